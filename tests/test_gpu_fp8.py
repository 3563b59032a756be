"""GPU parity of the fp8 cache (E4M3 codes + one exponent byte per row; the format is this library's own, the
paper only names quantisation as an orthogonal direction in Sec. 5: parity unpinned by the paper).

Stored codes and exponent bytes are compared bit for bit with the oracle's quantiser after every layer; the
attention is compared with the oracle's attention over the read-back values of the cached scales (the step's
own K/V stay unquantised, as in the library), within the tolerances of the bf16 path."""
import math

import numpy as np
import pytest
import torch

import heatkv_workloads as W
from oracle import heatkv_oracle as O

pytestmark = pytest.mark.gpu

ATOL_MAX, ATOL_MEAN = 1e-2, 1e-3


@pytest.fixture(scope="module")
def hk():
    import paper_2605_14877_b200 as hk
    return hk


def _f64(x):
    return O.bf16_bits_to_f64(W.bf16_bits(x))


def _run_fp8(hk, sh, ref, make_schedule, kernel, seed=0, bias=None, fused=False, mutate=None):
    """Whole generation with the fp8 cache, every (sequence, layer, head) checked."""
    from paper_2605_14877_b200.sweep import Session
    n_seq = sh.n_seq
    sm = 1.0 / math.sqrt(sh.d)
    pool_rows = n_seq * (sh.L * sh.H * (sh.c[-2] + 64 * sh.K) + 64)
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows, layout=hk.LAYOUT_PAGED, kernel=kernel,
                 cache_dtype=hk.CACHE_FP8_E4M3) as ses:
        sch = make_schedule(ses)
        ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(n_seq)]
        layers = [W.qkv_layer(sh, seed, l, device="cuda", n_seq=n_seq) for l in range(sh.L)]
        if mutate is not None:
            layers = [mutate(l, *layers[l]) for l in range(sh.L)]
        outs = [torch.zeros_like(layers[l][0]) for l in range(sh.L)]
        host = [[_f64(x) for x in layers[l]] for l in range(sh.L)]
        # what the cache gives back: quantise + read back every row once, with the oracle
        hat, codes, exps = [], [], []
        for l in range(sh.L):
            per = []
            for x in host[l][1:]:
                c, e = O.quantize_rows_e4m3(x.reshape(-1, sh.d))
                per.append((c.reshape(x.shape), e.reshape(x.shape[:-1]), O.dequantize_rows_e4m3(c, e).reshape(x.shape)))
            codes.append((per[0][0], per[1][0]))
            exps.append((per[0][1], per[1][1]))
            hat.append((per[0][2], per[1][2]))
        bias_dev = None if bias is None else torch.from_numpy(bias).cuda()

        def after(step, layer):
            if step + 1 >= sh.K:
                return
            for s_ in range(n_seq):
                for h in range(sh.H):
                    idx = O.token_indices(ref, O.stored_scales_after_layer(ref, step + 1, layer, h))
                    got_idx = hk.heatkv_retained_indices(ses.ctx, ids[s_], layer, h, sh.c[-1])
                    assert np.array_equal(got_idx, idx), (step, layer, h)
                    n = max(len(idx), 1)
                    kc = torch.zeros(n, sh.d, dtype=torch.uint8, device="cuda")
                    vc = torch.zeros_like(kc)
                    ke = torch.zeros(n, dtype=torch.int8, device="cuda")
                    ve = torch.zeros_like(ke)
                    hk.heatkv_export_head_fp8(ses.ctx, ids[s_], layer, h, kc, vc, ke, ve)
                    m = len(idx)
                    assert np.array_equal(kc.cpu().numpy()[:m], codes[layer][0][s_, h][idx]), (step, layer, h)
                    assert np.array_equal(vc.cpu().numpy()[:m], codes[layer][1][s_, h][idx]), (step, layer, h)
                    assert np.array_equal(ke.cpu().numpy()[:m], exps[layer][0][s_, h][idx]), (step, layer, h)
                    assert np.array_equal(ve.cpu().numpy()[:m], exps[layer][1][s_, h][idx]), (step, layer, h)

        ses.generate(ids, lambda l: layers[l], lambda l: outs[l],
                     (lambda l, k: bias_dev[l, k]) if bias is not None else None, after, fused)
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        err_sum, err_n, err_max = 0.0, 0, 0.0
        for s_ in range(n_seq):
            for l in range(sh.L):
                q, k, v = host[l]
                for h in range(sh.H):
                    for step in range(1, sh.K + 1):
                        lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
                        # cached scales come back quantised, the step's own rows are the fresh ones
                        k_use, v_use = hat[l][0][s_, h].copy(), hat[l][1][s_, h].copy()
                        k_use[lo:hi], v_use[lo:hi] = k[s_, h, lo:hi], v[s_, h, lo:hi]
                        brow = None if bias is None else bias[l, step - 1, h].astype(np.float64)
                        want = O.scale_attention(q[s_, h, lo:hi], k_use, v_use, ref, step, l, h, sm, brow)
                        got = outs[l][s_, h, lo:hi].to(torch.float64).cpu().numpy()
                        err = np.abs(got - want)
                        assert err.max() <= ATOL_MAX, (s_, l, h, step, err.max())
                        assert err.mean() <= ATOL_MEAN + 2.0 ** -9 * np.abs(want).mean(), (s_, l, h, step, err.mean())
                        err_sum, err_n, err_max = err_sum + float(err.sum()), err_n + err.size, max(err_max, float(err.max()))
        assert err_max <= ATOL_MAX and err_sum / err_n <= ATOL_MEAN
        kept = O.kept_tokens_after_step(ref, sh.K - 1)
        actual, closed = hk.heatkv_cache_bytes(ses.ctx, ids[0])
        assert actual == closed == O.cache_bytes_fp8(kept, sh.d)
        assert actual * 2 < O.cache_bytes(kept, sh.d) * 1.02 + 1          # about half of the bf16 cache
        st = hk.heatkv_allocator_stats(ses.ctx)
        assert st.open_seqs == n_seq and st.used_tokens == n_seq * int(kept.sum())
        # the bf16 export has no meaning here and says so
        with pytest.raises(hk.HeatKVError):
            hk.heatkv_export_head(ses.ctx, ids[0], 0, 0, torch.zeros(8, sh.d, dtype=torch.bfloat16, device="cuda"),
                                  torch.zeros(8, sh.d, dtype=torch.bfloat16, device="cuda"))
        ks = hk.heatkv_kernel_launches(ses.ctx)
        if kernel == hk.KERNEL_TCGEN05:
            assert ks.attention_generic == 0 and ks.attention_tcgen05 == sh.K * sh.L
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)
        hk.heatkv_schedule_free(sch)


@pytest.mark.parametrize("kernel", [1, 2], ids=["generic", "tcgen05"])
@pytest.mark.parametrize("fused", [False, True], ids=["separate", "one_call"])
def test_fp8_cache_mid_config(hk, kernel, fused):
    """d=128, 2 layers, 11 scales, budget 0.15, per-head bias: codes, exponents, attention, bytes."""
    sh = W.Shape("mid", L=2, H=4, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 4)
    ref = O.heatkv_schedule(scores, 0.15, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 3)
    _run_fp8(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.15), kernel, bias=bias, fused=fused)


def test_fp8_cache_full_budget_head_dim_64_wide_range(hk):
    """b = 1 (every scale cached and read back), 64-wide heads, rows scaled over 2^-12 .. 2^12 so that the
    exponent bytes differ from row to row; automatic kernel choice (both kernels take part)."""
    sh = W.Shape("full64", L=1, H=3, d=64, sides=W.SIDES_13[:10], n_seq=2, s=2)
    scores = W.synthetic_scas(sh, 1)
    ref = O.heatkv_schedule(scores, 1.0, sh.s, sh.sides)

    def mutate(l, q, k, v):
        tok = torch.arange(k.shape[2], device=k.device)
        scale = torch.exp2(((tok * 7) % 25 - 12).to(torch.float32)).to(torch.bfloat16)[None, None, :, None]
        # V rows over a wide range; K rows over a narrow one, so that the logits stay moderate
        kscale = torch.exp2(((tok * 5) % 3 - 1).to(torch.float32)).to(torch.bfloat16)[None, None, :, None]
        return q, k * kscale, v * scale * 2.0 ** -14      # |v| up to about 1: outputs stay where bf16 resolves 1e-2

    _run_fp8(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=1.0), hk.KERNEL_AUTO, mutate=mutate)


def test_fp8_cache_needs_paged_layout_and_enough_staging(hk):
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("mid", L=1, H=2, d=128, sides=W.SIDES_13[:9], n_seq=1, s=3)
    with pytest.raises(hk.HeatKVError):
        Session(sh.L, sh.H, sh.d, sh.t, sh.s, 4096, layout=hk.LAYOUT_RAGGED, kernel=hk.KERNEL_GENERIC,
                cache_dtype=hk.CACHE_FP8_E4M3)
    # staging of 64 rows: the first step that sees two half-tiles of cached keys cannot be expanded
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, 1 << 15, layout=hk.LAYOUT_PAGED, kernel=hk.KERNEL_GENERIC,
                 cache_dtype=hk.CACHE_FP8_E4M3, stage_bytes=64 * sh.d * 2 * 2) as ses:
        scores = W.synthetic_scas(sh, 1)
        sch = ses.schedule(scas=scores, b=1.0)
        ids = [hk.heatkv_seq_open(ses.ctx, sch)]
        q, k, v = W.qkv_layer(sh, 0, 0, device="cuda", n_seq=1)
        out = torch.zeros_like(q)
        with pytest.raises(hk.HeatKVError) as ei:
            ses.generate(ids, lambda l: (q, k, v), lambda l: out)
        assert ei.value.status == -4                      # HEATKV_ERR_OUT_OF_PAGES
        hk.heatkv_schedule_free(sch)


def test_fp8_cache_config2_full_size(hk):
    """Config 2 (16 heads, d=128, 13 scales, batch 2, 20x) with the fp8 cache at full size, automatic kernel
    choice, one call per (layer, step): every (sequence, head) unit against the oracle."""
    sh = W.CFG2
    scores = W.synthetic_scas(sh, 0)
    ref = O.heatkv_schedule(scores, 0.05, sh.s, sh.sides)
    bias = W.seg_bias_current_scale(sh, 0)
    _run_fp8(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.05), hk.KERNEL_AUTO, bias=bias, fused=True)
