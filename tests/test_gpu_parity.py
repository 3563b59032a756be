"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded
inputs.  Retained indices and cache contents bit-exact; attention within max-abs 1e-2 and
mean-abs 1e-3; calibration scores within 1e-3 relative."""
import math

import numpy as np
import pytest
import torch

import heatkv_workloads as W
from oracle import heatkv_oracle as O

pytestmark = pytest.mark.gpu

ATOL_MAX, ATOL_MEAN, RTOL_BETA = 1e-2, 1e-3, 1e-3


@pytest.fixture(scope="module")
def hk():
    import paper_2605_14877_b200 as hk
    return hk


def _session(hk, sh, pool_rows, layout, kernel=None, **kw):
    from paper_2605_14877_b200.sweep import Session
    return Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows, layout=layout,
                   kernel=hk.KERNEL_GENERIC if kernel is None else kernel, **kw)


def _f64(x):
    return O.bf16_bits_to_f64(W.bf16_bits(x))


class _ErrStats:
    """Accumulates |got - ref| over a whole workload: the stated bar (max-abs 1e-2, mean-abs
    1e-3) is applied to all outputs of the workload together."""

    def __init__(self):
        self.sum, self.n, self.max = 0.0, 0, 0.0

    def add(self, err):
        self.sum += float(err.sum())
        self.n += err.size
        self.max = max(self.max, float(err.max()))

    def check(self):
        assert self.n > 0 and self.max <= ATOL_MAX and self.sum / self.n <= ATOL_MEAN, (self.max, self.sum / self.n)


def _check_attention(got_bf16, ref_f64, what, stats=None):
    """Per block (one head at one step): max-abs within 1e-2, and mean-abs within 1e-3 plus the
    floor of the bf16 output format itself, 2^-9 * mean|ref| (a value in [2^e, 2^(e+1)) is
    stored with spacing 2^(e-7), i.e. a mean rounding error of about |x| * 2^-9.5)."""
    got = got_bf16.to(torch.float64).cpu().numpy()
    err = np.abs(got - ref_f64)
    assert err.max() <= ATOL_MAX, (what, err.max())
    assert err.mean() <= ATOL_MEAN + 2.0 ** -9 * np.abs(ref_f64).mean(), (what, err.mean())
    if stats is not None:
        stats.add(err)


def _run_full_parity(hk, sh, ref, make_schedule, layout, seed=0, bias=None, kernel=None, n_seq=None,
                     check_heads=None, check_cache=True, fused=False, mutate=None, want_kernels=None):
    """Whole generation of one batch; compares every (seq, layer, head, step) unless check_heads
    restricts the oracle work to a list of (seq, layer, head)."""
    n_seq = sh.n_seq if n_seq is None else n_seq
    sm = 1.0 / math.sqrt(sh.d)
    with _session(hk, sh, pool_rows=n_seq * (sh.L * sh.H * (sh.c[-2] + 64 * sh.K) + 64), layout=layout,
                  kernel=kernel) as ses:
        sch = make_schedule(ses)
        ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(n_seq)]
        layers = [W.qkv_layer(sh, seed, l, device="cuda", n_seq=n_seq) for l in range(sh.L)]
        if mutate is not None:
            layers = [mutate(l, *layers[l]) for l in range(sh.L)]
        outs = [torch.zeros_like(layers[l][0]) for l in range(sh.L)]
        host = [[_f64(x) for x in layers[l]] for l in range(sh.L)]
        bits = [[W.bf16_bits(x) for x in layers[l][1:]] for l in range(sh.L)]
        bias_dev = None if bias is None else torch.from_numpy(bias).cuda()
        heads = check_heads or [(s_, l, h) for s_ in range(n_seq) for l in range(sh.L) for h in range(sh.H)]

        def after(step, layer):
            if not check_cache or step + 1 >= sh.K:
                return
            for (s_, l, h) in heads:
                if l != layer:
                    continue
                idx, kk, vv = O.cache_after_layer(bits[l][0][s_, h], bits[l][1][s_, h], ref, step + 1, l, h)
                got_idx = hk.heatkv_retained_indices(ses.ctx, ids[s_], l, h, sh.c[-1])
                assert np.array_equal(got_idx, idx), (step, l, h)
                ko = torch.zeros(max(len(idx), 1), sh.d, dtype=torch.bfloat16, device="cuda")
                vo = torch.zeros_like(ko)
                hk.heatkv_export_head(ses.ctx, ids[s_], l, h, ko, vo)
                assert np.array_equal(W.bf16_bits(ko)[: len(idx)], kk), (step, l, h)
                assert np.array_equal(W.bf16_bits(vo)[: len(idx)], vv), (step, l, h)

        ses.generate(ids, lambda l: layers[l], lambda l: outs[l],
                     (lambda l, k: bias_dev[l, k]) if bias is not None else None, after, fused)
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        stats = _ErrStats()
        for (s_, l, h) in heads:
            q, k, v = host[l]
            for step in range(1, sh.K + 1):
                lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
                brow = None if bias is None else bias[l, step - 1, h].astype(np.float64)
                want = O.scale_attention(q[s_, h, lo:hi], k[s_, h], v[s_, h], ref, step, l, h, sm, brow)
                _check_attention(outs[l][s_, h, lo:hi], want, (s_, l, h, step), stats)
        stats.check()
        # closed form of the cache size at the end (last stored scale is K-1)
        kept = O.kept_tokens_after_step(ref, sh.K - 1)
        actual, closed = hk.heatkv_cache_bytes(ses.ctx, ids[0])
        reserved = hk.heatkv_seq_reservation(ses.ctx, ids[0])[1] * sh.d * 4
        assert actual == closed == O.cache_bytes(kept, sh.d) and reserved >= actual
        st = hk.heatkv_allocator_stats(ses.ctx)
        assert st.open_seqs == n_seq and st.used_tokens == n_seq * int(kept.sum())
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)
        assert hk.heatkv_allocator_stats(ses.ctx).reserved_rows == 0
        launches = hk.heatkv_launch_count(ses.ctx)
        ks = hk.heatkv_kernel_launches(ses.ctx)
        if kernel == hk.KERNEL_TCGEN05:                     # forced: the tensor-memory kernel took every attention launch
            assert ks.tcgen05_attention_ready == 1 and ks.attention_generic == 0 and ks.attention_tcgen05 >= sh.K * sh.L
        if kernel == hk.KERNEL_AUTO:                        # steps of 256 tokens and more go to the tensor-memory kernel,
            assert ks.tcgen05_attention_ready == 1          # steps of 128 and more once the call holds 64 (sequence, head) units
            big = [t >= 256 or (t >= 128 and n_seq * sh.H >= 64) for t in sh.t]
            assert ks.attention_tcgen05 == sh.L * sum(big)
            assert ks.attention_generic == sh.L * (len(big) - sum(big))
        if want_kernels is not None:
            assert (ks.attention_tcgen05, ks.attention_generic) == want_kernels
        hk.heatkv_schedule_free(sch)
    return launches


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
def test_tiny_config_end_to_end(hk, layout):
    """Config 1: 1 layer, 4 heads, d=64, sides {1,2,4,8}, per-head budgets {100,50,25,0} %."""
    sh = W.TINY
    frac = np.array([W.TINY_FRACTIONS])
    ref = O.explicit_schedule(frac, sh.s, sh.sides)
    n = _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(policy=hk.POLICY_EXPLICIT, fraction=frac), layout)
    assert n >= sh.K


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
@pytest.mark.parametrize("policy", [0, 1, 2], ids=["heatkv", "binary", "naive"])
def test_mid_config_multi_layer_with_bias(hk, layout, policy):
    """d=128, 3 layers, 11 scales (several key tiles, ragged tails 36/144/400), per-head logit bias."""
    sh = W.Shape("mid", L=3, H=4, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 4)
    cas = scores[:, :, 6].copy()
    ref = O.heatkv_schedule(cas if policy == 1 else scores, 0.15, sh.s, sh.sides, policy)
    bias = W.seg_bias_prior_lognormal(sh, 3)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, cas=cas, policy=policy, b=0.15), layout,
                     bias=bias)


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
def test_tensor_memory_kernel_mid_config(hk, layout):
    """Same mid workload with every step forced onto the tcgen05 kernel: single-row tiles,
    ragged tails, half-filled key tiles and the pool/own-scale boundary inside one tile."""
    sh = W.Shape("mid", L=2, H=4, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 4)
    ref = O.heatkv_schedule(scores, 0.15, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 3)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.15), layout, bias=bias,
                     kernel=hk.KERNEL_TCGEN05)


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
def test_tensor_memory_kernel_head_dim_64(hk, layout):
    """The tcgen05 kernel's head_dim-64 instantiation (one 64-column half per row, N = 64 PV products) on every
    step of a mid workload with bias, cache update in the same call; and a split launch (few heads, long ranges)."""
    sh = W.Shape("mid64", L=2, H=4, d=64, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 5)
    ref = O.heatkv_schedule(scores, 0.15, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 4)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.15), layout, bias=bias,
                     kernel=hk.KERNEL_TCGEN05, fused=True)
    if layout == 1:
        sh2 = W.Shape("split64", L=1, H=3, d=64, sides=W.SIDES_13[:12], n_seq=2, s=3)
        scores2 = W.synthetic_scas(sh2, 3)
        ref2 = O.heatkv_schedule(scores2, 0.6, sh2.s, sh2.sides)
        _run_full_parity(hk, sh2, ref2, lambda ses: ses.schedule(scas=scores2, b=0.6), hk.LAYOUT_PAGED,
                         kernel=hk.KERNEL_AUTO, check_cache=False)


@pytest.mark.parametrize("where", ["first_half", "second_half", "everywhere"])
def test_tensor_memory_kernel_outlier_keys(hk, where):
    """Sparse keys scaled by 16 (logits of +-40 and more) that first show up in later key tiles, in the first 64
    keys of a tile, in the last 64, or in both: the running reference of the online softmax has to move by tens
    of units in the middle of a head (rescaling O and the row sum), and the result must still match the oracle."""
    sh = W.Shape("outlier", L=1, H=2, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 2)
    ref = O.heatkv_schedule(scores, 0.5, sh.s, sh.sides)

    def mutate(l, q, k, v):
        k = k.clone()
        tok = torch.arange(k.shape[2], device=k.device)
        in_tile = tok % 128                                # position inside a 128-key stretch (tiles are not aligned to it: both halves get hit)
        pick = (tok >= 300) & (tok % 41 == 0)
        if where == "first_half":
            pick &= in_tile < 64
        elif where == "second_half":
            pick &= in_tile >= 64
        k[:, :, pick] = k[:, :, pick] * 16
        # attention is then close to one-hot, so outputs are single V rows: keep them below 1, where the bf16
        # output format itself resolves 1e-2
        return q, k, v * 0.25

    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.5), hk.LAYOUT_PAGED,
                     kernel=hk.KERNEL_TCGEN05, check_cache=False, fused=True, mutate=mutate)


def test_tensor_memory_kernel_full_cache(hk):
    """b = 1: long page tables (up to 4121 prior keys), tcgen05 kernel, no bias."""
    sh = W.Shape("full128", L=1, H=2, d=128, sides=W.SIDES_13[:12], n_seq=1, s=3)
    scores = W.synthetic_scas(sh, 1)
    ref = O.heatkv_schedule(scores, 1.0, sh.s, sh.sides)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=1.0), hk.LAYOUT_PAGED,
                     kernel=hk.KERNEL_TCGEN05, check_cache=False)


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
@pytest.mark.parametrize("kernel", [1, 2], ids=["generic", "tcgen05"])
def test_attention_with_cache_update_in_one_call(hk, layout, kernel):
    """heatkv_attention_append: in the paged layout the append rides on the attention launch (extra CTAs or spare warps)
    (both kernels); outputs, retained indices and cache contents after every layer as with separate calls."""
    sh = W.Shape("mid", L=2, H=4, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 4)
    ref = O.heatkv_schedule(scores, 0.15, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 3)
    n = _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.15), layout, bias=bias, kernel=kernel,
                         fused=True)
    if layout == 1:
        assert n == sh.K * sh.L                      # one launch per (step, layer): every update here is small


def test_config2_one_call_per_step_all_units(hk):
    sh = W.CFG2
    scores = W.synthetic_scas(sh, 0)
    ref = O.heatkv_schedule(scores, 0.05, sh.s, sh.sides)
    bias = W.seg_bias_current_scale(sh, 0)
    n = _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.05), hk.LAYOUT_PAGED, bias=bias,
                         kernel=hk.KERNEL_AUTO, fused=True, want_kernels=(7, 6))
    assert n == sh.K


def test_28_head_layer_width(hk):
    """A layer width that is not a power of two (28 heads of 128, the width the larger model's cache
    figures imply): heads beyond the 32-lane prefix chunk, odd head counts in the item tables."""
    sh = W.Shape("w28", L=1, H=28, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 6)
    ref = O.heatkv_schedule(scores, 0.1, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 6)
    heads = [(0, 0, 0), (1, 0, 13), (0, 0, 27)]
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.1), hk.LAYOUT_PAGED, bias=bias,
                     kernel=hk.KERNEL_AUTO, check_heads=heads, fused=True)


def test_40_head_layer_width(hk):
    """More heads than one 32-lane chunk of the work-item prefix sum in the tensor-memory kernel: items of
    heads 32..39 are found in the second chunk (sampled heads from both chunks, fused cache update)."""
    sh = W.Shape("w40", L=1, H=40, d=128, sides=W.SIDES_13[:10], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 8)
    ref = O.heatkv_schedule(scores, 0.2, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 8)
    heads = [(0, 0, 0), (1, 0, 31), (0, 0, 32), (1, 0, 39), (0, 0, 17)]
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.2), hk.LAYOUT_PAGED, bias=bias,
                     kernel=hk.KERNEL_AUTO, check_heads=heads, fused=True)


def test_key_range_splitting_is_used_and_exact(hk):
    """Few heads with long key ranges: the launch cuts them into pieces that meet in the scratch region
    (checked through heatkv_attention_split), and the merged outputs still match the oracle; a context
    without scratch runs the same workload unsplit."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("split", L=1, H=3, d=128, sides=W.SIDES_13[:12], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 3)
    ref = O.heatkv_schedule(scores, 0.6, sh.s, sh.sides)
    bias = W.seg_bias_prior_lognormal(sh, 5)
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K)) as ses:
        sch = ses.schedule(scas=scores, b=0.6)
        ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
        splits = [hk.heatkv_attention_split(ses.ctx, ids, 0, step) for step in range(sh.K)]
        assert any(st > 0 for st, _ in splits[6:]), splits
        assert all(items >= 1 for _, items in splits)
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)
        hk.heatkv_schedule_free(sch)
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=4096, scratch_bytes=1024) as ses:
        sch = ses.schedule(scas=scores, b=0.05)
        sid = hk.heatkv_seq_open(ses.ctx, sch)
        assert all(hk.heatkv_attention_split(ses.ctx, [sid], 0, step)[0] == 0 for step in range(sh.K))
        hk.heatkv_seq_close(ses.ctx, sid)
        hk.heatkv_schedule_free(sch)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.6), hk.LAYOUT_PAGED, bias=bias,
                     kernel=hk.KERNEL_AUTO)


def test_split_heads_are_reproducible_bit_for_bit(hk):
    """Pieces of a cut head are merged in piece order whichever arrives last: the same generation run four
    times gives identical output bits (steps of this workload are cut, see the test above)."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("split", L=1, H=3, d=128, sides=W.SIDES_13[:12], n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 3)
    q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
    runs = []
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K)) as ses:
        sch = ses.schedule(scas=scores, b=0.6)
        for _ in range(4):
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            out = torch.zeros_like(q)
            ses.generate(ids, lambda l: (q, k, v), lambda l: out, fused=True)
            torch.cuda.synchronize()
            runs.append(W.bf16_bits(out).copy())
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
        assert hk.heatkv_device_status(ses.ctx) == 0
        hk.heatkv_schedule_free(sch)
    for r in runs[1:]:
        assert np.array_equal(r, runs[0])


def test_full_budget_equals_uncompressed(hk):
    sh = W.Shape("full", L=1, H=2, d=64, sides=W.SIDES_13[:9], n_seq=1, s=2)
    scores = W.synthetic_scas(sh, 1)
    ref = O.heatkv_schedule(scores, 1.0, sh.s, sh.sides)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=1.0), hk.LAYOUT_PAGED)


def _calibrate(hk, sh, seeds, bias=None, with_out=False, kernel=None, mutate=None):
    from paper_2605_14877_b200.sweep import Session
    sm = 1.0 / math.sqrt(sh.d)
    ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64, kernel=hk.KERNEL_GENERIC if kernel is None else kernel)
    beta_dev = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
    bias_dev = None if bias is None else torch.from_numpy(bias).cuda()
    ref = np.zeros((sh.L, sh.H, sh.K, sh.K))
    n_samples = 0
    for seed in seeds:
        for l in range(sh.L):
            q, k, v = W.qkv_layer(sh, seed, l, device="cuda")
            if mutate is not None:
                q, k, v = mutate(q, k, v)
            out = torch.zeros_like(q) if with_out else None
            for step in range(sh.K):
                lo, hi = ses.step_slices(step)
                qs, ks, vs = q[:, :, lo:hi], k[:, :, :hi], v[:, :, :hi]
                os_ = out[:, :, lo:hi] if with_out else None
                st = hk.Strides.of(qs, ks, os_)
                hk.heatkv_calibrate_scores(ses.ctx, l, step, sh.n_seq, qs, ks, vs if with_out else None, st,
                                           None if bias is None else bias_dev[l, step], beta_dev, os_)
            qh, kh, vh = _f64(q), _f64(k), _f64(v)
            for s_ in range(sh.n_seq):
                for h in range(sh.H):
                    b_lh = None if bias is None else bias[l, :, h, :].astype(np.float64)
                    ref[l, h] += O.beta_sample(qh[s_, h], kh[s_, h], sh.sides, sm, b_lh)
            if with_out:
                full = O.explicit_schedule(np.ones((sh.L, sh.H)), sh.s, sh.sides)
                for h in range(sh.H):
                    for step in range(1, sh.K + 1):
                        lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
                        brow = None if bias is None else bias[l, step - 1, h].astype(np.float64)
                        want = O.scale_attention(qh[0, h, lo:hi], kh[0, h], vh[0, h], full, step, l, h, sm, brow)
                        _check_attention(out[0, h, lo:hi], want, ("calib-out", l, h, step))
        n_samples += sh.n_seq
    beta, scas, cas = hk.heatkv_finalize_scores(ses.ctx, beta_dev, n_samples, sh.L, sh.H, sh.K)
    ses.close()
    ref /= n_samples
    return beta, scas, cas, ref


def test_calibration_tiny_four_samples(hk):
    sh = W.TINY
    beta, scas, cas, ref = _calibrate(hk, sh, seeds=range(4))
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)
    assert np.all(np.triu(beta, 1) == 0)
    mask = ref > 1e-6
    assert np.all(np.abs(beta - ref)[mask] <= RTOL_BETA * ref[mask])
    for l in range(sh.L):
        for h in range(sh.H):
            assert np.allclose(scas[l, h], O.scas(ref[l, h], sh.s), rtol=RTOL_BETA, atol=1e-9)
            assert np.isclose(cas[l, h], O.cas(ref[l, h], sh.s), rtol=RTOL_BETA, atol=1e-9)


def test_calibration_mid_with_bias_and_output(hk):
    sh = W.Shape("mid", L=2, H=3, d=128, sides=W.SIDES_13[:10], n_seq=2, s=3)
    bias = W.seg_bias_prior_lognormal(sh, 8)
    beta, scas, cas, ref = _calibrate(hk, sh, seeds=[5], bias=bias, with_out=True)
    mask = ref > 1e-5
    assert np.all(np.abs(beta - ref)[mask] <= RTOL_BETA * ref[mask])
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)
    for l in range(sh.L):
        for h in range(sh.H):
            assert np.allclose(scas[l, h], O.scas(ref[l, h], sh.s), rtol=RTOL_BETA, atol=1e-9)


@pytest.mark.parametrize("d", [128, 64], ids=["d128", "d64"])
@pytest.mark.parametrize("with_bias", [False, True], ids=["plain", "bias"])
def test_calibration_tensor_memory_kernel(hk, with_bias, d):
    """Every step forced through the tcgen05 calibration kernel: one-row tiles, ragged source-scale
    borders inside key tiles (36, 144, 400 tokens), an odd number of half-tiles, two query tiles; heads of
    128 and of 64 dimensions."""
    sh = W.Shape("mid", L=2, H=3, d=d, sides=W.SIDES_13[:11], n_seq=2, s=3)
    bias = W.seg_bias_prior_lognormal(sh, 8) if with_bias else None
    beta, scas, cas, ref = _calibrate(hk, sh, seeds=[5], bias=bias, kernel=hk.KERNEL_TCGEN05)
    mask = ref > 1e-5
    assert np.all(np.abs(beta - ref)[mask] <= RTOL_BETA * ref[mask]), float((np.abs(beta - ref)[mask] / ref[mask]).max())
    assert np.all(np.triu(beta, 1) == 0)
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)
    for l in range(sh.L):
        for h in range(sh.H):
            assert np.allclose(scas[l, h], O.scas(ref[l, h], sh.s), rtol=RTOL_BETA, atol=1e-9)


def test_calibration_tensor_memory_kernel_outlier_keys(hk):
    """Sparse keys scaled by 16 beyond the first key tiles (logits of +-40 and more): the running reference of the
    calibration kernel's online softmax has to move by tens of units in the middle of a row, rescaling the masses
    parked for the finished source scales; beta must still match the oracle (Eq. 2)."""
    sh = W.Shape("calib_outlier", L=1, H=3, d=128, sides=W.SIDES_13[:11], n_seq=2, s=3)

    def mutate(q, k, v):
        k = k.clone()
        tok = torch.arange(k.shape[2], device=k.device)
        pick = (tok >= 300) & (tok % 41 == 0)
        k[:, :, pick] = k[:, :, pick] * 16
        return q, k, v

    beta, scas, cas, ref = _calibrate(hk, sh, seeds=[9], kernel=hk.KERNEL_TCGEN05, mutate=mutate)
    mask = ref > 1e-5
    assert np.all(np.abs(beta - ref)[mask] <= RTOL_BETA * ref[mask]), float((np.abs(beta - ref)[mask] / ref[mask]).max())
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)


def test_config2_calibration_full_size(hk):
    """Sec. 3.1, Eq. 2 and Eq. 4 at the size the bench calibrates at: 13 scales, 2 sequences x 16 heads, bias on
    the current scale, automatic kernel choice (tensor-memory kernel for the seven steps of 256 tokens and more:
    several waves of CTAs, 13 parked scales per row).  beta of four heads (both sequences summed, as the
    accumulator holds them) against the oracle at 1e-3 relative, S-CAS of the same heads, and what must hold for
    every head: rows of beta sum to 1, nothing above the diagonal."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG2
    sm = 1.0 / math.sqrt(sh.d)
    bias = W.seg_bias_current_scale(sh, 0)
    bias_dev = torch.from_numpy(bias).cuda()
    q, k, v = W.qkv_layer(sh, 100, 0, device="cuda")
    beta_dev = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64, kernel=hk.KERNEL_AUTO) as ses:
        for step in range(sh.K):
            lo, hi = ses.step_slices(step)
            qs, ks_ = q[:, :, lo:hi], k[:, :, :hi]
            hk.heatkv_calibrate_scores(ses.ctx, 0, step, sh.n_seq, qs, ks_, None, hk.Strides.of(qs, ks_),
                                       bias_dev[0, step], beta_dev, None)
        beta, scas, cas = hk.heatkv_finalize_scores(ses.ctx, beta_dev, sh.n_seq, sh.L, sh.H, sh.K)
        assert hk.heatkv_device_status(ses.ctx) == 0
        st = hk.heatkv_kernel_launches(ses.ctx)
        assert st.tcgen05_calibration_ready == 1
        assert (st.calibration_tcgen05, st.calibration_generic) == (sum(1 for t in sh.t if t >= 256), sum(1 for t in sh.t if t < 256))
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)
    assert np.all(np.triu(beta, 1) == 0)
    qh, kh = _f64(q), _f64(k)
    for h in (0, 5, 11, 15):
        ref = np.zeros((sh.K, sh.K))
        for s_ in range(sh.n_seq):
            ref += O.beta_sample(qh[s_, h], kh[s_, h], sh.sides, sm, bias[0, :, h, :].astype(np.float64))
        ref /= sh.n_seq
        mask = ref > 1e-5
        rel = np.abs(beta[0, h] - ref)[mask] / ref[mask]
        assert rel.max() <= RTOL_BETA, (h, float(rel.max()))
        assert np.allclose(scas[0, h], O.scas(ref, sh.s), rtol=RTOL_BETA, atol=1e-9)
        assert np.isclose(cas[0, h], O.cas(ref, sh.s), rtol=RTOL_BETA, atol=1e-9)


@pytest.mark.parametrize("with_bias", [False, True], ids=["plain", "bias"])
def test_calibration_all_steps_in_one_call(hk, with_bias):
    """heatkv_calibrate_scores_steps (Sec. 3.1, Eq. 2 for every step of a layer at once: one tensor-memory launch
    over the large steps, longest CTAs first) at the config-2 shape: equal to step-by-step calls up to the order of
    the fp32 sums, beta of two heads against the oracle, and a sub-range of steps on strided views."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG2
    sm = 1.0 / math.sqrt(sh.d)
    bias = W.seg_bias_current_scale(sh, 0)
    bias_dev = torch.from_numpy(bias).cuda()                       # [L, K, H, K]
    q, k, _ = W.qkv_layer(sh, 321, 0, device="cuda")
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64, kernel=hk.KERNEL_AUTO) as ses:
        one = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
        for step in range(sh.K):
            lo, hi = ses.step_slices(step)
            qs, ks_ = q[:, :, lo:hi], k[:, :, :hi]
            hk.heatkv_calibrate_scores(ses.ctx, 0, step, sh.n_seq, qs, ks_, None, hk.Strides.of(qs, ks_),
                                       bias_dev[0, step] if with_bias else None, one, None)
        n0 = hk.heatkv_kernel_launches(ses.ctx)
        allk = torch.zeros_like(one)
        hk.heatkv_calibrate_scores_steps(ses.ctx, 0, 0, sh.K, sh.n_seq, q, k, hk.Strides.of(q, k),
                                         bias_dev[0] if with_bias else None, allk)
        n1 = hk.heatkv_kernel_launches(ses.ctx)
        big = sum(1 for t in sh.t if t >= 256)
        assert n1.calibration_tcgen05 - n0.calibration_tcgen05 == 1                       # one launch for the large steps
        assert n1.calibration_generic - n0.calibration_generic == 1                       # ... and one for the small ones
        # steps 8 .. 11 only, on views of a wider buffer (strides differ from the dense ones)
        wide_q = torch.zeros(sh.n_seq, sh.H, sh.c[-1] + 8, sh.d, dtype=torch.bfloat16, device="cuda")
        wide_k = torch.zeros_like(wide_q)
        wide_q[:, :, : sh.c[-1]], wide_k[:, :, : sh.c[-1]] = q, k
        part = torch.zeros_like(one)
        vq, vk = wide_q[:, :, : sh.c[10]], wide_k[:, :, : sh.c[10]]
        hk.heatkv_calibrate_scores_steps(ses.ctx, 0, 7, 11, sh.n_seq, vq, vk, hk.Strides.of(vq, vk),
                                         bias_dev[0] if with_bias else None, part)
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        a, b, c = one.cpu().numpy()[0], allk.cpu().numpy()[0], part.cpu().numpy()[0]
    mask = a > 1e-5
    assert (np.abs(a - b)[mask] / a[mask]).max() <= 1e-4
    assert np.all(b[~mask] <= 2e-5)
    sel = np.zeros_like(mask)
    sel[:, 7:11, :] = mask[:, 7:11, :]
    assert (np.abs(a - c)[sel] / a[sel]).max() <= 1e-4
    rest = np.ones_like(mask)
    rest[:, 7:11, :] = False
    assert np.all(c[rest] == 0)
    qh, kh = _f64(q), _f64(k)
    for h in (3, 12):
        ref = np.zeros((sh.K, sh.K))
        for s_ in range(sh.n_seq):
            ref += O.beta_sample(qh[s_, h], kh[s_, h], sh.sides, sm, bias[0, :, h, :].astype(np.float64) if with_bias else None)
        m = ref > 1e-5 * sh.n_seq
        assert (np.abs(b[h] - ref)[m] / ref[m]).max() <= RTOL_BETA, h


def test_config3_calibration_sixteen_samples(hk):
    """Calibration as config 3 runs it, on one layer of its shape: 16 seeded samples (two calls of 8 sequences per
    step, accumulated in the same beta), per-head log-normal bias on the prior scales, automatic kernel choice.
    beta and S-CAS of three heads over all 16 samples against the oracle at 1e-3 relative; unit row sums and an empty
    upper triangle for every head."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("cfg3_layer", L=1, H=16, d=128, sides=W.SIDES_13, n_seq=8, s=3)
    sm = 1.0 / math.sqrt(sh.d)
    bias = W.seg_bias_prior_lognormal(sh, 0)
    bias_dev = torch.from_numpy(bias).cuda()
    beta_dev = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
    heads, batches = (1, 6, 12), 2
    ref = {h: np.zeros((sh.K, sh.K)) for h in heads}
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64, kernel=hk.KERNEL_AUTO) as ses:
        for bt in range(batches):
            q, k, _ = W.qkv_layer(sh, 200 + bt, 0, device="cuda")
            for step in range(sh.K):
                lo, hi = ses.step_slices(step)
                qs, ks_ = q[:, :, lo:hi], k[:, :, :hi]
                hk.heatkv_calibrate_scores(ses.ctx, 0, step, sh.n_seq, qs, ks_, None, hk.Strides.of(qs, ks_),
                                           bias_dev[0, step], beta_dev, None)
            for head in heads:
                qh, kh = _f64(q[:, head]), _f64(k[:, head])
                for s_ in range(sh.n_seq):
                    ref[head] += O.beta_sample(qh[s_], kh[s_], sh.sides, sm, bias[0, :, head, :].astype(np.float64))
        beta, scas, _ = hk.heatkv_finalize_scores(ses.ctx, beta_dev, batches * sh.n_seq, sh.L, sh.H, sh.K)
        assert hk.heatkv_device_status(ses.ctx) == 0
    assert np.allclose(beta.sum(axis=-1), 1.0, atol=2e-4)
    assert np.all(np.triu(beta, 1) == 0)
    for head in heads:
        want = ref[head] / (batches * sh.n_seq)
        mask = want > 1e-5
        rel = np.abs(beta[0, head] - want)[mask] / want[mask]
        assert rel.max() <= RTOL_BETA, (head, float(rel.max()))
        assert np.allclose(scas[0, head], O.scas(want, sh.s), rtol=RTOL_BETA, atol=1e-9)


def test_calibration_without_output_ignores_output_strides(hk):
    """A C caller that computes no attention output may leave the o_* strides zero (both calibration entry
    points); the result is the one the call with filled-in strides gives."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("strides", L=1, H=2, d=64, sides=W.SIDES_13[:7], n_seq=2, s=1)
    q, k, _ = W.qkv_layer(sh, 3, 0, device="cuda")
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64) as ses:
        outs = []
        for zero_o in (False, True):
            for entry in (hk.heatkv_calibrate_scores, hk.heatkv_calibrate_scores_static):
                beta_dev = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
                for step in range(sh.K):
                    lo, hi = ses.step_slices(step)
                    qs, ks_ = q[:, :, lo:hi], k[:, :, :hi]
                    st = hk.Strides.of(qs, ks_)
                    if zero_o:
                        st.o_seq = st.o_head = st.o_tok = 0
                    if entry is hk.heatkv_calibrate_scores:
                        entry(ses.ctx, 0, step, sh.n_seq, qs, ks_, None, st, None, beta_dev, None)
                    else:
                        entry(ses.ctx, 0, step, sh.n_seq, qs, ks_, st, None, beta_dev)
                outs.append(beta_dev.cpu().numpy())
        # (the accumulating entry point adds with atomics, so two runs agree only up to the order of the fp32 sums)
        assert np.allclose(outs[0], outs[2], rtol=0, atol=1e-5) and np.allclose(outs[1], outs[3], rtol=0, atol=1e-6)
        assert np.allclose(outs[0], outs[1], rtol=0, atol=1e-5)


def test_scas_stability_through_the_cuda_calibration(hk):
    """Appendix on S-CAS stability, end to end: three seeded calibration sets through the CUDA calibration
    (Eq. 2) -> S-CAS (Eq. 4) -> rank dispersion in the library, against the oracle's beta -> S-CAS -> dispersion
    on the same inputs.  A head's rank must agree wherever its S-CAS is further than 2e-3 relative from both
    neighbours in the oracle's order (closer scores may legitimately swap: the tie reading of the schedule
    builder); when every rank agrees the dispersions are the same numbers."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("stab", L=2, H=4, d=64, sides=W.SIDES_13[:9], n_seq=2, s=2)
    sm = 1.0 / math.sqrt(sh.d)
    bias = W.seg_bias_prior_lognormal(sh, 11)
    bias_dev = torch.from_numpy(bias).cuda()
    got_runs, ref_runs = [], []
    for seed in (21, 22, 23):
        with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64, kernel=hk.KERNEL_AUTO) as ses:
            beta_dev = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
            ref = np.zeros((sh.L, sh.H, sh.K))
            for l in range(sh.L):
                q, k, _ = W.qkv_layer(sh, seed, l, device="cuda")
                for step in range(sh.K):
                    lo, hi = ses.step_slices(step)
                    qs, ks_ = q[:, :, lo:hi], k[:, :, :hi]
                    hk.heatkv_calibrate_scores(ses.ctx, l, step, sh.n_seq, qs, ks_, None, hk.Strides.of(qs, ks_),
                                               bias_dev[l, step], beta_dev, None)
                qh, kh = _f64(q), _f64(k)
                for h in range(sh.H):
                    b = sum(O.beta_sample(qh[s_, h], kh[s_, h], sh.sides, sm, bias[l, :, h, :].astype(np.float64))
                            for s_ in range(sh.n_seq)) / sh.n_seq
                    ref[l, h] = O.scas(b, sh.s)
            _, scas, _ = hk.heatkv_finalize_scores(ses.ctx, beta_dev, sh.n_seq, sh.L, sh.H, sh.K)
        assert np.allclose(scas, ref, rtol=RTOL_BETA, atol=1e-9)
        got_runs.append(scas)
        ref_runs.append(ref)
    got_runs, ref_runs = np.stack(got_runs), np.stack(ref_runs)
    T = sh.L * sh.H
    all_equal = True
    for r in range(3):
        for kk in range(sh.s, sh.K - 1):
            ro = O.order_from_scores(ref_runs[r].reshape(T, sh.K)[:, kk])
            go = O.order_from_scores(got_runs[r].reshape(T, sh.K)[:, kk])
            vals = ref_runs[r].reshape(T, sh.K)[ro, kk]
            for pos in range(T):
                gaps = [abs(vals[pos] - vals[j]) / max(vals[pos], 1e-30) for j in (pos - 1, pos + 1) if 0 <= j < T]
                if min(gaps) > 2e-3:
                    assert go[pos] == ro[pos], (r, kk, pos)
                else:
                    all_equal &= go[pos] == ro[pos]
    got = hk.heatkv_rank_dispersion(got_runs, sh.s)
    want = O.scas_rank_dispersion(ref_runs, sh.s)
    assert np.all(got[: sh.s] == 0) and got[sh.K - 1] == 0
    if all_equal:
        assert np.allclose(got, want, rtol=0, atol=1e-12)
    else:
        assert np.allclose(got, want, rtol=0, atol=2.0 / T)


def test_config2_all_units(hk):
    """Config 2 (2B single layer, 16 heads, d=128, 13 scales, batch 2, 20x) at full size in the
    launch configuration the bench times; the oracle checks all 32 (sequence, head) units."""
    sh = W.CFG2
    scores = W.synthetic_scas(sh, 0)
    ref = O.heatkv_schedule(scores, 0.05, sh.s, sh.sides)
    bias = W.seg_bias_current_scale(sh, 0)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(scas=scores, b=0.05), hk.LAYOUT_PAGED, bias=bias,
                     kernel=hk.KERNEL_AUTO)                  # every one of the 32 (sequence, head) units


def test_bounded_wait_runs_out_and_reports(hk):
    """A hand-over that never comes: the library's self-test kernel waits (short limit) on a barrier nothing
    signals.  The wait must end by itself, the call must answer DEVICE_TIMEOUT, the context must stay in that
    state, and the device must go on working for other contexts."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("expiry", L=1, H=2, d=64, sides=W.SIDES_13[:5], n_seq=1, s=1)
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=256) as ses:
        assert hk.heatkv_device_status(ses.ctx) == 0
        assert hk.heatkv_selftest_wait_expiry(ses.ctx) == -7
        assert hk.heatkv_device_status(ses.ctx) == -7
    ref = O.explicit_schedule(np.ones((sh.L, sh.H)), sh.s, sh.sides)
    _run_full_parity(hk, sh, ref, lambda ses: ses.schedule(policy=hk.POLICY_EXPLICIT, fraction=np.ones((sh.L, sh.H))),
                     hk.LAYOUT_PAGED)


def test_step_order_and_pool_errors(hk):
    sh = W.Shape("err", L=2, H=2, d=64, sides=W.SIDES_13[:8], n_seq=1, s=1)
    scores = W.synthetic_scas(sh, 2)
    from paper_2605_14877_b200.sweep import Session
    ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=1024)
    sch = ses.schedule(scas=scores, b=1.0)
    # full cache of this shape needs more rows than the pool has
    with pytest.raises(hk.HeatKVError) as e:
        hk.heatkv_seq_open(ses.ctx, sch)
    assert e.value.status == -4
    sch2 = ses.schedule(scas=scores, b=0.1)
    sid = hk.heatkv_seq_open(ses.ctx, sch2)
    q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
    out = torch.zeros_like(q)
    with pytest.raises(hk.HeatKVError) as e:            # step 1 before step 0
        ses.run_layer_step([sid], 0, 1, q, k, v, out)
    assert e.value.status == -5
    ses.run_layer_step([sid], 0, 0, q, k, v, out)
    with pytest.raises(hk.HeatKVError) as e:            # same step twice
        ses.run_layer_step([sid], 0, 0, q, k, v, out)
    assert e.value.status == -5
    with pytest.raises(hk.HeatKVError):                 # unknown sequence
        ses.run_layer_step([sid + 7], 0, 1, q, k, v, out)
    with pytest.raises(hk.HeatKVError):                 # misaligned pointer
        hk.heatkv_scale_attention(ses.ctx, [sid], 1, 0, q.data_ptr() + 2, k, v, None, None, out)
    hk.heatkv_seq_close(ses.ctx, sid)
    hk.heatkv_schedule_free(sch)
    hk.heatkv_schedule_free(sch2)
    ses.close()


def test_config2_graph_replay_sampled_heads(hk):
    """Config 2 at full size in the launch configuration the bench times: the 13-step sweep (one
    heatkv_attention_append call per scale) recorded once into a CUDA graph (per-scale contiguous buffers,
    default strides) and replayed; outputs of
    the replay against the oracle on all 32 (sequence, head) units."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG2
    scores = W.synthetic_scas(sh, 0)
    ref = O.heatkv_schedule(scores, 0.05, sh.s, sh.sides)
    bias_np = W.seg_bias_current_scale(sh, 0)
    sm = 1.0 / math.sqrt(sh.d)
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=2 * sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K)) as ses:
        sch = ses.schedule(scas=scores, b=0.05)
        bias = torch.from_numpy(bias_np).cuda()
        q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
        qs, ks, vs, outs = [], [], [], []
        for step in range(sh.K):
            lo, hi = ses.step_slices(step)
            qs.append(q[:, :, lo:hi].contiguous()); ks.append(k[:, :, lo:hi].contiguous())
            vs.append(v[:, :, lo:hi].contiguous()); outs.append(torch.zeros_like(qs[-1]))

        def sweep():
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            for step in range(sh.K):
                ses.pre_step(ids, step)
                hk.heatkv_attention_append(ses.ctx, ids, 0, step, qs[step], ks[step], vs[step], None, bias[0, step],
                                           outs[step])
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)

        sweep()                                   # plan upload and one-time kernel attributes happen here
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            sweep()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            sweep()
        for o in outs:
            o.zero_()
        graph.replay()
        graph.replay()
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        qh, kh, vh = _f64(q), _f64(k), _f64(v)
        stats = _ErrStats()
        for (s_, h) in [(a, b) for a in range(sh.n_seq) for b in range(sh.H)]:
            for step in range(1, sh.K + 1):
                brow = bias_np[0, step - 1, h].astype(np.float64)
                lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
                want = O.scale_attention(qh[s_, h, lo:hi], kh[s_, h], vh[s_, h], ref, step, 0, h, sm, brow)
                _check_attention(outs[step - 1][s_, h], want, ("graph", s_, h, step), stats)
        stats.check()
        hk.heatkv_schedule_free(sch)
