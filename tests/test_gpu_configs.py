"""GPU parity at the full sizes of the multi-layer workloads: the 2B-class full model cache (32 layers,
batch 8, budgets 1/5, 1/10, 1/20), the larger-model shape (40 layers x 32 heads, batch 16, 1/20) and
the serving sweep (64 concurrent images, mixed per-request budgets, paged cache, staggered admission).

Every (sequence, layer, head) unit runs on the GPU through the C ABI in generation order; the oracle
checks a seeded sample of units (attention of all 13 scales within max-abs 1e-2 / mean-abs 1e-3, retained
indices and cache contents bit-exact) and, for every unit, what holds at any size: cache bytes equal the
closed form sum of kept tokens x d x 2 x 2 bytes, and allocator occupancy.  Besides a few fixed units the
sample is chosen by rule (`_rule_units`): per scale from the eighth on, the heaviest and the lightest head by
visible keys and heads long enough to be cut into pieces.

Inputs: the 2B full workload uses distinct seeded Q/K/V per layer.  The two larger ones would need
more than 160 GB of activations that way, so there all layers share one layer's seeded Q/K/V (the
schedule, the cache and the bias still differ per layer, which is what the kernels see)."""
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


def _schedule(hk, sh, scores, b):
    """Schedule handle built without a context (only the shape is read) and the pool rows one sequence
    of it reserves in the paged layout."""
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    sch = hk.heatkv_build_schedule(cfg, scas=scores, b=b)
    peak, rows = hk.heatkv_schedule_footprint(sch, hk.LAYOUT_PAGED)
    return sch, peak, rows


def _rule_units(sh, ref_of, n_seq, layers, first_step=8, extra_from=7):
    """Units picked by rule rather than by hand: for every scale from `first_step` on (the steps the tensor-memory
    kernel cuts into pieces and dispatches by key count), the head with the most and the head with the fewest
    visible keys among `layers`, in a sequence that rotates with the scale; every head of those layers whose key
    range is long enough to be cut (8 key tiles of 128 and more, twice the shortest piece a cut makes) comes
    with the heaviest.  Returned as (seq, layer, head, first step checked): these extra units are compared
    with the oracle from scale `extra_from` on."""
    units = {}
    for step in range(first_step, sh.K + 1):
        s_ = (step * 5) % n_seq
        ref = ref_of(s_)
        counts = {(l, h): sum(sh.t[i - 1] for i in O.visible_scales(ref, step, l, h)) + sh.t[step - 1]
                  for l in layers for h in range(sh.H)}
        order = sorted(counts, key=lambda lh: (counts[lh], lh))
        picks = [order[0], order[-1]] + [lh for lh in order if counts[lh] >= 8 * 128 and lh[1] % 4 == step % 4][-2:]
        for (l, h) in picks:
            units.setdefault((s_, l, h), extra_from)
    return [(s_, l, h, f) for (s_, l, h), f in sorted(units.items())]


def _check_units(hk, ses, sh, ref, ids, units, layer_data, outs_of, bias):
    """Oracle comparison of sampled (seq, layer, head[, first step]) units after a finished generation."""
    sm = 1.0 / math.sqrt(sh.d)
    tot, n, worst = 0.0, 0, 0.0
    for unit in units:
        (s_, l, h), first = unit[:3], (unit[3] if len(unit) > 3 else 1)
        q, k, v = layer_data(l)
        qh, kh, vh = _f64(q[s_, h]), _f64(k[s_, h]), _f64(v[s_, h])
        out = outs_of(l)
        for step in range(first, sh.K + 1):
            lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
            brow = None if bias is None else bias[l, step - 1, h].astype(np.float64)
            want = O.scale_attention(qh[lo:hi], kh, vh, ref(s_), step, l, h, sm, brow)
            got = out[s_, h, lo:hi].to(torch.float64).cpu().numpy()
            err = np.abs(got - want)
            assert err.max() <= ATOL_MAX, ((s_, l, h, step), err.max())
            assert err.mean() <= ATOL_MEAN + 2.0 ** -9 * np.abs(want).mean(), ((s_, l, h, step), err.mean())
            tot += float(err.sum()); n += err.size; worst = max(worst, float(err.max()))
        # cache at the end of the generation (after scale K-1; the last scale is never stored)
        idx, kk, vv = O.cache_after_layer(W.bf16_bits(k[s_, h]), W.bf16_bits(v[s_, h]), ref(s_), sh.K - 1, l, h)
        got_idx = hk.heatkv_retained_indices(ses.ctx, ids[s_], l, h, sh.c[-1])
        assert np.array_equal(got_idx, idx), (s_, l, h)
        ko = torch.zeros(max(len(idx), 1), sh.d, dtype=torch.bfloat16, device="cuda")
        vo = torch.zeros_like(ko)
        hk.heatkv_export_head(ses.ctx, ids[s_], l, h, ko, vo)
        assert np.array_equal(W.bf16_bits(ko)[: len(idx)], kk), (s_, l, h)
        assert np.array_equal(W.bf16_bits(vo)[: len(idx)], vv), (s_, l, h)
    assert worst <= ATOL_MAX and tot / n <= ATOL_MEAN, (worst, tot / n)


def test_2b_full_model_three_budgets(hk):
    """32 layers x 16 heads, batch 8, distinct seeded activations per layer, prior-scale log-normal bias;
    full generation at budgets 1/5, 1/10 and 1/20."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG3
    scores = W.synthetic_scas(sh, 0)
    bias = W.seg_bias_prior_lognormal(sh, 0)
    bias_dev = torch.from_numpy(bias).cuda()
    layers = [W.qkv_layer(sh, 0, l, device="cuda") for l in range(sh.L)]
    outs = [torch.zeros_like(layers[l][0]) for l in range(sh.L)]
    fixed = [(0, 0, 0), (3, 7, 5), (5, 18, 11), (7, 31, 15)]
    for b in (1 / 5, 1 / 10, 1 / 20):
        ref = O.heatkv_schedule(scores, b, sh.s, sh.sides)
        units = fixed + [u for u in _rule_units(sh, lambda s_: ref, sh.n_seq, range(sh.L)) if u[:3] not in fixed]
        assert len(units) >= 12
        sch, peak, rows = _schedule(hk, sh, scores, b)
        assert peak <= ref.B                                      # the budget holds at every checkpoint
        with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=sh.n_seq * rows + 64, meta_bytes=64 << 20) as ses:
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            ses.generate(ids, lambda l: layers[l], lambda l: outs[l], lambda l, k: bias_dev[l, k])
            torch.cuda.synchronize()
            assert hk.heatkv_device_status(ses.ctx) == 0
            kept = O.kept_tokens_after_step(ref, sh.K - 1)
            for i in ids:
                actual, closed = hk.heatkv_cache_bytes(ses.ctx, i)
                reserved = hk.heatkv_seq_reservation(ses.ctx, i)[1] * sh.d * 4
                assert actual == closed == O.cache_bytes(kept, sh.d) and reserved >= actual
            # end-of-generation size obeys the budget: N heads at c_s, the rest at c_{K-1} (Sec. 3.2)
            assert int(kept.sum()) <= ref.B
            st = hk.heatkv_allocator_stats(ses.ctx)
            assert st.open_seqs == sh.n_seq and st.used_tokens == sh.n_seq * int(kept.sum())
            _check_units(hk, ses, sh, lambda s_: ref, ids, units, lambda l: layers[l], lambda l: outs[l], bias)
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
            hk.heatkv_schedule_free(sch)


def test_larger_model_shape_20x(hk):
    """40 layers x 32 heads, batch 16, budget 1/20: the uncompressed cache of this shape is tens of GB,
    the compressed one a few; all layers share one layer's activations (see the file header)."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG4
    b = 1 / 20
    scores = W.synthetic_scas(sh, 1)
    bias = W.seg_bias_prior_lognormal(sh, 1)
    bias_dev = torch.from_numpy(bias).cuda()
    ref = O.heatkv_schedule(scores, b, sh.s, sh.sides)
    data = W.qkv_layer(sh, 1, 0, device="cuda")
    fixed = [(0, 0, 3), (9, 21, 30), (15, 39, 17)]
    units = fixed + [u for u in _rule_units(sh, lambda s_: ref, sh.n_seq, (0, 21, 39)) if u[:3] not in fixed]
    assert len(units) >= 12
    keep_layers = sorted({u[1] for u in units})
    outs = {l: torch.zeros_like(data[0]) for l in keep_layers}
    scratch_out = torch.zeros_like(data[0])
    sch, peak, rows = _schedule(hk, sh, scores, b)
    assert peak <= ref.B                                          # the budget holds at every checkpoint
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=sh.n_seq * rows + 64, meta_bytes=128 << 20) as ses:
        ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
        ses.generate(ids, lambda l: data, lambda l: outs.get(l, scratch_out), lambda l, k: bias_dev[l, k])
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        kept = O.kept_tokens_after_step(ref, sh.K - 1)
        actual, closed = hk.heatkv_cache_bytes(ses.ctx, ids[-1])
        reserved = hk.heatkv_seq_reservation(ses.ctx, ids[-1])[1] * sh.d * 4
        assert actual == closed == O.cache_bytes(kept, sh.d)
        full = sh.L * sh.H * sh.c[-2] * sh.d * 4
        assert actual <= b * full and reserved < 0.2 * full
        _check_units(hk, ses, sh, lambda s_: ref, ids, units, lambda l: data, lambda l: outs[l], bias)
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)
        hk.heatkv_schedule_free(sch)


def test_serving_sweep_mixed_budgets_staggered(hk):
    """64 concurrent images of the 2B shape, per-request budgets from {1/5, 1/10, 1/20, 1/40} by hash,
    paged cache with 64-token pages, four admission waves one scale apart; every call mixes sequences of
    different schedules.  All layers share one layer's activations (see the file header)."""
    from paper_2605_14877_b200.sweep import Session
    sh = W.CFG5
    budgets = W.serving_budgets(sh.n_seq, 0)
    scores = W.synthetic_scas(sh, 2)
    bias = W.seg_bias_prior_lognormal(sh, 2)
    bias_dev = torch.from_numpy(bias).cuda()
    refs = {b: O.heatkv_schedule(scores, b, sh.s, sh.sides) for b in sorted(set(budgets))}
    data = W.qkv_layer(sh, 2, 0, device="cuda")
    fixed = [(0, 0, 0), (17, 9, 4), (38, 20, 13), (63, 31, 7)]
    units = fixed + [u for u in _rule_units(sh, lambda s_: refs[budgets[s_]], sh.n_seq, (0, 9, 20, 31)) if u[:3] not in fixed]
    assert len(units) >= 12
    keep_layers = sorted({u[1] for u in units})
    outs = {l: torch.zeros_like(data[0]) for l in keep_layers}
    scratch_out = torch.zeros_like(data[0])
    n_waves, wave = 4, sh.n_seq // 4
    built = {b: _schedule(hk, sh, scores, b) for b in refs}
    schs = {b: built[b][0] for b in refs}
    pool_rows = sum(built[b][2] for b in budgets) + 64
    with Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=pool_rows, meta_bytes=256 << 20, layout=hk.LAYOUT_PAGED) as ses:
        ids = [None] * sh.n_seq
        peak_occupancy = 0.0
        # tick t: wave w is at scale t - w (admitted at tick w, finished after tick w + K - 1)
        for tick in range(sh.K + n_waves - 1):
            for w in range(n_waves):
                step = tick - w
                if step < 0 or step >= sh.K:
                    continue
                members = list(range(w * wave, (w + 1) * wave))
                if step == 0:
                    for s_ in members:
                        ids[s_] = hk.heatkv_seq_open(ses.ctx, schs[budgets[s_]])
                wid = [ids[s_] for s_ in members]
                lo, hi = ses.step_slices(step)
                ses.pre_step(wid, step)
                for l in range(sh.L):
                    q, k, v = (x[members[0]: members[-1] + 1, :, lo:hi] for x in data)
                    o = outs.get(l, scratch_out)[members[0]: members[-1] + 1, :, lo:hi]
                    st = hk.Strides.of(q, k, o)
                    hk.heatkv_scale_attention(ses.ctx, wid, l, step, q, k, v, st, bias_dev[l, step], o)
                    hk.heatkv_append_compact(ses.ctx, wid, l, step, k, v, st)
            st = hk.heatkv_allocator_stats(ses.ctx)
            peak_occupancy = max(peak_occupancy, st.used_tokens / max(st.reserved_rows, 1))
            assert st.reserved_rows <= st.pool_rows
        torch.cuda.synchronize()
        assert hk.heatkv_device_status(ses.ctx) == 0
        st = hk.heatkv_allocator_stats(ses.ctx)
        assert st.open_seqs == sh.n_seq and st.plans == len(refs)
        want_tokens = sum(int(O.kept_tokens_after_step(refs[budgets[s_]], sh.K - 1).sum()) for s_ in range(sh.n_seq))
        assert st.used_tokens == want_tokens
        assert 0.3 < peak_occupancy <= 1.0, peak_occupancy
        for s_ in (0, 17, 38, 63):
            actual, closed = hk.heatkv_cache_bytes(ses.ctx, ids[s_])
            assert actual == closed == O.cache_bytes(O.kept_tokens_after_step(refs[budgets[s_]], sh.K - 1), sh.d)
        _check_units(hk, ses, sh, lambda s_: refs[budgets[s_]], ids, units, lambda l: data, lambda l: outs[l], bias)
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)
        assert hk.heatkv_allocator_stats(ses.ctx).reserved_rows == 0
        for sch in schs.values():
            hk.heatkv_schedule_free(sch)
