"""CPU tests of the library's host side: the shared object loads and exports the declared
symbols, the C++ schedule builder agrees with the oracle on identical scores, and the static
cache plan (page tables, append targets, ragged moves) replays to exactly the cache the
oracle defines.  No CUDA call is made."""
import os
import re

import numpy as np
import pytest

import heatkv_workloads as W
from oracle import heatkv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hk():
    from paper_2605_14877_b200 import build
    build.build_library()
    import paper_2605_14877_b200 as hk
    return hk


def test_library_exports_every_declared_symbol(hk):
    import ctypes
    header = open(os.path.join(ROOT, "include", "heatkv.h")).read()
    declared = re.findall(r"^(?:int|const char\*)\s+(heatkv_\w+)\s*\(", header, flags=re.M)
    assert len(declared) >= 19
    lib = ctypes.CDLL(hk.lib_path())
    for name in declared:
        assert hasattr(lib, name), name
    assert set(declared) == set(hk.exported_symbols())
    assert hk.heatkv_strerror(0) == "ok" and "budget" in hk.heatkv_strerror(-3)


def _oracle_masks(sch):
    K, L, H, s = sch.K, sch.L, sch.H, sch.s
    am = np.zeros((K, L, H), dtype=np.uint16)
    km = np.zeros((K, L, H), dtype=np.uint16)
    for k in range(1, K + 1):
        for l in range(L):
            for h in range(H):
                a = sum(1 << (i - 1) for i in O.visible_scales(sch, k, l, h))
                am[k - 1, l, h] = a
                if k < K:
                    km[k - 1, l, h] = sum(1 << (i - 1) for i in O.stored_scales_after_layer(sch, k, l, h))
                else:
                    km[k - 1, l, h] = a
    return am, km


SHAPES = [
    W.Shape("mid", L=6, H=4, d=64, sides=W.SIDES_13, n_seq=1, s=3),
    W.Shape("s0", L=3, H=5, d=64, sides=W.SIDES_13[:9], n_seq=1, s=0),
    W.Shape("one_layer", L=1, H=16, d=128, sides=W.SIDES_13, n_seq=1, s=3),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("policy", [0, 1, 2])
@pytest.mark.parametrize("accounting", [0, 1])
@pytest.mark.parametrize("b", [0.05, 0.1, 0.3, 1.0])
def test_schedule_matches_oracle(hk, shape, policy, accounting, b):
    scores = W.synthetic_scas(shape, 3)
    cas = scores[:, :, min(5, shape.K - 1)].copy()
    cfg = hk.Config.make(shape.L, shape.H, shape.d, shape.t, shape.s)
    try:
        ref = O.heatkv_schedule(cas if policy == 1 else scores, b, shape.s, shape.sides, policy, accounting)
    except ValueError:
        with pytest.raises(hk.HeatKVError) as e:
            hk.heatkv_build_schedule(cfg, scas=scores, cas=cas, policy=policy, accounting=accounting, b=b)
        assert e.value.status == -3
        return
    sch = hk.heatkv_build_schedule(cfg, scas=scores, cas=cas, policy=policy, accounting=accounting, b=b)
    am, km, nk, B = hk.heatkv_schedule_masks(sch, shape.K, shape.L, shape.H)
    hk.heatkv_schedule_free(sch)
    ram, rkm = _oracle_masks(ref)
    assert B == ref.B
    assert list(nk[:-1]) == list(ref.N) and nk[-1] == 0
    assert np.array_equal(am, ram)
    assert np.array_equal(km, rkm)


def test_schedule_2b_shape_matches_oracle(hk):
    sh = W.CFG3
    scores = W.synthetic_scas(sh, 0)
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    for b in (0.05, 0.2):
        ref = O.heatkv_schedule(scores, b, sh.s, sh.sides)
        sch = hk.heatkv_build_schedule(cfg, scas=scores, b=b)
        am, km, nk, B = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
        hk.heatkv_schedule_free(sch)
        ram, rkm = _oracle_masks(ref)
        assert np.array_equal(am, ram) and np.array_equal(km, rkm) and B == ref.B


def test_schedule_ties_break_by_head_index(hk):
    sh = W.Shape("ties", L=2, H=4, d=64, sides=W.SIDES_13[:8], n_seq=1, s=1)
    scores = np.ones((sh.L, sh.H, sh.K))
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    ref = O.heatkv_schedule(scores, 0.3, sh.s, sh.sides)
    sch = hk.heatkv_build_schedule(cfg, scas=scores, b=0.3)
    am, km, _, _ = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
    hk.heatkv_schedule_free(sch)
    ram, rkm = _oracle_masks(ref)
    assert np.array_equal(am, ram) and np.array_equal(km, rkm)


def test_schedule_matches_hand_worked_pop_order(hk):
    """The C++ builder against the hand-derived GreedyEarlyPruning instance (Sec. 3.3, Algorithm 1: Sort of
    R_k by layer descending, source scale descending, rank ascending) -- expected values come from the
    golden file, not from the oracle."""
    from golden_reader import read_early_pruning_instance
    inst, cases = read_early_pruning_instance()
    L, H, K = inst["L"], inst["H"], len(inst["sides"])
    t = [a * a for a in inst["sides"]]
    cfg = hk.Config.make(L, H, 64, t, inst["s"])
    for case in cases:
        accs = {"physical": [0], "printed": [1], "both": [0, 1]}[case["accounting"]]
        for acc in accs:
            sch = hk.heatkv_build_schedule(cfg, scas=inst["scas_array"], cas=inst["cas_array"],
                                           policy=1 if case["policy"] == "binary" else 0, accounting=acc, b=inst["b"])
            am, _, nk, B = hk.heatkv_schedule_masks(sch, K, L, H)
            hk.heatkv_schedule_free(sch)
            assert B == inst["B"] and list(nk[:-1]) == inst["N"]
            for (k, layer, head), vis in case["visible"].items():
                assert am[k - 1, layer - 1, head - 1] == sum(1 << (i - 1) for i in vis), (case["policy"], acc, k, layer, head)


def test_explicit_policy_matches_oracle(hk):
    sh = W.TINY
    frac = np.array([W.TINY_FRACTIONS])
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    sch = hk.heatkv_build_schedule(cfg, policy=hk.POLICY_EXPLICIT, fraction=frac)
    am, km, nk, B = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
    hk.heatkv_schedule_free(sch)
    ram, rkm = _oracle_masks(O.explicit_schedule(frac, sh.s, sh.sides))
    assert B == -1 and np.array_equal(am, ram) and np.array_equal(km, rkm)
    sh = W.Shape("mid", L=3, H=4, d=64, sides=W.SIDES_13, n_seq=1, s=3)
    frac = W.uniform01(5, W.STREAM_BUDGET, 12).reshape(3, 4)
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    sch = hk.heatkv_build_schedule(cfg, policy=hk.POLICY_EXPLICIT, fraction=frac)
    am, km, _, _ = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
    hk.heatkv_schedule_free(sch)
    ram, rkm = _oracle_masks(O.explicit_schedule(frac, sh.s, sh.sides))
    assert np.array_equal(am, ram) and np.array_equal(km, rkm)


def test_schedule_error_paths(hk):
    sh = W.CFG2
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    scores = W.synthetic_scas(sh, 0)
    with pytest.raises(hk.HeatKVError) as e:
        hk.heatkv_build_schedule(cfg, scas=scores, b=0.001)          # b*c_{K-1} < c_s
    assert e.value.status == -3
    bad = scores.copy()
    bad[0, 3, 7] = np.nan
    with pytest.raises(hk.HeatKVError) as e:
        hk.heatkv_build_schedule(cfg, scas=bad, b=0.1)
    assert e.value.status == -6
    for b in (0.0, -1.0, 1.5, float("nan")):
        with pytest.raises(hk.HeatKVError) as e:
            hk.heatkv_build_schedule(cfg, scas=scores, b=b)
        assert e.value.status == -1
    with pytest.raises(hk.HeatKVError):
        hk.heatkv_build_schedule(cfg, scas=None, b=0.1)
    with pytest.raises(hk.HeatKVError):
        hk.heatkv_build_schedule(cfg, scas=scores, b=0.1, policy=9)
    bad_cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, 20)
    with pytest.raises(hk.HeatKVError):
        hk.heatkv_build_schedule(bad_cfg, scas=scores, b=0.1)


# ------------------------------------------------------------------ plan replay
class _Plan:
    def __init__(self, words):
        self.w = words
        self.L, self.H, self.K, self.n_desc = (int(x) for x in words[:4])
        names = ["desc", "attn_begin", "attn_cnt", "app_begin", "app_cnt", "order", "move",
                 "pre_begin", "pre_cnt", "post_begin", "post_cnt"]
        self.off = {n: int(words[4 + i]) for i, n in enumerate(names)}
        self.n_move = int(words[15])
        n = self.K * self.L * self.H
        self.desc = words[self.off["desc"]: self.off["desc"] + 2 * self.n_desc].reshape(-1, 2)
        self.move = words[self.off["move"]: self.off["move"] + 4 * self.n_move].reshape(-1, 4)
        for name in names:
            if name not in ("desc", "move"):
                setattr(self, name, words[self.off[name]: self.off[name] + n].reshape(self.K, self.L, self.H))

    def rows(self, begin, cnt):
        """(pool rows, source scales) listed by descriptors begin .. begin+cnt-1."""
        rows, segs = [], []
        for row, meta in self.desc[begin: begin + cnt]:
            n, sg = int(meta) & 0xff, (int(meta) >> 8) & 0xff
            assert 1 <= n <= 64
            rows += list(range(int(row), int(row) + n))
            segs += [sg] * n
        return rows, segs


def _replay(hk, shape, sch_handle, ref, layout):
    """Runs the whole generation against a numpy 'pool' that stores token ids; checks every
    attention page table and every post-layer cache against the oracle's index lists."""
    words = hk.heatkv_schedule_plan(sch_handle, layout)
    peak, reserved = hk.heatkv_schedule_footprint(sch_handle, layout)
    P = _Plan(words)
    assert (P.L, P.H, P.K) == (shape.L, shape.H, shape.K)
    pool = np.full(reserved, -1, dtype=np.int64)                # value = head * 2^20 + token index
    owner = np.full(reserved, -1, dtype=np.int64)               # which head may read a row
    t, c = shape.t, shape.c
    live_peak = 0
    for k in range(shape.K):
        for l in range(shape.L):                                # eviction before the step
            for h in range(shape.H):
                for m in range(P.pre_begin[k, l, h], P.pre_begin[k, l, h] + P.pre_cnt[k, l, h]):
                    src, dst, n, _ = (int(x) for x in P.move[m])
                    assert dst < src
                    pool[dst: dst + n] = pool[src: src + n].copy()
        for l in range(shape.L):
            for h in range(shape.H):
                hd = l * shape.H + h
                rows, segs = P.rows(P.attn_begin[k, l, h], P.attn_cnt[k, l, h])
                assert all(0 <= r < reserved for r in rows)
                want = O.token_indices(ref, O.visible_scales(ref, k + 1, l, h))
                assert [int(pool[r]) for r in rows] == [hd * (1 << 20) + int(x) for x in want], (k, l, h)
                seg_want = [i - 1 for i in O.visible_scales(ref, k + 1, l, h) for _ in range(t[i - 1])]
                assert segs == seg_want
            if k + 1 < shape.K:
                for h in range(shape.H):
                    for m in range(P.post_begin[k, l, h], P.post_begin[k, l, h] + P.post_cnt[k, l, h]):
                        src, dst, n, _ = (int(x) for x in P.move[m])
                        assert dst < src
                        pool[dst: dst + n] = pool[src: src + n].copy()
                for h in range(shape.H):
                    hd = l * shape.H + h
                    rows, segs = P.rows(P.app_begin[k, l, h], P.app_cnt[k, l, h])
                    stores = k + 1 in O.stored_scales_after_layer(ref, k + 1, l, h)
                    assert len(rows) == (t[k] if stores else 0)
                    assert all(sg == k for sg in segs)
                    for j, r in enumerate(rows):
                        pool[r] = hd * (1 << 20) + (c[k] - t[k] + j)
                        owner[r] = hd
            order = list(P.order[k, l])
            assert sorted(order) == list(range(shape.H))
            cnts = [P.attn_cnt[k, l, h] for h in order]
            vis = [sum(t[i - 1] for i in O.visible_scales(ref, k + 1, l, h)) for h in order]
            assert vis == sorted(vis, reverse=True)
        if k + 1 < shape.K:
            live = int(O.kept_tokens_after_step(ref, k + 1).sum())
            live_peak = max(live_peak, live)
    assert peak >= live_peak
    assert reserved % 64 == 0 and reserved >= peak
    return peak, reserved


@pytest.mark.parametrize("layout", [0, 1], ids=["ragged", "paged"])
@pytest.mark.parametrize("case", ["heatkv", "binary", "naive", "explicit", "full"])
def test_plan_replay_matches_oracle(hk, layout, case):
    sh = W.Shape("mid", L=4, H=3, d=64, sides=W.SIDES_13[:11], n_seq=1, s=3)
    scores = W.synthetic_scas(sh, 9)
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    if case == "explicit":
        frac = W.uniform01(1, W.STREAM_BUDGET, sh.L * sh.H).reshape(sh.L, sh.H)
        ref = O.explicit_schedule(frac, sh.s, sh.sides)
        sch = hk.heatkv_build_schedule(cfg, policy=hk.POLICY_EXPLICIT, fraction=frac)
    else:
        policy = {"heatkv": 0, "binary": 1, "naive": 2, "full": 0}[case]
        b = 1.0 if case == "full" else 0.12
        sc = scores[:, :, 6].copy() if policy == 1 else scores
        ref = O.heatkv_schedule(sc, b, sh.s, sh.sides, policy)
        sch = hk.heatkv_build_schedule(cfg, scas=scores, cas=scores[:, :, 6].copy(), policy=policy, b=b)
    peak, reserved = _replay(hk, sh, sch, ref, layout)
    hk.heatkv_schedule_free(sch)
    if case == "full":
        assert peak == sh.L * sh.H * sh.c[-2]


def test_plan_tiny_workload(hk):
    sh = W.TINY
    frac = np.array([W.TINY_FRACTIONS])
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    ref = O.explicit_schedule(frac, sh.s, sh.sides)
    sch = hk.heatkv_build_schedule(cfg, policy=hk.POLICY_EXPLICIT, fraction=frac)
    for layout in (0, 1):
        peak, _ = _replay(hk, sh, sch, ref, layout)
        assert peak == 21 + 5 + 5 + 0
    hk.heatkv_schedule_free(sch)


def test_paged_reservation_is_tighter_than_ragged_at_2b_shape(hk):
    """Heads peak at different times, so one dense run per head sized for its own peak
    reserves far more than pages handed out over time."""
    sh = W.CFG3
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    sch = hk.heatkv_build_schedule(cfg, scas=W.synthetic_scas(sh, 0), b=0.05)
    peak_r, rows_r = hk.heatkv_schedule_footprint(sch, hk.LAYOUT_RAGGED)
    peak_p, rows_p = hk.heatkv_schedule_footprint(sch, hk.LAYOUT_PAGED)
    hk.heatkv_schedule_free(sch)
    B = O.budget_tokens(0.05, sh.L * sh.H, np.array(sh.c))
    assert peak_r == peak_p <= B
    assert rows_p < rows_r and rows_p < 1.35 * B


def test_scas_rank_dispersion_matches_oracle():
    from paper_2605_14877_b200.analysis import scas_rank_dispersion
    rng = np.random.default_rng(3)
    runs = rng.random((7, 3, 4, 9))
    runs[2, 1, 2, 5] = runs[2, 0, 1, 5]                        # a tie: broken by head index on both sides
    assert np.allclose(scas_rank_dispersion(runs, 3), O.scas_rank_dispersion(runs, 3), rtol=0, atol=1e-12)


# ---- key-range splitting of the attention launch (pure host search, no GPU)
def _pieces_valid(tiles, pieces, min_piece=4):
    for t, n in zip(tiles, pieces):
        assert n >= 1
        piece = -(-t // n)
        assert (n - 1) * piece < t                      # every piece holds at least one tile
        if n > 1:
            assert piece >= min_piece


def test_rank_dispersion_entry_point_errors(hk):
    runs = np.ones((2, 1, 3, 5))
    assert np.all(hk.heatkv_rank_dispersion(runs, 1) == 0)          # equal scores: ties by head index in every run
    bad = runs.copy()
    bad[1, 0, 2, 2] = np.nan
    with pytest.raises(hk.HeatKVError) as e:
        hk.heatkv_rank_dispersion(bad, 1)
    assert e.value.status == -6
    with pytest.raises(hk.HeatKVError) as e:
        hk.heatkv_rank_dispersion(runs, 5)
    assert e.value.status == -1


def test_split_plan_leaves_full_launches_whole():
    import paper_2605_14877_b200 as hk
    # 64 (sequence, head) units x 16 query tile pairs of equal length: 1024 items for 148 SMs, nothing to gain
    pieces, whole, cut = hk.heatkv_split_plan([34] * 32, n_qp=16, n_seq=2)
    assert pieces == [1] * 32 and cut == whole


def test_split_plan_cuts_few_long_heads():
    import paper_2605_14877_b200 as hk
    # 2 heads, one query tile pair, 83 key tiles each: two items for 148 SMs
    pieces, whole, cut = hk.heatkv_split_plan([83, 83], n_qp=1, n_seq=1)
    _pieces_valid([83, 83], pieces)
    assert min(pieces) > 1 and cut < 0.95 * whole
    # the scratch region bounds the cut: no slots, no cut
    pieces0, _, _ = hk.heatkv_split_plan([83, 83], n_qp=1, n_seq=1, max_slots=0)
    assert pieces0 == [1, 1]
    # a longest-run rule (calls that mix schedules): equal heads get equal piece counts
    pieces1, _, _ = hk.heatkv_split_plan([83, 83], n_qp=1, n_seq=1, per_head=False)
    assert pieces1[0] == pieces1[1] > 1


def test_split_plan_ragged_heads_and_invariants():
    import paper_2605_14877_b200 as hk
    rng = np.random.default_rng(0)
    for _ in range(40):
        H = int(rng.integers(1, 40))
        tiles = sorted((int(x) for x in rng.integers(1, 90, size=H)), reverse=True)
        n_qp, n_seq = int(rng.integers(1, 17)), int(rng.integers(1, 9))
        pieces, whole, cut = hk.heatkv_split_plan(tiles, n_qp=n_qp, n_seq=n_seq)
        _pieces_valid(tiles, pieces)
        assert cut <= whole                              # a cut is only taken when the estimate improves
        if pieces != [1] * H:
            assert cut < 0.95 * whole
    # one long head among a few short ones that cannot fill the SMs: the long head is cut, the short ones are not
    tiles = [60] + [8] * 5
    pieces, whole, cut = hk.heatkv_split_plan(tiles, n_qp=2, n_seq=2)
    _pieces_valid(tiles, pieces)
    assert pieces[0] >= 2 and cut < whole and all(n <= 2 for n in pieces[1:])


def test_split_plan_rejects_bad_input():
    import paper_2605_14877_b200 as hk
    with pytest.raises(hk.HeatKVError):
        hk.heatkv_split_plan([3, 5], n_qp=1, n_seq=1)       # not in dispatch (descending) order
    with pytest.raises(hk.HeatKVError):
        hk.heatkv_split_plan([4, 0], n_qp=1, n_seq=1)


def test_fp8_plan_renumbers_attention_rows_into_staging_slots(hk):
    """Plan of a context with the fp8 cache against the plain paged plan of the same schedule: same tables, the
    attention descriptors of every (step, layer) sit in consecutive 64-row staging slots in descriptor order, the
    extra table holds the pool rows the plain plan has in their place, append descriptors keep their pool rows,
    and the staging rows asked for are 64 per visible half-tile of the busiest (step, layer)."""
    sh = W.Shape("mid", L=3, H=4, d=128, sides=W.SIDES_13[:11], n_seq=1, s=3)
    cfg = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    sch = hk.heatkv_build_schedule(cfg, scas=W.synthetic_scas(sh, 4), b=0.15)
    plain = hk.heatkv_schedule_plan(sch, hk.LAYOUT_PAGED)
    fp8, stage_rows = hk.heatkv_schedule_plan_fp8(sch)
    hk.heatkv_schedule_free(sch)
    n_desc = int(plain[3])
    assert int(fp8[3]) == n_desc and int(plain[17]) == 0 and int(fp8[17]) > 0
    for w in range(4, 15):                               # every table of the plain plan sits at the same offset
        assert int(plain[w]) == int(fp8[w])
    pd = plain[int(plain[4]): int(plain[4]) + 2 * n_desc].reshape(n_desc, 2)
    fd = fp8[int(fp8[4]): int(fp8[4]) + 2 * n_desc].reshape(n_desc, 2)
    src = fp8[int(fp8[17]): int(fp8[17]) + n_desc]
    assert np.array_equal(pd[:, 1], fd[:, 1])            # valid rows and source scales unchanged
    assert np.array_equal(src, pd[:, 0])                 # the pool rows moved into the extra table
    n_units = sh.K * sh.L * sh.H
    ab, ac = plain[int(plain[5]): int(plain[5]) + n_units], plain[int(plain[6]): int(plain[6]) + n_units]
    pb, pc = plain[int(plain[7]): int(plain[7]) + n_units], plain[int(plain[8]): int(plain[8]) + n_units]
    is_attn = np.zeros(n_desc, dtype=bool)
    busiest = 0
    for k in range(sh.K):
        for l in range(sh.L):
            u0 = (k * sh.L + l) * sh.H
            first, end = int(ab[u0]), int(ab[u0 + sh.H - 1] + ac[u0 + sh.H - 1])
            for h in range(sh.H):                        # the layer's heads follow one another without gaps
                assert int(ab[u0 + h]) == first + int(ac[u0: u0 + h].sum())
            assert np.array_equal(fd[first:end, 0], 64 * np.arange(end - first))
            is_attn[first:end] = True
            busiest = max(busiest, end - first)
    for u in range(n_units):                             # append descriptors keep pool rows
        b0, n = int(pb[u]), int(pc[u])
        assert not is_attn[b0: b0 + n].any() and np.array_equal(fd[b0: b0 + n, 0], pd[b0: b0 + n, 0])
    assert stage_rows == 64 * busiest and busiest > 0
