"""Pins for the CPU oracle: every oracle function is checked against something other than
itself -- values the paper prints, closed forms in exact rational arithmetic, invariants the
paper states, library routines on special cases, and brute force on tiny inputs."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import heatkv_workloads as W
from oracle import heatkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _head_f64(shape, seed=0, layer=0, seq=0):
    q, k, v = W.qkv_layer(shape, seed, layer, n_seq=seq + 1)
    f = lambda x: O.bf16_bits_to_f64(W.bf16_bits(x[seq]))
    return f(q), f(k), f(v)


def test_bf16_widening_is_exact():
    x = torch.tensor([0.0, -0.0, 1.0, -2.5, 3.0e-5, 65280.0, 1.0 / 3.0], dtype=torch.bfloat16)
    got = O.bf16_bits_to_f64(W.bf16_bits(x))
    assert np.array_equal(got, x.to(torch.float64).numpy())


def test_scale_table_13():
    t, c = O.scale_table(W.SIDES_13)
    assert list(t) == [1, 4, 16, 36, 64, 144, 256, 400, 576, 1024, 1600, 2304, 4096]
    assert list(c) == [1, 5, 21, 57, 121, 265, 521, 921, 1497, 2521, 4121, 6425, 10521]


# ------------------------------------------------------------------ attention (P1, P2, P3)
@pytest.mark.parametrize("with_bias", [False, True])
def test_full_budget_equals_library_attention(with_bias):
    """b = 1 => N_k = 0 => the retained set is everything: must equal plain attention,
    computed here by torch's fp64 scaled_dot_product_attention."""
    sh = W.TINY
    q, k, v = _head_f64(sh)
    scores = W.synthetic_scas(sh, 1)
    sch = O.heatkv_schedule(scores, 1.0, 1, sh.sides)
    assert np.all(sch.N == 0)
    sm = 1.0 / math.sqrt(sh.d)
    rng = np.random.default_rng(0)
    for h in range(sh.H):
        for step in range(1, sh.K + 1):
            lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
            bias_row = rng.normal(size=sh.K) if with_bias else None
            got = O.scale_attention(q[h, lo:hi], k[h], v[h], sch, step, 0, h, sm, bias_row)
            mask = None
            if with_bias:
                col = np.concatenate([np.full(sh.t[i], bias_row[i]) for i in range(step)])
                mask = torch.from_numpy(np.broadcast_to(col, (hi - lo, hi)).copy())
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q[h, lo:hi])[None], torch.from_numpy(k[h, :hi])[None],
                torch.from_numpy(v[h, :hi])[None], attn_mask=mask, scale=sm)[0].numpy()
            assert np.allclose(got, ref, rtol=0, atol=1e-12)


def test_zero_budget_is_current_scale_only_and_first_step_returns_v():
    sh = W.TINY
    q, k, v = _head_f64(sh)
    sch = O.explicit_schedule(np.zeros((1, sh.H)), 0, sh.sides)
    sm = 1.0 / math.sqrt(sh.d)
    for step in range(1, sh.K + 1):
        lo, hi = (sh.c[step - 2] if step > 1 else 0), sh.c[step - 1]
        assert O.visible_scales(sch, step, 0, 0) == []
        got = O.scale_attention(q[0, lo:hi], k[0], v[0], sch, step, 0, 0, sm)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[0, lo:hi])[None], torch.from_numpy(k[0, lo:hi])[None],
            torch.from_numpy(v[0, lo:hi])[None], scale=sm)[0].numpy()
        assert np.allclose(got, ref, rtol=0, atol=1e-12)
    # one query, one key: softmax is 1, output is V
    got = O.scale_attention(q[0, :1], k[0], v[0], sch, 1, 0, 0, sm)
    assert np.array_equal(got, v[0, :1])


def test_softmax_and_beta_rows_sum_to_one_and_upper_triangle_is_zero():
    sh = W.TINY
    q, k, _ = _head_f64(sh)
    sm = 1.0 / math.sqrt(sh.d)
    alpha = O.attention_rows(q[1, 21:85], k[1, :85], sm)
    assert np.allclose(alpha.sum(axis=1), 1.0, atol=1e-13)
    beta = O.beta_sample(q[1], k[1], sh.sides, sm)
    assert np.allclose(beta.sum(axis=1), 1.0, atol=1e-13)
    assert np.all(np.triu(beta, 1) == 0.0)
    assert np.all(beta >= 0)


# ------------------------------------------------------------------ beta / CAS / S-CAS (P4)
def test_beta_brute_force_tiny():
    """Eq. 2 spelled out with scalar loops and math.exp, no shared helper."""
    sh = W.TINY
    q, k, _ = _head_f64(sh)
    h = 2
    sm = 1.0 / math.sqrt(sh.d)
    bias = np.random.default_rng(3).normal(size=(sh.K, sh.K))
    got = O.beta_sample(q[h], k[h], sh.sides, sm, bias)
    t, c = sh.t, sh.c
    seg_of = []
    for i, ti in enumerate(t):
        seg_of += [i] * ti
    ref = np.zeros((sh.K, sh.K))
    for k1 in range(sh.K):
        lo, hi = c[k1] - t[k1], c[k1]
        for n in range(lo, hi):
            logit = [sm * sum(q[h, n, j] * k[h, m, j] for j in range(sh.d)) + bias[k1, seg_of[m]]
                     for m in range(hi)]
            mx = max(logit)
            e = [math.exp(x - mx) for x in logit]
            z = sum(e)
            for m in range(hi):
                ref[k1, seg_of[m]] += e[m] / z / t[k1]
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


def test_beta_constant_logits_closed_form():
    """Q = 0 makes every logit equal: beta[k1,k2] = t_{k2} / c_{k1}."""
    sh = W.TINY
    _, k, _ = _head_f64(sh)
    beta = O.beta_sample(np.zeros_like(k[0]), k[0], sh.sides, 0.125)
    for k1 in range(sh.K):
        for k2 in range(sh.K):
            want = sh.t[k2] / sh.c[k1] if k2 <= k1 else 0.0
            assert abs(beta[k1, k2] - want) < 1e-14


def test_cas_scas_closed_form_on_asymmetric_beta():
    """Eq. 3 / Eq. 4 on a beta whose entries are distinct rationals, against exact fractions.
    beta[k1,k2] = (k2+1)/(sum_{j<=k1}(j+1)) is row-stochastic and far from symmetric, so a
    transposed index or a shifted summation range changes the value."""
    K, s = 7, 2
    B = [[Fraction(k2 + 1, sum(j + 1 for j in range(k1 + 1))) if k2 <= k1 else Fraction(0)
          for k2 in range(K)] for k1 in range(K)]
    beta = np.array([[float(x) for x in row] for row in B])
    want_cas = sum(B[K - 1][tau - 1] for tau in range(s + 1, K)) / (K - s)
    assert abs(O.cas(beta, s) - float(want_cas)) < 1e-15
    got = O.scas(beta, s)
    for k in range(1, K + 1):
        if s + 1 <= k <= K - 1:
            want = sum(B[tau - 1][k - 1] for tau in range(k + 1, K + 1)) / (K - k)
            assert abs(got[k - 1] - float(want)) < 1e-15
        else:
            assert got[k - 1] == 0.0


def test_beta_mean_is_dataset_average():
    a = np.arange(9.0).reshape(3, 3)
    assert np.array_equal(O.beta_mean([a, 3 * a]), 2 * a)


# ------------------------------------------------------------------ N_k (P5)
def _nk_eq5(b: Fraction, T: int, s: int, c):
    K = len(c)
    out = []
    for k in range(1, K):
        if k <= s:
            out.append(0)
            continue
        x = Fraction(T) * (c[k - 1] - b * c[K - 2]) / (c[k - 1] - c[s - 1] if s > 0 else c[k - 1])
        out.append(min(T, max(0, math.ceil(x))))
    return out


@pytest.mark.parametrize("b", [Fraction(1, 20), Fraction(1, 10), Fraction(1, 5), Fraction(1, 25), Fraction(1, 3), Fraction(1)])
@pytest.mark.parametrize("T", [16, 512, 1280])
def test_nk_matches_eq5_in_exact_arithmetic(b, T):
    _, c = O.scale_table(W.SIDES_13)
    got = O.n_pruned_heads(float(b), T, 3, c)
    assert list(got) == _nk_eq5(b, T, 3, [int(x) for x in c])


def test_nk_golden_hand_values():
    _, c = O.scale_table(W.SIDES_13)
    for line in open(os.path.join(GOLDEN, "nk_13scale.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        got = O.n_pruned_heads(float(parts[0]), 512, 3, c)
        assert list(got) == [int(x) for x in parts[1:]]


def test_nk_infeasible_budget_raises():
    _, c = O.scale_table(W.SIDES_13)
    with pytest.raises(ValueError):
        O.n_pruned_heads(0.001, 16, 3, c)       # 0.001 * 6425 < c_3 = 21


def test_budget_tokens_guard():
    _, c = O.scale_table(W.SIDES_13)
    assert O.budget_tokens(0.05, 512, c) == 164480
    assert O.budget_tokens(1 / 20, 16, c) == 5140
    assert O.budget_tokens(0.1, 3, c) == 1927          # 1927.5 -> floor


# ------------------------------------------------------------------ schedule invariants (P6)
def _simulate_checkpoints(sch, policy_sets=None):
    """Independent physical simulation of the cache: a python set of head-scales per head,
    updated in generation order; yields (step, layer_done, total_tokens)."""
    K, L, H, s, t = sch.K, sch.L, sch.H, sch.s, sch.t
    held = {(l, h): set() for l in range(L) for h in range(H)}
    for k in range(1, K):
        A, G = sch.A[k - 1], sch.G[k - 1]
        for (l, h), st in held.items():                       # eviction before the scale starts
            for i in list(st):
                if i > s and A[i - 1, l, h]:
                    st.discard(i)
        yield k, 0, sum(int(t[i - 1]) for st in held.values() for i in st)
        for l in range(L):
            for h in range(H):
                st = held[(l, h)]
                st.add(k)                                      # append, then drop what is in G_k
                for i in list(st):
                    if i > s and G[i - 1, l, h]:
                        st.discard(i)
            yield k, l + 1, sum(int(t[i - 1]) for st in held.values() for i in st)


@pytest.mark.parametrize("policy", [O.POLICY_HEATKV, O.POLICY_BINARY, O.POLICY_NAIVE])
@pytest.mark.parametrize("accounting", [O.ACCOUNT_PHYSICAL, O.ACCOUNT_LITERAL])
@pytest.mark.parametrize("b", [0.05, 0.2])
def test_schedule_invariants(policy, accounting, b):
    sh = W.Shape("mid", L=6, H=4, d=64, sides=W.SIDES_13, n_seq=1, s=3)
    T = sh.L * sh.H
    scores = W.synthetic_scas(sh, 7)
    if policy == O.POLICY_BINARY:
        scores = scores[:, :, 5]
    sch = O.heatkv_schedule(scores, b, sh.s, sh.sides, policy, accounting)
    t, c = sch.t, sch.c
    cs = int(c[sh.s - 1])
    for k in range(1, sh.K):
        G, E, A = sch.G[k - 1], sch.E[k - 1], sch.A[k - 1]
        Gp = sch.G[k - 2] if k > 1 else np.zeros_like(G)
        N = int(sch.N[k - 1])
        assert k > sh.s or N == 0                              # N_k = 0 for k <= s
        assert not np.any(Gp & ~G)                             # G_{k-1} subset of G_k
        assert not np.any(E & ~(G & ~Gp))                      # E_k subset of G_k \ G_{k-1}
        assert np.array_equal(A, Gp | E)                       # A_k = G_{k-1} u E_k
        for i in range(1, sh.K + 1):                           # each source scale absent from N_k heads
            hi = sh.K - 1 if policy == O.POLICY_BINARY else k   # binary: whole head, all scales
            want = N if sh.s < i <= hi else 0
            assert int(G[i - 1].sum()) == want
        # end-of-scale total = N_k c_s + (T - N_k) c_k  (Sec. 3.2)
        assert int(O.kept_tokens_after_step(sch, k).sum()) == N * cs + (T - N) * int(c[k - 1]) or k <= sh.s
    assert np.array_equal(sch.A[sh.K - 1], sch.G[sh.K - 2])
    # the budget holds at every checkpoint of an independent simulation (Sec. 3.3)
    peak = 0
    for k, l_done, total in _simulate_checkpoints(sch):
        assert total <= sch.B, (k, l_done, total, sch.B)
        peak = max(peak, total)
    assert peak > 0.8 * sch.B                                  # and the budget is actually used


def test_heatkv_prunes_less_early_than_naive():
    """Sec. 3.3: pruning before a scale and not after stays under budget but wastes it; the
    greedy set is never larger than the naive one and is strictly smaller somewhere."""
    sh = W.Shape("mid", L=6, H=4, d=64, sides=W.SIDES_13, n_seq=1, s=3)
    scores = W.synthetic_scas(sh, 7)
    a = O.heatkv_schedule(scores, 0.1, sh.s, sh.sides, O.POLICY_HEATKV)
    n = O.heatkv_schedule(scores, 0.1, sh.s, sh.sides, O.POLICY_NAIVE)
    sizes_a = [int(e.sum()) for e in a.E]
    sizes_n = [int(e.sum()) for e in n.E]
    assert all(x <= y for x, y in zip(sizes_a, sizes_n))
    assert sum(sizes_a) < sum(sizes_n)
    for ea, en in zip(a.E, n.E):
        assert not np.any(ea & ~en)


def test_literal_accounting_never_prunes_less_than_physical():
    sh = W.Shape("mid", L=6, H=4, d=64, sides=W.SIDES_13, n_seq=1, s=3)
    scores = W.synthetic_scas(sh, 11)
    p = O.heatkv_schedule(scores, 0.1, sh.s, sh.sides, O.POLICY_HEATKV, O.ACCOUNT_PHYSICAL)
    l = O.heatkv_schedule(scores, 0.1, sh.s, sh.sides, O.POLICY_HEATKV, O.ACCOUNT_LITERAL)
    assert all(int(a.sum()) <= int(b.sum()) for a, b in zip(p.E, l.E))


def test_cache_size_after_layer_matches_simulation():
    """Algorithm 2 (physical reading) against the set-based simulation, at every checkpoint."""
    sh = W.Shape("mid", L=5, H=3, d=64, sides=W.SIDES_13[:9], n_seq=1, s=2)
    scores = W.synthetic_scas(sh, 5)
    sch = O.heatkv_schedule(scores, 0.15, sh.s, sh.sides)
    for k, l_done, total in _simulate_checkpoints(sch):
        if l_done == 0:
            continue
        Gp = sch.G[k - 2] if k > 1 else np.zeros_like(sch.G[0])
        got = O.cache_size_after_layer(k, l_done, sch.G[k - 1], Gp, sch.E[k - 1], sh.s, sch.t, sch.c)
        assert got == total


def test_cached_tokens_printed_formula():
    """CachedTokens (Appendix A) on a hand case: s=1, t=(1,4,16,36), k=4, P = {scale 3}."""
    t, c = O.scale_table((1, 2, 4, 6))
    P = np.zeros((4, 1, 1), dtype=bool)
    P[2, 0, 0] = True
    assert O.cached_tokens(4, 0, 0, P, 1, t, c) == 1 + 4 + 36
    assert O.cached_tokens(4, 0, 0, P, 1, t, c, upto=3) == 1 + 4
    assert O.cached_tokens(1, 0, 0, P, 3, t, c) == 1           # fewer than s scales exist


# ------------------------------------------------------------------ greedy optimality (P7)
def test_greedy_early_pruning_is_minimum_cardinality_binary():
    nontrivial = sum(_greedy_vs_brute_force(seed) for seed in range(6))
    assert nontrivial >= 4          # the instances really need early pruning


def _greedy_vs_brute_force(seed):
    """Proposition 1: in the binary setting the greedy early-pruning set has minimum
    cardinality among feasible subsets of G_k \\ G_{k-1}; checked by enumerating all subsets
    with an independent per-layer simulation."""
    sides = (1, 2, 3, 4, 5, 6)
    L, H, s, b = 4, 2, 1, 0.3
    T = L * H
    rng = np.random.default_rng(seed)
    cas = rng.random((L, H))
    sch = O.heatkv_schedule(cas, b, s, sides, O.POLICY_BINARY)
    t, c = [int(x) for x in sch.t], [int(x) for x in sch.c]
    K = len(t)
    order = list(np.argsort(cas.reshape(-1), kind="stable"))
    nonempty = 0
    for k in range(1, K):
        N_prev = int(sch.N[k - 2]) if k > 1 else 0
        Gk_heads = set(order[: int(sch.N[k - 1])])
        Gp_heads = set(order[:N_prev])
        cand = sorted(Gk_heads - Gp_heads)

        def feasible(E):
            absent = Gp_heads | set(E)
            size = {hd: (c[min(s, k - 1) - 1] if min(s, k - 1) > 0 else 0) if hd in absent
                    else (c[k - 2] if k > 1 else 0) for hd in range(T)}
            if sum(size.values()) > sch.B:
                return False
            for l in range(L):
                for h in range(H):
                    hd = l * H + h
                    size[hd] = c[min(s, k) - 1] if hd in Gk_heads else c[k - 1]
                if sum(size.values()) > sch.B:
                    return False
            return True

        best = None
        for r in range(len(cand) + 1):
            if any(feasible(E) for E in itertools.combinations(cand, r)):
                best = r
                break
        assert best is not None
        greedy_heads = {l * H + h for i in range(K) for l in range(L) for h in range(H)
                        if sch.E[k - 1][i, l, h]}
        assert greedy_heads <= set(cand)
        assert feasible(greedy_heads)
        assert len(greedy_heads) == best
        nonempty += best
    return nonempty


# ------------------------------------------------------------------ cache contents + bytes (P8, P9)
def _golden_early_pruning_cases():
    from golden_reader import read_early_pruning_instance
    inst, cases = read_early_pruning_instance()
    out = []
    for case in cases:
        accs = {"physical": [O.ACCOUNT_PHYSICAL], "printed": [O.ACCOUNT_LITERAL],
                "both": [O.ACCOUNT_PHYSICAL, O.ACCOUNT_LITERAL]}[case["accounting"]]
        for acc in accs:
            out.append((inst, case, acc))
    return out


@pytest.mark.parametrize("inst,case,accounting", _golden_early_pruning_cases(),
                         ids=lambda x: x["policy"] if isinstance(x, dict) and "policy" in x else None)
def test_early_pruning_pop_order_hand_worked(inst, case, accounting):
    """Sec. 3.3 / Algorithm 1, the Sort of R_k: candidates leave by layer descending, then source scale
    descending (head-scale policy), then rank ascending.  The expected E_k and visible sets come from a
    derivation written out by hand in tests/golden/early_pruning_order.txt; with either secondary key
    reversed the instance yields a different E_4."""
    binary = case["policy"] == "binary"
    scores = inst["cas_array"] if binary else inst["scas_array"]
    sch = O.heatkv_schedule(scores, inst["b"], inst["s"], inst["sides"],
                            O.POLICY_BINARY if binary else O.POLICY_HEATKV, accounting)
    assert sch.B == inst["B"] and list(sch.N) == inst["N"]
    K = sch.K
    for k, want in case["E"].items():
        got = {(i + 1, l + 1, h + 1) for i in range(K) for l in range(sch.L) for h in range(sch.H) if sch.E[k - 1][i, l, h]}
        if binary:   # the file lists heads; a popped head takes all its non-sink source scales with it
            want = {(i, l, h) for (l, h) in want for i in range(inst["s"] + 1, K)}
        assert got == want, (k, got, want)
    for (k, layer, head), vis in case["visible"].items():
        assert O.visible_scales(sch, k, layer - 1, head - 1) == vis, (k, layer, head)


def test_cache_contents_brute_force_and_bytes():
    sh = W.Shape("small", L=3, H=4, d=64, sides=W.SIDES_13[:8], n_seq=1, s=2)
    scores = W.synthetic_scas(sh, 2)
    sch = O.heatkv_schedule(scores, 0.25, sh.s, sh.sides)
    for l in range(sh.L):
        q, k, v = W.qkv_layer(sh, 0, l)
        kb, vb = W.bf16_bits(k[0]), W.bf16_bits(v[0])
        for h in range(sh.H):
            for step in range(1, sh.K):
                idx, kk, vv = O.cache_after_layer(kb[h], vb[h], sch, step, l, h)
                want = [m for i in range(1, step + 1)
                        if i <= sh.s or not sch.G[step - 1][i - 1, l, h]
                        for m in range(sh.c[i - 1] - sh.t[i - 1], sh.c[i - 1])]
                assert list(idx) == want
                assert np.array_equal(kk, kb[h][want]) and np.array_equal(vv, vb[h][want])
                idx2, _, _ = O.cache_before_step(kb[h], vb[h], sch, step + 1, l, h)
                assert set(idx2) <= set(idx)                   # eviction only removes
    for step in range(sh.s + 1, sh.K):
        kept = O.kept_tokens_after_step(sch, step)
        N, T = int(sch.N[step - 1]), sh.L * sh.H
        closed = (N * sh.c[sh.s - 1] + (T - N) * sh.c[step - 1]) * sh.d * 2 * 2
        assert O.cache_bytes(kept, sh.d) == closed


def test_table1_full_cache_megabytes():
    """b = 1 keeps c_{K-1} tokens per head; with the shapes in the fixture the byte count
    reproduces the 'Full Cache' figures the paper prints in Table 1."""
    for line in open(os.path.join(GOLDEN, "table1_cache_mb.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, mb, L, width, seqs = line.split()
        d = 128
        H = int(width) // d
        sh = W.Shape(name, L=int(L), H=H, d=d, sides=W.SIDES_13, n_seq=1, s=3)
        sch = O.explicit_schedule(np.ones((sh.L, sh.H)), sh.s, sh.sides)
        kept = O.kept_tokens_after_step(sch, sh.K - 1)
        assert np.all(kept == 6425)
        total_mb = int(seqs) * O.cache_bytes(kept, d) / 2 ** 20
        assert abs(total_mb - int(mb)) < 0.6


# ------------------------------------------------------------------ explicit per-head fractions
def test_explicit_policy_patterns_tiny():
    sh = W.TINY
    sch = O.explicit_schedule(np.array([W.TINY_FRACTIONS]), sh.s, sh.sides)
    vis = lambda h: [O.visible_scales(sch, k, 0, h) for k in (2, 3, 4)]
    assert vis(0) == [[1], [1, 2], [1, 2, 3]]
    assert vis(1) == [[1], [1, 2], [1, 2]]        # M = ceil(.5 * 21) = 11 -> scales 1..2
    assert vis(2) == [[1], [1, 2], [1, 2]]        # M = 6 -> scales 1..2
    assert vis(3) == [[], [], []]
    kept = O.kept_tokens_after_step(sch, 3)
    assert list(kept[0]) == [21, 5, 5, 0]


def test_workload_generator_is_seeded_and_sliceable():
    a = W.qkv_layer(W.TINY, 0, 0)
    b = W.qkv_layer(W.TINY, 0, 0)
    c = W.qkv_layer(W.TINY, 1, 0)
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    assert not torch.equal(a[0], c[0])
    two = W.qkv_layer(W.TINY, 0, 0, n_seq=2)
    second = W.qkv_layer(W.TINY, 0, 0, n_seq=1, seq0=1)
    assert torch.equal(two[1][1], second[1][0])


def test_scas_rank_dispersion_pins():
    """Appendix on S-CAS stability: identical runs give zero dispersion; two runs that swap two adjacent
    heads give those two heads a rank std of 1/2 each; scales outside the prunable range stay 0."""
    rng = np.random.default_rng(0)
    L, H, K, s = 2, 3, 6, 2
    base = rng.random((L, H, K))
    same = np.stack([base] * 4)
    assert np.all(O.scas_rank_dispersion(same, s) == 0)
    swapped = base.copy()
    k = 3                                                    # 0-based source scale inside [s, K-2]
    order = np.argsort(base.reshape(-1, K)[:, k], kind="stable")
    a, b = order[1], order[2]
    flat = swapped.reshape(-1, K)
    flat[a, k], flat[b, k] = flat[b, k], flat[a, k]
    d = O.scas_rank_dispersion(np.stack([base, swapped]), s)
    assert np.isclose(d[k], 2 * 0.5 / (L * H))
    assert np.all(d[:s] == 0) and d[K - 1] == 0
    assert np.all(np.delete(d, k) == 0)


# ----------------------------------------------------------------------------- fp8 cache format (build-defined)
def _fp8_golden_rows():
    rows = []
    for raw in open(os.path.join(GOLDEN, "fp8_rows.txt")):
        line = raw.split("#")[0].strip()
        if not line:
            continue
        a, b, c = line.split(":")
        rows.append((int(a.split()[1]), [float(v) for v in b.split()], [int(v, 16) for v in c.split()]))
    return rows


def test_fp8_rows_hand_worked():
    """Exponent byte and E4M3 codes of the rows derived by hand in tests/golden/fp8_rows.txt (ties to even,
    subnormals, signed zero, the exact-fit exponent)."""
    for e, x, codes in _fp8_golden_rows():
        got_c, got_e = O.quantize_rows_e4m3(np.array([x], dtype=np.float64))
        assert int(got_e[0]) == e
        assert [int(v) for v in got_c[0]] == codes


def test_e4m3_table_closed_forms():
    """The code table against the format's closed forms: 0x38 = 1, 0x7e = 448 (largest finite), 0x08 = 2^-6
    (smallest normal), 0x01 = 2^-9 (smallest subnormal), NaN only at S.1111.111, odd symmetry, strictly
    ascending positive half."""
    v = O.e4m3_values()
    assert v[0x38] == 1.0 and v[0x7E] == 448.0 and v[0x08] == 2.0 ** -6 and v[0x01] == 2.0 ** -9 and v[0] == 0.0
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF]) and np.isnan(v).sum() == 2
    assert (np.diff(v[:0x7F]) > 0).all()
    assert (v[0x80:0xFF] == -v[0x00:0x7F]).all()


def test_fp8_quantiser_matches_a_library_conversion():
    """Inside the finite range the rounding is the one of a library float32 -> float8_e4m3fn conversion
    (round to nearest even); the row exponent is minimal; the read-back value is exactly a bf16; reading and
    quantising again changes no value; the error stays below half a grid step."""
    import torch
    rng = np.random.default_rng(7)
    x = rng.standard_normal((96, 128)) * np.exp2(rng.integers(-30, 30, (96, 1)).astype(np.float64))
    x[5] = 0.0
    x[6, :] = 448.0 * 2.0 ** 3
    x[7, 3] = -x[7].max() * 4
    x = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()          # exactly bf16 values
    codes, e = O.quantize_rows_e4m3(x)
    y = x * np.exp2(-e.astype(np.float64))[:, None]
    amax = np.abs(y).max(axis=1)
    assert (amax <= 448.0).all()
    nz = np.abs(x).max(axis=1) > 0
    assert ((amax[nz] * 2 > 448.0) | (e[nz] == O.FP8_EXP_MIN)).all()              # e - 1 would not fit
    lib = torch.from_numpy(y).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert (lib == codes).all()
    xh = O.dequantize_rows_e4m3(codes, e)
    assert (torch.from_numpy(xh).to(torch.bfloat16).to(torch.float64).numpy() == xh).all()
    c2, e2 = O.quantize_rows_e4m3(xh)
    assert (O.dequantize_rows_e4m3(c2, e2) == xh).all()
    # half a step of the grid at the row's largest value: 2^(e + 8 - 3) / 2
    assert (np.abs(xh - x) <= np.exp2(e.astype(np.float64) + 4)[:, None]).all()
    # elementwise: relative error at most 2^-4 for values in the normal range of the scaled grid
    normal = np.abs(y) >= 2.0 ** -6
    assert (np.abs(xh - x)[normal] <= np.abs(x)[normal] * 2.0 ** -4).all()


def test_fp8_cache_bytes_closed_form():
    kept = np.array([[10, 0], [7, 3]])
    assert O.cache_bytes_fp8(kept, 128) == 20 * 129 * 2
    assert O.cache_bytes_fp8(kept, 128) * 2 < O.cache_bytes(kept, 128) * 1.01 + 1
