"""CPU oracle for the HeatKV hot path -- TEST INFRASTRUCTURE, not the product.

A plain, slow, fp64 restatement of what the paper defines: scale attention mass
(beta), CAS / S-CAS, the removal orders, N_k, Algorithm 1 (HeatKV, Binary-HeatKV,
and the naive boundary policy), Algorithm 2 (CacheSizeAfterLayer / CachedTokens),
the visible key set of every (step, layer, head), the masked attention output,
the cache contents after every layer, and the cache byte count.

Only tests, the smoke check and the bench's cpu_baseline / reference arm may
import this file.  It shares no code with the CUDA path and never imports it.

Conventions: scales, layers and heads are 1-based in the paper; every array here
is 0-based, so "scale k" of the paper is index k-1.  Sets of head-scales are
boolean arrays G[i, l, h] (source scale i, layer l, head h).

Readings taken where the paper is silent or ambiguous (each is also listed in the
design notes): see `cache_size_after_layer` (physical vs. literal future-layer
accounting), `budget_tokens` (integer budget), `order_from_scores` (tie order),
`heatkv_schedule` (last step), `explicit_schedule` (per-head fraction policy, which
has no counterpart in the paper: parity unpinned), and the fp8 cache format at the end of
the file (`quantize_rows_e4m3` / `dequantize_rows_e4m3`: the paper only points at
quantisation, so the format is this library's own: parity unpinned by the paper; the
rounding itself is pinned to the published E4M3 encoding and to a library conversion).
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np

POLICY_HEATKV = 0     # Algorithm 1, green: head-scale units, orders O_i from S-CAS
POLICY_BINARY = 1     # Algorithm 1, blue: head units, one order O from CAS
POLICY_NAIVE = 2      # boundary policy of Sec. 3.3: prune before a scale, E_k = G_k \ G_{k-1}
ACCOUNT_PHYSICAL = 0  # future layers hold what they held when scale k started
ACCOUNT_LITERAL = 1   # Algorithm 2 exactly as printed


# ----------------------------------------------------------------------------- basics
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    u32 = bits.astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def scale_table(sides: Sequence[int]):
    """t_k = w_k * h_k and c_k = sum_{tau<=k} t_tau (Sec. 3.1, first paragraph)."""
    t = np.array([int(a) * int(a) for a in sides], dtype=np.int64)
    c = np.cumsum(t)
    return t, c


def _c_at(c: np.ndarray, k: int) -> int:
    """c_k for a 1-based k, with c_0 = 0."""
    return 0 if k <= 0 else int(c[k - 1])


# ----------------------------------------------------------------------------- calibration
def attention_rows(q: np.ndarray, k: np.ndarray, sm_scale: float,
                   col_bias: Optional[np.ndarray] = None) -> np.ndarray:
    """alpha in R^{t_k x c_k}: row-softmax of sm_scale * q k^T (+ an additive per-column
    bias), every column visible (Sec. 3.1: each row sums to 1 over all c_k tokens)."""
    logits = sm_scale * (q @ k.T)
    if col_bias is not None:
        logits = logits + col_bias[None, :]
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    return e / e.sum(axis=1, keepdims=True)


def beta_row(alpha: np.ndarray, step: int, t: np.ndarray, c: np.ndarray, K: int) -> np.ndarray:
    """Eq. 2 for k1 = step (1-based): beta[k1, k2] = mean over the t_{k1} rows of the
    probability mass on the tokens of scale k2 (columns c_{k2}-t_{k2}+1 .. c_{k2}); 0 for k2 > k1."""
    out = np.zeros(K, dtype=np.float64)
    tk = alpha.shape[0]
    for k2 in range(1, step + 1):
        lo, hi = _c_at(c, k2) - int(t[k2 - 1]), _c_at(c, k2)
        out[k2 - 1] = alpha[:, lo:hi].sum() / tk
    return out


def beta_sample(q: np.ndarray, k: np.ndarray, sides: Sequence[int], sm_scale: float,
                seg_bias: Optional[np.ndarray] = None) -> np.ndarray:
    """beta^d_{l,h} in R^{K x K} (Eq. 2) for one data point and one head.

    q, k: [c_K, d] float64, the head's queries and keys of all scales in generation
    order.  seg_bias: optional [K(step), K(source)] additive logit bias per source scale.
    """
    t, c = scale_table(sides)
    K = len(t)
    beta = np.zeros((K, K), dtype=np.float64)
    for step in range(1, K + 1):
        lo, hi = _c_at(c, step - 1), _c_at(c, step)
        col_bias = None
        if seg_bias is not None:
            col_bias = np.concatenate([np.full(int(t[i]), float(seg_bias[step - 1, i])) for i in range(step)])
        alpha = attention_rows(q[lo:hi], k[:hi], sm_scale, col_bias)
        beta[step - 1] = beta_row(alpha, step, t, c, K)
    return beta


def beta_mean(betas: Sequence[np.ndarray]) -> np.ndarray:
    """beta_{l,h} = 1/|D| * sum_d beta^d_{l,h} (text after Eq. 2)."""
    return np.mean(np.stack(list(betas), axis=0), axis=0)


def cas(beta: np.ndarray, s: int) -> float:
    """Eq. 3: CAS = 1/(K-s) * sum_{tau=s+1}^{K-1} beta[K, tau] (normaliser as printed)."""
    K = beta.shape[0]
    return float(sum(beta[K - 1, tau - 1] for tau in range(s + 1, K))) / (K - s)


def scas(beta: np.ndarray, s: int) -> np.ndarray:
    """Eq. 4: S-CAS[k] = 1/(K-k) * sum_{tau=k+1}^{K} beta[tau, k] for k in [s+1, K-1]; 0 elsewhere."""
    K = beta.shape[0]
    out = np.zeros(K, dtype=np.float64)
    for k in range(s + 1, K):
        out[k - 1] = sum(beta[tau - 1, k - 1] for tau in range(k + 1, K + 1)) / (K - k)
    return out


# ----------------------------------------------------------------------------- schedule
def order_from_scores(scores_flat: np.ndarray) -> np.ndarray:
    """Heads sorted from least to most dependent (Sec. 3.1 last sentence, Sec. 3.3):
    ascending score; equal scores by ascending flat head index l*H+h (a reading: the paper
    does not say how ties are broken)."""
    return np.argsort(scores_flat, kind="stable")


def budget_tokens(b: float, T: int, c: np.ndarray) -> int:
    """B = b * T * c_{K-1} (Algorithm 1, first line) as an integer number of tokens.

    Cache sizes are integers, so 'size > B' equals 'size > floor(B)'.  b arrives as a
    binary fraction (1/20 is not exact), so the floor is taken after a relative guard of
    1e-12: a product within that distance below an integer counts as that integer."""
    K = len(c)
    x = float(b) * float(T) * float(_c_at(c, K - 1))
    return int(np.floor(x * (1.0 + 1e-12) + 1e-9))


def n_pruned_heads(b: float, T: int, s: int, c: np.ndarray) -> np.ndarray:
    """N_k of Eq. 5 for k = 1..K-1 (index k-1): 0 for k <= s; otherwise the smallest
    integer N in [0, T] with N*c_s + (T-N)*c_k <= B, which is Eq. 5's ceiling evaluated in
    integers and clamped to [0, T] (Eq. 5 is negative while c_k < b*c_{K-1}).
    Raises ValueError when even N = T does not fit (b*c_{K-1} < c_s)."""
    K = len(c)
    B = budget_tokens(b, T, c)
    cs = _c_at(c, s)
    out = np.zeros(K - 1, dtype=np.int64)
    for k in range(1, K):
        if k <= s:
            continue
        ck = _c_at(c, k)
        found = None
        for N in range(0, T + 1):
            if N * cs + (T - N) * ck <= B:
                found = N
                break
        if found is None:
            raise ValueError("budget infeasible: even sink-only heads exceed B")
        out[k - 1] = found
    return out


def cached_tokens(k: int, l: int, h: int, P: np.ndarray, s: int, t: np.ndarray, c: np.ndarray,
                  upto: Optional[int] = None) -> int:
    """CachedTokens(k, l, h, P), scale-dependent form (Appendix A):
    c_s + sum_{i=s+1}^{upto} t_i * 1[(i,l,h) not in P], upto = k as printed.
    Where fewer than s scales exist yet, c_{min(upto, s)} replaces c_s (a reading)."""
    upto = k if upto is None else upto
    m = _c_at(c, min(upto, s))
    for i in range(s + 1, upto + 1):
        if not P[i - 1, l, h]:
            m += int(t[i - 1])
    return m


def cache_size_after_layer(k: int, l_done: int, G_k: np.ndarray, G_km1: np.ndarray, E_k: np.ndarray,
                           s: int, t: np.ndarray, c: np.ndarray, accounting: int = ACCOUNT_PHYSICAL) -> int:
    """Algorithm 2: total cached tokens once layers 1..l_done (1-based count) of scale k ran.

    Layers already executed have applied every scale-k removal (set G_k) and hold scale k.
    For layers not yet executed the printed formula sums source scales up to i = k, which
    counts scale-k tokens those layers have not produced yet.  ACCOUNT_LITERAL keeps that.
    ACCOUNT_PHYSICAL (the reading used by default) counts what such a layer really holds at
    that moment: scales up to k-1 minus A_k = G_{k-1} u E_k.  Both agree at l_done = L."""
    A_k = G_km1 | E_k
    _, L, H = G_k.shape
    M = 0
    for l in range(L):
        for h in range(H):
            if l < l_done:
                M += cached_tokens(k, l, h, G_k, s, t, c)
            elif accounting == ACCOUNT_LITERAL:
                M += cached_tokens(k, l, h, A_k, s, t, c)
            else:
                M += cached_tokens(k, l, h, A_k, s, t, c, upto=k - 1)
    return M


@dataclasses.dataclass
class Schedule:
    """Static schedule: G[k-1], E[k-1], A[k-1] are boolean [K, L, H] sets of head-scales for
    step k = 1..K (G, E defined for k <= K-1; A for k <= K)."""
    K: int
    L: int
    H: int
    s: int
    t: np.ndarray
    c: np.ndarray
    N: np.ndarray
    B: int
    G: List[np.ndarray]
    E: List[np.ndarray]
    A: List[np.ndarray]


def heatkv_schedule(scores: np.ndarray, b: float, s: int, sides: Sequence[int],
                    policy: int = POLICY_HEATKV, accounting: int = ACCOUNT_PHYSICAL) -> Schedule:
    """Algorithm 1.

    scores: [L, H, K] S-CAS (POLICY_HEATKV / POLICY_NAIVE) or [L, H] CAS (POLICY_BINARY).
    For every k = 1..K-1: G_k = union over prunable source scales s < i <= k of
    Prefix(O_i, N_k) (binary: Prefix(O, N_k) applied to every prunable source scale of the
    head); R_k = G_k \\ G_{k-1} sorted by (layer desc, source scale desc, rank asc);
    for l = 1..L: while CacheSizeAfterLayer > B pop R_k into E_k; A_k = G_{k-1} u E_k.
    The loop range is not printed; the last scale is never cached (Sec. 3, Motivation), so
    the loop stops at K-1 and the last step attends with A_K = G_{K-1} (a reading).
    POLICY_NAIVE sets E_k = G_k \\ G_{k-1} (prune before a scale and not after).
    Source scale K has no order (orders exist for s < i < K) and is never stored."""
    t, c = scale_table(sides)
    K = len(t)
    L, H = scores.shape[0], scores.shape[1]
    T = L * H
    N = n_pruned_heads(b, T, s, c)
    B = budget_tokens(b, T, c)

    rank = np.zeros((K, T), dtype=np.int64)        # rank[i-1, head] = position of head in O_i
    order = np.zeros((K, T), dtype=np.int64)
    for i in range(s + 1, K):
        flat = scores.reshape(T, -1)[:, i - 1] if policy != POLICY_BINARY else scores.reshape(T)
        o = order_from_scores(np.asarray(flat, dtype=np.float64))
        order[i - 1] = o
        rank[i - 1, o] = np.arange(T)

    G_prev = np.zeros((K, L, H), dtype=bool)
    Gs, Es, As = [], [], []
    for k in range(1, K):
        G_k = np.zeros((K, L, H), dtype=bool)
        # HeatKV: prunable source scales s < i <= k.  Binary: a pruned head is in sink-only mode,
        # i.e. every non-sink source scale of it (also those not generated yet) is in G_k, which
        # makes the head-scale CachedTokens equal to the binary one (c_s if the head is in P).
        for i in range(s + 1, K if policy == POLICY_BINARY else k + 1):
            for head in order[i - 1, : int(N[k - 1])]:
                G_k[i - 1, head // H, head % H] = True
        E_k = np.zeros((K, L, H), dtype=bool)
        new = G_k & ~G_prev
        if policy == POLICY_NAIVE:
            E_k = new.copy()
        else:
            if policy == POLICY_BINARY:
                # the prunable object is a head: candidates are the heads that enter the prefix
                # at this scale, sorted by (layer desc, rank asc); popping one moves all of its
                # new head-scales into E_k.
                N_prev = int(N[k - 2]) if k >= 2 else 0
                heads = [int(x) for x in order[s, N_prev: int(N[k - 1])]] if s + 1 < K else []
                heads.sort(key=lambda hd: (-(hd // H), rank[s, hd]))
                cand = [[(i, hd // H, hd % H) for i in range(K) if new[i, hd // H, hd % H]] for hd in heads]
            else:
                units = [(i, l, h) for i in range(K) for l in range(L) for h in range(H) if new[i, l, h]]
                units.sort(key=lambda e: (-e[1], -e[0], rank[e[0], e[1] * H + e[2]]))
                cand = [[u] for u in units]
            pos = 0
            for l_done in range(1, L + 1):
                while cache_size_after_layer(k, l_done, G_k, G_prev, E_k, s, t, c, accounting) > B:
                    if pos >= len(cand):
                        raise ValueError("budget infeasible: removal list exhausted")
                    for (i, l, h) in cand[pos]:
                        E_k[i, l, h] = True
                    pos += 1
        Gs.append(G_k)
        Es.append(E_k)
        As.append(G_prev | E_k)
        G_prev = G_k
    As.append(G_prev.copy())                      # step K attends with A_K = G_{K-1}
    return Schedule(K, L, H, s, t, c, N, B, Gs, Es, As)


def explicit_schedule(fractions: np.ndarray, s: int, sides: Sequence[int]) -> Schedule:
    """Per-head fraction policy ("prefix retention"); no counterpart in the paper -- parity unpinned.

    Head (l,h) with fraction f gets the absolute token budget M = ceil(f * c_{K-1}); it stores
    scales 1..j with j = max{ j <= K-1 : c_j <= M }, at least the s sink scales, and refuses
    every later scale.  Nothing is evicted once stored, so E_k is empty and
    A_k = G_{k-1} = {(i,l,h) : i > j_{l,h}, i <= k-1}.  f = 1 is the full cache; f = 0 with
    s = 0 leaves only the current scale visible."""
    t, c = scale_table(sides)
    K = len(t)
    L, H = fractions.shape
    j = np.zeros((L, H), dtype=np.int64)
    for l in range(L):
        for h in range(H):
            M = int(np.ceil(float(fractions[l, h]) * _c_at(c, K - 1) - 1e-9))
            jj = 0
            for cand in range(1, K):
                if _c_at(c, cand) <= M:
                    jj = cand
            j[l, h] = max(jj, min(s, K - 1))
    Gs, Es, As = [], [], []
    G_prev = np.zeros((K, L, H), dtype=bool)
    for k in range(1, K):
        G_k = np.zeros((K, L, H), dtype=bool)
        for i in range(1, k + 1):
            G_k[i - 1] = i > j
        Gs.append(G_k)
        Es.append(np.zeros((K, L, H), dtype=bool))
        As.append(G_prev.copy())
        G_prev = G_k
    As.append(G_prev.copy())
    return Schedule(K, L, H, s, t, c, np.zeros(K - 1, dtype=np.int64), -1, Gs, Es, As)


# ----------------------------------------------------------------------------- cache + attention
def visible_scales(sch: Schedule, step: int, l: int, h: int) -> List[int]:
    """1-based source scales whose cached tokens head (l,h) attends to at step `step`
    (besides its own scale): sinks 1..min(s, step-1), and non-sink i <= step-1 with
    (i,l,h) not in A_step -- A_k is the set absent at the beginning of scale k (Sec. 3.3)."""
    A = sch.A[step - 1]
    out = []
    for i in range(1, step):
        if i <= sch.s or not A[i - 1, l, h]:
            out.append(i)
    return out


def stored_scales_after_layer(sch: Schedule, step: int, l: int, h: int) -> List[int]:
    """1-based source scales in the cache of head (l,h) right after its layer ran at `step`
    (step <= K-1): sinks 1..min(s, step) and non-sink i <= step with (i,l,h) not in G_step;
    the elements of G_k \\ A_k leave immediately after their layer has executed (Sec. 3.3)."""
    G = sch.G[step - 1]
    return [i for i in range(1, step + 1) if i <= sch.s or not G[i - 1, l, h]]


def token_indices(sch: Schedule, scales: Sequence[int]) -> np.ndarray:
    """Global token indices c_{i-1} + j (0-based) of the given scales, ascending scale,
    raster order inside a scale."""
    parts = [np.arange(_c_at(sch.c, i - 1), _c_at(sch.c, i), dtype=np.int64) for i in scales]
    return np.concatenate(parts) if parts else np.zeros(0, dtype=np.int64)


def scale_attention(q_step: np.ndarray, k_all: np.ndarray, v_all: np.ndarray, sch: Schedule,
                    step: int, l: int, h: int, sm_scale: float,
                    seg_bias_row: Optional[np.ndarray] = None) -> np.ndarray:
    """Attention output of head (l,h) at `step`: softmax over the retained prior tokens plus
    the step's own t_k tokens (all of them, no mask inside the scale), times V.

    q_step: [t_k, d]; k_all, v_all: [c_K, d] the head's K/V for all scales (the cache holds
    verbatim copies, so indexing the originals is the definition).  seg_bias_row: optional [K]
    additive logit bias per source scale.  Textbook definition in fp64."""
    vis = visible_scales(sch, step, l, h) + [step]
    idx = token_indices(sch, vis)
    logits = sm_scale * (q_step @ k_all[idx].T)
    if seg_bias_row is not None:
        col = np.concatenate([np.full(int(sch.t[i - 1]), float(seg_bias_row[i - 1])) for i in vis])
        logits = logits + col[None, :]
    logits = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v_all[idx]


def cache_after_layer(k_bits: np.ndarray, v_bits: np.ndarray, sch: Schedule, step: int, l: int, h: int):
    """(retained token indices, K bytes, V bytes) of head (l,h) after its layer ran at `step`.
    k_bits, v_bits: [c_K, d] uint16 bf16 patterns of the head's K/V; survivors keep their order."""
    idx = token_indices(sch, stored_scales_after_layer(sch, step, l, h))
    return idx, k_bits[idx], v_bits[idx]


def cache_before_step(k_bits: np.ndarray, v_bits: np.ndarray, sch: Schedule, step: int, l: int, h: int):
    """Same, at the beginning of `step` (after E_step was evicted): the visible prior scales."""
    idx = token_indices(sch, visible_scales(sch, step, l, h))
    return idx, k_bits[idx], v_bits[idx]


def kept_tokens_after_step(sch: Schedule, step: int) -> np.ndarray:
    """[L, H] tokens in each head's cache at the end of scale `step` (<= K-1)."""
    out = np.zeros((sch.L, sch.H), dtype=np.int64)
    for l in range(sch.L):
        for h in range(sch.H):
            out[l, h] = sum(int(sch.t[i - 1]) for i in stored_scales_after_layer(sch, step, l, h))
    return out


def cache_bytes(kept: np.ndarray, d: int, dtype_bytes: int = 2) -> int:
    """sum over (layer, head) of kept_tokens * head_dim * 2 (K and V) * dtype bytes."""
    return int(kept.sum()) * d * 2 * dtype_bytes


# ----------------------------------------------------------------------------- S-CAS stability (Appendix C)
def scas_rank_dispersion(scas_runs: np.ndarray, s: int) -> np.ndarray:
    """Stability of the S-CAS head ordering across calibration runs (Appendix, "S-CAS stability").

    scas_runs: [R, L, H, K] S-CAS of R independent calibration sets.  For every prunable source scale
    k in [s+1, K-1] each run orders the heads (order_from_scores); a head's rank position is recorded per
    run, its standard deviation around the head's own mean rank is taken over the runs (population form,
    1/R), and these are averaged over the heads.  Returns [K] (0 outside the prunable scales)."""
    R, L, H, K = scas_runs.shape
    T = L * H
    out = np.zeros(K, dtype=np.float64)
    for k in range(s + 1, K):
        ranks = np.zeros((R, T), dtype=np.float64)
        for r in range(R):
            o = order_from_scores(np.asarray(scas_runs[r].reshape(T, K)[:, k - 1], dtype=np.float64))
            for pos in range(T):
                ranks[r, o[pos]] = pos
        acc = 0.0
        for head in range(T):
            mean = sum(ranks[r, head] for r in range(R)) / R
            var = sum((ranks[r, head] - mean) ** 2 for r in range(R)) / R
            acc += var ** 0.5
        out[k - 1] = acc / T
    return out


# ----------------------------------------------------------------------------- fp8 K/V cache (build-defined)
# The paper names cache quantisation only as an orthogonal direction (Sec. 5 and the conclusion) and defines
# no format, so everything below is this library's own definition: PARITY UNPINNED BY THE PAPER.  What the
# format borrows is public: the 8-bit E4M3 encoding of the OCP "8-bit floating point" specification
# (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; subnormals; no infinities; S.1111.111 is NaN;
# largest finite value 448), and power-of-two block scales as in microscaling formats.
#
# A cached row (the d values of one token of one head, K or V) is stored as d E4M3 codes plus one signed
# byte e: code_j = RN_even_E4M3(x_j * 2^-e), where e is the smallest integer >= FP8_EXP_MIN with
# max_j |x_j| * 2^-e <= 448.  Reading the cache gives x^_j = value(code_j) * 2^e, which a bf16 holds exactly;
# attention then runs on x^ exactly as it does on an unquantised cache.
FP8_EXP_MIN = -120
FP8_MAX = 448.0


def e4m3_values() -> np.ndarray:
    """value[code] for the 256 E4M3 codes, from the format's definition (NaN for 0x7f and 0xff)."""
    out = np.zeros(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        ex, man = (code >> 3) & 0xF, code & 0x7
        if ex == 0xF and man == 0x7:
            out[code] = np.nan
        elif ex == 0:
            out[code] = sign * (man / 8.0) * 2.0 ** (-6)
        else:
            out[code] = sign * (1.0 + man / 8.0) * 2.0 ** (ex - 7)
    return out


def fp8_row_exponents(x: np.ndarray) -> np.ndarray:
    """[n] the exponent byte of every row of x [n, d] (finite values)."""
    amax = np.abs(x).max(axis=1)
    e = np.full(x.shape[0], FP8_EXP_MIN, dtype=np.int64)
    for r in range(x.shape[0]):
        a = float(amax[r])
        if a == 0.0:
            continue
        k = int(np.ceil(np.log2(a / FP8_MAX))) - 2      # start below the answer, then walk up exactly
        while a * 2.0 ** (-k) > FP8_MAX:
            k += 1
        e[r] = max(k, FP8_EXP_MIN)
    return e


def quantize_rows_e4m3(x: np.ndarray):
    """x [n, d] float64 (bf16 values widened exactly) -> (codes uint8 [n, d], exps int8 [n]).
    Round to nearest on the E4M3 grid, ties to the code with an even mantissa; zero keeps its sign."""
    vals = e4m3_values()
    pos = vals[:0x7F]                                     # codes 0 .. 0x7e ascend from 0 to 448
    e = fp8_row_exponents(x)
    y = x * np.exp2(-e.astype(np.float64))[:, None]       # exact: a power-of-two scaling
    a = np.abs(y)
    hi = np.searchsorted(pos, a, side="left")             # first code with value >= a
    hi = np.minimum(hi, 0x7E)
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = pos[hi] - a, a - pos[lo]
    take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(take_lo, lo, hi).astype(np.uint8)
    code = np.where(np.signbit(y), code | 0x80, code).astype(np.uint8)
    return code, e.astype(np.int8)


def dequantize_rows_e4m3(codes: np.ndarray, exps: np.ndarray) -> np.ndarray:
    """[n, d] float64: value(code) * 2^e, exactly."""
    return e4m3_values()[codes] * np.exp2(exps.astype(np.float64))[:, None]


def cache_bytes_fp8(kept: np.ndarray, d: int) -> int:
    """sum over (layer, head) of kept_tokens * (head_dim codes + 1 exponent byte) * 2 (K and V)."""
    return int(kept.sum()) * (d + 1) * 2
