"""Seeded synthetic inputs for the HeatKV hot path (shared by oracle tests, GPU tests, bench).

This module holds input generation only: shapes, scale lists and pseudo-random
values.  It contains none of the method's arithmetic (no softmax, no scores, no
schedule, no cache logic), so both the CPU oracle's tests and the CUDA path may
draw inputs from it without sharing any computation.

Values come from a counter-based generator written in integer tensor ops that
give bit-identical results on the CPU and on a CUDA device:

    u      = splitmix64(seed * GOLDEN + stream * STREAM_MUL + linear_index)
    value  = NORMAL_TABLE[u >> 48]            (bf16-rounded N(0,1) quantiles)

The workloads stand in for the paper's Infinity-2B / 8B runs (Experimental
Results, "Base Models"), whose weights and prompts are not available: Q/K/V are
i.i.d. N(0,1) in bf16 with the paper's 13-scale 1024x1024 token schedule, and
head-to-head variation of attention locality is injected through an additive
per-(head, source scale) logit bias.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

# Side lengths of the 13 scales of a 1024x1024 generation (t_k = side^2).
SIDES_13 = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
SIDES_TINY = (1, 2, 4, 8)

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_STREAM_MUL = 0xD1342543DE82EF95
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

# Stream ids: one independent random stream per tensor kind.
STREAM_Q, STREAM_K, STREAM_V, STREAM_HEAD, STREAM_SCORE, STREAM_BUDGET = 1, 2, 3, 4, 5, 6


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the int64 with the same bit pattern."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift on int64 tensors (torch's >> is arithmetic)."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping arithmetic), any device."""
    z = x + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


_TABLE_CACHE: Dict[str, torch.Tensor] = {}


def normal_table(device: str | torch.device = "cpu") -> torch.Tensor:
    """65 536 bf16 values: the N(0,1) quantile at (j + 1/2) / 65536, rounded to bf16.

    Always built on the CPU in fp64 and then moved, so every device sees the same bits.
    """
    key = str(device)
    if key not in _TABLE_CACHE:
        if "cpu" not in _TABLE_CACHE:
            p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
            z = math.sqrt(2.0) * torch.erfinv(2.0 * p - 1.0)
            _TABLE_CACHE["cpu"] = z.to(torch.float32).to(torch.bfloat16)
        _TABLE_CACHE[key] = _TABLE_CACHE["cpu"].to(device)
    return _TABLE_CACHE[key]


def hash_u64(seed: int, stream: int, start: int, count: int,
             device: str | torch.device = "cpu") -> torch.Tensor:
    """int64 tensor of `count` hashed words for linear indices start .. start+count-1."""
    base = _s64(seed * _GOLDEN + stream * _STREAM_MUL + start)
    idx = torch.arange(count, dtype=torch.int64, device=device) + base
    return splitmix64(idx)


def normal_bf16(seed: int, stream: int, shape: Sequence[int], offset: int = 0,
                device: str | torch.device = "cpu") -> torch.Tensor:
    """bf16 tensor of the given shape; element with flat index i uses counter offset + i."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    table = normal_table(device)
    chunk = 1 << 24
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        u = hash_u64(seed, stream, offset + s, c, device)
        out[s:s + c] = table[_lsr(u, 48)]
    return out.view(*shape)


def uniform01(seed: int, stream: int, count: int, offset: int = 0) -> np.ndarray:
    """float64 uniforms in [0,1) (53 bits), always computed on the CPU."""
    u = hash_u64(seed, stream, offset, count, "cpu")
    return (_lsr(u, 11).to(torch.float64) * (1.0 / (1 << 53))).numpy()


def std_normal(seed: int, stream: int, count: int, offset: int = 0) -> np.ndarray:
    """float64 N(0,1) draws (inverse-CDF of uniform01), always computed on the CPU."""
    p = torch.from_numpy(uniform01(seed, stream, count, offset)).clamp_(1e-12, 1 - 1e-12)
    return (math.sqrt(2.0) * torch.erfinv(2.0 * p - 1.0)).numpy()


@dataclasses.dataclass(frozen=True)
class Shape:
    """Static shape of one workload."""
    name: str
    L: int
    H: int
    d: int
    sides: Tuple[int, ...]
    n_seq: int
    s: int                      # sink scales

    @property
    def K(self) -> int:
        return len(self.sides)

    @property
    def t(self) -> List[int]:
        return [a * a for a in self.sides]

    @property
    def c(self) -> List[int]:
        out, acc = [], 0
        for a in self.t:
            acc += a
            out.append(acc)
        return out

    @property
    def n_tokens(self) -> int:
        return self.c[-1]


# The five workload shapes (batch = number of sequences).
TINY = Shape("tiny", L=1, H=4, d=64, sides=SIDES_TINY, n_seq=1, s=0)
CFG2 = Shape("2b_single_layer", L=1, H=16, d=128, sides=SIDES_13, n_seq=2, s=3)
CFG3 = Shape("2b_full", L=32, H=16, d=128, sides=SIDES_13, n_seq=8, s=3)
CFG4 = Shape("larger", L=40, H=32, d=128, sides=SIDES_13, n_seq=16, s=3)
CFG5 = Shape("serving", L=32, H=16, d=128, sides=SIDES_13, n_seq=64, s=3)

TINY_FRACTIONS = (1.0, 0.5, 0.25, 0.0)          # per-head budgets of the tiny workload
SERVING_BUDGETS = (1 / 5, 1 / 10, 1 / 20, 1 / 40)


def qkv_layer(shape: Shape, seed: int, layer: int, device: str | torch.device = "cpu",
              n_seq: Optional[int] = None, seq0: int = 0):
    """Q, K, V of one layer for all scales: three bf16 tensors [n_seq, H, n_tokens, d].

    Token axis is the concatenation of the K scales in generation order (raster order
    inside a scale).  The counter of an element is its flat index in the conceptual
    [seq, layer, head, token, dim] array, so any slice can be regenerated alone.
    """
    n_seq = shape.n_seq if n_seq is None else n_seq
    per_head = shape.n_tokens * shape.d
    outs = []
    for stream in (STREAM_Q, STREAM_K, STREAM_V):
        x = torch.empty(n_seq, shape.H, shape.n_tokens, shape.d, dtype=torch.bfloat16, device=device)
        for si in range(n_seq):
            off = (((seq0 + si) * shape.L + layer) * shape.H) * per_head
            x[si] = normal_bf16(seed, stream, (shape.H, shape.n_tokens, shape.d), off, device)
        outs.append(x)
    return tuple(outs)


def seg_bias_current_scale(shape: Shape, seed: int) -> np.ndarray:
    """float32 [L, K(step), H, K(source scale)]: a_h ~ U[0,4] added to the logits of the
    current scale's own keys (source == step), 0 elsewhere.  2B single-layer workload.
    The slice [layer, step] is the contiguous [H, K] table one attention call takes."""
    a = 4.0 * uniform01(seed, STREAM_HEAD, shape.L * shape.H).reshape(shape.L, shape.H)
    bias = np.zeros((shape.L, shape.K, shape.H, shape.K), dtype=np.float32)
    for k in range(shape.K):
        bias[:, k, :, k] = a.astype(np.float32)
    return bias


def seg_bias_prior_lognormal(shape: Shape, seed: int) -> np.ndarray:
    """float32 [L, K(step), H, K(source scale)]: ln g added to the logits of keys of every
    prior source scale i < step, 0 on the current scale.  ln g = z_{l,h} + z'_{l,h,i} / 2
    with z, z' ~ N(0,1): a log-normal per-head strength, modulated per source scale so
    that heads differ in which scales they depend on."""
    zh = std_normal(seed, STREAM_HEAD, shape.L * shape.H).reshape(shape.L, shape.H, 1)
    zs = std_normal(seed, STREAM_HEAD, shape.L * shape.H * shape.K,
                    offset=shape.L * shape.H).reshape(shape.L, shape.H, shape.K)
    lng = (zh + 0.5 * zs).astype(np.float32)
    bias = np.zeros((shape.L, shape.K, shape.H, shape.K), dtype=np.float32)
    for k in range(shape.K):
        bias[:, k, :, :k] = lng[:, :, :k]
    return bias


def synthetic_scas(shape: Shape, seed: int) -> np.ndarray:
    """float64 [L, H, K] positive pseudo-scores (no attention involved) for tests and
    benches that need a schedule without running calibration: exp(N(0,1)) / K."""
    z = std_normal(seed, STREAM_SCORE, shape.L * shape.H * shape.K)
    return (np.exp(z) / shape.K).reshape(shape.L, shape.H, shape.K)


def serving_budgets(n_seq: int, seed: int) -> List[float]:
    """Per-request budget b drawn from SERVING_BUDGETS by hash."""
    u = uniform01(seed, STREAM_BUDGET, n_seq)
    return [SERVING_BUDGETS[int(x * len(SERVING_BUDGETS))] for x in u]


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of a bf16 tensor (on the CPU)."""
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
