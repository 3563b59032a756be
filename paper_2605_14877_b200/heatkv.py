"""ctypes binding of libheatkv: argument marshalling only, same names as the C entry points.

Tensors are passed as device pointers (`tensor.data_ptr()`), streams as the raw
`cudaStream_t` of `torch.cuda.current_stream()` unless one is given.  Every function raises
`HeatKVError` when the library returns a negative status.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

__all__ = [
    "HeatKVError", "Config", "Strides", "AllocStats", "lib_path", "exported_symbols",
    "LAYOUT_RAGGED", "LAYOUT_PAGED", "POLICY_HEATKV", "POLICY_BINARY", "POLICY_NAIVE", "POLICY_EXPLICIT",
    "ACCOUNT_PHYSICAL", "ACCOUNT_LITERAL", "KERNEL_AUTO", "KERNEL_GENERIC", "KERNEL_TCGEN05",
    "MAX_K", "MAX_BATCH", "PAGE_TOKENS",
    "heatkv_create", "heatkv_destroy", "heatkv_calibrate_scores", "heatkv_calibrate_scores_steps", "heatkv_calibrate_scores_static",
    "heatkv_finalize_scores", "heatkv_build_schedule", "heatkv_schedule_free", "heatkv_schedule_masks", "heatkv_schedule_footprint",
    "heatkv_schedule_plan", "heatkv_schedule_plan_fp8", "heatkv_seq_open", "heatkv_seq_close", "heatkv_append_compact", "heatkv_scale_attention",
    "heatkv_attention_append", "heatkv_split_plan",
    "heatkv_cache_bytes", "heatkv_retained_indices", "heatkv_export_head", "heatkv_export_head_fp8", "heatkv_allocator_stats",
    "CACHE_BF16", "CACHE_FP8_E4M3", "heatkv_launch_count", "heatkv_kernel_launches", "heatkv_rank_dispersion", "heatkv_seq_reservation", "KernelStats",
    "heatkv_selftest_wait_expiry", "heatkv_device_status", "heatkv_strerror", "heatkv_attention_split", "arena_bytes_for",
]

MAX_K, MAX_BATCH, PAGE_TOKENS = 16, 128, 64
CACHE_BF16, CACHE_FP8_E4M3 = 0, 1
LAYOUT_RAGGED, LAYOUT_PAGED = 0, 1
POLICY_HEATKV, POLICY_BINARY, POLICY_NAIVE, POLICY_EXPLICIT = 0, 1, 2, 3
ACCOUNT_PHYSICAL, ACCOUNT_LITERAL = 0, 1
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_TCGEN05 = 0, 1, 2


class HeatKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {heatkv_strerror(status)} ({status})")


class Config(C.Structure):
    _fields_ = [("L", C.c_int32), ("H", C.c_int32), ("d", C.c_int32), ("K", C.c_int32),
                ("t", C.c_int32 * MAX_K), ("s", C.c_int32), ("layout", C.c_int32), ("kernel", C.c_int32),
                ("sm_scale", C.c_float), ("arena", C.c_void_p), ("arena_bytes", C.c_uint64),
                ("meta_bytes", C.c_uint64), ("scratch_bytes", C.c_uint64),
                ("cache_dtype", C.c_int32), ("reserved0", C.c_int32), ("stage_bytes", C.c_uint64)]

    @classmethod
    def make(cls, L: int, H: int, d: int, t: Sequence[int], s: int, layout: int = LAYOUT_PAGED,
             kernel: int = KERNEL_AUTO, sm_scale: float = 0.0, arena: Optional[torch.Tensor] = None,
             meta_bytes: int = 0, scratch_bytes: int = 0, cache_dtype: int = 0, stage_bytes: int = 0) -> "Config":
        cfg = cls()
        cfg.L, cfg.H, cfg.d, cfg.K, cfg.s = L, H, d, len(t), s
        for i, v in enumerate(t):
            cfg.t[i] = int(v)
        cfg.layout, cfg.kernel, cfg.sm_scale, cfg.meta_bytes = layout, kernel, sm_scale, meta_bytes
        cfg.scratch_bytes = scratch_bytes
        cfg.cache_dtype, cfg.stage_bytes = cache_dtype, stage_bytes
        if arena is not None:
            cfg.arena = arena.data_ptr()
            cfg.arena_bytes = arena.numel() * arena.element_size()
        return cfg


class Strides(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("q_seq", "q_head", "q_tok", "kv_seq", "kv_head", "kv_tok",
                                         "o_seq", "o_head", "o_tok")]

    @classmethod
    def of(cls, q: torch.Tensor, kv: torch.Tensor, o: Optional[torch.Tensor] = None) -> "Strides":
        """Strides of [n_seq, H, t, d] views (d contiguous)."""
        o = q if o is None else o
        for x in (q, kv, o):
            assert x.dim() == 4 and x.stride(3) == 1
        return cls(q.stride(0), q.stride(1), q.stride(2), kv.stride(0), kv.stride(1), kv.stride(2),
                   o.stride(0), o.stride(1), o.stride(2))


class AllocStats(C.Structure):
    _fields_ = [("pool_rows", C.c_uint64), ("reserved_rows", C.c_uint64), ("used_tokens", C.c_uint64),
                ("peak_reserved_rows", C.c_uint64), ("meta_bytes_used", C.c_uint64),
                ("open_seqs", C.c_uint32), ("plans", C.c_uint32)]


class KernelStats(C.Structure):
    _fields_ = [("tcgen05_attention_ready", C.c_uint32), ("tcgen05_calibration_ready", C.c_uint32),
                ("attention_tcgen05", C.c_uint64), ("attention_generic", C.c_uint64),
                ("calibration_tcgen05", C.c_uint64), ("calibration_generic", C.c_uint64),
                ("append", C.c_uint64), ("compact", C.c_uint64), ("other", C.c_uint64)]


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libheatkv.so")


def exported_symbols():
    """Names declared in include/heatkv.h, in declaration order."""
    return ["heatkv_create", "heatkv_destroy", "heatkv_calibrate_scores", "heatkv_calibrate_scores_steps", "heatkv_calibrate_scores_static",
            "heatkv_finalize_scores",
            "heatkv_build_schedule", "heatkv_schedule_free", "heatkv_schedule_masks",
            "heatkv_schedule_footprint", "heatkv_schedule_plan", "heatkv_schedule_plan_fp8", "heatkv_seq_open", "heatkv_seq_close", "heatkv_append_compact",
            "heatkv_scale_attention", "heatkv_attention_append", "heatkv_cache_bytes", "heatkv_seq_reservation",
            "heatkv_retained_indices", "heatkv_export_head", "heatkv_export_head_fp8",
            "heatkv_attention_split", "heatkv_split_plan", "heatkv_allocator_stats", "heatkv_launch_count",
            "heatkv_kernel_launches", "heatkv_rank_dispersion", "heatkv_selftest_wait_expiry", "heatkv_device_status",
            "heatkv_strerror"]


def _load() -> C.CDLL:
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python paper_2605_14877_b200/build.py` "
                          "(the CUDA library is the only implementation; there is no fallback)")
    return C.CDLL(path)


_lib = _load()
_lib.heatkv_strerror.restype = C.c_char_p
_lib.heatkv_strerror.argtypes = [C.c_int]
_P = C.c_void_p
_lib.heatkv_create.argtypes = [C.POINTER(Config), _P, C.POINTER(_P)]
_lib.heatkv_destroy.argtypes = [_P]
_lib.heatkv_calibrate_scores.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, _P, C.POINTER(Strides), _P, _P, _P, _P]
_lib.heatkv_calibrate_scores_static.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, C.POINTER(Strides), _P, _P, _P]
_lib.heatkv_calibrate_scores_steps.argtypes = [_P, C.c_int, C.c_int, C.c_int, C.c_int, _P, _P, C.POINTER(Strides), _P, _P, _P]
_lib.heatkv_finalize_scores.argtypes = [_P, _P, C.c_int, _P, _P, _P, _P]
_lib.heatkv_build_schedule.argtypes = [C.POINTER(Config), _P, _P, C.c_int, C.c_int, C.c_double, _P, C.POINTER(_P)]
_lib.heatkv_schedule_free.argtypes = [_P]
_lib.heatkv_schedule_masks.argtypes = [_P, _P, _P, _P, C.POINTER(C.c_int64)]
_lib.heatkv_schedule_footprint.argtypes = [_P, C.c_int, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
_lib.heatkv_schedule_plan.argtypes = [_P, C.c_int, _P, C.POINTER(C.c_int64)]
_lib.heatkv_schedule_plan_fp8.argtypes = [_P, _P, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
_lib.heatkv_seq_open.argtypes = [_P, _P, _P, C.POINTER(C.c_int)]
_lib.heatkv_seq_close.argtypes = [_P, C.c_int]
_lib.heatkv_append_compact.argtypes = [_P, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, _P, _P, C.POINTER(Strides), _P]
_lib.heatkv_scale_attention.argtypes = [_P, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, _P, _P, _P,
                                        C.POINTER(Strides), _P, _P, _P]
_lib.heatkv_attention_append.argtypes = [_P, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, _P, _P, _P,
                                         C.POINTER(Strides), _P, _P, _P]
_lib.heatkv_split_plan.argtypes = [C.POINTER(C.c_int32), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_uint64,
                                   C.POINTER(C.c_int32), C.POINTER(C.c_double), C.POINTER(C.c_double)]
_lib.heatkv_attention_split.argtypes = [_P, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int32),
                                        C.POINTER(C.c_int32)]
_lib.heatkv_cache_bytes.argtypes = [_P, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
_lib.heatkv_retained_indices.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, C.POINTER(C.c_int)]
_lib.heatkv_export_head.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, _P]
_lib.heatkv_export_head_fp8.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, _P, _P, _P]
_lib.heatkv_allocator_stats.argtypes = [_P, C.POINTER(AllocStats)]
_lib.heatkv_launch_count.argtypes = [_P, C.POINTER(C.c_uint64)]
_lib.heatkv_device_status.argtypes = [_P, _P]
_lib.heatkv_selftest_wait_expiry.argtypes = [_P, _P]
_lib.heatkv_kernel_launches.argtypes = [_P, C.POINTER(KernelStats)]
_lib.heatkv_rank_dispersion.argtypes = [_P, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, _P]
_lib.heatkv_seq_reservation.argtypes = [_P, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
for _n in exported_symbols():
    if _n != "heatkv_strerror":
        getattr(_lib, _n).restype = C.c_int


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return int(x)


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise HeatKVError(rc, where)


def _ids(seq_ids: Sequence[int]):
    return (C.c_int * len(seq_ids))(*[int(i) for i in seq_ids]), len(seq_ids)


def heatkv_strerror(status: int) -> str:
    return _lib.heatkv_strerror(int(status)).decode()


def arena_bytes_for(pool_rows: int, d: int, meta_bytes: int = 1 << 24, scratch_bytes: int = 1 << 26,
                    cache_dtype: int = 0, stage_bytes: int = 0) -> int:
    """Arena size that yields at least `pool_rows` rows in each of the K and V pools when the context is
    created with the same (non-zero) `meta_bytes`, `scratch_bytes` and, for the fp8 cache, `stage_bytes`."""
    rows = (pool_rows + PAGE_TOKENS - 1) // PAGE_TOKENS * PAGE_TOKENS
    fixed = (meta_bytes + 1023) // 1024 * 1024 + (scratch_bytes + 1023) // 1024 * 1024
    if cache_dtype == CACHE_FP8_E4M3:
        return fixed + stage_bytes + 2 * rows * (d + 1)
    return fixed + 2 * rows * d * 2


def heatkv_create(cfg: Config, stream=None) -> int:
    out = _P()
    _check(_lib.heatkv_create(C.byref(cfg), _stream(stream), C.byref(out)), "heatkv_create")
    return out.value


def heatkv_destroy(ctx: int) -> None:
    _check(_lib.heatkv_destroy(ctx), "heatkv_destroy")


def heatkv_calibrate_scores(ctx, layer, step, n_seq, q, k_full, v_full, strides, seg_bias, beta_accum, out,
                            stream=None) -> None:
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_calibrate_scores(ctx, layer, step, n_seq, _ptr(q), _ptr(k_full), _ptr(v_full), st,
                                        _ptr(seg_bias), _ptr(beta_accum), _ptr(out), _stream(stream)),
           "heatkv_calibrate_scores")


def heatkv_calibrate_scores_steps(ctx, layer, step_begin, step_end, n_seq, q_all, k_all, strides, seg_bias, beta_accum,
                                  stream=None) -> None:
    """Eq. 2 for steps step_begin .. step_end - 1 of one layer in one call (q_all, k_all: [n_seq, H, tokens, d] with
    all scales on the token axis; seg_bias: [step_end, H, K] or None)."""
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_calibrate_scores_steps(ctx, layer, step_begin, step_end, n_seq, _ptr(q_all), _ptr(k_all), st,
                                              _ptr(seg_bias), _ptr(beta_accum), _stream(stream)),
           "heatkv_calibrate_scores_steps")


def heatkv_calibrate_scores_static(ctx, layer, step, n_seq, q, k_full, strides, seg_bias, beta_accum,
                                   stream=None) -> None:
    """Same beta update as heatkv_calibrate_scores, for callers that must not allocate device memory:
    the scratch is an array inside the library.  Raises HeatKVError(-10) when the call is too large."""
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_calibrate_scores_static(ctx, layer, step, n_seq, _ptr(q), _ptr(k_full), st, _ptr(seg_bias),
                                               _ptr(beta_accum), _stream(stream)), "heatkv_calibrate_scores_static")


def heatkv_finalize_scores(ctx, beta_accum, n_samples, L, H, K, stream=None):
    """Returns (beta [L,H,K,K], scas [L,H,K], cas [L,H]) as float64 numpy arrays."""
    beta = np.zeros((L, H, K, K), dtype=np.float64)
    scas = np.zeros((L, H, K), dtype=np.float64)
    cas = np.zeros((L, H), dtype=np.float64)
    _check(_lib.heatkv_finalize_scores(ctx, _ptr(beta_accum), n_samples, _ptr(beta), _ptr(scas), _ptr(cas),
                                       _stream(stream)), "heatkv_finalize_scores")
    return beta, scas, cas


def heatkv_build_schedule(cfg: Config, scas=None, cas=None, policy: int = POLICY_HEATKV,
                          accounting: int = ACCOUNT_PHYSICAL, b: float = 1.0, fraction=None) -> int:
    keep = [None if a is None else np.ascontiguousarray(a, dtype=np.float64) for a in (scas, cas, fraction)]
    out = _P()
    _check(_lib.heatkv_build_schedule(C.byref(cfg), _ptr(keep[0]), _ptr(keep[1]), policy, accounting, float(b),
                                      _ptr(keep[2]), C.byref(out)), "heatkv_build_schedule")
    return out.value


def heatkv_schedule_free(sch: int) -> None:
    _check(_lib.heatkv_schedule_free(sch), "heatkv_schedule_free")


def heatkv_schedule_masks(sch: int, K: int, L: int, H: int):
    """Returns (attn_mask [K,L,H] uint16, keep_mask [K,L,H] uint16, n_k [K] int32, budget_tokens)."""
    am = np.zeros((K, L, H), dtype=np.uint16)
    km = np.zeros((K, L, H), dtype=np.uint16)
    nk = np.zeros(K, dtype=np.int32)
    b = C.c_int64()
    _check(_lib.heatkv_schedule_masks(sch, _ptr(am), _ptr(km), _ptr(nk), C.byref(b)), "heatkv_schedule_masks")
    return am, km, nk, b.value


def heatkv_schedule_footprint(sch: int, layout: int):
    peak, rows = C.c_int64(), C.c_int64()
    _check(_lib.heatkv_schedule_footprint(sch, layout, C.byref(peak), C.byref(rows)), "heatkv_schedule_footprint")
    return peak.value, rows.value


def heatkv_schedule_plan(sch: int, layout: int) -> np.ndarray:
    """The plan tables as one int32 array (see include/heatkv.h for the layout)."""
    n = C.c_int64(0)
    _check(_lib.heatkv_schedule_plan(sch, layout, None, C.byref(n)), "heatkv_schedule_plan")
    words = np.zeros(n.value, dtype=np.int32)
    _check(_lib.heatkv_schedule_plan(sch, layout, _ptr(words), C.byref(n)), "heatkv_schedule_plan")
    return words


def heatkv_schedule_plan_fp8(sch: int):
    """(plan tables of a context with the fp8 cache as one int32 array, staging rows a sequence needs per call)."""
    n, rows = C.c_int64(0), C.c_int64(0)
    _check(_lib.heatkv_schedule_plan_fp8(sch, None, C.byref(n), None), "heatkv_schedule_plan_fp8")
    words = np.zeros(n.value, dtype=np.int32)
    _check(_lib.heatkv_schedule_plan_fp8(sch, _ptr(words), C.byref(n), C.byref(rows)), "heatkv_schedule_plan_fp8")
    return words, rows.value


def heatkv_seq_open(ctx: int, sch: int, stream=None) -> int:
    out = C.c_int()
    _check(_lib.heatkv_seq_open(ctx, sch, _stream(stream), C.byref(out)), "heatkv_seq_open")
    return out.value


def heatkv_seq_close(ctx: int, seq_id: int) -> None:
    _check(_lib.heatkv_seq_close(ctx, seq_id), "heatkv_seq_close")


def heatkv_append_compact(ctx, seq_ids, layer, step, k_new, v_new, strides=None, stream=None) -> None:
    ids, n = _ids(seq_ids)
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_append_compact(ctx, ids, n, layer, step, _ptr(k_new), _ptr(v_new), st, _stream(stream)),
           "heatkv_append_compact")


def heatkv_scale_attention(ctx, seq_ids, layer, step, q, k_new, v_new, strides, seg_bias, out, stream=None) -> None:
    ids, n = _ids(seq_ids)
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_scale_attention(ctx, ids, n, layer, step, _ptr(q), _ptr(k_new), _ptr(v_new), st,
                                       _ptr(seg_bias), _ptr(out), _stream(stream)), "heatkv_scale_attention")


def heatkv_attention_append(ctx, seq_ids, layer, step, q, k_new, v_new, strides, seg_bias, out, stream=None) -> None:
    """Attention of the layer at the step followed by its cache update, one launch in the paged layout."""
    ids, n = _ids(seq_ids)
    st = C.byref(strides) if strides is not None else None
    _check(_lib.heatkv_attention_append(ctx, ids, n, layer, step, _ptr(q), _ptr(k_new), _ptr(v_new), st,
                                        _ptr(seg_bias), _ptr(out), _stream(stream)), "heatkv_attention_append")


def heatkv_attention_split(ctx, seq_ids, layer, step):
    """(longest piece in 128-key tiles among the heads that are cut, 0 = whole heads; work items of the launch)
    for this attention call."""
    ids, n = _ids(seq_ids)
    a, b = C.c_int32(), C.c_int32()
    _check(_lib.heatkv_attention_split(ctx, ids, n, layer, step, C.byref(a), C.byref(b)), "heatkv_attention_split")
    return a.value, b.value


def heatkv_split_plan(tiles, n_qp: int, n_seq: int, n_sm: int = 148, per_head: bool = True,
                      max_slots: int = 1 << 40, max_ctrs: int = 1 << 40):
    """Pieces per head (tiles in descending order) and the estimated makespans (whole heads, chosen cut)."""
    n = len(tiles)
    t = (C.c_int32 * n)(*[int(x) for x in tiles])
    out = (C.c_int32 * n)()
    a, b = C.c_double(), C.c_double()
    _check(_lib.heatkv_split_plan(t, n, n_qp, n_seq, n_sm, int(per_head), max_slots, max_ctrs, out, C.byref(a), C.byref(b)),
           "heatkv_split_plan")
    return [int(x) for x in out], a.value, b.value


def heatkv_cache_bytes(ctx: int, seq_id: int):
    """(bytes of the rows the plan placed for what the sequence stores, closed form from the schedule's masks)."""
    a, r = C.c_uint64(), C.c_uint64()
    _check(_lib.heatkv_cache_bytes(ctx, seq_id, C.byref(a), C.byref(r)), "heatkv_cache_bytes")
    return a.value, r.value


def heatkv_seq_reservation(ctx: int, seq_id: int):
    """(first pool row, rows) reserved for the sequence."""
    a, r = C.c_uint64(), C.c_uint64()
    _check(_lib.heatkv_seq_reservation(ctx, seq_id, C.byref(a), C.byref(r)), "heatkv_seq_reservation")
    return a.value, r.value


def heatkv_retained_indices(ctx: int, seq_id: int, layer: int, head: int, max_tokens: int) -> np.ndarray:
    idx = np.zeros(max_tokens, dtype=np.int32)
    n = C.c_int()
    _check(_lib.heatkv_retained_indices(ctx, seq_id, layer, head, _ptr(idx), C.byref(n)), "heatkv_retained_indices")
    return idx[: n.value].copy()


def heatkv_export_head_fp8(ctx, seq_id, layer, head, k_codes, v_codes, k_exps, v_exps, stream=None) -> None:
    _check(_lib.heatkv_export_head_fp8(ctx, seq_id, layer, head, _ptr(k_codes), _ptr(v_codes), _ptr(k_exps), _ptr(v_exps),
                                       _stream(stream)), "heatkv_export_head_fp8")


def heatkv_export_head(ctx, seq_id, layer, head, k_out, v_out, stream=None) -> None:
    _check(_lib.heatkv_export_head(ctx, seq_id, layer, head, _ptr(k_out), _ptr(v_out), _stream(stream)),
           "heatkv_export_head")


def heatkv_allocator_stats(ctx: int) -> AllocStats:
    st = AllocStats()
    _check(_lib.heatkv_allocator_stats(ctx, C.byref(st)), "heatkv_allocator_stats")
    return st


def heatkv_launch_count(ctx: int) -> int:
    n = C.c_uint64()
    _check(_lib.heatkv_launch_count(ctx, C.byref(n)), "heatkv_launch_count")
    return n.value


def heatkv_kernel_launches(ctx: int) -> KernelStats:
    st = KernelStats()
    _check(_lib.heatkv_kernel_launches(ctx, C.byref(st)), "heatkv_kernel_launches")
    return st


def heatkv_rank_dispersion(scas_runs, s: int) -> np.ndarray:
    """scas_runs [R, L, H, K] float64 -> [K] mean standard deviation of the heads' rank positions."""
    a = np.ascontiguousarray(scas_runs, dtype=np.float64)
    R, L, H, K = a.shape
    out = np.zeros(K, dtype=np.float64)
    _check(_lib.heatkv_rank_dispersion(_ptr(a), R, L, H, K, int(s), _ptr(out)), "heatkv_rank_dispersion")
    return out


def heatkv_selftest_wait_expiry(ctx: int, stream=None) -> int:
    """Status of the bounded-wait self-test: -7 (a wait ran out, as it must) is the expected answer."""
    return _lib.heatkv_selftest_wait_expiry(ctx, _stream(stream))


def heatkv_device_status(ctx: int, stream=None) -> int:
    return _lib.heatkv_device_status(ctx, _stream(stream))
