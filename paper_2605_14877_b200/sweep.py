"""Generation-order driver: issues the C-ABI calls of one image batch in the order a
next-scale model would (for every scale: evict E_k, then per layer attention followed by
the cache update).  Pure call sequencing; every computation happens inside the library."""
from __future__ import annotations

from typing import Callable, Optional, Sequence

import torch

from . import heatkv as hk


class Session:
    """A context plus its arena.  `pool_rows` rows are available to each of the K and V pools."""

    def __init__(self, L: int, H: int, d: int, t: Sequence[int], s: int, pool_rows: int,
                 layout: int = hk.LAYOUT_PAGED, kernel: int = hk.KERNEL_AUTO, sm_scale: float = 0.0,
                 meta_bytes: int = 1 << 24, device: str = "cuda:0", scratch_bytes: int = 1 << 26,
                 cache_dtype: int = hk.CACHE_BF16, stage_bytes: int = 0):
        self.L, self.H, self.d, self.t, self.s = L, H, d, list(t), s
        self.K = len(self.t)
        self.c = [sum(self.t[: i + 1]) for i in range(self.K)]
        self.device = torch.device(device)
        if cache_dtype == hk.CACHE_FP8_E4M3 and stage_bytes == 0:
            stage_bytes = 64 << 20                     # bf16 staging rows of one attention call (K and V)
        nbytes = hk.arena_bytes_for(pool_rows, d, meta_bytes, scratch_bytes, cache_dtype, stage_bytes)
        self.arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
        off = (-self.arena.data_ptr()) % 1024
        self._arena_view = self.arena[off: off + nbytes]
        self.cfg = hk.Config.make(L, H, d, self.t, s, layout, kernel, sm_scale, self._arena_view, meta_bytes,
                                  scratch_bytes, cache_dtype, stage_bytes)
        self.ctx = hk.heatkv_create(self.cfg)

    def close(self) -> None:
        if self.ctx is not None:
            torch.cuda.synchronize(self.device)
            hk.heatkv_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def schedule(self, **kw) -> int:
        return hk.heatkv_build_schedule(self.cfg, **kw)

    def step_slices(self, step: int):
        lo = self.c[step - 1] if step > 0 else 0
        return lo, self.c[step]

    def run_layer_step(self, seq_ids, layer: int, step: int, q, k, v, out, seg_bias=None, fused: bool = False) -> None:
        """q, k, v, out: [n_seq, H, n_tokens, d] tensors holding all scales; uses the slice of `step`.
        `fused`: one heatkv_attention_append call instead of attention followed by the cache update."""
        lo, hi = self.step_slices(step)
        qs, ks, vs, os_ = q[:, :, lo:hi], k[:, :, lo:hi], v[:, :, lo:hi], out[:, :, lo:hi]
        st = hk.Strides.of(qs, ks, os_)
        if fused:
            hk.heatkv_attention_append(self.ctx, seq_ids, layer, step, qs, ks, vs, st, seg_bias, os_)
            return
        hk.heatkv_scale_attention(self.ctx, seq_ids, layer, step, qs, ks, vs, st, seg_bias, os_)
        hk.heatkv_append_compact(self.ctx, seq_ids, layer, step, ks, vs, st)

    def pre_step(self, seq_ids, step: int) -> None:
        hk.heatkv_append_compact(self.ctx, seq_ids, -1, step, None, None, None)

    def generate(self, seq_ids, qkv_of_layer: Callable[[int], tuple], out_of_layer: Callable[[int], torch.Tensor],
                 bias_of: Optional[Callable[[int, int], Optional[torch.Tensor]]] = None,
                 after: Optional[Callable[[int, int], None]] = None, fused: bool = False) -> None:
        """Whole sweep: steps outer, layers inner.  `after(step, layer)` runs after each layer."""
        for step in range(self.K):
            self.pre_step(seq_ids, step)
            for layer in range(self.L):
                q, k, v = qkv_of_layer(layer)
                bias = bias_of(layer, step) if bias_of else None
                self.run_layer_step(seq_ids, layer, step, q, k, v, out_of_layer(layer), bias, fused)
                if after:
                    after(step, layer)
