// Append of one destination half-tile (up to 64 rows) of a head's new K and V into the rows the plan
// assigns (Sec. 3.3: the scale is stored unless (k, l, h) is in G_k).  Shared by the stand-alone append
// kernel and by the attention kernels, whose launches can carry the append (extra CTAs of the generic
// kernel, spare warps of the tensor-memory kernel).
#pragma once
#include "device_common.cuh"

namespace heatkv {

// `u` = (step * L + layer) * H + head.  Returns at once when the head does not store half-tile `j`.
// All `nthreads` threads of the CTA call it with their `tid`; rows are copied verbatim in 16-byte words.
__device__ __forceinline__ void append_half_tile(const int32_t* plan, int64_t base_row, int u, int j,
                                                 const __nv_bfloat16* __restrict__ k_src,
                                                 const __nv_bfloat16* __restrict__ v_src, int64_t kv_tok,
                                                 __nv_bfloat16* __restrict__ k_pool, __nv_bfloat16* __restrict__ v_pool,
                                                 int d, int tid, int nthreads) {
  constexpr int UNROLL = 4;
  PlanView pv(plan);
  const int cnt = pv.app_cnt()[u];
  if (j >= cnt) return;
  const int2* descs = pv.descs() + pv.app_begin()[u];
  int tok0 = 0;
  for (int i = 0; i < j; ++i) tok0 += descs[i].y & 0xff;
  const int2 dsc = descs[j];
  const int n = dsc.y & 0xff;
  const int64_t row = base_row + dsc.x;
  const int ch_per_row = d / 8;
  const int total = n * ch_per_row;                      // 16-byte chunks per tensor
  const int64_t src_off = (int64_t)tok0 * kv_tok;
  for (int base = tid; base < total; base += nthreads * UNROLL) {
    int4 kv[UNROLL], vv[UNROLL];
#pragma unroll
    for (int uu = 0; uu < UNROLL; ++uu) {
      const int i = base + uu * nthreads;
      if (i < total) {
        const int r = i / ch_per_row, ch = i % ch_per_row;
        const int64_t off = src_off + (int64_t)r * kv_tok + ch * 8;
        kv[uu] = __ldg(reinterpret_cast<const int4*>(k_src + off));
        vv[uu] = __ldg(reinterpret_cast<const int4*>(v_src + off));
      }
    }
#pragma unroll
    for (int uu = 0; uu < UNROLL; ++uu) {
      const int i = base + uu * nthreads;
      if (i < total) {
        const int r = i / ch_per_row, ch = i % ch_per_row;
        const int64_t off = (row + r) * d + ch * 8;
        *reinterpret_cast<int4*>(k_pool + off) = kv[uu];
        *reinterpret_cast<int4*>(v_pool + off) = vv[uu];
      }
    }
  }
}

}  // namespace heatkv
