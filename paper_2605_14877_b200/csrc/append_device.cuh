// Append of one destination half-tile (up to 64 rows) of a head's new K and V into the rows the plan
// assigns (Sec. 3.3: the scale is stored unless (k, l, h) is in G_k).  Shared by the stand-alone append
// kernel and by the attention kernels, whose launches can carry the append (extra CTAs of the generic
// kernel, spare warps of the tensor-memory kernel).
#pragma once
#include <cuda_fp16.h>

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

// ---------------------------------------------------------------- fp8 cache (E4M3 codes + one exponent byte per row)
// The format is the library's own (the paper only names quantisation as an orthogonal direction, Sec. 5):
// code = round-to-nearest-even of x * 2^-e on the E4M3 grid, e the smallest integer >= -120 with
// max|x| * 2^-e <= 448 over the row.  Both conversions below are exact up to that one rounding: the
// scaling is by a power of two, and the read-back value(code) * 2^e fits a bf16.
constexpr int FP8_EXP_MIN = -120;

// Exponent byte of a row from the largest |x| of the row, given as bf16 bits without the sign.
// |x| = (1 + m/128) * 2^(E-127) fits under 448 = 1.75 * 2^8 after scaling by 2^-(E-135) when m <= 96
// (1 + 96/128 = 1.75), else one more.
__device__ __forceinline__ int fp8_row_exponent(uint32_t amax_bits) {
  const int E = (int)(amax_bits >> 7), m = (int)(amax_bits & 0x7f);
  const int e = E - 135 + (m > 96 ? 1 : 0);
  return amax_bits == 0 ? FP8_EXP_MIN : max(e, FP8_EXP_MIN);
}
__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(127 + e) << 23); }   // -126 <= e <= 127
// two floats -> two E4M3 codes, `lo` in bits 0..7 (round to nearest even, finite inputs stay finite)
__device__ __forceinline__ uint32_t to_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// two E4M3 codes (bits 0..15) -> two floats, exactly
__device__ __forceinline__ void from_e4m3x2(uint32_t codes, float& lo, float& hi) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
  const __half2 v = *reinterpret_cast<const __half2*>(&h2);
  lo = __low2float(v);
  hi = __high2float(v);
}
// 8 bf16 (one 16-byte chunk) -> largest |x| as bf16 bits
__device__ __forceinline__ uint32_t chunk_amax_bits(const int4& v) {
  const uint32_t w[4] = {(uint32_t)v.x, (uint32_t)v.y, (uint32_t)v.z, (uint32_t)v.w};
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) m = max(m, max(w[i] & 0x7fffu, (w[i] >> 16) & 0x7fffu));
  return m;
}
__device__ __forceinline__ uint2 chunk_to_codes(const int4& v, float scale) {
  const uint32_t w[4] = {(uint32_t)v.x, (uint32_t)v.y, (uint32_t)v.z, (uint32_t)v.w};
  uint32_t c[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)      // a bf16 is the upper half of a float
    c[i] = to_e4m3x2(__uint_as_float(w[i] << 16) * scale, __uint_as_float(w[i] & 0xffff0000u) * scale);
  return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

// The same for the fp8 cache: destination half-tile `j` of the head's new K and V, quantised row by row on the way.
// The d / 8 lanes that hold one row (consecutive lanes of one warp) agree on the row's largest magnitude by
// shuffles, then every lane converts its own 8 values of K and of V.  `nthreads` must be a multiple of 32 and
// every thread of the calling warps must take part (the shuffles name the whole warp); `base_row` is the
// sequence's first row in the code pools.
__device__ __forceinline__ void append_half_tile_fp8(const int32_t* plan, int64_t base_row, int u, int j,
                                                     const __nv_bfloat16* __restrict__ k_src,
                                                     const __nv_bfloat16* __restrict__ v_src, int64_t kv_tok,
                                                     uint8_t* __restrict__ k8_pool, uint8_t* __restrict__ v8_pool,
                                                     int8_t* __restrict__ k_exp, int8_t* __restrict__ v_exp, int d, int tid,
                                                     int nthreads) {
  PlanView pv(plan);
  if (j >= pv.app_cnt()[u]) return;
  const int2* descs = pv.descs() + pv.app_begin()[u];
  int tok0 = 0;
  for (int i = 0; i < j; ++i) tok0 += descs[i].y & 0xff;
  const int2 dsc = descs[j];
  const int n = dsc.y & 0xff;
  const int64_t row0 = base_row + dsc.x;
  const int ch_per_row = d / 8;                          // 16 or 8: a power of two that divides the warp
  const int total = n * ch_per_row;
  const int64_t src_off = (int64_t)tok0 * kv_tok;
  const int rounds = (total + nthreads - 1) / nthreads;
  for (int it = 0; it < rounds; ++it) {                  // every thread runs every round: the shuffles need whole warps
    const int i = it * nthreads + tid;
    const bool live = i < total;                         // whole rows are live or not (ch_per_row divides 32)
    const int r = i / ch_per_row, ch = i % ch_per_row;
    int4 kv = make_int4(0, 0, 0, 0), vv = make_int4(0, 0, 0, 0);
    if (live) {
      const int64_t off = src_off + (int64_t)r * kv_tok + ch * 8;
      kv = __ldg(reinterpret_cast<const int4*>(k_src + off));
      vv = __ldg(reinterpret_cast<const int4*>(v_src + off));
    }
    uint32_t ka = chunk_amax_bits(kv), va = chunk_amax_bits(vv);
    for (int o = 1; o < ch_per_row; o <<= 1) {
      ka = max(ka, __shfl_xor_sync(0xffffffffu, ka, o));
      va = max(va, __shfl_xor_sync(0xffffffffu, va, o));
    }
    if (live) {
      const int ke = fp8_row_exponent(ka), ve = fp8_row_exponent(va);
      const int64_t row = row0 + r;
      *reinterpret_cast<uint2*>(k8_pool + row * d + ch * 8) = chunk_to_codes(kv, pow2f(-ke));
      *reinterpret_cast<uint2*>(v8_pool + row * d + ch * 8) = chunk_to_codes(vv, pow2f(-ve));
      if (ch == 0) {
        k_exp[row] = (int8_t)ke;
        v_exp[row] = (int8_t)ve;
      }
    }
  }
}

}  // namespace heatkv
