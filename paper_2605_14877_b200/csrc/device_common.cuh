// Device-side structures and small PTX wrappers shared by the kernels of libheatkv.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "heatkv.h"

namespace heatkv {

// One sequence of a batched call: device address of its plan blob and the first pool row
// of its reservation.
struct SeqRef {
  const int32_t* plan;
  int64_t base_row;
};

struct AttnParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_new;     // own-scale keys (calibration: all keys)
  const __nv_bfloat16* v_new;
  __nv_bfloat16* out;             // may be null in calibration mode
  const __nv_bfloat16* k_pool;
  const __nv_bfloat16* v_pool;
  const float* seg_bias;          // [H][K] or null
  float* beta_row;                // calibration: &beta_accum[layer][0][step][0]
  int64_t q_seq, q_head, q_tok;
  int64_t kv_seq, kv_head, kv_tok;
  int64_t o_seq, o_head, o_tok;
  int32_t t_q;                    // queries of this step
  int32_t n_own;                  // keys read from k_new (t_q, or c[step] in calibration)
  int32_t step, layer, H, K, L;
  float scale_log2;               // sm_scale * log2(e)
  int32_t c[HEATKV_MAX_K];        // cumulative tokens (calibration: column -> source scale)
  uint32_t* status;               // device status word (non-zero = a bounded wait gave up)
  SeqRef seqs[HEATKV_MAX_BATCH];
  float* partials;                // calibration with a fixed summation order: per-warp partial masses, else null
  // ---- key-range splitting of the tensor-memory attention kernel (split_tiles == 0: no splitting)
  int32_t n_seq;                  // sequences of the call (work items interleave them)
  int32_t split_tiles;            // longest run of 128-key tiles one CTA takes; a head with more is cut into pieces
  int32_t items_per_seq;          // work items (head, piece, query tile pair) of one sequence, an upper bound
  int32_t slots_per_seq;          // partial-result slots reserved per sequence
  int32_t ctrs_per_seq;           // arrival counters reserved per sequence
  int32_t table_heads;            // > 0: every sequence of the call follows one plan and the tables below hold, for
                                  // its heads by descending key count, the head index, its key tiles and its pieces
  int16_t table_head[64];
  int16_t table_tiles[64];
  int16_t table_split[64];        // pieces the head's key range is cut into (1: whole head)
  int32_t longest_piece;          // host report: longest piece among the heads that are cut (0: none is)
  int32_t append_tiles;           // > 0: the launch also stores the step's K/V (paged layout): that many destination
                                  // half-tile slots per (sequence, head) follow the attention work
  int32_t attn_items, store_items;  // tensor-memory kernel: attention work items; cache-update items (destination half-tiles)
  float* split_partials;          // [n_seq * slots_per_seq][SPLIT_SLOT_FLOATS]
  uint32_t* split_counters;       // [n_seq * ctrs_per_seq], zero between launches
  // generic kernel, with table_heads > 0: per head in dispatch order, the half-tile descriptors of its visible
  // prior keys (count, and word offset of the first in the plan blob)
  int16_t table_ndesc[64];
  int32_t table_desc_begin[64];
  // generic kernel, calibration over several steps in one launch (cal_n > 0): the query tiles of step cal_step[e]
  // are blocks cal_tile_begin[e] .. cal_tile_begin[e + 1] - 1 of grid.x; q holds the queries of all scales, beta_row
  // is beta_accum[layer][0][0], seg_bias the bias of step 0 with cal_bias_stride floats between steps
  int32_t cal_n;
  int32_t cal_tile_begin[HEATKV_MAX_K + 1];
  int32_t cal_step[HEATKV_MAX_K];
  int64_t cal_bias_stride;
  // fp8 cache (k8_pool != null): seqs[i].base_row numbers the bf16 staging rows the attention reads; a cache update
  // riding on the launch quantises the new rows into the code pools, where sequence i starts at pool_base[i]
  uint8_t* k8_pool;
  uint8_t* v8_pool;
  int8_t* k_exp;
  int8_t* v_exp;
  int32_t pool_base[HEATKV_MAX_BATCH];
};

struct CopyParams {
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  __nv_bfloat16* k_pool;
  __nv_bfloat16* v_pool;
  int64_t kv_seq, kv_head, kv_tok;
  int32_t t_k, step, layer, H, K, L, d;
  int32_t phase;                  // compaction: 0 = before the step, 1 = after the layer
  int32_t layer_begin, n_layers;  // compaction before a step may cover all layers
  SeqRef seqs[HEATKV_MAX_BATCH];
  // ---- fp8 cache: code pools [rows][d], one exponent byte per row, and the first staging row of every
  // sequence of the call (the bf16 staging rows are k_pool / v_pool)
  uint8_t* k8_pool;
  uint8_t* v8_pool;
  int8_t* k_exp;
  int8_t* v_exp;
  int32_t stage_base[HEATKV_MAX_BATCH];
};

// ---- plan blob accessors (see PlanHeader in internal.h: word offsets from the blob start)
struct PlanView {
  const int32_t* w;
  __device__ __forceinline__ explicit PlanView(const int32_t* p) : w(p) {}
  __device__ __forceinline__ int L() const { return w[0]; }
  __device__ __forceinline__ int H() const { return w[1]; }
  __device__ __forceinline__ int K() const { return w[2]; }
  __device__ __forceinline__ const int2* descs() const { return reinterpret_cast<const int2*>(w + w[4]); }
  __device__ __forceinline__ const int32_t* attn_begin() const { return w + w[5]; }
  __device__ __forceinline__ const int32_t* attn_cnt() const { return w + w[6]; }
  __device__ __forceinline__ const int32_t* app_begin() const { return w + w[7]; }
  __device__ __forceinline__ const int32_t* app_cnt() const { return w + w[8]; }
  __device__ __forceinline__ const int32_t* order() const { return w + w[9]; }
  __device__ __forceinline__ const int4* moves() const { return reinterpret_cast<const int4*>(w + w[10]); }
  __device__ __forceinline__ const int32_t* pre_begin() const { return w + w[11]; }
  __device__ __forceinline__ const int32_t* pre_cnt() const { return w + w[12]; }
  __device__ __forceinline__ const int32_t* post_begin() const { return w + w[13]; }
  __device__ __forceinline__ const int32_t* post_cnt() const { return w + w[14]; }
  __device__ __forceinline__ const int32_t* src_rows() const { return w + w[17]; }   // fp8 cache only
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace heatkv
