// Cache update kernels (Sec. 3.3): append of a new scale's K/V into the rows the plan
// assigns, and the in-place left compaction of the ragged layout after an eviction.
// Both are pure byte movers: 16-byte vector loads and stores, rows copied verbatim.
// For the fp8 cache: the quantising append and the expansion of the visible rows into bf16 staging rows.
#include <cuda_fp16.h>

#include "append_device.cuh"

namespace heatkv {

constexpr int CP_THREADS = 128;

// ---------------------------------------------------------------- append
// grid = (destination half-tile, head, sequence).  Destination half-tile j of a storing head
// receives the next n_valid tokens of the step's K and V.
__global__ void __launch_bounds__(CP_THREADS) append_kernel(const __grid_constant__ CopyParams p) {
  const int seq = blockIdx.z, head = blockIdx.y, j = blockIdx.x;
  const int u = (p.step * p.L + p.layer) * p.H + head;
  const int64_t src = seq * p.kv_seq + head * p.kv_head;
  append_half_tile(p.seqs[seq].plan, p.seqs[seq].base_row, u, j, p.k_new + src, p.v_new + src, p.kv_tok, p.k_pool,
                   p.v_pool, p.d, threadIdx.x, CP_THREADS);
}

// ---------------------------------------------------------------- in-place compaction
// grid = (64-byte column slice, head * 2 + {K,V}, sequence * n_layers + layer).  One CTA walks the
// head's moves in order; every move goes left (dst < src) and may overlap itself, so a chunk
// is read completely (barrier) before it is written.  Later chunks never read what an earlier
// chunk wrote, because destinations stay below the sources still to be read.
constexpr int CM_ROWS = 128;       // rows per chunk: 128 rows x 64 B = 8 KB in registers per CTA

__global__ void __launch_bounds__(CP_THREADS) compact_kernel(const __grid_constant__ CopyParams p) {
  const int slice = blockIdx.x;
  const int head = blockIdx.y >> 1;
  const bool is_v = blockIdx.y & 1;
  const int seq = blockIdx.z / p.n_layers;
  const int layer = p.layer_begin + blockIdx.z % p.n_layers;
  PlanView pv(p.seqs[seq].plan);
  const int u = (p.step * p.L + layer) * p.H + head;
  const int cnt = p.phase == 0 ? pv.pre_cnt()[u] : pv.post_cnt()[u];
  if (cnt == 0) return;
  const int4* moves = pv.moves() + (p.phase == 0 ? pv.pre_begin()[u] : pv.post_begin()[u]);
  __nv_bfloat16* pool = is_v ? p.v_pool : p.k_pool;
  const int64_t base_row = p.seqs[seq].base_row;
  const int col = slice * 32;                            // 32 bf16 = 64 bytes per slice
  // thread -> (row within chunk, 16-byte piece of the slice)
  const int piece = threadIdx.x & 3;
  const int r_in = threadIdx.x >> 2;                     // 0..31
  for (int m = 0; m < cnt; ++m) {
    const int4 mv = moves[m];                            // src, dst, n
    for (int r0 = 0; r0 < mv.z; r0 += CM_ROWS) {
      int4 buf[CM_ROWS / 32];
#pragma unroll
      for (int q = 0; q < CM_ROWS / 32; ++q) {
        int r = r0 + q * 32 + r_in;
        if (r < mv.z)
          buf[q] = *reinterpret_cast<const int4*>(pool + (base_row + mv.x + r) * p.d + col + piece * 8);
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < CM_ROWS / 32; ++q) {
        int r = r0 + q * 32 + r_in;
        if (r < mv.z)
          *reinterpret_cast<int4*>(pool + (base_row + mv.y + r) * p.d + col + piece * 8) = buf[q];
      }
    }
  }
}

// ---------------------------------------------------------------- fp8 cache (conversions: append_device.cuh)
// grid = (destination half-tile, head, sequence), as append_kernel.
__global__ void __launch_bounds__(CP_THREADS) append_fp8_kernel(const __grid_constant__ CopyParams p) {
  const int seq = blockIdx.z, head = blockIdx.y, j = blockIdx.x;
  const int u = (p.step * p.L + p.layer) * p.H + head;
  const int64_t src = seq * p.kv_seq + head * p.kv_head;
  append_half_tile_fp8(p.seqs[seq].plan, p.seqs[seq].base_row, u, j, p.k_new + src, p.v_new + src, p.kv_tok, p.k8_pool,
                       p.v8_pool, p.k_exp, p.v_exp, p.d, threadIdx.x, CP_THREADS);
}

// Expansion of the visible head-scales of one (step, layer) into the bf16 staging rows the attention kernels
// read: grid = (visible half-tile of the layer in descriptor order, sequence, K | V).  Staging slot j of the
// sequence takes the n_valid rows behind descriptor first + j; rows past n_valid keep whatever finite values
// an earlier call left there (the kernels mask them).
__global__ void __launch_bounds__(CP_THREADS) dequant_fp8_kernel(const __grid_constant__ CopyParams p) {
  const int seq = blockIdx.y, j = blockIdx.x;
  const bool is_v = blockIdx.z != 0;
  PlanView pv(p.seqs[seq].plan);
  const int u0 = (p.step * p.L + p.layer) * p.H;
  const int first = pv.attn_begin()[u0];
  const int count = pv.attn_begin()[u0 + p.H - 1] + pv.attn_cnt()[u0 + p.H - 1] - first;
  if (j >= count) return;
  const int n = pv.descs()[first + j].y & 0xff;
  const int64_t src_row = p.seqs[seq].base_row + pv.src_rows()[first + j];
  const int64_t dst_row = (int64_t)p.stage_base[seq] + (int64_t)j * HEATKV_PAGE_TOKENS;
  const uint8_t* codes = (is_v ? p.v8_pool : p.k8_pool) + src_row * p.d;
  const int8_t* exps = (is_v ? p.v_exp : p.k_exp) + src_row;
  __nv_bfloat16* dst = (is_v ? p.v_pool : p.k_pool) + dst_row * p.d;
  const int ch_per_row = p.d / 8;
  for (int i = threadIdx.x; i < n * ch_per_row; i += CP_THREADS) {
    const int r = i / ch_per_row, ch = i % ch_per_row;
    const uint2 c = __ldg(reinterpret_cast<const uint2*>(codes + (int64_t)r * p.d + ch * 8));
    const float scale = pow2f((int)exps[r]);
    const uint32_t w[4] = {c.x & 0xffffu, c.x >> 16, c.y & 0xffffu, c.y >> 16};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float lo, hi;
      from_e4m3x2(w[q], lo, hi);
      o[q] = pack_bf16(lo * scale, hi * scale);          // exact: at most four significant bits times a power of two
    }
    *reinterpret_cast<int4*>(dst + (int64_t)r * p.d + ch * 8) = make_int4((int)o[0], (int)o[1], (int)o[2], (int)o[3]);
  }
}

cudaError_t launch_append_fp8(const CopyParams& p, int n_seq, cudaStream_t stream) {
  dim3 grid((p.t_k + HEATKV_PAGE_TOKENS - 1) / HEATKV_PAGE_TOKENS + 1, p.H, n_seq);
  append_fp8_kernel<<<grid, CP_THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

// `slots` = the largest number of visible half-tiles any sequence of the call has at (step, layer)
cudaError_t launch_dequant_fp8(const CopyParams& p, int n_seq, int slots, cudaStream_t stream) {
  if (slots < 1) return cudaSuccess;
  dim3 grid(slots, n_seq, 2);
  dequant_fp8_kernel<<<grid, CP_THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append(const CopyParams& p, int n_seq, cudaStream_t stream) {
  dim3 grid((p.t_k + HEATKV_PAGE_TOKENS - 1) / HEATKV_PAGE_TOKENS + 1, p.H, n_seq);
  append_kernel<<<grid, CP_THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_compact(const CopyParams& p, int n_seq, cudaStream_t stream) {
  dim3 grid(p.d / 32, p.H * 2, n_seq * p.n_layers);
  compact_kernel<<<grid, CP_THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace heatkv
