// Cache update kernels (Sec. 3.3): append of a new scale's K/V into the rows the plan
// assigns, and the in-place left compaction of the ragged layout after an eviction.
// Both are pure byte movers: 16-byte vector loads and stores, rows copied verbatim.
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
