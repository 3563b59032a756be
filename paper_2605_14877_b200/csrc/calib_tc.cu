// Tensor-memory calibration kernel (Sec. 3.1, Eq. 2) for the large scale steps (head_dim 128 or 64).
//
// beta[step][i] needs, for every query row of the step, the share of its softmax mass that falls on
// the keys of source scale i.  Only S = Q K^T is a contraction here: there is no PV product and no
// output, so the kernel is the attention kernel's front half with the per-scale bookkeeping fused into
// the softmax pass; the attention matrix is never written anywhere.
//
// One CTA owns 256 queries of one (sequence, head) as two 128-row tiles A and B.  Warp roles:
//   warp 0      TMA producer: Q tiles once, then K half-tiles (64 rows x 128 dims) of the full key set,
//               cut at source-scale borders (descriptor list built on the host), 3 stages.
//   warp 1      MMA issuer: S_x = Q_x K^T into TMEM as soon as the softmax warps have read the
//               previous S_x into registers (they say so right after the load, before the exponentials).
//   warps 4-11  tile A, warps 12-19 tile B: TWO threads per query row, one for keys 0..63 and one for keys
//               64..127 of every key tile (warps w and w + 4 share a TMEM lane quadrant).  Nothing here needs
//               a reference common to a row while the tiles stream by (there is no P to hand to a product),
//               so each thread keeps a running max, a sum and the mass of the scale it is inside of its own --
//               a half-tile lies inside one source scale -- parks finished scales in shared memory relative to
//               its own reference and rescales them when that moves (rare).  Four softmax warps per SM
//               sub-partition instead of two keep the exponential unit fed.
// At the end the two halves of every row are brought to a common reference, the row's masses are divided by
// its row sum, summed over the CTA's rows and added to beta with one atomicAdd per (CTA, source scale).  Every
// wait is bounded as in the attention kernel.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "internal.h"
#include "tc_common.cuh"

namespace heatkv {

namespace calib {

using namespace tc;

// (the shared-memory map is sized for 128-wide heads; 64-wide ones use half of each tile)
constexpr int BM = 128;                 // rows per Q tile
constexpr int BN = 128;                 // keys per tile (two 64-row half-tiles)
constexpr int HALF = 64;
constexpr int THREADS = 640;             // 4 utility warps + 16 softmax warps
constexpr int REGS_UTIL = 40, REGS_SOFTMAX = 104, REGS_LAUNCH = 96;   // ptxas assigns 96 under __launch_bounds__(640, 1)
static_assert(128 * REGS_UTIL + 512 * REGS_SOFTMAX <= THREADS * REGS_LAUNCH, "register hand-over exceeds the CTA's allocation");
constexpr int K_STAGES = 3;               // with the per-thread scale masses of two threads per row, four would not fit
constexpr uint32_t HALF_COLS_BYTES = 128 * 128;        // one 64-column half of a 128-row tile: 16 KB
constexpr uint32_t TILE_BYTES = 2 * HALF_COLS_BYTES;   // 32 KB
constexpr uint32_t SLOT_BYTES = HALF * 128;            // 64 rows x 128 B inside one column half

constexpr uint32_t SM_Q = 0;                                   // 2 tiles
constexpr uint32_t SM_K = SM_Q + 2 * TILE_BYTES;               // K_STAGES tiles
constexpr uint32_t SM_SEG = SM_K + K_STAGES * TILE_BYTES;      // float[2 tiles][2 key halves][16 scales][128 rows]
constexpr uint32_t SM_STAT = SM_SEG + 4 * HEATKV_MAX_K * BM * 4;  // float[2 tiles][2 key halves][2][128 rows]: reference, sum
constexpr uint32_t SM_ACC = SM_STAT + 4 * 2 * BM * 4;          // float[16]: the CTA's sums per scale
constexpr uint32_t SM_BAR = SM_ACC + HEATKV_MAX_K * 4;
constexpr uint32_t SM_TOTAL = SM_BAR + 256;
constexpr uint32_t SM_ALLOC = SM_TOTAL + 1024;                 // slack for manual alignment
static_assert(SM_ALLOC <= 227 * 1024, "shared memory of one CTA");

enum Bar : uint32_t {
  Q_FULL = 0,                   // +x (2)
  K_FULL = 2, K_EMPTY = 6,      // +stage (K_STAGES each, room for 4)
  S_FULL = 10,                  // +x  S_x of tile j is in TMEM
  S_READ = 12,                  // +x  the 128 rows of S_x of tile j are in registers (256 arrivals: two threads per row)
  N_BARS = 14
};
constexpr uint32_t SM_TMEM_PTR = SM_BAR + N_BARS * 8;
constexpr uint32_t SM_ABORT = SM_TMEM_PTR + 4;
constexpr uint32_t TMEM_COLS = 256;

struct Maps {
  CUtensorMap q, k;
};

// The steps one launch covers (one for heatkv_calibrate_scores, several for heatkv_calibrate_scores_steps): CTAs
// cta_begin[e] .. cta_begin[e + 1] - 1 belong to entry e, query tile pair fastest, then sequence, then head.
// Entries are ordered by descending work, so the long CTAs are dispatched first.
struct StepTable {
  int n;
  int cta_begin[HEATKV_MAX_K + 1];
  int step[HEATKV_MAX_K];
  int t_q[HEATKV_MAX_K];        // queries of the step
  int q_tok0[HEATKV_MAX_K];     // first query token of the step on the token axis of the q map
  int desc_first[HEATKV_MAX_K]; // the step's key half-tiles in the descriptor table
  int n_slots[HEATKV_MAX_K];
};

struct HalfTile {
  int row;          // first key row inside k_full
  int n_valid;      // real rows of the 64
  int seg;          // source scale
};

__device__ __forceinline__ HalfTile get_half(int i, const int2* descs, int n_slots) {
  const bool valid = i < n_slots;
  const int2 d = descs[valid ? i : n_slots - 1];     // padding half-tile: re-read finite data, mask everything
  HalfTile h;
  h.row = d.x;
  h.n_valid = valid ? (d.y & 0xff) : 0;
  h.seg = (d.y >> 8) & 0xff;
  return h;
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
calib_tc_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ Maps maps, const int2* __restrict__ all_descs,
                const __grid_constant__ StepTable tab, int n_seq, int64_t bias_step_stride) {
  static_assert(D == 64 || D == 128, "head dimension");
  constexpr int NCH = D / 64;                               // 64-column halves per row
  constexpr uint32_t LOAD_BYTES = NCH * HALF_COLS_BYTES;    // bytes one tile's copies deliver
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sbase = (raw + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - raw);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(sgen + SM_ABORT);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(sgen + SM_TMEM_PTR);
  float* acc_smem = reinterpret_cast<float*>(sgen + SM_ACC);
  auto bar = [&](uint32_t which) { return sbase + SM_BAR + which * 8; };

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  int e = 0;
  while (e + 1 < tab.n && (int)blockIdx.x >= tab.cta_begin[e + 1]) ++e;
  const int step = tab.step[e], t_q = tab.t_q[e], n_slots = tab.n_slots[e];
  const int2* descs = all_descs + tab.desc_first[e];
  const int n_qp = (t_q + 2 * BM - 1) / (2 * BM);
  const int local = (int)blockIdx.x - tab.cta_begin[e];
  const int seq = (local / n_qp) % n_seq, head = local / (n_qp * n_seq);
  const int q0 = (local % n_qp) * (2 * BM);             // first query of the CTA inside its step
  const int q_tok = tab.q_tok0[e] + q0;                 // ... and on the token axis of the q map
  const int nq = (q0 + BM < t_q) ? 2 : 1;               // does tile B hold any query?
  const int n_tiles = (n_slots + 1) / 2;

  if (threadIdx.x == 0) {
    *abort_flag = *reinterpret_cast<volatile uint32_t*>(p.status) != 0;   // an earlier CTA gave up: do not wait again
    for (int i = 0; i < HEATKV_MAX_K; ++i) acc_smem[i] = 0.f;
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(Q_FULL + x), 1);
      mbar_init(bar(S_FULL + x), 1);
      mbar_init(bar(S_READ + x), 2 * BM);
    }
    for (int s = 0; s < K_STAGES; ++s) {
      mbar_init(bar(K_FULL + s), 1);
      mbar_init(bar(K_EMPTY + s), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + SM_TMEM_PTR), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_ptr_smem;

  // register budget per warpgroup: 128*40 + 512*104 <= 640*96
  if (warp < 4) {
    reg_dealloc<REGS_UTIL>();
    if (warp == 0) {
      // ------------------------------------------------------------------ TMA producer
      const bool leader = elect_one();
      uint32_t armed = 0;                               // stage -> a copy was issued at least once
      uint32_t par[K_STAGES] = {};
      if (leader) {
        for (int x = 0; x < nq; ++x) {
          mbar_expect_tx(bar(Q_FULL + x), LOAD_BYTES);
          for (int ch = 0; ch < NCH; ++ch)
            for (int hf = 0; hf < 2; ++hf)
              tma_load_4d(sbase + SM_Q + x * TILE_BYTES + ch * HALF_COLS_BYTES + hf * SLOT_BYTES, &maps.q, ch * 64,
                          q_tok + x * BM + hf * HALF, head, seq, bar(Q_FULL + x));
        }
      }
      bool ok = true;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j % K_STAGES;
        const uint32_t use = (uint32_t)(j / K_STAGES);
        const HalfTile h0 = get_half(2 * j, descs, n_slots), h1 = get_half(2 * j + 1, descs, n_slots);
        if (use > 0) ok = warp_wait(bar(K_EMPTY + st), (use - 1) & 1, abort_flag, p.status);
        if (!ok) break;
        armed |= 1u << st;
        par[st] = use & 1;
        if (leader) {
          mbar_expect_tx(bar(K_FULL + st), LOAD_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            for (int ch = 0; ch < NCH; ++ch)
              tma_load_4d(sbase + SM_K + st * TILE_BYTES + ch * HALF_COLS_BYTES + hf * SLOT_BYTES, &maps.k, ch * 64,
                          hf == 0 ? h0.row : h1.row, head, seq, bar(K_FULL + st));
        }
        __syncwarp();
      }
      if (!ok) {
        // leaving early: let every copy this warp started land before the CTA exits
        for (int s = 0; s < K_STAGES; ++s)
          if (armed & (1u << s))
            for (uint32_t it = 0; it < WAIT_LIMIT && !mbar_try(bar(K_FULL + s), par[s]); ++it) {}
        for (int x = 0; x < nq; ++x)
          for (uint32_t it = 0; it < WAIT_LIMIT && !mbar_try(bar(Q_FULL + x), 0); ++it) {}
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------------ MMA issuer
      const bool leader = elect_one();
      constexpr uint32_t IDESC_S = instr_desc(BM, BN, 0, 0);     // Q, K both K-major
      bool ok = true;
      for (int x = 0; x < nq && ok; ++x) ok = warp_wait(bar(Q_FULL + x), 0, abort_flag, p.status);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j % K_STAGES;
        ok = warp_wait(bar(K_FULL + st), (uint32_t)(j / K_STAGES) & 1, abort_flag, p.status);
        for (int x = 0; x < nq && ok; ++x) {
          if (j > 0) ok = warp_wait(bar(S_READ + x), (j - 1) & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          if (leader) {
            const uint32_t qa = sbase + SM_Q + x * TILE_BYTES, ka = sbase + SM_K + st * TILE_BYTES;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint32_t off = (ks >> 2) * HALF_COLS_BYTES + (ks & 3) * 32;
              mma_ss(tmem + x * 128, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024), IDESC_S, ks > 0);
            }
            tc_commit(bar(S_FULL + x));
          }
          __syncwarp();
        }
        if (ok && leader) tc_commit(bar(K_EMPTY + st));
        __syncwarp();
      }
    }
  } else {
    reg_alloc<REGS_SOFTMAX>();
    // ------------------------------------------------------------------ softmax with per-scale masses
    const int x = (warp - 4) >> 3;                      // 0: tile A (warps 4-11), 1: tile B (warps 12-19)
    const int g = ((warp - 4) >> 2) & 1;                // which 64 keys of every key tile
    const int row = (warp & 3) * 32 + lane;             // row inside the tile == TMEM lane
    float* seg_smem = reinterpret_cast<float*>(sgen + SM_SEG) + (x * 2 + g) * (HEATKV_MAX_K * BM);   // [scale][row]
    float* stat_smem = reinterpret_cast<float*>(sgen + SM_STAT) + (x * 2 + g) * (2 * BM);           // [reference | sum][row]
    float m_ref = -INFINITY, l_sum = 0.f;
    int cur_seg = -1;                                   // the scale whose mass is being collected (warp-uniform)
    float cur_sum = 0.f;
    bool ok = true;
    if (x < nq) {
      const uint32_t t_s = tmem + ((uint32_t)((warp & 3) * 32) << 16) + x * 128 + g * 64;
      const float* bias_h = p.seg_bias ? p.seg_bias + step * bias_step_stride + head * p.K : nullptr;
      const float LOG2E = 1.4426950408889634f;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const HalfTile sg = get_half(2 * j + g, descs, n_slots);
        const float bg = bias_h ? bias_h[sg.seg] * LOG2E : 0.f;
        ok = __all_sync(0xffffffffu, mbar_wait_hint(bar(S_FULL + x), j & 1, abort_flag, p.status));
        if (!ok) break;
        tc_fence_after();
        uint32_t r0[32], r1[32];
        tmem_ld32(t_s, r0);
        tmem_ld32(t_s + 32, r1);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(S_READ + x));                   // the next S_x may overwrite these columns
        if (sg.n_valid == 0) continue;                  // padding half-tile (warp-uniform): nothing to add
        if (sg.n_valid < HALF) {                        // ragged half-tile (warp-uniform): mask by -inf
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (i >= sg.n_valid) r0[i] = 0xff800000u;
            if (i + 32 >= sg.n_valid) r1[i] = 0xff800000u;
          }
        }
        // maximum of the 64 logits: the logit is raw * scale + bias(half) with scale > 0, so take the raw maximum
        float mq[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) mq[c] = fmaxf(__uint_as_float(r0[c]), __uint_as_float(r1[c]));
#pragma unroll
        for (int i = 4; i < 32; i += 4) {
#pragma unroll
          for (int c = 0; c < 4; ++c) mq[c] = fmax3(mq[c], __uint_as_float(r0[i + c]), __uint_as_float(r1[i + c]));
        }
        const float mx = fmaf(fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3])), p.scale_log2, bg);
        const float m_new = fmaxf(m_ref, mx);
        const bool grow = m_new > m_ref + RESCALE_THRESHOLD;   // also true on the first tile (m_ref = -inf)
        if (grow) {
          if (m_ref > -INFINITY) {
            // everything collected so far is relative to m_ref: move it to the new reference
            const float f = exp2f(m_ref - m_new);
            l_sum *= f;
            cur_sum *= f;
            for (int s = 0; s < cur_seg; ++s) seg_smem[s * BM + row] *= f;
          }
          m_ref = m_new;
        }
        __syncwarp();
        const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2);
        const uint64_t bb = pack2(bg - m_ref, bg - m_ref);
        uint64_t sum_a = pack2(0.f, 0.f), sum_b = pack2(0.f, 0.f);
        auto exp_sum = [&](const uint32_t (&rc)[32], uint64_t& sum2) {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const uint64_t xx = fma2(pack2(__uint_as_float(rc[i]), __uint_as_float(rc[i + 1])), scale2, bb);
            float e0, e1;
            if (((i >> 1) % 3) == 2) {                  // one pair in three on the FMA pipe (measured best for this kernel)
              exp2_poly2(xx, e0, e1);
            } else {
              float x0, x1;
              unpack2(xx, x0, x1);
              e0 = ex2_approx(x0);
              e1 = ex2_approx(x1);
            }
            sum2 = add2(sum2, pack2(e0, e1));
          }
        };
        exp_sum(r0, sum_a);
        exp_sum(r1, sum_b);
        float a0, a1, c0, c1;
        unpack2(sum_a, a0, a1);
        unpack2(sum_b, c0, c1);
        const float h = (a0 + a1) + (c0 + c1);
        l_sum += h;
        // source scales arrive in ascending order, each as one run of half-tiles
        if (sg.seg != cur_seg) {
          if (cur_seg >= 0) seg_smem[cur_seg * BM + row] = cur_sum;
          // scales this thread never sees between the two (their half-tiles all went to the partner) stay zero
          for (int s = cur_seg + 1; s < sg.seg; ++s) seg_smem[s * BM + row] = 0.f;
          cur_seg = sg.seg;
          cur_sum = 0.f;
        }
        cur_sum += h;
      }
      if (ok) {
        if (cur_seg >= 0) seg_smem[cur_seg * BM + row] = cur_sum;
        for (int s = cur_seg + 1; s <= step; ++s) seg_smem[s * BM + row] = 0.f;
        stat_smem[row] = m_ref;
        stat_smem[BM + row] = l_sum;
      }
    }
  }

  // ---- the two halves of every row meet: thread (row, keys 0..63) brings both to a common reference
  tc_fence_before();
  __syncthreads();
  if (warp >= 4 && ((warp - 4) >> 2 & 1) == 0 && *abort_flag == 0) {
    const int x = (warp - 4) >> 3;
    if (x < nq) {
      const int row = (warp & 3) * 32 + lane;
      const float* seg0 = reinterpret_cast<const float*>(sgen + SM_SEG) + (x * 2) * (HEATKV_MAX_K * BM);
      const float* seg1 = seg0 + HEATKV_MAX_K * BM;
      const float* st0 = reinterpret_cast<const float*>(sgen + SM_STAT) + (x * 2) * (2 * BM);
      const float* st1 = st0 + 2 * BM;
      // Eq. 2: mean over the step's rows of mass(row, scale) / rowsum(row); rows past t_q are padding.  A thread
      // that saw no valid key keeps the reference -inf and contributes nothing.
      const float m0 = st0[row], m1 = st1[row];
      const float m = fmaxf(m0, m1);
      const float w0 = m0 > -INFINITY ? exp2f(m0 - m) : 0.f, w1 = m1 > -INFINITY ? exp2f(m1 - m) : 0.f;
      const float l = st0[BM + row] * w0 + st1[BM + row] * w1;
      const bool live = q0 + x * BM + row < t_q;
      const float inv = live ? 1.f / l : 0.f;
      for (int s = 0; s <= step; ++s) {
        float v = live ? (seg0[s * BM + row] * w0 + seg1[s * BM + row] * w1) * inv : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) atomicAdd(acc_smem + s, v);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  // p.beta_row is beta_accum[layer][0][0]: the row of (head, step) follows
  if ((int)threadIdx.x <= step && *abort_flag == 0)
    atomicAdd(p.beta_row + ((int64_t)head * p.K + step) * p.K + threadIdx.x, acc_smem[threadIdx.x] / (float)t_q);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace calib

// ---------------------------------------------------------------------------------- host side
struct CalibTcState {
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  std::vector<int2> host_descs;          // all steps, concatenated (kept alive for the upload)
  std::vector<int> first, count;         // per step
  const int2* dev_descs = nullptr;
  int d = 0;                             // head dimension of the context (64 or 128)
  bool ready = false;
};

uint64_t calib_tc_desc_bytes(const heatkv_config& cfg) {
  uint64_t n = 0;
  for (int step = 0; step < cfg.K; ++step)
    for (int i = 0; i <= step; ++i) n += (uint64_t)(cfg.t[i] + calib::HALF - 1) / calib::HALF;
  return n * sizeof(int2);
}

// `dev_table` is device memory of calib_tc_desc_bytes(cfg) bytes inside the context's metadata region.
int calib_tc_create(const heatkv_config& cfg, void* dev_table, cudaStream_t stream, CalibTcState** out) {
  *out = nullptr;
  CalibTcState* st = new (std::nothrow) CalibTcState;
  if (!st) return HEATKV_ERR_HOST_MEMORY;
  *out = st;
  if ((cfg.d != 64 && cfg.d != 128) || !dev_table) return HEATKV_OK;   // other head dimensions: generic kernel only
  st->d = cfg.d;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    return HEATKV_OK;
  }
  st->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  try {
    for (int step = 0; step < cfg.K; ++step) {
      st->first.push_back((int)st->host_descs.size());
      int row0 = 0;
      for (int i = 0; i <= step; ++i) {
        for (int off = 0; off < cfg.t[i]; off += calib::HALF) {
          int n = cfg.t[i] - off < calib::HALF ? cfg.t[i] - off : calib::HALF;
          st->host_descs.push_back(make_int2(row0 + off, n | (i << 8)));
        }
        row0 += cfg.t[i];
      }
      st->count.push_back((int)st->host_descs.size() - st->first.back());
    }
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (cudaMemcpyAsync(dev_table, st->host_descs.data(), st->host_descs.size() * sizeof(int2), cudaMemcpyHostToDevice,
                      stream) != cudaSuccess)
    return HEATKV_ERR_CUDA;
  // later calls may come on other streams: the table must be in place before create returns
  if (cudaStreamSynchronize(stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  st->dev_descs = static_cast<const int2*>(dev_table);
  const void* kern = cfg.d == 128 ? (const void*)calib::calib_tc_kernel<128> : (const void*)calib::calib_tc_kernel<64>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)calib::SM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    return HEATKV_OK;
  }
  cudaFuncAttributes attr;
  if (cudaFuncGetAttributes(&attr, kern) != cudaSuccess) {
    cudaGetLastError();
    return HEATKV_OK;
  }
  // the register hand-over inside the kernel must fit in what the launch really allocates
  if (attr.numRegs * calib::THREADS < 128 * calib::REGS_UTIL + 512 * calib::REGS_SOFTMAX) return HEATKV_ERR_CUDA;
  st->ready = true;
  return HEATKV_OK;
}

void calib_tc_destroy(CalibTcState* st) { delete st; }

bool calib_tc_ready(const CalibTcState* st) { return st && st->ready; }

bool calib_tc_supported(const CalibTcState* st, const AttnParams& p, int d, int n_seq) {
  if (!st || !st->ready || d != st->d || n_seq > 65535 || p.H > 65535) return false;
  const int64_t s[6] = {p.q_seq, p.q_head, p.q_tok, p.kv_seq, p.kv_head, p.kv_tok};
  for (int64_t v : s)
    if (v & 7) return false;
  return true;
}

namespace {
bool encode_4d(CalibTcState* st, CUtensorMap* m, const void* base, int t, int H, int n_seq, int64_t s_tok, int64_t s_head,
               int64_t s_seq) {
  cuuint64_t dims[4] = {(cuuint64_t)st->d, (cuuint64_t)t, (cuuint64_t)H, (cuuint64_t)n_seq};
  auto fix = [](int64_t s) { return (cuuint64_t)((s > 0 ? s : 8) * 2); };
  cuuint64_t strides[3] = {fix(s_tok), fix(s_head), fix(s_seq)};
  cuuint32_t box[4] = {64, (cuuint32_t)calib::HALF, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return st->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

// One launch for the given steps of one layer.  `p` carries the common fields: q = the queries at token 0 of the
// q map (`q_tokens` tokens per head), k_new = the keys (`k_tokens` per head), strides, H, K, seg_bias (of step 0
// when `bias_step_stride` != 0, else of the one step), beta_row = beta_accum[layer][0][0].  `q_tok0[i]` is the first
// query token of steps[i] on the q map's token axis.
cudaError_t launch_calib_tc_steps(CalibTcState* st, const AttnParams& p, int n_seq, const int* steps, const int* t_q,
                                  const int* q_tok0, int n_steps, int q_tokens, int k_tokens, int64_t bias_step_stride,
                                  cudaStream_t stream) {
  if (n_steps < 1 || n_steps > HEATKV_MAX_K) return cudaErrorInvalidValue;
  calib::Maps maps;
  if (!encode_4d(st, &maps.q, p.q, q_tokens, p.H, n_seq, p.q_tok, p.q_head, p.q_seq) ||
      !encode_4d(st, &maps.k, p.k_new, k_tokens, p.H, n_seq, p.kv_tok, p.kv_head, p.kv_seq))
    return cudaErrorInvalidValue;
  // longest CTAs first: entries by descending key half-tiles (the CTAs of one step are all alike)
  int order[HEATKV_MAX_K];
  for (int i = 0; i < n_steps; ++i) order[i] = i;
  std::sort(order, order + n_steps, [&](int a, int b) { return st->count[steps[a]] > st->count[steps[b]]; });
  calib::StepTable tab;
  std::memset(&tab, 0, sizeof(tab));
  tab.n = n_steps;
  int ctas = 0;
  for (int e = 0; e < n_steps; ++e) {
    const int i = order[e];
    tab.cta_begin[e] = ctas;
    tab.step[e] = steps[i];
    tab.t_q[e] = t_q[i];
    tab.q_tok0[e] = q_tok0[i];
    tab.desc_first[e] = st->first[steps[i]];
    tab.n_slots[e] = st->count[steps[i]];
    ctas += (t_q[i] + 2 * calib::BM - 1) / (2 * calib::BM) * n_seq * p.H;
  }
  tab.cta_begin[n_steps] = ctas;
  dim3 grid((unsigned)ctas);
  if (st->d == 128)
    calib::calib_tc_kernel<128><<<grid, calib::THREADS, calib::SM_ALLOC, stream>>>(p, maps, st->dev_descs, tab, n_seq, bias_step_stride);
  else
    calib::calib_tc_kernel<64><<<grid, calib::THREADS, calib::SM_ALLOC, stream>>>(p, maps, st->dev_descs, tab, n_seq, bias_step_stride);
  return cudaGetLastError();
}

// One step: p.q = the step's queries, p.t_q of them; p.k_new = all p.n_own keys; p.beta_row = beta_accum[layer][0][step]
// as the generic kernel takes it.
cudaError_t launch_calib_tc(CalibTcState* st, const AttnParams& p, int n_seq, cudaStream_t stream) {
  AttnParams q = p;
  q.beta_row = p.beta_row - (int64_t)p.step * p.K;       // back to beta_accum[layer][0][0]
  const int step = p.step, t_q = p.t_q, tok0 = 0;
  return launch_calib_tc_steps(st, q, n_seq, &step, &t_q, &tok0, 1, p.t_q, p.n_own, 0, stream);
}

}  // namespace heatkv
