// Generic ragged attention kernel (warp-level MMA, online softmax), used for the small,
// bandwidth / latency bound scale steps and for calibration.
//
// One CTA = 64 queries of one (sequence, head); 4 warps x 16 query rows.  Keys arrive as a
// sequence of half-tiles of up to 64 rows: first the head's retained prior keys, listed by
// the plan's page table (Sec. 3.3: the head-scales not in A_k), then the step's own keys
// from k_new.  In calibration mode (Eq. 2) every key comes from k_full and the per-row
// probability mass of every source scale is accumulated next to the online softmax, so the
// attention matrix alpha is never formed.
#include <atomic>
#include "append_device.cuh"

namespace heatkv {

constexpr int GM = 64;    // queries per CTA
constexpr int GN = 64;    // keys per half-tile
constexpr int GTHREADS = 128;
constexpr int GSTAGES = 2;   // key/value half-tiles in flight or in use per CTA (3 measured no faster: the small steps are bound by the warp-level MMA rate)

template <int D>
struct GenericSmem {
  static constexpr int TILE_BYTES = GN * D * 2;
  // q | k[GSTAGES] | v[GSTAGES] | seg_sum[GM][16] | seg_ref[GM][16]
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = GM * D * 2;
  static constexpr int V_OFF = K_OFF + GSTAGES * TILE_BYTES;
  static constexpr int SEG_OFF = V_OFF + GSTAGES * TILE_BYTES;
  static constexpr int BYTES = SEG_OFF + 2 * GM * HEATKV_MAX_K * 4;
  static constexpr int ATTN_BYTES = SEG_OFF;             // without the calibration sums: two CTAs of head_dim 128 fit an SM
};

// byte offset of 16-byte chunk `ch` of row `r` in a [rows][D] bf16 tile (XOR swizzle)
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int ch) {
  return (uint32_t)((r * (D / 8) + (ch ^ (r & 7))) * 16);
}

// copies `rows` rows (row-major, D bf16 each, `stride` elements apart) into a swizzled tile;
// rows >= n_valid are zero-filled.
template <int D>
__device__ __forceinline__ void load_tile(uint32_t smem_base, const __nv_bfloat16* src, int64_t stride,
                                          int n_valid, int tid) {
  constexpr int CH = D / 8;
  constexpr int ROWS_PER_PASS = GTHREADS / CH;
  const int ch = tid % CH;
  const int r0 = tid / CH;
#pragma unroll
  for (int r = r0; r < GN; r += ROWS_PER_PASS) {
    const bool ok = r < n_valid;
    const __nv_bfloat16* p = ok ? src + (int64_t)r * stride + ch * 8 : src;
    cp_async16(smem_base + tile_off<D>(r, ch), p, ok ? 16 : 0);
  }
}

// Scratch of heatkv_calibrate_scores_static: one partial mass per (CTA, warp, source scale).  It lives in
// the library image, so that entry point needs no allocation; every GPU that loads the library holds
// these 4 MiB until the process exits.
constexpr int STATIC_PARTIAL_FLOATS = 1 << 20;
static __device__ __align__(256) float g_static_partials[STATIC_PARTIAL_FLOATS];

template <int D, bool CALIB, bool PARTIALS = false>
__global__ void __launch_bounds__(GTHREADS, 2) attn_generic_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  using SM = GenericSmem<D>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, qd = lane & 3;
  // attention: grid = (query tiles, sequences, heads by descending key count), so the heaviest heads of
  // every sequence are dispatched first; calibration: grid = (query tiles, heads, sequences)
  if (!CALIB && (int)blockIdx.x >= (p.t_q + GM - 1) / GM) {
    // cache update riding on this launch: one CTA per (destination half-tile, sequence, head)
    const int sq = blockIdx.y, hd = blockIdx.z, j = blockIdx.x - (p.t_q + GM - 1) / GM;
    const int64_t src = sq * p.kv_seq + hd * p.kv_head;
    if (p.k8_pool)
      append_half_tile_fp8(p.seqs[sq].plan, p.pool_base[sq], (p.step * p.L + p.layer) * p.H + hd, j, p.k_new + src,
                           p.v_new + src, p.kv_tok, p.k8_pool, p.v8_pool, p.k_exp, p.v_exp, D, threadIdx.x, GTHREADS);
    else
      append_half_tile(p.seqs[sq].plan, p.seqs[sq].base_row, (p.step * p.L + p.layer) * p.H + hd, j, p.k_new + src,
                       p.v_new + src, p.kv_tok, const_cast<__nv_bfloat16*>(p.k_pool), const_cast<__nv_bfloat16*>(p.v_pool),
                       D, threadIdx.x, GTHREADS);
    return;
  }
  const int seq = CALIB ? blockIdx.z : blockIdx.y;
  int head = CALIB ? blockIdx.y : blockIdx.z;
  // What a CTA works on comes from the launch parameters; a calibration launch may cover several steps
  // (heatkv_calibrate_scores_steps), its query tiles laid side by side along grid.x.
  int t_q = p.t_q, n_own = p.n_own, step = p.step, q0 = blockIdx.x * GM;
  const __nv_bfloat16* q_base = p.q;
  float* beta_row = p.beta_row;
  const float* seg_bias = p.seg_bias;
  if (CALIB && p.cal_n > 0) {
    int e = 0;
    while (e + 1 < p.cal_n && (int)blockIdx.x >= p.cal_tile_begin[e + 1]) ++e;
    step = p.cal_step[e];
    n_own = p.c[step];
    t_q = n_own - (step > 0 ? p.c[step - 1] : 0);
    q0 = ((int)blockIdx.x - p.cal_tile_begin[e]) * GM;
    q_base = p.q + (int64_t)(n_own - t_q) * p.q_tok;        // the step's queries on the token axis of all scales
    beta_row = p.beta_row + (int64_t)step * p.K;              // p.beta_row is beta_accum[layer][0][0] here
    if (seg_bias) seg_bias += (int64_t)step * p.cal_bias_stride;
  }

  const int2* descs = nullptr;
  int n_desc = 0;
  int64_t base_row = 0;
  if (!CALIB) {
    if (p.table_heads > 0) {
      // one schedule for the whole call: the host listed, per head in dispatch order, where its descriptors
      // start, so the first key tile is two dependent loads away instead of four
      head = p.table_head[blockIdx.z];
      descs = reinterpret_cast<const int2*>(p.seqs[seq].plan + p.table_desc_begin[blockIdx.z]);
      n_desc = p.table_ndesc[blockIdx.z];
    } else {
      PlanView pv(p.seqs[seq].plan);
      const int u = (p.step * p.L + p.layer) * p.H;
      head = pv.order()[u + blockIdx.z];                   // heavy heads first
      descs = pv.descs() + pv.attn_begin()[u + head];
      n_desc = pv.attn_cnt()[u + head];
    }
    base_row = p.seqs[seq].base_row;
  }
  const int n_own_tiles = (n_own + GN - 1) / GN;
  const int n_tiles = n_desc + n_own_tiles;

  const uint32_t sbase = smem_u32(smem);
  float* seg_sum = reinterpret_cast<float*>(smem + SM::SEG_OFF);
  float* seg_ref = seg_sum + GM * HEATKV_MAX_K;

  const __nv_bfloat16* kown = p.k_new + seq * p.kv_seq + head * p.kv_head;
  const __nv_bfloat16* vown = p.v_new ? p.v_new + seq * p.kv_seq + head * p.kv_head : nullptr;

  // descriptors are fetched one tile ahead of the copy they steer: `dsc_next` belongs to the tile issued next
  int2 dsc_next = n_desc > 0 ? descs[0] : make_int2(0, 0);
  auto issue_tile = [&](int j, int stage) {
    const __nv_bfloat16 *ks, *vs;
    int64_t stride;
    int nv;
    if (j < n_desc) {
      int2 dsc = dsc_next;
      int64_t row = base_row + dsc.x;
      ks = p.k_pool + row * D;
      vs = p.v_pool + row * D;
      stride = D;
      nv = dsc.y & 0xff;
    } else {
      int jj = j - n_desc;
      ks = kown + (int64_t)jj * GN * p.kv_tok;
      vs = vown ? vown + (int64_t)jj * GN * p.kv_tok : nullptr;
      stride = p.kv_tok;
      nv = min(GN, n_own - jj * GN);
    }
    load_tile<D>(sbase + SM::K_OFF + stage * SM::TILE_BYTES, ks, stride, nv, tid);
    if (vs) load_tile<D>(sbase + SM::V_OFF + stage * SM::TILE_BYTES, vs, stride, nv, tid);
    if (j + 1 < n_desc) dsc_next = descs[j + 1];
  };

  // ---- prologue: Q tile and the first GSTAGES - 1 key tiles, one copy group each (empty groups keep the count)
  {
    const __nv_bfloat16* qsrc = q_base + seq * p.q_seq + head * p.q_head + (int64_t)q0 * p.q_tok;
    load_tile<D>(sbase + SM::Q_OFF, qsrc, p.q_tok, min(GM, t_q - q0), tid);
    cp_async_commit();
    for (int j = 0; j < GSTAGES - 1; ++j) {
      if (j < n_tiles) issue_tile(j, j);
      cp_async_commit();
    }
  }
  if (CALIB) {
    for (int i = tid; i < GM * HEATKV_MAX_K; i += GTHREADS) {
      seg_sum[i] = 0.f;
      seg_ref[i] = -INFINITY;
    }
  }
  cp_async_wait<GSTAGES - 1>();                        // Q has landed
  __syncthreads();

  uint32_t qf[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    int ch = ks * 2 + (lane >> 4);
    ldmatrix_x4(qf[ks], sbase + SM::Q_OFF + tile_off<D>(r, ch));
  }

  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};

  for (int j = 0; j < n_tiles; ++j) {
    const int stage = j % GSTAGES;
    cp_async_wait<GSTAGES - 2>();                      // all groups but the newest GSTAGES - 2: tile j is among them
    __syncthreads();                                   // tile j landed for everyone; everyone left tile j-1
    if (j + GSTAGES - 1 < n_tiles) issue_tile(j + GSTAGES - 1, (j + GSTAGES - 1) % GSTAGES);   // into tile j-1's stage
    cp_async_commit();

    // tile attributes (warp-uniform)
    int nv, seg_lo, seg_hi, col0 = 0;
    if (j < n_desc) {
      int2 dsc = descs[j];
      nv = dsc.y & 0xff;
      seg_lo = seg_hi = (dsc.y >> 8) & 0xff;
    } else {
      int jj = j - n_desc;
      nv = min(GN, n_own - jj * GN);
      col0 = jj * GN;
      seg_lo = seg_hi = step;
      if (CALIB) {
        seg_lo = 0;
        while (p.c[seg_lo] <= col0) ++seg_lo;
        seg_hi = seg_lo;
        while (p.c[seg_hi] < col0 + nv) ++seg_hi;
      }
    }

    // ---- S = Q K^T
    float s[GN / 8][4];
#pragma unroll
    for (int i = 0; i < GN / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
    const uint32_t kbase = sbase + SM::K_OFF + stage * SM::TILE_BYTES;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < GN / 16; ++np) {
        uint32_t b[4];
        int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
        int ch = ks * 2 + ((lane >> 3) & 1);
        ldmatrix_x4(b, kbase + tile_off<D>(r, ch));
        mma_bf16(s[2 * np], qf[ks], b[0], b[1]);
        mma_bf16(s[2 * np + 1], qf[ks], b[2], b[3]);
      }
    }

    // ---- scale, bias, mask, online softmax
    const float* bias_h = seg_bias ? seg_bias + head * p.K : nullptr;
    const float LOG2E = 1.4426950408889634f;
    float tile_bias = bias_h ? bias_h[seg_lo] * LOG2E : 0.f;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int n = 0; n < GN / 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int col = n * 8 + qd * 2 + (e & 1);
        float bias = tile_bias;
        if (CALIB && bias_h && seg_lo != seg_hi) {
          int sg = seg_lo;
          while (p.c[sg] <= col0 + col && sg < seg_hi) ++sg;
          bias = bias_h[sg] * LOG2E;
        }
        float v = col < nv ? fmaf(s[n][e], p.scale_log2, bias) : -INFINITY;
        s[n][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      float m_new = fmaxf(m_run[r], mx[r]);
      corr[r] = exp2f(m_run[r] - m_new);
      m_run[r] = m_new;
      l_run[r] *= corr[r];
    }
    float psum[2] = {0.f, 0.f};
#pragma unroll
    for (int n = 0; n < GN / 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float pv = exp2f(s[n][e] - m_run[e >> 1]);
        s[n][e] = pv;
        psum[e >> 1] += pv;
      }
    }
    l_run[0] += psum[0];
    l_run[1] += psum[1];

    if (CALIB) {
      // per-row mass of every source scale that intersects this tile, kept as (sum, reference max)
      for (int sg = seg_lo; sg <= seg_hi; ++sg) {
        const int lo = sg > 0 ? p.c[sg - 1] : 0, hi = p.c[sg];
        float part[2] = {0.f, 0.f};
#pragma unroll
        for (int n = 0; n < GN / 8; ++n) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            int col = col0 + n * 8 + qd * 2 + (e & 1);
            if (col >= lo && col < hi) part[e >> 1] += s[n][e];
          }
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          part[r] += __shfl_xor_sync(0xffffffffu, part[r], 1);
          part[r] += __shfl_xor_sync(0xffffffffu, part[r], 2);
          if (qd == 0) {
            int row = warp * 16 + g + r * 8;
            float old = seg_sum[row * HEATKV_MAX_K + sg];
            float ref = seg_ref[row * HEATKV_MAX_K + sg];
            seg_sum[row * HEATKV_MAX_K + sg] = old * exp2f(ref - m_run[r]) + part[r];
            seg_ref[row * HEATKV_MAX_K + sg] = m_run[r];
          }
        }
      }
    }

    // ---- O = O * corr + P V
    if (!CALIB || p.out) {
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        o[i][0] *= corr[0];
        o[i][1] *= corr[0];
        o[i][2] *= corr[1];
        o[i][3] *= corr[1];
      }
      const uint32_t vbase = sbase + SM::V_OFF + stage * SM::TILE_BYTES;
#pragma unroll
      for (int kk = 0; kk < GN / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
        pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
        pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int dp = 0; dp < D / 16; ++dp) {
          uint32_t b[4];
          int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          int ch = dp * 2 + (lane >> 4);
          ldmatrix_x4_trans(b, vbase + tile_off<D>(r, ch));
          mma_bf16(o[2 * dp], pa, b[0], b[1]);
          mma_bf16(o[2 * dp + 1], pa, b[2], b[3]);
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- epilogue
  float inv_l[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    float l = l_run[r];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    inv_l[r] = 1.f / l;
  }

  if (CALIB) {
    // beta[step][sg] += (1/t) * sum over rows of mass(row, sg) / l(row)     (Eq. 2)
    float* beta = beta_row + (int64_t)head * p.K * p.K;
    for (int sg = 0; sg <= step; ++sg) {
      float acc = 0.f;
      if (qd == 0) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          int row = warp * 16 + g + r * 8;
          if (q0 + row < t_q)
            acc += seg_sum[row * HEATKV_MAX_K + sg] * exp2f(seg_ref[row * HEATKV_MAX_K + sg] - m_run[r]) * inv_l[r];
        }
      }
      acc += __shfl_xor_sync(0xffffffffu, acc, 4);
      acc += __shfl_xor_sync(0xffffffffu, acc, 8);
      acc += __shfl_xor_sync(0xffffffffu, acc, 16);
      if (PARTIALS) {
        // slot of (CTA, warp, source scale); reduce_partials_kernel adds them up in a fixed order
        const int64_t cta = blockIdx.x + (int64_t)gridDim.x * (blockIdx.y + (int64_t)gridDim.y * blockIdx.z);
        if (lane == 0) p.partials[(cta * (GTHREADS / 32) + warp) * HEATKV_MAX_K + sg] = acc / (float)t_q;
      } else {
        if (lane == 0) atomicAdd(beta + sg, acc / (float)t_q);
      }
    }
  }

  if (p.out) {
    __syncthreads();                                   // all warps are done with the K/V stages
    // stage the bf16 tile in shared memory (reusing the Q region), then 16-byte row stores
#pragma unroll
    for (int n = 0; n < D / 8; ++n) {
      int r0 = warp * 16 + g;
      uint32_t lo = pack_bf16(o[n][0] * inv_l[0], o[n][1] * inv_l[0]);
      uint32_t hi = pack_bf16(o[n][2] * inv_l[1], o[n][3] * inv_l[1]);
      *reinterpret_cast<uint32_t*>(smem + SM::Q_OFF + tile_off<D>(r0, n) + qd * 4) = lo;
      *reinterpret_cast<uint32_t*>(smem + SM::Q_OFF + tile_off<D>(r0 + 8, n) + qd * 4) = hi;
    }
    __syncthreads();
    constexpr int CH = D / 8;
    __nv_bfloat16* dst = p.out + seq * p.o_seq + head * p.o_head + (int64_t)q0 * p.o_tok;
    for (int i = tid; i < GM * CH; i += GTHREADS) {
      int r = i / CH, ch = i % CH;
      if (q0 + r < t_q) {
        int4 v = *reinterpret_cast<const int4*>(smem + SM::Q_OFF + tile_off<D>(r, ch));
        *reinterpret_cast<int4*>(dst + (int64_t)r * p.o_tok + ch * 8) = v;
      }
    }
  }
}

// beta[head][step][sg] += sum of the partials of that head in the order (sequence, query tile, warp):
// one thread per (head, source scale), so the result does not depend on scheduling.
__global__ void reduce_partials_kernel(const float* partials, float* beta_row, int n_qtiles, int H, int n_seq, int K,
                                       int step) {
  const int head = blockIdx.x, sg = threadIdx.x;
  if (sg > step) return;
  float acc = 0.f;
  for (int seq = 0; seq < n_seq; ++seq)
    for (int qt = 0; qt < n_qtiles; ++qt) {
      const int64_t cta = qt + (int64_t)n_qtiles * (head + (int64_t)H * seq);
      for (int w = 0; w < GTHREADS / 32; ++w) acc += partials[(cta * (GTHREADS / 32) + w) * HEATKV_MAX_K + sg];
    }
  beta_row[(int64_t)head * K * K + sg] += acc;
}

constexpr int MAX_DEVICES = 64;

template <int D, bool CALIB>
static cudaError_t launch_one(const AttnParams& p, int n_seq, cudaStream_t stream) {
  auto kern = attn_generic_kernel<D, CALIB>;
  constexpr int bytes = CALIB ? GenericSmem<D>::BYTES : GenericSmem<D>::ATTN_BYTES;
  // the attribute belongs to the (function, device) pair: set it once on every device that launches
  static std::atomic<bool> configured[MAX_DEVICES];
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (!configured[dev].load(std::memory_order_acquire)) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    configured[dev].store(true, std::memory_order_release);
  }
  const int q_tiles = CALIB && p.cal_n > 0 ? p.cal_tile_begin[p.cal_n] : (p.t_q + GM - 1) / GM;
  dim3 grid(q_tiles + (CALIB ? 0 : p.append_tiles), CALIB ? p.H : n_seq, CALIB ? n_seq : p.H);
  kern<<<grid, GTHREADS, bytes, stream>>>(p);
  return cudaGetLastError();
}

// Calibration pass whose scratch is the static array above.  Returns cudaErrorInvalidValue when the
// launch would need more partial slots than the array has.  The array's device address is looked up
// once per device (cudaGetSymbolAddress; the symbol's name itself is only a host-side handle).
cudaError_t launch_calibrate_static(const AttnParams& p_in, int d, int n_seq, cudaStream_t stream, bool* too_large) {
  *too_large = false;
  const int n_qtiles = (p_in.t_q + GM - 1) / GM;
  const int64_t slots = (int64_t)n_qtiles * p_in.H * n_seq * (GTHREADS / 32) * HEATKV_MAX_K;
  if (slots > STATIC_PARTIAL_FLOATS) {
    *too_large = true;
    return cudaErrorInvalidValue;
  }
  static std::atomic<float*> scratch_of_device[MAX_DEVICES];
  static std::atomic<bool> configured[MAX_DEVICES][2];
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  float* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&scratch), g_static_partials);
    if (e != cudaSuccess) return e;
    scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  AttnParams p = p_in;
  p.partials = scratch;
  p.out = nullptr;
  p.v_new = nullptr;
  const int which = d == 128 ? 1 : 0;
  dim3 grid(n_qtiles, p.H, n_seq);
  if (d == 128) {
    auto kern = attn_generic_kernel<128, true, true>;
    if (!configured[dev][which].load(std::memory_order_acquire)) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GenericSmem<128>::BYTES);
      if (e != cudaSuccess) return e;
      configured[dev][which].store(true, std::memory_order_release);
    }
    kern<<<grid, GTHREADS, GenericSmem<128>::BYTES, stream>>>(p);
  } else if (d == 64) {
    auto kern = attn_generic_kernel<64, true, true>;
    if (!configured[dev][which].load(std::memory_order_acquire)) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GenericSmem<64>::BYTES);
      if (e != cudaSuccess) return e;
      configured[dev][which].store(true, std::memory_order_release);
    }
    kern<<<grid, GTHREADS, GenericSmem<64>::BYTES, stream>>>(p);
  } else {
    return cudaErrorInvalidValue;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  reduce_partials_kernel<<<p.H, HEATKV_MAX_K, 0, stream>>>(p.partials, p.beta_row, n_qtiles, p.H, n_seq, p.K, p.step);
  return cudaGetLastError();
}

cudaError_t launch_attn_generic(const AttnParams& p, int d, int n_seq, bool calib, cudaStream_t stream) {
  if (d == 128) return calib ? launch_one<128, true>(p, n_seq, stream) : launch_one<128, false>(p, n_seq, stream);
  if (d == 64) return calib ? launch_one<64, true>(p, n_seq, stream) : launch_one<64, false>(p, n_seq, stream);
  return cudaErrorInvalidValue;
}

}  // namespace heatkv
