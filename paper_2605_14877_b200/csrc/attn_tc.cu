// Tensor-memory attention kernel for the large scale steps (head_dim 128 or 64).
//
// The launch is a list of work items handed out through a counter: one CTA per SM stays resident and takes
// item after item, so the loads and first products of the next item run under the epilogue of the current
// one.  An attention item is 256 queries of one (sequence, head) as two 128-row tiles A and B that share
// the key/value stream, over the head's whole key range or one piece of it.  When the call carries the
// cache update, the rows of the step's own K/V are copied by two otherwise idle warps, which take
// destination half-tiles from a counter of their own.  Warp roles:
//   warp 0      fetches and decodes items (a two-entry ring in shared memory) and is the TMA producer:
//               Q tiles once per item, then K and V half-tiles (64 rows x 128 dims each) gathered
//               through the plan's page table, followed by the step's own keys.
//   warp 1      MMA issuer: S = Q K^T and O += P V with tcgen05.mma, accumulators in TMEM.
//   warps 2-3   cache update (only when the call carries it).
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one thread per query row
//               reads its row of S from TMEM, keeps the running max / sum, writes P (bf16)
//               back into the columns S occupied, and rescales O only when the row max grew
//               by more than 2^8 since the last reference (the sum keeps the same reference,
//               so the result is exact).  The same warps write the item's result.
// TMEM columns: S_A/P_A 0..127, S_B/P_B 128..255, O_A 256..383, O_B 384..511.
// The MMA order S_A S_B (PV_A S_A' PV_B S_B')* lets the softmax of one tile overlap the
// tensor work of the other.  The host may cut a head's key range into pieces (a count per head); their
// unnormalised results meet in a scratch region, where, for every group of 32 rows, the warp that arrives
// last adds them up in piece order.  All barrier phases run on across items.  Every wait is bounded; on expiry the
// CTA records a status word, drains its own copies and leaves.
#include <algorithm>

#include "append_device.cuh"
#include "internal.h"
#include "tc_common.cuh"

namespace heatkv {

namespace tc {

constexpr int BM = 128;                 // rows per Q tile
constexpr int BN = 128;                 // keys per tile (two 64-row half-tiles)
constexpr int HALF = 64;
constexpr int THREADS = 384;
constexpr int KV_STAGES = 2;
// Registers are handed from the four utility warps to the eight softmax warps.  setmaxnreg only moves
// registers inside the CTA's own allocation (threads x registers at launch), so the two budgets must fit
// in it; an increase that cannot be served would block for ever.
constexpr int REGS_LAUNCH = 168;        // what ptxas assigns under __launch_bounds__(384, 1)
constexpr int REGS_SMALL = 72;
constexpr int REGS_SOFTMAX = 216;
static_assert(128 * REGS_SMALL + 256 * REGS_SOFTMAX <= THREADS * REGS_LAUNCH, "register hand-over exceeds the CTA's allocation");
constexpr uint32_t HALF_COLS_BYTES = 128 * 128;        // one 64-column half of a 128-row tile: 16 KB
constexpr uint32_t SLOT_BYTES = HALF * 128;            // 64 rows x 128 B inside one column half
constexpr uint32_t STAGE_BYTES = 4096;                 // per softmax warp: two buffers of 32 rows x 64 B for the output rows

// Sizes that follow the head dimension D (64 or 128): a 128-row tile is D / 64 column halves of 16 KB.
template <int D>
struct Layout {
  static_assert(D == 64 || D == 128, "head dimension");
  static constexpr int NCH = D / 64;                             // 64-column halves per row
  static constexpr uint32_t TILE_BYTES = NCH * HALF_COLS_BYTES;  // 16 or 32 KB
  // shared memory map (bytes from a 1024-aligned base)
  static constexpr uint32_t SM_Q = 0;                                   // 2 tiles
  static constexpr uint32_t SM_K = SM_Q + 2 * TILE_BYTES;               // KV_STAGES tiles
  static constexpr uint32_t SM_V = SM_K + KV_STAGES * TILE_BYTES;       // KV_STAGES tiles
  static constexpr uint32_t SM_OUT = SM_V + KV_STAGES * TILE_BYTES;     // output staging of the eight softmax warps
  static constexpr uint32_t SM_BAR = SM_OUT + 8 * STAGE_BYTES;          // barriers + scalars + item ring
  static constexpr uint32_t SM_TOTAL = SM_BAR + 512;
  static constexpr uint32_t SM_ALLOC = SM_TOTAL + 1024;                 // slack for manual alignment
  static_assert(SM_ALLOC <= 227 * 1024, "shared memory of one CTA");
  // One partial result of a split head: unnormalised O of both query tiles (fp32, groups of four columns
  // outermost so that a warp's 32 rows touch consecutive 16-byte words), then the rows' running references
  // and row sums.
  static constexpr int SPLIT_SLOT_FLOATS = 2 * BM * D + 2 * 2 * BM;
};

// barrier slots (8 bytes each) inside SM_BAR
enum Bar : uint32_t {
  Q_FULL = 0, Q_EMPTY = 2,      // +x
  K_FULL = 4, K_EMPTY = 6,      // +stage
  V_FULL = 8, V_EMPTY = 10,     // +stage
  S_FULL = 12,                  // +x  S_x of the tile is in TMEM
  P_FULL = 14,                  // +2x+h  half h (keys 64h..64h+63) of P_x of the tile is in TMEM (128 arrivals)
  PV_DONE = 18,                 // +x  O_x includes the item's last tile (one completion per item)
  ITEM_FULL = 20, ITEM_EMPTY = 22,  // +ring entry; EMPTY takes one arrival from the MMA warp and each softmax warp
  N_BARS = 24
};
constexpr uint32_t BAR_TMEM_PTR = N_BARS * 8;                  // offsets inside the barrier region
constexpr uint32_t BAR_ABORT = BAR_TMEM_PTR + 4;
constexpr uint32_t BAR_RING = 256;                             // 2 entries x int32[16]
enum ItemKind : int { ATTENTION = 0, STOP = 2, NOTHING = 3 };
// ring entry words
enum ItemWord : int { W_KIND = 0, W_HEAD, W_SEQ, W_TILES, W_NSPLIT, W_SUB, W_SLOT, W_CTR, W_DESC, W_NDESC };
constexpr int WORK_COUNTER_WORD = 16;                          // word of the status region that hands out the attention items
constexpr int STORE_COUNTER_WORD = 17;                         // ... and the cache-update items


struct Maps {
  CUtensorMap q, k_own, v_own, k_pool, v_pool;
};

// One key half-tile: where it comes from and how many of its 64 rows are real.
struct Slot {
  int pool_row;     // >= 0: row in the pool; < 0: own-scale tokens starting at -(pool_row + 1)
  int n_valid;
  int seg;
};

__device__ __forceinline__ Slot get_slot(int i, const int2* descs, int n_desc, int n_slots, int64_t base_row,
                                         int t_own, int step) {
  Slot s;
  int valid = i < n_slots;
  if (!valid) i = n_slots - 1;                      // padding half-tile: re-read finite data, mask everything
  if (i < n_desc) {
    int2 d = descs[i];
    s.pool_row = (int)(base_row + d.x);
    s.n_valid = d.y & 0xff;
    s.seg = (d.y >> 8) & 0xff;
  } else {
    int tok0 = (i - n_desc) * HALF;
    s.pool_row = -(tok0 + 1);
    s.n_valid = min(HALF, t_own - tok0);
    s.seg = step;
  }
  if (!valid) s.n_valid = 0;
  return s;
}

// What every role derives from a ring entry of kind ATTENTION.
struct Item {
  int head, seq, n_split, sub, piece, qp, q0, nq, j0, n_tiles, slot_base, ctr_base, n_desc, n_slots, desc_begin;
};
__device__ __forceinline__ Item read_item(const volatile int32_t* ring, const AttnParams& p, int n_qp) {
  Item it;
  it.head = ring[W_HEAD];
  it.seq = ring[W_SEQ];
  it.n_split = ring[W_NSPLIT];
  it.sub = ring[W_SUB];
  it.slot_base = ring[W_SLOT];
  it.ctr_base = ring[W_CTR];
  it.desc_begin = ring[W_DESC];
  it.n_desc = ring[W_NDESC];
  const int tiles = ring[W_TILES];
  it.piece = it.sub / n_qp;
  it.qp = it.sub % n_qp;
  it.q0 = it.qp * (2 * BM);
  it.nq = (it.q0 + BM < p.t_q) ? 2 : 1;             // does tile B hold any query?
  it.n_slots = it.n_desc + (p.n_own + HALF - 1) / HALF;
  // this item's run of key tiles: [j0, j0 + n_tiles) of the head's ceil(n_slots / 2)
  const int piece_tiles = (tiles + it.n_split - 1) / it.n_split;
  it.j0 = it.piece * piece_tiles;
  it.n_tiles = min(tiles, it.j0 + piece_tiles) - it.j0;
  return it;
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
attn_tc_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ Maps maps) {
  using L = Layout<D>;
  constexpr int NCH = L::NCH;
  constexpr uint32_t TILE_BYTES = L::TILE_BYTES, SM_Q = L::SM_Q, SM_K = L::SM_K, SM_V = L::SM_V, SM_OUT = L::SM_OUT,
                     SM_BAR = L::SM_BAR, SM_TMEM_PTR = L::SM_BAR + BAR_TMEM_PTR, SM_ABORT = L::SM_BAR + BAR_ABORT,
                     SM_RING = L::SM_BAR + BAR_RING;
  constexpr int SPLIT_SLOT_FLOATS = L::SPLIT_SLOT_FLOATS;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sbase = (raw + 1023u) & ~1023u;
  unsigned char* sgen = smem_raw + (sbase - raw);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(sgen + SM_ABORT);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(sgen + SM_TMEM_PTR);
  volatile int32_t* ring_base = reinterpret_cast<volatile int32_t*>(sgen + SM_RING);
  auto bar = [&](uint32_t which) { return sbase + SM_BAR + which * 8; };

  // the shuffle makes the warp index provably warp-uniform, so role code stays on the uniform datapath
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int u = (p.step * p.L + p.layer) * p.H;
  const int n_qp = (p.t_q + 2 * BM - 1) / (2 * BM);

  if (threadIdx.x == 0) {
    *abort_flag = *reinterpret_cast<volatile uint32_t*>(p.status) != 0;   // an earlier CTA gave up: do not wait again
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(Q_FULL + x), 1);
      mbar_init(bar(Q_EMPTY + x), 1);
      mbar_init(bar(S_FULL + x), 1);
      mbar_init(bar(P_FULL + 2 * x), BM);
      mbar_init(bar(P_FULL + 2 * x + 1), BM);
      mbar_init(bar(PV_DONE + x), 1);
      mbar_init(bar(ITEM_FULL + x), 1);
      mbar_init(bar(ITEM_EMPTY + x), 9);
    }
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(bar(K_FULL + s), 1);
      mbar_init(bar(K_EMPTY + s), 1);
      mbar_init(bar(V_FULL + s), 1);
      mbar_init(bar(V_EMPTY + s), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + SM_TMEM_PTR), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_ptr_smem;

  // register budget per warpgroup: 128*72 + 256*216 <= 64K
  if (warp < 4) {
    reg_dealloc<REGS_SMALL>();
  if (warp == 0) {
    // ------------------------------------------------------------------ item fetch + TMA producer
    const bool leader = elect_one();
    const int own_slots = (p.n_own + HALF - 1) / HALF;
    uint32_t* work_counter = p.status + WORK_COUNTER_WORD;
    uint32_t g = 0;                                    // key tiles handed to the copy engine so far (all items)
    uint32_t iq[2] = {0, 0};                           // items that loaded query tile x so far
    uint32_t armed_k = 0, armed_v = 0, armed_q = 0;    // bit per barrier: a copy was issued at least once
    uint32_t par_k = 0, par_v = 0, par_q = 0;          // bit per barrier: parity of the phase its last copy completes
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      // The first item of a CTA is its block index; later ones come from the counter.  Every CTA ends with
      // one fetch past the end, so the launch makes exactly attn_items fetches and the last resets the counter.
      int idx = blockIdx.x;
      if (it > 0) {
        uint32_t old = 0;
        if (lane == 0) {
          old = atomicAdd(work_counter, 1u);
          if (old == (uint32_t)p.attn_items - 1u) *reinterpret_cast<volatile uint32_t*>(work_counter) = 0;
        }
        idx = (int)gridDim.x + (int)__shfl_sync(0xffffffffu, old, 0);
      }
      const uint32_t slot = it & 1;
      volatile int32_t* ring = ring_base + slot * 16;
      if (it >= 2) ok = warp_wait(bar(ITEM_EMPTY + slot), ((it >> 1) - 1) & 1, abort_flag, p.status);
      if (!ok) break;
      if (idx >= p.attn_items) {
        if (lane == 0) ring[W_KIND] = STOP;
        __syncwarp();
        if (leader) mbar_arrive(bar(ITEM_FULL + slot));
        break;
      }
      // Attention items: sequences interleaved; the items of one sequence run over its heads by descending
      // key count (the plan's order); a head may be cut into equal pieces of its key range (the count comes
      // from the host's table, else from the launch's longest run), and every (piece, query tile pair) is
      // one item, pieces outermost.  A prefix sum over the
      // heads finds the item.
      const int seq = idx % p.n_seq;
      const int item = idx / p.n_seq;
      PlanView pv(p.seqs[seq].plan);
      if (lane == 0) ring[W_KIND] = NOTHING;            // sequences of a call may differ in item count
      __syncwarp();
      int before = 0, slots_before = 0, ctrs_before = 0;
      for (int base = 0; base < p.H; base += 32) {
        const int i = base + lane;
        int h = 0, tiles = 0, ns = 0, cnt = 0;
        if (i < p.H) {
          if (p.table_heads > 0) {                            // the host put the per-head table into the launch parameters
            h = p.table_head[i];
            tiles = p.table_tiles[i];
            ns = p.table_split[i];
          } else {
            h = pv.order()[u + i];
            tiles = (pv.attn_cnt()[u + h] + own_slots + 1) >> 1;
            ns = p.split_tiles > 0 ? (tiles + p.split_tiles - 1) / p.split_tiles : 1;
          }
          cnt = n_qp * ns;
        }
        const int scnt = ns > 1 ? cnt : 0, ccnt = ns > 1 ? n_qp : 0;
        int inc = cnt, sinc = scnt, cinc = ccnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v0 = __shfl_up_sync(0xffffffffu, inc, o), v1 = __shfl_up_sync(0xffffffffu, sinc, o),
                    v2 = __shfl_up_sync(0xffffffffu, cinc, o);
          if (lane >= o) { inc += v0; sinc += v1; cinc += v2; }
        }
        const int excl = before + inc - cnt;
        const bool mine = cnt > 0 && item >= excl && item < excl + cnt;
        if (mine) {
          ring[W_HEAD] = h;
          ring[W_SEQ] = seq;
          ring[W_TILES] = tiles;
          ring[W_NSPLIT] = ns;
          ring[W_SUB] = item - excl;                        // piece * n_qp + query tile pair
          ring[W_SLOT] = slots_before + sinc - scnt;        // first partial slot of this head
          ring[W_CTR] = ctrs_before + cinc - ccnt;          // first arrival counter group of this head
          ring[W_DESC] = pv.attn_begin()[u + h];
          ring[W_NDESC] = pv.attn_cnt()[u + h];
          ring[W_KIND] = ATTENTION;
        }
        const bool any = __any_sync(0xffffffffu, mine);
        before += __shfl_sync(0xffffffffu, inc, 31);
        slots_before += __shfl_sync(0xffffffffu, sinc, 31);
        ctrs_before += __shfl_sync(0xffffffffu, cinc, 31);
        if (any) break;
      }
      __syncwarp();
      const bool is_attn = ring[W_KIND] == ATTENTION;
      Item im;
      if (is_attn) im = read_item(ring, p, n_qp);
      __syncwarp();
      if (leader) mbar_arrive(bar(ITEM_FULL + slot));
      if (!is_attn) continue;
      const int2* descs = pv.descs() + im.desc_begin;
      const int64_t base_row = p.seqs[seq].base_row;
      for (int j = 0; j < im.n_tiles && ok; ++j, ++g) {
        const uint32_t st = g % KV_STAGES;
        const uint32_t use = g / KV_STAGES;
        Slot sl[2];
        for (int hf = 0; hf < 2; ++hf)
          sl[hf] = get_slot(2 * (im.j0 + j) + hf, descs, im.n_desc, im.n_slots, base_row, p.n_own, p.step);
        // K first: the S product of the next tile needs it earliest
        if (use > 0) ok = warp_wait(bar(K_EMPTY + st), (use - 1) & 1, abort_flag, p.status);
        if (!ok) break;
        armed_k |= 1u << st;
        par_k = (par_k & ~(1u << st)) | ((use & 1) << st);
        if (leader) {
          mbar_expect_tx(bar(K_FULL + st), TILE_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            for (int ch = 0; ch < NCH; ++ch) {
              uint32_t dst = sbase + SM_K + st * TILE_BYTES + ch * HALF_COLS_BYTES + hf * SLOT_BYTES;
              if (sl[hf].pool_row >= 0) tma_load_2d(dst, &maps.k_pool, ch * 64, sl[hf].pool_row, bar(K_FULL + st));
              else tma_load_4d(dst, &maps.k_own, ch * 64, -sl[hf].pool_row - 1, im.head, seq, bar(K_FULL + st));
            }
        }
        if (j == 0) {
          // the item's query tiles, once the last S product of the previous item has read the old ones
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            if (x >= im.nq || !ok) continue;
            if (iq[x] > 0) ok = warp_wait(bar(Q_EMPTY + x), (iq[x] - 1) & 1, abort_flag, p.status);
            if (!ok) continue;
            armed_q |= 1u << x;
            par_q = (par_q & ~(1u << x)) | ((iq[x] & 1) << x);
            ++iq[x];
            if (leader) {
              mbar_expect_tx(bar(Q_FULL + x), TILE_BYTES);
              for (int ch = 0; ch < NCH; ++ch)
                for (int hf = 0; hf < 2; ++hf)
                  tma_load_4d(sbase + SM_Q + x * TILE_BYTES + ch * HALF_COLS_BYTES + hf * SLOT_BYTES, &maps.q, ch * 64,
                              im.q0 + x * BM + hf * HALF, im.head, seq, bar(Q_FULL + x));
            }
          }
          if (!ok) break;
        }
        if (use > 0) ok = warp_wait(bar(V_EMPTY + st), (use - 1) & 1, abort_flag, p.status);
        if (!ok) break;
        armed_v |= 1u << st;
        par_v = (par_v & ~(1u << st)) | ((use & 1) << st);
        if (leader) {
          mbar_expect_tx(bar(V_FULL + st), TILE_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            for (int ch = 0; ch < NCH; ++ch) {
              uint32_t dst = sbase + SM_V + st * TILE_BYTES + ch * HALF_COLS_BYTES + hf * SLOT_BYTES;
              if (sl[hf].pool_row >= 0) tma_load_2d(dst, &maps.v_pool, ch * 64, sl[hf].pool_row, bar(V_FULL + st));
              else tma_load_4d(dst, &maps.v_own, ch * 64, -sl[hf].pool_row - 1, im.head, seq, bar(V_FULL + st));
            }
        }
        __syncwarp();
      }
    }
    if (!ok || *abort_flag) {
      // leaving early: let every copy this warp started land before the CTA exits
      for (int s = 0; s < KV_STAGES; ++s) {
        if (armed_k & (1u << s))
          for (uint32_t t = 0; t < WAIT_LIMIT && !mbar_try(bar(K_FULL + s), (par_k >> s) & 1); ++t) {}
        if (armed_v & (1u << s))
          for (uint32_t t = 0; t < WAIT_LIMIT && !mbar_try(bar(V_FULL + s), (par_v >> s) & 1); ++t) {}
      }
      for (int x = 0; x < 2; ++x)
        if (armed_q & (1u << x))
          for (uint32_t t = 0; t < WAIT_LIMIT && !mbar_try(bar(Q_FULL + x), (par_q >> x) & 1); ++t) {}
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const bool leader = elect_one();
    constexpr uint32_t IDESC_S = instr_desc(BM, BN, 0, 0);     // Q, K both K-major
    constexpr uint32_t IDESC_PV = instr_desc(BM, D, 0, 1);     // P from TMEM, V MN-major
    bool ok = true;
    auto issue_s = [&](int x, int st) {
      const uint32_t qa = sbase + SM_Q + x * TILE_BYTES, ka = sbase + SM_K + st * TILE_BYTES;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t off = (ks >> 2) * HALF_COLS_BYTES + (ks & 3) * 32;
        mma_ss(tmem + x * 128, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024), IDESC_S, ks > 0);
      }
    };
    // keys 64h .. 64h+63 of the tile: four K=16 steps
    auto issue_pv = [&](int x, int st, int h, bool first) {
      const uint32_t va = sbase + SM_V + st * TILE_BYTES;
#pragma unroll
      for (int ks = 4 * h; ks < 4 * h + 4; ++ks)
        mma_ts(tmem + 256 + x * 128, tmem + x * 128 + ks * 8, smem_desc(va + ks * 2048, HALF_COLS_BYTES, 1024),
               IDESC_PV, !(first && ks == 0));
    };
    uint32_t g = 0;                                    // key tiles consumed so far (all items)
    uint32_t cx[2] = {0, 0};                           // key tiles of query tile x so far
    uint32_t iq[2] = {0, 0};                           // items with query tile x so far
    for (uint32_t it = 0; ok; ++it) {
      const uint32_t slot = it & 1;
      volatile int32_t* ring = ring_base + slot * 16;
      ok = warp_wait(bar(ITEM_FULL + slot), (it >> 1) & 1, abort_flag, p.status);
      if (!ok) break;
      const int kind = ring[W_KIND];
      if (kind == STOP) break;
      if (kind == ATTENTION) {
        const Item im = read_item(ring, p, n_qp);
        const int nq = im.nq, n_tiles = im.n_tiles;
        const uint32_t st0 = g % KV_STAGES, par0 = (g / KV_STAGES) & 1;
#pragma unroll
        for (int x = 0; x < 2; ++x)
          if (x < nq && ok) ok = warp_wait(bar(Q_FULL + x), iq[x] & 1, abort_flag, p.status);
        if (ok) ok = warp_wait(bar(K_FULL + st0), par0, abort_flag, p.status);
        if (ok) {
          tc_fence_after();
          if (leader) {
            for (int x = 0; x < nq; ++x) {
              issue_s(x, st0);
              tc_commit(bar(S_FULL + x));
              if (n_tiles == 1) tc_commit(bar(Q_EMPTY + x));
            }
            tc_commit(bar(K_EMPTY + st0));
          }
          __syncwarp();
        }
        // Waits for K and V sit where the tensor pipe still has queued work: the next tile's V at the end
        // of an iteration, the next tile's K between the two halves of PV_A.  The hand-over of P is then
        // the only wait between the last S product of one tile and the first PV product of the next.
        if (ok) ok = warp_wait(bar(V_FULL + st0), par0, abort_flag, p.status);
        for (int j = 0; j < n_tiles && ok; ++j) {
          const uint32_t st = (g + j) % KV_STAGES, stn = (g + j + 1) % KV_STAGES;
          const uint32_t parn = ((g + j + 1) / KV_STAGES) & 1;
          const bool more = j + 1 < n_tiles;
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            if (x >= nq || !ok) continue;
            const uint32_t ph = (cx[x] + j) & 1;
            ok = warp_wait(bar(P_FULL + 2 * x), ph, abort_flag, p.status);
            if (!ok) continue;
            tc_fence_after();
            if (leader) issue_pv(x, st, 0, j == 0);
            __syncwarp();
            // the next tile's keys are waited for here, off the path between the last half of P and the next S
            if (more && x == 0) ok = warp_wait(bar(K_FULL + stn), parn, abort_flag, p.status);
            if (!ok) continue;
            ok = warp_wait(bar(P_FULL + 2 * x + 1), ph, abort_flag, p.status);
            if (!ok) continue;
            tc_fence_after();
            if (leader) {
              issue_pv(x, st, 1, false);
              if (!more) tc_commit(bar(PV_DONE + x));                   // only the epilogue waits for it
            }
            __syncwarp();
            if (more) {
              if (leader) {
                issue_s(x, stn);
                tc_commit(bar(S_FULL + x));
                if (j + 2 == n_tiles) tc_commit(bar(Q_EMPTY + x));     // the item's last product that reads Q_x
              }
              __syncwarp();
            }
          }
          if (ok && leader) {
            tc_commit(bar(V_EMPTY + st));
            if (more) tc_commit(bar(K_EMPTY + stn));
          }
          __syncwarp();
          if (ok && more) ok = warp_wait(bar(V_FULL + stn), parn, abort_flag, p.status);
        }
        g += n_tiles;
#pragma unroll
        for (int x = 0; x < 2; ++x)
          if (x < nq) {
            cx[x] += n_tiles;
            ++iq[x];
          }
      }
      __syncwarp();
      if (ok && leader) mbar_arrive(bar(ITEM_EMPTY + slot));
    }
  } else if (p.store_items > 0) {
    // ------------------------------------------------------------------ cache update (warps 2 and 3)
    // Each warp takes destination half-tiles of (sequence, head) units from a counter of its own and copies
    // their rows while the other warps work on attention items.  Every store warp of the launch ends with one
    // fetch past the end; the last of those store_items + 2 * CTAs fetches resets the counter.
    uint32_t* store_counter = p.status + STORE_COUNTER_WORD;
    const uint32_t fetches = (uint32_t)p.store_items + 2u * gridDim.x;
    for (;;) {
      uint32_t old = 0;
      if (lane == 0) {
        old = atomicAdd(store_counter, 1u);
        if (old == fetches - 1u) *reinterpret_cast<volatile uint32_t*>(store_counter) = 0;
      }
      const int a = (int)__shfl_sync(0xffffffffu, old, 0);
      if (a >= p.store_items) break;
      const int sq = a % p.n_seq, hd = (a / p.n_seq) % p.H, j = a / (p.n_seq * p.H);
      const int64_t src = sq * p.kv_seq + hd * p.kv_head;
      append_half_tile(p.seqs[sq].plan, p.seqs[sq].base_row, u + hd, j, p.k_new + src, p.v_new + src, p.kv_tok,
                       const_cast<__nv_bfloat16*>(p.k_pool), const_cast<__nv_bfloat16*>(p.v_pool), D, lane, 32);
    }
  }
  } else {
    reg_alloc<REGS_SOFTMAX>();
    // ------------------------------------------------------------------ softmax + epilogue + cache-update items
    const int x = (warp - 4) >> 2;                      // 0: tile A, 1: tile B
    const int row = (warp & 3) * 32 + lane;             // row inside the tile == TMEM lane
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + lane_base + x * 128;
    const uint32_t t_o = tmem + lane_base + 256 + x * 128;
    unsigned char* stage = sgen + SM_OUT + (warp - 4) * STAGE_BYTES;
    const float LOG2E = 1.4426950408889634f;
    uint32_t cx = 0;                                    // key tiles of this query tile so far (all items)
    uint32_t items_x = 0;                               // items in which this query tile held rows so far
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      const uint32_t slot = it & 1;
      volatile int32_t* ring = ring_base + slot * 16;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(ITEM_FULL + slot), (it >> 1) & 1, abort_flag, p.status));
      if (!ok) break;
      const int kind = ring[W_KIND];
      if (kind == STOP) break;
      if (kind == ATTENTION) {
        // Only what the tile loop needs stays in registers; the epilogue reads the ring entry again.
        int n_tiles, nq;
        {
          const Item im = read_item(ring, p, n_qp);
          n_tiles = im.n_tiles;
          nq = im.nq;
        }
        if (x < nq) {
          int j0, n_desc, n_slots;
          const int2* descs;
          const float* bias_h;
          {
            const Item im = read_item(ring, p, n_qp);
            j0 = im.j0; n_desc = im.n_desc; n_slots = im.n_slots;
            descs = PlanView(p.seqs[im.seq].plan).descs() + im.desc_begin;
            bias_h = p.seg_bias ? p.seg_bias + im.head * p.K : nullptr;
          }
          float m_ref = -INFINITY, l_sum = 0.f;
          for (int j = 0; j < n_tiles && ok; ++j) {
            const uint32_t ph = (cx + j) & 1;
            Slot s0 = get_slot(2 * (j0 + j), descs, n_desc, n_slots, 0, p.n_own, p.step);       // row numbers unused here
            Slot s1 = get_slot(2 * (j0 + j) + 1, descs, n_desc, n_slots, 0, p.n_own, p.step);
            const float b0 = bias_h ? bias_h[s0.seg] * LOG2E : 0.f;
            const float b1 = bias_h ? bias_h[s1.seg] * LOG2E : 0.f;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(S_FULL + x), ph, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            // whole row of S into registers (one wait for the four loads)
            uint32_t r0[32], r1[32], r2[32], r3[32];
            tmem_ld32(t_s, r0);
            tmem_ld32(t_s + 32, r1);
            tmem_ld32(t_s + 64, r2);
            tmem_ld32(t_s + 96, r3);
            tmem_wait_ld();
            if (s0.n_valid < HALF || s1.n_valid < HALF) {            // ragged tile (warp-uniform): mask by -inf
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                if (i >= s0.n_valid) r0[i] = 0xff800000u;
                if (i + 32 >= s0.n_valid) r1[i] = 0xff800000u;
                if (i >= s1.n_valid) r2[i] = 0xff800000u;
                if (i + 32 >= s1.n_valid) r3[i] = 0xff800000u;
              }
            }
            // row maximum: the logit is raw * scale + bias(half) with scale > 0, so take the raw maxima
            // (eight independent chains keep the dependent depth short)
            float mq[8];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              mq[c] = fmaxf(__uint_as_float(r0[c]), __uint_as_float(r1[c]));
              mq[4 + c] = fmaxf(__uint_as_float(r2[c]), __uint_as_float(r3[c]));
            }
#pragma unroll
            for (int i = 4; i < 32; i += 4) {
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                mq[c] = fmax3(mq[c], __uint_as_float(r0[i + c]), __uint_as_float(r1[i + c]));
                mq[4 + c] = fmax3(mq[4 + c], __uint_as_float(r2[i + c]), __uint_as_float(r3[i + c]));
              }
            }
            const float mx0 = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3]));
            const float mx1 = fmaxf(fmaxf(mq[4], mq[5]), fmaxf(mq[6], mq[7]));
            const float mx = fmaxf(fmaf(mx0, p.scale_log2, b0), fmaf(mx1, p.scale_log2, b1));
            const float m_new = fmaxf(m_ref, mx);
            const bool grow = m_new > m_ref + RESCALE_THRESHOLD;   // also true on the first tile (m_ref = -inf)
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
              // O_x holds tiles < j relative to m_ref: rescale the rows whose reference moves.  O_x is complete:
              // S_x of this tile was issued after the PV products of tile j - 1 by the same thread, and the
              // commit behind S_FULL covers every product issued before it.
              const float f = grow ? exp2f(m_ref - m_new) : 1.f;
#pragma unroll
              for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(t_o + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
                tmem_st32(t_o + c * 32, r);
              }
              tmem_wait_st();
              l_sum *= f;
            }
            if (grow) m_ref = m_new;
            // p = exp2(logit - m_ref); row sum in fp32; P as bf16 pairs into the columns S occupied
            // (keys 32c..32c+31 -> P columns 16c..16c+15; the whole row of S is already in registers).
            // One pair in four takes the polynomial on the FMA pipe, the rest the MUFU unit: the tile's
            // 16 384 exponentials would otherwise keep MUFU busy as long as the tensor pipe needs for
            // the tile's two products.
            const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2);
            uint64_t sum2 = pack2(0.f, 0.f);
            auto exp_chunk = [&](const uint32_t (&rc)[32], uint64_t bb2, int c) {
              uint32_t pk[16];
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const uint64_t xx = fma2(pack2(__uint_as_float(rc[i]), __uint_as_float(rc[i + 1])), scale2, bb2);
                float e0, e1;
                if (((i >> 1) & POLY_MASK) == POLY_MASK) {
                  exp2_poly2(xx, e0, e1);
                } else {
                  float x0, x1;
                  unpack2(xx, x0, x1);
                  e0 = ex2_approx(x0);
                  e1 = ex2_approx(x1);
                }
                sum2 = add2(sum2, pack2(e0, e1));
                pk[i >> 1] = pack_bf16(e0, e1);
              }
              tmem_st16(t_s + c * 16, pk);
            };
            const uint64_t bb0 = pack2(b0 - m_ref, b0 - m_ref), bb1 = pack2(b1 - m_ref, b1 - m_ref);
            exp_chunk(r0, bb0, 0);
            exp_chunk(r1, bb0, 1);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(P_FULL + 2 * x));                      // the PV product of keys 0..63 may start
            exp_chunk(r2, bb1, 2);
            exp_chunk(r3, bb1, 3);
            float sa, sb;
            unpack2(sum2, sa, sb);
            l_sum += sa + sb;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(P_FULL + 2 * x + 1));
          }
          if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(PV_DONE + x), items_x & 1, abort_flag, p.status));
          ++items_x;
          cx += n_tiles;
          const Item im = read_item(ring, p, n_qp);
          const int seq = im.seq;
          const int q_row0 = im.q0 + x * BM;
          __nv_bfloat16* dst = p.out + seq * p.o_seq + im.head * p.o_head + (int64_t)q_row0 * p.o_tok;
          // Normalised rows leave through this warp's staging buffer: per group of 32 columns every thread
          // parks its 64 bytes (16-byte chunks, chunk ^ (row / 2 mod 4) against bank conflicts), then four
          // lanes write each row's 64 bytes.  The two halves of the buffer alternate between groups.
          auto store_rows = [&](const float (&acc)[32], float inv, int c) {
            unsigned char* buf = stage + (c & 1) * 2048;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              int4 v;
              v.x = (int)pack_bf16(acc[i] * inv, acc[i + 1] * inv);
              v.y = (int)pack_bf16(acc[i + 2] * inv, acc[i + 3] * inv);
              v.z = (int)pack_bf16(acc[i + 4] * inv, acc[i + 5] * inv);
              v.w = (int)pack_bf16(acc[i + 6] * inv, acc[i + 7] * inv);
              const int chunk = i >> 3;
              *reinterpret_cast<int4*>(buf + lane * 64 + ((chunk ^ ((lane >> 1) & 3)) << 4)) = v;
            }
            __syncwarp();
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2) {
              const int rl = 8 * k2 + (lane >> 2), chunk = lane & 3;
              const int rr = (warp & 3) * 32 + rl;
              if (q_row0 + rr < p.t_q) {
                const int4 v = *reinterpret_cast<const int4*>(buf + rl * 64 + ((chunk ^ ((rl >> 1) & 3)) << 4));
                *reinterpret_cast<int4*>(dst + (int64_t)rr * p.o_tok + c * 32 + chunk * 8) = v;
              }
            }
          };
          if (ok && im.n_split == 1) {
            tc_fence_after();
            const float inv = 1.f / l_sum;
            // the whole row of O in one go, so the four groups' conversions and stores overlap
            uint32_t o[D / 32][32];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) tmem_ld32(t_o + c * 32, o[c]);
            tmem_wait_ld();
            auto out_group = [&](const uint32_t (&r)[32], int c) {
              float acc[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) acc[i] = __uint_as_float(r[i]);
              store_rows(acc, inv, c);
            };
#pragma unroll
            for (int c = 0; c < D / 32; ++c) out_group(o[c], c);
          } else if (ok) {
            // A piece of a split head: publish the unnormalised O of this row with its reference and row
            // sum; the warp that arrives last at the counter of these 32 rows merges
            // sum over pieces of 2^(m_piece - m) * (O_piece, l_piece).
            tc_fence_after();
            const int n_split = im.n_split, piece = im.piece, qp = im.qp;
            float* slots = p.split_partials + ((int64_t)seq * p.slots_per_seq + im.slot_base) * SPLIT_SLOT_FLOATS;
            float* slot_own = slots + (int64_t)im.sub * SPLIT_SLOT_FLOATS;
            int4* ocol = reinterpret_cast<int4*>(slot_own) + x * BM + row;
            uint32_t* ctr = p.split_counters + ((int64_t)seq * p.ctrs_per_seq + im.ctr_base + qp) * 8 + (warp - 4);
            // Every other piece of these 32 rows published already?  Then this warp's own stays in TMEM and it merges at once.
            uint32_t last = 0;
            if (lane == 0) {
              uint32_t seen;
              asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(ctr) : "memory");
              last = seen == (uint32_t)(n_split - 1);
              if (last) *reinterpret_cast<volatile uint32_t*>(ctr) = 0;     // ready for the next launch
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (!last) {
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(t_o + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int gq = 0; gq < 8; ++gq)
                  ocol[(c * 8 + gq) * (2 * BM)] = make_int4((int)r[4 * gq], (int)r[4 * gq + 1], (int)r[4 * gq + 2], (int)r[4 * gq + 3]);
              }
              slot_own[2 * BM * D + x * BM + row] = m_ref;
              slot_own[2 * BM * D + 2 * BM + x * BM + row] = l_sum;
              __threadfence();
              __syncwarp();
              if (lane == 0) {
                const uint32_t old = atomicAdd(ctr, 1u);
                last = old == (uint32_t)(n_split - 1);
                if (last) *reinterpret_cast<volatile uint32_t*>(ctr) = 0;   // ready for the next launch
              }
              last = __shfl_sync(0xffffffffu, last, 0);
            }
            if (last) {
              __threadfence();
              // The pieces are added in piece order, this warp's own (still in TMEM) at its place among them, so
              // the result does not depend on which piece happened to arrive last.
              // references and row sums of up to MERGE_FAST pieces are read once, all loads in flight together;
              // a head cut finer than that reads them again where it needs them
              constexpr int MERGE_FAST = 4;
              float mp[MERGE_FAST], lp[MERGE_FAST];
#pragma unroll
              for (int s2 = 0; s2 < MERGE_FAST; ++s2) {
                const float* sl = slots + (int64_t)(s2 * n_qp + qp) * SPLIT_SLOT_FLOATS;
                const bool other = s2 < n_split && s2 != piece;
                mp[s2] = other ? __ldcg(sl + 2 * BM * D + x * BM + row) : (s2 == piece ? m_ref : -INFINITY);
                lp[s2] = other ? __ldcg(sl + 2 * BM * D + 2 * BM + x * BM + row) : (s2 == piece ? l_sum : 0.f);
              }
              float m_all = -INFINITY;                                // common reference and total row sum
#pragma unroll
              for (int s2 = 0; s2 < MERGE_FAST; ++s2) m_all = fmaxf(m_all, mp[s2]);
              for (int s2 = MERGE_FAST; s2 < n_split; ++s2) {
                const float* sl = slots + (int64_t)(s2 * n_qp + qp) * SPLIT_SLOT_FLOATS;
                m_all = fmaxf(m_all, s2 == piece ? m_ref : __ldcg(sl + 2 * BM * D + x * BM + row));
              }
              float l_all = 0.f;
#pragma unroll
              for (int s2 = 0; s2 < MERGE_FAST; ++s2) {               // piece order, as below
                mp[s2] = s2 < n_split ? exp2f(mp[s2] - m_all) : 0.f;  // from here on: the piece's weight
                l_all = fmaf(lp[s2], mp[s2], l_all);
              }
              for (int s2 = MERGE_FAST; s2 < n_split; ++s2) {
                const float* sl = slots + (int64_t)(s2 * n_qp + qp) * SPLIT_SLOT_FLOATS;
                const float l2 = s2 == piece ? l_sum : __ldcg(sl + 2 * BM * D + 2 * BM + x * BM + row);
                const float m2 = s2 == piece ? m_ref : __ldcg(sl + 2 * BM * D + x * BM + row);
                l_all = fmaf(l2, exp2f(m2 - m_all), l_all);
              }
              const float inv = 1.f / l_all;
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(t_o + c * 32, r);
                tmem_wait_ld();
                float acc[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[i] = 0.f;
                for (int s2 = 0; s2 < n_split; ++s2) {
                  if (s2 == piece) {
                    const float w_own = exp2f(m_ref - m_all);
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] = fmaf(__uint_as_float(r[i]), w_own, acc[i]);
                    continue;
                  }
                  const float* sl = slots + (int64_t)(s2 * n_qp + qp) * SPLIT_SLOT_FLOATS;
                  float w;
                  if (s2 < MERGE_FAST) {
                    w = s2 == 0 ? mp[0] : s2 == 1 ? mp[1] : s2 == 2 ? mp[2] : mp[3];
                  } else {
                    w = exp2f(__ldcg(sl + 2 * BM * D + x * BM + row) - m_all);
                  }
                  const float4* oc = reinterpret_cast<const float4*>(sl) + (c * 8) * (2 * BM) + x * BM + row;
#pragma unroll
                  for (int i = 0; i < 8; ++i) {
                    const float4 v = __ldcg(oc + i * (2 * BM));
                    acc[4 * i] = fmaf(v.x, w, acc[4 * i]);
                    acc[4 * i + 1] = fmaf(v.y, w, acc[4 * i + 1]);
                    acc[4 * i + 2] = fmaf(v.z, w, acc[4 * i + 2]);
                    acc[4 * i + 3] = fmaf(v.w, w, acc[4 * i + 3]);
                  }
                }
                store_rows(acc, inv, c);
              }
            }
          }
          // the next item's first P hand-over orders this item's reads of O before the next PV product
          tc_fence_before();
        }
      }
      __syncwarp();
      if (ok && lane == 0) mbar_arrive(bar(ITEM_EMPTY + slot));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// Self-test of the bounded wait: one thread waits on a barrier nobody will ever arrive at, with a short limit,
// and reports what the wait returned.  The wait must give up, set the status word and return false.
__global__ void wait_expiry_kernel(uint32_t* status, uint32_t* result) {
  __shared__ __align__(8) unsigned long long barrier_word;
  __shared__ uint32_t abort_word;
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(smem_u32(&barrier_word), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(smem_u32(&barrier_word), 0, &abort_word, status, 2048u);
    result[0] = ok ? 1u : (abort_word ? 2u : 3u);
  }
}

}  // namespace tc

cudaError_t launch_wait_expiry(uint32_t* status, uint32_t* result, cudaStream_t stream) {
  tc::wait_expiry_kernel<<<1, 32, 0, stream>>>(status, result);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------- host side
struct TcState {
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  CUtensorMap k_pool, v_pool;
  int n_sm = 148;
  int d = 0;                 // head dimension of the context (64 or 128)
  bool ready = false;
};

namespace {

bool encode_2d(TcState* st, CUtensorMap* m, void* base, uint64_t rows) {
  cuuint64_t dims[2] = {(cuuint64_t)st->d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)st->d * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)tc::HALF};
  cuuint32_t estr[2] = {1, 1};
  return st->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [n_seq, H, t, d] view with element strides -> 4-D map (d, token, head, sequence)
bool encode_4d(TcState* st, CUtensorMap* m, const void* base, int t, int H, int n_seq, int64_t s_tok, int64_t s_head,
               int64_t s_seq) {
  cuuint64_t dims[4] = {(cuuint64_t)st->d, (cuuint64_t)t, (cuuint64_t)H, (cuuint64_t)n_seq};
  // a stride of 0 is not encodable; a dimension of extent 1 may carry any positive stride
  auto fix = [](int64_t s) { return (cuuint64_t)((s > 0 ? s : 8) * 2); };
  cuuint64_t strides[3] = {fix(s_tok), fix(s_head), fix(s_seq)};
  cuuint32_t box[4] = {64, (cuuint32_t)tc::HALF, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return st->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int tc_create(const heatkv_config& cfg, void* k_pool, void* v_pool, uint64_t pool_rows, TcState** out) {
  *out = nullptr;
  TcState* st = new (std::nothrow) TcState;
  if (!st) return HEATKV_ERR_HOST_MEMORY;
  *out = st;
  if (cfg.d != 64 && cfg.d != 128) return HEATKV_OK;    // other head dimensions run on the generic kernel only
  st->d = cfg.d;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    return HEATKV_OK;                                   // no driver entry point: generic kernel only
  }
  st->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  if (!encode_2d(st, &st->k_pool, k_pool, pool_rows) || !encode_2d(st, &st->v_pool, v_pool, pool_rows))
    return HEATKV_OK;
  const void* kern = cfg.d == 128 ? (const void*)tc::attn_tc_kernel<128> : (const void*)tc::attn_tc_kernel<64>;
  const int smem = cfg.d == 128 ? (int)tc::Layout<128>::SM_ALLOC : (int)tc::Layout<64>::SM_ALLOC;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
    cudaGetLastError();
    return HEATKV_OK;
  }
  // the register hand-over inside the kernel must fit in what the launch really allocates
  cudaFuncAttributes attr;
  if (cudaFuncGetAttributes(&attr, kern) != cudaSuccess) {
    cudaGetLastError();
    return HEATKV_OK;
  }
  if (attr.numRegs * tc::THREADS < 128 * tc::REGS_SMALL + 256 * tc::REGS_SOFTMAX) return HEATKV_ERR_CUDA;
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n_sm > 0)
    st->n_sm = n_sm;
  st->ready = true;
  return HEATKV_OK;
}

void tc_destroy(TcState* st) { delete st; }

bool tc_ready(const TcState* st) { return st && st->ready; }

int tc_split_slot_floats(int d) { return d == 64 ? tc::Layout<64>::SPLIT_SLOT_FLOATS : tc::Layout<128>::SPLIT_SLOT_FLOATS; }

bool tc_supported(const TcState* st, const AttnParams& p, int d, int n_seq, bool calib) {
  if (!st || !st->ready || calib || d != st->d || n_seq > 65535) return false;
  // TMA needs 16-byte aligned bases (checked by the caller) and strides that are multiples of 16 bytes
  const int64_t s[6] = {p.q_seq, p.q_head, p.q_tok, p.kv_seq, p.kv_head, p.kv_tok};
  for (int64_t v : s)
    if (v & 7) return false;
  return true;
}

cudaError_t launch_attn_tc(TcState* st, const AttnParams& p, int d, int n_seq, bool calib, cudaStream_t stream,
                           int* launches) {
  (void)d; (void)calib;
  tc::Maps maps;
  maps.k_pool = st->k_pool;
  maps.v_pool = st->v_pool;
  if (!encode_4d(st, &maps.q, p.q, p.t_q, p.H, n_seq, p.q_tok, p.q_head, p.q_seq) ||
      !encode_4d(st, &maps.k_own, p.k_new, p.n_own, p.H, n_seq, p.kv_tok, p.kv_head, p.kv_seq) ||
      !encode_4d(st, &maps.v_own, p.v_new, p.n_own, p.H, n_seq, p.kv_tok, p.kv_head, p.kv_seq))
    return cudaErrorInvalidValue;
  if (p.n_seq != n_seq || p.items_per_seq < 1) return cudaErrorInvalidValue;
  // one resident CTA per SM takes the attention items in turn; its two spare warps take the cache-update items
  AttnParams q = p;
  q.attn_items = p.items_per_seq * n_seq;
  q.store_items = p.append_tiles * p.H * n_seq;
  dim3 grid((unsigned)std::min(q.attn_items, st->n_sm));
  if (st->d == 128) tc::attn_tc_kernel<128><<<grid, tc::THREADS, tc::Layout<128>::SM_ALLOC, stream>>>(q, maps);
  else tc::attn_tc_kernel<64><<<grid, tc::THREADS, tc::Layout<64>::SM_ALLOC, stream>>>(q, maps);
  *launches = 1;
  return cudaGetLastError();
}

}  // namespace heatkv
