// C ABI of libheatkv: context, arena bookkeeping, sequence admission and the launch logic
// of every entry point declared in heatkv.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <memory>
#include <new>
#include <vector>

#include "device_common.cuh"
#include "internal.h"

namespace heatkv {
cudaError_t launch_attn_generic(const AttnParams& p, int d, int n_seq, bool calib, cudaStream_t stream);
cudaError_t launch_calibrate_static(const AttnParams& p, int d, int n_seq, cudaStream_t stream, bool* too_large);
cudaError_t launch_append(const CopyParams& p, int n_seq, cudaStream_t stream);
cudaError_t launch_compact(const CopyParams& p, int n_seq, cudaStream_t stream);
cudaError_t launch_append_fp8(const CopyParams& p, int n_seq, cudaStream_t stream);
cudaError_t launch_dequant_fp8(const CopyParams& p, int n_seq, int slots, cudaStream_t stream);
struct TcState;
int tc_create(const heatkv_config& cfg, void* k_pool, void* v_pool, uint64_t pool_rows, TcState** out);
void tc_destroy(TcState* st);
bool tc_ready(const TcState* st);
bool tc_supported(const TcState* st, const AttnParams& p, int d, int n_seq, bool calib);
cudaError_t launch_attn_tc(TcState* st, const AttnParams& p, int d, int n_seq, bool calib, cudaStream_t stream,
                           int* launches);
int tc_split_slot_floats(int d);
cudaError_t launch_wait_expiry(uint32_t* status, uint32_t* result, cudaStream_t stream);
struct CalibTcState;
uint64_t calib_tc_desc_bytes(const heatkv_config& cfg);
int calib_tc_create(const heatkv_config& cfg, void* dev_table, cudaStream_t stream, CalibTcState** out);
void calib_tc_destroy(CalibTcState* st);
bool calib_tc_ready(const CalibTcState* st);
bool calib_tc_supported(const CalibTcState* st, const AttnParams& p, int d, int n_seq);
cudaError_t launch_calib_tc(CalibTcState* st, const AttnParams& p, int n_seq, cudaStream_t stream);
cudaError_t launch_calib_tc_steps(CalibTcState* st, const AttnParams& p, int n_seq, const int* steps, const int* t_q,
                                  const int* q_tok0, int n_steps, int q_tokens, int k_tokens, int64_t bias_step_stride,
                                  cudaStream_t stream);
}  // namespace heatkv

using namespace heatkv;

struct heatkv_schedule {
  Schedule s;
};

namespace {

constexpr uint64_t META_ALIGN = 256;
constexpr uint64_t STATUS_BYTES = 256;
// largest cache update (bytes read + written) that rides on the attention launch, per kernel
constexpr uint64_t FUSE_LIMIT_TC_BYTES = 1ull << 30, FUSE_LIMIT_GENERIC_BYTES = 8ull << 20;

// first-fit allocator over [0, size) in abstract units
struct RangeAlloc {
  std::map<uint64_t, uint64_t> free_;   // start -> length
  void reset(uint64_t start, uint64_t len) {
    free_.clear();
    if (len) free_[start] = len;
  }
  bool alloc(uint64_t len, uint64_t* start) {
    for (auto it = free_.begin(); it != free_.end(); ++it) {
      if (it->second >= len) {
        *start = it->first;
        uint64_t rest = it->second - len, s2 = it->first + len;
        free_.erase(it);
        if (rest) free_[s2] = rest;
        return true;
      }
    }
    return false;
  }
  void release(uint64_t start, uint64_t len) {
    auto it = free_.emplace(start, len).first;
    auto nx = std::next(it);
    if (nx != free_.end() && it->first + it->second == nx->first) {
      it->second += nx->second;
      free_.erase(nx);
    }
    if (it != free_.begin()) {
      auto pv = std::prev(it);
      if (pv->first + pv->second == it->first) {
        pv->second += it->second;
        free_.erase(it);
      }
    }
  }
};

struct PlanEntry {
  uint64_t uid = 0;
  Schedule sched;
  Plan plan;
  uint64_t meta_off = 0, meta_len = 0;
  int refs = 0;
};

struct Seq {
  bool open = false;
  int plan = -1;
  uint64_t base_row = 0, rows = 0;
  std::vector<int16_t> done_step;   // per layer: last step whose post-layer update ran (-1 = none)
  std::vector<int16_t> pre_step;    // per layer: last step whose pre-step eviction ran
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

struct heatkv_ctx {
  heatkv_config cfg;
  int c[HEATKV_MAX_K];
  float sm_scale;
  unsigned char* meta = nullptr;
  __nv_bfloat16* k_pool = nullptr;
  __nv_bfloat16* v_pool = nullptr;
  uint64_t pool_rows = 0, meta_bytes = 0;
  // fp8 cache: k_pool / v_pool above are then the bf16 staging rows the attention kernels read (stage_rows of
  // them), and the cache proper is these code pools [pool_rows][d] with one exponent byte per row
  bool fp8 = false;
  uint8_t* k8_pool = nullptr;
  uint8_t* v8_pool = nullptr;
  int8_t* k_exp = nullptr;
  int8_t* v_exp = nullptr;
  uint64_t stage_rows = 0;
  uint32_t* status = nullptr;
  RangeAlloc rows, metas;
  std::vector<std::unique_ptr<PlanEntry>> plans;
  std::vector<Seq> seqs;
  uint64_t reserved_rows = 0, peak_reserved = 0, meta_used = 0;
  uint64_t launches = 0;
  heatkv_kernel_stats kstats = {};             // launches per kernel
  TcState* tc = nullptr;
  CalibTcState* calib_tc = nullptr;
  // key-range splitting of the tensor-memory attention kernel
  float* split_partials = nullptr;
  uint32_t* split_counters = nullptr;
  uint64_t split_slots = 0, split_ctrs = 0;
  int n_sm = 148;
  std::map<uint64_t, SplitChoice> split_choice;   // (plan uid, step, layer, n_seq) -> pieces per head of the attention launch
};

namespace {

int find_or_load_plan(heatkv_ctx* ctx, const Schedule& s, cudaStream_t stream, int* idx) {
  for (size_t i = 0; i < ctx->plans.size(); ++i)
    if (ctx->plans[i] && ctx->plans[i]->uid == s.uid) { *idx = (int)i; return HEATKV_OK; }
  if (s.L != ctx->cfg.L || s.H != ctx->cfg.H || s.K != ctx->cfg.K || s.s != ctx->cfg.s)
    return HEATKV_ERR_SHAPE_MISMATCH;
  for (int i = 0; i < s.K; ++i)
    if (s.t[i] != ctx->cfg.t[i]) return HEATKV_ERR_SHAPE_MISMATCH;
  std::unique_ptr<PlanEntry> e(new (std::nothrow) PlanEntry);
  if (!e) return HEATKV_ERR_HOST_MEMORY;
  e->uid = s.uid;
  e->sched = s;
  int rc = build_plan(s, ctx->cfg.layout, &e->plan, ctx->fp8);
  if (rc != HEATKV_OK) return rc;
  uint64_t bytes = ((uint64_t)e->plan.blob.size() * 4 + META_ALIGN - 1) / META_ALIGN * META_ALIGN;
  uint64_t off = 0;
  bool ok = ctx->metas.alloc(bytes, &off);
  if (!ok) {                                    // drop resident plans nobody uses and retry
    for (auto& pe : ctx->plans)
      if (pe && pe->refs == 0) {
        ctx->metas.release(pe->meta_off, pe->meta_len);
        ctx->meta_used -= pe->meta_len;
        pe.reset();
      }
    ok = ctx->metas.alloc(bytes, &off);
  }
  if (!ok) return HEATKV_ERR_OUT_OF_PAGES;
  e->meta_off = off;
  e->meta_len = bytes;
  if (cudaMemcpyAsync(ctx->meta + off, e->plan.blob.data(), e->plan.blob.size() * 4, cudaMemcpyHostToDevice,
                      stream) != cudaSuccess) {
    ctx->metas.release(off, bytes);
    return HEATKV_ERR_CUDA;
  }
  // the blob is pageable host memory: wait so the vector may be touched again safely
  if (cudaStreamSynchronize(stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  ctx->meta_used += bytes;
  size_t slot = ctx->plans.size();
  for (size_t i = 0; i < ctx->plans.size(); ++i)
    if (!ctx->plans[i]) { slot = i; break; }
  if (slot == ctx->plans.size()) ctx->plans.emplace_back();
  ctx->plans[slot] = std::move(e);
  *idx = (int)slot;
  return HEATKV_OK;
}

inline Seq* get_seq(heatkv_ctx* ctx, int id) {
  if (id < 0 || id >= (int)ctx->seqs.size() || !ctx->seqs[id].open) return nullptr;
  return &ctx->seqs[id];
}

// scales head (l,h) of the sequence holds right now
uint16_t stored_mask(const heatkv_ctx* ctx, const Seq& q, int l, int h) {
  const Schedule& s = ctx->plans[q.plan]->sched;
  int done = q.done_step[l];
  uint16_t m = done >= 0 ? s.keep_mask[s.at(done, l, h)] : 0;
  if (q.pre_step[l] > done && q.pre_step[l] < s.K) m &= s.attn_mask[s.at(q.pre_step[l], l, h)];
  return m;
}

// does the eviction before `step` remove anything from layer l?
bool pre_needed(const Schedule& s, int step, int l) {
  if (step == 0) return false;
  for (int h = 0; h < s.H; ++h)
    if (s.keep_mask[s.at(step - 1, l, h)] & ~s.attn_mask[s.at(step, l, h)]) return true;
  return false;
}

int check_strides(const heatkv_ctx* ctx, const heatkv_strides* st, int t, heatkv_strides* out, bool has_output = true) {
  const int64_t d = ctx->cfg.d, H = ctx->cfg.H;
  if (!st) {
    out->q_tok = out->kv_tok = out->o_tok = d;
    out->q_head = out->kv_head = out->o_head = d * t;
    out->q_seq = out->kv_seq = out->o_seq = d * t * H;
    return HEATKV_OK;
  }
  *out = *st;
  if (!has_output) {                               // nothing is written: the caller may leave o_* unset
    out->o_seq = out->q_seq; out->o_head = out->q_head; out->o_tok = out->q_tok;
  }
  const int64_t* v = &out->q_seq;
  for (int i = 0; i < 9; ++i)
    if (v[i] < 0 || (v[i] & 7)) return HEATKV_ERR_INVALID_ARG;
  if (out->q_tok < d || out->kv_tok < d || out->o_tok < d) return HEATKV_ERR_INVALID_ARG;
  return HEATKV_OK;
}

void fill_common(const heatkv_ctx* ctx, AttnParams* p, const heatkv_strides& s) {
  p->q_seq = s.q_seq; p->q_head = s.q_head; p->q_tok = s.q_tok;
  p->kv_seq = s.kv_seq; p->kv_head = s.kv_head; p->kv_tok = s.kv_tok;
  p->o_seq = s.o_seq; p->o_head = s.o_head; p->o_tok = s.o_tok;
  p->H = ctx->cfg.H; p->K = ctx->cfg.K; p->L = ctx->cfg.L;
  p->scale_log2 = ctx->sm_scale * 1.4426950408889634f;
  for (int i = 0; i < HEATKV_MAX_K; ++i) p->c[i] = i < ctx->cfg.K ? ctx->c[i] : 0x7fffffff;
  p->k_pool = ctx->k_pool; p->v_pool = ctx->v_pool;
  p->status = ctx->status;
}

// Validates ids and per-layer progress for a batched call and fills the SeqRef table.
int gather_seqs(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, SeqRef* refs) {
  if (!seq_ids || n_seq < 1 || n_seq > HEATKV_MAX_BATCH) return HEATKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || step < 0 || step >= ctx->cfg.K) return HEATKV_ERR_INVALID_ARG;
  for (int i = 0; i < n_seq; ++i) {
    Seq* q = get_seq(ctx, seq_ids[i]);
    if (!q) return HEATKV_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (seq_ids[j] == seq_ids[i]) return HEATKV_ERR_INVALID_ARG;
    const PlanEntry& pe = *ctx->plans[q->plan];
    if (q->done_step[layer] != step - 1) return HEATKV_ERR_BAD_STEP_ORDER;
    if (q->pre_step[layer] != step && pre_needed(pe.sched, step, layer)) return HEATKV_ERR_BAD_STEP_ORDER;
    refs[i].plan = reinterpret_cast<const int32_t*>(ctx->meta + pe.meta_off);
    refs[i].base_row = (int64_t)q->base_row;
  }
  return HEATKV_OK;
}

// ---- key-range splitting of the tensor-memory attention kernel -----------------------------------------
// Key tiles of the heads of (step, layer), in the plan's dispatch order (descending key count).
std::vector<int> ordered_tiles(const PlanEntry& pe, int step, int layer, int own_slots) {
  const Schedule& s = pe.sched;
  const PlanHeader& h = pe.plan.header();
  const int32_t* blob = pe.plan.blob.data();
  const int32_t* cnt = blob + h.off_attn_cnt + s.at(step, layer, 0);
  const int32_t* order = blob + h.off_order + s.at(step, layer, 0);
  std::vector<int> t(s.H);
  for (int i = 0; i < s.H; ++i) t[i] = (cnt[order[i]] + own_slots + 1) / 2;
  return t;
}

// Head table of a call whose sequences all follow one schedule (generic kernel): heads in dispatch order with
// the place of their descriptors, so the kernel starts without walking the plan.
void fill_head_table(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int step, int layer, AttnParams* p) {
  p->table_heads = 0;
  const PlanEntry& pe0 = *ctx->plans[ctx->seqs[seq_ids[0]].plan];
  if (pe0.sched.H > 64) return;
  for (int i = 1; i < n_seq; ++i)
    if (ctx->seqs[seq_ids[i]].plan != ctx->seqs[seq_ids[0]].plan) return;
  const PlanHeader& hdr = pe0.plan.header();
  const int32_t* blob = pe0.plan.blob.data();
  const int at = pe0.sched.at(step, layer, 0);
  const int32_t *order = blob + hdr.off_order + at, *cnt = blob + hdr.off_attn_cnt + at, *begin = blob + hdr.off_attn_begin + at;
  for (int i = 0; i < pe0.sched.H; ++i) {
    if (cnt[order[i]] > 32767) return;
    p->table_head[i] = (int16_t)order[i];
    p->table_ndesc[i] = (int16_t)cnt[order[i]];
    p->table_desc_begin[i] = hdr.off_desc + 2 * begin[order[i]];
  }
  p->table_heads = pe0.sched.H;
}

// Fills the splitting fields of the launch parameters.  When the whole call follows one schedule the choice
// is a piece count per head: long heads are cut to a common longest run, and the heads dispatched last may be
// cut further so that the last round of items fills the SMs.  It is cached per (schedule, step, layer, batch
// size).  Calls that mix schedules use one longest run for all of them.
void choose_split(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int step, int layer, AttnParams* p) {
  const int n_qp = (p->t_q + 255) / 256, own_slots = (p->n_own + HEATKV_PAGE_TOKENS - 1) / HEATKV_PAGE_TOKENS;
  const PlanEntry& pe0 = *ctx->plans[ctx->seqs[seq_ids[0]].plan];
  bool one_plan = pe0.sched.H <= 64;
  for (int i = 1; i < n_seq && one_plan; ++i) one_plan = ctx->seqs[seq_ids[i]].plan == ctx->seqs[seq_ids[0]].plan;
  const std::vector<int> tiles = ordered_tiles(pe0, step, layer, own_slots);
  const int H = (int)tiles.size();
  for (int t : tiles) one_plan = one_plan && t <= 32767;
  const uint64_t key = (pe0.uid << 24) ^ ((uint64_t)step << 20) ^ ((uint64_t)layer << 8) ^ (uint64_t)n_seq ^
                       (one_plan ? 0ull : 1ull << 63);
  auto fits = [&](const SplitShape& sh) {
    return (uint64_t)sh.slots * n_seq <= ctx->split_slots &&
           (uint64_t)sh.ctrs * n_seq * SPLIT_CTRS_PER_GROUP <= ctx->split_ctrs;
  };
  auto it = ctx->split_choice.find(key);
  if (it == ctx->split_choice.end())
    it = ctx->split_choice.emplace(key, split_search(tiles, n_qp, n_seq, ctx->n_sm, one_plan, ctx->split_slots,
                                                     ctx->split_ctrs)).first;
  const SplitChoice& ch = it->second;
  SplitShape m = split_shape(tiles, ch.ns, n_qp);
  int lmax = ch.lmax > 0 ? ch.lmax : 0;
  if (!one_plan) {
    // other schedules in the batch follow the same longest run; the per-sequence bounds cover all of them
    auto bounds = [&](int lm) {
      SplitShape b;
      int last_plan = -1;
      for (int i = 0; i < n_seq; ++i) {
        const int pi = ctx->seqs[seq_ids[i]].plan;
        if (pi == last_plan) continue;
        last_plan = pi;
        const std::vector<int> t = ordered_tiles(*ctx->plans[pi], step, layer, own_slots);
        std::vector<int> ns(t.size());
        for (size_t k = 0; k < t.size(); ++k) ns[k] = split_pieces_for(t[k], lm);
        const SplitShape sh = split_shape(t, ns, n_qp);
        b.items = std::max(b.items, sh.items); b.slots = std::max(b.slots, sh.slots); b.ctrs = std::max(b.ctrs, sh.ctrs);
      }
      return b;
    };
    m = bounds(lmax);
    if (lmax > 0 && !fits(m)) {
      lmax = 0;                                             // another schedule in the batch needs more scratch: whole heads
      m = bounds(0);
    }
  }
  // one plan for the whole call (the usual case): its heads, by descending key count, travel in the parameters
  p->table_heads = 0;
  p->longest_piece = 0;
  if (one_plan) {
    const int32_t* order = pe0.plan.blob.data() + pe0.plan.header().off_order + pe0.sched.at(step, layer, 0);
    for (int i = 0; i < H; ++i) {
      p->table_head[i] = (int16_t)order[i];
      p->table_tiles[i] = (int16_t)tiles[i];
      p->table_split[i] = (int16_t)ch.ns[i];
      if (ch.ns[i] > 1) p->longest_piece = std::max(p->longest_piece, (tiles[i] + ch.ns[i] - 1) / ch.ns[i]);
    }
    p->table_heads = H;
  } else {
    p->longest_piece = lmax;
  }
  p->n_seq = n_seq;
  p->split_tiles = lmax;
  p->items_per_seq = m.items;
  p->slots_per_seq = m.slots;
  p->ctrs_per_seq = m.ctrs;
  p->split_partials = ctx->split_partials;
  p->split_counters = ctx->split_counters;
}

}  // namespace

extern "C" {

const char* heatkv_strerror(int status) {
  switch (status) {
    case HEATKV_OK: return "ok";
    case HEATKV_ERR_INVALID_ARG: return "invalid argument";
    case HEATKV_ERR_SHAPE_MISMATCH: return "shape mismatch between schedule, context or call";
    case HEATKV_ERR_BUDGET_INFEASIBLE: return "budget infeasible";
    case HEATKV_ERR_OUT_OF_PAGES: return "cache pool or metadata region exhausted";
    case HEATKV_ERR_BAD_STEP_ORDER: return "call out of generation order";
    case HEATKV_ERR_NAN_SCORE: return "score is not finite";
    case HEATKV_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case HEATKV_ERR_CUDA: return "CUDA runtime error";
    case HEATKV_ERR_HOST_MEMORY: return "host allocation failed";
    case HEATKV_ERR_TOO_LARGE: return "call needs more built-in scratch than the library holds";
    default: return "unknown status";
  }
}

int heatkv_create(const heatkv_config* cfg, void* stream_, heatkv_ctx** out) {
  if (!cfg || !out) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (cfg->L < 1 || cfg->H < 1 || cfg->K < 1 || cfg->K > HEATKV_MAX_K) return HEATKV_ERR_INVALID_ARG;
  if (cfg->d != 64 && cfg->d != 128) return HEATKV_ERR_INVALID_ARG;
  if (cfg->s < 0 || cfg->s > (cfg->K > 1 ? cfg->K - 1 : 0)) return HEATKV_ERR_INVALID_ARG;
  if (cfg->layout != HEATKV_LAYOUT_RAGGED && cfg->layout != HEATKV_LAYOUT_PAGED) return HEATKV_ERR_INVALID_ARG;
  if (cfg->kernel < HEATKV_KERNEL_AUTO || cfg->kernel > HEATKV_KERNEL_TCGEN05) return HEATKV_ERR_INVALID_ARG;
  if (cfg->cache_dtype != HEATKV_CACHE_BF16 && cfg->cache_dtype != HEATKV_CACHE_FP8_E4M3) return HEATKV_ERR_INVALID_ARG;
  const bool fp8 = cfg->cache_dtype == HEATKV_CACHE_FP8_E4M3;
  if (fp8 && cfg->layout != HEATKV_LAYOUT_PAGED) return HEATKV_ERR_INVALID_ARG;
  if (!cfg->arena || (reinterpret_cast<uintptr_t>(cfg->arena) & 1023)) return HEATKV_ERR_INVALID_ARG;
  for (int i = 0; i < cfg->K; ++i)
    if (cfg->t[i] < 1 || cfg->t[i] > (1 << 20)) return HEATKV_ERR_INVALID_ARG;
  std::unique_ptr<heatkv_ctx> ctx(new (std::nothrow) heatkv_ctx);
  if (!ctx) return HEATKV_ERR_HOST_MEMORY;
  ctx->cfg = *cfg;
  for (int i = 0, acc = 0; i < cfg->K; ++i) { acc += cfg->t[i]; ctx->c[i] = acc; }
  ctx->sm_scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / std::sqrt((float)cfg->d);
  uint64_t meta = cfg->meta_bytes;
  if (meta == 0) meta = std::min<uint64_t>(std::max<uint64_t>(cfg->arena_bytes / 16, 1u << 20), 256u << 20);
  meta = (meta + 1023) / 1024 * 1024;
  if (meta < STATUS_BYTES + META_ALIGN || cfg->arena_bytes < meta + 2ull * HEATKV_PAGE_TOKENS * cfg->d * 2)
    return HEATKV_ERR_INVALID_ARG;
  uint64_t scratch = cfg->scratch_bytes;
  if (scratch == 0) scratch = std::min<uint64_t>(cfg->arena_bytes / 8, 128u << 20);
  scratch = (scratch + 1023) / 1024 * 1024;
  if (cfg->arena_bytes < meta + scratch + 2ull * HEATKV_PAGE_TOKENS * cfg->d * 2) return HEATKV_ERR_INVALID_ARG;
  const uint64_t row_bytes = (uint64_t)cfg->d * 2;
  // bf16 cache: the rest of the arena is the K pool and the V pool.  fp8 cache: first the bf16 staging rows
  // (K and V), then the two code pools and the two exponent arrays.
  uint64_t stage_rows = 0, rows = 0;
  if (fp8) {
    uint64_t stage = cfg->stage_bytes ? cfg->stage_bytes : cfg->arena_bytes / 8;
    stage_rows = stage / (2 * row_bytes) / HEATKV_PAGE_TOKENS * HEATKV_PAGE_TOKENS;
    if (stage_rows > 0x7fffffc0ull) stage_rows = 0x7fffffc0ull;
    const uint64_t used = meta + scratch + 2 * stage_rows * row_bytes;
    if (stage_rows == 0 || cfg->arena_bytes < used + 2ull * HEATKV_PAGE_TOKENS * (cfg->d + 1)) return HEATKV_ERR_INVALID_ARG;
    rows = (cfg->arena_bytes - used) / (2ull * (cfg->d + 1));
  } else {
    rows = (cfg->arena_bytes - meta - scratch) / (2 * row_bytes);
  }
  rows = rows / HEATKV_PAGE_TOKENS * HEATKV_PAGE_TOKENS;
  if (rows > 0x7fffffffull) rows = 0x7fffffc0ull;
  ctx->meta = static_cast<unsigned char*>(cfg->arena);
  ctx->meta_bytes = meta;
  ctx->fp8 = fp8;
  ctx->stage_rows = stage_rows;
  ctx->k_pool = reinterpret_cast<__nv_bfloat16*>(ctx->meta + meta + scratch);
  {   // scratch region: arrival counters first (kept zero between launches), then the partial-result slots
    const uint64_t ctr_bytes = std::min<uint64_t>(scratch / 4, 256u << 10) / 1024 * 1024;
    const uint64_t slot_bytes = (uint64_t)tc_split_slot_floats(cfg->d) * 4;
    ctx->split_counters = reinterpret_cast<uint32_t*>(ctx->meta + meta);
    ctx->split_ctrs = ctr_bytes / 4;
    ctx->split_partials = reinterpret_cast<float*>(ctx->meta + meta + ctr_bytes);
    ctx->split_slots = (scratch - ctr_bytes) / slot_bytes;
    if (ctr_bytes && cudaMemsetAsync(ctx->split_counters, 0, ctr_bytes, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n_sm > 0)
      ctx->n_sm = n_sm;
  }
  const uint64_t bf16_rows = fp8 ? stage_rows : rows;           // rows of the two bf16 arrays the attention kernels read
  ctx->v_pool = ctx->k_pool + bf16_rows * cfg->d;
  ctx->pool_rows = rows;
  if (fp8) {
    ctx->k8_pool = reinterpret_cast<uint8_t*>(ctx->v_pool + bf16_rows * cfg->d);
    ctx->v8_pool = ctx->k8_pool + rows * cfg->d;
    ctx->k_exp = reinterpret_cast<int8_t*>(ctx->v8_pool + rows * cfg->d);
    ctx->v_exp = ctx->k_exp + rows;
  }
  ctx->status = reinterpret_cast<uint32_t*>(ctx->meta);
  ctx->rows.reset(0, rows);
  ctx->metas.reset(STATUS_BYTES, meta - STATUS_BYTES);
  // zero the status word and both pools: half-tiles are read whole, rows past a tile's valid
  // count must hold finite values
  if (cudaMemsetAsync(ctx->meta, 0, STATUS_BYTES, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  if (cudaMemsetAsync(ctx->k_pool, 0, 2 * bf16_rows * row_bytes, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  if (fp8 && cudaMemsetAsync(ctx->k8_pool, 0, 2 * rows * ((uint64_t)cfg->d + 1), stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  int rc = tc_create(ctx->cfg, ctx->k_pool, ctx->v_pool, bf16_rows, &ctx->tc);
  if (rc != HEATKV_OK) {
    tc_destroy(ctx->tc);
    return rc;
  }
  // the calibration kernel's half-tile table (key rows cut at source-scale borders) sits in the metadata region
  void* calib_table = nullptr;
  {
    uint64_t bytes = (calib_tc_desc_bytes(ctx->cfg) + META_ALIGN - 1) / META_ALIGN * META_ALIGN, off = 0;
    if (bytes && ctx->metas.alloc(bytes, &off)) {
      calib_table = ctx->meta + off;
      ctx->meta_used += bytes;
    }
  }
  rc = calib_tc_create(ctx->cfg, calib_table, stream, &ctx->calib_tc);
  // A context that may use the tensor-memory kernels must really have them: on a device of compute capability
  // 10.x a failed set-up (driver entry point, tensor maps, shared-memory or register limits) is an error, never
  // a quiet switch to the warp-level kernel.  HEATKV_KERNEL_TCGEN05 demands them on any device.
  if (rc == HEATKV_OK && cfg->kernel != HEATKV_KERNEL_GENERIC) {
    int dev = 0, major = 0;
    const bool sm100 = cudaGetDevice(&dev) == cudaSuccess &&
                       cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10;
    const bool have = tc_ready(ctx->tc) && (calib_tc_ready(ctx->calib_tc) || !calib_table);
    if (!have && (sm100 || cfg->kernel == HEATKV_KERNEL_TCGEN05)) rc = HEATKV_ERR_CUDA;
  }
  if (rc != HEATKV_OK) {
    tc_destroy(ctx->tc);
    calib_tc_destroy(ctx->calib_tc);
    return rc;
  }
  *out = ctx.release();
  return HEATKV_OK;
}

int heatkv_destroy(heatkv_ctx* ctx) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  tc_destroy(ctx->tc);
  calib_tc_destroy(ctx->calib_tc);
  delete ctx;
  return HEATKV_OK;
}

int heatkv_build_schedule(const heatkv_config* cfg, const double* scas, const double* cas, int policy,
                          int accounting, double b, const double* fraction, heatkv_schedule** out) {
  if (!cfg || !out) return HEATKV_ERR_INVALID_ARG;
  std::unique_ptr<heatkv_schedule> s(new (std::nothrow) heatkv_schedule);
  if (!s) return HEATKV_ERR_HOST_MEMORY;
  int rc;
  try {
    rc = build_schedule(*cfg, scas, cas, policy, accounting, b, fraction, &s->s);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (rc != HEATKV_OK) return rc;
  *out = s.release();
  return HEATKV_OK;
}

int heatkv_schedule_free(heatkv_schedule* sch) {
  delete sch;
  return HEATKV_OK;
}

int heatkv_schedule_masks(const heatkv_schedule* sch, uint16_t* attn_mask, uint16_t* keep_mask, int32_t* n_k,
                          int64_t* budget_tokens) {
  if (!sch) return HEATKV_ERR_INVALID_ARG;
  const Schedule& s = sch->s;
  if (attn_mask) std::memcpy(attn_mask, s.attn_mask.data(), s.attn_mask.size() * 2);
  if (keep_mask) std::memcpy(keep_mask, s.keep_mask.data(), s.keep_mask.size() * 2);
  if (n_k) std::memcpy(n_k, s.n_k.data(), s.n_k.size() * 4);
  if (budget_tokens) *budget_tokens = s.budget;
  return HEATKV_OK;
}

int heatkv_schedule_footprint(const heatkv_schedule* sch, int layout, int64_t* peak_tokens, int64_t* reserved_rows) {
  if (!sch) return HEATKV_ERR_INVALID_ARG;
  Plan plan;
  int rc;
  try {
    rc = build_plan(sch->s, layout, &plan);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (rc != HEATKV_OK) return rc;
  if (peak_tokens) *peak_tokens = plan.peak_tokens;
  if (reserved_rows) *reserved_rows = plan.reserved_rows;
  return HEATKV_OK;
}

int heatkv_schedule_plan(const heatkv_schedule* sch, int layout, int32_t* words, int64_t* n_words) {
  if (!sch || !n_words) return HEATKV_ERR_INVALID_ARG;
  Plan plan;
  int rc;
  try {
    rc = build_plan(sch->s, layout, &plan);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (rc != HEATKV_OK) return rc;
  if (words) {
    if (*n_words < (int64_t)plan.blob.size()) return HEATKV_ERR_INVALID_ARG;
    std::memcpy(words, plan.blob.data(), plan.blob.size() * 4);
  }
  *n_words = (int64_t)plan.blob.size();
  return HEATKV_OK;
}

int heatkv_schedule_plan_fp8(const heatkv_schedule* sch, int32_t* words, int64_t* n_words, int64_t* stage_rows) {
  if (!sch || !n_words) return HEATKV_ERR_INVALID_ARG;
  Plan plan;
  int rc;
  try {
    rc = build_plan(sch->s, HEATKV_LAYOUT_PAGED, &plan, true);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (rc != HEATKV_OK) return rc;
  if (words) {
    if (*n_words < (int64_t)plan.blob.size()) return HEATKV_ERR_INVALID_ARG;
    std::memcpy(words, plan.blob.data(), plan.blob.size() * 4);
  }
  *n_words = (int64_t)plan.blob.size();
  if (stage_rows) *stage_rows = plan.stage_rows;
  return HEATKV_OK;
}

int heatkv_seq_open(heatkv_ctx* ctx, const heatkv_schedule* sch, void* stream_, int* seq_id) {
  if (!ctx || !sch || !seq_id) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int pi = -1, rc;
  try {
    rc = find_or_load_plan(ctx, sch->s, stream, &pi);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (rc != HEATKV_OK) return rc;
  PlanEntry& pe = *ctx->plans[pi];
  uint64_t start = 0;
  if (!ctx->rows.alloc((uint64_t)pe.plan.reserved_rows, &start)) return HEATKV_ERR_OUT_OF_PAGES;
  int id = -1;
  for (size_t i = 0; i < ctx->seqs.size(); ++i)
    if (!ctx->seqs[i].open) { id = (int)i; break; }
  if (id < 0) { ctx->seqs.emplace_back(); id = (int)ctx->seqs.size() - 1; }
  Seq& q = ctx->seqs[id];
  q.open = true;
  q.plan = pi;
  q.base_row = start;
  q.rows = (uint64_t)pe.plan.reserved_rows;
  q.done_step.assign(ctx->cfg.L, -1);
  q.pre_step.assign(ctx->cfg.L, -1);
  pe.refs++;
  ctx->reserved_rows += q.rows;
  ctx->peak_reserved = std::max(ctx->peak_reserved, ctx->reserved_rows);
  *seq_id = id;
  return HEATKV_OK;
}

int heatkv_seq_close(heatkv_ctx* ctx, int seq_id) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q) return HEATKV_ERR_INVALID_ARG;
  ctx->rows.release(q->base_row, q->rows);
  ctx->reserved_rows -= q->rows;
  ctx->plans[q->plan]->refs--;
  q->open = false;
  return HEATKV_OK;
}

// Attention of one layer at one step; with `with_update` the cache update after the layer follows: inside the
// same launch in the paged layout (the plan never puts the new scale on a page this step still reads), as
// the separate kernels otherwise.
static int attention_impl(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, const void* q,
                          const void* k_new, const void* v_new, const heatkv_strides* st, const float* seg_bias,
                          void* out, void* stream_, bool with_update) {
  if (!ctx || !q || !k_new || !v_new || !out) return HEATKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  int rc = gather_seqs(ctx, seq_ids, n_seq, layer, step, p.seqs);
  if (rc != HEATKV_OK) return rc;
  heatkv_strides s;
  rc = check_strides(ctx, st, ctx->cfg.t[step], &s);
  if (rc != HEATKV_OK) return rc;
  fill_common(ctx, &p, s);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.seg_bias = seg_bias;
  p.t_q = p.n_own = ctx->cfg.t[step];
  p.step = step;
  p.layer = layer;
  const bool stores = step + 1 < ctx->cfg.K;                  // the last scale is never cached
  const int choice = ctx->cfg.kernel;
  bool use_tc = choice != HEATKV_KERNEL_GENERIC && tc_supported(ctx->tc, p, ctx->cfg.d, n_seq, false);
  // AUTO: steps of 256 queries and more, and steps of 128 and more once the call holds 64 (sequence, head) units:
  // from there on the warp-level kernel is bound by its mma.sync rate (144 queries, 128 units: 52 us against 23 us)
  if (choice == HEATKV_KERNEL_AUTO && !(p.t_q >= 256 || (p.t_q >= 128 && (int64_t)n_seq * ctx->cfg.H >= 64))) use_tc = false;
  if (choice == HEATKV_KERNEL_TCGEN05 && !use_tc) return HEATKV_ERR_INVALID_ARG;   // never a silent substitute
  if (ctx->fp8) {
    // The attention kernels read bf16 rows: expand the visible head-scales of this (layer, step) from the code
    // pools into the staging rows first (every sequence gets the rows its plan needs, one after the other),
    // then point the kernels' row numbering at them.
    CopyParams cp;
    std::memset(&cp, 0, sizeof(cp));
    cp.k_pool = ctx->k_pool; cp.v_pool = ctx->v_pool;
    cp.k8_pool = ctx->k8_pool; cp.v8_pool = ctx->v8_pool; cp.k_exp = ctx->k_exp; cp.v_exp = ctx->v_exp;
    cp.step = step; cp.layer = layer; cp.H = ctx->cfg.H; cp.K = ctx->cfg.K; cp.L = ctx->cfg.L; cp.d = ctx->cfg.d;
    uint64_t next = 0;
    int slots = 0;
    for (int i = 0; i < n_seq; ++i) {
      const PlanEntry& pe = *ctx->plans[ctx->seqs[seq_ids[i]].plan];
      const PlanHeader& hd = pe.plan.header();
      const int32_t* blob = pe.plan.blob.data();
      const size_t u0 = pe.sched.at(step, layer, 0), u1 = pe.sched.at(step, layer, pe.sched.H - 1);
      const int count = blob[hd.off_attn_begin + u1] + blob[hd.off_attn_cnt + u1] - blob[hd.off_attn_begin + u0];
      slots = std::max(slots, count);
      cp.seqs[i] = p.seqs[i];
      cp.stage_base[i] = (int32_t)next;
      next += (uint64_t)count * HEATKV_PAGE_TOKENS;
    }
    if (next > ctx->stage_rows) return HEATKV_ERR_OUT_OF_PAGES;
    if (launch_dequant_fp8(cp, n_seq, slots, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
    if (slots > 0) {
      ctx->launches += 1;
      ctx->kstats.other += 1;
    }
    for (int i = 0; i < n_seq; ++i) {
      p.pool_base[i] = (int32_t)p.seqs[i].base_row;         // where a cache update riding on the launch writes
      p.seqs[i].base_row = cp.stage_base[i];
    }
    p.k8_pool = ctx->k8_pool; p.v8_pool = ctx->v8_pool; p.k_exp = ctx->k_exp; p.v_exp = ctx->v_exp;
  }
  // fp8 cache: only the generic kernel carries the quantising update (the same branch in the tensor-memory kernel's
  // spare warps measured 1.5 % on the bf16 path's largest launch and 8 % on its smallest)
  bool fuse = with_update && stores && ctx->cfg.layout == HEATKV_LAYOUT_PAGED && !(ctx->fp8 && use_tc);
  if (fuse) {
    // The tensor-memory kernel copies the new rows with two spare warps per SM beside the attention work, so
    // the update rides along whatever its size.  The generic kernel carries it as extra CTAs of its own
    // footprint, which only pays while the update is a launch-bound copy; a larger one keeps its own kernel.
    const uint64_t limit = use_tc ? FUSE_LIMIT_TC_BYTES : FUSE_LIMIT_GENERIC_BYTES;
    uint64_t storing = 0;
    for (int i = 0; i < n_seq; ++i) {
      const PlanEntry& pe = *ctx->plans[ctx->seqs[seq_ids[i]].plan];
      const int32_t* cnt = pe.plan.blob.data() + pe.plan.header().off_app_cnt + pe.sched.at(step, layer, 0);
      for (int hd = 0; hd < pe.sched.H; ++hd) storing += cnt[hd] > 0;
    }
    fuse = storing * (uint64_t)ctx->cfg.t[step] * ctx->cfg.d * 8 <= limit;
    // (fp8 cache: a step that does not ride along goes through heatkv_append_compact below, which takes the
    // sequences' pool rows from the context, not from p)
  }
  if (fuse) p.append_tiles = (ctx->cfg.t[step] + HEATKV_PAGE_TOKENS - 1) / HEATKV_PAGE_TOKENS + 1;
  cudaError_t e;
  if (use_tc) {
    int n = 0;
    try {
      choose_split(ctx, seq_ids, n_seq, step, layer, &p);
    } catch (const std::bad_alloc&) {
      return HEATKV_ERR_HOST_MEMORY;
    }
    e = launch_attn_tc(ctx->tc, p, ctx->cfg.d, n_seq, false, stream, &n);
    ctx->launches += n;
    ctx->kstats.attention_tcgen05 += n;
  } else {
    fill_head_table(ctx, seq_ids, n_seq, step, layer, &p);
    e = launch_attn_generic(p, ctx->cfg.d, n_seq, false, stream);
    ctx->launches += 1;
    ctx->kstats.attention_generic += 1;
  }
  if (e != cudaSuccess) return HEATKV_ERR_CUDA;
  if (!with_update) return HEATKV_OK;
  if (fuse || !stores) {
    for (int i = 0; i < n_seq; ++i) ctx->seqs[seq_ids[i]].done_step[layer] = (int16_t)step;
    return HEATKV_OK;
  }
  return heatkv_append_compact(ctx, seq_ids, n_seq, layer, step, k_new, v_new, st, stream_);
}

int heatkv_scale_attention(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, const void* q,
                           const void* k_new, const void* v_new, const heatkv_strides* st, const float* seg_bias,
                           void* out, void* stream_) {
  return attention_impl(ctx, seq_ids, n_seq, layer, step, q, k_new, v_new, st, seg_bias, out, stream_, false);
}

int heatkv_attention_append(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, const void* q,
                            const void* k_new, const void* v_new, const heatkv_strides* st, const float* seg_bias,
                            void* out, void* stream_) {
  return attention_impl(ctx, seq_ids, n_seq, layer, step, q, k_new, v_new, st, seg_bias, out, stream_, true);
}

int heatkv_attention_split(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, int32_t* split_tiles,
                           int32_t* items) {
  if (!ctx || !seq_ids || n_seq < 1 || n_seq > HEATKV_MAX_BATCH) return HEATKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || step < 0 || step >= ctx->cfg.K) return HEATKV_ERR_INVALID_ARG;
  for (int i = 0; i < n_seq; ++i)
    if (!get_seq(ctx, seq_ids[i])) return HEATKV_ERR_INVALID_ARG;
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  p.t_q = p.n_own = ctx->cfg.t[step];
  try {
    choose_split(ctx, seq_ids, n_seq, step, layer, &p);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (split_tiles) *split_tiles = p.longest_piece;
  if (items) *items = p.items_per_seq * n_seq;
  return HEATKV_OK;
}

int heatkv_calibrate_scores(heatkv_ctx* ctx, int layer, int step, int n_seq, const void* q, const void* k_full,
                            const void* v_full, const heatkv_strides* st, const float* seg_bias, float* beta_accum,
                            void* out, void* stream_) {
  if (!ctx || !q || !k_full || !beta_accum) return HEATKV_ERR_INVALID_ARG;
  if (out && !v_full) return HEATKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_full) || !aligned16(v_full) || !aligned16(out)) return HEATKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || step < 0 || step >= ctx->cfg.K || n_seq < 1 || n_seq > 65535)
    return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  heatkv_strides s;
  if (!st) {   // dense: q/out [n_seq,H,t,d], k/v [n_seq,H,c[step],d]
    const int64_t d = ctx->cfg.d, H = ctx->cfg.H, t = ctx->cfg.t[step], c = ctx->c[step];
    s.q_tok = s.kv_tok = s.o_tok = d;
    s.q_head = s.o_head = d * t; s.kv_head = d * c;
    s.q_seq = s.o_seq = d * t * H; s.kv_seq = d * c * H;
  } else {
    int rc = check_strides(ctx, st, ctx->cfg.t[step], &s, out != nullptr);
    if (rc != HEATKV_OK) return rc;
  }
  fill_common(ctx, &p, s);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_full);
  p.v_new = out ? static_cast<const __nv_bfloat16*>(v_full) : nullptr;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.seg_bias = seg_bias;
  p.t_q = ctx->cfg.t[step];
  p.n_own = ctx->c[step];
  p.step = step;
  p.layer = layer;
  p.beta_row = beta_accum + (((int64_t)layer * ctx->cfg.H) * ctx->cfg.K + step) * ctx->cfg.K;
  // without an attention output the pass is S = Q K^T plus bookkeeping: the tensor-memory kernel takes it
  const int choice = ctx->cfg.kernel;
  bool use_tc = !out && choice != HEATKV_KERNEL_GENERIC && calib_tc_supported(ctx->calib_tc, p, ctx->cfg.d, n_seq);
  if (choice == HEATKV_KERNEL_AUTO && p.t_q < 256) use_tc = false;
  cudaError_t e = use_tc ? launch_calib_tc(ctx->calib_tc, p, n_seq, stream)
                         : launch_attn_generic(p, ctx->cfg.d, n_seq, true, stream);
  ctx->launches += 1;
  (use_tc ? ctx->kstats.calibration_tcgen05 : ctx->kstats.calibration_generic) += 1;
  return e == cudaSuccess ? HEATKV_OK : HEATKV_ERR_CUDA;
}

int heatkv_calibrate_scores_steps(heatkv_ctx* ctx, int layer, int step_begin, int step_end, int n_seq, const void* q_all,
                                  const void* k_all, const heatkv_strides* st, const float* seg_bias, float* beta_accum,
                                  void* stream_) {
  if (!ctx || !q_all || !k_all || !beta_accum) return HEATKV_ERR_INVALID_ARG;
  if (!aligned16(q_all) || !aligned16(k_all)) return HEATKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || step_begin < 0 || step_begin >= step_end || step_end > ctx->cfg.K || n_seq < 1 ||
      n_seq > 65535)
    return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int64_t d = ctx->cfg.d, H = ctx->cfg.H, K = ctx->cfg.K, tokens = ctx->c[step_end - 1];
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  heatkv_strides s;
  if (!st) {   // dense: [n_seq, H, tokens, d]
    s.q_tok = s.kv_tok = s.o_tok = d;
    s.q_head = s.kv_head = s.o_head = d * tokens;
    s.q_seq = s.kv_seq = s.o_seq = d * tokens * H;
  } else {
    int rc = check_strides(ctx, st, (int)tokens, &s, false);
    if (rc != HEATKV_OK) return rc;
  }
  fill_common(ctx, &p, s);
  p.layer = layer;
  float* beta_layer = beta_accum + (int64_t)layer * H * K * K;
  // the steps the tensor-memory kernel takes, as one launch
  int big[HEATKV_MAX_K], big_t[HEATKV_MAX_K], big_tok0[HEATKV_MAX_K], n_big = 0;
  const int choice = ctx->cfg.kernel;
  p.q = static_cast<const __nv_bfloat16*>(q_all);
  p.k_new = static_cast<const __nv_bfloat16*>(k_all);
  const bool tc_ok = choice != HEATKV_KERNEL_GENERIC && calib_tc_supported(ctx->calib_tc, p, ctx->cfg.d, n_seq);
  // the small steps share one launch of the generic kernel (their query tiles side by side), longest first
  AttnParams g = p;
  g.cal_n = 0;
  for (int k = step_end - 1; k >= step_begin; --k) {
    const bool use_tc = tc_ok && !(choice == HEATKV_KERNEL_AUTO && ctx->cfg.t[k] < 256);
    if (use_tc) {
      big[n_big] = k; big_t[n_big] = ctx->cfg.t[k]; big_tok0[n_big] = ctx->c[k] - ctx->cfg.t[k];
      ++n_big;
      continue;
    }
    g.cal_step[g.cal_n] = k;
    g.cal_tile_begin[g.cal_n + 1] = g.cal_tile_begin[g.cal_n] + (ctx->cfg.t[k] + 63) / 64;
    ++g.cal_n;
  }
  if (g.cal_n > 0) {
    g.seg_bias = seg_bias;
    g.cal_bias_stride = H * K;
    g.beta_row = beta_layer;
    if (launch_attn_generic(g, ctx->cfg.d, n_seq, true, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
    ctx->launches += 1;
    ctx->kstats.calibration_generic += 1;
  }
  if (n_big > 0) {
    p.seg_bias = seg_bias;
    p.beta_row = beta_layer;
    if (launch_calib_tc_steps(ctx->calib_tc, p, n_seq, big, big_t, big_tok0, n_big, (int)tokens, (int)tokens,
                              seg_bias ? H * K : 0, stream) != cudaSuccess)
      return HEATKV_ERR_CUDA;
    ctx->launches += 1;
    ctx->kstats.calibration_tcgen05 += 1;
  }
  return HEATKV_OK;
}

int heatkv_calibrate_scores_static(heatkv_ctx* ctx, int layer, int step, int n_seq, const void* q, const void* k_full,
                                   const heatkv_strides* st, const float* seg_bias, float* beta_accum, void* stream_) {
  if (!ctx || !q || !k_full || !beta_accum) return HEATKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_full)) return HEATKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || step < 0 || step >= ctx->cfg.K || n_seq < 1 || n_seq > 65535)
    return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  heatkv_strides s;
  if (!st) {   // dense: q [n_seq,H,t,d], k [n_seq,H,c[step],d]
    const int64_t d = ctx->cfg.d, H = ctx->cfg.H, t = ctx->cfg.t[step], c = ctx->c[step];
    s.q_tok = s.kv_tok = s.o_tok = d;
    s.q_head = s.o_head = d * t; s.kv_head = d * c;
    s.q_seq = s.o_seq = d * t * H; s.kv_seq = d * c * H;
  } else {
    int rc = check_strides(ctx, st, ctx->cfg.t[step], &s, false);
    if (rc != HEATKV_OK) return rc;
  }
  fill_common(ctx, &p, s);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_full);
  p.seg_bias = seg_bias;
  p.t_q = ctx->cfg.t[step];
  p.n_own = ctx->c[step];
  p.step = step;
  p.layer = layer;
  p.beta_row = beta_accum + (((int64_t)layer * ctx->cfg.H) * ctx->cfg.K + step) * ctx->cfg.K;
  bool too_large = false;
  cudaError_t e = launch_calibrate_static(p, ctx->cfg.d, n_seq, stream, &too_large);
  if (too_large) return HEATKV_ERR_TOO_LARGE;
  if (e != cudaSuccess) return HEATKV_ERR_CUDA;
  ctx->launches += 2;
  ctx->kstats.calibration_generic += 1;
  ctx->kstats.other += 1;
  return HEATKV_OK;
}

int heatkv_finalize_scores(heatkv_ctx* ctx, const float* beta_accum, int n_samples, double* beta, double* scas,
                           double* cas, void* stream_) {
  if (!ctx || !beta_accum || n_samples < 1) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int L = ctx->cfg.L, H = ctx->cfg.H, K = ctx->cfg.K, s = ctx->cfg.s;
  const size_t n = (size_t)L * H * K * K;
  std::vector<float> host;
  try {
    host.resize(n);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  if (cudaMemcpyAsync(host.data(), beta_accum, n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return HEATKV_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  for (size_t i = 0; i < n; ++i)
    if (!std::isfinite(host[i])) return HEATKV_ERR_NAN_SCORE;
  const double inv = 1.0 / (double)n_samples;
  for (int hd = 0; hd < L * H; ++hd) {
    const float* b = &host[(size_t)hd * K * K];
    if (beta)
      for (int i = 0; i < K * K; ++i) beta[(size_t)hd * K * K + i] = (double)b[i] * inv;
    if (cas) {   // Eq. 3: last scale's mass on the cached non-sink scales, normaliser 1/(K-s)
      double acc = 0.0;
      for (int tau = s; tau <= K - 2; ++tau) acc += (double)b[(size_t)(K - 1) * K + tau] * inv;
      cas[hd] = acc / (double)(K - s);
    }
    if (scas)    // Eq. 4: mean over the future scales tau > k of beta[tau][k], for s <= k <= K-2 (0-based)
      for (int k = 0; k < K; ++k) {
        double acc = 0.0;
        if (k >= s && k <= K - 2) {
          for (int tau = k + 1; tau < K; ++tau) acc += (double)b[(size_t)tau * K + k] * inv;
          acc /= (double)(K - 1 - k);
        }
        scas[(size_t)hd * K + k] = acc;
      }
  }
  return HEATKV_OK;
}

// Does the plan move any row at `step` in layers [l0, l1)?  phase 0: the eviction before the step (E_step),
// phase 1: the eviction after a layer (G_step minus A_step of that layer).  The ragged layout launches its compaction
// kernel only then.
static bool plan_moves_rows(const Plan& pl, int phase, int step, int l0, int l1) {
  const PlanHeader& hd = pl.header();
  if (hd.n_move <= 0) return false;
  const int32_t* cnt = pl.blob.data() + (phase == 0 ? hd.off_pre_cnt : hd.off_post_cnt);
  for (int l = l0; l < l1; ++l)
    for (int h = 0; h < hd.H; ++h)
      if (cnt[((size_t)step * hd.L + l) * hd.H + h] > 0) return true;
  return false;
}

int heatkv_append_compact(heatkv_ctx* ctx, const int* seq_ids, int n_seq, int layer, int step, const void* k_new,
                          const void* v_new, const heatkv_strides* st, void* stream_) {
  if (!ctx || !seq_ids || n_seq < 1 || n_seq > HEATKV_MAX_BATCH) return HEATKV_ERR_INVALID_ARG;
  if (step < 0 || step >= ctx->cfg.K || layer >= ctx->cfg.L) return HEATKV_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int L = ctx->cfg.L;
  CopyParams p;
  std::memset(&p, 0, sizeof(p));
  p.k_pool = ctx->k_pool; p.v_pool = ctx->v_pool;
  p.step = step; p.H = ctx->cfg.H; p.K = ctx->cfg.K; p.L = L; p.d = ctx->cfg.d;
  p.t_k = ctx->cfg.t[step];

  if (!k_new) {
    // ---- eviction before the step starts (E_step)
    const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? L : layer + 1;
    bool moves = false;
    for (int i = 0; i < n_seq; ++i) {
      Seq* q = get_seq(ctx, seq_ids[i]);
      if (!q) return HEATKV_ERR_INVALID_ARG;
      for (int j = 0; j < i; ++j)
        if (seq_ids[j] == seq_ids[i]) return HEATKV_ERR_INVALID_ARG;
      for (int l = l0; l < l1; ++l)
        if (q->done_step[l] != step - 1 || q->pre_step[l] >= step) return HEATKV_ERR_BAD_STEP_ORDER;
      const PlanEntry& pe = *ctx->plans[q->plan];
      p.seqs[i].plan = reinterpret_cast<const int32_t*>(ctx->meta + pe.meta_off);
      p.seqs[i].base_row = (int64_t)q->base_row;
      moves |= plan_moves_rows(pe.plan, 0, step, l0, l1);
    }
    if (ctx->cfg.layout == HEATKV_LAYOUT_RAGGED && moves && step > 0) {
      p.phase = 0; p.layer_begin = l0; p.n_layers = l1 - l0; p.layer = l0;
      if (launch_compact(p, n_seq, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
      ctx->launches += 1;
      ctx->kstats.compact += 1;
    }
    for (int i = 0; i < n_seq; ++i)
      for (int l = l0; l < l1; ++l) ctx->seqs[seq_ids[i]].pre_step[l] = (int16_t)step;
    return HEATKV_OK;
  }

  // ---- update after the layer ran: drop G_step \ A_step of this layer, store the new scale
  if (!aligned16(k_new) || !aligned16(v_new)) return HEATKV_ERR_INVALID_ARG;
  int rc = gather_seqs(ctx, seq_ids, n_seq, layer, step, p.seqs);
  if (rc != HEATKV_OK) return rc;
  heatkv_strides s;
  rc = check_strides(ctx, st, ctx->cfg.t[step], &s, false);
  if (rc != HEATKV_OK) return rc;
  p.kv_seq = s.kv_seq; p.kv_head = s.kv_head; p.kv_tok = s.kv_tok;
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.layer = layer;
  if (step + 1 < ctx->cfg.K) {                  // the last scale is never cached
    if (ctx->cfg.layout == HEATKV_LAYOUT_RAGGED) {
      bool moves = false;
      for (int i = 0; i < n_seq; ++i) moves |= plan_moves_rows(ctx->plans[ctx->seqs[seq_ids[i]].plan]->plan, 1, step, layer, layer + 1);
      if (moves) {
        p.phase = 1; p.layer_begin = layer; p.n_layers = 1;
        if (launch_compact(p, n_seq, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
        ctx->launches += 1;
        ctx->kstats.compact += 1;
      }
    }
    p.k8_pool = ctx->k8_pool; p.v8_pool = ctx->v8_pool; p.k_exp = ctx->k_exp; p.v_exp = ctx->v_exp;
    if ((ctx->fp8 ? launch_append_fp8(p, n_seq, stream) : launch_append(p, n_seq, stream)) != cudaSuccess) return HEATKV_ERR_CUDA;
    ctx->launches += 1;
    ctx->kstats.append += 1;
  }
  for (int i = 0; i < n_seq; ++i) ctx->seqs[seq_ids[i]].done_step[layer] = (int16_t)step;
  return HEATKV_OK;
}

int heatkv_cache_bytes(heatkv_ctx* ctx, int seq_id, uint64_t* actual, uint64_t* closed_form) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q) return HEATKV_ERR_INVALID_ARG;
  const PlanEntry& pe = *ctx->plans[q->plan];
  const Schedule& s = pe.sched;
  const PlanHeader& hd = pe.plan.header();
  const int32_t* blob = pe.plan.blob.data();
  const Desc* descs = reinterpret_cast<const Desc*>(blob + hd.off_desc);
  uint64_t tokens = 0, placed = 0;
  for (int l = 0; l < s.L; ++l)
    for (int h = 0; h < s.H; ++h) {
      const uint16_t m = stored_mask(ctx, *q, l, h);
      for (int i = 0; i < s.K; ++i) {
        if (!((m >> i) & 1)) continue;
        tokens += s.t[i];
        // rows the plan gave this head-scale when it was appended (valid rows of its destination half-tiles)
        const size_t u = s.at(i, l, h);
        const int32_t b0 = blob[hd.off_app_begin + u], cnt = blob[hd.off_app_cnt + u];
        for (int j = 0; j < cnt; ++j) placed += descs[b0 + j].meta & 0xff;
      }
    }
  const uint64_t row_bytes = ctx->fp8 ? (uint64_t)ctx->cfg.d + 1 : (uint64_t)ctx->cfg.d * 2;   // per row of K or of V
  if (actual) *actual = placed * row_bytes * 2;
  if (closed_form) *closed_form = tokens * row_bytes * 2;
  return HEATKV_OK;
}

int heatkv_seq_reservation(heatkv_ctx* ctx, int seq_id, uint64_t* first_row, uint64_t* rows) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q) return HEATKV_ERR_INVALID_ARG;
  if (first_row) *first_row = q->base_row;
  if (rows) *rows = q->rows;
  return HEATKV_OK;
}

int heatkv_retained_indices(heatkv_ctx* ctx, int seq_id, int layer, int head, int32_t* idx, int* n) {
  if (!ctx || !n) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q || layer < 0 || layer >= ctx->cfg.L || head < 0 || head >= ctx->cfg.H) return HEATKV_ERR_INVALID_ARG;
  const Schedule& s = ctx->plans[q->plan]->sched;
  uint16_t m = stored_mask(ctx, *q, layer, head);
  int cnt = 0;
  for (int i = 0; i < s.K; ++i)
    if ((m >> i) & 1)
      for (int j = 0; j < s.t[i]; ++j) {
        if (idx) idx[cnt] = s.c[i] - s.t[i] + j;
        ++cnt;
      }
  *n = cnt;
  return HEATKV_OK;
}

int heatkv_export_head(heatkv_ctx* ctx, int seq_id, int layer, int head, void* k_out, void* v_out, void* stream_) {
  if (!ctx || !k_out || !v_out || ctx->fp8) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q || layer < 0 || layer >= ctx->cfg.L || head < 0 || head >= ctx->cfg.H) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const PlanEntry& pe = *ctx->plans[q->plan];
  const Schedule& s = pe.sched;
  const PlanHeader& h = pe.plan.header();
  const int32_t* blob = pe.plan.blob.data();
  const Desc* descs = reinterpret_cast<const Desc*>(blob + h.off_desc);
  const uint16_t m = stored_mask(ctx, *q, layer, head);
  const size_t row_bytes = (size_t)ctx->cfg.d * 2;
  size_t out_row = 0;
  int64_t dense = pe.plan.head_base[layer * s.H + head];
  for (int i = 0; i < s.K; ++i) {
    if (!((m >> i) & 1)) continue;
    if (ctx->cfg.layout == HEATKV_LAYOUT_PAGED) {
      // a head-scale keeps the rows it was appended to for its whole life
      size_t u = s.at(i, layer, head);
      const int32_t b0 = blob[h.off_app_begin + u], cnt = blob[h.off_app_cnt + u];
      for (int j = 0; j < cnt; ++j) {
        const Desc& dsc = descs[b0 + j];
        const int nrow = dsc.meta & 0xff;
        const int64_t row = (int64_t)q->base_row + dsc.row;
        if (cudaMemcpyAsync(static_cast<char*>(k_out) + out_row * row_bytes, ctx->k_pool + row * ctx->cfg.d,
                            nrow * row_bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
            cudaMemcpyAsync(static_cast<char*>(v_out) + out_row * row_bytes, ctx->v_pool + row * ctx->cfg.d,
                            nrow * row_bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
          return HEATKV_ERR_CUDA;
        out_row += nrow;
      }
    } else {
      const int64_t row = (int64_t)q->base_row + dense;
      if (cudaMemcpyAsync(static_cast<char*>(k_out) + out_row * row_bytes, ctx->k_pool + row * ctx->cfg.d,
                          s.t[i] * row_bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
          cudaMemcpyAsync(static_cast<char*>(v_out) + out_row * row_bytes, ctx->v_pool + row * ctx->cfg.d,
                          s.t[i] * row_bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return HEATKV_ERR_CUDA;
      out_row += s.t[i];
      dense += s.t[i];
    }
  }
  return HEATKV_OK;
}

int heatkv_export_head_fp8(heatkv_ctx* ctx, int seq_id, int layer, int head, void* k_codes, void* v_codes, void* k_exps,
                           void* v_exps, void* stream_) {
  if (!ctx || !k_codes || !v_codes || !k_exps || !v_exps || !ctx->fp8) return HEATKV_ERR_INVALID_ARG;
  Seq* q = get_seq(ctx, seq_id);
  if (!q || layer < 0 || layer >= ctx->cfg.L || head < 0 || head >= ctx->cfg.H) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const PlanEntry& pe = *ctx->plans[q->plan];
  const Schedule& s = pe.sched;
  const PlanHeader& h = pe.plan.header();
  const int32_t* blob = pe.plan.blob.data();
  const Desc* descs = reinterpret_cast<const Desc*>(blob + h.off_desc);
  const uint16_t m = stored_mask(ctx, *q, layer, head);
  const size_t d = (size_t)ctx->cfg.d;
  size_t out_row = 0;
  for (int i = 0; i < s.K; ++i) {
    if (!((m >> i) & 1)) continue;
    // a head-scale keeps the rows it was appended to for its whole life (append descriptors carry pool rows)
    const size_t u = s.at(i, layer, head);
    const int32_t b0 = blob[h.off_app_begin + u], cnt = blob[h.off_app_cnt + u];
    for (int j = 0; j < cnt; ++j) {
      const Desc& dsc = descs[b0 + j];
      const size_t nrow = (size_t)(dsc.meta & 0xff);
      const int64_t row = (int64_t)q->base_row + dsc.row;
      if (cudaMemcpyAsync(static_cast<char*>(k_codes) + out_row * d, ctx->k8_pool + row * d, nrow * d,
                          cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
          cudaMemcpyAsync(static_cast<char*>(v_codes) + out_row * d, ctx->v8_pool + row * d, nrow * d,
                          cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
          cudaMemcpyAsync(static_cast<char*>(k_exps) + out_row, ctx->k_exp + row, nrow, cudaMemcpyDeviceToDevice,
                          stream) != cudaSuccess ||
          cudaMemcpyAsync(static_cast<char*>(v_exps) + out_row, ctx->v_exp + row, nrow, cudaMemcpyDeviceToDevice,
                          stream) != cudaSuccess)
        return HEATKV_ERR_CUDA;
      out_row += nrow;
    }
  }
  return HEATKV_OK;
}

int heatkv_allocator_stats(heatkv_ctx* ctx, heatkv_alloc_stats* out) {
  if (!ctx || !out) return HEATKV_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->pool_rows = ctx->pool_rows;
  out->reserved_rows = ctx->reserved_rows;
  out->peak_reserved_rows = ctx->peak_reserved;
  out->meta_bytes_used = ctx->meta_used;
  for (size_t i = 0; i < ctx->seqs.size(); ++i)
    if (ctx->seqs[i].open) {
      out->open_seqs++;
      uint64_t bytes = 0;
      heatkv_cache_bytes(ctx, (int)i, nullptr, &bytes);
      out->used_tokens += bytes / (ctx->fp8 ? ((uint64_t)ctx->cfg.d + 1) * 2 : (uint64_t)ctx->cfg.d * 4);
    }
  for (auto& pe : ctx->plans)
    if (pe) out->plans++;
  return HEATKV_OK;
}

int heatkv_launch_count(heatkv_ctx* ctx, uint64_t* n) {
  if (!ctx || !n) return HEATKV_ERR_INVALID_ARG;
  *n = ctx->launches;
  return HEATKV_OK;
}

int heatkv_kernel_launches(heatkv_ctx* ctx, heatkv_kernel_stats* out) {
  if (!ctx || !out) return HEATKV_ERR_INVALID_ARG;
  *out = ctx->kstats;
  out->tcgen05_attention_ready = tc_ready(ctx->tc) ? 1u : 0u;
  out->tcgen05_calibration_ready = calib_tc_ready(ctx->calib_tc) ? 1u : 0u;
  return HEATKV_OK;
}

int heatkv_rank_dispersion(const double* scas_runs, int n_runs, int L, int H, int K, int s, double* out) {
  if (!scas_runs || !out || n_runs < 1 || L < 1 || H < 1 || K < 1 || K > HEATKV_MAX_K || s < 0 || s >= K)
    return HEATKV_ERR_INVALID_ARG;
  const int T = L * H;
  try {
    std::vector<int> order(T);
    std::vector<double> rank((size_t)n_runs * T);
    for (int k = 0; k < K; ++k) {
      out[k] = 0.0;
      if (k < s || k > K - 2) continue;                  // orders exist for the prunable source scales only
      for (int r = 0; r < n_runs; ++r) {
        const double* sc = scas_runs + (size_t)r * T * K;
        for (int i = 0; i < T; ++i) {
          if (!std::isfinite(sc[(size_t)i * K + k])) return HEATKV_ERR_NAN_SCORE;
          order[i] = i;
        }
        // least to most dependent; equal scores by ascending head index, as the schedule builder orders them
        std::stable_sort(order.begin(), order.end(),
                         [&](int a, int b) { return sc[(size_t)a * K + k] < sc[(size_t)b * K + k]; });
        for (int pos = 0; pos < T; ++pos) rank[(size_t)r * T + order[pos]] = (double)pos;
      }
      double acc = 0.0;
      for (int i = 0; i < T; ++i) {
        double mean = 0.0, var = 0.0;
        for (int r = 0; r < n_runs; ++r) mean += rank[(size_t)r * T + i];
        mean /= (double)n_runs;
        for (int r = 0; r < n_runs; ++r) {
          const double dlt = rank[(size_t)r * T + i] - mean;
          var += dlt * dlt;
        }
        acc += std::sqrt(var / (double)n_runs);
      }
      out[k] = acc / (double)T;
    }
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  return HEATKV_OK;
}

int heatkv_selftest_wait_expiry(heatkv_ctx* ctx, void* stream_) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // word 32 of the status region receives what the wait returned (the work counters sit in words 16 and 17)
  uint32_t* result = ctx->status + 32;
  if (cudaMemsetAsync(result, 0, 4, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  if (launch_wait_expiry(ctx->status, result, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  ctx->launches += 1;
  ctx->kstats.other += 1;
  uint32_t host[2] = {0, 0};
  if (cudaMemcpyAsync(&host[0], result, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemcpyAsync(&host[1], ctx->status, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return HEATKV_ERR_CUDA;
  // the wait gave up, flagged its CTA and the context: exactly what a stuck hand-over inside a kernel does
  if (host[0] == 2u && host[1] != 0u) return HEATKV_ERR_DEVICE_TIMEOUT;
  return host[0] == 1u ? HEATKV_OK : HEATKV_ERR_CUDA;
}

int heatkv_device_status(heatkv_ctx* ctx, void* stream_) {
  if (!ctx) return HEATKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, ctx->status, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return HEATKV_ERR_CUDA;
  return word == 0 ? HEATKV_OK : HEATKV_ERR_DEVICE_TIMEOUT;
}

}  // extern "C"
