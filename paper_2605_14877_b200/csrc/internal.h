// Internal host-side declarations shared by the translation units of libheatkv.
#pragma once
#include <cstdint>
#include <vector>

#include "heatkv.h"

namespace heatkv {

// ---------------------------------------------------------------- schedule (host)
struct Schedule {
  int L = 0, H = 0, K = 0, s = 0;
  int t[HEATKV_MAX_K] = {0};
  int c[HEATKV_MAX_K] = {0};             // c[i] = t[0] + .. + t[i]
  int policy = 0;
  int64_t budget = -1;                   // B in tokens, -1 for EXPLICIT
  std::vector<int32_t> n_k;              // [K]
  std::vector<uint16_t> attn_mask;       // [K][L][H]
  std::vector<uint16_t> keep_mask;       // [K][L][H]
  uint64_t uid = 0;                      // identity used to cache plans per context
  size_t at(int step, int l, int h) const { return ((size_t)step * L + l) * H + h; }
};

// ---------------------------------------------------------------- plan (host image of device tables)
// One key half-tile: up to 64 consecutive pool rows that belong to one source scale.
struct Desc {
  int32_t row;      // row relative to the sequence's reservation
  int32_t meta;     // n_valid (bits 0..7) | source scale (bits 8..15)
};
// One in-place move of the ragged layout: n rows from src to dst (dst < src), relative rows.
struct Move {
  int32_t src, dst, n, pad;
};

// Offsets (in 4-byte words from the start of the blob) of the tables of a plan.  The blob
// is what lives in the metadata region; kernels receive its device address.
struct PlanHeader {
  int32_t L, H, K, n_desc;
  int32_t off_desc;        // Desc[n_desc]
  int32_t off_attn_begin;  // int32[K*L*H] first desc of the visible prior keys
  int32_t off_attn_cnt;    // int32[K*L*H]
  int32_t off_app_begin;   // int32[K*L*H] first desc of the rows the step's K/V go to
  int32_t off_app_cnt;     // int32[K*L*H] 0 = the head does not store this scale
  int32_t off_order;       // int32[K*L*H] heads of a (step, layer) sorted by visible keys, descending
  int32_t off_move;        // Move[n_move]
  int32_t off_pre_begin;   // int32[K*L*H] moves of the eviction before the step   (ragged)
  int32_t off_pre_cnt;
  int32_t off_post_begin;  // int32[K*L*H] moves of the eviction after the layer   (ragged)
  int32_t off_post_cnt;
  int32_t n_move;
  int32_t total_words;
  int32_t off_src;         // fp8 cache only, else 0: int32[n_desc] pool row (relative to the reservation) behind
                           // every descriptor; the attention descriptors then carry staging rows instead
  int32_t pad[2];
};
static_assert(sizeof(PlanHeader) % 16 == 0, "header must keep 16-byte alignment");

struct Plan {
  int layout = 0;
  int64_t reserved_rows = 0;            // multiple of HEATKV_PAGE_TOKENS
  int64_t peak_tokens = 0;
  int64_t stage_rows = 0;               // fp8 cache: staging rows one attention call needs per sequence (64 per
                                        // visible half-tile of the busiest (step, layer))
  std::vector<int32_t> blob;            // PlanHeader followed by the tables
  // host-only bookkeeping for introspection -------------------------------------------------
  // place[(l*H+h)*K + i] = first relative row of source scale i in the paged layout (-1: never stored)
  std::vector<int32_t> place;
  // ragged: base row and capacity of every head
  std::vector<int32_t> head_base, head_cap;
  // tokens cached after the pre-step eviction of step k / after layer l of step k
  std::vector<int64_t> tokens_pre;      // [K]
  std::vector<int64_t> tokens_post;     // [K][L]
  const PlanHeader& header() const { return *reinterpret_cast<const PlanHeader*>(blob.data()); }
};

// ---- key-range splitting of the tensor-memory attention launch (split.cpp)
constexpr int SPLIT_MIN_PIECE = 4;        // shorter pieces measured slower (their fixed cost dominates)
constexpr int SPLIT_CTRS_PER_GROUP = 8;   // arrival counters per (head, query tile pair): one per 32 rows
// How one attention launch cuts its heads: pieces per head in dispatch order; `lmax` > 0 when that is the
// same as "no run longer than lmax tiles" (the rule a call with several schedules applies to all of them).
struct SplitChoice {
  std::vector<int> ns;
  int lmax = 0;
};
// Items of one sequence: count, partial slots, counter groups.
struct SplitShape {
  int items = 0, slots = 0, ctrs = 0;
};
// Pieces of a head under a longest run of `lmax` tiles (0: the whole head).
inline int split_pieces_for(int tiles, int lmax) { return lmax > 0 ? (tiles + lmax - 1) / lmax : 1; }
// Every piece of an equal cut must hold at least one tile.
inline bool split_cut_ok(int tiles, int ns) { return ns >= 1 && (ns - 1) * ((tiles + ns - 1) / ns) < tiles; }
SplitShape split_shape(const std::vector<int>& tiles, const std::vector<int>& ns, int n_qp);
double split_makespan(const std::vector<int>& tiles, const std::vector<int>& ns, int n_qp, int n_seq, int n_sm);
SplitChoice split_search(const std::vector<int>& tiles, int n_qp, int n_seq, int n_sm, bool per_head, uint64_t max_slots,
                         uint64_t max_ctrs);

int build_schedule(const heatkv_config& cfg, const double* scas, const double* cas, int policy,
                   int accounting, double b, const double* fraction, Schedule* out);
// `fp8`: plan for a context with the fp8 cache (paged layout only): the attention descriptors of every
// (step, layer) are renumbered to consecutive 64-row staging slots, in descriptor order across the layer's heads,
// and a table of the pool rows behind them is added.
int build_plan(const Schedule& sch, int layout, Plan* out, bool fp8 = false);

}  // namespace heatkv
