// Key-range splitting of the tensor-memory attention launch: the host-side choice of how many pieces every
// head's key range is cut into.  Pure host code (no CUDA): the launch is described by the key tiles of its
// heads in dispatch order (descending), the query tile pairs per head, the sequences of the call and the SMs.
#include <algorithm>
#include <vector>

#include "internal.h"

namespace heatkv {

SplitShape split_shape(const std::vector<int>& tiles, const std::vector<int>& ns, int n_qp) {
  SplitShape r;
  for (size_t i = 0; i < tiles.size(); ++i) {
    r.items += n_qp * ns[i];
    if (ns[i] > 1) { r.slots += n_qp * ns[i]; r.ctrs += n_qp; }
  }
  return r;
}

// Estimated makespan (in units of one 128-key tile) of the launch.  Items are taken by the resident CTAs in
// dispatch order (heads by descending key count, pieces, query tile pairs, sequences interleaved); for very
// large launches the list-scheduling bound total / SMs + longest is used.  The per-item constants were fitted
// to clock stamps of the kernel: an item costs its tiles plus the result's way out and the next item's start;
// a piece writes fp32 partials instead, and the piece that arrives last reads the others.
double split_makespan(const std::vector<int>& tiles, const std::vector<int>& ns, int n_qp, int n_seq, int n_sm) {
  constexpr double FIXED = 2.0, PUBLISH = 1.0, MERGE_PER_PIECE = 1.5;
  std::vector<double> costs;
  double total = 0.0, longest = 0.0;
  for (size_t i = 0; i < tiles.size(); ++i) {
    const int piece = (tiles[i] + ns[i] - 1) / ns[i];
    for (int pc = 0; pc < ns[i]; ++pc) {
      const int len = std::min(tiles[i], (pc + 1) * piece) - pc * piece;
      const double c = len + FIXED + (ns[i] > 1 ? PUBLISH + MERGE_PER_PIECE * (ns[i] - 1) / ns[i] : 0.0);
      for (int q = 0; q < n_qp; ++q) costs.push_back(c);
      total += c * n_qp;
      longest = std::max(longest, c);
    }
  }
  const size_t n_items = costs.size() * (size_t)n_seq;
  if (n_items > 8192) return total * n_seq / n_sm + longest;
  std::vector<double> sm(n_sm, 0.0);                       // binary min-heap of SM finish times
  auto cmp = [](double a, double b) { return a > b; };
  for (double c : costs)
    for (int q = 0; q < n_seq; ++q) {
      std::pop_heap(sm.begin(), sm.end(), cmp);
      sm.back() += c;
      std::push_heap(sm.begin(), sm.end(), cmp);
    }
  return *std::max_element(sm.begin(), sm.end());
}

// The search.  Long heads are cut to a common longest run (candidates: the longest head divided by 2..16), and,
// when `per_head` allows a piece count of its own for every head, the heads dispatched last may be cut two or
// three times finer so that the last round of items fills the SMs.  A cut is taken when it shortens the
// estimate by 5 %; pieces are never shorter than SPLIT_MIN_PIECE tiles, and the partial slots and arrival
// counters the cut needs per sequence (times n_seq) must fit max_slots / max_ctrs.
SplitChoice split_search(const std::vector<int>& tiles, int n_qp, int n_seq, int n_sm, bool per_head, uint64_t max_slots,
                         uint64_t max_ctrs) {
  const int H = (int)tiles.size();
  SplitChoice best;
  best.ns.assign(H, 1);
  if (H == 0) return best;
  double best_t = split_makespan(tiles, best.ns, n_qp, n_seq, n_sm);
  auto fits = [&](const SplitShape& sh) {
    return (uint64_t)sh.slots * n_seq <= max_slots && (uint64_t)sh.ctrs * n_seq * SPLIT_CTRS_PER_GROUP <= max_ctrs;
  };
  const int max_tiles = *std::max_element(tiles.begin(), tiles.end());
  std::vector<int> lmaxes = {0};
  for (int div : {2, 3, 4, 6, 8, 12, 16}) {
    const int cand = (max_tiles + div - 1) / div;
    if (cand < SPLIT_MIN_PIECE) break;
    lmaxes.push_back(cand);
  }
  for (int lmax : lmaxes) {
    std::vector<int> base(H);
    for (int i = 0; i < H; ++i) base[i] = split_pieces_for(tiles[i], lmax);
    for (int extra = 1; extra <= (per_head ? 3 : 1); ++extra)
      for (int tail = (extra == 1 ? 0 : 1); tail <= (extra == 1 ? 0 : H); ++tail) {
        std::vector<int> ns = base;
        bool ok = true;
        for (int i = H - tail; i < H; ++i) {
          ns[i] = base[i] * extra;
          ok = ok && (tiles[i] + ns[i] - 1) / ns[i] >= SPLIT_MIN_PIECE;
        }
        for (int i = 0; i < H; ++i) ok = ok && split_cut_ok(tiles[i], ns[i]);
        if (!ok || (lmax == 0 && tail == 0)) continue;
        if (!fits(split_shape(tiles, ns, n_qp))) continue;
        const double t = split_makespan(tiles, ns, n_qp, n_seq, n_sm);
        if (t < 0.95 * best_t) { best_t = t; best.ns = ns; best.lmax = tail == 0 ? lmax : -1; }
      }
  }
  return best;
}

}  // namespace heatkv

extern "C" int heatkv_split_plan(const int32_t* tiles, int n_heads, int n_qp, int n_seq, int n_sm, int per_head,
                                 uint64_t max_slots, uint64_t max_ctrs, int32_t* pieces, double* makespan_whole,
                                 double* makespan_cut) {
  if (!tiles || !pieces || n_heads < 1 || n_qp < 1 || n_seq < 1 || n_sm < 1) return HEATKV_ERR_INVALID_ARG;
  for (int i = 0; i < n_heads; ++i)
    if (tiles[i] < 1 || (i > 0 && tiles[i] > tiles[i - 1])) return HEATKV_ERR_INVALID_ARG;
  try {
    const std::vector<int> t(tiles, tiles + n_heads);
    const heatkv::SplitChoice ch = heatkv::split_search(t, n_qp, n_seq, n_sm, per_head != 0, max_slots, max_ctrs);
    for (int i = 0; i < n_heads; ++i) pieces[i] = ch.ns[i];
    if (makespan_whole) *makespan_whole = heatkv::split_makespan(t, std::vector<int>(n_heads, 1), n_qp, n_seq, n_sm);
    if (makespan_cut) *makespan_cut = heatkv::split_makespan(t, ch.ns, n_qp, n_seq, n_sm);
  } catch (const std::bad_alloc&) {
    return HEATKV_ERR_HOST_MEMORY;
  }
  return HEATKV_OK;
}
