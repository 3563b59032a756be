// Static cache plan: because the schedule is fixed before generation starts, the physical
// position of every head-scale at every (step, layer) is known at admission.  The planner
// replays the whole generation once on the host with a private row space and emits the page
// tables (lists of <=64-row half-tiles), the append destinations and, for the ragged
// layout, the in-place moves of every eviction.  Rows are relative to the sequence's
// reservation, so one plan serves every sequence that uses the schedule.
#include <algorithm>
#include <functional>
#include <queue>

#include "internal.h"

namespace heatkv {
namespace {

constexpr int P = HEATKV_PAGE_TOKENS;

inline int32_t pack_meta(int n_valid, int scale) { return (int32_t)(n_valid | (scale << 8)); }

struct Builder {
  const Schedule& S;
  std::vector<Desc> descs;
  std::vector<Move> moves;
  std::vector<int32_t> attn_begin, attn_cnt, app_begin, app_cnt, order;
  std::vector<int32_t> pre_begin, pre_cnt, post_begin, post_cnt;
  std::vector<int32_t> src;                 // fp8 cache: pool row behind every descriptor
  explicit Builder(const Schedule& s) : S(s) {
    size_t n = (size_t)S.K * S.L * S.H;
    attn_begin.assign(n, 0); attn_cnt.assign(n, 0); app_begin.assign(n, 0); app_cnt.assign(n, 0);
    order.assign(n, 0);
    pre_begin.assign(n, 0); pre_cnt.assign(n, 0); post_begin.assign(n, 0); post_cnt.assign(n, 0);
  }
  // rows [row, row+n) of one source scale -> half-tile descriptors
  void emit_rows(int row, int n, int scale) {
    for (int off = 0; off < n; off += P)
      descs.push_back({row + off, pack_meta(std::min(P, n - off), scale)});
  }
  void finish(Plan* out) {
    PlanHeader h{};
    h.L = S.L; h.H = S.H; h.K = S.K;
    h.n_desc = (int32_t)descs.size();
    h.n_move = (int32_t)moves.size();
    std::vector<int32_t>& b = out->blob;
    b.assign(sizeof(PlanHeader) / 4, 0);
    auto put = [&](const void* p, size_t bytes) {
      while (b.size() % 4) b.push_back(0);               // 16-byte alignment of every table
      int32_t off = (int32_t)b.size();
      const int32_t* w = static_cast<const int32_t*>(p);
      b.insert(b.end(), w, w + bytes / 4);
      return off;
    };
    h.off_desc = put(descs.data(), descs.size() * sizeof(Desc));
    h.off_attn_begin = put(attn_begin.data(), attn_begin.size() * 4);
    h.off_attn_cnt = put(attn_cnt.data(), attn_cnt.size() * 4);
    h.off_app_begin = put(app_begin.data(), app_begin.size() * 4);
    h.off_app_cnt = put(app_cnt.data(), app_cnt.size() * 4);
    h.off_order = put(order.data(), order.size() * 4);
    h.off_move = put(moves.data(), moves.size() * sizeof(Move));
    h.off_pre_begin = put(pre_begin.data(), pre_begin.size() * 4);
    h.off_pre_cnt = put(pre_cnt.data(), pre_cnt.size() * 4);
    h.off_post_begin = put(post_begin.data(), post_begin.size() * 4);
    h.off_post_cnt = put(post_cnt.data(), post_cnt.size() * 4);
    if (!src.empty()) h.off_src = put(src.data(), src.size() * 4);
    while (b.size() % 4) b.push_back(0);
    h.total_words = (int32_t)b.size();
    *reinterpret_cast<PlanHeader*>(b.data()) = h;
  }
};

// visible prior tokens of (k, l, h) -> used to sort heads heavy-first
inline int visible_tokens(const Schedule& S, uint16_t mask) {
  int n = 0;
  for (int i = 0; i < S.K; ++i)
    if ((mask >> i) & 1) n += S.t[i];
  return n;
}

void fill_order(const Schedule& S, Builder& B) {
  std::vector<int> key(S.H);
  for (int k = 0; k < S.K; ++k)
    for (int l = 0; l < S.L; ++l) {
      int32_t* o = &B.order[S.at(k, l, 0)];
      for (int h = 0; h < S.H; ++h) {
        o[h] = h;
        key[h] = visible_tokens(S, S.attn_mask[S.at(k, l, h)]);
      }
      std::stable_sort(o, o + S.H, [&](int x, int y) { return key[x] > key[y]; });
    }
}

}  // namespace

int build_plan(const Schedule& S, int layout, Plan* out, bool fp8) {
  if (layout != HEATKV_LAYOUT_PAGED && layout != HEATKV_LAYOUT_RAGGED) return HEATKV_ERR_INVALID_ARG;
  if (fp8 && layout != HEATKV_LAYOUT_PAGED) return HEATKV_ERR_INVALID_ARG;
  const int L = S.L, H = S.H, K = S.K, s = S.s, T = L * H;
  Builder B(S);
  fill_order(S, B);
  out->layout = layout;
  out->tokens_pre.assign(K, 0);
  out->tokens_post.assign((size_t)K * L, 0);
  out->place.assign((size_t)T * K, -1);
  out->head_base.assign(T, 0);
  out->head_cap.assign(T, 0);
  std::vector<uint16_t> stored(T, 0);
  int64_t live_tokens = 0, peak_tokens = 0;
  auto tokens_of = [&](uint16_t m) { return (int64_t)visible_tokens(S, m); };
  const int c_s = s > 0 ? S.c[s - 1] : 0;

  if (layout == HEATKV_LAYOUT_PAGED) {
    // Pages of 64 rows.  The sink scales of a head share one block of ceil(c_s/64) pages; every
    // other head-scale owns ceil(t_i/64) pages from its append until its eviction (a page freed after a
    // layer is reusable from the next layer's append on).  Lowest
    // free page first, so the highest page ever used equals the peak number of live pages.
    std::priority_queue<int, std::vector<int>, std::greater<int>> free_pages;
    int next_page = 0;
    auto alloc = [&]() {
      if (!free_pages.empty()) { int p = free_pages.top(); free_pages.pop(); return p; }
      return next_page++;
    };
    // pages[(hd*K + i)] = pages of head-scale i (sink block stored under scale 0)
    std::vector<std::vector<int>> pages((size_t)T * K);
    auto release = [&](int hd, uint16_t gone) {
      for (int i = s; i < K; ++i)
        if ((gone >> i) & 1) {
          for (int p : pages[(size_t)hd * K + i]) free_pages.push(p);
          pages[(size_t)hd * K + i].clear();
        }
    };
    auto emit_scale = [&](int hd, int i) {     // descriptors of stored source scale i
      if (i < s) {
        const std::vector<int>& pg = pages[(size_t)hd * K + 0];
        int off0 = i > 0 ? S.c[i - 1] : 0;     // position inside the sink block
        for (int off = off0; off < S.c[i];) {
          int n = std::min(S.c[i] - off, P - off % P);
          B.descs.push_back({pg[off / P] * P + off % P, pack_meta(n, i)});
          off += n;
        }
      } else {
        const std::vector<int>& pg = pages[(size_t)hd * K + i];
        for (size_t j = 0; j < pg.size(); ++j)
          B.descs.push_back({pg[j] * P, pack_meta(std::min(P, S.t[i] - (int)j * P), i)});
      }
    };
    for (int k = 0; k < K; ++k) {
      for (int hd = 0; hd < T; ++hd) {         // eviction before the scale starts (E_k)
        uint16_t keep = S.attn_mask[(size_t)k * T + hd];
        uint16_t gone = (uint16_t)(stored[hd] & ~keep);
        if (gone) { release(hd, gone); live_tokens -= tokens_of(gone); stored[hd] &= keep; }
      }
      out->tokens_pre[k] = live_tokens;
      for (int l = 0; l < L; ++l) {
        for (int h = 0; h < H; ++h) {          // page table of the attention at (k, l, h)
          int hd = l * H + h;
          size_t u = S.at(k, l, h);
          B.attn_begin[u] = (int32_t)B.descs.size();
          for (int i = 0; i < k; ++i)
            if ((stored[hd] >> i) & 1) emit_scale(hd, i);
          B.attn_cnt[u] = (int32_t)B.descs.size() - B.attn_begin[u];
        }
        if (k + 1 < K) {
          for (int h = 0; h < H; ++h) {
            int hd = l * H + h;
            size_t u = S.at(k, l, h);
            uint16_t keep = S.keep_mask[u];
            B.app_begin[u] = (int32_t)B.descs.size();
            if ((keep >> k) & 1) {
              if (k < s) {
                if (pages[(size_t)hd * K].empty())
                  for (int j = 0; j < (c_s + P - 1) / P; ++j) pages[(size_t)hd * K].push_back(alloc());
              } else {
                for (int j = 0; j < (S.t[k] + P - 1) / P; ++j) pages[(size_t)hd * K + k].push_back(alloc());
              }
              emit_scale(hd, k);
              int first = B.descs[B.app_begin[u]].row;
              out->place[(size_t)hd * K + k] = first;
              stored[hd] |= (uint16_t)(1u << k);
              live_tokens += S.t[k];
            }
            B.app_cnt[u] = (int32_t)B.descs.size() - B.app_begin[u];
          }
          // Pages evicted after this layer are released only now: the new scale never lands on a page the
          // same step's attention still reads, so the append may run inside the attention launch.
          for (int h = 0; h < H; ++h) {
            int hd = l * H + h;
            uint16_t keep = S.keep_mask[S.at(k, l, h)];
            uint16_t gone = (uint16_t)(stored[hd] & ~keep);
            if (gone) { release(hd, gone); live_tokens -= tokens_of(gone); stored[hd] &= keep; }
          }
        }
        out->tokens_post[(size_t)k * L + l] = live_tokens;
        peak_tokens = std::max(peak_tokens, live_tokens);
      }
    }
    out->reserved_rows = (int64_t)std::max(next_page, 1) * P;
  } else {
    // Ragged-contiguous: every head owns one dense run (K pool and V pool alike) sized for the
    // most tokens it ever holds; stored scales sit in ascending order without gaps, so an
    // eviction slides the later survivors left and the new scale is appended at the tail.
    std::vector<int> cap(T, 0);
    {   // capacity pass: peak stored tokens per head over all checkpoints
      std::vector<uint16_t> st(T, 0);
      for (int k = 0; k < K; ++k)
        for (int hd = 0; hd < T; ++hd) {
          st[hd] &= S.attn_mask[(size_t)k * T + hd];
          cap[hd] = std::max(cap[hd], visible_tokens(S, st[hd]));
          if (k + 1 < K) {
            st[hd] = S.keep_mask[(size_t)k * T + hd];
            cap[hd] = std::max(cap[hd], visible_tokens(S, st[hd]));
          }
        }
    }
    int64_t base = 0;
    for (int hd = 0; hd < T; ++hd) {
      out->head_base[hd] = (int32_t)base;
      out->head_cap[hd] = cap[hd];
      base += cap[hd];
      if (base > INT32_MAX) return HEATKV_ERR_OUT_OF_PAGES;
    }
    out->reserved_rows = std::max<int64_t>((base + P - 1) / P * P, P);
    // Moves that take the dense layout of `from` to the dense layout of `to` (a subset of
    // `from`); adjacent surviving scales merge into one move.  Returns the tokens kept.
    auto emit_moves = [&](int hd, uint16_t from, uint16_t to, int32_t first_move) {
      int src = 0, dst = 0;
      for (int i = 0; i < K; ++i) {
        if (!((from >> i) & 1)) continue;
        if ((to >> i) & 1) {
          if (src != dst) {
            int a = out->head_base[hd] + src, d = out->head_base[hd] + dst;
            if ((int32_t)B.moves.size() > first_move && B.moves.back().src + B.moves.back().n == a)
              B.moves.back().n += S.t[i];
            else
              B.moves.push_back({a, d, S.t[i], 0});
          }
          dst += S.t[i];
        }
        src += S.t[i];
      }
      return dst;
    };
    for (int k = 0; k < K; ++k) {
      for (int l = 0; l < L; ++l)
        for (int h = 0; h < H; ++h) {          // eviction before the scale starts
          int hd = l * H + h;
          size_t u = S.at(k, l, h);
          uint16_t keep = (uint16_t)(stored[hd] & S.attn_mask[u]);
          B.pre_begin[u] = (int32_t)B.moves.size();
          if (keep != stored[hd]) {
            emit_moves(hd, stored[hd], keep, B.pre_begin[u]);
            live_tokens -= tokens_of((uint16_t)(stored[hd] & ~keep));
            stored[hd] = keep;
          }
          B.pre_cnt[u] = (int32_t)B.moves.size() - B.pre_begin[u];
        }
      out->tokens_pre[k] = live_tokens;
      for (int l = 0; l < L; ++l) {
        for (int h = 0; h < H; ++h) {
          int hd = l * H + h;
          size_t u = S.at(k, l, h);
          B.attn_begin[u] = (int32_t)B.descs.size();
          int off = 0;
          for (int i = 0; i < k; ++i)
            if ((stored[hd] >> i) & 1) { B.emit_rows(out->head_base[hd] + off, S.t[i], i); off += S.t[i]; }
          B.attn_cnt[u] = (int32_t)B.descs.size() - B.attn_begin[u];
        }
        if (k + 1 < K) {
          for (int h = 0; h < H; ++h) {
            int hd = l * H + h;
            size_t u = S.at(k, l, h);
            uint16_t keepm = S.keep_mask[u];
            uint16_t keep = (uint16_t)(stored[hd] & keepm);
            B.post_begin[u] = (int32_t)B.moves.size();
            int dst = emit_moves(hd, stored[hd], keep, B.post_begin[u]);
            B.post_cnt[u] = (int32_t)B.moves.size() - B.post_begin[u];
            live_tokens -= tokens_of((uint16_t)(stored[hd] & ~keep));
            stored[hd] = keep;
            B.app_begin[u] = (int32_t)B.descs.size();
            if ((keepm >> k) & 1) {
              B.emit_rows(out->head_base[hd] + dst, S.t[k], k);
              stored[hd] |= (uint16_t)(1u << k);
              live_tokens += S.t[k];
            }
            B.app_cnt[u] = (int32_t)B.descs.size() - B.app_begin[u];
          }
        }
        out->tokens_post[(size_t)k * L + l] = live_tokens;
        peak_tokens = std::max(peak_tokens, live_tokens);
      }
    }
  }
  out->peak_tokens = peak_tokens;
  out->stage_rows = 0;
  if (fp8) {
    // The attention kernels read bf16 staging rows that the call fills from the fp8 pool just before: the
    // visible half-tiles of a (step, layer) take consecutive 64-row slots in descriptor order (the layer's
    // heads are emitted one after the other), and `src` keeps the pool row of every descriptor.
    B.src.resize(B.descs.size());
    for (size_t i = 0; i < B.descs.size(); ++i) B.src[i] = B.descs[i].row;
    for (int k = 0; k < K; ++k)
      for (int l = 0; l < L; ++l) {
        const int32_t first = B.attn_begin[S.at(k, l, 0)];
        const int32_t end = B.attn_begin[S.at(k, l, H - 1)] + B.attn_cnt[S.at(k, l, H - 1)];
        for (int32_t i = first; i < end; ++i) B.descs[i].row = (i - first) * P;
        out->stage_rows = std::max<int64_t>(out->stage_rows, (int64_t)(end - first) * P);
      }
  }
  B.finish(out);
  return HEATKV_OK;
}

}  // namespace heatkv
