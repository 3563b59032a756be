// Host-side schedule construction: Eq. 5 (N_k), Algorithm 1 (G_k, E_k, A_k) with
// GreedyEarlyPruning, Algorithm 2 (CacheSizeAfterLayer / CachedTokens), and the
// per-head-fraction policy.  Everything after the sort is integer arithmetic.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <numeric>

#include "internal.h"

namespace heatkv {
namespace {

struct Unit {          // one prunable object: a head-scale, or (binary) a head with all its new scales
  int layer, head, scale, rank;
  uint16_t bits;
};

// CachedTokens (Appendix A) for one head: sinks present so far plus every non-sink source
// scale up to `upto` (0-based, inclusive) that is not in the absent set.
inline int64_t cached_tokens(const Schedule& S, uint16_t absent, int upto) {
  if (upto < 0) return 0;
  int64_t m = 0;
  if (S.s > 0) m = S.c[std::min(upto, S.s - 1)];
  for (int i = S.s; i <= upto; ++i)
    if (!((absent >> i) & 1)) m += S.t[i];
  return m;
}

}  // namespace

int build_schedule(const heatkv_config& cfg, const double* scas, const double* cas, int policy,
                   int accounting, double b, const double* fraction, Schedule* out) {
  Schedule S;
  S.L = cfg.L; S.H = cfg.H; S.K = cfg.K; S.s = cfg.s; S.policy = policy;
  if (S.L < 1 || S.H < 1 || S.K < 1 || S.K > HEATKV_MAX_K || S.s < 0 || S.s > std::max(S.K - 1, 0))
    return HEATKV_ERR_INVALID_ARG;
  if ((int64_t)S.L * S.H > (1 << 20)) return HEATKV_ERR_INVALID_ARG;
  for (int i = 0, acc = 0; i < S.K; ++i) {
    if (cfg.t[i] < 1) return HEATKV_ERR_INVALID_ARG;
    S.t[i] = cfg.t[i];
    acc += cfg.t[i];
    S.c[i] = acc;
  }
  if (accounting != HEATKV_ACCOUNT_PHYSICAL && accounting != HEATKV_ACCOUNT_LITERAL)
    return HEATKV_ERR_INVALID_ARG;
  const int L = S.L, H = S.H, K = S.K, s = S.s, T = L * H;
  S.n_k.assign(K, 0);
  S.attn_mask.assign((size_t)K * T, 0);
  S.keep_mask.assign((size_t)K * T, 0);

  std::vector<uint16_t> g((size_t)K * T, 0);   // G_k as absent-bits per head, k = 0..K-2
  std::vector<uint16_t> a((size_t)K * T, 0);   // A_k, k = 0..K-1

  if (policy == HEATKV_POLICY_EXPLICIT) {
    if (!fraction) return HEATKV_ERR_INVALID_ARG;
    const int64_t cfull = K >= 2 ? S.c[K - 2] : 0;
    for (int hd = 0; hd < T; ++hd) {
      double f = fraction[hd];
      if (!std::isfinite(f)) return HEATKV_ERR_NAN_SCORE;
      if (f < 0.0 || f > 1.0) return HEATKV_ERR_INVALID_ARG;
      int64_t M = (int64_t)std::ceil(f * (double)cfull - 1e-9);
      int j = 0;                                  // number of leading scales the head stores
      for (int cand = 1; cand <= K - 1; ++cand)
        if (S.c[cand - 1] <= M) j = cand;
      j = std::max(j, std::min(s, K - 1));
      uint16_t refused = 0;                       // scales j .. K-1 are never stored
      for (int i = j; i < K; ++i) refused |= (uint16_t)(1u << i);
      for (int k = 0; k < K; ++k) {
        g[(size_t)k * T + hd] = refused;
        a[(size_t)k * T + hd] = refused;
      }
    }
    S.budget = -1;
  } else if (policy == HEATKV_POLICY_HEATKV || policy == HEATKV_POLICY_BINARY ||
             policy == HEATKV_POLICY_NAIVE) {
    const bool binary = policy == HEATKV_POLICY_BINARY;
    const double* score = binary ? cas : scas;
    if (!score) return HEATKV_ERR_INVALID_ARG;
    if (!(b > 0.0) || !(b <= 1.0)) return HEATKV_ERR_INVALID_ARG;
    const int64_t cfull = K >= 2 ? S.c[K - 2] : 0;
    // B = b*T*c_{K-1} in whole tokens; the guard keeps 0.05*512*6425 at 164480.
    const double x = b * (double)T * (double)cfull;
    S.budget = (int64_t)std::floor(x * (1.0 + 1e-12) + 1e-9);
    const int64_t B = S.budget;
    const int64_t cs = s > 0 ? S.c[s - 1] : 0;
    // Eq. 5: smallest N with N*c_s + (T-N)*c_k <= B, 0 while scale k is a sink.
    for (int k = 0; k + 1 < K; ++k) {
      if (k < s) continue;
      int64_t need = (int64_t)T * S.c[k] - B;
      if (need <= 0) continue;
      int64_t den = S.c[k] - cs;
      int64_t N = (need + den - 1) / den;
      if (N > T) return HEATKV_ERR_BUDGET_INFEASIBLE;
      S.n_k[k] = (int32_t)N;
    }
    // Removal orders O_i for the prunable source scales s <= i <= K-2 (0-based).
    std::vector<int32_t> order((size_t)K * T, 0), rank((size_t)K * T, 0);
    for (int i = s; i + 1 < K; ++i) {
      int32_t* o = &order[(size_t)i * T];
      std::iota(o, o + T, 0);
      for (int hd = 0; hd < T; ++hd) {
        double v = binary ? score[hd] : score[(size_t)hd * K + i];
        if (!std::isfinite(v)) return HEATKV_ERR_NAN_SCORE;
      }
      std::stable_sort(o, o + T, [&](int32_t x1, int32_t x2) {
        double v1 = binary ? score[x1] : score[(size_t)x1 * K + i];
        double v2 = binary ? score[x2] : score[(size_t)x2 * K + i];
        return v1 < v2;
      });
      for (int r = 0; r < T; ++r) rank[(size_t)i * T + o[r]] = r;
    }
    // G_k: union over prunable source scales of Prefix(O_i, N_k).  Binary: a pruned head is in
    // sink-only mode, so every non-sink scale of it is in G_k.
    for (int k = 0; k + 1 < K; ++k) {
      const int ihi = binary ? K - 2 : k;
      for (int i = s; i <= ihi; ++i)
        for (int r = 0; r < S.n_k[k]; ++r)
          g[(size_t)k * T + order[(size_t)i * T + r]] |= (uint16_t)(1u << i);
    }
    // GreedyEarlyPruning per scale.
    std::vector<int64_t> after(L), before(L);
    std::vector<uint16_t> e(T);
    std::vector<Unit> units;
    for (int k = 0; k + 1 < K; ++k) {
      const uint16_t* Gk = &g[(size_t)k * T];
      const uint16_t* Gp = k > 0 ? &g[(size_t)(k - 1) * T] : nullptr;
      std::fill(e.begin(), e.end(), 0);
      units.clear();
      if (binary) {
        const int n_prev = k > 0 ? S.n_k[k - 1] : 0;
        for (int r = n_prev; r < S.n_k[k] && s + 1 < K; ++r) {
          int hd = order[(size_t)s * T + r];
          uint16_t nb = (uint16_t)(Gk[hd] & ~(Gp ? Gp[hd] : 0));
          if (nb) units.push_back({hd / H, hd, 0, r, nb});
        }
        std::sort(units.begin(), units.end(), [](const Unit& u, const Unit& v) {
          if (u.layer != v.layer) return u.layer > v.layer;
          return u.rank < v.rank;
        });
      } else {
        for (int hd = 0; hd < T; ++hd) {
          uint16_t nb = (uint16_t)(Gk[hd] & ~(Gp ? Gp[hd] : 0));
          for (int i = 0; i < K; ++i)
            if ((nb >> i) & 1)
              units.push_back({hd / H, hd, i, rank[(size_t)i * T + hd], (uint16_t)(1u << i)});
        }
        std::sort(units.begin(), units.end(), [](const Unit& u, const Unit& v) {
          if (u.layer != v.layer) return u.layer > v.layer;
          if (u.scale != v.scale) return u.scale > v.scale;
          return u.rank < v.rank;
        });
      }
      if (policy == HEATKV_POLICY_NAIVE) {
        for (const Unit& u : units) e[u.head] |= u.bits;
      } else {
        // Algorithm 2.  Executed layers hold scale k and have applied G_k.  Layers still to
        // run: as printed they are summed up to source scale k (LITERAL); physically they
        // hold only scales < k (PHYSICAL).
        const int upto_future = accounting == HEATKV_ACCOUNT_LITERAL ? k : k - 1;
        for (int l = 0; l < L; ++l) {
          after[l] = before[l] = 0;
          for (int h = 0; h < H; ++h) {
            int hd = l * H + h;
            after[l] += cached_tokens(S, Gk[hd], k);
            before[l] += cached_tokens(S, Gp ? Gp[hd] : 0, upto_future);
          }
        }
        size_t pos = 0;
        for (int done = 1; done <= L; ++done) {
          for (;;) {
            int64_t M = 0;
            for (int l = 0; l < L; ++l) M += l < done ? after[l] : before[l];
            if (M <= B) break;
            if (pos >= units.size()) return HEATKV_ERR_BUDGET_INFEASIBLE;
            const Unit& u = units[pos++];
            for (int i = s; i <= upto_future; ++i)
              if (((u.bits >> i) & 1) && !((e[u.head] >> i) & 1)) before[u.layer] -= S.t[i];
            e[u.head] |= u.bits;
          }
        }
      }
      for (int hd = 0; hd < T; ++hd) a[(size_t)k * T + hd] = (uint16_t)((Gp ? Gp[hd] : 0) | e[hd]);
    }
    if (K >= 2)
      for (int hd = 0; hd < T; ++hd) a[(size_t)(K - 1) * T + hd] = g[(size_t)(K - 2) * T + hd];
  } else {
    return HEATKV_ERR_INVALID_ARG;
  }

  // Masks: sinks are always present; a non-sink scale is visible at step k unless in A_k and
  // stored after the layer ran unless in G_k.
  const uint16_t sink_bits = (uint16_t)((1u << s) - 1);
  for (int k = 0; k < K; ++k) {
    const uint16_t below = (uint16_t)((1u << k) - 1);          // bits i < k
    const uint16_t upto = (uint16_t)((1u << (k + 1)) - 1);     // bits i <= k
    for (int hd = 0; hd < T; ++hd) {
      uint16_t am = (uint16_t)(below & (sink_bits | (uint16_t)~a[(size_t)k * T + hd]));
      S.attn_mask[(size_t)k * T + hd] = am;
      uint16_t km = k + 1 < K ? (uint16_t)(upto & (sink_bits | (uint16_t)~g[(size_t)k * T + hd])) : am;
      S.keep_mask[(size_t)k * T + hd] = km;
    }
  }
  static std::atomic<uint64_t> next_uid{1};       // schedules may be built from several threads
  S.uid = next_uid.fetch_add(1, std::memory_order_relaxed);
  *out = std::move(S);
  return HEATKV_OK;
}

}  // namespace heatkv
