// Host-side routing of a batch onto the SP tree (paper Sec. 4.1.2: cost model; Sec. 4.1.3: Algorithm 1, "Prefix-Completion
// SP-Tree Routing"). No device code: this file is part of the library so that a caller gets the planner, its cost
// table and the attention kernels behind one C ABI.
//
// Tree: the full binary tree over P = 2^(n_levels-1) GPUs; node (l, i) covers GPUs [i * 2^l, (i + 1) * 2^l) and
// runs its samples at SP degree 2^l (paper Sec. 4.1.1, Def. 1). The cost model is additive: cost[j * n_levels + l] is
// the load placed on every GPU of a level-l node by sample j, so the per-GPU load C_p of a plan is a plain sum.
// Token loads (the paper's Tok_p) are kept in units of 1/P token, which keeps them integers.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <numeric>
#include <vector>
#include "../../include/nsp.h"

namespace {

struct State {
  std::vector<int8_t> lvl;    // per sample in visiting order; only the first `placed` entries are meaningful
  std::vector<int32_t> idx;
  std::vector<int64_t> C, T;  // per GPU
  int64_t crit = 0;           // max_p C_p
  int last = 0;               // level of the sample placed last (monotone-SP constraint)
};

int64_t vmax(const std::vector<int64_t>& v) {
  int64_t m = std::numeric_limits<int64_t>::min();
  for (int64_t x : v) m = std::max(m, x);
  return v.empty() ? 0 : m;
}

}  // namespace

extern "C" int nsp_route_sp_tree(const int32_t* lengths, const int64_t* cost, int32_t n_samples, int32_t n_levels,
                                 int32_t prefix_k, int32_t beam_w, int64_t b_tok, int32_t monotone,
                                 int32_t* level_out, int32_t* index_out, int64_t* load_out, int64_t* tok_out,
                                 int32_t* feasible_out) {
  if (n_samples < 0 || n_levels < 1 || n_levels > 11 || prefix_k < 0 || beam_w < 1 || b_tok < 0)
    return NSP_ERR_INVALID_ARG;
  if (n_samples > 0 && (!lengths || !cost || !level_out || !index_out)) return NSP_ERR_INVALID_ARG;
  const int M = n_samples, K = n_levels - 1, P = 1 << K;
  for (int j = 0; j < M; ++j)
    if (lengths[j] < 0) return NSP_ERR_INVALID_ARG;
  for (int64_t t = 0; t < static_cast<int64_t>(M) * n_levels; ++t)
    if (cost[t] < 0) return NSP_ERR_INVALID_ARG;
  const int64_t budget = b_tok > std::numeric_limits<int64_t>::max() / P ? std::numeric_limits<int64_t>::max() : b_tok * P;

  // samples by nonincreasing length (equal lengths keep their order)
  std::vector<int> order(M);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return lengths[a] > lengths[b]; });
  const int nH = std::min(prefix_k, M);

  std::vector<State> Q(1);
  Q[0].lvl.assign(M, 0);
  Q[0].idx.assign(M, 0);
  Q[0].C.assign(P, 0);
  Q[0].T.assign(P, 0);
  Q[0].last = K;

  // ---- long-prefix tree search: every retained state is extended by every feasible node, token-infeasible
  // extensions are dropped at once, the beam_w states with the smallest critical load survive
  for (int t = 0; t < nH; ++t) {
    const int j = order[t];
    std::vector<State> N;
    for (const State& S : Q) {
      for (int l = K; l >= 0; --l) {
        if (monotone && l > S.last) continue;
        const int64_t c = cost[static_cast<int64_t>(j) * n_levels + l];
        const int64_t tok = static_cast<int64_t>(lengths[j]) * (P >> l);
        for (int i = 0; i < (P >> l); ++i) {
          bool fits = true;
          for (int p = i << l; p < (i + 1) << l; ++p)
            if (S.T[p] + tok > budget) { fits = false; break; }
          if (!fits) continue;  // GPUs outside the node keep their (already feasible) token loads
          N.push_back(S);
          State& X = N.back();
          X.lvl[t] = static_cast<int8_t>(l);
          X.idx[t] = i;
          for (int p = i << l; p < (i + 1) << l; ++p) X.C[p] += c, X.T[p] += tok;
          X.crit = vmax(X.C);
          X.last = l;
        }
      }
    }
    if (N.empty()) return NSP_ERR_INFEASIBLE;  // no token-feasible placement of the prefix
    std::stable_sort(N.begin(), N.end(), [](const State& a, const State& b) { return a.crit < b.crit; });
    if (static_cast<int>(N.size()) > beam_w) N.resize(beam_w);
    Q.swap(N);
  }

  // ---- greedy completion of the short tail on the leaves, for every surviving state
  int best = -1;
  bool best_feasible = false;
  for (size_t q = 0; q < Q.size(); ++q) {
    State& S = Q[q];
    for (int t = nH; t < M; ++t) {
      const int j = order[t];
      const int64_t tok = static_cast<int64_t>(lengths[j]) * P;
      int u = -1;
      for (int p = 0; p < P; ++p)  // least-loaded leaf that stays within the token budget
        if (S.T[p] + tok <= budget && (u < 0 || S.C[p] < S.C[u])) u = p;
      if (u < 0) {  // none: the leaf with the smallest token load
        u = 0;
        for (int p = 1; p < P; ++p)
          if (S.T[p] < S.T[u]) u = p;
      }
      S.lvl[t] = 0;
      S.idx[t] = u;
      S.C[u] += cost[static_cast<int64_t>(j) * n_levels];
      S.T[u] += tok;
    }
    S.crit = vmax(S.C);
    const bool feas = vmax(S.T) <= budget;
    if (best < 0 || (feas && !best_feasible) || (feas == best_feasible && S.crit < Q[best].crit)) {
      best = static_cast<int>(q);
      best_feasible = feas;
    }
  }
  const State& R = Q[best];
  for (int t = 0; t < M; ++t) {
    level_out[order[t]] = R.lvl[t];
    index_out[order[t]] = R.idx[t];
  }
  if (load_out)
    for (int p = 0; p < P; ++p) load_out[p] = R.C[p];
  if (tok_out)
    for (int p = 0; p < P; ++p) tok_out[p] = R.T[p];
  if (feasible_out) *feasible_out = best_feasible ? 1 : 0;
  return NSP_OK;
}

extern "C" int nsp_cost_table(const int32_t* lengths, int32_t n_samples, int32_t n_levels, int32_t hq, int32_t hkv,
                              int32_t head_dim, const double* tcomp_ns, const double* link_gbs,
                              double other_ns_per_token, int64_t* cost_out) {
  if (n_samples < 0 || n_levels < 1 || n_levels > 11 || hq <= 0 || hkv <= 0 || head_dim <= 0 ||
      !(other_ns_per_token >= 0.0))
    return NSP_ERR_INVALID_ARG;
  if (!tcomp_ns || !link_gbs || (n_samples > 0 && (!lengths || !cost_out))) return NSP_ERR_INVALID_ARG;
  for (int l = 0; l < n_levels; ++l) {
    if (l > 0 && !(link_gbs[l] > 0.0)) return NSP_ERR_INVALID_ARG;
    for (int b = 0; b < NSP_COST_BUCKETS; ++b)
      if (!(tcomp_ns[l * NSP_COST_BUCKETS + b] >= 0.0)) return NSP_ERR_INVALID_ARG;
  }
  for (int j = 0; j < n_samples; ++j) {
    const int64_t L = lengths[j];
    if (L < 0) return NSP_ERR_INVALID_ARG;
    int b = 0;  // length class: floor(log2 L) clipped to [5, 20], minus 5
    while (b < NSP_COST_BUCKETS - 1 && (static_cast<int64_t>(64) << b) <= L) ++b;
    const double pairs = static_cast<double>(L) * static_cast<double>(L + 1) / 2.0;
    for (int l = 0; l < n_levels; ++l) {
      const double d = static_cast<double>(1 << l);
      // SP-backend level: compute = causal pairs x local q heads x profiled time per (pair, head), forward + backward
      const double comp = pairs * (static_cast<double>(hq) / d) * tcomp_ns[l * NSP_COST_BUCKETS + b];
      // prologue + epilogue: the all-to-alls move Q, K, V in and O out in the forward pass and their gradients the
      // other way in the backward pass; a GPU keeps 1/d of its L/d tokens' data and exchanges the rest
      double comm = 0.0;
      if (l > 0) {
        const double bytes_per_token = 2.0 * 2.0 * head_dim * (2.0 * hq + 2.0 * hkv);
        comm = (static_cast<double>(L) / d) * ((d - 1.0) / d) * bytes_per_token / link_gbs[l];  // bytes / (GB/s) = ns
      }
      // model level: projections and MLP scale with the tokens that stay on the GPU
      const double other = (static_cast<double>(L) / d) * other_ns_per_token;
      cost_out[static_cast<int64_t>(j) * n_levels + l] = std::llround(comp + comm + other);
    }
  }
  return NSP_OK;
}
