// seq_tree_build / seq_tree_speedup_search: Sequoia's tree construction (Section 3.1, Algorithm 1, with the depth
// bound and the per-depth acceptance matrix of the appendix) and the hardware-aware choice of size and depth
// (Section 4.1).  Host code: the tree is built once, offline, and then fixed for the whole run.
//
// T[d][b][n] = best F of a tree with exactly n nodes, depth <= d, root fan-out exactly b, no fan-out above B.
// Which (n, d, b) admit a tree at all is known in closed form -- the b subtrees hold 1 .. cap(d-1) nodes each,
// cap(d) = 1 + B + ... + B^d -- so the recursion only ever touches feasible entries: no sentinels, and the inner
// loop is a plain max-plus convolution over contiguous memory.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>

#include "seq_tree.h"

namespace {

struct Dp {
  int N, D, B;
  std::vector<int64_t> cap;     // cap[d] = most nodes a tree of depth <= d can hold, clamped to N
  std::vector<double> T;        // [D+1][B+1][N+1]
  std::vector<double> G;        // [D+1][N+1]: max over b
  std::vector<int32_t> arg_m;   // [D+1][B+1][N+1]: size of the last child's subtree
  std::vector<int32_t> arg_b;   // [D+1][N+1]
  double* t(int d, int b) { return T.data() + ((size_t)d * (B + 1) + b) * (N + 1); }
  int32_t* am(int d, int b) { return arg_m.data() + ((size_t)d * (B + 1) + b) * (N + 1); }
  double* g(int d) { return G.data() + (size_t)d * (N + 1); }
  int32_t* ab(int d) { return arg_b.data() + (size_t)d * (N + 1); }
  // n nodes, depth <= d, root fan-out b: possible?
  bool feasible(int n, int d, int b) const {
    if (b == 0) return n == 1;
    if (d == 0) return false;
    return n - 1 >= b && n - 1 <= (int64_t)b * cap[d - 1];
  }
};

void run_dp(Dp& dp, const double* rates, int rate_rows) {
  const int N = dp.N, D = dp.D, B = dp.B;
  const double ninf = -std::numeric_limits<double>::infinity();
  dp.cap.assign(D + 1, 1);
  for (int d = 1; d <= D; ++d) dp.cap[d] = std::min<int64_t>(N, 1 + (int64_t)B * dp.cap[d - 1]);
  dp.T.assign((size_t)(D + 1) * (B + 1) * (N + 1), ninf);
  dp.G.assign((size_t)(D + 1) * (N + 1), ninf);
  dp.arg_m.assign(dp.T.size(), 0);
  dp.arg_b.assign(dp.G.size(), 0);
  for (int d = 0; d <= D; ++d) {
    dp.t(d, 0)[1] = 1.0;  // the root alone generates one token per step
    dp.g(d)[1] = 1.0;
  }
  for (int d = 1; d <= D; ++d) {
    // a tree that may still grow d levels hangs below a node at depth D - d: its root's children use that row
    const double* P = rates + (size_t)(rate_rows == 1 ? 0 : D - d) * B;
    const double* sub = dp.g(d - 1);  // best subtree of each size one level down
    const int64_t cap = dp.cap[d - 1];
    for (int b = 1; b <= B; ++b) {
      const double pb = P[b - 1];
      const double* left = dp.t(d, b - 1);
      double* out = dp.t(d, b);
      int32_t* arg = dp.am(d, b);
      const int n_hi = (int)std::min<int64_t>(N, 1 + (int64_t)b * cap);
      for (int n = b + 1; n <= n_hi; ++n) {
        // m nodes in the b-th child's subtree; the other b-1 subtrees and the root keep n - m
        const int m_lo = (int)std::max<int64_t>(1, n - 1 - (int64_t)(b - 1) * cap);
        const int m_hi = (int)std::min<int64_t>(cap, n - b);
        double best = ninf;
        int best_m = 0;
        for (int m = m_lo; m <= m_hi; ++m) {
          const double v = left[n - m] + pb * sub[m];
          if (v > best) { best = v; best_m = m; }
        }
        out[n] = best;
        arg[n] = best_m;
      }
    }
    double* g = dp.g(d);
    int32_t* ab = dp.ab(d);
    for (int n = 2; n <= N; ++n)
      for (int b = 1; b <= B; ++b)
        if (dp.feasible(n, d, b) && dp.t(d, b)[n] > g[n]) { g[n] = dp.t(d, b)[n]; ab[n] = b; }
  }
}

}  // namespace

extern "C" int seq_tree_build(const seq_tree_build_params* p) {
  if (p == nullptr || p->acc_rates == nullptr || p->parent_out == nullptr || p->size_out == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->max_size < 1 || p->max_size > SEQ_MAX_TREE || p->max_depth < 0 || p->max_branch < 1) return SEQ_ERR_INVALID_ARG;
  if (p->acc_rows != 1 && p->acc_rows < p->max_depth) return SEQ_ERR_INVALID_ARG;
  const int N = p->max_size, B = std::min(p->max_branch, N - 1 > 0 ? N - 1 : 1);
  const int D = std::min(p->max_depth, N - 1);  // deeper than a chain of N nodes is never used
  // (the clamp of D moves no row of an acceptance matrix: rows are indexed from the root down)
  const int rows_used = p->acc_rows == 1 ? 1 : std::max(D, 1);
  std::vector<double> rates((size_t)rows_used * B);
  for (int r = 0; r < rows_used; ++r)
    for (int b = 0; b < B; ++b) {
      const double v = p->acc_rates[(size_t)r * p->max_branch + b];
      if (!(v >= 0.0 && v <= 1.0)) return SEQ_ERR_INVALID_ARG;
      rates[(size_t)r * B + b] = v;
    }
  if ((double)(D + 1) * (B + 1) * (N + 1) > 1e8) return SEQ_ERR_UNSUPPORTED;  // tables above a GB
  Dp dp;
  dp.N = N; dp.D = D; dp.B = B;
  // with a matrix, row index = depth of the parent = D - d for the table at d, D being the clamped depth
  run_dp(dp, rates.data(), rows_used == 1 ? 1 : rows_used);

  // the budget's best tree: more nodes never lower F (scores are >= 0), so the largest feasible size on ties
  int n_best = 1;
  for (int n = 2; n <= N; ++n)
    if (dp.g(D)[n] >= dp.g(D)[n_best]) n_best = n;
  // level-order numbering: siblings contiguous, in rank order, every parent before its children
  struct Item { int node, n, d; };
  std::vector<Item> level{{0, n_best, D}}, next;
  int count = 1;
  p->parent_out[0] = -1;
  std::vector<int> sizes;
  while (!level.empty()) {
    next.clear();
    for (const Item& it : level) {
      if (it.n == 1) continue;
      sizes.clear();
      int n = it.n;
      for (int b = dp.ab(it.d)[it.n]; b > 0; --b) {
        const int m = dp.am(it.d, b)[n];
        sizes.push_back(m);
        n -= m;
      }
      for (auto s = sizes.rbegin(); s != sizes.rend(); ++s) {
        p->parent_out[count] = it.node;
        next.push_back({count, *s, it.d - 1});
        ++count;
      }
    }
    level.swap(next);
  }
  *p->size_out = count;
  if (p->expected_out != nullptr) *p->expected_out = dp.g(D)[n_best];
  if (p->table_out != nullptr) {
    const double ninf = -std::numeric_limits<double>::infinity();
    for (int n = 0; n <= N; ++n)
      for (int d = 0; d <= p->max_depth; ++d)
        p->table_out[(size_t)n * (p->max_depth + 1) + d] = n == 0 ? ninf : dp.g(std::min(d, D))[n];
  }
  return SEQ_OK;
}

extern "C" int seq_tree_speedup_search(const double* table, int32_t max_size, int32_t max_depth, const double* t_of_n,
                                       double c, int32_t* n_out, int32_t* d_out, double* speedup_out) {
  if (table == nullptr || t_of_n == nullptr || n_out == nullptr || d_out == nullptr) return SEQ_ERR_INVALID_ARG;
  if (max_size < 1 || max_depth < 0 || !(c >= 0.0)) return SEQ_ERR_INVALID_ARG;
  double best = -std::numeric_limits<double>::infinity();
  int bn = 0, bd = 0;
  for (int n = 1; n <= max_size; ++n) {
    if (!(t_of_n[n] > 0.0)) return SEQ_ERR_INVALID_ARG;
    for (int d = 0; d <= max_depth; ++d) {
      const double g = table[(size_t)n * (max_depth + 1) + d];
      if (std::isinf(g)) continue;
      const double s = g / (t_of_n[n] + d * c);
      if (s > best) { best = s; bn = n; bd = d; }
    }
  }
  if (bn == 0) return SEQ_ERR_INVALID_ARG;
  *n_out = bn; *d_out = bd;
  if (speedup_out != nullptr) *speedup_out = best;
  return SEQ_OK;
}
