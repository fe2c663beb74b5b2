// Host-side plan for spreading the communities over several GPUs (Section 2 of the paper: every community
// can be handed to an agent of its own; Section 3.1: a further agent holds the weights; Appendix A, Eq. 4:
// the first-order messages p and the second-order messages s that neighbouring agents exchange).
//
// A rank owns a contiguous range of communities, hence a contiguous range of rows in the community order of
// GraphIndex, with about the same number of stored entries of A + I per rank.  For every ordered pair
// (receiver r, sender s) the plan lists the rows of s that r depends on:
//   first order   rows of s adjacent to a row of r.  These are the rows r must hold a copy of before a pass:
//                 Z_{l-1} for the propagation A~ Z_{l-1} on r's rows, and the next layer's pre-activation,
//                 auxiliary variable and dual (H_{l+1}, Z_{l+1}, U) for the gradient and the step-size
//                 search of r's Z_{l,m} blocks.  The owner computes those rows; r only receives them, so the
//                 second-order information of Eq. 4 (what a neighbouring community aggregates from its own
//                 neighbours) arrives already folded into H_{l+1}.
//   second order  rows of s that are neither r's own nor first-order rows of r but adjacent to a first-order
//                 row of r: the rows whose Z_l reaches r's objectives only through a neighbour's
//                 aggregation.  Nothing is sent for them in the owner-computes scheme; the list sizes what a
//                 rank would have to fetch if it recomputed its neighbours' pre-activations itself, and is
//                 what the paper's second-order message replaces.
// All lists are ascending in new ids and unique.  The send list of (s -> r) is the receive list of (r <- s).
// Nothing here touches a device; no collective is issued by this library (every handle works on one GPU).
#pragma once
#include <algorithm>
#include <vector>

#include "graph_index.hpp"

namespace gcn_admm_host {

struct ShardPlan {
  int n_ranks = 0;
  std::vector<int> comm_begin;   // [R+1] rank r owns communities comm_begin[r] .. comm_begin[r+1]-1
  std::vector<int> row_begin;    // [R+1] and rows row_begin[r] .. row_begin[r+1]-1
  std::vector<int> rank_of_row;  // [n]
  // lists[r * R + s], r = receiver, s = sender (empty for r == s)
  std::vector<std::vector<int>> first_order, second_order;
};

// Contiguous community ranges with balanced stored entries: rank r ends at the first community boundary
// at or past (r+1)/R of the stored entries, leaving at least one community for every later rank.
inline bool build_shard_plan(const GraphIndex& g, int n_ranks, ShardPlan& plan) {
  if (n_ranks < 1 || n_ranks > g.n_comm) return false;
  const int R = n_ranks, M = g.n_comm;
  plan = ShardPlan{};
  plan.n_ranks = R;
  plan.comm_begin.assign(R + 1, 0);
  plan.row_begin.assign(R + 1, 0);
  int m = 0;
  for (int r = 0; r < R; ++r) {
    plan.comm_begin[r] = m;
    const long long want = g.nnz * (long long)(r + 1) / R;
    ++m;                                                      // at least one community per rank
    while (m < M - (R - 1 - r) && g.row_ptr[g.comm_ptr[m]] < want) ++m;
    if (r == R - 1) m = M;
  }
  plan.comm_begin[R] = M;
  for (int r = 0; r <= R; ++r) plan.row_begin[r] = g.comm_ptr[plan.comm_begin[r]];
  plan.rank_of_row.resize((size_t)g.n);
  for (int r = 0; r < R; ++r)
    for (int i = plan.row_begin[r]; i < plan.row_begin[r + 1]; ++i) plan.rank_of_row[(size_t)i] = r;

  plan.first_order.assign((size_t)R * R, {});
  plan.second_order.assign((size_t)R * R, {});
  std::vector<char> mark((size_t)g.n);
  for (int r = 0; r < R; ++r) {
    const int lo = plan.row_begin[r], hi = plan.row_begin[r + 1];
    // mark: 1 = first-order row of r, 2 = second-order row of r
    std::fill(mark.begin(), mark.end(), 0);
    std::vector<int> halo;
    for (int i = lo; i < hi; ++i)
      for (int p = g.row_ptr[i]; p < g.row_ptr[i + 1]; ++p) {
        const int j = g.col[p];
        if ((j < lo || j >= hi) && !mark[(size_t)j]) { mark[(size_t)j] = 1; halo.push_back(j); }
      }
    std::vector<int> halo2;
    for (int j : halo)
      for (int p = g.row_ptr[j]; p < g.row_ptr[j + 1]; ++p) {
        const int k = g.col[p];
        if ((k < lo || k >= hi) && !mark[(size_t)k]) { mark[(size_t)k] = 2; halo2.push_back(k); }
      }
    std::sort(halo.begin(), halo.end());
    std::sort(halo2.begin(), halo2.end());
    for (int j : halo) plan.first_order[(size_t)r * R + plan.rank_of_row[(size_t)j]].push_back(j);
    for (int k : halo2) plan.second_order[(size_t)r * R + plan.rank_of_row[(size_t)k]].push_back(k);
  }
  return true;
}

}  // namespace gcn_admm_host
