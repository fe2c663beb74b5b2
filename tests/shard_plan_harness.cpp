// Test harness (host only): reads a graph and a community assignment as text, builds the index tables and
// the multi-GPU shard plan, prints the plan as text; with the argument "index" it prints the index tables
// instead.  Built and run by test_shard_plan.py and test_graph_index_host.py.
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../paper_2112_09335_b200/csrc/shard_plan.hpp"

template <typename V> void print_row(const V& v) {
  std::printf("%zu", v.size());
  for (auto x : v) std::printf(" %d", (int)x);
  std::printf("\n");
}

int main(int argc, char** argv) {
  long long n; int n_comm, n_ranks;
  if (std::scanf("%lld %d %d", &n, &n_comm, &n_ranks) != 3) return 2;
  std::vector<long long> row_ptr(n + 1);
  for (auto& v : row_ptr) if (std::scanf("%lld", &v) != 1) return 2;
  std::vector<int> col(row_ptr[n]), comm(n);
  for (auto& v : col) if (std::scanf("%d", &v) != 1) return 2;
  for (auto& v : comm) if (std::scanf("%d", &v) != 1) return 2;
  gcn_admm_host::GraphIndex g;
  std::string err;
  if (gcn_admm_host::build_graph_index(n, row_ptr.data(), col.data(), n_comm, comm.data(), g, err) != 0) {
    std::fprintf(stderr, "%s\n", err.c_str());
    return 3;
  }
  if (argc > 1 && std::strcmp(argv[1], "index") == 0) {
    std::printf("ok\n");
    print_row(g.perm); print_row(g.inv); print_row(g.comm_ptr); print_row(g.row_comm); print_row(g.row_ptr);
    print_row(g.col); print_row(g.col_comm); print_row(g.seg_row_ptr); print_row(g.seg_comm); print_row(g.seg_begin);
    for (float d : g.dinv) std::printf("%.9g ", d);
    std::printf("\n");
    return 0;
  }
  gcn_admm_host::ShardPlan plan;
  if (!gcn_admm_host::build_shard_plan(g, n_ranks, plan)) { std::printf("refused\n"); return 0; }
  std::printf("ok\n");
  for (int v : plan.comm_begin) std::printf("%d ", v);
  std::printf("\n");
  for (int v : plan.row_begin) std::printf("%d ", v);
  std::printf("\n");
  for (const auto* lists : {&plan.first_order, &plan.second_order})
    for (const auto& l : *lists) {
      std::printf("%zu", l.size());
      for (int v : l) std::printf(" %d", v);
      std::printf("\n");
    }
  return 0;
}
