// Test harness (host only): reads a graph and a community assignment as text, builds the index
// tables and the long-row work items, prints them as text.  Built and run by test_long_row_tables.py.
#include <cstdio>
#include <string>
#include <vector>

#include "../paper_2112_09335_b200/csrc/graph_index.hpp"

int main() {
  long long n; int n_comm, limit;
  if (std::scanf("%lld %d %d", &n, &n_comm, &limit) != 3) return 2;
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
  gcn_admm_host::LongRowTables t;
  gcn_admm_host::build_long_row_tables(g, limit, t);
  std::printf("%lld\n", g.nnz);
  for (int v : g.row_ptr) std::printf("%d ", v);
  std::printf("\n");
  for (int v : g.col) std::printf("%d ", v);
  std::printf("\n");
  for (int v : g.row_comm) std::printf("%d ", v);
  std::printf("\n");
  for (const auto* tab : {&t.items, &t.split, &t.rows}) {
    std::printf("%zu\n", tab->size());
    for (const auto& q : *tab) std::printf("%d %d %d %d\n", q.x, q.y, q.z, q.w);
  }
  return 0;
}
