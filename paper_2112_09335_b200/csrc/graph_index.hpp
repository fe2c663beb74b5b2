// Host-side community reordering and index tables (Section 2 of the paper: V_m, N_m and the
// block split of A~; Appendix A: first- and second-order neighbour rows).  Runs once at
// creation, outside every ADMM iteration.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <string>
#include <vector>

namespace gcn_admm_host {

struct GraphIndex {
  long long n = 0;
  int n_comm = 0;
  long long nnz = 0;               // stored entries of A + I
  std::vector<int> perm, inv;      // new -> original, original -> new
  std::vector<int> comm_ptr;       // [M+1]
  std::vector<int> row_comm;       // community of each new id
  std::vector<int> row_ptr, col;   // A + I in new ids, ascending columns
  std::vector<float> dinv;         // (deg_A + 1)^(-1/2) per new id
  std::vector<int> seg_row_ptr, seg_comm, seg_begin;
};

enum { IDX_OK = 0, IDX_BAD_GRAPH = 1, IDX_BAD_COMMUNITY = 2 };

// Validates the CSR of A and the community assignment and fills `g`.
inline int build_graph_index(long long n, const long long* row_ptr, const int* col_idx, int n_comm,
                             const int* community, GraphIndex& g, std::string& err) {
  g.n = n;
  g.n_comm = n_comm;
  if (row_ptr[0] != 0) { err = "row_ptr[0] must be 0"; return IDX_BAD_GRAPH; }
  for (long long i = 0; i < n; ++i)
    if (row_ptr[i + 1] < row_ptr[i]) { err = "row_ptr is not ascending"; return IDX_BAD_GRAPH; }
  if (row_ptr[n] + n > 2147483647LL) { err = "more than 2^31-1 stored entries"; return IDX_BAD_GRAPH; }
  // Symmetry: every entry above the diagonal must have its mirror below it (a binary search in the
  // sorted row), and there must be as many entries below as above; rows hold no duplicates, so the
  // mirrors found are distinct and the counts then force every lower entry to be one of them.
  int bad = 0;
  long long upper = 0, lower = 0;
#pragma omp parallel for schedule(dynamic, 4096) reduction(| : bad) reduction(+ : upper, lower)
  for (long long i = 0; i < n; ++i) {
    for (long long p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
      const int j = col_idx[p];
      if (j < 0 || j >= n) { bad |= 1; continue; }
      if (p > row_ptr[i] && col_idx[p - 1] >= j) bad |= 2;
      if (j > i) {
        ++upper;
        const int* lo = col_idx + row_ptr[j];
        const int* hi = col_idx + row_ptr[j + 1];
        if (!std::binary_search(lo, hi, (int)i)) bad |= 4;
      } else if (j < i) {
        ++lower;
      }
    }
  }
  if (upper != lower) bad |= 4;
  if (bad & 1) { err = "column index out of range"; return IDX_BAD_GRAPH; }
  if (bad & 2) { err = "columns of a row are not strictly ascending"; return IDX_BAD_GRAPH; }
  if (bad & 4) { err = "adjacency is not symmetric"; return IDX_BAD_GRAPH; }

  // nodes sorted by (community, original id): a stable counting sort
  g.comm_ptr.assign(n_comm + 1, 0);
  for (long long i = 0; i < n; ++i) {
    const int c = community[i];
    if (c < 0 || c >= n_comm) { err = "community id out of range"; return IDX_BAD_COMMUNITY; }
    g.comm_ptr[c + 1]++;
  }
  for (int m = 0; m < n_comm; ++m) {
    if (g.comm_ptr[m + 1] == 0) { err = "empty community"; return IDX_BAD_COMMUNITY; }
    g.comm_ptr[m + 1] += g.comm_ptr[m];
  }
  g.perm.resize(n);
  g.inv.resize(n);
  g.row_comm.resize(n);
  {
    std::vector<int> cursor(g.comm_ptr.begin(), g.comm_ptr.end() - 1);
    for (long long i = 0; i < n; ++i) {
      const int pos = cursor[community[i]]++;
      g.perm[pos] = (int)i;
      g.inv[i] = pos;
      g.row_comm[pos] = community[i];
    }
  }

  // A + I in new ids: row lengths, then columns (self loops of the input dropped, one identity)
  g.row_ptr.assign(n + 1, 0);
  g.dinv.resize(n);
#pragma omp parallel for schedule(static)
  for (long long i = 0; i < n; ++i) {
    const long long o = g.perm[i];
    int deg = 0;
    for (long long p = row_ptr[o]; p < row_ptr[o + 1]; ++p) deg += (col_idx[p] != o);
    g.row_ptr[i + 1] = deg + 1;
    g.dinv[i] = (float)(1.0 / std::sqrt((double)deg + 1.0));
  }
  for (long long i = 0; i < n; ++i) g.row_ptr[i + 1] += g.row_ptr[i];
  g.nnz = g.row_ptr[n];
  g.col.resize(g.nnz);
  g.seg_row_ptr.assign(n + 1, 0);
#pragma omp parallel for schedule(dynamic, 4096)
  for (long long i = 0; i < n; ++i) {
    const long long o = g.perm[i];
    int* dst = g.col.data() + g.row_ptr[i];
    int k = 0;
    for (long long p = row_ptr[o]; p < row_ptr[o + 1]; ++p)
      if (col_idx[p] != o) dst[k++] = g.inv[col_idx[p]];
    dst[k++] = (int)i;
    std::sort(dst, dst + k);
    int segs = 0;
    for (int t = 0; t < k; ++t)
      if (t == 0 || g.row_comm[dst[t]] != g.row_comm[dst[t - 1]]) ++segs;
    g.seg_row_ptr[i + 1] = segs;
  }
  for (long long i = 0; i < n; ++i) g.seg_row_ptr[i + 1] += g.seg_row_ptr[i];
  const long long n_seg = g.seg_row_ptr[n];
  g.seg_comm.resize(n_seg);
  g.seg_begin.resize(n_seg + 1);
#pragma omp parallel for schedule(dynamic, 4096)
  for (long long i = 0; i < n; ++i) {
    int s = g.seg_row_ptr[i];
    for (int p = g.row_ptr[i]; p < g.row_ptr[i + 1]; ++p) {
      if (p == g.row_ptr[i] || g.row_comm[g.col[p]] != g.row_comm[g.col[p - 1]]) {
        g.seg_comm[s] = g.row_comm[g.col[p]];
        g.seg_begin[s] = p;
        ++s;
      }
    }
  }
  g.seg_begin[n_seg] = (int)g.nnz;
  return IDX_OK;
}

// ------------------------------------------------------------------------------------------
// Work items for long rows.  Row lengths follow a power law, and a warp walks the stored entries
// of its row one after the other: a row of thousands of entries keeps one warp busy long after
// every other row is done.  Rows with more than `limit` stored entries are therefore cut into
// items of at most `limit` entries, each handled by a warp of its own.  Cuts fall between
// community segments wherever a segment fits (an item of whole segments can be scored without
// help in the Z search); a segment longer than `limit` is cut into even pieces whose partial
// sums are put together afterwards.
//   items[k] = {row, first entry, one past the last entry, split}   split = -1: whole segments,
//                                                                   else index into `split`
//   split[s] = {row, community, first item, number of items}        (pieces are consecutive items)
//   rows[r]  = {row, first item, number of items, 0}                (items of a row are consecutive)
// ------------------------------------------------------------------------------------------
struct Quad { int x, y, z, w; };
struct LongRowTables {
  std::vector<Quad> items, split, rows;
};

template <typename ItemFn, typename SplitFn>
inline void walk_long_row(const GraphIndex& g, int row, int limit, ItemFn&& item, SplitFn&& split) {
  int group_beg = g.row_ptr[row];
  for (int s = g.seg_row_ptr[row]; s < g.seg_row_ptr[row + 1]; ++s) {
    const int sb = g.seg_begin[s], se = g.seg_begin[s + 1], len = se - sb;
    if (len > limit) {
      if (sb > group_beg) item(group_beg, sb, false);
      const int pieces = (len + limit - 1) / limit;
      split(g.seg_comm[s], pieces);
      for (int k = 0; k < pieces; ++k)
        item(sb + (int)((long long)len * k / pieces), sb + (int)((long long)len * (k + 1) / pieces), true);
      group_beg = se;
    } else if (se - group_beg > limit) {
      item(group_beg, sb, false);
      group_beg = sb;
    }
  }
  if (group_beg < g.row_ptr[row + 1]) item(group_beg, g.row_ptr[row + 1], false);
}

inline void build_long_row_tables(const GraphIndex& g, int limit, LongRowTables& t) {
  t.items.clear(); t.split.clear(); t.rows.clear();
  std::vector<int> long_rows;
  for (long long i = 0; i < g.n; ++i)
    if (g.row_ptr[i + 1] - g.row_ptr[i] > limit) long_rows.push_back((int)i);
  const long long nl = (long long)long_rows.size();
  if (nl == 0) return;
  std::vector<long long> item_at(nl + 1, 0), split_at(nl + 1, 0);
#pragma omp parallel for schedule(dynamic, 256)
  for (long long r = 0; r < nl; ++r) {
    long long ni = 0, ns = 0;
    walk_long_row(g, long_rows[r], limit, [&](int, int, bool) { ++ni; }, [&](int, int) { ++ns; });
    item_at[r + 1] = ni;
    split_at[r + 1] = ns;
  }
  for (long long r = 0; r < nl; ++r) { item_at[r + 1] += item_at[r]; split_at[r + 1] += split_at[r]; }
  t.items.resize((size_t)item_at[nl]);
  t.split.resize((size_t)split_at[nl]);
  t.rows.resize((size_t)nl);
#pragma omp parallel for schedule(dynamic, 256)
  for (long long r = 0; r < nl; ++r) {
    const int row = long_rows[r];
    long long ni = item_at[r], ns = split_at[r];
    int cur_split = -1;
    walk_long_row(
        g, row, limit,
        [&](int b, int e, bool piece) { t.items[(size_t)ni++] = Quad{row, b, e, piece ? cur_split : -1}; },
        [&](int comm, int pieces) {
          cur_split = (int)ns;
          t.split[(size_t)ns++] = Quad{row, comm, (int)ni, pieces};
        });
    t.rows[(size_t)r] = Quad{row, (int)item_at[r], (int)(item_at[r + 1] - item_at[r]), 0};
  }
}

// First-order neighbour rows of community m: new ids outside V_m adjacent to V_m, ascending.
inline std::vector<int> halo1_of(const GraphIndex& g, int m) {
  std::vector<int> out;
  const int lo = g.comm_ptr[m], hi = g.comm_ptr[m + 1];
  for (int i = lo; i < hi; ++i)
    for (int p = g.row_ptr[i]; p < g.row_ptr[i + 1]; ++p) {
      const int j = g.col[p];
      if (j < lo || j >= hi) out.push_back(j);
    }
  std::sort(out.begin(), out.end());
  out.erase(std::unique(out.begin(), out.end()), out.end());
  return out;
}

// Second-order neighbour rows: outside V_m and halo1(m), adjacent to halo1(m), ascending.
inline std::vector<int> halo2_of(const GraphIndex& g, int m) {
  const std::vector<int> h1 = halo1_of(g, m);
  std::vector<int> out;
  const int lo = g.comm_ptr[m], hi = g.comm_ptr[m + 1];
  for (int j : h1)
    for (int p = g.row_ptr[j]; p < g.row_ptr[j + 1]; ++p) {
      const int k = g.col[p];
      if (k >= lo && k < hi) continue;
      if (std::binary_search(h1.begin(), h1.end(), k)) continue;
      out.push_back(k);
    }
  std::sort(out.begin(), out.end());
  out.erase(std::unique(out.begin(), out.end()), out.end());
  return out;
}

// N_m: communities other than m that own a node adjacent to V_m, ascending.
inline std::vector<int> nbr_of(const GraphIndex& g, int m) {
  std::vector<char> seen(g.n_comm, 0);
  const int lo = g.comm_ptr[m], hi = g.comm_ptr[m + 1];
  for (int i = lo; i < hi; ++i)
    for (int s = g.seg_row_ptr[i]; s < g.seg_row_ptr[i + 1]; ++s) seen[g.seg_comm[s]] = 1;
  std::vector<int> out;
  for (int c = 0; c < g.n_comm; ++c)
    if (seen[c] && c != m) out.push_back(c);
  return out;
}

}  // namespace gcn_admm_host
