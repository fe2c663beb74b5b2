// Host-side community reordering and index tables (Section 2 of the paper: V_m, N_m and the
// block split of A~; Appendix A: first- and second-order neighbour rows).  Runs once at
// creation, outside every ADMM iteration.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <new>
#include <string>
#include <utility>
#include <vector>
#include <sys/mman.h>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace gcn_admm_host {

// Allocator of the tables that hold one element per stored entry (hundreds of MB): `resize` leaves the
// elements uninitialised, so the threads that fill a table are the first to touch its pages (no serial zero
// fill), and blocks of 4 MB or more are 2 MB-aligned and marked for transparent huge pages (512 times fewer
// page faults where the system grants them).
template <class T>
struct TableAlloc {
  using value_type = T;
  TableAlloc() = default;
  template <class U> TableAlloc(const TableAlloc<U>&) {}
  T* allocate(std::size_t count) {
    const std::size_t bytes = count * sizeof(T), huge = (std::size_t)2 << 20;
    void* p;
    if (bytes >= 2 * huge) {
      const std::size_t rounded = (bytes + huge - 1) / huge * huge;
      p = std::aligned_alloc(huge, rounded);
      if (p) madvise(p, rounded, MADV_HUGEPAGE);
    } else {
      p = std::malloc(bytes ? bytes : 1);
    }
    if (!p) throw std::bad_alloc();
    return static_cast<T*>(p);
  }
  void deallocate(T* p, std::size_t) { std::free(p); }
  template <class U> void construct(U* p) { ::new (static_cast<void*>(p)) U; }
  template <class U, class... A> void construct(U* p, A&&... a) { ::new (static_cast<void*>(p)) U(std::forward<A>(a)...); }
  template <class U> bool operator==(const TableAlloc<U>&) const { return true; }
  template <class U> bool operator!=(const TableAlloc<U>&) const { return false; }
};
template <class T> using Table = std::vector<T, TableAlloc<T>>;

struct GraphIndex {
  long long n = 0;
  int n_comm = 0;
  long long nnz = 0;               // stored entries of A + I
  std::vector<int> perm, inv;      // new -> original, original -> new
  std::vector<int> comm_ptr;       // [M+1]
  std::vector<int> row_comm;       // community of each new id
  std::vector<int> row_ptr;        // A + I in new ids
  Table<int> col;                  // its columns, ascending in each row
  Table<unsigned short> col_comm;  // community of every stored column (n_comm <= 65535)
  std::vector<float> dinv;         // (deg_A + 1)^(-1/2) per new id
  std::vector<int> seg_row_ptr;
  Table<int> seg_comm, seg_begin;
};

enum { IDX_OK = 0, IDX_BAD_GRAPH = 1, IDX_BAD_COMMUNITY = 2 };

// Two independent 64-bit mixers (finalisers in the style of splitmix64 with different constants) for the
// fingerprints of the symmetry check.
inline uint64_t fingerprint_a(uint64_t x) {
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ULL;
  x ^= x >> 27; x *= 0x94d049bb133111ebULL;
  return x ^ (x >> 31);
}
inline uint64_t fingerprint_b(uint64_t x) {
  x += 0x9e3779b97f4a7c15ULL;
  x ^= x >> 33; x *= 0xff51afd7ed558ccdULL;
  x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ULL;
  return x ^ (x >> 33);
}

// Validates the CSR of A and the community assignment and fills `g`.
inline int build_graph_index(long long n, const long long* row_ptr, const int* col_idx, int n_comm,
                             const int* community, GraphIndex& g, std::string& err) {
  g.n = n;
  g.n_comm = n_comm;
  if (n_comm < 1 || n_comm > 65535) { err = "the number of communities must lie in 1..65535"; return IDX_BAD_COMMUNITY; }
  if (row_ptr[0] != 0) { err = "row_ptr[0] must be 0"; return IDX_BAD_GRAPH; }
  for (long long i = 0; i < n; ++i)
    if (row_ptr[i + 1] < row_ptr[i]) { err = "row_ptr is not ascending"; return IDX_BAD_GRAPH; }
  if (row_ptr[n] + n > 2147483647LL) { err = "more than 2^31-1 stored entries"; return IDX_BAD_GRAPH; }
  // One streaming pass over the entries: range, strictly ascending columns, self loops, symmetry.
  // Symmetry: rows hold no duplicates, so A is symmetric exactly when the set of unordered pairs {i, j}
  // stored above the diagonal equals the set stored below it.  The two sets are compared by their sizes
  // and by two independent 64-bit sums of mixed pair keys (a set difference survives only if both sums
  // collide); a mirror search per entry costs a cache miss each and was a third of the whole index build.
  int bad = 0;
  long long upper = 0, lower = 0;
  uint64_t ua = 0, ub = 0, la = 0, lb = 0;
  std::vector<unsigned char> self_loop((size_t)n, 0);
#pragma omp parallel for schedule(dynamic, 4096) reduction(| : bad) reduction(+ : upper, lower, ua, ub, la, lb)
  for (long long i = 0; i < n; ++i) {
    for (long long p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
      const int j = col_idx[p];
      if (j < 0 || j >= n) { bad |= 1; continue; }
      if (p > row_ptr[i] && col_idx[p - 1] >= j) bad |= 2;
      if (j > i) {
        const uint64_t key = ((uint64_t)i << 32) | (uint64_t)(uint32_t)j;
        ++upper; ua += fingerprint_a(key); ub += fingerprint_b(key);
      } else if (j < i) {
        const uint64_t key = ((uint64_t)j << 32) | (uint64_t)(uint32_t)i;
        ++lower; la += fingerprint_a(key); lb += fingerprint_b(key);
      } else {
        self_loop[(size_t)i] = 1;
      }
    }
  }
  if (upper != lower || ua != la || ub != lb) bad |= 4;
  if (bad & 1) { err = "column index out of range"; return IDX_BAD_GRAPH; }
  if (bad & 2) { err = "columns of a row are not strictly ascending"; return IDX_BAD_GRAPH; }
  if (bad & 4) { err = "adjacency is not symmetric"; return IDX_BAD_GRAPH; }

  // nodes sorted by (community, original id): a stable counting sort, the nodes cut into one slice per
  // thread (a histogram per slice, then every slice scatters its nodes behind those of the slices before it)
  g.comm_ptr.assign(n_comm + 1, 0);
  g.perm.resize(n);
  g.inv.resize(n);
  g.row_comm.resize(n);
  {
    int n_slices = 1;
#ifdef _OPENMP
    n_slices = std::max(1, std::min(omp_get_max_threads(), (int)std::min<long long>(64, (long long)(32 << 20) / std::max(n_comm, 1))));
#endif
    n_slices = (int)std::max<long long>(1, std::min<long long>(n_slices, n / 1024));
    std::vector<int> hist((size_t)n_slices * n_comm, 0);
    int out_of_range = 0;
#pragma omp parallel for schedule(static, 1) reduction(| : out_of_range)
    for (int t = 0; t < n_slices; ++t) {
      int* mine = hist.data() + (size_t)t * n_comm;
      for (long long i = n * t / n_slices; i < n * (t + 1) / n_slices; ++i) {
        const int c = community[i];
        if (c < 0 || c >= n_comm) { out_of_range = 1; continue; }
        ++mine[c];
      }
    }
    if (out_of_range) { err = "community id out of range"; return IDX_BAD_COMMUNITY; }
    int at = 0;
    for (int m = 0; m < n_comm; ++m) {
      g.comm_ptr[m] = at;
      for (int t = 0; t < n_slices; ++t) {
        const int here = hist[(size_t)t * n_comm + m];
        hist[(size_t)t * n_comm + m] = at;
        at += here;
      }
      if (at == g.comm_ptr[m]) { err = "empty community"; return IDX_BAD_COMMUNITY; }
    }
    g.comm_ptr[n_comm] = at;
#pragma omp parallel for schedule(static, 1)
    for (int t = 0; t < n_slices; ++t) {
      int* cursor = hist.data() + (size_t)t * n_comm;
      for (long long i = n * t / n_slices; i < n * (t + 1) / n_slices; ++i) {
        const int pos = cursor[community[i]]++;
        g.perm[pos] = (int)i;
        g.inv[i] = pos;
        g.row_comm[pos] = community[i];
      }
    }
  }

  // A + I in new ids: row lengths, then columns (self loops of the input dropped, one identity)
  g.row_ptr.assign(n + 1, 0);
  g.dinv.resize(n);
#pragma omp parallel for schedule(static)
  for (long long i = 0; i < n; ++i) {
    const long long o = g.perm[i];
    const int deg = (int)(row_ptr[o + 1] - row_ptr[o]) - (int)self_loop[(size_t)o];
    g.row_ptr[i + 1] = deg + 1;
    g.dinv[i] = (float)(1.0 / std::sqrt((double)deg + 1.0));
  }
  for (long long i = 0; i < n; ++i) g.row_ptr[i + 1] += g.row_ptr[i];
  g.nnz = g.row_ptr[n];
  g.col.resize(g.nnz);
  g.col_comm.resize(g.nnz);
  g.seg_row_ptr.assign(n + 1, 0);
  // New ids ascend with (community, original id) and the given rows ascend in original id, so a sorted row in
  // new ids is the given row partitioned by community with the order inside each community kept: a counting
  // sort over the communities the row touches (a comparison sort of every row was three quarters of this pass).
  // The row's own index (the identity entry) enters the walk where the original id says.
  {
    std::vector<uint64_t> where((size_t)n);   // community and new id of an original id, side by side
#pragma omp parallel for schedule(static)
    for (long long j = 0; j < n; ++j) where[(size_t)j] = ((uint64_t)(uint32_t)community[j] << 32) | (uint32_t)g.inv[j];
#pragma omp parallel
    {
      std::vector<int> count((size_t)n_comm, 0), touched, ids;
      std::vector<unsigned short> comms;
#pragma omp for schedule(dynamic, 4096)
      for (long long i = 0; i < n; ++i) {
        const long long o = g.perm[i];
        const long long len = row_ptr[o + 1] - row_ptr[o];
        if ((long long)ids.size() < len + 1) { ids.resize((size_t)len + 1); comms.resize((size_t)len + 1); }
        touched.clear();
        int k = 0;
        auto put = [&](int id, int c) {
          ids[(size_t)k] = id;
          comms[(size_t)k] = (unsigned short)c;
          if (count[(size_t)c]++ == 0) touched.push_back(c);
          ++k;
        };
        bool self_in = false;
        for (long long p = row_ptr[o]; p < row_ptr[o + 1]; ++p) {
          const int j = col_idx[p];
          if (!self_in && j >= o) { put((int)i, g.row_comm[i]); self_in = true; }
          if (j != o) { const uint64_t w = where[(size_t)j]; put((int)(uint32_t)w, (int)(w >> 32)); }
        }
        if (!self_in) put((int)i, g.row_comm[i]);
        std::sort(touched.begin(), touched.end());
        int base = 0;
        for (int c : touched) { const int here = count[(size_t)c]; count[(size_t)c] = base; base += here; }
        int* dst = g.col.data() + g.row_ptr[i];
        unsigned short* cdst = g.col_comm.data() + g.row_ptr[i];
        for (int t = 0; t < k; ++t) {
          const int at = count[comms[(size_t)t]]++;
          dst[at] = ids[(size_t)t];
          cdst[at] = comms[(size_t)t];
        }
        for (int c : touched) count[(size_t)c] = 0;
        g.seg_row_ptr[i + 1] = (int)touched.size();
      }
    }
  }
  for (long long i = 0; i < n; ++i) g.seg_row_ptr[i + 1] += g.seg_row_ptr[i];
  const long long n_seg = g.seg_row_ptr[n];
  g.seg_comm.resize(n_seg);
  g.seg_begin.resize(n_seg + 1);
#pragma omp parallel for schedule(dynamic, 4096)
  for (long long i = 0; i < n; ++i) {
    int s = g.seg_row_ptr[i];
    for (int p = g.row_ptr[i]; p < g.row_ptr[i + 1]; ++p) {
      if (p == g.row_ptr[i] || g.col_comm[p] != g.col_comm[p - 1]) {
        g.seg_comm[s] = g.col_comm[p];
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
