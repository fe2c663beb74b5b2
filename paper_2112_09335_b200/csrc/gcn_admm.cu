// C-ABI library of the community-based ADMM GCN trainer: host orchestration of the kernels in
// kernels.cuh.  See include/gcn_admm.h for the contract of every entry point.
#include "../../include/gcn_admm.h"

#include <climits>
#include <cmath>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "gemm_tc.cuh"
#include "graph_index.hpp"
#include "kernels.cuh"
#include "shard_plan.hpp"

using gcn_admm_host::GraphIndex;

namespace {
// Named range on the profiler timeline (NVTX; a no-op unless a tool is attached) for the life of the object.
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};
}  // namespace
using gk::SearchCtl;

namespace {

constexpr int kLogPasses = 256;
constexpr int kSmCount = 148;
constexpr long long kImageMinRows = 16384;   // row count from which the weight operand is pre-split
constexpr int kZBlockRows = 32;      // rows per block of the hidden-layer gradient's closing sweep
constexpr int kChunksPerGroup = 256; // chunks whose sums one block of k_reduce_chunks adds up
constexpr int kCandZ = 4;           // theta candidates scored per sweep (2..4; steady-state searches close at trial 0..2)
constexpr int kDefaultLongRow = 256;   // stored entries one warp walks before a row is cut into items

thread_local std::string g_create_error;

inline int ldpad(int c) { return (c + 3) & ~3; }
constexpr int kMaxWidth = 1 << 24;   // widest matrix an entry point accepts (keeps the padded width inside int)

// Output function of the splitmix64 generator applied to the state x + 0x9E3779B97F4A7C15.
inline unsigned long long splitmix64(unsigned long long x) {
  unsigned long long z = x + 0x9E3779B97F4A7C15ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
inline long long cdiv(long long a, long long b) { return (a + b - 1) / b; }

struct Fail {
  int code;
  std::string msg;
};

#define CU(expr)                                                                           \
  do {                                                                                     \
    cudaError_t e__ = (expr);                                                              \
    if (e__ != cudaSuccess)                                                                \
      throw Fail{GCN_ADMM_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)};  \
  } while (0)

template <typename T>
T* dalloc(size_t count) {
  void* p = nullptr;
  cudaError_t e = cudaMalloc(&p, std::max<size_t>(count, 1) * sizeof(T));
  if (e != cudaSuccess)
    throw Fail{e == cudaErrorMemoryAllocation ? GCN_ADMM_ERR_ALLOC : GCN_ADMM_ERR_CUDA,
               std::string("cudaMalloc: ") + cudaGetErrorString(e)};
  return static_cast<T*>(p);
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link the driver API directly).
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      p = nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Tensor map of a row-major rows x ld fp32 matrix for 128-row x 32-column tiles written with the 128-byte
// swizzle; elements outside the matrix read as zero.  False when the map cannot be made (the caller then
// stages the operand through registers).
bool make_a_tile_map(const float* A, long long rows, int ld, CUtensorMap* map) {
  EncodeTiledFn fn = encode_tiled();
  if (fn == nullptr || ld < gtc::kChunkK) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)ld, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)gtc::kChunkK, (cuuint32_t)gtc::kBlockM};
  const cuuint32_t elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(A), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool is_device_pointer(const void* p) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged;
}

}  // namespace

struct ProfStat {
  long long launches = 0;
  double ms = 0.0, bytes = 0.0, flops = 0.0;
};
struct ProfPending {
  ProfStat* stat;
  cudaEvent_t a, b;
};

struct gcn_admm {
  gcn_admm_params p{};
  // launch accounting: every kernel launch goes through a Scope (below)
  long long launches = 0;
  bool profiling = false;
  std::map<std::string, ProfStat> prof;
  std::vector<ProfPending> pending;
  std::vector<cudaEvent_t> event_pool;
  cudaEvent_t get_event() {
    if (!event_pool.empty()) { cudaEvent_t e = event_pool.back(); event_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  // Counts `kernels` launches; when profiling, brackets them with events on the handle's stream and
  // books the algorithmic bytes / flops of the work under `name`.
  struct Scope {
    gcn_admm* h;
    cudaEvent_t b = nullptr;
    Scope(gcn_admm* h_, const char* name, int kernels, double bytes, double flops) : h(h_) {
      h->launches += kernels;
      if (!h->profiling) return;
      ProfStat& st = h->prof[name];
      st.launches += kernels;
      st.bytes += bytes;
      st.flops += flops;
      cudaEvent_t a = h->get_event();
      b = h->get_event();
      cudaEventRecord(a, h->stream);
      h->pending.push_back(ProfPending{&st, a, b});
    }
    ~Scope() { if (b) cudaEventRecord(b, h->stream); }
  };
  void collect_profile() {
    cudaStreamSynchronize(stream);
    for (ProfPending& q : pending) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, q.a, q.b) == cudaSuccess) q.stat->ms += ms;
      event_pool.push_back(q.a);
      event_pool.push_back(q.b);
    }
    pending.clear();
  }

  cudaStream_t stream = nullptr;
  int L = 0;
  long long n = 0;
  int M = 0;
  int n_train = 0;
  std::vector<int> C, ld;   // widths C_0..C_L and their padded leading dimensions
  int max_ld = 0;
  GraphIndex gi;
  std::vector<void*> owned;  // every device allocation, for destroy

  int *d_row_ptr = nullptr, *d_col = nullptr, *d_row_comm = nullptr, *d_perm = nullptr;
  int* d_y = nullptr;
  float* d_dinv = nullptr;
  unsigned short* d_col_comm = nullptr;   // community of every stored column
  // rows too long for one warp, cut into items (see gcn_admm_host::LongRowTables)
  int4 *d_items = nullptr, *d_split = nullptr, *d_long_rows = nullptr;
  int n_items = 0, n_split = 0, n_long = 0, long_len = 0;
  float* item_sums = nullptr;             // n_items x max_ld
  size_t item_sums_elems = 0;
  unsigned char* d_train = nullptr;
  int* d_train_rows = nullptr;            // new ids of the training rows, ascending
  float* d_fista_momentum = nullptr;      // (t_j - 1) / t_{j+1}, j = 1..fista_iters

  std::vector<float*> W, Wt, Z, P, H;   // 1..L
  float* U = nullptr;
  float *B0 = nullptr, *B1 = nullptr, *B2 = nullptr;   // N x max_ld scratch
  float* grad = nullptr;     // max over l of C_{l-1} x ld_l
  float* grad_t = nullptr;   // its transpose, C_l x ld_{l-1} (K-major operand of the tensor-core product)
  int* tc_error = nullptr;   // raised by a tensor-core product whose bounded wait ran out
  uint8_t* b_image = nullptr;   // split weight operand in the staged layout (see gtc::k_split_b)
  size_t b_image_bytes = 0;
  float* part = nullptr;     // split partial sums of the transposed product
  size_t part_elems = 0;
  SearchCtl *ctl_w = nullptr, *ctl_z = nullptr;   // [L+1], [(L+1) * M]
  double *sums_w = nullptr, *sums_z = nullptr, *obj = nullptr;
  double* red_part = nullptr;               // per-block partial sums awaiting their fixed-order reduction
  int2* d_zblocks = nullptr;                // row blocks of at most kZBlockRows rows, none crossing a community
  int* d_comm_block_ptr = nullptr;          // [M+1] first row block of every community
  int n_zblocks = 0;
  int *n_active = nullptr, *status = nullptr, *d_pass = nullptr;
  // Z scoring: units in chunks of about equally many stored entries, dealt to the warps of the grid in a fixed order
  int* d_chunk_ptr = nullptr;
  int* d_row_order = nullptr;               // rows per community by falling length: the order of the kernels that put several rows in a warp
  int* d_chunk_ptr_sorted = nullptr;        // chunk table of the units in that order
  int n_chunks_sorted = 0;
  int n_chunks = 0;
  double* z_chunk_part = nullptr;           // [chunk][M][candidates] sums of one sweep, per chunk of units
  double* z_group_part = nullptr;           // [group of chunks][M][candidates], chunks added in order
  int* chunk_counter = nullptr;             // hands the chunks out to the warps of a sweep
  int n_groups = 0;
  double* split_scores = nullptr;           // [n_split][candidates] sums of the segments scored in pieces
  int *d_split_order = nullptr, *d_split_ptr = nullptr;   // split entries grouped by community
  cudaGraphExec_t pass_graph = nullptr;   // one pass of Algorithm 1, recorded once and replayed
  int *log_trial_w = nullptr, *log_trial_z = nullptr;
  double *log_q_w = nullptr, *log_q_z = nullptr;
  long long log_count = 0;
  long long launches_per_pass = 0;
  bool fresh = false;        // P_l, H_l agree with the stored W, Z
  std::string err;
  std::vector<int> ix_cache[16];
  gcn_admm_host::ShardPlan shard_plan;      // last plan asked for (host only)
  std::vector<int> shard_ranges;

  template <typename T>
  T* alloc(size_t count) {
    T* p_ = dalloc<T>(count);
    owned.push_back(p_);
    return p_;
  }
  int grid_for(long long work_items, int per_block = 256) const {
    return (int)std::max<long long>(1, std::min<long long>(cdiv(work_items, per_block), (long long)kSmCount * 8));
  }

  // ---- launches -----------------------------------------------------------------------
  void spmm(const float* x, float* out, int ldx) {
    char name[48];
    std::snprintf(name, sizeof name, "spmm@%d", ldx);
    Scope sc(this, name, 1, 4.0 * gi.nnz + 8.0 * n + 8.0 * (double)n * ldx, 2.0 * (double)gi.nnz * ldx);
    // Long rows go as items unless the operand is wider than the item buffer was sized for (a
    // caller's matrix wider than every layer): then they are walked whole, slower but the same sums.
    const bool cut = n_items > 0 && (size_t)n_items * ldx <= item_sums_elems;
    spmm_launch(d_row_ptr, d_col, d_dinv, d_row_order, (int)n, d_items, cut ? n_items : 0, cut ? long_len : INT_MAX, x, out, ldx);
    if (cut) {
      gk::k_spmm_long_rows<<<(unsigned)n_long, 64, 0, stream>>>(d_long_rows, reinterpret_cast<const float4*>(item_sums),
                                                                reinterpret_cast<float4*>(out), ldx / 4);
      CU(cudaGetLastError());
      ++launches;   // booked with the propagation it completes
    }
  }

  // The propagation kernel on a graph given by its tables (the handle's own, or a rank's local part of it):
  // rows 0 .. nn-1 of out = A~ x, columns of `cl` index rows of x.  `order` lists the rows by falling length
  // (used by the forms that put several rows in a warp).
  void spmm_launch(const int* rp, const int* cl, const float* dv, const int* order, int nn, const int4* its, int items_used,
                   int long_eff, const float* x, float* out, int ldx) {
    const int ld4 = ldx / 4;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    float4* o4 = reinterpret_cast<float4*>(out);
    // 64-thread blocks: rows differ widely in length, small blocks keep the SMs evenly loaded.
#define SPMM_CASE(G, V, UN)                                                                    \
  {                                                                                            \
    const long long threads = ((long long)nn + items_used) * (G);                              \
    /* several rows per warp (G < 32): rows of equal length side by side */                     \
    gk::k_spmm<G, V, UN, ((G) < 32)><<<(unsigned)cdiv(threads, 64), 64, 0, stream>>>(rp, cl, dv, x4, o4, nn, ld4, \
        its, items_used, long_eff, reinterpret_cast<float4*>(item_sums), order);               \
  }
    if (ld4 <= 1) SPMM_CASE(1, 1, 4)
    else if (ld4 <= 2) SPMM_CASE(2, 1, 4)
    else if (ld4 <= 4) SPMM_CASE(4, 1, 8)
    else if (ld4 <= 8) SPMM_CASE(8, 1, 8)
    else if (ld4 <= 16) SPMM_CASE(16, 1, 8)
    else if (ld4 <= 32) SPMM_CASE(32, 1, 4)
    else SPMM_CASE(32, 2, 2)   // two neighbours in flight per lane beat four (fewer registers, more warps): measured
#undef SPMM_CASE
    CU(cudaGetLastError());
  }

  // C = A B.  B is handed over twice: row-major K x N (ldb) for the fp32-ALU kernels and K-major
  // N x K (Bk, ldbk; may be NULL) for the tensor-core kernel, which is used whenever it applies
  // (K capped at 2048 because its accumulator error grows with K, about 2.5e-9 K of the magnitude).
  void gemm_nn(const float* A, int lda, const float* B, int ldb, const float* Bk, int ldbk, float* Cm, int ldc,
               long long Mr, int N, int K, const int* skip = nullptr) {
    char name[48];
    if (p.tensor_cores && Bk != nullptr && K >= 8 && K <= 2048 && Mr >= 512) {
      std::snprintf(name, sizeof name, "gemm_tc@%dx%d", K, N);
      Scope sc(this, name, 1, 4.0 * ((double)Mr * (lda + ldc) + (double)K * ldb), 2.0 * (double)Mr * N * K);
      const int tiles = (int)cdiv(Mr, gtc::kBlockM);
      CUtensorMap tmap;
      std::memset(&tmap, 0, sizeof tmap);
      // With many row tiles the weight operand is split once into an image of the staged layout and
      // fetched by bulk copies; with few (launch-bound problems) the extra launch costs more than the
      // producers' repeated work.  tensor_cores = 2 takes the image at every size.
#define TC_WS(NT)                                                                                              \
  {                                                                                                            \
    const size_t smem = gtc::WsCfg<NT>::kSmem;                                                                 \
    const int groups = (int)cdiv(N, NT);                                                                       \
    const size_t image_bytes = (size_t)groups * cdiv(K, gtc::kChunkK) * 2 * (NT) * gtc::kChunkK * 4;            \
    dim3 grid((unsigned)std::max(1, std::min(tiles, kSmCount / groups)), (unsigned)groups);                    \
    if ((p.tensor_cores == 2 || Mr >= kImageMinRows) && image_bytes <= b_image_bytes) {                        \
      const long long work = (long long)groups * cdiv(K, gtc::kChunkK) * (NT) * 8;                             \
      gtc::k_split_b<<<(unsigned)std::min<long long>(cdiv(work, 256), 4 * kSmCount), 256, 0, stream>>>(Bk, ldbk, N, K, NT, b_image); \
      ++launches;                                                                                              \
      /* up to 128 columns: A tiles by tensor copies into a ring of their own (at 256 columns shared memory    \
         leaves no room for it, and the form measured no faster there) */                                      \
      if ((NT) <= 128 && make_a_tile_map(A, Mr, lda, &tmap)) {                                                 \
        const size_t smem_ring = gtc::WsCfg<NT>::kSmemRing;                                                    \
        CU(cudaFuncSetAttribute(gtc::k_gemm_tc_ws<NT, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_ring)); \
        gtc::k_gemm_tc_ws<NT, true, true><<<grid, gtc::WsCfg<NT>::kThreads + 32, smem_ring, stream>>>(A, lda, Bk, ldbk, Cm, ldc, (int)Mr, N, K, skip, tc_error, b_image, tmap); \
      } else {                                                                                                 \
        CU(cudaFuncSetAttribute(gtc::k_gemm_tc_ws<NT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        gtc::k_gemm_tc_ws<NT, true><<<grid, gtc::WsCfg<NT>::kThreads, smem, stream>>>(A, lda, Bk, ldbk, Cm, ldc, (int)Mr, N, K, skip, tc_error, b_image, tmap); \
      }                                                                                                        \
    } else {                                                                                                   \
      CU(cudaFuncSetAttribute(gtc::k_gemm_tc_ws<NT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
      gtc::k_gemm_tc_ws<NT, false><<<grid, gtc::WsCfg<NT>::kThreads, smem, stream>>>(A, lda, Bk, ldbk, Cm, ldc, (int)Mr, N, K, skip, tc_error, nullptr, tmap); \
    }                                                                                                          \
  }
      if (N <= 16) TC_WS(16)
      else if (N <= 32) TC_WS(32)
      else if (N <= 48) TC_WS(48)
      else if (N <= 64) TC_WS(64)
      else if (N <= 128) TC_WS(128)
      // 129..256 columns with a short reduction (K <= 128: a tile has at most four chunks of MMAs, so the epilogue
      // that the single accumulator set of the 256-column form leaves uncovered dominates): two groups of 128 columns
      // in the tensor-copy form instead, whose two accumulator sets put the epilogue under the next tile's MMAs
      // (measured on 1.2 M rows: 0.372 -> 0.326 ms at K = 47, 0.560 -> 0.463 at 100, 0.518 -> 0.456 at 128; no gain at 256)
      else if (K <= 128 && lda >= gtc::kChunkK && Mr >= kImageMinRows) TC_WS(128)
      else TC_WS(256)
#undef TC_WS
      CU(cudaGetLastError());
      return;
    }
    std::snprintf(name, sizeof name, "gemm_nn@%dx%d", K, N);
    Scope sc(this, name, 1, 4.0 * ((double)Mr * (lda + ldc) + (double)K * ldb), 2.0 * (double)Mr * N * K);
#define NN_CASE(BM, BN, BK, TM, TN)                                                             \
  {                                                                                             \
    dim3 grid((unsigned)cdiv(Mr, BM), (unsigned)cdiv(ldc, BN));                                  \
    gk::k_gemm_nn<BM, BN, BK, TM, TN><<<grid, (BM / TM) * (BN / TN), 0, stream>>>(A, lda, B, ldb, Cm, ldc, (int)Mr, N, K, skip); \
  }
    if (N > 64) NN_CASE(128, 128, 16, 8, 8)
    else if (N > 16) NN_CASE(128, 64, 16, 8, 4)
    else NN_CASE(256, 16, 16, 4, 4)
#undef NN_CASE
    CU(cudaGetLastError());
  }

  // out[Ka x ldp] = A^T B over `rows` rows, through split partial sums reduced in a fixed order.
  // Whether P^T R runs on the tensor cores (that form can also build a hidden layer's R itself).
  bool tn_on_tensor_cores(long long rows) const { return p.tensor_cores != 0 && rows >= 4096; }

  // With `zres` (tensor-core form only) B holds pre-activations H and the operand is
  // h > 0 ? nu (h - z) : 0, formed while staging: the residual matrix is never stored.
  void gemm_tn(const float* A, int lda, const float* B, int ldb, float* out, int ldp, long long rows, int Ka,
               int Nb, const float* zres = nullptr, float nu = 0.f) {
    int splits = 1;
    long long rps = rows;
    char name[48];
    if (zres && !tn_on_tensor_cores(rows)) throw Fail{GCN_ADMM_ERR_ARG, "fused residual needs the tensor-core product"};
    if (tn_on_tensor_cores(rows)) {
      std::snprintf(name, sizeof name, zres ? "gemm_tn_tc.resid@%dx%d" : "gemm_tn_tc@%dx%d", Ka, Nb);
      Scope sc(this, name, 2, 4.0 * ((double)rows * (lda + (zres ? 2 : 1) * ldb) + (double)Ka * ldp), 2.0 * (double)rows * Ka * Nb);
      const int nt_tn = Nb <= 16 ? 16 : Nb <= 32 ? 32 : Nb <= 48 ? 48 : Nb <= 64 ? 64 : Nb <= 128 ? 128 : 256;
      const int nb_groups = (int)cdiv(Nb, nt_tn);
      const int groups = (int)cdiv(Ka, gtc::kBlockM);
      // at most 2048 rows (256 MMAs) per accumulator: the tensor core rounds the running sum toward zero at
      // every MMA, so long sums are cut into splits whose partial results are added in fp64
      splits = (int)std::max<long long>(std::max(1, kSmCount / (groups * nb_groups)), cdiv(rows, 2048));
      {   // whole waves: with more CTAs than SMs (one CTA per SM), round the count up to a multiple of the SM count
        const long long per = (long long)groups * nb_groups;
        if (splits * per > kSmCount) splits = (int)(cdiv(splits * per, kSmCount) * kSmCount / per);
      }
      splits = (int)std::min<long long>(splits, cdiv(rows, 256));
      splits = (int)std::min<long long>(splits, (long long)(part_elems / ((size_t)Ka * ldp)));
      rps = cdiv(rows, splits);
      splits = (int)cdiv(rows, rps);
#define TN_TC(NT)                                                                                              \
  {                                                                                                            \
    const size_t smem = gtc::TnCfg<NT>::kSmem;                                                                 \
    dim3 grid((unsigned)groups, (unsigned)splits, (unsigned)nb_groups);                                        \
    if (zres) {                                                                                                \
      CU(cudaFuncSetAttribute(gtc::k_gemm_tn_tc<NT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
      gtc::k_gemm_tn_tc<NT, true><<<grid, gtc::kTnThreads, smem, stream>>>(A, lda, B, ldb, part, ldp, rows, rps, Ka, Nb, tc_error, zres, nu); \
    } else {                                                                                                   \
      CU(cudaFuncSetAttribute(gtc::k_gemm_tn_tc<NT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
      gtc::k_gemm_tn_tc<NT, false><<<grid, gtc::kTnThreads, smem, stream>>>(A, lda, B, ldb, part, ldp, rows, rps, Ka, Nb, tc_error, nullptr, 0.f); \
    }                                                                                                          \
  }
      if (Nb <= 16) TN_TC(16)
      else if (Nb <= 32) TN_TC(32)
      else if (Nb <= 48) TN_TC(48)
      else if (Nb <= 64) TN_TC(64)
      else if (Nb <= 128) TN_TC(128)
      else TN_TC(256)
#undef TN_TC
      CU(cudaGetLastError());
      const long long elems_tc = (long long)Ka * ldp;
      gk::k_reduce_splits<<<(unsigned)cdiv(elems_tc, 256), 256, 0, stream>>>(part, out, elems_tc, splits);
      CU(cudaGetLastError());
      return;
    }
    std::snprintf(name, sizeof name, "gemm_tn@%dx%d", Ka, Nb);
    Scope sc(this, name, 2, 4.0 * ((double)rows * (lda + ldb) + (double)Ka * ldp), 2.0 * (double)rows * Ka * Nb);
#define TN_CASE(BM, BN, BK, TM, TN)                                                             \
  {                                                                                             \
    const long long tiles = cdiv(Ka, BM) * cdiv(ldp, BN);                                        \
    splits = (int)std::max<long long>(1, std::min<long long>((4LL * kSmCount) / tiles, cdiv(rows, 64))); \
    splits = (int)std::min<long long>(splits, (long long)(part_elems / ((size_t)Ka * ldp)));     \
    rps = cdiv(rows, splits);                                                                    \
    splits = (int)cdiv(rows, rps);                                                               \
    dim3 grid((unsigned)cdiv(Ka, BM), (unsigned)cdiv(ldp, BN), (unsigned)splits);                \
    gk::k_gemm_tn<BM, BN, BK, TM, TN><<<grid, (BM / TM) * (BN / TN), 0, stream>>>(A, lda, B, ldb, part, ldp, rows, rps, Ka, Nb); \
  }
    if (Nb > 64) TN_CASE(128, 128, 16, 8, 8)
    else if (Nb > 16) TN_CASE(128, 64, 16, 8, 4)
    else if (Nb > 8) TN_CASE(128, 16, 16, 8, 1)
    else TN_CASE(128, 8, 16, 4, 1)
#undef TN_CASE
    CU(cudaGetLastError());
    const long long elems = (long long)Ka * ldp;
    gk::k_reduce_splits<<<(unsigned)cdiv(elems, 256), 256, 0, stream>>>(part, out, elems, splits);
    CU(cudaGetLastError());
  }

  void resid(int l, float* R) {   // derivative of phi_l with respect to H_l, at the stored H_l
    const long long n4 = n * ld[l] / 4;
    Scope sc(this, l < L ? "resid_hidden" : "resid_out", 1, 16.0 * n4 * (l < L ? 3 : 4), 0.0);
    if (l < L)
      gk::k_resid_hidden<<<grid_for(n4), 256, 0, stream>>>((const float4*)H[l], (const float4*)Z[l], (float4*)R, n4, p.nu);
    else
      gk::k_resid_out<<<grid_for(n4), 256, 0, stream>>>((const float4*)H[l], (const float4*)Z[l], (const float4*)U,
                                                        (float4*)R, n4, p.rho);
    CU(cudaGetLastError());
  }

  int n_passes(int cand) const { return (p.bt_max_trials + cand - 1) / cand; }

  long long z_per_pass() const { return (long long)std::max(L - 1, 0) * M; }

  void begin_log_pass() {
    const long long zc = z_per_pass();
    Scope sc(this, "small", zc > 0 ? 2 : 1, 0.0, 0.0);
    gk::k_log_clear<<<1, 64, 0, stream>>>(log_trial_w, d_pass, L, kLogPasses);
    if (zc > 0) gk::k_log_clear<<<grid_for(zc), 256, 0, stream>>>(log_trial_z, d_pass, zc, kLogPasses);
    CU(cudaGetLastError());
  }
  void end_log_pass() {
    Scope sc(this, "small", 1, 0.0, 0.0);
    gk::k_pass_advance<<<1, 1, 0, stream>>>(d_pass);
    CU(cudaGetLastError());
    ++log_count;
  }

  // ---- W_l block (Section 3.1) --------------------------------------------------------
  void update_W(int l) {
    Range range("gcn_admm: W block");
    const int Kp = C[l - 1], Cn = C[l], ldc = ld[l];
    const long long n4 = n * ldc / 4;
    SearchCtl* ctl = ctl_w + l;
    if (l < L && tn_on_tensor_cores(n)) {                               // grad = P_l^T R_l, R_l formed inside the product
      gemm_tn(P[l], ld[l - 1], H[l], ldc, grad, ldc, n, Kp, Cn, Z[l], p.nu);
    } else {
      resid(l, B0);                                                     // R_l
      gemm_tn(P[l], ld[l - 1], B0, ldc, grad, ldc, n, Kp, Cn);          // grad = P_l^T R_l
    }
    {
      Scope sc(this, "small", 3, 0.0, 0.0);
      gk::k_transpose_small<<<(unsigned)cdiv((long long)Kp * Cn, 256), 256, 0, stream>>>(grad, ldc, grad_t, ld[l - 1], Kp, Cn);
      gk::k_two_sumsq<<<1, 1024, 0, stream>>>(grad, W[l], (long long)Kp * ldc, sums_w);
      gk::k_search_begin<<<1, 32, 0, stream>>>(ctl, sums_w, p.bt_shrink, p.bt_growth, status);
      CU(cudaGetLastError());
    }
    gemm_nn(P[l], ld[l - 1], grad, ldc, grad_t, ld[l - 1], B1, ldc, n, Cn, Kp, &ctl->done);   // D = P_l grad
    gk::DecideArgs a{};
    a.growth = p.bt_growth;
    a.max_trials = p.bt_max_trials;
    a.cand = gk::kCand;
    const int score_grid = grid_for(n4);   // every block of a scoring sweep leaves its sums in red_part
    if (l == L) {
      {
        Scope sc(this, "score_w_out", 1, 32.0 * n4, 0.0);
        gk::k_score_w_out<<<score_grid, 256, 0, stream>>>((const float4*)B1, (const float4*)B0, n4, ctl, red_part);
      }
      a.mode = 1;
      a.quad_coef = 0.5 * p.rho;
      a.last_pass = 1;
      Scope sc(this, "small", 1, 0.0, 0.0);
      gk::k_search_decide_w<<<1, 256, 0, stream>>>(ctl, red_part, score_grid, 2, a, status);
    } else {
      a.mode = 0;
      a.scale = 0.5 * p.nu;
      const int passes = n_passes(gk::kCand);
      for (int ps = 0; ps < passes; ++ps) {
        {   // passes after the first almost always find the search finished and return at once
          Scope sc(this, ps == 0 ? "score_w_hidden" : "score_w_hidden.retry", 1, ps == 0 ? 48.0 * n4 : 0.0, 0.0);
          gk::k_score_w_hidden<<<score_grid, 256, 0, stream>>>((const float4*)H[l], (const float4*)B1,
                                                               (const float4*)Z[l], n4, ctl, red_part);
        }
        a.last_pass = (ps == passes - 1);
        Scope sc(this, "small", 1, 0.0, 0.0);
        gk::k_search_decide_w<<<1, 256, 0, stream>>>(ctl, red_part, score_grid, gk::kCand, a, status);
      }
    }
    CU(cudaGetLastError());
    {
      Scope sc(this, "small", 2, 0.0, 0.0);
      gk::k_log_decisions<<<1, 32, 0, stream>>>(ctl, 1, log_trial_w, log_q_w, d_pass, L, l - 1, kLogPasses);
      gk::k_apply_w<<<(unsigned)cdiv((long long)Kp * Cn, 256), 256, 0, stream>>>(W[l], Wt[l], grad, Kp, Cn, ldc,
                                                                               ld[l - 1], ctl);
    }
    Scope sc(this, "axpy_h", 1, 48.0 * n4, 0.0);
    gk::k_axpy_ctl<<<grid_for(n4), 256, 0, stream>>>((float4*)H[l], (const float4*)B1, n4, ctl);   // H_l at W^{k+1}
    CU(cudaGetLastError());
  }

  // ---- Z_{l,m}, l < L, every community (Appendix A, Eq. 5/6 and 8-10) ------------------
  void update_Z_hidden(int l) {
    Range range("gcn_admm: hidden Z blocks");
    const int ldl = ld[l], ldn = ld[l + 1];
    SearchCtl* ctl = ctl_z + (size_t)l * M;
    resid(l + 1, B0);                                                    // R'_{l+1}
    spmm(B0, B1, ldn);                                                   // S = A~ R'
    gemm_nn(B1, ldn, Wt[l + 1], ldl, W[l + 1], ldn, B2, ldl, n, C[l], C[l + 1]);        // S W_{l+1}^T
    CU(cudaMemsetAsync(n_active, 0, sizeof(int), stream));
    {
      Scope sc(this, "zgrad_finish", 1, 16.0 * 4.0 * (double)n * (ldl / 4), 0.0);
      gk::k_zgrad_finish<<<(unsigned)n_zblocks, 256, 0, stream>>>((float4*)B2, (const float4*)Z[l], (const float4*)H[l],
                                                                 ldl / 4, d_zblocks, p.nu, red_part);
    }
    const bool out = (l + 1 == L);
    const int per = out ? 2 : kCandZ;
    {
      Scope sc(this, "small", 1, 0.0, 0.0);
      gk::k_search_begin_z<<<(unsigned)cdiv((long long)M * 32, 128), 128, 0, stream>>>(
          ctl, M, red_part, d_comm_block_ptr, sums_z, p.bt_shrink, p.bt_growth, n_active, status);
      CU(cudaGetLastError());
    }
    gemm_nn(B2, ldl, W[l + 1], ldn, Wt[l + 1], ldl, B1, ldn, n, C[l + 1], C[l]);         // T = G W_{l+1}
    gk::DecideArgs a{};
    a.growth = p.bt_growth;
    a.max_trials = p.bt_max_trials;
    a.cand = kCandZ;
    a.own_nu = p.nu;
    const int ld4 = ldn / 4;
    const int warps = 8;
    const size_t smem = (size_t)warps * M * per * sizeof(double);
    const int use_smem = smem <= 96 * 1024;
    const size_t dyn = use_smem ? smem : 0;
    // after a sweep: the chunks' sums are added group by group, in chunk order (first stage of the ordered sum)
    int groups_used = 0;   // groups of chunks the last sweep filled (the chunk table depends on the kernel)
    auto reduce_chunks = [&](int chunks) {
      groups_used = (int)cdiv(chunks, kChunksPerGroup);
      gk::k_reduce_chunks<<<(unsigned)groups_used, 256, 0, stream>>>(z_chunk_part, chunks, kChunksPerGroup, M * per,
                                                                     z_group_part, n_active);
      ++launches;
    };
#define SCORE_Z_U(V, OUT, UNZ)                                                                                 \
  {                                                                                                       \
    const size_t dynv = dyn + (size_t)warps * 2 * (V) * 32 * sizeof(float4);   /* per-warp copy of the row's a, b */ \
    if (dynv > 48 * 1024)                                                                                 \
      CU(cudaFuncSetAttribute(gk::k_score_z<V, OUT, UNZ, kCandZ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dynv)); \
    int occ = 1;                                                                                          \
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gk::k_score_z<V, OUT, UNZ, kCandZ>, warps * 32, dynv));     \
    const unsigned grid = (unsigned)std::min<long long>(cdiv(n_chunks, warps), (long long)kSmCount * std::max(occ, 1)); \
    CU(cudaMemsetAsync(chunk_counter, 0, sizeof(int), stream));                                           \
    gk::k_score_z<V, OUT, UNZ, kCandZ><<<grid, warps * 32, dynv, stream>>>(d_row_ptr, d_col, d_col_comm, d_dinv,       \
        (const float4*)B1, (const float4*)H[l + 1], (const float4*)Z[l + 1], (const float4*)B0, ld4, (int)n, ctl, M, \
        z_chunk_part, n_active, use_smem, d_chunk_ptr, n_chunks, chunk_counter, d_items, n_items, long_len,      \
        reinterpret_cast<float4*>(item_sums), nullptr);                                                         \
    reduce_chunks(n_chunks);                                                                              \
    if (n_split > 0) {                                                                                    \
      gk::k_score_z_split<V, OUT, kCandZ><<<(unsigned)cdiv(n_split, warps), warps * 32, 0, stream>>>(d_split, n_split, d_dinv, \
          reinterpret_cast<const float4*>(item_sums), (const float4*)H[l + 1], (const float4*)Z[l + 1], (const float4*)B0, \
          ld4, ctl, split_scores, n_active);                                                              \
      ++launches;                                                                                         \
    }                                                                                                     \
  }
#define SCORE_Z_ANY(OUT)                        \
  {                                             \
    if (ld4 <= 32) SCORE_Z_U(1, OUT, 4)         \
    else if (ld4 <= 64) SCORE_Z_U(2, OUT, 4)    \
    else if (ld4 <= 128) SCORE_Z_U(4, OUT, 4)   \
    else SCORE_Z_U(8, OUT, 4)                   \
  }
    auto decide = [&](const gk::DecideArgs& args) {
      Scope sc(this, "small", 1, 0.0, 0.0);
      gk::k_search_decide_z<<<(unsigned)cdiv((long long)M * 32, 128), 128, 0, stream>>>(
          ctl, M, z_group_part, groups_used, per, split_scores, d_split_order, d_split_ptr, sums_z, args, n_active, status);
    };
    char zname[48];
    std::snprintf(zname, sizeof zname, out ? "score_z_out@%d" : "score_z_hidden@%d", ldn);
    const std::string zretry = std::string(zname) + ".retry";
    const double zbytes = 6.0 * gi.nnz + 8.0 * n +
                          4.0 * (double)n * ldn * (out ? 2 : 3);
    if (out) {
      {
        Scope sc(this, zname, 1, zbytes, 2.0 * (double)gi.nnz * ldn);
        const size_t smem_h = (size_t)2 * warps * M * 2 * sizeof(double);
        if (ld4 <= 16 && smem_h <= 96 * 1024) {   // narrow output layer: two rows per warp (see k_score_z_out_half)
          if (smem_h > 48 * 1024)
            CU(cudaFuncSetAttribute(gk::k_score_z_out_half<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_h));
          int occ = 1;
          CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gk::k_score_z_out_half<4>, warps * 32, smem_h));
          const unsigned grid = (unsigned)std::min<long long>(cdiv(n_chunks_sorted, warps), (long long)kSmCount * std::max(occ, 1));
          CU(cudaMemsetAsync(chunk_counter, 0, sizeof(int), stream));
          gk::k_score_z_out_half<4><<<grid, warps * 32, smem_h, stream>>>(d_row_ptr, d_col, d_col_comm, d_dinv,
              (const float4*)B1, (const float4*)B0, ld4, (int)n, ctl, M, z_chunk_part, n_active, d_chunk_ptr_sorted, n_chunks_sorted,
              chunk_counter, d_items, n_items, long_len, reinterpret_cast<float4*>(item_sums), d_row_order);
          reduce_chunks(n_chunks_sorted);
          if (n_split > 0) {
            gk::k_score_z_split<1, true, kCandZ><<<(unsigned)cdiv(n_split, warps), warps * 32, 0, stream>>>(d_split, n_split, d_dinv,
                reinterpret_cast<const float4*>(item_sums), (const float4*)H[l + 1], (const float4*)Z[l + 1], (const float4*)B0,
                ld4, ctl, split_scores, n_active);
            ++launches;
          }
        } else {
          SCORE_Z_ANY(true)
        }
      }
      a.mode = 1;
      a.quad_coef = 0.5 * p.rho;
      a.last_pass = 1;
      decide(a);
    } else {
      a.mode = 0;
      a.scale = 0.5 * p.nu;
      const int passes = n_passes(kCandZ);
      for (int ps = 0; ps < passes; ++ps) {
        {   // later passes touch only the segments of communities still searching
          Scope sc(this, ps == 0 ? zname : zretry.c_str(), 1, ps == 0 ? zbytes : 0.0,
                   ps == 0 ? 2.0 * (double)gi.nnz * ldn : 0.0);
          SCORE_Z_ANY(false)
        }
        a.last_pass = (ps == passes - 1);
        decide(a);
      }
    }
#undef SCORE_Z_ANY
#undef SCORE_Z_U
    CU(cudaGetLastError());
    {
      Scope sc(this, "small", 1, 0.0, 0.0);
      gk::k_log_decisions<<<(unsigned)cdiv(M, 128), 128, 0, stream>>>(ctl, M, log_trial_z, log_q_z, d_pass, z_per_pass(),
                                                                      (long long)(l - 1) * M, kLogPasses);
    }
    Scope sc(this, "apply_z", 1, 12.0 * (double)n * ldl, 0.0);
    gk::k_apply_z<<<grid_for(n * (ldl / 4)), 256, 0, stream>>>((float4*)Z[l], (const float4*)B2, ldl / 4, n, d_row_comm, ctl);
    CU(cudaGetLastError());
  }

  // ---- Z_L (Eq. 7) and, in the same sweep, the dual as printed in Eq. 3 -----------------
  void update_output(bool dual_now, bool update_z) {
    Range range("gcn_admm: output layer and dual");
    const int warps = 8;
    Scope sc(this, "output_rows", 1, 4.0 * (double)n * ld[L] * (3 + (update_z ? 1 : 0) + (dual_now ? 1 : 0)), 0.0);
    // rows without a loss term: closed form, plain sweep; training rows: one warp each (FISTA)
    gk::k_output_plain<<<grid_for(n * (ld[L] / 4)), 256, 0, stream>>>((float4*)Z[L], (float4*)U, (const float4*)H[L],
                                                                      ld[L] / 4, n, d_train, p.rho, dual_now ? 1 : 0,
                                                                      update_z ? 1 : 0);
    CU(cudaGetLastError());
    if (n_train > 0) {
#define OUTPUT_ROWS(CPL)                                                                                          \
  gk::k_output_rows<CPL><<<(unsigned)cdiv(n_train, warps), warps * 32, 0, stream>>>(                              \
      Z[L], U, H[L], ld[L], C[L], n_train, d_y, d_train, p.rho, p.loss_scale, p.fista_iters, dual_now ? 1 : 0,    \
      update_z ? 1 : 0, d_train_rows, d_fista_momentum);
      if (C[L] <= 32) OUTPUT_ROWS(1)
      else if (C[L] <= 64) OUTPUT_ROWS(2)
      else if (C[L] <= 96) OUTPUT_ROWS(3)
      else OUTPUT_ROWS(4)
#undef OUTPUT_ROWS
      CU(cudaGetLastError());
      ++launches;
    }
  }

  void dual_from_stored() {   // U + rho (Z_L - H_L) with H_L = A~ Z_{L-1} W_L of the stored iterates
    const long long n4 = n * ld[L] / 4;
    Scope sc(this, "dual", 1, 64.0 * n4, 0.0);
    gk::k_dual<<<grid_for(n4), 256, 0, stream>>>((float4*)U, (const float4*)Z[L], (const float4*)H[L], n4, p.rho);
    CU(cudaGetLastError());
  }

  // P_l = A~ Z_{l-1} (l >= 2; P_1 is constant) and H_l = P_l W_l from the stored W, Z.
  // keep_h1: the caller knows that H_1 already is P_1 W_1.  After a pass it is: P_1 never changes and
  // the W_1 step left H_1 - D/tau = P_1 (W_1 - grad/tau) behind, so the product is skipped; to keep
  // rounding from piling up over many passes it is still formed afresh every kH1RefreshEvery passes.
  static constexpr int kH1RefreshEvery = 16;
  int h1_age = 0;
  bool capturing = false;
  void refresh(bool keep_h1 = false) {
    Range range("gcn_admm: refresh P_l, H_l");
    for (int l = 2; l <= L; ++l) spmm(Z[l - 1], P[l], ld[l - 1]);
    const bool skip_h1 = keep_h1 && !capturing && h1_age + 1 < kH1RefreshEvery;
    h1_age = skip_h1 ? h1_age + 1 : 0;
    for (int l = skip_h1 ? 2 : 1; l <= L; ++l)
      gemm_nn(P[l], ld[l - 1], W[l], ld[l], Wt[l], ld[l - 1], H[l], ld[l], n, C[l], C[l - 1]);
    fresh = true;
  }

  // The serial schedule of Section 4.1: the same block updates, one after the other in the order
  // W_1, Z_1, .., W_L, Z_L, U, each reading the latest value of every other block.
  void iterate_sequential() {
    if (!fresh) refresh();
    begin_log_pass();
    for (int l = 1; l <= L; ++l) {
      if (l >= 2) {   // Z_{l-1} has just moved: P_l and H_l follow it (H_{l+1} still matches the untouched Z_l)
        spmm(Z[l - 1], P[l], ld[l - 1]);
        gemm_nn(P[l], ld[l - 1], W[l], ld[l], Wt[l], ld[l - 1], H[l], ld[l], n, C[l], C[l - 1]);
      }
      update_W(l);
      if (l < L) update_Z_hidden(l);
      else update_output(false, true);
    }
    refresh(true);
    dual_from_stored();
    end_log_pass();
  }

  void iterate() {   // Algorithm 1, one pass
    if (p.schedule == 1) { iterate_sequential(); return; }
    if (!fresh) refresh();
    begin_log_pass();
    for (int l = 1; l <= L; ++l) update_W(l);
    for (int l = 1; l < L; ++l) update_Z_hidden(l);
    update_output(p.dual_mode == 0, true);
    refresh(true);
    if (p.dual_mode != 0) dual_from_stored();
    end_log_pass();
  }

  // logits of Problem 1's forward pass with the stored W, left in B0 (N x ld_L)
  void forward_logits() {
    gemm_nn(P[1], ld[0], W[1], ld[1], Wt[1], ld[0], B0, ld[1], n, C[1], C[0]);
    for (int l = 1; l < L; ++l) {
      const long long n4 = n * ld[l] / 4;
      Scope sc(this, "relu", 1, 32.0 * n4, 0.0);
      gk::k_relu_inplace<<<grid_for(n4), 256, 0, stream>>>((float4*)B0, n4);
      CU(cudaGetLastError());
      spmm(B0, B1, ld[l]);
      gemm_nn(B1, ld[l], W[l + 1], ld[l + 1], Wt[l + 1], ld[l], B0, ld[l + 1], n, C[l + 1], C[l]);
    }
  }

  void check_status() {
    int s = 0, t = 0;
    CU(cudaMemcpyAsync(&s, status, sizeof(int), cudaMemcpyDeviceToHost, stream));
    CU(cudaMemcpyAsync(&t, tc_error, sizeof(int), cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    if (t != 0) {
      CU(cudaMemsetAsync(tc_error, 0, sizeof(int), stream));
      throw Fail{GCN_ADMM_ERR_CUDA, "a tensor-core product gave up waiting on its pipeline"};
    }
    if (s & 1) {
      CU(cudaMemsetAsync(status, 0, sizeof(int), stream));
      throw Fail{GCN_ADMM_ERR_NONFINITE, "a non-finite value reached a step-size decision"};
    }
  }

  // rows in the caller's order (dense, width c) <-> internal (community order, padded)
  void rows_to_host(const float* dev, int c, float* host_out) {
    float* dense = B2;
    Scope sc(this, "permute_rows", 1, 8.0 * (double)n * c, 0.0);
    gk::k_permute_rows<<<grid_for(n * ldpad(c)), 256, 0, stream>>>(dev, dense, d_perm, n, c, ldpad(c), 0);
    CU(cudaGetLastError());
    CU(cudaMemcpyAsync(host_out, dense, sizeof(float) * n * c, cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
  }
  void rows_from_host(const float* host_in, int c, float* dev) {
    float* dense = B2;
    CU(cudaMemcpyAsync(dense, host_in, sizeof(float) * n * c, cudaMemcpyHostToDevice, stream));
    Scope sc(this, "permute_rows", 1, 8.0 * (double)n * c, 0.0);
    gk::k_permute_rows<<<grid_for(n * ldpad(c)), 256, 0, stream>>>(dense, dev, d_perm, n, c, ldpad(c), 1);
    CU(cudaGetLastError());
    CU(cudaStreamSynchronize(stream));
  }
  void upload_weight(int l, const float* host_w) {
    const int r = C[l - 1], c = C[l];
    std::vector<float> w((size_t)r * ld[l], 0.f), wt((size_t)c * ld[l - 1], 0.f);
    for (int i = 0; i < r; ++i)
      for (int j = 0; j < c; ++j) {
        w[(size_t)i * ld[l] + j] = host_w[(size_t)i * c + j];
        wt[(size_t)j * ld[l - 1] + i] = host_w[(size_t)i * c + j];
      }
    CU(cudaMemcpyAsync(W[l], w.data(), w.size() * sizeof(float), cudaMemcpyHostToDevice, stream));
    CU(cudaMemcpyAsync(Wt[l], wt.data(), wt.size() * sizeof(float), cudaMemcpyHostToDevice, stream));
    CU(cudaStreamSynchronize(stream));
  }
};

namespace {

template <typename F>
int guarded(gcn_admm* h, F&& body) {
  if (h == nullptr) return GCN_ADMM_ERR_ARG;
  try {
    cudaError_t e = cudaSetDevice(h->p.device);
    if (e != cudaSuccess) throw Fail{GCN_ADMM_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e)};
    body();
    return GCN_ADMM_OK;
  } catch (const Fail& f) {
    h->err = f.msg;
    return f.code;
  } catch (const std::bad_alloc&) {
    h->err = "host allocation failed";
    return GCN_ADMM_ERR_ALLOC;
  } catch (...) {
    h->err = "unexpected failure";
    return GCN_ADMM_ERR_CUDA;
  }
}

// View of `count` elements on the host: the caller's buffer itself when it is host memory, a copy when
// it lives on the device.
template <typename T>
struct HostView {
  std::vector<T> copy;
  const T* ptr = nullptr;
  HostView(const T* p, size_t count) {
    if (count > 0 && is_device_pointer(p)) {
      copy.resize(count);
      CU(cudaMemcpy(copy.data(), p, count * sizeof(T), cudaMemcpyDeviceToHost));
      ptr = copy.data();
    } else {
      ptr = p;
    }
  }
  const T* data() const { return ptr; }
  const T& operator[](size_t i) const { return ptr[i]; }
};

template <typename T, typename A>
T* upload(gcn_admm* h, const std::vector<T, A>& v) {
  T* d = h->alloc<T>(v.size());
  if (!v.empty()) CU(cudaMemcpy(d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice));
  return d;
}

void create_impl(gcn_admm* h, long long n, const long long* row_ptr, const int* col_idx, const float* X, const int* y,
                 const unsigned char* train_mask, int n_layers, const int* widths, int n_comm, const int* community) {
  const gcn_admm_params& p = h->p;
  h->L = n_layers;
  h->n = n;
  h->M = n_comm;
  h->C.assign(widths, widths + n_layers + 1);
  h->ld.resize(n_layers + 1);
  for (int l = 0; l <= n_layers; ++l) {
    if (h->C[l] < 1) throw Fail{GCN_ADMM_ERR_WIDTHS, "a layer width is smaller than 1"};
    h->ld[l] = ldpad(h->C[l]);
    h->max_ld = std::max(h->max_ld, h->ld[l]);
  }
  if (h->C[n_layers] > 32 * gk::kMaxClassesPerLane)
    throw Fail{GCN_ADMM_ERR_WIDTHS, "more than 128 classes are not supported"};
  for (int l = 2; l <= n_layers; ++l)
    if (h->ld[l] / 4 > 256) throw Fail{GCN_ADMM_ERR_WIDTHS, "layer widths above 1024 are supported for C_0 and C_1 only"};
  for (int l = 1; l <= n_layers; ++l)   // the Z scoring addresses rows of an N x C_l matrix by 32-bit float4 offsets
    if (n * (long long)(h->ld[l] / 4) >= (1LL << 32))
      throw Fail{GCN_ADMM_ERR_WIDTHS, "n x layer width exceeds 2^34 elements"};

  // host copies of the graph-side inputs, then the index tables
  HostView<long long> rp(row_ptr, (size_t)n + 1);
  if (rp[n] < 0 || rp[0] != 0) throw Fail{GCN_ADMM_ERR_GRAPH, "row_ptr must start at 0 and be ascending"};
  HostView<int> ci(col_idx, (size_t)rp[n]);
  HostView<int> comm(community, (size_t)n);
  HostView<int> yy(y, (size_t)n);
  HostView<unsigned char> tm(train_mask, (size_t)n);
  std::string msg;
  const int rc = gcn_admm_host::build_graph_index(n, rp.data(), ci.data(), n_comm, comm.data(), h->gi, msg);
  if (rc == gcn_admm_host::IDX_BAD_GRAPH) throw Fail{GCN_ADMM_ERR_GRAPH, msg};
  if (rc == gcn_admm_host::IDX_BAD_COMMUNITY) throw Fail{GCN_ADMM_ERR_COMMUNITY, msg};
  { std::vector<long long>().swap(rp.copy); std::vector<int>().swap(ci.copy); }
  const GraphIndex& g = h->gi;
  std::vector<int> y_new(n);
  std::vector<unsigned char> t_new(n);
  h->n_train = 0;
  for (long long i = 0; i < n; ++i) {
    y_new[i] = yy[g.perm[i]];
    t_new[i] = tm[g.perm[i]] ? 1 : 0;
    h->n_train += t_new[i];
    if (t_new[i] && (y_new[i] < 0 || y_new[i] >= h->C[n_layers]))
      throw Fail{GCN_ADMM_ERR_WIDTHS, "a training label lies outside 0..C_L-1"};
    if (y_new[i] < 0 || y_new[i] >= h->C[n_layers]) y_new[i] = 0;
  }
  // all host-side validation is done; from here on a CUDA device is required
  int dev_count = 0;
  CU(cudaGetDeviceCount(&dev_count));
  if (p.device < 0 || p.device >= dev_count) throw Fail{GCN_ADMM_ERR_CUDA, "no such CUDA device"};
  CU(cudaSetDevice(p.device));
  h->stream = static_cast<cudaStream_t>(p.stream);
  h->d_row_ptr = upload(h, g.row_ptr);
  h->d_col = upload(h, g.col);
  h->d_row_comm = upload(h, g.row_comm);
  h->d_perm = upload(h, g.perm);
  h->d_dinv = upload(h, g.dinv);
  h->d_col_comm = upload(h, g.col_comm);
  { gcn_admm_host::Table<unsigned short>().swap(h->gi.col_comm); }   // needed on the device only
  h->d_y = upload(h, y_new);
  h->d_train = upload(h, t_new);
  {
    std::vector<int> tr;
    tr.reserve((size_t)h->n_train);
    for (long long i = 0; i < n; ++i)
      if (t_new[i]) tr.push_back((int)i);
    h->d_train_rows = upload(h, tr);
  }
  {
    std::vector<float> mom((size_t)std::max(p.fista_iters, 1), 0.f);
    double t = 1.0;
    for (int j = 0; j < p.fista_iters; ++j) {
      const double tn = 0.5 * (1.0 + std::sqrt(1.0 + 4.0 * t * t));
      mom[(size_t)j] = (float)((t - 1.0) / tn);
      t = tn;
    }
    h->d_fista_momentum = upload(h, mom);
  }
  {
    h->long_len = p.long_row > 0 ? p.long_row : kDefaultLongRow;
    gcn_admm_host::LongRowTables lt;
    gcn_admm_host::build_long_row_tables(g, h->long_len, lt);
    static_assert(sizeof(gcn_admm_host::Quad) == sizeof(int4), "tables are uploaded as int4");
    h->n_items = (int)lt.items.size();
    h->n_split = (int)lt.split.size();
    h->n_long = (int)lt.rows.size();
    h->d_items = reinterpret_cast<int4*>(upload(h, lt.items));
    h->d_split = reinterpret_cast<int4*>(upload(h, lt.split));
    {   // split entries grouped by community (stable), for the ordered sums of k_search_decide_z
      std::vector<int> sptr((size_t)n_comm + 1, 0), order(lt.split.size());
      for (const auto& q : lt.split) ++sptr[(size_t)q.y + 1];
      for (int m = 0; m < n_comm; ++m) sptr[m + 1] += sptr[m];
      std::vector<int> at(sptr.begin(), sptr.end() - 1);
      for (size_t k = 0; k < lt.split.size(); ++k) order[(size_t)at[lt.split[k].y]++] = (int)k;
      h->d_split_order = upload(h, order);
      h->d_split_ptr = upload(h, sptr);
      h->split_scores = h->alloc<double>(std::max<size_t>(1, lt.split.size() * gk::kCand));
    }
    std::vector<int> row_order((size_t)n);
    for (long long i = 0; i < n; ++i) row_order[(size_t)i] = (int)i;
#pragma omp parallel for schedule(dynamic, 1)
    for (int m = 0; m < n_comm; ++m)   // inside a community: longest rows first, ties by row id
      std::stable_sort(row_order.begin() + g.comm_ptr[m], row_order.begin() + g.comm_ptr[m + 1], [&](int a, int b) {
        return g.row_ptr[a + 1] - g.row_ptr[a] > g.row_ptr[b + 1] - g.row_ptr[b];
      });
    h->d_row_order = upload(h, row_order);
    {   // chunks of units (items first, then rows) holding about the same number of stored entries each,
        // once for rows in storage order and once for rows in the sorted order
      const long long n_units = (long long)lt.items.size() + n;
      const long long warps_guess = (long long)kSmCount * 3 * 8;
      // few enough chunks that their sums (M x candidates doubles each) stay small next to the entries they cover
      const long long target = std::max<long long>({64, std::min<long long>(1024, (long long)g.nnz / (warps_guess * 16)), 16LL * n_comm});
      auto build_chunks = [&](const int* order) {
        std::vector<int> cp;
        cp.push_back(0);
        long long in_chunk = 0;
        for (long long u = 0; u < n_units; ++u) {
          long long len;
          if (u < (long long)lt.items.size()) len = lt.items[(size_t)u].z - lt.items[(size_t)u].y;
          else {
            const long long k = u - (long long)lt.items.size();
            const long long r = order ? order[k] : k;
            len = g.row_ptr[r + 1] - g.row_ptr[r];
            if (len > h->long_len) len = 0;                 // walked as items
          }
          in_chunk += len + 2;                              // a unit costs a little even when it is short
          if (in_chunk >= target) { cp.push_back((int)(u + 1)); in_chunk = 0; }
        }
        if (cp.back() != (int)n_units) cp.push_back((int)n_units);
        return cp;
      };
      const std::vector<int> plain = build_chunks(nullptr), sorted = build_chunks(row_order.data());
      h->n_chunks = (int)plain.size() - 1;
      h->d_chunk_ptr = upload(h, plain);
      h->n_chunks_sorted = (int)sorted.size() - 1;
      h->d_chunk_ptr_sorted = upload(h, sorted);
    }
    h->d_long_rows = reinterpret_cast<int4*>(upload(h, lt.rows));
  }

  const int L = n_layers;
  const size_t rows = (size_t)n;
  h->W.assign(L + 1, nullptr); h->Wt.assign(L + 1, nullptr); h->Z.assign(L + 1, nullptr);
  h->P.assign(L + 1, nullptr); h->H.assign(L + 1, nullptr);
  size_t grad_elems = 1, grad_t_elems = 1;
  h->part_elems = 1;
  for (int l = 1; l <= L; ++l) {
    h->W[l] = h->alloc<float>((size_t)h->C[l - 1] * h->ld[l]);
    h->Wt[l] = h->alloc<float>((size_t)h->C[l] * h->ld[l - 1]);
    h->Z[l] = h->alloc<float>(rows * h->ld[l]);
    h->P[l] = h->alloc<float>(rows * h->ld[l - 1]);
    h->H[l] = h->alloc<float>(rows * h->ld[l]);
    const size_t ge = (size_t)h->C[l - 1] * h->ld[l];
    grad_elems = std::max(grad_elems, ge);
    grad_t_elems = std::max(grad_t_elems, (size_t)h->C[l] * h->ld[l - 1]);
    h->part_elems = std::max(h->part_elems, ge * 4 * kSmCount);
  }
  for (int l = 1; l <= L; ++l)   // room for one split per 2048 rows (tensor-core form of the transposed product)
    h->part_elems = std::max(h->part_elems, (size_t)h->C[l - 1] * h->ld[l] * (size_t)(cdiv(n, 2048) + kSmCount));
  h->part_elems = std::min<size_t>(h->part_elems, (size_t)256 << 20);   // at most 1 GB of partial sums
  h->part_elems = std::max(h->part_elems, grad_elems);
  h->U = h->alloc<float>(rows * h->ld[L]);
  h->B0 = h->alloc<float>(rows * h->max_ld);
  h->B1 = h->alloc<float>(rows * h->max_ld);
  h->B2 = h->alloc<float>(rows * h->max_ld);
  h->item_sums_elems = std::max<size_t>(1, (size_t)h->n_items * h->max_ld);
  h->item_sums = h->alloc<float>(h->item_sums_elems);
  h->grad = h->alloc<float>(grad_elems);
  h->grad_t = h->alloc<float>(grad_t_elems);
  h->tc_error = h->alloc<int>(1);
  h->b_image_bytes = (size_t)16 << 20;   // e.g. 1024 columns x 2048 K
  h->b_image = h->alloc<uint8_t>(h->b_image_bytes);
  CU(cudaMemset(h->tc_error, 0, sizeof(int)));
  CU(cudaMemset(h->grad_t, 0, grad_t_elems * sizeof(float)));
  h->part = h->alloc<float>(h->part_elems);
  h->ctl_w = h->alloc<SearchCtl>(L + 1);
  h->ctl_z = h->alloc<SearchCtl>((size_t)(L + 1) * n_comm);
  h->sums_w = h->alloc<double>(2);
  h->sums_z = h->alloc<double>((size_t)3 * n_comm);
  h->obj = h->alloc<double>(8);
  {   // row blocks of the hidden-layer gradient's closing sweep, cut at community boundaries
    std::vector<int2> zb;
    std::vector<int> cbp((size_t)n_comm + 1, 0);
    for (int m = 0; m < n_comm; ++m) {
      cbp[m] = (int)zb.size();
      for (int r = g.comm_ptr[m]; r < g.comm_ptr[m + 1]; r += kZBlockRows)
        zb.push_back(make_int2(r, std::min(r + kZBlockRows, g.comm_ptr[m + 1])));
    }
    cbp[n_comm] = (int)zb.size();
    h->n_zblocks = (int)zb.size();
    h->d_zblocks = upload(h, zb);
    h->d_comm_block_ptr = upload(h, cbp);
  }
  const int max_chunks = std::max(h->n_chunks, h->n_chunks_sorted);
  h->n_groups = (int)cdiv(max_chunks, kChunksPerGroup);
  h->z_chunk_part = h->alloc<double>((size_t)max_chunks * n_comm * gk::kCand);
  h->z_group_part = h->alloc<double>((size_t)h->n_groups * n_comm * gk::kCand);
  h->chunk_counter = h->alloc<int>(1);
  h->red_part = h->alloc<double>(std::max<size_t>({(size_t)kSmCount * 8 * gk::kCand, (size_t)h->n_zblocks * 3,
                                                   (size_t)cdiv(n, 8) * 2}));
  h->n_active = h->alloc<int>(1);
  h->status = h->alloc<int>(1);
  h->d_pass = h->alloc<int>(1);
  CU(cudaMemset(h->d_pass, 0, sizeof(int)));
  h->log_trial_w = h->alloc<int>((size_t)kLogPasses * L);
  h->log_q_w = h->alloc<double>((size_t)kLogPasses * L);
  h->log_trial_z = h->alloc<int>((size_t)kLogPasses * std::max(L - 1, 0) * n_comm);
  h->log_q_z = h->alloc<double>((size_t)kLogPasses * std::max(L - 1, 0) * n_comm);
  CU(cudaMemset(h->status, 0, sizeof(int)));
  CU(cudaMemset(h->n_active, 0, sizeof(int)));
  CU(cudaMemset(h->U, 0, rows * h->ld[L] * sizeof(float)));

  {
    std::vector<SearchCtl> cw(L + 1), cz((size_t)(L + 1) * n_comm);
    std::memset(cw.data(), 0, cw.size() * sizeof(SearchCtl));
    std::memset(cz.data(), 0, cz.size() * sizeof(SearchCtl));
    for (auto& c : cw) { c.t_prev = p.tau0; c.done = 1; c.trial = -3; }
    for (auto& c : cz) { c.t_prev = p.theta0; c.done = 1; c.trial = -3; }
    CU(cudaMemcpy(h->ctl_w, cw.data(), cw.size() * sizeof(SearchCtl), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(h->ctl_z, cz.data(), cz.size() * sizeof(SearchCtl), cudaMemcpyHostToDevice));
  }

  // Z_0 in community order, then P_1 = A~ Z_0 (Z_0 never changes, so neither does P_1)
  {
    float* dense = nullptr;
    const bool on_device = is_device_pointer(X);
    if (!on_device) {
      dense = dalloc<float>(rows * h->C[0]);
      cudaError_t e = cudaMemcpy(dense, X, rows * h->C[0] * sizeof(float), cudaMemcpyHostToDevice);
      if (e != cudaSuccess) { cudaFree(dense); throw Fail{GCN_ADMM_ERR_CUDA, cudaGetErrorString(e)}; }
    }
    float* x_pad = nullptr;
    try {
      x_pad = dalloc<float>(rows * h->ld[0]);
      gcn_admm::Scope sc(h, "permute_rows", 1, 8.0 * (double)n * h->C[0], 0.0);
      gk::k_permute_rows<<<h->grid_for(n * h->ld[0]), 256, 0, h->stream>>>(on_device ? X : dense, x_pad, h->d_perm, n,
                                                                           h->C[0], h->ld[0], 1);
      CU(cudaGetLastError());
      h->spmm(x_pad, h->P[1], h->ld[0]);
      CU(cudaStreamSynchronize(h->stream));
    } catch (...) {
      if (dense) cudaFree(dense);
      if (x_pad) cudaFree(x_pad);
      throw;
    }
    if (dense) cudaFree(dense);
    cudaFree(x_pad);
  }

  for (int l = 1; l <= L; ++l) {
    if (p.w_init != nullptr) { h->upload_weight(l, p.w_init[l - 1]); continue; }
    // no weights given: Glorot-uniform from a counter-based generator (see the header for the definition)
    const int r = h->C[l - 1], c = h->C[l];
    std::vector<float> w((size_t)r * c);
    const double a = std::sqrt(6.0 / ((double)r + (double)c));
    for (size_t e = 0; e < w.size(); ++e) {
      const double u = (double)(splitmix64(p.seed + ((unsigned long long)l << 32) + e) >> 40) / 16777216.0;
      w[e] = (float)(a * (2.0 * u - 1.0));
    }
    h->upload_weight(l, w.data());
  }
  // forward pass of Problem 1 with the same kernels that later recompute H_l, so that the
  // initial residuals are exactly zero
  for (int l = 1; l <= L; ++l) {
    if (l >= 2) h->spmm(h->Z[l - 1], h->P[l], h->ld[l - 1]);
    h->gemm_nn(h->P[l], h->ld[l - 1], h->W[l], h->ld[l], h->Wt[l], h->ld[l - 1], h->H[l], h->ld[l], n, h->C[l], h->C[l - 1]);
    const size_t bytes = rows * h->ld[l] * sizeof(float);
    CU(cudaMemcpyAsync(h->Z[l], h->H[l], bytes, cudaMemcpyDeviceToDevice, h->stream));
    if (l < L) {
      const long long n4 = n * h->ld[l] / 4;
      gcn_admm::Scope sc(h, "relu", 1, 32.0 * n4, 0.0);
      gk::k_relu_inplace<<<h->grid_for(n4), 256, 0, h->stream>>>((float4*)h->Z[l], n4);
      CU(cudaGetLastError());
    }
  }
  h->fresh = true;
  CU(cudaStreamSynchronize(h->stream));
}

}  // namespace

extern "C" {

void gcn_admm_default_params(gcn_admm_params* p) {
  if (!p) return;
  std::memset(p, 0, sizeof(*p));
  p->nu = 1e-3f; p->rho = 1e-3f;
  p->tau0 = 1.f; p->theta0 = 1.f;
  p->bt_growth = 2.f; p->bt_shrink = 0.5f;
  p->bt_max_trials = 40;
  p->fista_iters = 30;
  p->loss_scale = 1.f;
  p->dual_mode = 0;
  p->tensor_cores = 1;
  p->use_graph = 2;
  p->schedule = 0;
  p->long_row = 0;
  p->seed = 0;
  p->w_init = nullptr;
  p->device = 0;
  p->stream = nullptr;
}

int gcn_admm_create(gcn_admm** out, long long n, const long long* row_ptr, const int* col_idx, const float* X,
                    const int* y, const unsigned char* train_mask, int n_layers, const int* widths,
                    const gcn_admm_params* p, int n_comm, const int* community) {
  if (out) *out = nullptr;
  if (!out || !row_ptr || !X || !y || !train_mask || !widths || !p || !community || !col_idx) {
    g_create_error = "NULL argument";
    return GCN_ADMM_ERR_ARG;
  }
  if (n < 1 || n > 2147483647LL / 2 || n_comm < 1) { g_create_error = "n and n_comm must be positive"; return GCN_ADMM_ERR_ARG; }
  if (n_comm > 65535) { g_create_error = "more than 65535 communities are not supported"; return GCN_ADMM_ERR_COMMUNITY; }
  if (n_layers < 1 || n_layers > 64) { g_create_error = "n_layers must be 1..64"; return GCN_ADMM_ERR_WIDTHS; }
  for (int l = 0; p->w_init && l < n_layers; ++l)
    if (!p->w_init[l]) { g_create_error = "w_init holds a NULL pointer"; return GCN_ADMM_ERR_ARG; }
  if (!(p->nu > 0.f) || !(p->rho > 0.f) || !(p->bt_growth > 1.f) || !(p->bt_shrink > 0.f) || p->bt_max_trials < 1 ||
      p->bt_max_trials > 64 || p->fista_iters < 0 || p->schedule < 0 || p->schedule > 1 || p->long_row < 0 || !(p->tau0 > 0.f) || !(p->theta0 > 0.f) || !(p->loss_scale > 0.f)) {
    g_create_error = "a parameter is out of range";
    return GCN_ADMM_ERR_ARG;
  }
  gcn_admm* h = new (std::nothrow) gcn_admm();
  if (!h) { g_create_error = "host allocation failed"; return GCN_ADMM_ERR_ALLOC; }
  h->p = *p;
  int code = GCN_ADMM_OK;
  try {
    create_impl(h, n, row_ptr, col_idx, X, y, train_mask, n_layers, widths, n_comm, community);
  } catch (const Fail& f) {
    code = f.code; g_create_error = f.msg;
  } catch (const std::bad_alloc&) {
    code = GCN_ADMM_ERR_ALLOC; g_create_error = "host allocation failed";
  } catch (...) {
    code = GCN_ADMM_ERR_CUDA; g_create_error = "unexpected failure";
  }
  if (code != GCN_ADMM_OK) {
    gcn_admm_destroy(h);
    return code;
  }
  h->p.w_init = nullptr;   // the caller's pointers are not kept
  *out = h;
  return GCN_ADMM_OK;
}

void gcn_admm_destroy(gcn_admm* h) {
  if (!h) return;
  if (cudaSetDevice(h->p.device) == cudaSuccess) {
    cudaStreamSynchronize(h->stream);
    h->collect_profile();
    if (h->pass_graph) cudaGraphExecDestroy(h->pass_graph);
    for (cudaEvent_t e : h->event_pool) cudaEventDestroy(e);
    for (void* q : h->owned) cudaFree(q);
  }
  cudaGetLastError();
  delete h;
}

const char* gcn_admm_last_error(const gcn_admm* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

int gcn_admm_step(gcn_admm* h, int n_iters) {
  return guarded(h, [&] {
    if (n_iters < 0) throw Fail{GCN_ADMM_ERR_ARG, "n_iters must be >= 0"};
    h->log_count = 0;
    CU(cudaMemsetAsync(h->d_pass, 0, sizeof(int), h->stream));
    // A pass is a fixed sequence of launches (every decision is taken on the device), so on a stream
    // that can be captured it is recorded once and replayed: the small workloads are launch-bound.
    // use_graph 1: always; 2: only where a pass is short enough for launch overhead to matter
    const bool wanted = h->p.use_graph == 1 || (h->p.use_graph == 2 && h->n * (long long)h->max_ld < (1LL << 27));
    const bool replay = wanted && h->stream != nullptr && !h->profiling && n_iters >= 2;
    if (!replay) {
      for (int k = 0; k < n_iters; ++k) h->iterate();
      return;
    }
    if (!h->fresh) h->refresh();
    if (h->pass_graph == nullptr) {
      cudaGraph_t graph = nullptr;
      CU(cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
      const long long launches_before = h->launches, log_before = h->log_count;
      h->capturing = true;          // the recorded pass is replayed many times: it forms every product
      try {
        h->iterate();
        h->capturing = false;
      } catch (...) {
        h->capturing = false;
        cudaStreamEndCapture(h->stream, &graph);
        if (graph) cudaGraphDestroy(graph);
        throw;
      }
      CU(cudaStreamEndCapture(h->stream, &graph));
      h->launches_per_pass = h->launches - launches_before;
      h->launches = launches_before;       // recording launched nothing
      h->log_count = log_before;
      cudaError_t e = cudaGraphInstantiate(&h->pass_graph, graph, 0);
      cudaGraphDestroy(graph);
      if (e != cudaSuccess) throw Fail{GCN_ADMM_ERR_CUDA, std::string("cudaGraphInstantiate: ") + cudaGetErrorString(e)};
    }
    for (int k = 0; k < n_iters; ++k) {
      CU(cudaGraphLaunch(h->pass_graph, h->stream));
      h->launches += h->launches_per_pass;
      ++h->log_count;
    }
  });
}

int gcn_admm_step_block(gcn_admm* h, int phase, int layer) {
  return guarded(h, [&] {
    const int L = h->L;
    if (phase == GCN_ADMM_PHASE_W || phase == GCN_ADMM_PHASE_Z)
      if (layer < 1 || layer > L) throw Fail{GCN_ADMM_ERR_ARG, "layer out of range"};
    if (!h->fresh) h->refresh();
    h->log_count = 0;
    CU(cudaMemsetAsync(h->d_pass, 0, sizeof(int), h->stream));
    h->begin_log_pass();
    if (phase == GCN_ADMM_PHASE_W) {
      h->update_W(layer);
    } else if (phase == GCN_ADMM_PHASE_Z) {
      if (layer < L) h->update_Z_hidden(layer);
      else h->update_output(false, true);
      h->fresh = false;
    } else if (phase == GCN_ADMM_PHASE_U) {
      h->dual_from_stored();
    } else {
      throw Fail{GCN_ADMM_ERR_ARG, "unknown phase"};
    }
    h->end_log_pass();
  });
}

int gcn_admm_objective(gcn_admm* h, double out[6]) {
  return guarded(h, [&] {
    if (!out) throw Fail{GCN_ADMM_ERR_ARG, "NULL output"};
    if (!h->fresh) h->refresh();
    const int L = h->L;
    cudaStream_t s = h->stream;
    CU(cudaMemsetAsync(h->obj, 0, 8 * sizeof(double), s));
    // every sum: per-block partials, then one block adds them in a fixed order
    for (int l = 1; l < L; ++l) {
      const long long n4 = h->n * h->ld[l] / 4;
      gcn_admm::Scope sc(h, "objective_sums", 2, 32.0 * n4, 0.0);
      const int grid = h->grid_for(n4);
      gk::k_sum_hidden_penalty<<<grid, 256, 0, s>>>((const float4*)h->Z[l], (const float4*)h->H[l], n4, h->red_part);
      gk::k_add_partials<<<1, 256, 0, s>>>(h->red_part, grid, 1, h->obj + 2);
    }
    const long long n4 = h->n * h->ld[L] / 4;
    const int warps = 8;
    const int row_blocks = (int)cdiv(h->n, warps);
    {
      gcn_admm::Scope sc_obj(h, "objective_sums", 4, 48.0 * n4, 0.0);
      const int grid = h->grid_for(n4);
      gk::k_sum_constraint<<<grid, 256, 0, s>>>((const float4*)h->Z[L], (const float4*)h->H[L], (const float4*)h->U, n4,
                                                h->red_part);
      gk::k_add_partials<<<1, 256, 0, s>>>(h->red_part, grid, 2, h->obj + 3);
      gk::k_row_loss_argmax<<<row_blocks, warps * 32, 0, s>>>(h->Z[L], nullptr, h->ld[L], h->C[L], (int)h->n, h->d_y,
                                                              h->d_train, nullptr, h->red_part);
      gk::k_add_partials<<<1, 256, 0, s>>>(h->red_part, row_blocks, 2, h->obj);      // obj[0] = cross-entropy sum
      CU(cudaGetLastError());
    }
    h->forward_logits();
    {
      gcn_admm::Scope sc_obj(h, "objective_sums", 2, 4.0 * (double)h->n * h->ld[L], 0.0);
      gk::k_row_loss_argmax<<<row_blocks, warps * 32, 0, s>>>(nullptr, h->B0, h->ld[L], h->C[L], (int)h->n, h->d_y,
                                                              h->d_train, nullptr, h->red_part);
      gk::k_add_partials<<<1, 256, 0, s>>>(h->red_part, row_blocks, 2, h->obj + 5);  // obj[6] = correct training rows
      CU(cudaGetLastError());
    }
    double v[8];
    CU(cudaMemcpyAsync(v, h->obj, 8 * sizeof(double), cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    const double R = h->p.loss_scale * v[0];
    const double pen = 0.5 * h->p.nu * v[2];
    const double ur = v[3];
    const double rr = 0.5 * h->p.rho * v[4];
    out[0] = R + pen + ur + rr;
    out[1] = R; out[2] = pen; out[3] = ur; out[4] = rr;
    out[5] = h->n_train > 0 ? v[6] / h->n_train : 0.0;
    h->check_status();
  });
}

int gcn_admm_weights(gcn_admm* h, int layer, float* out) {
  return gcn_admm_get_state(h, GCN_ADMM_ST_W, layer, out);
}

int gcn_admm_predict(gcn_admm* h, float* logits, int* labels) {
  return guarded(h, [&] {
    const int L = h->L;
    h->forward_logits();
    if (labels) {
      const int warps = 8;
      int* d_lab = reinterpret_cast<int*>(h->B1);
      gcn_admm::Scope sc(h, "row_argmax", 1, 4.0 * (double)h->n * h->ld[L], 0.0);
      gk::k_row_loss_argmax<<<(unsigned)cdiv(h->n, warps), warps * 32, 0, h->stream>>>(
          nullptr, h->B0, h->ld[L], h->C[L], (int)h->n, h->d_y, h->d_train, d_lab, h->red_part);
      CU(cudaGetLastError());
      std::vector<int> lab(h->n);
      CU(cudaMemcpyAsync(lab.data(), d_lab, sizeof(int) * h->n, cudaMemcpyDeviceToHost, h->stream));
      CU(cudaStreamSynchronize(h->stream));
      for (long long i = 0; i < h->n; ++i) labels[h->gi.perm[i]] = lab[i];
    }
    if (logits) h->rows_to_host(h->B0, h->C[L], logits);
    CU(cudaStreamSynchronize(h->stream));
  });
}

int gcn_admm_propagate(gcn_admm* h, const float* x, int width, float* out) {
  return guarded(h, [&] {
    if (!x || !out || width < 1 || width > kMaxWidth) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    const int ldw = ldpad(width);
    const size_t rows = (size_t)h->n;
    const bool dev_in = is_device_pointer(x), dev_out = is_device_pointer(out);
    if (dev_in != dev_out) throw Fail{GCN_ADMM_ERR_ARG, "x and out must both be host or both be device pointers"};
    float *dense = nullptr, *a = nullptr, *b = nullptr;
    try {
      dense = dalloc<float>(rows * width);
      a = dalloc<float>(rows * ldw);
      b = dalloc<float>(rows * ldw);
      CU(cudaMemcpyAsync(dense, x, rows * width * sizeof(float), dev_in ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice,
                         h->stream));
      gcn_admm::Scope sc(h, "permute_rows", 2, 16.0 * (double)h->n * width, 0.0);
      gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(dense, a, h->d_perm, h->n, width, ldw, 1);
      CU(cudaGetLastError());
      h->spmm(a, b, ldw);
      gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(b, dense, h->d_perm, h->n, width, ldw, 0);
      CU(cudaGetLastError());
      CU(cudaMemcpyAsync(out, dense, rows * width * sizeof(float), dev_out ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost,
                         h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } catch (...) {
      cudaFree(dense); cudaFree(a); cudaFree(b);
      throw;
    }
    cudaFree(dense); cudaFree(a); cudaFree(b);
  });
}

int gcn_admm_dense_product(gcn_admm* h, const float* A, const float* B, float* C, long long m, int n, int k,
                           int tensor_cores) {
  return guarded(h, [&] {
    if (!A || !B || !C || m < 1 || n < 1 || k < 1 || m > 2147483647LL) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    if (!is_device_pointer(A) || !is_device_pointer(B) || !is_device_pointer(C))
      throw Fail{GCN_ADMM_ERR_ARG, "A, B and C must be device pointers"};
    const int lda = ldpad(k), ldb = ldpad(n), ldc = ldpad(n), ldbk = ldpad(k);
    float *a = nullptr, *b = nullptr, *bk = nullptr, *c = nullptr;
    const int saved = h->p.tensor_cores;
    try {
      a = dalloc<float>((size_t)m * lda);
      b = dalloc<float>((size_t)k * ldb);
      bk = dalloc<float>((size_t)n * ldbk);
      c = dalloc<float>((size_t)m * ldc);
      CU(cudaMemsetAsync(a, 0, (size_t)m * lda * 4, h->stream));
      CU(cudaMemsetAsync(b, 0, (size_t)k * ldb * 4, h->stream));
      CU(cudaMemsetAsync(bk, 0, (size_t)n * ldbk * 4, h->stream));
      CU(cudaMemcpy2DAsync(a, (size_t)lda * 4, A, (size_t)k * 4, (size_t)k * 4, (size_t)m, cudaMemcpyDeviceToDevice, h->stream));
      CU(cudaMemcpy2DAsync(b, (size_t)ldb * 4, B, (size_t)n * 4, (size_t)n * 4, (size_t)k, cudaMemcpyDeviceToDevice, h->stream));
      gk::k_transpose_small<<<(unsigned)cdiv((long long)k * n, 256), 256, 0, h->stream>>>(b, ldb, bk, ldbk, k, n);
      CU(cudaGetLastError());
      h->p.tensor_cores = tensor_cores;
      h->gemm_nn(a, lda, b, ldb, tensor_cores ? bk : nullptr, ldbk, c, ldc, m, n, k);
      h->p.tensor_cores = saved;
      CU(cudaMemcpy2DAsync(C, (size_t)n * 4, c, (size_t)ldc * 4, (size_t)n * 4, (size_t)m, cudaMemcpyDeviceToDevice, h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } catch (...) {
      h->p.tensor_cores = saved;
      cudaFree(a); cudaFree(b); cudaFree(bk); cudaFree(c);
      throw;
    }
    cudaFree(a); cudaFree(b); cudaFree(bk); cudaFree(c);
    h->check_status();
  });
}

int gcn_admm_dense_product_tn(gcn_admm* h, const float* A, const float* B, float* C, long long rows, int ka, int nb,
                              int tensor_cores) {
  return guarded(h, [&] {
    if (!A || !B || !C || rows < 1 || ka < 1 || nb < 1) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    if (!is_device_pointer(A) || !is_device_pointer(B) || !is_device_pointer(C))
      throw Fail{GCN_ADMM_ERR_ARG, "A, B and C must be device pointers"};
    const int lda = ldpad(ka), ldb = ldpad(nb), ldp = ldpad(nb);
    if ((size_t)ka * ldp > h->part_elems) throw Fail{GCN_ADMM_ERR_ARG, "ka x nb exceeds the handle's partial-sum scratch"};
    float *a = nullptr, *b = nullptr, *c = nullptr;
    const int saved = h->p.tensor_cores;
    try {
      a = dalloc<float>((size_t)rows * lda);
      b = dalloc<float>((size_t)rows * ldb);
      c = dalloc<float>((size_t)ka * ldp);
      CU(cudaMemsetAsync(a, 0, (size_t)rows * lda * 4, h->stream));
      CU(cudaMemsetAsync(b, 0, (size_t)rows * ldb * 4, h->stream));
      CU(cudaMemcpy2DAsync(a, (size_t)lda * 4, A, (size_t)ka * 4, (size_t)ka * 4, (size_t)rows, cudaMemcpyDeviceToDevice, h->stream));
      CU(cudaMemcpy2DAsync(b, (size_t)ldb * 4, B, (size_t)nb * 4, (size_t)nb * 4, (size_t)rows, cudaMemcpyDeviceToDevice, h->stream));
      h->p.tensor_cores = tensor_cores;
      h->gemm_tn(a, lda, b, ldb, c, ldp, rows, ka, nb);
      h->p.tensor_cores = saved;
      CU(cudaMemcpy2DAsync(C, (size_t)nb * 4, c, (size_t)ldp * 4, (size_t)nb * 4, (size_t)ka, cudaMemcpyDeviceToDevice, h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } catch (...) {
      h->p.tensor_cores = saved;
      cudaFree(a); cudaFree(b); cudaFree(c);
      throw;
    }
    cudaFree(a); cudaFree(b); cudaFree(c);
    h->check_status();
  });
}

// ---- propagation for callers that may not allocate ---------------------------------------------
// The two padded staging matrices of gcn_admm_propagate live in one file-scope device array, so
// this entry point reserves nothing at call time.  Every GPU that loads the library carries the
// array (32 MiB) until the process exits.
namespace {
constexpr long long kStaticHalf = 4LL << 20;                       // floats per staging matrix
static __device__ __align__(256) float g_propagate_scratch[2 * kStaticHalf];
std::mutex g_scratch_mutex;
float* g_scratch_addr[64] = {nullptr};

// Device address of g_propagate_scratch on `device` (which must be current).  In host code the
// array's name is only a handle for the runtime, never an address a kernel may be given.
float* static_scratch(int device) {
  if (device < 0 || device >= 64) throw Fail{GCN_ADMM_ERR_ARG, "device ordinal above 63"};
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[device] == nullptr) {
    float* ptr = nullptr;
    CU(cudaGetSymbolAddress((void**)&ptr, g_propagate_scratch));
    g_scratch_addr[device] = ptr;
  }
  return g_scratch_addr[device];
}
}  // namespace

int gcn_admm_propagate_static(gcn_admm* h, const float* x, int width, float* out) {
  return guarded(h, [&] {
    if (!x || !out || width < 1 || width > kMaxWidth) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    const int ldw = ldpad(width);
    if ((long long)h->n * ldw > kStaticHalf)
      throw Fail{GCN_ADMM_ERR_ARG, "n * padded width exceeds the static scratch of 4194304 floats per staging matrix"};
    if (!is_device_pointer(x) || !is_device_pointer(out))
      throw Fail{GCN_ADMM_ERR_ARG, "x and out must be device pointers"};
    float* a = static_scratch(h->p.device);
    float* b = a + kStaticHalf;
    struct Untimed {   // event creation reserves memory: launches here are counted, never timed
      gcn_admm* h; bool saved;
      explicit Untimed(gcn_admm* h_) : h(h_), saved(h_->profiling) { h->profiling = false; }
      ~Untimed() { h->profiling = saved; }
    } untimed(h);
    {
      gcn_admm::Scope sc(h, "permute_rows", 1, 8.0 * (double)h->n * width, 0.0);
      gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(x, a, h->d_perm, h->n, width, ldw, 1);
      CU(cudaGetLastError());
    }
    h->spmm(a, b, ldw);
    gcn_admm::Scope sc(h, "permute_rows", 1, 8.0 * (double)h->n * width, 0.0);
    gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(b, out, h->d_perm, h->n, width, ldw, 0);
    CU(cudaGetLastError());
  });
}

int gcn_admm_index(gcn_admm* h, int which, int comm, const int** data, long long* len) {
  return guarded(h, [&] {
    if (!data || !len || which < 0 || which > GCN_ADMM_IX_SEG_BEGIN) throw Fail{GCN_ADMM_ERR_ARG, "bad selector"};
    const GraphIndex& g = h->gi;
    auto give = [&](const auto& v) { *data = v.data(); *len = (long long)v.size(); };
    switch (which) {
      case GCN_ADMM_IX_PERM: give(g.perm); break;
      case GCN_ADMM_IX_INV_PERM: give(g.inv); break;
      case GCN_ADMM_IX_COMM_PTR: give(g.comm_ptr); break;
      case GCN_ADMM_IX_CSR_ROW_PTR: give(g.row_ptr); break;
      case GCN_ADMM_IX_CSR_COL: give(g.col); break;
      case GCN_ADMM_IX_SEG_ROW_PTR: give(g.seg_row_ptr); break;
      case GCN_ADMM_IX_SEG_COMM: give(g.seg_comm); break;
      case GCN_ADMM_IX_SEG_BEGIN: give(g.seg_begin); break;
      default: {
        if (comm < 0 || comm >= h->M) throw Fail{GCN_ADMM_ERR_ARG, "community out of range"};
        std::vector<int>& c = h->ix_cache[which];
        if (which == GCN_ADMM_IX_NBR) c = gcn_admm_host::nbr_of(g, comm);
        else if (which == GCN_ADMM_IX_HALO1) c = gcn_admm_host::halo1_of(g, comm);
        else c = gcn_admm_host::halo2_of(g, comm);
        give(c);
      }
    }
  });
}

namespace {
void ensure_shard_plan(gcn_admm* h, int n_ranks) {
  if (h->shard_plan.n_ranks == n_ranks) return;
  if (!gcn_admm_host::build_shard_plan(h->gi, n_ranks, h->shard_plan))
    throw Fail{GCN_ADMM_ERR_ARG, "n_ranks must be between 1 and the number of communities"};
  h->shard_ranges = h->shard_plan.comm_begin;
  h->shard_ranges.insert(h->shard_ranges.end(), h->shard_plan.row_begin.begin(), h->shard_plan.row_begin.end());
}
}  // namespace

int gcn_admm_shard_plan(gcn_admm* h, int n_ranks, int which, int receiver, int sender, const int** data, long long* len) {
  return guarded(h, [&] {
    if (!data || !len || which < GCN_ADMM_SHARD_RANGES || which > GCN_ADMM_SHARD_SECOND_ORDER)
      throw Fail{GCN_ADMM_ERR_ARG, "bad selector"};
    ensure_shard_plan(h, n_ranks);
    const std::vector<int>* v = &h->shard_ranges;
    if (which != GCN_ADMM_SHARD_RANGES) {
      if (receiver < 0 || receiver >= n_ranks || sender < 0 || sender >= n_ranks)
        throw Fail{GCN_ADMM_ERR_ARG, "rank out of range"};
      const auto& lists = which == GCN_ADMM_SHARD_FIRST_ORDER ? h->shard_plan.first_order : h->shard_plan.second_order;
      v = &lists[(size_t)receiver * n_ranks + sender];
    }
    *data = v->data();
    *len = (long long)v->size();
  });
}

// The propagation as the ranks of a sharded run would carry it out, rank after rank on this one device.
int gcn_admm_propagate_sharded(gcn_admm* h, int n_ranks, const float* x, int width, float* out, long long* staged_rows) {
  return guarded(h, [&] {
    if (!x || !out || width < 1 || width > kMaxWidth) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    ensure_shard_plan(h, n_ranks);
    const gcn_admm_host::ShardPlan& plan = h->shard_plan;
    const gcn_admm_host::GraphIndex& g = h->gi;
    const int ldw = ldpad(width), R = n_ranks;
    const size_t rows = (size_t)h->n;
    const bool dev_in = is_device_pointer(x), dev_out = is_device_pointer(out);
    if (dev_in != dev_out) throw Fail{GCN_ADMM_ERR_ARG, "x and out must both be host or both be device pointers"};
    std::vector<void*> mine;   // freed on every way out
    auto take = [&](size_t bytes) { void* q = dalloc<char>(std::max<size_t>(bytes, 16)); mine.push_back(q); return q; };
    auto release = [&] { for (void* q : mine) cudaFree(q); mine.clear(); };
    long long staged = 0;
    try {
      float* dense = static_cast<float*>(take(rows * width * sizeof(float)));
      float* a = static_cast<float*>(take(rows * ldw * sizeof(float)));
      float* b = static_cast<float*>(take(rows * ldw * sizeof(float)));
      CU(cudaMemcpyAsync(dense, x, rows * width * sizeof(float), dev_in ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice,
                         h->stream));
      gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(dense, a, h->d_perm, h->n, width, ldw, 1);
      CU(cudaGetLastError());
      for (int r = 0; r < R; ++r) {
        const int lo = plan.row_begin[r], hi = plan.row_begin[r + 1], n_own = hi - lo;
        // rows this rank holds: its own, then the first-order rows of every sender (ascending in new ids,
        // because senders own ascending row ranges)
        std::vector<int> held((size_t)n_own);
        for (int i = 0; i < n_own; ++i) held[(size_t)i] = lo + i;
        for (int sdr = 0; sdr < R; ++sdr) {
          const std::vector<int>& f = plan.first_order[(size_t)r * R + sdr];
          held.insert(held.end(), f.begin(), f.end());
        }
        const int n_held = (int)held.size();
        staged += n_held - n_own;
        // local tables: the rank's rows of A + I with columns renumbered to positions in `held`
        // (entry order kept, so every row is summed in the order of the unsharded kernel)
        std::vector<int> rp((size_t)n_own + 1), order((size_t)n_own);
        const long long e0 = g.row_ptr[lo], e1 = g.row_ptr[hi];
        std::vector<int> cl((size_t)(e1 - e0));
        std::vector<float> dv((size_t)n_held);
        for (int k = 0; k < n_held; ++k) dv[(size_t)k] = g.dinv[(size_t)held[(size_t)k]];
        for (int i = 0; i <= n_own; ++i) rp[(size_t)i] = (int)(g.row_ptr[lo + i] - e0);
        for (long long e = e0; e < e1; ++e) {
          const int j = g.col[(size_t)e];
          int local;
          if (j >= lo && j < hi) local = j - lo;
          else {
            const auto it = std::lower_bound(held.begin() + n_own, held.end(), j);
            if (it == held.end() || *it != j) throw Fail{GCN_ADMM_ERR_CUDA, "plan misses a neighbour row"};
            local = (int)(it - held.begin());
          }
          cl[(size_t)(e - e0)] = local;
        }
        for (int i = 0; i < n_own; ++i) order[(size_t)i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int p_, int q_) { return rp[p_ + 1] - rp[p_] > rp[q_ + 1] - rp[q_]; });
        int* d_rp = static_cast<int*>(take(rp.size() * sizeof(int)));
        int* d_cl = static_cast<int*>(take(cl.size() * sizeof(int)));
        int* d_order = static_cast<int*>(take(order.size() * sizeof(int)));
        int* d_held = static_cast<int*>(take(held.size() * sizeof(int)));
        float* d_dv = static_cast<float*>(take(dv.size() * sizeof(float)));
        float* xl = static_cast<float*>(take((size_t)n_held * ldw * sizeof(float)));
        CU(cudaMemcpyAsync(d_rp, rp.data(), rp.size() * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        if (!cl.empty()) CU(cudaMemcpyAsync(d_cl, cl.data(), cl.size() * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        if (n_own > 0) CU(cudaMemcpyAsync(d_order, order.data(), order.size() * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        if (n_held > 0) {
          CU(cudaMemcpyAsync(d_held, held.data(), held.size() * sizeof(int), cudaMemcpyHostToDevice, h->stream));
          CU(cudaMemcpyAsync(d_dv, dv.data(), dv.size() * sizeof(float), cudaMemcpyHostToDevice, h->stream));
          // own rows and, behind them, the copies of the first-order rows: on several devices the second part
          // is what the receives from the rows' owners fill
          gk::k_gather_rows<<<h->grid_for((long long)n_held * (ldw / 4)), 256, 0, h->stream>>>(
              reinterpret_cast<const float4*>(a), d_held, reinterpret_cast<float4*>(xl), ldw / 4, n_held);
          CU(cudaGetLastError());
          ++h->launches;
        }
        if (n_own > 0) {
          gcn_admm::Scope sc(h, "spmm.sharded", 1, 0.0, 0.0);
          h->spmm_launch(d_rp, d_cl, d_dv, d_order, n_own, nullptr, 0, INT_MAX, xl, b + (size_t)lo * ldw, ldw);
        }
        CU(cudaStreamSynchronize(h->stream));   // the host vectors of this rank go out of scope
      }
      gk::k_permute_rows<<<h->grid_for(h->n * ldw), 256, 0, h->stream>>>(b, dense, h->d_perm, h->n, width, ldw, 0);
      CU(cudaGetLastError());
      h->launches += 2;   // the two row permutations
      CU(cudaMemcpyAsync(out, dense, rows * width * sizeof(float), dev_out ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost,
                         h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } catch (...) {
      release();
      throw;
    }
    release();
    if (staged_rows) *staged_rows = staged;
  });
}

int gcn_admm_get_state(gcn_admm* h, int which, int layer, void* out) {
  return guarded(h, [&] {
    if (!out) throw Fail{GCN_ADMM_ERR_ARG, "NULL output"};
    const int L = h->L;
    auto need_layer = [&](int lo, int hi) {
      if (layer < lo || layer > hi) throw Fail{GCN_ADMM_ERR_ARG, "layer out of range"};
    };
    if (which == GCN_ADMM_ST_W) {
      need_layer(1, L);
      const int r = h->C[layer - 1], c = h->C[layer], ldw = h->ld[layer];
      std::vector<float> w((size_t)r * ldw);
      CU(cudaMemcpyAsync(w.data(), h->W[layer], w.size() * sizeof(float), cudaMemcpyDeviceToHost, h->stream));
      CU(cudaStreamSynchronize(h->stream));
      float* o = static_cast<float*>(out);
      for (int i = 0; i < r; ++i) std::memcpy(o + (size_t)i * c, w.data() + (size_t)i * ldw, c * sizeof(float));
    } else if (which == GCN_ADMM_ST_Z) {
      need_layer(1, L);
      h->rows_to_host(h->Z[layer], h->C[layer], static_cast<float*>(out));
    } else if (which == GCN_ADMM_ST_U) {
      h->rows_to_host(h->U, h->C[L], static_cast<float*>(out));
    } else if (which == GCN_ADMM_ST_TAU) {
      need_layer(1, L);
      SearchCtl c;
      CU(cudaMemcpyAsync(&c, h->ctl_w + layer, sizeof(c), cudaMemcpyDeviceToHost, h->stream));
      CU(cudaStreamSynchronize(h->stream));
      *static_cast<double*>(out) = c.t_prev;
    } else if (which == GCN_ADMM_ST_THETA) {
      need_layer(1, L - 1);
      std::vector<SearchCtl> c(h->M);
      CU(cudaMemcpyAsync(c.data(), h->ctl_z + (size_t)layer * h->M, c.size() * sizeof(SearchCtl), cudaMemcpyDeviceToHost,
                         h->stream));
      CU(cudaStreamSynchronize(h->stream));
      for (int m = 0; m < h->M; ++m) static_cast<double*>(out)[m] = c[m].t_prev;
    } else if (which == GCN_ADMM_ST_PIPELINE_FLAG) {
      CU(cudaMemcpyAsync(out, h->tc_error, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } else {
      throw Fail{GCN_ADMM_ERR_ARG, "unknown state selector"};
    }
  });
}

int gcn_admm_set_state(gcn_admm* h, int which, int layer, const void* in) {
  return guarded(h, [&] {
    if (!in) throw Fail{GCN_ADMM_ERR_ARG, "NULL input"};
    const int L = h->L;
    auto need_layer = [&](int lo, int hi) {
      if (layer < lo || layer > hi) throw Fail{GCN_ADMM_ERR_ARG, "layer out of range"};
    };
    if (which == GCN_ADMM_ST_W) {
      need_layer(1, L);
      h->upload_weight(layer, static_cast<const float*>(in));
      h->fresh = false;
    } else if (which == GCN_ADMM_ST_Z) {
      need_layer(1, L);
      h->rows_from_host(static_cast<const float*>(in), h->C[layer], h->Z[layer]);
      h->fresh = false;
    } else if (which == GCN_ADMM_ST_U) {
      h->rows_from_host(static_cast<const float*>(in), h->C[L], h->U);
    } else if (which == GCN_ADMM_ST_TAU) {
      need_layer(1, L);
      const double t = *static_cast<const double*>(in);
      if (!(t > 0.0)) throw Fail{GCN_ADMM_ERR_ARG, "tau must be positive"};
      CU(cudaMemcpyAsync(&h->ctl_w[layer].t_prev, &t, sizeof(double), cudaMemcpyHostToDevice, h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } else if (which == GCN_ADMM_ST_THETA) {
      need_layer(1, L - 1);
      const double* t = static_cast<const double*>(in);
      for (int m = 0; m < h->M; ++m) {
        if (!(t[m] > 0.0)) throw Fail{GCN_ADMM_ERR_ARG, "theta must be positive"};
        CU(cudaMemcpyAsync(&h->ctl_z[(size_t)layer * h->M + m].t_prev, t + m, sizeof(double), cudaMemcpyHostToDevice,
                           h->stream));
      }
      CU(cudaStreamSynchronize(h->stream));
    } else if (which == GCN_ADMM_ST_PIPELINE_FLAG) {
      CU(cudaMemcpyAsync(h->tc_error, in, sizeof(int), cudaMemcpyHostToDevice, h->stream));
      CU(cudaStreamSynchronize(h->stream));
    } else {
      throw Fail{GCN_ADMM_ERR_ARG, "unknown state selector"};
    }
  });
}

int gcn_admm_launches(gcn_admm* h, long long* count) {
  return guarded(h, [&] {
    if (!count) throw Fail{GCN_ADMM_ERR_ARG, "NULL output"};
    *count = h->launches;
  });
}

int gcn_admm_profile(gcn_admm* h, int enable) {
  return guarded(h, [&] {
    h->collect_profile();
    if (enable) h->prof.clear();
    h->profiling = enable != 0;
  });
}

int gcn_admm_profile_read(gcn_admm* h, int max_entries, int* n_entries, char* names, long long* launches, double* ms,
                          double* bytes, double* flops) {
  return guarded(h, [&] {
    if (!n_entries || max_entries < 0) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    h->collect_profile();
    int k = 0;
    for (const auto& kv : h->prof) {
      if (k >= max_entries) break;
      if (names) { std::strncpy(names + (size_t)k * 48, kv.first.c_str(), 47); names[(size_t)k * 48 + 47] = 0; }
      if (launches) launches[k] = kv.second.launches;
      if (ms) ms[k] = kv.second.ms;
      if (bytes) bytes[k] = kv.second.bytes;
      if (flops) flops[k] = kv.second.flops;
      ++k;
    }
    *n_entries = k;
  });
}

int gcn_admm_decisions(gcn_admm* h, int max_passes, int* n_passes, int* trial_w, double* q_w, int* trial_z,
                       double* q_z) {
  return guarded(h, [&] {
    if (!n_passes || max_passes < 0) throw Fail{GCN_ADMM_ERR_ARG, "bad argument"};
    const int L = h->L;
    const long long have = std::min<long long>(h->log_count, kLogPasses);
    const int take = (int)std::min<long long>(have, max_passes);
    const size_t zper = (size_t)std::max(L - 1, 0) * h->M;
    CU(cudaStreamSynchronize(h->stream));
    for (int k = 0; k < take; ++k) {
      const long long pass = h->log_count - have + k;   // oldest kept pass first
      const long long slot = pass % kLogPasses;
      if (trial_w) CU(cudaMemcpy(trial_w + (size_t)k * L, h->log_trial_w + slot * L, L * sizeof(int), cudaMemcpyDeviceToHost));
      if (q_w) CU(cudaMemcpy(q_w + (size_t)k * L, h->log_q_w + slot * L, L * sizeof(double), cudaMemcpyDeviceToHost));
      if (zper && trial_z)
        CU(cudaMemcpy(trial_z + k * zper, h->log_trial_z + slot * zper, zper * sizeof(int), cudaMemcpyDeviceToHost));
      if (zper && q_z) CU(cudaMemcpy(q_z + k * zper, h->log_q_z + slot * zper, zper * sizeof(double), cudaMemcpyDeviceToHost));
    }
    *n_passes = take;
    h->check_status();
  });
}

}  // extern "C"
