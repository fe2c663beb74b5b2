// Dense product C[M x N] = A[M x K] * B on the 5th-generation tensor cores (tcgen05, accumulator
// in tensor memory), used for the feature-by-weight contractions of every layer:
//   H_l = P_l W_l,  D = P_l grad,  G = S W_{l+1}^T,  T = G W_{l+1}.
//
// fp32 accuracy from TF32 hardware: each operand x is split into x_hi + x_lo with both halves held
// at TF32 resolution (x_hi = x rounded to 10 mantissa bits, x_lo = x - x_hi, at most 2^-11 of x), and
//   A B ~= A_lo B_hi + A_hi B_lo + A_hi B_hi
// is accumulated in fp32.  The dropped terms are below 2^-21 of |a||b| per product, which keeps the
// products inside the 1e-5 single-block tolerance; one TF32 pass (2^-11) would not.  The tensor core
// rounds its fp32 accumulator toward zero at every MMA (measured: the error grows with the number of
// MMAs per accumulator), so the main product A_hi B_hi and the two small correction products get
// separate accumulators in tensor memory and are added once, in the epilogue; the residual error is
// about (K/8) * 2^-24 of the accumulated magnitude, which is why K is capped by the caller.
//
// Operand padding: leading dimensions are multiples of 4 floats and the columns K .. ld-1 of A and of
// Bk hold zeros (the library's layout invariant), so a 128-bit load that straddles K needs no masking --
// which matters: touching a loaded value right after the load would stall the prefetch.
//
// Shapes: A is M x K row-major (K contiguous), B is given K-major too: Bk[n][k] = B[k][n], N x K
// row-major (the library keeps W_l and its transpose, so one of them always has this form).
// One CTA owns 128 rows of A and all N <= 256 columns; the accumulators (128 lanes x 2 NT columns of
// fp32) live in tensor memory.  K is walked in chunks of 32 floats = one 128-byte swizzle row.
// Producer warps stage each chunk (128-bit loads from global memory, split into hi/lo, stores into shared
// memory in the canonical K-major 128-byte-swizzled operand layout); one thread issues the MMAs
// (4 steps of K = 8, three products each; up to 128 columns two of the three share one MMA, see the
// issuing loop) and commits them to the mbarrier that frees the stage; epilogue warps
// drain finished accumulators (see k_gemm_tc_ws).  Every wait on an mbarrier is bounded; a wait that runs
// out raises `*error_flag` and the CTA leaves through the normal exit (tensor memory released).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gtc {

constexpr int kBlockM = 128;
constexpr int kChunkK = 32;                 // floats per K chunk (128 bytes)
constexpr int kATileBytes = kBlockM * kChunkK * 4;     // 16 KiB, one of hi / lo
constexpr long long kWaitClocks = 1LL << 31;   // bound of every mbarrier wait, in SM clocks (about a second)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// Instruction descriptor: D fp32, A and B TF32, both K-major, M = 128, N = nt.
__device__ __forceinline__ uint32_t instr_desc(int nt) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(nt >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);
}

// Shared-memory operand descriptor of a K-major tile with the 128-byte swizzle, 8-row groups 1024 bytes
// apart: the low word holds the start address (in 16-byte units) and the LBO field (= 1), the high word the
// SBO, the version and the swizzle mode, and is the same for every tile.  The MMA wrapper takes the low
// words: the one issuing thread of a CTA then spends one addition per operand (its instruction count per
// chunk is a floor of the whole pipeline: rebuilding 64-bit descriptors and dividing by the chunk count
// there cost 16 % of the narrow products).
constexpr uint32_t kOperandDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // SBO, version 1, SWIZZLE_128B
__device__ __forceinline__ uint32_t operand_desc_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3fffu) | (1u << 16); }
__device__ __forceinline__ void mma_tf32_lo(uint32_t tmem_d, uint32_t da_lo, uint32_t db_lo, uint32_t idesc, uint32_t accumulate,
                                            uint32_t desc_hi = kOperandDescHi) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "r"(da_lo), "r"(db_lo), "r"(idesc), "r"(accumulate), "r"(0u), "r"(desc_hi)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define GTC_TMEM_LD16(v, addr)                                                                                       \
  asm volatile(                                                                                                      \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];" \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),   \
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])                      \
      : "r"(addr)                                                                                                    \
      : "memory")

// x -> (hi, lo): hi = x rounded to TF32 (ties away; zero in the 13 low mantissa bits, so the tensor
// core reads it exactly), lo = x - hi exactly (|lo| <= 2^-11 |x|).  lo is handed over as it is: whatever
// the hardware does with its low 13 bits moves it by at most 2^-10 |lo| <= 2^-21 |x|.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  hi = __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
  lo = x - hi;
}

// Swizzled byte offset of the 16-byte unit `c16` (0..7) of row `r` inside a K-major operand tile.
__device__ __forceinline__ uint32_t swz(int r, int c16) { return (uint32_t)r * 128u + (uint32_t)((c16 ^ (r & 7)) << 4); }

// ------------------------------------------------------------------------------------------------
// The product kernel: work split by role, so that staging, MMA issue and the epilogue overlap.
//   warps 0-7   producers: 128-bit loads of the A and B chunks (two chunks ahead, in registers),
//               hi/lo split, swizzled stores, fence, arrive on full[stage]
//   warps 8-11 (8-15 with one accumulator set)  epilogue: wait for a finished accumulator set,
//               tensor memory -> registers -> C, arrive on acc_empty[set]  (warp w reads lanes
//               32 (w mod 4) .. +31; with eight warps the two of a quarter take the column steps in turn)
//   next warp   MMA: waits full[stage] (and, at the first chunk of a tile, acc_empty[set]), issues
//               the chunk's MMAs, commits to empty[stage] and, at the last chunk, to acc_full[set]
// Up to 128 output columns, two accumulator sets (main + correction each) alternate between consecutive
// tiles (4 NT <= 512 columns of tensor memory); from 129 to 256 columns there is room for one set, and
// the MMAs of the next tile wait for the epilogue of the current one while the producers keep staging.
// A wait that runs out raises a shared abort flag that every other wait polls; all roles then meet
// at the closing barrier and tensor memory is released.
// ------------------------------------------------------------------------------------------------


// One arrival for the whole warp: an mbarrier arrival is an atomic update of one shared-memory word, and 256
// of them per K chunk, one after the other, were the floor of about 1,600 clocks per chunk that no change to
// the staging itself had moved.  Every lane has made its shared-memory stores visible to the async proxy
// (fence.proxy.async) before the call; __syncwarp orders them before lane 0's releasing arrival.
__device__ __forceinline__ void mbar_arrive_warp(uint32_t bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Waits for a phase, giving up when another role has raised the abort flag or after kWaitClocks (a try_wait
// may itself suspend the thread for a while, so the bound is on elapsed clocks, not on attempts).
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  long long t0 = 0;   // read only once the wait has proved long: a wait that succeeds at once costs one try
  for (uint32_t i = 0;; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((i & 63u) == 63u) {
      if (*abort_flag) return false;
      if (t0 == 0) t0 = clock64();
      else if (clock64() - t0 > kWaitClocks) break;
    }
  }
  *abort_flag = 1;
  return false;
}

template <int NT>
struct WsCfg {
  static constexpr int kSets = NT > 128 ? 1 : 2;                        // accumulator sets (main + correction each)
  // With one accumulator set (more than 128 columns) the epilogue of a tile is not covered by MMAs:
  // eight epilogue warps then, two per quarter of the tensor-memory lanes, taking the column steps in
  // turn (measured 3-8 % faster); with two sets four warps are enough and leave more registers.
  static constexpr int kEpiWarps = NT > 128 ? 8 : 4;
  static constexpr int kMmaWarp = 8 + kEpiWarps;
  static constexpr int kThreads = (kMmaWarp + 1) * 32;
  static constexpr int kStagesWs = NT > 128 ? 2 : NT > 64 ? 3 : 4;
  static constexpr int kBTile = NT * kChunkK * 4;                       // one of hi / lo
  static constexpr int kStage = 2 * kATileBytes + 2 * kBTile;
  static constexpr int kAccCols = kSets * 2 * NT;
  static constexpr uint32_t kTmemCols = kAccCols <= 64 ? 64 : kAccCols <= 128 ? 128 : kAccCols <= 256 ? 256 : 512;
  static constexpr size_t kSmem = (size_t)kStagesWs * kStage + kEpiWarps * 4096 + 1024;   // + the epilogue warps' buffers
  // Tensor-copy form (NT <= 128): a ring of R slots {raw A tile (read in place as the hi operand), B_hi, B_lo},
  // filled by copies alone and therefore a DRAM latency ahead of the MMAs, and a ring of S A_lo tiles that the
  // producers fill from the raw tiles; a lo tile is held only from the producers' stores to the end of its MMAs.
  static constexpr int kRawSlots = NT > 64 ? 3 : 5;
  static constexpr int kLoStages = 3;
  static constexpr int kRawSlot = kATileBytes + 2 * kBTile;
  static constexpr size_t kSmemRing = (size_t)kRawSlots * kRawSlot + (size_t)kLoStages * kATileBytes + kEpiWarps * 4096 + 1024;
};

// The weight operand split once, in the layout the MMA descriptors read: for column group g and K
// chunk kc, the 128-byte-swizzled NT x 32 tile of B_hi followed by that of B_lo, one contiguous block
// of 2 * NT * 128 bytes at block index g * chunks + kc.  With it (IMG = true) a stage's B tiles arrive
// by one bulk copy issued by one thread, and the producers stage A only; without it they load, split
// and store B again for every 128-row tile.
__global__ void k_split_b(const float* __restrict__ Bk, int ldbk, int N, int K, int nt, uint8_t* __restrict__ image) {
  const int kc_count = (K + kChunkK - 1) / kChunkK;
  const int groups = (N + nt - 1) / nt;
  const long long total = (long long)groups * kc_count * nt * 8;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int c16 = (int)(i & 7);
    const int nrow = (int)((i >> 3) % nt);
    const long long blk = i / (8LL * nt);
    const int kc = (int)(blk % kc_count), g = (int)(blk / kc_count);
    const int k0 = kc * kChunkK + c16 * 4, n = g * nt + nrow;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (n < N && k0 < K) v = *reinterpret_cast<const float4*>(Bk + (long long)n * ldbk + k0);
    float4 h, l;
    split_tf32(v.x, h.x, l.x); split_tf32(v.y, h.y, l.y); split_tf32(v.z, h.z, l.z); split_tf32(v.w, h.w, l.w);
    uint8_t* dst = image + (size_t)blk * (size_t)(2 * nt * kChunkK * 4) + swz(nrow, c16);
    *reinterpret_cast<float4*>(dst) = h;
    *reinterpret_cast<float4*>(dst + (size_t)nt * kChunkK * 4) = l;
  }
}

// TMA = true (needs IMG): the A operand is not loaded by the producers at all.  One more warp (its lane 0)
// fetches each 128 x 32 tile of A with a tensor copy (cp.async.bulk.tensor, 128-byte swizzle: the copy
// engine writes exactly the K-major layout the MMA descriptors read) and the chunk's two weight tiles with
// a bulk copy into slot j mod R of a ring that only copies fill, up to R chunks ahead of the MMAs.  The
// tensor core reads a 32-bit operand as TF32 by dropping its 13 low mantissa bits, so the raw tile IS the
// hi operand, hi = x with those bits cleared, and the producers only form lo = x - hi from the tile in
// shared memory (exact) and store it into stage j mod S of a second ring: no global loads and half the
// stores, and the A stream no longer passes through L1.  A slot is freed by the commit of its chunk's
// MMAs (raw_empty), a lo stage likewise (empty).  Rows past M and columns past the matrix are filled with
// zeros by the copy.
template <int NT, bool IMG, bool TMA = false>
__global__ void __launch_bounds__(WsCfg<NT>::kThreads + (TMA ? 32 : 0), 1)
k_gemm_tc_ws(const float* __restrict__ A, int lda, const float* __restrict__ Bk, int ldbk, float* __restrict__ C, int ldc,
             int M, int N, int K, const int* __restrict__ skip, int* __restrict__ error_flag,
             const uint8_t* __restrict__ b_image, const __grid_constant__ CUtensorMap tmap_a) {
  static_assert(!TMA || IMG, "the tensor-copy form stages no B tile");
  using Cfg = WsCfg<NT>;
  constexpr int S = TMA ? Cfg::kLoStages : Cfg::kStagesWs;   // stages of the ring the producers fill
  constexpr int R = TMA ? Cfg::kRawSlots : 1;                // slots of the ring the copies fill (tensor-copy form only)
  constexpr int B_PASSES = (NT + 31) / 32;
  constexpr int A_PASSES = kBlockM / 32;
  constexpr int SETS = Cfg::kSets;
  static_assert(NT <= 256 && NT % 16 == 0, "NT");
  if (skip != nullptr && *skip) return;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * S + 4 + 2 * R];      // full[S], empty[S], acc_full[2], acc_empty[2], raw_full[R], raw_empty[R]
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[S]);
  const uint32_t bar_acc_full = smem_u32(&bars[2 * S]), bar_acc_empty = smem_u32(&bars[2 * S + 2]);
  const uint32_t bar_raw_full = smem_u32(&bars[2 * S + 4]), bar_raw_empty = smem_u32(&bars[2 * S + 4 + R]);
  // shared-memory map of the tensor-copy form: R slots of {raw A, B_hi, B_lo}, then S tiles of A_lo
  constexpr uint32_t kRawSlot = (uint32_t)Cfg::kRawSlot;
  constexpr uint32_t kLoBase = (uint32_t)R * kRawSlot;
  constexpr uint32_t kStageBytes = TMA ? (uint32_t)kATileBytes : (uint32_t)Cfg::kStage;
  constexpr uint32_t kRingBytes = TMA ? kLoBase + (uint32_t)S * kStageBytes : (uint32_t)S * kStageBytes;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8 * s, 8); mbar_init(bar_empty + 8 * s, 1); }   // full: one arrival per producer warp
    for (int r = 0; r < R; ++r) { mbar_init(bar_raw_full + 8 * r, 1); mbar_init(bar_raw_empty + 8 * r, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, Cfg::kEpiWarps); }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == Cfg::kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(Cfg::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;

  const int kc_count = (K + kChunkK - 1) / kChunkK;
  const int n_tiles = (M + kBlockM - 1) / kBlockM;
  const int my_tiles = (n_tiles > (int)blockIdx.x) ? (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int total = my_tiles * kc_count;
  const int n0 = blockIdx.y * NT;
  const int n_loc = min(NT, N - n0);

  if (warp < 8) {
    // ---------------- producers ----------------
    const int ld_c16 = tid & 7, ld_row = tid >> 3;
    constexpr int DEPTH = IMG ? 4 : (NT > 128 ? 1 : 2);   // chunks a thread holds in registers ahead of the one it stores
    float4 ra[DEPTH][A_PASSES], rb[DEPTH][IMG ? 1 : B_PASSES];
    // chunks are loaded strictly in order, so tile and K chunk of the next load are counters (no division per chunk)
    int ld_j = 0, ld_kc = 0, st_kc = 0;
    long long ld_row0 = (long long)blockIdx.x * kBlockM;
    auto load_chunk = [&](float4* pa, float4* pb) {
      if (ld_j >= total) return;
      const int k0 = ld_kc * kChunkK + ld_c16 * 4;
      const long long row0 = ld_row0;
      ++ld_j;
      if (++ld_kc == kc_count) { ld_kc = 0; ld_row0 += (long long)gridDim.x * kBlockM; }
#pragma unroll
      for (int i = 0; i < A_PASSES; ++i) {
        const long long r = row0 + ld_row + 32 * i;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < M && k0 < K) {
          v = *reinterpret_cast<const float4*>(A + r * lda + k0);
        }
        pa[i] = v;
      }
      if (!IMG) {
#pragma unroll
        for (int i = 0; i < B_PASSES; ++i) {
          const int nrow = ld_row + 32 * i;
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (nrow < n_loc && k0 < K) {
            v = *reinterpret_cast<const float4*>(Bk + (long long)(n0 + nrow) * ldbk + k0);
          }
          pb[i] = v;
        }
      }
    };
    auto store_chunk = [&](int stage, const float4* pa, const float4* pb) {
      uint8_t* st = smem + (size_t)stage * Cfg::kStage;
#pragma unroll
      for (int i = 0; i < A_PASSES; ++i) {
        float4 h, l;
        split_tf32(pa[i].x, h.x, l.x); split_tf32(pa[i].y, h.y, l.y);
        split_tf32(pa[i].z, h.z, l.z); split_tf32(pa[i].w, h.w, l.w);
        const uint32_t off = swz(ld_row + 32 * i, ld_c16);
        *reinterpret_cast<float4*>(st + off) = h;
        *reinterpret_cast<float4*>(st + kATileBytes + off) = l;
      }
      if (!IMG) {
#pragma unroll
        for (int i = 0; i < B_PASSES; ++i) {
          const int nrow = ld_row + 32 * i;
          if (nrow < NT) {
            float4 h, l;
            split_tf32(pb[i].x, h.x, l.x); split_tf32(pb[i].y, h.y, l.y);
            split_tf32(pb[i].z, h.z, l.z); split_tf32(pb[i].w, h.w, l.w);
            const uint32_t off = swz(nrow, ld_c16);
            *reinterpret_cast<float4*>(st + 2 * kATileBytes + off) = h;
            *reinterpret_cast<float4*>(st + 2 * kATileBytes + Cfg::kBTile + off) = l;
          }
        }
      }
    };
    if (TMA) {
      // chunk j: raw tile and weight tiles in slot j mod R (see the copy warp below), lo in stage j mod S
      int stage = 0, slot = 0;
      uint32_t empty_parity = 1, raw_parity = 0;   // a fresh barrier passes a wait on parity 1
      for (int j = 0; j < total; ++j) {
        if (!__all_sync(0xffffffffu, mbar_wait_abortable(bar_empty + 8 * stage, empty_parity, abortp))) break;   // warp-uniform: the arrival below is per warp
        if (!__all_sync(0xffffffffu, mbar_wait_abortable(bar_raw_full + 8 * slot, raw_parity, abortp))) break;
        const uint8_t* raw = smem + (size_t)slot * kRawSlot;
        uint8_t* st = smem + kLoBase + (size_t)stage * kStageBytes;
#pragma unroll
        for (int i = 0; i < A_PASSES; ++i) {
          const uint32_t off = swz(ld_row + 32 * i, ld_c16);
          const float4 x = *reinterpret_cast<const float4*>(raw + off);
          float4 l;
          l.x = x.x - __uint_as_float(__float_as_uint(x.x) & 0xffffe000u);
          l.y = x.y - __uint_as_float(__float_as_uint(x.y) & 0xffffe000u);
          l.z = x.z - __uint_as_float(__float_as_uint(x.z) & 0xffffe000u);
          l.w = x.w - __uint_as_float(__float_as_uint(x.w) & 0xffffe000u);
          *reinterpret_cast<float4*>(st + off) = l;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive_warp(bar_full + 8 * stage);
        if (++stage == S) { stage = 0; empty_parity ^= 1u; }
        if (++slot == R) { slot = 0; raw_parity ^= 1u; }
      }
    } else {
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) load_chunk(ra[d], rb[d]);
    bool stop = false;
    for (int j0 = 0; j0 < total && !stop; j0 += DEPTH) {
#pragma unroll
      for (int d = 0; d < DEPTH; ++d) {
        const int j = j0 + d;
        if (j >= total) break;
        const int stage = j % S;
        if (j >= S && !__all_sync(0xffffffffu, mbar_wait_abortable(bar_empty + 8 * stage, ((j / S) - 1) & 1, abortp))) { stop = true; break; }
        if (IMG && tid == 0) {
          // the stage is free (its MMAs have retired): fetch both B tiles of this chunk with one bulk copy
          // that reports its bytes to the stage's full barrier; this thread's own arrival comes below
          const uint32_t bytes = 2u * (uint32_t)Cfg::kBTile;
          const uint8_t* src = b_image + ((size_t)blockIdx.y * kc_count + (size_t)st_kc) * bytes;
          const uint32_t dst = smem_base + (uint32_t)stage * Cfg::kStage + 2u * kATileBytes;
          asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar_full + 8 * stage), "r"(bytes) : "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                       ::"r"(dst), "l"(src), "r"(bytes), "r"(bar_full + 8 * stage)
                       : "memory");
        }
        if (++st_kc == kc_count) st_kc = 0;
        store_chunk(stage, ra[d], rb[d]);
        load_chunk(ra[d], rb[d]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive_warp(bar_full + 8 * stage);
      }
    }
    }
  } else if (TMA && warp == Cfg::kMmaWarp + 1) {
    // ---------------- copies (tensor-copy form only): A tile and weight tiles of chunk j as soon as slot j mod R is free ----------------
    if (lane == 0) {
      const uint32_t b_bytes = 2u * (uint32_t)Cfg::kBTile;
      const uint8_t* const b_src = b_image + (size_t)blockIdx.y * kc_count * b_bytes;
      int kc = 0, tile = blockIdx.x, slot = 0;
      uint32_t empty_parity = 1;   // a fresh barrier passes a wait on parity 1
      for (int j = 0; j < total; ++j) {
        if (!mbar_wait_abortable(bar_raw_empty + 8 * slot, empty_parity, abortp)) break;
        const uint32_t dst_a = smem_base + (uint32_t)slot * kRawSlot;
        const uint32_t raw_bar = bar_raw_full + 8 * slot;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(raw_bar), "r"((uint32_t)kATileBytes + b_bytes) : "memory");
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                     ::"r"(dst_a), "l"(&tmap_a), "r"(kc * kChunkK), "r"(tile * kBlockM), "r"(raw_bar)
                     : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst_a + (uint32_t)kATileBytes), "l"(b_src + (size_t)kc * b_bytes), "r"(b_bytes), "r"(raw_bar)
                     : "memory");
        if (++kc == kc_count) { kc = 0; tile += gridDim.x; }
        if (++slot == R) { slot = 0; empty_parity ^= 1u; }
      }
    }
  } else if (warp == Cfg::kMmaWarp) {
    // ---------------- MMA issue ----------------
    // One thread issues everything, so its instruction count per chunk is a floor of the whole pipeline
    // (no division by kc_count, no 64-bit descriptor arithmetic: counters that wrap, one addition per operand).
    if (lane == 0) {
      const uint32_t idesc = instr_desc(NT), idesc2 = instr_desc(NT <= 128 ? 2 * NT : NT);
      int stage = 0, kc = 0, tile_i = 0, slot = 0;
      uint32_t full_parity = 0;
      for (int j = 0; j < total; ++j) {
        const int set = SETS == 1 ? 0 : (tile_i & 1);
        if (kc == 0 && tile_i >= SETS && !mbar_wait_abortable(bar_acc_empty + 8 * set, ((tile_i / SETS) - 1) & 1, abortp)) break;
        if (!mbar_wait_abortable(bar_full + 8 * stage, full_parity, abortp)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // shared memory ends below 2^18, so additions to a descriptor's low word never carry out of the address field
        const uint32_t a_hi = operand_desc_lo(TMA ? smem_base + slot * kRawSlot : smem_base + stage * kStageBytes);
        const uint32_t a_lo = TMA ? operand_desc_lo(smem_base + kLoBase + stage * kStageBytes) : a_hi + (kATileBytes >> 4);
        const uint32_t b_hi = TMA ? a_hi + (kATileBytes >> 4) : a_hi + (2 * kATileBytes >> 4), b_lo = b_hi + (Cfg::kBTile >> 4);
        const uint32_t acc = tmem_base + (uint32_t)(set * 2 * NT);
#pragma unroll
        for (int ks = 0; ks < kChunkK / 8; ++ks) {
          const uint32_t o = ks * 2;   // 32 bytes per K step, in 16-byte units
          const uint32_t first = (ks > 0) ? 1u : (kc > 0 ? 1u : 0u);
          if constexpr (NT <= 128) {
            // B_lo follows B_hi in shared memory in the same 8-row groups, so the two are one operand of 2 NT
            // rows: A_hi [B_hi; B_lo] fills the main accumulator (columns 0 .. NT-1) and starts the correction
            // (columns NT .. 2 NT - 1) in one MMA; A_lo B_hi is added to the correction.  Two MMAs per K step
            // instead of three: narrow MMAs have a floor on their duration, and each one costs the issuing thread.
            mma_tf32_lo(acc, a_hi + o, b_hi + o, idesc2, first);
            mma_tf32_lo(acc + NT, a_lo + o, b_hi + o, idesc, 1u);
          } else {
            mma_tf32_lo(acc + NT, a_lo + o, b_hi + o, idesc, first);   // corrections
            mma_tf32_lo(acc + NT, a_hi + o, b_lo + o, idesc, 1u);
            mma_tf32_lo(acc, a_hi + o, b_hi + o, idesc, first);        // main product
          }
        }
        mma_commit(bar_empty + 8 * stage);
        if (TMA) {
          mma_commit(bar_raw_empty + 8 * slot);
          if (++slot == R) slot = 0;
        }
        if (++kc == kc_count) {
          mma_commit(bar_acc_full + 8 * set);
          kc = 0;
          ++tile_i;
        }
        if (++stage == S) { stage = 0; full_parity ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue ----------------
    // In tensor memory a lane holds one row, so a direct store would have the 32 lanes of a warp write
    // 16 bytes each to 32 different rows.  The sums of CW columns go through a per-warp buffer in shared
    // memory instead (128-byte rows, 16-byte slots XORed with the row index) and leave as whole lines:
    // 32 / (CW/4) rows of CW contiguous floats per store instruction.
    const int quarter = warp & 3;
    constexpr int CW = (NT % 32 == 0) ? 32 : 16;      // columns per step
    constexpr int SLOTS = CW / 4;                      // float4 per row and step
    constexpr int ROWS_PER_STORE = 32 / SLOTS;
    const int turn = (warp - 8) >> 2;                  // which of the quarter's two warps this is
    uint8_t* tbuf = smem + kRingBytes + (size_t)(warp - 8) * 4096;
    for (int tile_i = 0; tile_i < my_tiles; ++tile_i) {
      const int set = tile_i % SETS;
      if (!__all_sync(0xffffffffu, mbar_wait_abortable(bar_acc_full + 8 * set, (tile_i / SETS) & 1, abortp))) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long row0 = (long long)(blockIdx.x + tile_i * gridDim.x) * kBlockM + quarter * 32;
#pragma unroll 1
      for (int cstep = turn; cstep < NT / CW; cstep += Cfg::kEpiWarps / 4) {
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(set * 2 * NT + cstep * CW);
#pragma unroll
        for (int half = 0; half < CW / 16; ++half) {
          uint32_t v[16], w[16];
          GTC_TMEM_LD16(v, taddr + (uint32_t)(half * 16));
          GTC_TMEM_LD16(w, taddr + (uint32_t)(NT + half * 16));
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int slot = (half * 4 + q) ^ (lane & (SLOTS - 1));
            *reinterpret_cast<float4*>(tbuf + lane * 128 + slot * 16) =
                make_float4(__uint_as_float(v[q * 4]) + __uint_as_float(w[q * 4]),
                            __uint_as_float(v[q * 4 + 1]) + __uint_as_float(w[q * 4 + 1]),
                            __uint_as_float(v[q * 4 + 2]) + __uint_as_float(w[q * 4 + 2]),
                            __uint_as_float(v[q * 4 + 3]) + __uint_as_float(w[q * 4 + 3]));
          }
        }
        __syncwarp();
        const int c4 = lane & (SLOTS - 1);
        const int col = n0 + cstep * CW + c4 * 4;
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) {
          const int r = i * ROWS_PER_STORE + lane / SLOTS;
          const float4 val = *reinterpret_cast<const float4*>(tbuf + r * 128 + ((c4 ^ (r & (SLOTS - 1))) * 16));
          if (row0 + r < M && col < ldc) *reinterpret_cast<float4*>(C + (row0 + r) * ldc + col) = val;
        }
        __syncwarp();
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive_warp(bar_acc_empty + 8 * set);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0 && abort_flag) atomicExch(error_flag, 1);
  if (warp == Cfg::kMmaWarp) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Transposed product on the tensor cores:  part[s][Ka x Nb] = sum over the rows of split s of
// A[r,:]^T B[r,:]  (the weight gradient P^T R, reduction over the node dimension).
// Here the reduction index r is the MMA's K, and both operands are stored with their own index
// (ka, nb) contiguous: "MN-major" operands, for which 32-bit elements have exactly one shared-memory
// form: 128-byte rows swizzled at 32-byte granularity.  A chunk is 32 rows; atom (g, q) holds rows
// 4q..4q+3 of column group g (32 columns = 128 bytes per row), 512 bytes, and inside it the 32-byte
// unit u of row r sits at unit u ^ (r mod 4); successive column groups are 4096 bytes apart (the
// descriptor's leading byte offset), successive groups of 4 rows 512 bytes apart (its stride byte
// offset).  One MMA consumes 8 rows (K = 8), i.e. two atoms.  Same hi/lo split, same separate correction accumulator, same roles as
// above (8 producer warps, one MMA warp); a CTA owns 128 columns of A (blockIdx.x), NT columns of B
// (blockIdx.z) and one row split (blockIdx.y) and writes its 128 x NT partial sum once, at the end.
// The column groups of A are the fastest grid index: the CTAs that read the same rows of B start
// together, and the second one finds them in L2.
// ------------------------------------------------------------------------------------------------
constexpr int kTnThreads = 9 * 32;
constexpr int kTnRows = 32;                       // rows (reduction steps) per chunk

// MN-major tile: LBO = 4096, SBO = 512, version 1, 128-byte swizzle with 32-byte base (low / high word as above)
constexpr uint32_t kOperandDescMnHi = (512u >> 4) | (1u << 14) | (1u << 29);
__device__ __forceinline__ uint32_t operand_desc_mn_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3fffu) | ((4096u >> 4) << 16); }
__device__ __forceinline__ uint32_t instr_desc_mn(int nt) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(nt >> 3) << 17) |
         ((uint32_t)(kBlockM >> 4) << 24);
}
// byte offset of float4 number c4 (columns 4 c4 .. 4 c4 + 3) of chunk row r in an MN-major tile
__device__ __forceinline__ uint32_t swz_mn(int r, int c4) {
  return (uint32_t)(c4 >> 3) * 4096u + (uint32_t)(r >> 2) * 512u + (uint32_t)(r & 3) * 128u +
         (uint32_t)(((((c4 & 7) >> 1) ^ (r & 3)) << 5) | ((c4 & 1) << 4));
}

template <int NT>
struct TnCfg {
  static constexpr int kGroupsB = (NT + 31) / 32;
  static constexpr int kATile = 4 * 4096;                 // 128 columns x 32 rows, one of hi / lo
  static constexpr int kBTile = kGroupsB * 4096;
  static constexpr int kStage = 2 * kATile + 2 * kBTile;
  static constexpr int kStagesTn = kStage > 72 * 1024 ? 2 : 3;
  static constexpr uint32_t kTmemCols = 2 * NT <= 32 ? 32 : 2 * NT <= 64 ? 64 : 2 * NT <= 128 ? 128 : 2 * NT <= 256 ? 256 : 512;
  static constexpr size_t kSmem = (size_t)kStagesTn * kStage + 1024;
};

// RESID: B is not stored.  The operand is the derivative of a hidden layer's penalty with respect to
// its pre-activation, formed while staging from the pre-activation H (passed as B) and the layer's
// Z (Zres, same leading dimension):  b = h > 0 ? nu (h - z) : 0.  Both rows are fetched one chunk
// ahead (A stays two chunks ahead), so the second matrix costs no further registers.
template <int NT, bool RESID>
__global__ void __launch_bounds__(kTnThreads, 1)
k_gemm_tn_tc(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb, float* __restrict__ part, int ldp,
             long long rows, long long rows_per_split, int Ka, int Nb, int* __restrict__ error_flag,
             const float* __restrict__ Zres, float nu) {
  using Cfg = TnCfg<NT>;
  constexpr int S = Cfg::kStagesTn;
  constexpr int A_PASSES = 4;                              // 1024 float4 / 256 threads
  constexpr int B_F4 = kTnRows * (NT / 4);
  constexpr int B_PASSES = (B_F4 + 255) / 256;
  static_assert(NT % 16 == 0 && NT <= 256, "NT");

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * S + 1];       // full[S], empty[S], acc_full
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[S]), bar_acc = smem_u32(&bars[2 * S]);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8 * s, 8); mbar_init(bar_empty + 8 * s, 1); }   // full: one arrival per producer warp
    mbar_init(bar_acc, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(Cfg::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;

  const long long r_begin = (long long)blockIdx.y * rows_per_split;
  const long long r_end = min(rows, r_begin + rows_per_split);
  const int total = r_end > r_begin ? (int)((r_end - r_begin + kTnRows - 1) / kTnRows) : 0;
  const int ka0 = blockIdx.x * kBlockM;
  const int nb0 = blockIdx.z * NT;                 // first column of B (and of the partial sum) of this CTA

  if (warp < 8) {
    // ---------------- producers ----------------
    float4 ra[2][A_PASSES], rb[2][B_PASSES];
    auto load_a = [&](int j, float4* pa) {
      if (j >= total) return;
      const long long r0 = r_begin + (long long)j * kTnRows;
#pragma unroll
      for (int i = 0; i < A_PASSES; ++i) {
        const int f = tid + 256 * i, rr = f >> 5, c4 = f & 31;
        const long long r = r0 + rr;
        const int col = ka0 + 4 * c4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < r_end && col < Ka) v = *reinterpret_cast<const float4*>(A + r * lda + col);   // zero padding beyond Ka
        pa[i] = v;
      }
    };
    auto load_b = [&](int j, const float* __restrict__ src, float4* pb) {
      if (j >= total) return;
      const long long r0 = r_begin + (long long)j * kTnRows;
#pragma unroll
      for (int i = 0; i < B_PASSES; ++i) {
        const int f = tid + 256 * i;
        const int rr = f / (NT / 4), c4 = f % (NT / 4);
        const long long r = r0 + rr;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (f < B_F4 && r < r_end && nb0 + 4 * c4 < Nb) v = *reinterpret_cast<const float4*>(src + r * ldb + nb0 + 4 * c4);
        pb[i] = v;
      }
    };
    auto store_chunk = [&](int stage, const float4* pa, const float4* pb, const float4* pz) {
      uint8_t* st = smem + (size_t)stage * Cfg::kStage;
#pragma unroll
      for (int i = 0; i < A_PASSES; ++i) {
        const int f = tid + 256 * i, rr = f >> 5, c4 = f & 31;
        float4 h, l;
        split_tf32(pa[i].x, h.x, l.x); split_tf32(pa[i].y, h.y, l.y);
        split_tf32(pa[i].z, h.z, l.z); split_tf32(pa[i].w, h.w, l.w);
        const uint32_t off = swz_mn(rr, c4);
        *reinterpret_cast<float4*>(st + off) = h;
        *reinterpret_cast<float4*>(st + Cfg::kATile + off) = l;
      }
#pragma unroll
      for (int i = 0; i < B_PASSES; ++i) {
        const int f = tid + 256 * i;
        if (f < B_F4) {
          const int rr = f / (NT / 4), c4 = f % (NT / 4);
          float4 b = pb[i];
          if (RESID) {
            const float4 z = pz[i];
            b.x = b.x > 0.f ? nu * (b.x - z.x) : 0.f;
            b.y = b.y > 0.f ? nu * (b.y - z.y) : 0.f;
            b.z = b.z > 0.f ? nu * (b.z - z.z) : 0.f;
            b.w = b.w > 0.f ? nu * (b.w - z.w) : 0.f;
          }
          float4 h, l;
          split_tf32(b.x, h.x, l.x); split_tf32(b.y, h.y, l.y);
          split_tf32(b.z, h.z, l.z); split_tf32(b.w, h.w, l.w);
          const uint32_t off = swz_mn(rr, c4);
          *reinterpret_cast<float4*>(st + 2 * Cfg::kATile + off) = h;
          *reinterpret_cast<float4*>(st + 2 * Cfg::kATile + Cfg::kBTile + off) = l;
        }
      }
    };
    load_a(0, ra[0]);
    load_a(1, ra[1]);
    if (RESID) {   // rb[0] = rows of H, rb[1] = rows of Z, both of the next chunk
      load_b(0, B, rb[0]);
      load_b(0, Zres, rb[1]);
    } else {
      load_b(0, B, rb[0]);
      load_b(1, B, rb[1]);
    }
    for (int j = 0; j < total; ++j) {
      const int stage = j % S;
      if (j >= S && !__all_sync(0xffffffffu, mbar_wait_abortable(bar_empty + 8 * stage, ((j / S) - 1) & 1, abortp))) break;
      if (RESID) {
        if (j & 1) { store_chunk(stage, ra[1], rb[0], rb[1]); load_a(j + 2, ra[1]); }
        else       { store_chunk(stage, ra[0], rb[0], rb[1]); load_a(j + 2, ra[0]); }
        load_b(j + 1, B, rb[0]);
        load_b(j + 1, Zres, rb[1]);
      } else {
        if (j & 1) { store_chunk(stage, ra[1], rb[1], nullptr); load_a(j + 2, ra[1]); load_b(j + 2, B, rb[1]); }
        else       { store_chunk(stage, ra[0], rb[0], nullptr); load_a(j + 2, ra[0]); load_b(j + 2, B, rb[0]); }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive_warp(bar_full + 8 * stage);
    }
  } else if (lane == 0) {
    // ---------------- MMA issue ----------------
    // one issuing thread: counters that wrap and one addition per operand descriptor (see k_gemm_tc_ws)
    const uint32_t idesc = instr_desc_mn(NT);
    int stage = 0;
    uint32_t full_parity = 0;
    for (int j = 0; j < total; ++j) {
      if (!mbar_wait_abortable(bar_full + 8 * stage, full_parity, abortp)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_hi = operand_desc_mn_lo(smem_base + stage * Cfg::kStage), a_lo = a_hi + (Cfg::kATile >> 4);
      const uint32_t b_hi = a_hi + (2 * Cfg::kATile >> 4), b_lo = b_hi + (Cfg::kBTile >> 4);
#pragma unroll
      for (int ks = 0; ks < kTnRows / 8; ++ks) {
        const uint32_t o = ks * (1024 >> 4);       // the next group of 8 rows, in 16-byte units
        const uint32_t first = (ks > 0) ? 1u : (j > 0 ? 1u : 0u);
        mma_tf32_lo(tmem_base + NT, a_lo + o, b_hi + o, idesc, first, kOperandDescMnHi);   // corrections
        mma_tf32_lo(tmem_base + NT, a_hi + o, b_lo + o, idesc, 1u, kOperandDescMnHi);
        mma_tf32_lo(tmem_base, a_hi + o, b_hi + o, idesc, first, kOperandDescMnHi);        // main product
      }
      mma_commit(bar_empty + 8 * stage);
      if (j + 1 == total) mma_commit(bar_acc);
      if (++stage == S) { stage = 0; full_parity ^= 1u; }
    }
  }
  __syncwarp();
  // ---------------- epilogue: warps 0-3, one tensor-memory lane (= column of A) per thread ----------------
  if (warp < 4) {
    bool ok = true;
    if (total > 0) ok = mbar_wait_abortable(bar_acc, 0, abortp);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int ka = ka0 + warp * 32 + lane;
    float* dst = part + ((long long)blockIdx.y * Ka + ka) * ldp;
#pragma unroll 1
    for (int cchunk = 0; cchunk < NT / 16; ++cchunk) {
      uint32_t v[16], w[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) v[q] = w[q] = 0u;
      if (ok && total > 0) {
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(cchunk * 16);
        GTC_TMEM_LD16(v, taddr);
        GTC_TMEM_LD16(w, taddr + (uint32_t)NT);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      }
      if (ka < Ka) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int col = nb0 + cchunk * 16 + q * 4;
          if (col < ldp)
            *reinterpret_cast<float4*>(dst + col) =
                make_float4(__uint_as_float(v[q * 4]) + __uint_as_float(w[q * 4]),
                            __uint_as_float(v[q * 4 + 1]) + __uint_as_float(w[q * 4 + 1]),
                            __uint_as_float(v[q * 4 + 2]) + __uint_as_float(w[q * 4 + 2]),
                            __uint_as_float(v[q * 4 + 3]) + __uint_as_float(w[q * 4 + 3]));
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0 && abort_flag) atomicExch(error_flag, 1);
  if (warp == 8) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
  }
}

}  // namespace gtc
