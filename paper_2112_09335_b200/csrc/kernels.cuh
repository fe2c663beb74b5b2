// Device kernels of the community-based ADMM GCN trainer (sm_100a).
//
// Layout: every N x C matrix is row-major fp32 with a leading dimension padded to a multiple
// of 4 floats, rows in community order, so that a row starts on a 16-byte boundary and can be
// moved with 128-bit loads.  Padding columns are kept at zero.
// Scalars that decide a step size (descent sums, squared norms) are accumulated in fp64.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gk {

constexpr int kCand = 4;        // step-size candidates scored per pass
constexpr int kMaxClassesPerLane = 4;   // C_L <= 128

// Control block of one quadratic-approximation search (one per W_l, one per Z_{l,m}).
struct SearchCtl {
  double t_prev;   // accepted parameter of the previous search (tau_l or theta_{l,m})
  double t_base;   // first candidate of the current pass
  double gg;       // ||grad||^2
  double xx;       // ||x||^2 of the block
  double q;        // (f(x) - f(x+)) / (gg / 2t) at the accepted trial
  float inv_step;  // 1/t of the accepted trial, 0 when the block stays
  int done;        // search finished (accepted, skipped or exhausted)
  int trial;       // accepted trial index, -1 skipped, -2 exhausted
  int pass;        // passes already scored
  float inv_cand[kCand];  // 1/t of the candidates of the current pass
};

__device__ __forceinline__ float relu(float x) { return x > 0.f ? x : 0.f; }

// relu(h) - relu(h - s) without forming h - s when both sides are active, so that a step s far
// below the rounding unit of h still registers exactly.  With pos = max(h, 0) and neg = max(-h, 0)
// (one of them is zero) the drop is min(s + neg, pos): for h > 0 that is min(s, h), for h <= 0 it
// is min(s - h, 0).  The caller forms pos and neg once per element and passes s = k * inv as the
// two factors, so a candidate costs one fused multiply-add and one minimum.
__device__ __forceinline__ float relu_drop(float k, float inv, float neg, float pos) {
  return fminf(fmaf(k, inv, neg), pos);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sum of `v` over the block; valid in thread 0.  `sh` holds >= 32 doubles.
__device__ __forceinline__ double block_sum(double v, double* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  const int nw = (blockDim.x + 31) >> 5;
  v = (threadIdx.x < nw) ? sh[threadIdx.x] : 0.0;
  if (w == 0) v = warp_sum(v);
  return v;
}

// ------------------------------------------------------------------------------------------
// Propagation  out = A~ x,  A~_ij = dinv_i dinv_j on the pattern of A + I (Problem 1).
// G lanes share one row; each lane owns the float4 columns lane, lane+G, .. of a block of
// G*V float4 columns; wider rows loop over column blocks.
// A lane group walks its stored entries one after the other, so a row of thousands of entries
// (row lengths follow a power law) would keep one warp busy long after the rest of the grid is
// done.  Rows longer than `long_len` are therefore not handled as rows: they come as `n_items`
// items {row, first entry, one past the last} (first in the grid), whose partial sums go to
// `scratch` (one padded row per item) and are added up, in item order, by k_spmm_long_rows.
// With ORDERED, rows are taken in the order `row_order` lists them (inside every community by falling
// length): where several rows share a warp (narrow operands) its lane groups then walk rows of about the
// same length and finish together (-20 % measured at 48 columns; at 256 columns, one row per warp, the
// scattered order costs 13 %, so the caller passes no order there).
// ------------------------------------------------------------------------------------------
template <int G, int V, int UN, bool ORDERED>
__global__ void __launch_bounds__(256)
k_spmm(const int* __restrict__ row_ptr, const int* __restrict__ col, const float* __restrict__ dinv,
       const float4* __restrict__ x, float4* __restrict__ out, int n, int ld4,
       const int4* __restrict__ items, int n_items, int long_len, float4* __restrict__ scratch,
       const int* __restrict__ row_order) {
  const int lane = threadIdx.x & 31;
  const int gl = lane & (G - 1);
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(G - 1)));
  const long long unit = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / G;
  if (unit >= (long long)n + n_items) return;
  long long row;
  int rs, re;
  float4* dst;
  if (unit < n_items) {
    const int4 it = items[unit];
    row = it.x; rs = it.y; re = it.z;
    dst = scratch + unit * ld4;
  } else {
    row = unit - n_items;
    if (ORDERED) row = row_order[row];
    rs = row_ptr[row]; re = row_ptr[row + 1];
    if (re - rs > long_len) return;
    dst = out + row * ld4;
  }
  const float di = dinv[row];
  for (int cb = 0; cb < ld4; cb += G * V) {
    float4 acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    // Narrow operands (several rows per warp): a chunk of G entries costs three dependent load latencies
    // (column, weight of that column, operand row) and moves little data, so the columns are fetched two
    // chunks ahead and their weights one chunk ahead.  (At one row per warp the same prefetch was measured
    // slower, and this kernel's load order is touchy there: the wide form keeps the plain loop.)
    constexpr bool kAhead = G < 32;
    int c_n = 0, c_n2 = 0;
    float w_n = 0.f;
    if (kAhead) {
      if (rs + gl < re) c_n = col[rs + gl];
      if (rs + G + gl < re) c_n2 = col[rs + G + gl];
      if (rs + gl < re) w_n = dinv[c_n];
    }
    for (int base = rs; base < re; base += G) {
      const int idx = base + gl;
      int c = 0;
      float w = 0.f;
      if (kAhead) {
        c = c_n; w = w_n;
        c_n = c_n2;
        c_n2 = (idx + 2 * G < re) ? col[idx + 2 * G] : 0;
        w_n = (idx + G < re) ? dinv[c_n] : 0.f;
      } else if (idx < re) { c = col[idx]; w = dinv[c]; }
      const int cnt = min(G, re - base);
      for (int t = 0; t < cnt; t += UN) {
        int cj[UN];
        float wj[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {   // lanes past the row's end hold (column 0, weight 0)
          cj[u] = __shfl_sync(gmask, c, (t + u) & (G - 1), G);
          wj[u] = __shfl_sync(gmask, w, (t + u) & (G - 1), G);
          if (t + u >= G) wj[u] = 0.f;
        }
#pragma unroll
        for (int v = 0; v < V; ++v) {
          const int f = cb + gl + G * v;
          if (f < ld4) {
            float4 xv[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) xv[u] = __ldg(x + (long long)cj[u] * ld4 + f);
#pragma unroll
            for (int u = 0; u < UN; ++u) {
              acc[v].x = fmaf(wj[u], xv[u].x, acc[v].x);
              acc[v].y = fmaf(wj[u], xv[u].y, acc[v].y);
              acc[v].z = fmaf(wj[u], xv[u].z, acc[v].z);
              acc[v].w = fmaf(wj[u], xv[u].w, acc[v].w);
            }
          }
        }
      }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const int f = cb + gl + G * v;
      if (f < ld4)
        dst[f] = make_float4(di * acc[v].x, di * acc[v].y, di * acc[v].z, di * acc[v].w);
    }
  }
}

// Rows that k_spmm handled as items: out[row] = sum of the row's item sums, in item order.
// rows[r] = {row, first item, number of items}; one block per row.
__global__ void k_spmm_long_rows(const int4* __restrict__ rows, const float4* __restrict__ scratch,
                                 float4* __restrict__ out, int ld4) {
  const int4 r = rows[blockIdx.x];
  for (int f = threadIdx.x; f < ld4; f += blockDim.x) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < r.z; ++k) {
      const float4 v = scratch[(long long)(r.y + k) * ld4 + f];
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    out[(long long)r.x * ld4 + f] = s;
  }
}

// ------------------------------------------------------------------------------------------
// Dense products.
//   k_gemm_nn : C[M x N] = A[M x K] B[K x N]          (H = P W, D = P grad, G = S W^T, T = G W)
//   k_gemm_tn : part[s][Ka x Nb] = sum over the rows of split s of A[r,:]^T B[r,:]   (grad = P^T R)
// fp32 FFMA register tiles; `skip`, when given, points at a flag that cancels the launch.
// ------------------------------------------------------------------------------------------
template <int BM, int BN, int BK, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), 2)
k_gemm_nn(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
          float* __restrict__ C, int ldc, int M, int N, int K, const int* __restrict__ skip) {
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int TX = BN / TN;
  constexpr int A_F4 = BM * BK / 4, B_F4 = BK * BN / 4;
  constexpr int A_PER = (A_F4 + NT - 1) / NT, B_PER = (B_F4 + NT - 1) / NT;
  constexpr int PAD = 4;
  static_assert(TN == 4 || TN == 8, "TN");
  static_assert(TM == 4 || TM == 8, "TM");
  if (skip != nullptr && *skip) return;
  __shared__ __align__(16) float As[2][BK][BM + PAD];
  __shared__ __align__(16) float Bs[2][BK][BN];
  const int tid = threadIdx.x;
  const int tx = tid % TX, ty = tid / TX;
  const long long row0 = (long long)blockIdx.x * BM;
  const int col0 = blockIdx.y * BN;

  float4 ra[A_PER], rb[B_PER];
  auto load_tiles = [&](int k0) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int f = tid + i * NT;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (f < A_F4) {
        const int r = f / (BK / 4), kq = (f % (BK / 4)) * 4;
        const long long gr = row0 + r;
        const int gk = k0 + kq;
        if (gr < M && gk < K) {
          v = *reinterpret_cast<const float4*>(A + gr * lda + gk);   // lda % 4 == 0, gk % 4 == 0
          if (gk + 1 >= K) v.y = 0.f;
          if (gk + 2 >= K) v.z = 0.f;
          if (gk + 3 >= K) v.w = 0.f;
        }
      }
      ra[i] = v;
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int f = tid + i * NT;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (f < B_F4) {
        const int kr = f / (BN / 4), c = (f % (BN / 4)) * 4;
        const int gk = k0 + kr, gc = col0 + c;
        if (gk < K && gc < N) {
          v = *reinterpret_cast<const float4*>(B + (long long)gk * ldb + gc);  // ldb % 4 == 0
          if (gc + 1 >= N) v.y = 0.f;
          if (gc + 2 >= N) v.z = 0.f;
          if (gc + 3 >= N) v.w = 0.f;
        }
      }
      rb[i] = v;
    }
  };
  auto store_tiles = [&](int buf) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int f = tid + i * NT;
      if (f < A_F4) {
        const int r = f / (BK / 4), kq = (f % (BK / 4)) * 4;
        As[buf][kq + 0][r] = ra[i].x;
        As[buf][kq + 1][r] = ra[i].y;
        As[buf][kq + 2][r] = ra[i].z;
        As[buf][kq + 3][r] = ra[i].w;
      }
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int f = tid + i * NT;
      if (f < B_F4) {
        const int kr = f / (BN / 4), c = (f % (BN / 4)) * 4;
        *reinterpret_cast<float4*>(&Bs[buf][kr][c]) = rb[i];
      }
    }
  };

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  load_tiles(0);
  store_tiles(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < K; k0 += BK) {
    const bool more = (k0 + BK) < K;
    if (more) load_tiles(k0 + BK);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[TM], b[TN];
#pragma unroll
      for (int i = 0; i < TM; i += 4) {
        const float4 v = *reinterpret_cast<const float4*>(&As[buf][k][ty * TM + i]);
        a[i] = v.x; a[i + 1] = v.y; a[i + 2] = v.z; a[i + 3] = v.w;
      }
      {
        const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
        b[0] = v.x; b[1] = v.y; b[2] = v.z; b[3] = v.w;
      }
      if constexpr (TN == 8) {
        const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][k][BN / 2 + tx * 4]);
        b[TN - 4] = v.x; b[TN - 3] = v.y; b[TN - 2] = v.z; b[TN - 1] = v.w;
      }
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) {
      store_tiles(buf ^ 1);
      __syncthreads();
      buf ^= 1;
    }
  }
  // columns N..ldc-1 (padding) receive the zeros accumulated from the masked B columns
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const long long gr = row0 + ty * TM + i;
    if (gr >= M) continue;
#pragma unroll
    for (int h = 0; h < TN / 4; ++h) {
      const int gc = col0 + (h == 0 ? tx * 4 : BN / 2 + tx * 4);
      if (gc < ldc)
        *reinterpret_cast<float4*>(C + gr * ldc + gc) =
            make_float4(acc[i][h * 4], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]);
    }
  }
}

// part[(split * Ka + ka) * ldp + nb].  A: rows x Ka (lda), B: rows x Nb (ldb).
// Split s owns rows [s * rows_per_split, min(rows, (s+1) * rows_per_split)).
template <int BM, int BN, int BK, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), 2)
k_gemm_tn(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
          float* __restrict__ part, int ldp, long long rows, long long rows_per_split, int Ka, int Nb) {
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int TX = BN / TN;
  constexpr int A_F4 = BK * BM / 4, B_F4 = BK * BN / 4;
  constexpr int A_PER = (A_F4 + NT - 1) / NT, B_PER = (B_F4 + NT - 1) / NT;
  static_assert(TM == 4 || TM == 8, "TM");
  static_assert(BN % 4 == 0, "BN");
  __shared__ __align__(16) float As[2][BK][BM];
  __shared__ __align__(16) float Bs[2][BK][BN];
  const int tid = threadIdx.x;
  const int tx = tid % TX, ty = tid / TX;
  const int a0 = blockIdx.x * BM, b0 = blockIdx.y * BN;
  const long long r_begin = (long long)blockIdx.z * rows_per_split;
  const long long r_end = min(rows, r_begin + rows_per_split);

  float4 ra[A_PER], rb[B_PER];
  auto load_tiles = [&](long long r0) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int f = tid + i * NT;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (f < A_F4) {
        const int rr = f / (BM / 4), c = (f % (BM / 4)) * 4;
        const long long gr = r0 + rr;
        const int gc = a0 + c;
        if (gr < r_end && gc < Ka) {
          v = *reinterpret_cast<const float4*>(A + gr * lda + gc);
          if (gc + 1 >= Ka) v.y = 0.f;
          if (gc + 2 >= Ka) v.z = 0.f;
          if (gc + 3 >= Ka) v.w = 0.f;
        }
      }
      ra[i] = v;
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int f = tid + i * NT;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (f < B_F4) {
        const int rr = f / (BN / 4), c = (f % (BN / 4)) * 4;
        const long long gr = r0 + rr;
        const int gc = b0 + c;
        if (gr < r_end && gc < Nb) {
          v = *reinterpret_cast<const float4*>(B + gr * ldb + gc);
          if (gc + 1 >= Nb) v.y = 0.f;
          if (gc + 2 >= Nb) v.z = 0.f;
          if (gc + 3 >= Nb) v.w = 0.f;
        }
      }
      rb[i] = v;
    }
  };
  auto store_tiles = [&](int buf) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int f = tid + i * NT;
      if (f < A_F4) *reinterpret_cast<float4*>(&As[buf][f / (BM / 4)][(f % (BM / 4)) * 4]) = ra[i];
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int f = tid + i * NT;
      if (f < B_F4) *reinterpret_cast<float4*>(&Bs[buf][f / (BN / 4)][(f % (BN / 4)) * 4]) = rb[i];
    }
  };

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  if (r_begin < r_end) {
    load_tiles(r_begin);
    store_tiles(0);
    __syncthreads();
    int buf = 0;
    for (long long r0 = r_begin; r0 < r_end; r0 += BK) {
      const bool more = (r0 + BK) < r_end;
      if (more) load_tiles(r0 + BK);
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float a[TM], b[TN];
        {
          const float4 v = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
          a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
        }
        if constexpr (TM == 8) {
          const float4 v = *reinterpret_cast<const float4*>(&As[buf][k][BM / 2 + ty * 4]);
          a[TM - 4] = v.x; a[TM - 3] = v.y; a[TM - 2] = v.z; a[TM - 1] = v.w;
        }
        if constexpr (TN >= 4) {
          const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
          b[0] = v.x; b[1] = v.y; b[2] = v.z; b[3] = v.w;
          if constexpr (TN == 8) {
            const float4 w = *reinterpret_cast<const float4*>(&Bs[buf][k][BN / 2 + tx * 4]);
            b[TN - 4] = w.x; b[TN - 3] = w.y; b[TN - 2] = w.z; b[TN - 1] = w.w;
          }
        } else {
#pragma unroll
          for (int j = 0; j < TN; ++j) b[j] = Bs[buf][k][tx * TN + j];
        }
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
      if (more) {
        store_tiles(buf ^ 1);
        __syncthreads();
        buf ^= 1;
      }
    }
  }
  float* dst = part + (long long)blockIdx.z * Ka * ldp;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int ga = a0 + ((TM == 8 && i >= 4) ? BM / 2 + ty * 4 + (i - 4) : ty * 4 + i);
    if (ga >= Ka) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int gb;
      if (TN == 8) gb = b0 + (j >= 4 ? BN / 2 + tx * 4 + (j - 4) : tx * 4 + j);
      else if (TN == 4) gb = b0 + tx * 4 + j;
      else gb = b0 + tx * TN + j;
      if (gb < ldp) dst[(long long)ga * ldp + gb] = acc[i][j];
    }
  }
}

// grad[e] = sum over splits of part[s][e], summed in fp64 in split order (fixed order).
__global__ void k_reduce_splits(const float* __restrict__ part, float* __restrict__ grad, long long elems,
                                int splits) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= elems) return;
  double s = 0.0;
  for (int k = 0; k < splits; ++k) s += (double)part[(long long)k * elems + e];
  grad[e] = (float)s;
}

// out[0] = sum a^2, out[1] = sum b^2 over `elems` floats (one block, fixed order).
__global__ void k_two_sumsq(const float* __restrict__ a, const float* __restrict__ b, long long elems,
                            double* __restrict__ out) {
  __shared__ double sh[32];
  double sa = 0.0, sb = 0.0;
  for (long long e = threadIdx.x; e < elems; e += blockDim.x) {
    const double x = a[e], y = b[e];
    sa += x * x;
    sb += y * y;
  }
  sa = block_sum(sa, sh);
  sb = block_sum(sb, sh);
  if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; }
}

// ------------------------------------------------------------------------------------------
// Residuals with respect to the pre-activation H (derivatives of phi, Section 3):
//   hidden layer  R = nu (f(H) - Z) * f'(H)
//   last layer    R = -(U + rho (Z - H))
// ------------------------------------------------------------------------------------------
__global__ void k_resid_hidden(const float4* __restrict__ H, const float4* __restrict__ Z,
                               float4* __restrict__ R, long long n4, float nu) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 h = H[i], z = Z[i];
    float4 r;
    r.x = h.x > 0.f ? nu * (h.x - z.x) : 0.f;
    r.y = h.y > 0.f ? nu * (h.y - z.y) : 0.f;
    r.z = h.z > 0.f ? nu * (h.z - z.z) : 0.f;
    r.w = h.w > 0.f ? nu * (h.w - z.w) : 0.f;
    R[i] = r;
  }
}

__global__ void k_resid_out(const float4* __restrict__ H, const float4* __restrict__ Z,
                            const float4* __restrict__ U, float4* __restrict__ R, long long n4, float rho) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 h = H[i], z = Z[i], u = U[i];
    float4 r;
    r.x = -(u.x + rho * (z.x - h.x));
    r.y = -(u.y + rho * (z.y - h.y));
    r.z = -(u.z + rho * (z.z - h.z));
    r.w = -(u.w + rho * (z.w - h.w));
    R[i] = r;
  }
}

// ------------------------------------------------------------------------------------------
// Step-size search of a W block (Section 3.1).  Along W - grad/t the pre-activation is
// H - D/t with D = P grad, so every candidate is scored from H, D, Z without another product.
// ------------------------------------------------------------------------------------------
// Every block leaves its sums in `partial` (kCand, resp. 2, doubles per block); k_search_decide_w adds the
// blocks up in a fixed order, so a decision does not depend on how the blocks were scheduled.
// hidden layer: sum_j = sum ( (z - f(h - d/t_j))^2 - (z - f(h))^2 )   (times nu/2 at decision time)
__global__ void __launch_bounds__(256)
k_score_w_hidden(const float4* __restrict__ H, const float4* __restrict__ D, const float4* __restrict__ Z,
                 long long n4, const SearchCtl* __restrict__ ctl, double* __restrict__ partial) {
  if (ctl->done) return;
  __shared__ double sh[32];
  float inv[kCand];
#pragma unroll
  for (int j = 0; j < kCand; ++j) inv[j] = ctl->inv_cand[j];
  double s[kCand];
#pragma unroll
  for (int j = 0; j < kCand; ++j) s[j] = 0.0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 h4 = H[i], d4 = D[i], z4 = Z[i];
    const float h[4] = {h4.x, h4.y, h4.z, h4.w}, d[4] = {d4.x, d4.y, d4.z, d4.w},
                z[4] = {z4.x, z4.y, z4.z, z4.w};
    float part[kCand];
#pragma unroll
    for (int j = 0; j < kCand; ++j) part[j] = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float pos = fmaxf(h[c], 0.f), neg = fmaxf(-h[c], 0.f);
      const float e2 = 2.f * (z[c] - pos);
#pragma unroll
      for (int j = 0; j < kCand; ++j) {
        const float df = relu_drop(d[c], inv[j], neg, pos);
        part[j] = fmaf(df, e2 + df, part[j]);   // e1^2 - e0^2 = (e1 - e0)(e1 + e0), e1 - e0 = df
      }
    }
#pragma unroll
    for (int j = 0; j < kCand; ++j) s[j] += (double)part[j];
  }
#pragma unroll
  for (int j = 0; j < kCand; ++j) {
    const double v = block_sum(s[j], sh);
    if (threadIdx.x == 0) partial[(size_t)blockIdx.x * kCand + j] = v;
  }
}

// last layer: phi_L(t) - phi_L = -(1/t) <D, R> + (rho / 2t^2) ||D||^2 ; sums <D,R> and ||D||^2
__global__ void __launch_bounds__(256)
k_score_w_out(const float4* __restrict__ D, const float4* __restrict__ R, long long n4,
              const SearchCtl* __restrict__ ctl, double* __restrict__ partial) {
  if (ctl->done) return;
  __shared__ double sh[32];
  double s1 = 0.0, s2 = 0.0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 d = D[i], r = R[i];
    s1 += (double)(d.x * r.x + d.y * r.y + d.z * r.z + d.w * r.w);
    s2 += (double)(d.x * d.x + d.y * d.y + d.z * d.z + d.w * d.w);
  }
  s1 = block_sum(s1, sh);
  s2 = block_sum(s2, sh);
  if (threadIdx.x == 0) { partial[(size_t)blockIdx.x * 2] = s1; partial[(size_t)blockIdx.x * 2 + 1] = s2; }
}

__device__ __forceinline__ void set_candidates(SearchCtl* c, double growth) {
  double t = c->t_base;
#pragma unroll
  for (int j = 0; j < kCand; ++j) { c->inv_cand[j] = (float)(1.0 / t); t *= growth; }
}

// Starts one search from ||grad||^2 and ||x||^2 of its block.
__device__ __forceinline__ void begin_one(SearchCtl* c, double gg, double xx, double shrink, double growth,
                                          int* __restrict__ n_active, int* __restrict__ status) {
  c->gg = gg;
  c->xx = xx;
  c->pass = 0;
  c->q = 0.0;
  c->inv_step = 0.f;
  if (!(c->gg > 1e-24 * c->xx)) {          // zero up to rounding (also catches NaN): skip
    c->done = 1;
    const bool finite = (c->gg == c->gg) && (c->xx == c->xx) && c->gg < 1.0e300 && c->xx < 1.0e300;
    c->trial = finite ? -1 : -2;
    if (!finite) atomicOr(status, 1);     // a NaN or an infinity reached the gradient or the block itself
    return;
  }
  c->done = 0;
  c->trial = -2;
  c->t_base = fmax(c->t_prev * shrink, 1e-12);
  set_candidates(c, growth);
  if (n_active) atomicAdd(n_active, 1);
}

// Starts the search of a W block: sums[0] = ||grad||^2, sums[1] = ||W||^2.
__global__ void k_search_begin(SearchCtl* ctl, const double* __restrict__ sums, double shrink, double growth,
                               int* __restrict__ status) {
  if (threadIdx.x == 0 && blockIdx.x == 0) begin_one(ctl, sums[0], sums[1], shrink, growth, nullptr, status);
}

// Starts the searches of the `count` communities of a hidden layer, one warp each.  k_zgrad_finish left
// three sums per row block in `partial`; the blocks of community i are block_ptr[i] .. block_ptr[i+1]-1
// and are added up in a fixed order (lane-strided, then the shuffle tree).  sums[i*3 + ..] receives
// { ||G_i||^2, ||Z_i||^2, <Z_i - f(H_i), G_i> }.
__global__ void k_search_begin_z(SearchCtl* ctl, int count, const double* __restrict__ partial,
                                 const int* __restrict__ block_ptr, double* __restrict__ sums, double shrink,
                                 double growth, int* __restrict__ n_active, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int i = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (i >= count) return;
  double s0 = 0.0, s1 = 0.0, s2 = 0.0;
  for (int b = block_ptr[i] + lane; b < block_ptr[i + 1]; b += 32) {
    s0 += partial[(size_t)b * 3]; s1 += partial[(size_t)b * 3 + 1]; s2 += partial[(size_t)b * 3 + 2];
  }
  s0 = warp_sum(s0); s1 = warp_sum(s1); s2 = warp_sum(s2);
  if (lane != 0) return;
  sums[i * 3] = s0; sums[i * 3 + 1] = s1; sums[i * 3 + 2] = s2;
  begin_one(ctl + i, s0, s1, shrink, growth, n_active, status);
}

// One decision per search.  mode 0: `cand` sums of a scoring pass, delta_j = scale * sum[j]
// plus the quadratic own term; mode 1: closed form, delta(t) = -lin/t + quad/t^2, all trials at once.
//   own term (Z blocks only): -(nu/t) sag + (nu/2t^2) sgg with sag = <Z - f(H), G>, sgg = gg
struct DecideArgs {
  double growth;
  int max_trials;
  int mode;          // 0 scored candidates, 1 closed form
  int cand;          // mode 0: candidates scored per pass (<= kCand)
  double scale;      // multiplies the scored sums (nu/2)
  double quad_coef;  // closed form: delta = -sum[0]/t + quad_coef * sum[1] / t^2
  double own_nu;     // nu when the block has a quadratic own term, else 0
  int last_pass;     // this is the final pass: mark exhausted searches
};

__device__ __forceinline__ bool accept(SearchCtl* c, double delta, double t, int trial) {
  const double need = c->gg / (2.0 * t);
  if (delta <= -need) {          // f(x+) - f(x) <= -||g||^2 / (2t); false for NaN
    c->t_prev = t;
    c->q = -delta / need;
    c->inv_step = (float)(1.0 / t);
    c->trial = trial;
    c->done = 1;
    return true;
  }
  return false;
}

// Decision of one open search from the sums of the pass just scored.  Returns true when the search
// goes on to another pass (its candidates are then already set).
__device__ __forceinline__ bool decide_one(SearchCtl* c, const double* __restrict__ sums, double sag,
                                           const DecideArgs& a, int* __restrict__ n_active,
                                           int* __restrict__ status) {
  if (a.mode == 1) {
    double t = c->t_base;
    const double lin = sums[0], quad = a.quad_coef * sums[1];
    bool ok = false;
    for (int trial = 0; trial < a.max_trials && !ok; ++trial) {
      const double delta = -lin / t + quad / (t * t) - a.own_nu * sag / t + 0.5 * a.own_nu * c->gg / (t * t);
      ok = accept(c, delta, t, trial);
      t *= a.growth;
    }
    if (!ok) { c->done = 1; c->trial = -2; c->inv_step = 0.f; if (!(lin == lin && quad == quad)) atomicOr(status, 1); }
    if (n_active) atomicSub(n_active, 1);
    return false;
  }
  double t = c->t_base;
  bool ok = false, finite = true;
  for (int j = 0; j < a.cand && !ok; ++j) {
    const int trial = c->pass * a.cand + j;
    if (trial >= a.max_trials) break;
    const double sum = sums[j];
    finite = finite && (sum == sum);
    const double delta = a.scale * sum - a.own_nu * sag / t + 0.5 * a.own_nu * c->gg / (t * t);
    ok = accept(c, delta, t, trial);
    t *= a.growth;
  }
  if (!finite) atomicOr(status, 1);
  if (ok) { if (n_active) atomicSub(n_active, 1); return false; }
  c->pass += 1;
  if (a.last_pass || c->pass * a.cand >= a.max_trials) {
    c->done = 1; c->trial = -2; c->inv_step = 0.f;
    if (n_active) atomicSub(n_active, 1);
    return false;
  }
  c->t_base = t;
  set_candidates(c, a.growth);
  return true;
}

// Sums of a scoring sweep, first stage: group g adds the chunks g*per_group .. (g+1)*per_group - 1 in chunk
// order, value by value (width = communities x sums per community): group_part[g][v] = sum_ch chunk_part[ch][v].
__global__ void k_reduce_chunks(const double* __restrict__ chunk_part, int n_chunks, int per_group, int width,
                                double* __restrict__ group_part, const int* __restrict__ n_active) {
  if (*n_active <= 0) return;
  const int c0 = blockIdx.x * per_group, c1 = min(n_chunks, c0 + per_group);
  for (int v = threadIdx.x; v < width; v += blockDim.x) {
    double s = 0.0;
    for (int ch = c0; ch < c1; ++ch) s += chunk_part[(size_t)ch * width + v];
    group_part[(size_t)blockIdx.x * width + v] = s;
  }
}

// Decisions of the `count` communities of a hidden layer, one warp each.  k_reduce_chunks left the sweep's
// sums in block_part[(b*count + i)*per + j], b < n_blocks; they are added in a fixed order (lane-strided
// over b, then the shuffle tree), together with the sums of the segments scored in pieces
// (split_scores, in the order split_order lists those of community i: split_ptr[i] .. split_ptr[i+1]-1).
// own[i*3 + 2] = <Z_i - f(H_i), G_i>.
__global__ void k_search_decide_z(SearchCtl* ctl, int count, const double* __restrict__ block_part, int n_blocks,
                                  int per, const double* __restrict__ split_scores,
                                  const int* __restrict__ split_order, const int* __restrict__ split_ptr,
                                  const double* __restrict__ own, DecideArgs a, int* __restrict__ n_active,
                                  int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int i = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (i >= count) return;
  SearchCtl* c = ctl + i;
  if (c->done) return;
  double s[kCand];
#pragma unroll
  for (int j = 0; j < kCand; ++j) s[j] = 0.0;
  for (int b = lane; b < n_blocks; b += 32)
#pragma unroll
    for (int j = 0; j < kCand; ++j)
      if (j < per) s[j] += block_part[((size_t)b * count + i) * per + j];
  for (int k = split_ptr[i] + lane; k < split_ptr[i + 1]; k += 32) {
    const size_t at = (size_t)split_order[k] * per;
#pragma unroll
    for (int j = 0; j < kCand; ++j)
      if (j < per) s[j] += split_scores[at + j];
  }
#pragma unroll
  for (int j = 0; j < kCand; ++j) s[j] = warp_sum(s[j]);
  if (lane != 0) return;
  decide_one(c, s, own[i * 3 + 2], a, n_active, status);
}

// Decision of a W block: the `n_part` blocks of the scoring kernel left `per` sums each in `partial`;
// they are added in a fixed order (thread-strided, then the block tree) before the decision is taken.
// One block of 256 threads.
__global__ void __launch_bounds__(256)
k_search_decide_w(SearchCtl* c, const double* __restrict__ partial, int n_part, int per, DecideArgs a,
                  int* __restrict__ status) {
  if (c->done) return;
  __shared__ double sh[32];
  __shared__ double total[kCand];
  for (int j = 0; j < per; ++j) {
    double s = 0.0;
    for (int b = threadIdx.x; b < n_part; b += blockDim.x) s += partial[(size_t)b * per + j];
    s = block_sum(s, sh);
    if (threadIdx.x == 0) total[j] = s;
  }
  if (threadIdx.x == 0) decide_one(c, total, 0.0, a, nullptr, status);
}

// The decision log is a ring of `ring` passes; the slot in use is *pass mod ring, with the pass counter
// kept on the device so that a recorded launch sequence stays valid from one pass to the next.
// Copies the decision of each search into the slot of the current pass.
__global__ void k_log_decisions(const SearchCtl* __restrict__ ctl, int count, int* __restrict__ trial_base,
                                double* __restrict__ q_base, const int* __restrict__ pass, long long per_pass,
                                long long offset, int ring) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const long long at = (long long)(*pass % ring) * per_pass + offset + i;
  trial_base[at] = ctl[i].trial;
  q_base[at] = ctl[i].q;
}

// Marks every entry of the current pass's slot as "not run".
__global__ void k_log_clear(int* __restrict__ trial_base, const int* __restrict__ pass, long long per_pass, int ring) {
  const long long at0 = (long long)(*pass % ring) * per_pass;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < per_pass;
       i += (long long)gridDim.x * blockDim.x)
    trial_base[at0 + i] = -3;
}

__global__ void k_pass_advance(int* __restrict__ pass) { *pass += 1; }

// W <- W - grad / tau (and its transpose copy), C_prev x C matrices with padded leading dimensions.
__global__ void k_apply_w(float* __restrict__ W, float* __restrict__ Wt, const float* __restrict__ grad,
                          int rows, int cols, int ldw, int ldwt, const SearchCtl* __restrict__ ctl) {
  const float s = ctl->inv_step;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * cols) return;
  const int r = e / cols, c = e % cols;
  const float w = fmaf(-grad[r * ldw + c], s, W[r * ldw + c]);
  W[r * ldw + c] = w;
  Wt[c * ldwt + r] = w;
}

// Y <- Y - s X with s = ctl->inv_step (H <- H - D/tau).
__global__ void k_axpy_ctl(float4* __restrict__ Y, const float4* __restrict__ X, long long n4,
                           const SearchCtl* __restrict__ ctl) {
  const float s = ctl->inv_step;
  if (s == 0.f) return;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    float4 y = Y[i];
    const float4 x = X[i];
    y.x = fmaf(-s, x.x, y.x); y.y = fmaf(-s, x.y, y.y); y.z = fmaf(-s, x.z, y.z); y.w = fmaf(-s, x.w, y.w);
    Y[i] = y;
  }
}

// ------------------------------------------------------------------------------------------
// Hidden Z blocks (Appendix A).  The gradient of psi_m with respect to Z_{l,m} is the rows V_m of
//   G = nu (Z_l - f(H_l)) + (A~ R') W_{l+1}^T ,
// R' the residual of layer l+1 at the new W.  k_zgrad_finish adds the first term to the product and
// leaves, per row block, partial[b*3 + ..] = { ||G||^2, ||Z_l||^2, <Z_l - f(H_l), G> } over the block's
// rows.  blocks[b] = {first row, one past the last}: a block never crosses a community boundary, so
// the sums of a community are the sums of its blocks, added in a fixed order by k_search_begin_z.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_zgrad_finish(float4* __restrict__ G, const float4* __restrict__ Z, const float4* __restrict__ H, int ld4,
               const int2* __restrict__ blocks, float nu, double* __restrict__ partial) {
  __shared__ double sh[32];
  const int2 rb = blocks[blockIdx.x];
  double sgg = 0.0, szz = 0.0, sag = 0.0;
  const long long e0 = (long long)rb.x * ld4, e1 = (long long)rb.y * ld4;
  for (long long e = e0 + threadIdx.x; e < e1; e += blockDim.x) {
    const float4 z = Z[e], h = H[e];
    float4 g = G[e];
    const float ax = z.x - relu(h.x), ay = z.y - relu(h.y), az = z.z - relu(h.z), aw = z.w - relu(h.w);
    g.x = fmaf(nu, ax, g.x); g.y = fmaf(nu, ay, g.y); g.z = fmaf(nu, az, g.z); g.w = fmaf(nu, aw, g.w);
    G[e] = g;
    sgg += (double)(g.x * g.x + g.y * g.y + g.z * g.z + g.w * g.w);
    szz += (double)(z.x * z.x + z.y * z.y + z.z * z.z + z.w * z.w);
    sag += (double)(ax * g.x + ay * g.y + az * g.z + aw * g.w);
  }
  sgg = block_sum(sgg, sh); szz = block_sum(szz, sh); sag = block_sum(sag, sh);
  if (threadIdx.x == 0) {
    partial[(size_t)blockIdx.x * 3] = sgg; partial[(size_t)blockIdx.x * 3 + 1] = szz; partial[(size_t)blockIdx.x * 3 + 2] = sag;
  }
}

// Warp-wide sums of 4 (or 2) per-lane values with 6 (5) shuffles: lane 8*j (16*j) ends up holding
// the total of value j.
__device__ __forceinline__ float warp_sum4(float v0, float v1, float v2, float v3, int lane) {
  const bool up16 = lane & 16, up8 = lane & 8;
  const float r0 = __shfl_xor_sync(0xffffffffu, up16 ? v0 : v2, 16);
  const float r1 = __shfl_xor_sync(0xffffffffu, up16 ? v1 : v3, 16);
  const float a = (up16 ? v2 : v0) + r0, b = (up16 ? v3 : v1) + r1;
  float c = (up8 ? b : a) + __shfl_xor_sync(0xffffffffu, up8 ? a : b, 8);
  c += __shfl_xor_sync(0xffffffffu, c, 4);
  c += __shfl_xor_sync(0xffffffffu, c, 2);
  c += __shfl_xor_sync(0xffffffffu, c, 1);
  return c;
}
__device__ __forceinline__ float warp_sum2(float v0, float v1, int lane) {
  const bool up16 = lane & 16;
  float c = (up16 ? v1 : v0) + __shfl_xor_sync(0xffffffffu, up16 ? v0 : v1, 16);
  c += __shfl_xor_sync(0xffffffffu, c, 8);
  c += __shfl_xor_sync(0xffffffffu, c, 4);
  c += __shfl_xor_sync(0xffffffffu, c, 2);
  c += __shfl_xor_sync(0xffffffffu, c, 1);
  return c;
}

// Scoring of the theta candidates of every community in one sweep over the rows.
// With T = G W_{l+1}, the move of community m changes the pre-activation of row i by
//   -K_m[i] / theta_m ,  K_m[i] = sum over j in V_m of A~_ij T_j  (row i of A~_{comm(i),m} T_m),
// which is non-zero on V_m and its first-order neighbour rows only.  A warp owns row i and walks
// its stored entries once; col_comm gives the community of every entry, entries of one community
// are contiguous (ascending columns), and at every change of community the finished K_m[i] is scored:
//   OUT = false (layer l+1 < L, ReLU):  per community, sum_c (z - f(h - k/t_j))^2 - (z - f(h))^2 for j < NC
//                                        (NC = candidates scored per sweep, 2..4: a candidate costs two
//                                        instructions per element, and a search that needs more trials
//                                        than one sweep scores is served by a further sweep)
//   OUT = true  (layer l+1 = L):        sums <k, R'> and ||k||^2 per community   (closed form)
// Sums are kept per warp in shared memory (no atomics on the hot path) and leave the kernel per chunk of
// units (see the scheduling note in the kernel).  V = float4 columns per lane (width <= 128 V).
// Persistent grid.
//
// Rows longer than `long_len` come as `n_items` items {row, first entry, one past the last, split}
// (see k_spmm): an item of whole community segments (split < 0) is scored like a short row; an
// item that is one piece of a segment too long for one warp only leaves its part of K_m[i],
// unscaled, in `scratch` (one padded row per item), and k_score_z_split scores the sum of the pieces.

// 2 (z - f(h)): twice the row's current error, formed once per row and reused by every segment.
__device__ __forceinline__ float4 twice_error(const float4& h, const float4& z) {
  return make_float4(2.f * (z.x - relu(h.x)), 2.f * (z.y - relu(h.y)), 2.f * (z.z - relu(h.z)), 2.f * (z.w - relu(h.w)));
}

// Scores one finished K_m[i] (k, still without the factor di) against the row's a, b:
// OUT: a = R'; else a = h and b = twice_error(h, z).  The sums (2 when OUT, else NC) go to `slots`:
// how = 0 added by plain stores (the slots belong to this warp), 1 added atomically, 2 stored.
__device__ __forceinline__ void put_sum(double* dst, float r, int how) {
  if (how == 0) *dst += (double)r;
  else if (how == 1) atomicAdd(dst, (double)r);
  else *dst = (double)r;
}
template <int V, bool OUT, int NC>
__device__ __forceinline__ void score_segment(const float4 (&k)[V], float di, const float4 (&a)[V],
                                              const float4 (&b)[V], const SearchCtl* __restrict__ ctl,
                                              int cur, int lane, double* slots, int how) {
  if (OUT) {
    float p1 = 0.f, p2 = 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const float kx = di * k[v].x, ky = di * k[v].y, kz = di * k[v].z, kw = di * k[v].w;
      p1 += kx * a[v].x + ky * a[v].y + kz * a[v].z + kw * a[v].w;
      p2 += kx * kx + ky * ky + kz * kz + kw * kw;
    }
    const float r = warp_sum2(p1, p2, lane);
    if ((lane & 15) == 0) put_sum(slots + (lane >> 4), r, how);
  } else {
    static_assert(NC >= 2 && NC <= 4, "two to four candidates per sweep");
    float inv[NC], part[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) { inv[j] = di * ctl[cur].inv_cand[j]; part[j] = 0.f; }   // K_m[i] = di * k
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const float kk[4] = {k[v].x, k[v].y, k[v].z, k[v].w};
      const float hh[4] = {a[v].x, a[v].y, a[v].z, a[v].w};
      const float ee[4] = {b[v].x, b[v].y, b[v].z, b[v].w};   // 2 (z - f(h)), see twice_error
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float pos = fmaxf(hh[c], 0.f), neg = fmaxf(-hh[c], 0.f);
#pragma unroll
        for (int j = 0; j < NC; ++j) {
          const float df = relu_drop(kk[c], inv[j], neg, pos);
          part[j] = fmaf(df, ee[c] + df, part[j]);   // e1^2 - e0^2 = df (2 e0 + df)
        }
      }
    }
    if constexpr (NC >= 3) {
      const float r = warp_sum4(part[0], part[1], part[2], NC == 4 ? part[NC - 1] : 0.f, lane);
      if ((lane & 7) == 0 && (lane >> 3) < NC) put_sum(slots + (lane >> 3), r, how);
    } else {
      const float r = warp_sum2(part[0], part[1], lane);
      if ((lane & 15) == 0) put_sum(slots + (lane >> 4), r, how);
    }
  }
}

template <int V, bool OUT, int UN, int NC>
__global__ void __launch_bounds__(256, (V <= 1 ? 4 : V <= 2 ? 3 : 1))
k_score_z(const int* __restrict__ row_ptr, const int* __restrict__ col,
          const unsigned short* __restrict__ col_comm, const float* __restrict__ dinv,
          const float4* __restrict__ T, const float4* __restrict__ Hn, const float4* __restrict__ Zn,
          const float4* __restrict__ Rn, int ld4, int n, const SearchCtl* __restrict__ ctl, int n_comm,
          double* __restrict__ chunk_part, const int* __restrict__ n_active, int use_smem,
          const int* __restrict__ chunk_ptr, int n_chunks, int* __restrict__ chunk_counter,
          const int4* __restrict__ items, int n_items, int long_len, float4* __restrict__ scratch,
          const int* __restrict__ row_order) {
  if (*n_active <= 0) return;
  constexpr int PER = OUT ? 2 : NC;
  // dynamic shared memory: per warp the row's a, b (2 V float4 per lane; parked there during the
  // walk so that the registers hold gathered rows instead), then the per-warp sums
  extern __shared__ float4 s_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_per_block = blockDim.x >> 5;
  float4* row_ab = s_raw + (size_t)warp * (2 * V * 32) + lane;
  double* s_acc = reinterpret_cast<double*>(s_raw + (size_t)warps_per_block * (2 * V * 32));
  double* mine = nullptr;   // the sums of the chunk in hand, [community][PER]
  if (use_smem) {
    for (int i = threadIdx.x; i < warps_per_block * n_comm * PER; i += blockDim.x) s_acc[i] = 0.0;
    mine = s_acc + (size_t)warp * n_comm * PER;
  }
  __syncthreads();
  const float4* __restrict__ T_lane = T + lane;   // rows of T are addressed by 32-bit float4 offsets (n * ld4 < 2^32)
  bool in_row[V];
#pragma unroll
  for (int v = 0; v < V; ++v) in_row[v] = lane + 32 * v < ld4;
  // Units (items first, then rows) come in chunks of about equally many stored entries (chunk_ptr, built
  // on the host).  Chunks are handed out from a global counter (`chunk_counter`, zero at launch): row
  // lengths follow a power law and the time a chunk takes depends on what its rows find in L2, so any
  // static deal leaves most warps waiting for the unlucky ones.  A chunk is scored by one warp, units in
  // order, and its sums go to chunk_part[chunk][community][PER]; they are added up in chunk order
  // afterwards (k_reduce_chunks, k_search_decide_z), so no sum depends on which warp took which chunk.
  // With room in shared memory the chunk's sums are kept there and copied out at the end of the chunk;
  // otherwise (too many communities) the warp adds into the chunk's slice of chunk_part directly.
  for (;;) {
    int ch = 0;
    if (lane == 0) ch = atomicAdd(chunk_counter, 1);
    ch = __shfl_sync(0xffffffffu, ch, 0);
    if (ch >= n_chunks) break;
    double* const out_part = chunk_part + (size_t)ch * n_comm * PER;
    if (!use_smem) {
      for (int i = lane; i < n_comm * PER; i += 32) out_part[i] = 0.0;
      mine = out_part;
      __syncwarp();
    }
    const int chunk_end = chunk_ptr[ch + 1];
  for (int unit_base = chunk_ptr[ch]; unit_base < chunk_end; unit_base += 4) {
    const int unit_end = min(chunk_end, unit_base + 4);
    // lanes 0..3 fetch the descriptions of the four units together (one load latency, not four)
    int4 my_unit = make_int4(0, 0, 0, -1);   // row, first entry, one past the last, split (>= 0: a piece)
    if (lane < 4 && unit_base + lane < unit_end) {
      const int u = unit_base + lane;
      if (u < n_items) my_unit = items[u];
      else {
        const int r = row_order != nullptr ? row_order[u - n_items] : u - n_items;
        my_unit = make_int4(r, row_ptr[r], row_ptr[r + 1], -1);
        if (my_unit.z - my_unit.y > long_len) my_unit.z = my_unit.y;   // walked as items
      }
    }
    // column and community of a unit's first chunk are fetched while the unit before it is walked
    int c_first = 0, m_first = -1;
    {
      const int s0 = __shfl_sync(0xffffffffu, my_unit.y, 0), e0 = __shfl_sync(0xffffffffu, my_unit.z, 0);
      if (s0 + lane < e0) { c_first = col[s0 + lane]; m_first = col_comm[s0 + lane]; }
    }
  for (int unit = unit_base; unit < unit_end; ++unit) {
    const int q = unit - unit_base;
    const int row = __shfl_sync(0xffffffffu, my_unit.x, q);
    const int rs = __shfl_sync(0xffffffffu, my_unit.y, q), re = __shfl_sync(0xffffffffu, my_unit.z, q);
    const bool piece = __shfl_sync(0xffffffffu, my_unit.w, q) >= 0;
    int c_next = c_first, m_next = m_first;
    {
      const int s1 = __shfl_sync(0xffffffffu, my_unit.y, (q + 1) & 3), e1 = __shfl_sync(0xffffffffu, my_unit.z, (q + 1) & 3);
      m_first = -1;
      if (q + 1 < unit_end - unit_base && s1 + lane < e1) { c_first = col[s1 + lane]; m_first = col_comm[s1 + lane]; }
    }
    if (rs >= re) continue;
    __syncwarp();          // the previous unit's last segment has been scored
#pragma unroll
    for (int v = 0; v < V; ++v) {   // OUT: a = R' ; else a = h, b = 2 (z - f(h))
      const int f = lane + 32 * v;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (f < ld4 && !piece) {
        if (OUT) a = Rn[(long long)row * ld4 + f];
        else { a = Hn[(long long)row * ld4 + f]; b = twice_error(a, Zn[(long long)row * ld4 + f]); }
      }
      row_ab[32 * v] = a;
      if (!OUT) row_ab[32 * (V + v)] = b;
    }
    const float di = dinv[row];
    float4 k[V];
#pragma unroll
    for (int v = 0; v < V; ++v) k[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    int cur = -1;          // community of the segment being accumulated
    bool cur_on = false;   // its search is still running

    auto finish_segment = [&]() {
      if (!cur_on) return;
      if (piece) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
          const int f = lane + 32 * v;
          if (f < ld4) scratch[(long long)unit * ld4 + f] = k[v];
        }
        return;
      }
      float4 a[V], b[V];   // each lane reads back what it stored itself
#pragma unroll
      for (int v = 0; v < V; ++v) {
        a[v] = row_ab[32 * v];
        b[v] = OUT ? a[v] : row_ab[32 * (V + v)];
      }
      score_segment<V, OUT, NC>(k, di, a, b, ctl, cur, lane, mine + cur * PER, 0);
    };

    // column and community of a chunk are fetched while the chunk before it is walked; the two
    // loads that depend on them (weight, search state) are issued together, not one after the other
    for (int base = rs; base < re; base += 32) {
      const int idx = base + lane;
      const bool valid = idx < re;
      const int c = c_next, m = m_next;
      if (idx + 32 < re) { c_next = col[idx + 32]; m_next = col_comm[idx + 32]; }
      else m_next = -1;
      unsigned off = 0u;      // first float4 of the entry's row of T; lanes past the row's end hold (row 0, weight 0)
      float w = 0.f;
      bool live = false;      // the entry's community is still searching: its row of T is gathered
      if (valid) {
        const float wc = dinv[c];
        live = !ctl[m].done;
        if (live) { w = wc; off = (unsigned)c * (unsigned)ld4; }
      }
      // entries of one community are contiguous: bit t of `chg` says that entry t opens a new
      // segment, bit t of `on` that its row is gathered; both are the same in every lane, so the
      // walk below needs the community of an entry only where a segment starts
      int mprev = __shfl_up_sync(0xffffffffu, m, 1);
      if (lane == 0) mprev = cur;
      unsigned chg = __ballot_sync(0xffffffffu, valid && m != mprev);
      unsigned on = __ballot_sync(0xffffffffu, live);
      const int cnt = min(32, re - base);
      if (on == 0u) {   // nothing to gather in this chunk (the usual case in a sweep after the first)
        if (chg != 0u) {   // an open segment ends at the chunk's first entry; a later one starts from scratch
          finish_segment();
          cur = __shfl_sync(0xffffffffu, m, cnt - 1);
          cur_on = false;
        }
        continue;
      }
      for (int t = 0; t < cnt; t += UN, chg >>= UN, on >>= UN) {
        unsigned oj[UN];
        float wj[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
          oj[u] = __shfl_sync(0xffffffffu, off, t + u);
          wj[u] = __shfl_sync(0xffffffffu, w, t + u);
        }
        float4 xv[UN][V];   // set and read under the same condition (entry gathered, column inside the row)
#pragma unroll
        for (int u = 0; u < UN; ++u)
#pragma unroll
          for (int v = 0; v < V; ++v)
            if (((on >> u) & 1u) && in_row[v]) xv[u][v] = __ldg(T_lane + oj[u] + 32 * v);
#pragma unroll
        for (int u = 0; u < UN; ++u) {
          if ((chg >> u) & 1u) {                          // warp-uniform
            finish_segment();
            cur = __shfl_sync(0xffffffffu, m, t + u);
            cur_on = (on >> u) & 1u;
#pragma unroll
            for (int v = 0; v < V; ++v) k[v] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int v = 0; v < V; ++v)
            if (((on >> u) & 1u) && in_row[v]) {
              k[v].x = fmaf(wj[u], xv[u][v].x, k[v].x); k[v].y = fmaf(wj[u], xv[u][v].y, k[v].y);
              k[v].z = fmaf(wj[u], xv[u][v].z, k[v].z); k[v].w = fmaf(wj[u], xv[u][v].w, k[v].w);
            }
        }
      }
    }
    finish_segment();
  }
  }
    __syncwarp();
    if (use_smem)
      for (int i = lane; i < n_comm * PER; i += 32) { out_part[i] = mine[i]; mine[i] = 0.0; }
    __syncwarp();
  }
}

// The output-layer form of k_score_z (OUT = true) for rows of at most 16 float4 (C_L <= 64), two
// units per warp: each half-warp walks its own row or item, 16 stored entries per chunk.  With 12 of
// 32 lanes carrying columns (47 classes) the full-warp form spends most of its issue slots on lanes
// that hold nothing; here every instruction of the walk serves two rows.  Control flow is kept the
// same for both halves (loop bounds are the larger of the two, a half that has run out holds weight 0
// and no segment start), shuffles use width 16, and only the closing of a segment is a divergent
// branch, inside which nothing is exchanged beyond the half's own 16 lanes.  Sums go to one array
// per half-warp (the halves may close segments of the same community at the same time).
// Dynamic shared memory: 2 x warps x n_comm x 2 doubles (the caller uses k_score_z when that does not fit).
template <int UN>
__global__ void __launch_bounds__(256, 4)
k_score_z_out_half(const int* __restrict__ row_ptr, const int* __restrict__ col,
                   const unsigned short* __restrict__ col_comm, const float* __restrict__ dinv,
                   const float4* __restrict__ T, const float4* __restrict__ Rn, int ld4, int n,
                   const SearchCtl* __restrict__ ctl, int n_comm, double* __restrict__ chunk_part,
                   const int* __restrict__ n_active, const int* __restrict__ chunk_ptr, int n_chunks,
                   int* __restrict__ chunk_counter,
                   const int4* __restrict__ items, int n_items, int long_len, float4* __restrict__ scratch,
                   const int* __restrict__ row_order) {
  if (*n_active <= 0) return;
  static_assert(16 % UN == 0, "UN divides the chunk");
  extern __shared__ double s_half[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, half = lane >> 4, hl = lane & 15;
  const int warps_per_block = blockDim.x >> 5;
  const unsigned hmask = 0xffffu << (16 * half);
  for (int i = threadIdx.x; i < 2 * warps_per_block * n_comm * 2; i += blockDim.x) s_half[i] = 0.0;
  double* const mine = s_half + (size_t)(2 * warp + half) * n_comm * 2;   // the half-warp's sums of the chunk in hand
  __syncthreads();
  const bool in_row = hl < ld4;
  const float4* __restrict__ T_lane = T + hl;
  for (;;) {   // chunks from a global counter, their sums to chunk_part: see k_score_z
    int ch = 0;
    if (lane == 0) ch = atomicAdd(chunk_counter, 1);
    ch = __shfl_sync(0xffffffffu, ch, 0);
    if (ch >= n_chunks) break;
    const int chunk_end = chunk_ptr[ch + 1];
  for (int unit_base = chunk_ptr[ch]; unit_base < chunk_end; unit_base += 4) {
    for (int pair = 0; pair < 2; ++pair) {
      const int unit = unit_base + 2 * pair + half;
      int row = 0, rs = 0, re = 0;
      bool piece = false;
      if (unit < chunk_end) {
        if (unit < n_items) {
          const int4 it = items[unit];
          row = it.x; rs = it.y; re = it.z;
          piece = it.w >= 0;
        } else {
          row = row_order[unit - n_items];
          rs = row_ptr[row]; re = row_ptr[row + 1];
          if (re - rs > long_len) re = rs;          // walked as items
        }
      }
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      if (in_row && !piece && re > rs) a = Rn[(long long)row * ld4 + hl];
      const float di = dinv[row];
      float4 k = make_float4(0.f, 0.f, 0.f, 0.f);
      int cur = -1;
      bool cur_on = false;

      auto finish_segment = [&]() {   // called by one half at a time: exchanges stay inside hmask
        if (!cur_on) return;
        if (piece) {
          if (in_row) scratch[(long long)unit * ld4 + hl] = k;
          return;
        }
        const float kx = di * k.x, ky = di * k.y, kz = di * k.z, kw = di * k.w;
        const float p1 = kx * a.x + ky * a.y + kz * a.z + kw * a.w;
        const float p2 = kx * kx + ky * ky + kz * kz + kw * kw;
        const bool up8 = hl & 8;
        float c = (up8 ? p2 : p1) + __shfl_xor_sync(hmask, up8 ? p1 : p2, 8, 16);
        c += __shfl_xor_sync(hmask, c, 4, 16);
        c += __shfl_xor_sync(hmask, c, 2, 16);
        c += __shfl_xor_sync(hmask, c, 1, 16);
        if ((hl & 7) == 0) put_sum(mine + cur * 2 + (hl >> 3), c, 0);
      };

      const int len = re - rs;
      const int len_max = max(len, __shfl_xor_sync(0xffffffffu, len, 16));
      int c_next = 0, m_next = -1;   // fetched one chunk ahead, as in k_score_z
      if (rs + hl < re) { c_next = col[rs + hl]; m_next = col_comm[rs + hl]; }
      for (int o = 0; o < len_max; o += 16) {
        const int idx = rs + o + hl;
        const bool valid = idx < re;
        const int c = c_next, m = m_next;
        if (idx + 16 < re) { c_next = col[idx + 16]; m_next = col_comm[idx + 16]; }
        else m_next = -1;
        unsigned off = 0u;
        float w = 0.f;
        bool live = false;
        if (valid) {
          const float wc = dinv[c];
          live = !ctl[m].done;
          if (live) { w = wc; off = (unsigned)c * (unsigned)ld4; }
        }
        int mprev = __shfl_up_sync(0xffffffffu, m, 1, 16);
        if (hl == 0) mprev = cur;
        unsigned chg = (__ballot_sync(0xffffffffu, valid && m != mprev) >> (16 * half)) & 0xffffu;
        const unsigned on_both = __ballot_sync(0xffffffffu, live);
        unsigned on = (on_both >> (16 * half)) & 0xffffu;
        const int cnt_max = min(16, len_max - o);
        if (on_both == 0u) {   // neither half has anything to gather in this chunk
          if (chg != 0u) {     // per half: an open segment ends at the chunk's first entry
            finish_segment();
            cur = __shfl_sync(hmask, m, min(16, len - o) - 1, 16);
            cur_on = false;
          }
          continue;
        }
        for (int t = 0; t < cnt_max; t += UN, chg >>= UN, on >>= UN) {
          unsigned oj[UN];
          float wj[UN];
#pragma unroll
          for (int u = 0; u < UN; ++u) {
            oj[u] = __shfl_sync(0xffffffffu, off, t + u, 16);
            wj[u] = __shfl_sync(0xffffffffu, w, t + u, 16);
          }
          float4 xv[UN];   // set and read under the same condition
#pragma unroll
          for (int u = 0; u < UN; ++u)
            if (((on >> u) & 1u) && in_row) xv[u] = __ldg(T_lane + oj[u]);
#pragma unroll
          for (int u = 0; u < UN; ++u) {
            if ((chg >> u) & 1u) {                        // uniform within the half
              finish_segment();
              cur = col_comm[rs + o + t + u];
              cur_on = (on >> u) & 1u;
              k = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (((on >> u) & 1u) && in_row) {
              k.x = fmaf(wj[u], xv[u].x, k.x); k.y = fmaf(wj[u], xv[u].y, k.y);
              k.z = fmaf(wj[u], xv[u].z, k.z); k.w = fmaf(wj[u], xv[u].w, k.w);
            }
          }
        }
      }
      finish_segment();
      __syncwarp();
    }
  }
    // the chunk's sums: lower half-warp first, then the upper one
    double* const lo = s_half + (size_t)(2 * warp) * n_comm * 2;
    double* const hi = lo + (size_t)n_comm * 2;
    double* const out_part = chunk_part + (size_t)ch * n_comm * 2;
    for (int i = lane; i < n_comm * 2; i += 32) { out_part[i] = lo[i] + hi[i]; lo[i] = 0.0; hi[i] = 0.0; }
    __syncwarp();
  }
}

// Segments that k_score_z handled in pieces: K_m[i] = sum of the pieces (item order), then scored
// as above.  split[s] = {row, community, first item, number of items}; one warp per entry, whose sums
// go to split_scores[s*PER ..] (PER = 2 when OUT, else NC); k_search_decide_z adds them in table order.
template <int V, bool OUT, int NC>
__global__ void __launch_bounds__(256)
k_score_z_split(const int4* __restrict__ split, int n_split, const float* __restrict__ dinv,
                const float4* __restrict__ scratch, const float4* __restrict__ Hn, const float4* __restrict__ Zn,
                const float4* __restrict__ Rn, int ld4, const SearchCtl* __restrict__ ctl,
                double* __restrict__ split_scores, const int* __restrict__ n_active) {
  if (*n_active <= 0) return;
  const int lane = threadIdx.x & 31;
  const int s = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (s >= n_split) return;
  const int4 sp = split[s];
  if (ctl[sp.y].done) return;
  float4 a[V], b[V], k[V];
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int f = lane + 32 * v;
    a[v] = b[v] = k[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (f < ld4) {
      if (OUT) a[v] = Rn[(long long)sp.x * ld4 + f];
      else { a[v] = Hn[(long long)sp.x * ld4 + f]; b[v] = twice_error(a[v], Zn[(long long)sp.x * ld4 + f]); }
      for (int q = 0; q < sp.w; ++q) {
        const float4 t = scratch[(long long)(sp.z + q) * ld4 + f];
        k[v].x += t.x; k[v].y += t.y; k[v].z += t.z; k[v].w += t.w;
      }
    }
  }
  score_segment<V, OUT, NC>(k, dinv[sp.x], a, b, ctl, sp.y, lane, split_scores + (size_t)s * (OUT ? 2 : NC), 2);
}

// The rows of Eq. 7 without a loss term (not in the training set) have the closed form
// z = q - u / rho; with dual_now, U <- u + rho (z_old - q) first (Eq. 3 as printed).  Plain
// elementwise sweep; training rows are skipped (k_output_rows visits them).
__global__ void k_output_plain(float4* __restrict__ ZL, float4* __restrict__ U, const float4* __restrict__ HL, int ld4,
                               long long n, const unsigned char* __restrict__ train, float rho, int dual_now,
                               int update_z) {
  const long long total = n * ld4;
  const float inv_rho = 1.f / rho;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    if (train[e / ld4]) continue;
    const float4 q = HL[e], u = U[e];
    if (dual_now) {
      const float4 z = ZL[e];
      U[e] = make_float4(fmaf(rho, z.x - q.x, u.x), fmaf(rho, z.y - q.y, u.y), fmaf(rho, z.z - q.z, u.z),
                         fmaf(rho, z.w - q.w, u.w));
    }
    if (update_z)
      ZL[e] = make_float4(fmaf(-u.x, inv_rho, q.x), fmaf(-u.y, inv_rho, q.y), fmaf(-u.z, inv_rho, q.z),
                          fmaf(-u.w, inv_rho, q.w));
  }
}

// Z_l[i,:] <- Z_l[i,:] - G[i,:] / theta_{comm(i)}   (Eq. 10)
__global__ void k_apply_z(float4* __restrict__ Z, const float4* __restrict__ G, int ld4, long long n,
                          const int* __restrict__ row_comm, const SearchCtl* __restrict__ ctl) {
  const long long total = n * ld4;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const float s = ctl[row_comm[e / ld4]].inv_step;
    if (s == 0.f) continue;
    float4 z = Z[e];
    const float4 g = G[e];
    z.x = fmaf(-s, g.x, z.x); z.y = fmaf(-s, g.y, z.y); z.z = fmaf(-s, g.z, z.z); z.w = fmaf(-s, g.w, z.w);
    Z[e] = z;
  }
}

// ------------------------------------------------------------------------------------------
// Output layer rows (Eq. 7) and the dual (Eq. 3), one warp per row, classes spread over lanes.
//   q = row of A~ Z_{L-1}^k W_L^{k+1};  training rows: FISTA on
//   loss_scale * CE(z, y) + <u, z - q> + (rho/2)||z - q||^2 ;  other rows: z = q - u / rho.
//   dual_now != 0: U <- u + rho (z_old - q) in the same sweep (Eq. 3 as printed).
// `rows` (may be NULL = every row) lists the rows to visit: the training rows, when the rest is
// left to k_output_plain.  CPL = classes per lane (C <= 32 CPL).  momentum[j] = (t_j - 1) / t_{j+1}
// of FISTA's sequence t_1 = 1, t_{j+1} = (1 + sqrt(1 + 4 t_j^2)) / 2: the same for every row, so it
// is tabulated once (in fp64) instead of being recomputed by every lane in every iteration.
// ------------------------------------------------------------------------------------------
template <int CPL>
__global__ void __launch_bounds__(256)
k_output_rows(float* __restrict__ ZL, float* __restrict__ U, const float* __restrict__ HL, int ld, int C,
              int n, const int* __restrict__ y, const unsigned char* __restrict__ train, float rho,
              float loss_scale, int iters, int dual_now, int update_z, const int* __restrict__ rows,
              const float* __restrict__ momentum) {
  const int lane = threadIdx.x & 31;
  const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (slot >= n) return;
  const int row = rows != nullptr ? rows[slot] : slot;
  float q[CPL], u[CPL], z[CPL];
  const long long base = (long long)row * ld;
#pragma unroll
  for (int t = 0; t < CPL; ++t) {
    const int c = lane + 32 * t;
    q[t] = u[t] = z[t] = 0.f;
    if (c < C) { q[t] = HL[base + c]; u[t] = U[base + c]; z[t] = ZL[base + c]; }
  }
  if (dual_now) {
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      const int c = lane + 32 * t;
      if (c < C) U[base + c] = fmaf(rho, z[t] - q[t], u[t]);
    }
  }
  if (!update_z) return;
  if (!train[row]) {
    const float inv_rho = 1.f / rho;
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      const int c = lane + 32 * t;
      if (c < C) ZL[base + c] = fmaf(-u[t], inv_rho, q[t]);
    }
    return;
  }
  const int yi = y[row];
  const float step = 1.f / (0.5f * loss_scale + rho);
  float xp[CPL], v[CPL];
#pragma unroll
  for (int t = 0; t < CPL; ++t) { xp[t] = z[t]; v[t] = z[t]; }
  for (int it = 0; it < iters; ++it) {
    float mx = -3.0e38f;
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (lane + 32 * t < C) mx = fmaxf(mx, v[t]);
    mx = warp_max(mx);
    float ex[CPL], se = 0.f;
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      ex[t] = (lane + 32 * t < C) ? expf(v[t] - mx) : 0.f;
      se += ex[t];
    }
    se = warp_sum(se);
    const float inv_se = 1.f / se;
    const float mom = momentum[it];
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      const int c = lane + 32 * t;
      const float p = ex[t] * inv_se - (c == yi ? 1.f : 0.f);
      const float g = loss_scale * p + u[t] + rho * (v[t] - q[t]);
      const float x = fmaf(-step, g, v[t]);
      v[t] = fmaf(mom, x - xp[t], x);
      xp[t] = x;
    }
  }
#pragma unroll
  for (int t = 0; t < CPL; ++t) {
    const int c = lane + 32 * t;
    if (c < C) ZL[base + c] = xp[t];
  }
}

// ------------------------------------------------------------------------------------------
// Reporting (Eq. 1) and the forward pass of Problem 1.
// ------------------------------------------------------------------------------------------
// The sums below leave one partial per block in `partial`; k_add_partials adds the blocks in a fixed order.
// partial[b] = sum (z - f(h))^2 over the block's elements
__global__ void __launch_bounds__(256)
k_sum_hidden_penalty(const float4* __restrict__ Z, const float4* __restrict__ H, long long n4,
                     double* __restrict__ partial) {
  __shared__ double sh[32];
  double s = 0.0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 z = Z[i], h = H[i];
    const float a = z.x - relu(h.x), b = z.y - relu(h.y), c = z.z - relu(h.z), d = z.w - relu(h.w);
    s += (double)(a * a + b * b + c * c + d * d);
  }
  s = block_sum(s, sh);
  if (threadIdx.x == 0) partial[blockIdx.x] = s;
}

// partial[2b] = <U, Z - H>, partial[2b+1] = ||Z - H||^2 over the block's elements
__global__ void __launch_bounds__(256)
k_sum_constraint(const float4* __restrict__ Z, const float4* __restrict__ H, const float4* __restrict__ U,
                 long long n4, double* __restrict__ partial) {
  __shared__ double sh[32];
  double s1 = 0.0, s2 = 0.0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 z = Z[i], h = H[i], u = U[i];
    const float a = z.x - h.x, b = z.y - h.y, c = z.z - h.z, d = z.w - h.w;
    s1 += (double)(u.x * a + u.y * b + u.z * c + u.w * d);
    s2 += (double)(a * a + b * b + c * c + d * d);
  }
  s1 = block_sum(s1, sh);
  s2 = block_sum(s2, sh);
  if (threadIdx.x == 0) { partial[2 * (size_t)blockIdx.x] = s1; partial[2 * (size_t)blockIdx.x + 1] = s2; }
}

// out[j] += sum over b < n_part of partial[b*per + j], j < per; one block, fixed order
// (thread-strided, then the block tree).
__global__ void __launch_bounds__(256)
k_add_partials(const double* __restrict__ partial, int n_part, int per, double* __restrict__ out) {
  __shared__ double sh[32];
  for (int j = 0; j < per; ++j) {
    double s = 0.0;
    for (int b = threadIdx.x; b < n_part; b += blockDim.x) s += partial[(size_t)b * per + j];
    s = block_sum(s, sh);
    if (threadIdx.x == 0) out[j] += s;
  }
}

// Per row: cross-entropy of the row of Zrows with its label (training rows only); argmax of the row of
// `logits` (lowest index on ties) to labels[row]; whether a training row's argmax equals its label.
// One warp per row; partial[2b] = the block's cross-entropy sum, partial[2b+1] = its count of hits,
// rows added in row order.  Either of Zrows / logits may be NULL.
__global__ void __launch_bounds__(256)
k_row_loss_argmax(const float* __restrict__ Zrows, const float* __restrict__ logits, int ld, int C, int n,
                  const int* __restrict__ y, const unsigned char* __restrict__ train,
                  int* __restrict__ labels, double* __restrict__ partial) {
  __shared__ double s_loss[8], s_hit[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * (blockDim.x >> 5) + warp;
  double loss = 0.0, hit = 0.0;
  if (row < n) {
    const long long base = (long long)row * ld;
    const bool tr = train[row] != 0;
    if (Zrows != nullptr && tr) {
      float mx = -3.0e38f;
      for (int c = lane; c < C; c += 32) mx = fmaxf(mx, Zrows[base + c]);
      mx = warp_max(mx);
      float se = 0.f;
      for (int c = lane; c < C; c += 32) se += expf(Zrows[base + c] - mx);
      se = warp_sum(se);
      loss = (double)(mx + logf(se) - Zrows[base + y[row]]);
    }
    if (logits != nullptr) {
      float best = -3.0e38f;
      int arg = 0x7fffffff;
      for (int c = lane; c < C; c += 32) {
        const float v = logits[base + c];
        if (v > best) { best = v; arg = c; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
      }
      if (lane == 0 && labels) labels[row] = arg;
      if (tr && arg == y[row]) hit = 1.0;
    }
  }
  if (lane == 0) { s_loss[warp] = loss; s_hit[warp] = hit; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { a += s_loss[w]; b += s_hit[w]; }
    partial[2 * (size_t)blockIdx.x] = a;
    partial[2 * (size_t)blockIdx.x + 1] = b;
  }
}

// Y = relu(Y) in place.
__global__ void k_relu_inplace(float4* __restrict__ Y, long long n4) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    float4 y = Y[i];
    y.x = relu(y.x); y.y = relu(y.y); y.z = relu(y.z); y.w = relu(y.w);
    Y[i] = y;
  }
}

// U <- U + rho (Z - H)
__global__ void k_dual(float4* __restrict__ U, const float4* __restrict__ Z, const float4* __restrict__ H,
                       long long n4, float rho) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    float4 u = U[i];
    const float4 z = Z[i], h = H[i];
    u.x = fmaf(rho, z.x - h.x, u.x); u.y = fmaf(rho, z.y - h.y, u.y);
    u.z = fmaf(rho, z.z - h.z, u.z); u.w = fmaf(rho, z.w - h.w, u.w);
    U[i] = u;
  }
}

// dst[c][r] = src[r][c] for a small rows x cols matrix (weights and their gradients).
__global__ void k_transpose_small(const float* __restrict__ src, int lds, float* __restrict__ dst, int ldd, int rows,
                                  int cols) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * cols) return;
  const int r = e / cols, c = e % cols;
  dst[c * ldd + r] = src[r * lds + c];
}

__global__ void k_fill_int(int* __restrict__ p, long long count, int value) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count;
       i += (long long)gridDim.x * blockDim.x)
    p[i] = value;
}

// Row gather / scatter between the caller's dense layout (original order, width C) and the
// internal one (community order, leading dimension ld).  to_internal != 0: dst[new] = src[perm[new]].
// dst[r] = src[rows[r]] for padded rows of ld4 float4: the staging copy of the rows a rank does not own
// (what a receive from their owners would deliver) behind its own rows.
__global__ void k_gather_rows(const float4* __restrict__ src, const int* __restrict__ rows, float4* __restrict__ dst,
                              int ld4, long long count) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count * ld4;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / ld4;
    dst[i] = src[(long long)rows[r] * ld4 + (i - r * ld4)];
  }
}

__global__ void k_permute_rows(const float* __restrict__ src, float* __restrict__ dst, const int* __restrict__ perm,
                               long long n, int C, int ld, int to_internal) {
  const long long total = n * ld;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / ld;
    const int c = (int)(e % ld);
    if (to_internal) dst[e] = (c < C) ? src[(long long)perm[r] * C + c] : 0.f;
    else if (c < C) dst[(long long)perm[r] * C + c] = src[e];
  }
}

}  // namespace gk
