// Tiled CUDA-core product C = A * op(B) for a list of independent problems (ragged batch).
// Used where full float32 / float64 accumulation of float32 operands is required (the subspace
// iteration on the Gram matrix) and for the float32 configuration; bf16 operands are widened on
// load, so products are exact and only the float32 accumulation rounds.
#pragma once
#include "common.cuh"

namespace covspec {

constexpr int kGemmBM = 64, kGemmBN = 64, kGemmBK = 16;

// A [m x k] row-major (k contiguous).  B [n x k] row-major when !B_KN (C = A * B^T), or
// [k x n] row-major when B_KN (C = A * B).  C [m x n] row-major of TC.  Leading dimensions in
// elements; vector loads need ld % 4 == 0 and 16-byte aligned bases, which the caller guarantees.
// `lower_only`: skip tiles strictly above the diagonal and mirror the computed ones (C symmetric).
template <typename TA, typename TB, typename AccT, typename TC, bool B_KN>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const GemmProb* __restrict__ table, int nprob, GemmProb single, int lower_only) {
  __shared__ AccT As[kGemmBK][kGemmBM + 4];
  __shared__ AccT Bs[kGemmBK][kGemmBN + 4];
  GemmProb pr;
  if (table == nullptr) {
    pr = single;
  } else {
    int lo = 0, hi = nprob - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (table[mid].tile_start <= (int)blockIdx.x) lo = mid; else hi = mid - 1;
    }
    pr = table[lo];
  }
  int tile = blockIdx.x - pr.tile_start;
  int tm = tile / pr.tiles_n, tn = tile % pr.tiles_n;
  if (lower_only && tn > tm) return;
  int row0 = tm * kGemmBM, col0 = tn * kGemmBN;
  const TA* A = reinterpret_cast<const TA*>(pr.A);
  const TB* B = reinterpret_cast<const TB*>(pr.B);
  int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  AccT acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = AccT(0);

  // loader coordinates
  int a_row = tid >> 2, a_k = (tid & 3) * 4;           // A tile: 64 rows x 16 k
  int bkn_k = tid >> 4, bkn_n = (tid & 15) * 4;        // B tile when [k x n]: 16 k x 64 n

  // The next k-tile is fetched into registers while the current one is multiplied, so that the
  // global-memory latency overlaps the arithmetic (the problems here are small: few blocks, and a
  // loop that waited for every tile would be latency-bound).
  auto fetch = [&](int k0, float (&va)[4], float (&vb)[4]) {
#pragma unroll
    for (int e = 0; e < 4; ++e) { va[e] = 0.f; vb[e] = 0.f; }
    if (k0 >= pr.k) return;
    {
      int r = row0 + a_row, kk = k0 + a_k;
      if (r < pr.m) {
        const TA* src = A + (size_t)r * pr.lda + kk;
        if (kk + 3 < pr.k) load4(src, va);
        else for (int e = 0; e < 4; ++e) if (kk + e < pr.k) va[e] = to_float(src[e]);
      }
    }
    if (!B_KN) {
      int r = col0 + a_row, kk = k0 + a_k;
      if (r < pr.n) {
        const TB* src = B + (size_t)r * pr.ldb + kk;
        if (kk + 3 < pr.k) load4(src, vb);
        else for (int e = 0; e < 4; ++e) if (kk + e < pr.k) vb[e] = to_float(src[e]);
      }
    } else {
      int kk = k0 + bkn_k, c = col0 + bkn_n;
      if (kk < pr.k) {
        const TB* src = B + (size_t)kk * pr.ldb + c;
        if (c + 3 < pr.n) load4(src, vb);
        else for (int e = 0; e < 4; ++e) if (c + e < pr.n) vb[e] = to_float(src[e]);
      }
    }
  };
  float va[4], vb[4];
  fetch(0, va, vb);
  for (int k0 = 0; k0 < pr.k; k0 += kGemmBK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) As[a_k + e][a_row] = (AccT)va[e];
    if (!B_KN) {
#pragma unroll
      for (int e = 0; e < 4; ++e) Bs[a_k + e][a_row] = (AccT)vb[e];
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) Bs[bkn_k][bkn_n + e] = (AccT)vb[e];
    }
    __syncthreads();
    fetch(k0 + kGemmBK, va, vb);
#pragma unroll
    for (int kk = 0; kk < kGemmBK; ++kk) {
      AccT a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
    }
    __syncthreads();
  }
  TC* C = reinterpret_cast<TC*>(pr.C);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int r = row0 + ty * 4 + i;
    if (r >= pr.m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int c = col0 + tx * 4 + j;
      if (c >= pr.n) continue;
      C[(size_t)r * pr.ldc + c] = (TC)acc[i][j];
      if (lower_only && tn < tm) C[(size_t)c * pr.ldc + r] = (TC)acc[i][j];
    }
  }
}

}  // namespace covspec
