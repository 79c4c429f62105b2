// Small dense building blocks of the top-r subspace solver behind Eq. 14-15 (used by the fused
// kernel in subspace_fused.cuh).
//
// The energies c_i = sum_{k<=r} lambda_k V_ik^2 are the diagonal of the best rank-r approximation of
// the Gram matrix G = Z_M^T Z_M (lambda_k = sigma_k^2, V = right singular vectors of Z_M).  The
// library reaches the top-r eigenspace of G by block subspace iteration with p = r + oversample
// vectors.  Every step leaves the float64 Gram matrix B = Y^T Y of the new block as per-tile partial
// sums; its Cholesky factor L makes Q = Y L^-T an orthonormal basis.  After the last step
// Y' = G Q^T: Rayleigh-Ritz for G^2 on the span of the last `win` basis vectors, whose Ritz matrix
// is the trailing win x win block of B' = Y'^T Y' = Q G^2 Q^T.  Its Cholesky factor is diagonalised
// by one-sided Jacobi rotations (this file); the eigenvectors u_k of the p - r smallest Ritz values
// are kept.  For an orthonormal basis of a G-invariant subspace, sum_k lambda_k V_ik^2 =
// sum_j Y'_ij Q_ij; the energy in the top-r subspace is that total over all p basis vectors minus
// the part of the p - r smallest Ritz pairs,
//   c_i = sum_j Y'_ij Q_ij - sum_k (Y'_i,win u_k)(Q_i,win u_k).
// Only the Ritz pairs next to the cut at r have to be resolved individually: basis vectors more
// than 16 places above the cut are separated from the discarded ones by the same eigenvalue ratios
// that drive the subspace iteration itself, so the window has p - r + min(16, r) vectors (all p when
// the problem is small).
#pragma once
#include "subspace_tc.cuh"

namespace covspec {

using sub::kLbufStride;
using sub::kLtFloats;
using sub::kTriMax;
using sub::kXsLd;
using sub::lt_row_offset;
using sub::tri_index;

// Bytes of shared memory the blocked Cholesky factorisation needs for an n x n matrix (8 x 8 tiles
// of the lower triangle in float64, the original diagonal and the reciprocal pivots).
__host__ __device__ inline size_t cholesky_smem_bytes(int n) {
  int nb = (n + 7) / 8;
  return ((size_t)nb * (nb + 1) / 2 * 64 + 16 * nb) * sizeof(double);
}

// One-sided Jacobi on the w columns C[c * ldc + row] (w <= 4 * ROWS): rotate column pairs until
// they are mutually orthogonal.  Round-robin ordering, w/2 disjoint pairs per round, one 4-lane
// group per pair with the two columns held in registers between the inner products and the
// rotation, so that a round is a short instruction stream on few warps and the barrier between
// rounds spans only those warps (named barrier 1 over `nact` threads; the caller guarantees that
// exactly the threads tid < nact enter).  A pair is left alone when its inner product g is
// negligible against the two norms (g^2 <= 1e-12 |a|^2 |b|^2) or so small that the energies move by
// less than ~2e-5 of the problem's scale s1 (g^2 <= (2e-5 s1)^2 min(|a|^2, |b|^2)).  Returns false
// when max_sweeps sweeps did not reach a sweep without rotations.
template <int ROWS>
__device__ __forceinline__ bool jacobi_sweeps(float* C, int ldc, int w, float s1, int max_sweeps,
                                              int nact, volatile int* flag) {
  const int tid = threadIdx.x;
  const int np = (w + 1) & ~1, half = np >> 1;
  const int g = tid >> 2, gl = tid & 3;
  const float abs2 = (2e-5f * s1) * (2e-5f * s1);
  bool converged = w < 2;
  for (int sweep = 0; sweep < max_sweeps && !converged; ++sweep) {
    int rotated = 0;
    for (int round = 0; round < np - 1; ++round) {
      int a = 0, b = 0;
      bool active = g < half;
      if (active) {
        a = round + g; if (a >= np - 1) a -= np - 1;
        b = round - g; if (b < 0) b += np - 1;
        if (g == 0) { a = round; b = np - 1; }
        if (a > b) { int t = a; a = b; b = t; }
        active = b < w;
      }
      float* ca = C + a * ldc;
      float* cb = C + b * ldc;
      float xa[ROWS], xb[ROWS];
      float al = 0.f, be = 0.f, ga = 0.f;
#pragma unroll
      for (int q = 0; q < ROWS; ++q) {
        int row = gl + 4 * q;
        bool in = active && row < w;
        xa[q] = in ? ca[row] : 0.f;
        xb[q] = in ? cb[row] : 0.f;
        al += xa[q] * xa[q]; be += xb[q] * xb[q]; ga += xa[q] * xb[q];
      }
#pragma unroll
      for (int o = 2; o > 0; o >>= 1) {
        al += __shfl_xor_sync(0xffffffffu, al, o);
        be += __shfl_xor_sync(0xffffffffu, be, o);
        ga += __shfl_xor_sync(0xffffffffu, ga, o);
      }
      float g2 = ga * ga;
      float thr2 = fmaxf(1e-12f * al * be, abs2 * fminf(al, be));
      if (active && g2 > thr2 && g2 > 1e-37f) {
        // tan of the rotation angle: t = sign(d g) 2|g| / (|d| + sqrt(d^2 + 4 g^2)), d = |b|^2 - |a|^2
        float d = be - al;
        float t = __fdividef(2.f * ga, fabsf(d) + __fsqrt_rn(d * d + 4.f * g2));
        if (d < 0.f) t = -t;
        float c = rsqrtf(t * t + 1.f), sn = t * c;
#pragma unroll
        for (int q = 0; q < ROWS; ++q) {
          int row = gl + 4 * q;
          if (row < w) {
            ca[row] = c * xa[q] - sn * xb[q];
            cb[row] = sn * xa[q] + c * xb[q];
          }
        }
        rotated = 1;
      }
      sub::named_barrier(1, nact);
    }
    if (rotated) *flag = 1;
    sub::named_barrier(1, nact);
    converged = *flag == 0;
    sub::named_barrier(1, nact);
    if (tid == 0) *flag = 0;
    sub::named_barrier(1, nact);
  }
  return converged;
}

// Column stride of the window factor in shared memory: >= w and congruent to 4 modulo 32, so that
// the eight 4-lane groups of a warp, which hold consecutive columns, hit distinct banks.
__host__ __device__ inline int ritz_ldc(int w) { return (w + 27) / 32 * 32 + 4; }
// Bytes of dynamic shared memory of ritz_kernel for a window of w vectors.
__host__ __device__ inline size_t ritz_smem_bytes(int w) {
  return ((((size_t)w * ritz_ldc(w) + w + 1) & ~(size_t)1)) * sizeof(float) + cholesky_smem_bytes(w);
}

}  // namespace covspec
