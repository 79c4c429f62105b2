// Small dense kernels of the top-r subspace solver behind Eq. 14-15.
//
// The energies c_i = sum_{k<=r} lambda_k V_ik^2 are the diagonal of the best rank-r approximation of
// the Gram matrix G = Z_M^T Z_M (lambda_k = sigma_k^2, V = right singular vectors of Z_M).  The
// library reaches the top-r eigenspace of G by block subspace iteration with p = r + oversample
// vectors (power_tc_kernel).  Every step leaves the float64 Gram matrix B = Y^T Y of the new block
// as per-tile partial sums; this file holds
//   chol_kernel    B = L L^T (float64, one block per request), stored in the layout the next power
//                  step reads, so that Y L^-T is an orthonormal basis;
//   ritz_kernel    after the last step: the singular value decomposition of L by one-sided Jacobi
//                  rotations, L W = U diag(s).  With Y = G Q (Q the previous orthonormal basis),
//                  B = Q G^2 Q^T, so U holds the Ritz vectors of G^2 in the basis Q, s_k ~ lambda_k,
//                  and Y u_k / s_k is the Ritz vector after one more power step;
//   energy_kernel  c_i = sum_{k<r} (Y[i,:] a_k)^2 / s_k^3 with a_k = s_k u_k the rotated columns.
#pragma once
#include "subspace_tc.cuh"

namespace covspec {

using sub::kLbufStride;
using sub::kLtFloats;
using sub::kTriMax;
using sub::lt_row_offset;
using sub::tri_index;

// Sums the per-tile partial Gram matrices of a request in tile order (deterministic) into the
// packed lower triangle A, then factors it in place: on return A[tri(i,k)] (i > k) holds the
// unscaled column entries and piv[k] the (clamped) pivots of the square-root-free elimination, so
// that L[i][k] = A[tri(i,k)] / sqrt(piv[k]) and L[k][k] = sqrt(piv[k]).  A pivot that falls below
// 1e-12 of its original diagonal entry (a numerically dependent direction) is clamped there; the
// next multiplication by G restores the direction.  One __syncthreads per column.
__device__ __forceinline__ void gram_cholesky(const ReqPlan& rp, const double* __restrict__ partial,
                                              double* A, double* piv, double* d0) {
  const int p = rp.p, tri = p * (p + 1) / 2, tid = threadIdx.x, nt = blockDim.x;
  const int lane = tid & 31, w = tid >> 5, nw = nt >> 5;
  const int ntile = (rp.m + sub::kTile - 1) / sub::kTile;
  for (int e = tid; e < tri; e += nt) {
    double s = 0.0;
    for (int t = 0; t < ntile; ++t) s += partial[(size_t)(rp.ptile_off + t) * kTriMax + e];
    A[e] = s;
  }
  __syncthreads();
  for (int i = tid; i < p; i += nt) d0[i] = A[tri_index(i, i)];
  __syncthreads();
  for (int k = 0; k < p; ++k) {
    double pv = A[tri_index(k, k)], floor_ = 1e-12 * d0[k];
    if (!(pv > floor_)) pv = floor_ > 0.0 ? floor_ : 1.0;
    if (tid == 0) piv[k] = pv;
    double inv = 1.0 / pv;
    for (int i = k + 1 + w; i < p; i += nw) {
      double lik = A[tri_index(i, k)] * inv;
      double* row = A + tri_index(i, 0);
      for (int j = k + 1 + lane; j <= i; j += 32) row[j] -= lik * A[tri_index(j, k)];
    }
    __syncthreads();
  }
}

// Dynamic shared memory: (p(p+1)/2 + 2p) doubles.
__global__ void __launch_bounds__(512)
chol_kernel(const ReqPlan* __restrict__ plan, const double* __restrict__ partial,
            float* __restrict__ lbuf) {
  extern __shared__ double sm_d[];
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  const int p = rp.p, P = (p + 7) & ~7, tri = p * (p + 1) / 2;
  double* A = sm_d;
  double* piv = A + tri;
  double* d0 = piv + p;
  gram_cholesky(rp, partial, A, piv, d0);
  // rsqrt of the pivots once
  for (int k = threadIdx.x; k < p; k += blockDim.x) d0[k] = 1.0 / sqrt(piv[k]);
  __syncthreads();
  float* out = lbuf + (size_t)blockIdx.x * kLbufStride;
  // row i of the layout holds L[j][i] for j = (i & ~3) .. P-1; identity beyond p
  const int total = lt_row_offset(P, P);
  for (int i = threadIdx.x >> 5; i < P; i += blockDim.x >> 5) {
    int j0 = i & ~3;
    float* row = out + lt_row_offset(i, P) - j0;
    for (int j = j0 + (threadIdx.x & 31); j < P; j += 32) {
      float v = 0.f;
      if (i < p && j < p) {
        if (j == i) v = (float)sqrt(piv[i]);
        else if (j > i) v = (float)(A[tri_index(j, i)] * d0[i]);
      } else if (i == j) {
        v = 1.f;
      }
      row[j] = v;
    }
  }
  (void)total;
  for (int j = threadIdx.x; j < P; j += blockDim.x)
    out[kLtFloats + j] = j < p ? (float)d0[j] : 1.f;
}

// Dynamic shared memory: (p(p+1)/2 + 2p) doubles + p * ldc floats, ldc = p | 1.
__global__ void __launch_bounds__(1024)
ritz_kernel(const ReqPlan* __restrict__ plan, const double* __restrict__ partial,
            float* __restrict__ ut, float* __restrict__ theta, int max_sweeps, int* status) {
  extern __shared__ double sm_d[];
  __shared__ float s_max;
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  const int p = rp.p, tri = p * (p + 1) / 2, tid = threadIdx.x, nt = blockDim.x;
  double* A = sm_d;
  double* piv = A + tri;
  double* d0 = piv + p;
  const int ldc = p | 1;
  float* C = reinterpret_cast<float*>(d0 + p);          // columns of L: C[c * ldc + row]
  float* sig = C + (size_t)p * ldc;                     // [p] column norms at the end
  gram_cholesky(rp, partial, A, piv, d0);
  for (int k = tid; k < p; k += nt) d0[k] = 1.0 / sqrt(piv[k]);
  __syncthreads();
  for (int e = tid; e < p * p; e += nt) {
    int c = e / p, row = e % p;
    float v = 0.f;
    if (row == c) v = (float)sqrt(piv[c]);
    else if (row > c) v = (float)(A[tri_index(row, c)] * d0[c]);
    C[c * ldc + row] = v;
  }
  __syncthreads();
  // One-sided Jacobi: rotate column pairs until all columns are mutually orthogonal.  Round-robin
  // ordering, p/2 disjoint pairs per round, one 16-lane group per pair.
  const int np = (p + 1) & ~1, half = np >> 1;
  const int g = tid >> 4, gl = tid & 15, ng = nt >> 4;
  bool converged = p < 2;
  for (int sweep = 0; sweep < max_sweeps && !converged; ++sweep) {
    int rotated = 0;
    for (int round = 0; round < np - 1; ++round) {
      for (int base = 0; base < half; base += ng) {
        int i = base + g;
        int a = 0, b = 0;
        bool active = i < half;
        if (active) {
          a = i == 0 ? round : (round + i) % (np - 1);
          b = i == 0 ? np - 1 : (round - i + np - 1) % (np - 1);
          if (a > b) { int t = a; a = b; b = t; }
          active = b < p;
        }
        float* ca = C + a * ldc;
        float* cb = C + b * ldc;
        float al = 0.f, be = 0.f, ga = 0.f;
        if (active)
          for (int row = gl; row < p; row += 16) {
            float x = ca[row], y = cb[row];
            al += x * x; be += y * y; ga += x * y;
          }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
          al += __shfl_xor_sync(0xffffffffu, al, o);
          be += __shfl_xor_sync(0xffffffffu, be, o);
          ga += __shfl_xor_sync(0xffffffffu, ga, o);
        }
        if (active && fabsf(ga) > 1e-6f * sqrtf(al * be) && fabsf(ga) > 1e-36f) {
          float zeta = (be - al) / (2.f * ga);
          float t = (zeta >= 0.f ? 1.f : -1.f) / (fabsf(zeta) + sqrtf(zeta * zeta + 1.f));
          float c = rsqrtf(t * t + 1.f), s = t * c;
          for (int row = gl; row < p; row += 16) {
            float x = ca[row], y = cb[row];
            ca[row] = c * x - s * y;
            cb[row] = s * x + c * y;
          }
          rotated = 1;
        }
      }
      __syncthreads();
    }
    converged = __syncthreads_or(rotated) == 0;
  }
  if (!converged && tid == 0) atomicOr(status, kStatusNoConverge);
  // singular values = column norms
  for (int k = tid >> 5; k < p; k += nt >> 5) {
    float s = 0.f;
    for (int row = tid & 31; row < p; row += 32) { float x = C[k * ldc + row]; s += x * x; }
    s = warp_sum(s);
    if ((tid & 31) == 0) sig[k] = sqrtf(s);
  }
  if (tid == 0) s_max = 0.f;
  __syncthreads();
  if (tid < 32) {
    float m = 0.f;
    for (int k = tid; k < p; k += 32) m = fmaxf(m, sig[k]);
    m = warp_max(m);
    if (tid == 0) s_max = m;
  }
  __syncthreads();
  // rank the columns by singular value (descending, ties by index); the r largest, scaled by
  // s^-3/2, become the rows-by-rank matrix the energy kernel multiplies with: ut[j * r + rank]
  float* out_u = ut + (size_t)blockIdx.x * kPMax * kPMax;
  float* out_t = theta + (size_t)blockIdx.x * kPMax;
  const int r = rp.r;
  for (int k = tid >> 5; k < p; k += nt >> 5) {
    float sk = sig[k];
    int rank = 0;
    for (int q = tid & 31; q < p; q += 32) {
      float sq = sig[q];
      rank += (sq > sk) || (sq == sk && q < k);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
    if (rank < r) {
      float scale = sk > 1e-6f * s_max ? 1.f / (sk * sqrtf(sk)) : 0.f;
      for (int j = tid & 31; j < p; j += 32) out_u[j * r + rank] = C[k * ldc + j] * scale;
      if ((tid & 31) == 0) out_t[rank] = sk;
    }
  }
}

// Eq. 15 for the preselected tokens of every request: c_i = sum_{k<r} (sum_j Yf[i][j] ut[j][k])^2.
// Requests without stage 2 get zeros.  grid = (ceil(max M / 64), batch), 256 threads: one warp per
// token row, lanes over k.  Dynamic shared memory: p_max * r_max floats.
__global__ void __launch_bounds__(256)
energy_kernel(const ReqPlan* __restrict__ plan, const float* __restrict__ yf,
              const float* __restrict__ ut, float* __restrict__ energy) {
  extern __shared__ float sm_u[];
  ReqPlan rp = plan[blockIdx.y];
  const int row0 = blockIdx.x * 64;
  if (row0 >= rp.m) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (!rp.stage2) {
    for (int i = row0 + threadIdx.x; i < min(rp.m, row0 + 64); i += blockDim.x) energy[rp.presel_off + i] = 0.f;
    return;
  }
  const int p = rp.p, r = rp.r;
  const float* u = ut + (size_t)blockIdx.y * kPMax * kPMax;
  for (int e = threadIdx.x; e < p * r; e += blockDim.x) sm_u[e] = u[e];
  __syncthreads();
  for (int i = row0 + w; i < min(rp.m, row0 + 64); i += 8) {
    const float* y = yf + ((size_t)rp.presel_off + i) * kPMax;
    float acc[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
    for (int jc = 0; jc < p; jc += 32) {
      float yv = jc + lane < p ? y[jc + lane] : 0.f;
      int jn = min(32, p - jc);
      for (int jj = 0; jj < jn; ++jj) {
        float yj = __shfl_sync(0xffffffffu, yv, jj);
        const float* ur = sm_u + (jc + jj) * r;
#pragma unroll
        for (int kk = 0; kk < 5; ++kk) {
          int k = lane + 32 * kk;
          if (k < r) acc[kk] += yj * ur[k];
        }
      }
    }
    float c = 0.f;
#pragma unroll
    for (int kk = 0; kk < 5; ++kk) c += acc[kk] * acc[kk];
    c = warp_sum(c);
    if (lane == 0) energy[rp.presel_off + i] = c;
  }
}

}  // namespace covspec
