// Small dense kernels of the top-r subspace solver behind Eq. 14-15.
//
// The energies c_i = sum_{k<=r} lambda_k V_ik^2 are the diagonal of the best rank-r approximation of
// the Gram matrix G = Z_M^T Z_M (lambda_k = sigma_k^2, V = right singular vectors of Z_M).  The
// library reaches the top-r eigenspace of G by block subspace iteration with p = r + oversample
// basis vectors, orthonormalised every step by a Cholesky QR whose p x p Gram matrix is accumulated
// and factored in float64, and finishes with a Rayleigh-Ritz step (p x p symmetric eigenproblem by
// cyclic Jacobi) that splits the p Ritz pairs at r.  Bases are stored transposed ([p x ldm], one
// basis vector per row) so that every large product is an A * B^T with contiguous k.
#pragma once
#include "common.cuh"

namespace covspec {

// Start basis: entries uniform in [-1, 1) from a counter hash of (request, vector, position).
__global__ void __launch_bounds__(256)
eig_init_kernel(const ReqPlan* __restrict__ plan, float* __restrict__ U) {
  ReqPlan rp = plan[blockIdx.y];
  if (!rp.stage2) return;
  int total = rp.p * rp.ldm;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
    int col = e % rp.ldm;
    unsigned h = (unsigned)e * 0x9E3779B1u ^ ((unsigned)blockIdx.y + 1u) * 0x85EBCA77u;
    h ^= h >> 16; h *= 0x7FEB352Du; h ^= h >> 15; h *= 0x846CA68Bu; h ^= h >> 16;
    float v = (float)(h >> 8) * (2.0f / 16777216.0f) - 1.0f;
    U[rp.u_off + e] = col < rp.m ? v : 0.f;
  }
}

// Cholesky factor of the p x p float64 Gram matrix Bm = L L^T and its inverse, one block per
// request.  Writes Linv (float32, [p x ldp], upper part zero) so that Linv * Z has orthonormal
// rows.  A pivot that falls below 1e-12 of its original diagonal entry (a numerically dependent
// direction) is clamped there; the next multiplication by G restores the direction.
// Dynamic shared memory: p*p + 2*p doubles.
__global__ void __launch_bounds__(1024)
chol_inv_kernel(const ReqPlan* __restrict__ plan, const double* __restrict__ Bm,
                float* __restrict__ Linv) {
  extern __shared__ double sm_d[];
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  int p = rp.p, ldp = (p + 3) & ~3, tid = threadIdx.x, nt = blockDim.x;
  double* L = sm_d;                 // [p][p]
  double* diag0 = sm_d + p * p;     // original diagonal
  double* col = diag0 + p;          // scratch column
  const double* src = Bm + (size_t)blockIdx.x * kPMax * kPMax;
  for (int e = tid; e < p * p; e += nt) L[e] = src[(e / p) * kPMax + (e % p)];
  __syncthreads();
  for (int i = tid; i < p; i += nt) diag0[i] = L[i * p + i];
  __syncthreads();
  for (int k = 0; k < p; ++k) {
    if (tid == 0) {
      double piv = L[k * p + k], floor_ = 1e-12 * diag0[k];
      if (!(piv > floor_)) piv = floor_ > 0.0 ? floor_ : 1.0;
      L[k * p + k] = sqrt(piv);
    }
    __syncthreads();
    double dk = L[k * p + k];
    for (int i = k + 1 + tid; i < p; i += nt) L[i * p + k] /= dk;
    __syncthreads();
    int rem = p - k - 1;
    for (int e = tid; e < rem * rem; e += nt) {
      int i = k + 1 + e / rem, j = k + 1 + e % rem;
      if (j <= i) L[i * p + j] -= L[i * p + k] * L[j * p + k];
    }
    __syncthreads();
  }
  // In-place inverse of the lower-triangular L, column by column from the right.
  int lane = tid & 31, w = tid >> 5, nw = nt >> 5;
  for (int j = p - 1; j >= 0; --j) {
    for (int i = j + 1 + tid; i < p; i += nt) col[i] = L[i * p + j];
    __syncthreads();
    double inv_jj = 1.0 / L[j * p + j];
    for (int i = j + 1 + w; i < p; i += nw) {
      double s = 0.0;
      for (int k = j + 1 + lane; k <= i; k += 32) s += L[i * p + k] * col[k];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) L[i * p + j] = -s * inv_jj;
    }
    if (tid == 0) L[j * p + j] = inv_jj;
    __syncthreads();
  }
  float* dst = Linv + (size_t)blockIdx.x * kPMax * kPMax;
  for (int e = tid; e < p * ldp; e += nt) {
    int i = e / ldp, j = e % ldp;
    dst[i * ldp + j] = (j <= i && j < p) ? (float)L[i * p + j] : 0.f;
  }
}

// Rayleigh-Ritz: eigen-decomposition of the symmetric p x p matrix S = Q G Q^T by cyclic Jacobi
// with a round-robin parallel ordering (p/2 disjoint rotations per round), one block per request.
// Rotations whose off-diagonal entry is negligible against the two diagonal entries are skipped.
// Outputs the r largest Ritz values (theta, descending) and the matching eigenvectors as rows of
// Wr ([r x ldp]).  Dynamic shared memory: 2 * p * (p + 1) floats + rotation table.
__global__ void __launch_bounds__(1024)
jacobi_kernel(const ReqPlan* __restrict__ plan, const float* __restrict__ Sm, float* __restrict__ Wr,
              float* __restrict__ theta, int max_sweeps, int* status) {
  extern __shared__ float sm_f[];
  __shared__ int n_rot;
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  int p = rp.p, ldp = (p + 3) & ~3, ld = p + 1, tid = threadIdx.x, nt = blockDim.x;
  int np = (p + 1) & ~1;            // padded to even: index p (if present) is a bye
  int half = np >> 1;
  float* S = sm_f;                  // [p][ld]
  float* W = S + p * ld;            // [p][ld]
  float* rc = W + p * ld;           // [half] cos
  float* rs = rc + half;            // [half] sin (0 = skipped)
  int* ra = reinterpret_cast<int*>(rs + half);
  int* rb = ra + half;
  const float* src = Sm + (size_t)blockIdx.x * kPMax * kPMax;
  for (int e = tid; e < p * p; e += nt) {
    int i = e / p, j = e % p;
    // symmetrise the input (it is Q G Q^T up to rounding)
    S[i * ld + j] = 0.5f * (src[i * ldp + j] + src[j * ldp + i]);
    W[i * ld + j] = i == j ? 1.f : 0.f;
  }
  __syncthreads();
  bool converged = p < 2;
  for (int sweep = 0; sweep < max_sweeps && !converged; ++sweep) {
    if (tid == 0) n_rot = 0;
    __syncthreads();
    for (int round = 0; round < np - 1; ++round) {
      for (int i = tid; i < half; i += nt) {
        int a = i == 0 ? round : (round + i) % (np - 1);
        int b = i == 0 ? np - 1 : (round - i + np - 1) % (np - 1);
        if (a > b) { int t = a; a = b; b = t; }
        float c = 1.f, s = 0.f;
        if (b < p) {
          float saa = S[a * ld + a], sbb = S[b * ld + b], sab = S[a * ld + b];
          if (fabsf(sab) > 2e-7f * sqrtf(fabsf(saa * sbb)) && fabsf(sab) > 1e-30f) {
            float th = (sbb - saa) / (2.f * sab);
            float t = (th >= 0.f ? 1.f : -1.f) / (fabsf(th) + sqrtf(th * th + 1.f));
            c = rsqrtf(t * t + 1.f);
            s = t * c;
            atomicAdd(&n_rot, 1);
          }
        }
        rc[i] = c; rs[i] = s; ra[i] = a; rb[i] = b;
      }
      __syncthreads();
      // columns: S <- S J, W <- W J
      for (int e = tid; e < half * p; e += nt) {
        int i = e / p, row = e % p;
        float s = rs[i];
        if (s == 0.f) continue;
        float c = rc[i];
        int a = ra[i], b = rb[i];
        float xa = S[row * ld + a], xb = S[row * ld + b];
        S[row * ld + a] = c * xa - s * xb;
        S[row * ld + b] = s * xa + c * xb;
        float wa = W[row * ld + a], wb = W[row * ld + b];
        W[row * ld + a] = c * wa - s * wb;
        W[row * ld + b] = s * wa + c * wb;
      }
      __syncthreads();
      // rows: S <- J^T S
      for (int e = tid; e < half * p; e += nt) {
        int i = e / p, colj = e % p;
        float s = rs[i];
        if (s == 0.f) continue;
        float c = rc[i];
        int a = ra[i], b = rb[i];
        float xa = S[a * ld + colj], xb = S[b * ld + colj];
        S[a * ld + colj] = c * xa - s * xb;
        S[b * ld + colj] = s * xa + c * xb;
      }
      __syncthreads();
      // the rotated pair is now decoupled: store exact zeros instead of rounding residue
      for (int i = tid; i < half; i += nt)
        if (rs[i] != 0.f) { S[ra[i] * ld + rb[i]] = 0.f; S[rb[i] * ld + ra[i]] = 0.f; }
      __syncthreads();
    }
    converged = n_rot == 0;
    __syncthreads();
  }
  if (!converged && tid == 0) atomicOr(status, kStatusNoConverge);
  // Rank the Ritz values (descending, ties by index) and emit the top r.
  float* out_w = Wr + (size_t)blockIdx.x * kPMax * kPMax;
  float* out_t = theta + (size_t)blockIdx.x * kPMax;
  for (int k = tid; k < p; k += nt) {
    float tk = S[k * ld + k];
    int rank = 0;
    for (int q = 0; q < p; ++q) {
      float tq = S[q * ld + q];
      rank += (tq > tk) || (tq == tk && q < k);
    }
    if (rank < rp.r) out_t[rank] = tk;
    // scatter column k of W into row `rank` of Wr
    if (rank < rp.r)
      for (int i = 0; i < ldp; ++i) out_w[rank * ldp + i] = i < p ? W[i * ld + k] : 0.f;
  }
}

// c_i = sum_{k<r} theta_k * Vt[k, i]^2 for the preselected tokens of every request (Eq. 15), where
// Vt = Wr * Q holds the Ritz vectors as rows.  Requests without stage 2 get zeros.
__global__ void __launch_bounds__(256)
energy_kernel(const ReqPlan* __restrict__ plan, const float* __restrict__ Vt,
              const float* __restrict__ theta, float* __restrict__ energy) {
  ReqPlan rp = plan[blockIdx.y];
  const float* th = theta + (size_t)blockIdx.y * kPMax;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < rp.m; i += gridDim.x * blockDim.x) {
    float c = 0.f;
    if (rp.stage2) {
      const float* v = Vt + rp.u_off + i;
      for (int k = 0; k < rp.r; ++k) { float x = v[(size_t)k * rp.ldm]; c += fmaxf(th[k], 0.f) * x * x; }
    }
    energy[rp.presel_off + i] = c;
  }
}

}  // namespace covspec
