// Small dense kernels of the top-r subspace solver behind Eq. 14-15.
//
// The energies c_i = sum_{k<=r} lambda_k V_ik^2 are the diagonal of the best rank-r approximation of
// the Gram matrix G = Z_M^T Z_M (lambda_k = sigma_k^2, V = right singular vectors of Z_M).  The
// library reaches the top-r eigenspace of G by block subspace iteration with p = r + oversample
// vectors (power_tc_kernel).  Every step leaves the float64 Gram matrix B = Y^T Y of the new block
// as per-tile partial sums; this file holds
//   chol_kernel    B = L L^T (float64, one block per request), stored in the layout the next power
//                  step reads, so that Q = Y L^-T is an orthonormal basis.
//   ritz_kernel    after the last step Y' = G Q^T: Rayleigh-Ritz for G^2 on the span of the last
//                  `win` basis vectors, whose Ritz matrix is the trailing win x win block of
//                  B' = Y'^T Y' = Q G^2 Q^T.  Its Cholesky factor is diagonalised by one-sided Jacobi
//                  rotations; the eigenvectors u_k of the p - r smallest Ritz values are kept.
//   energy_kernel  for an orthonormal basis of a G-invariant subspace, sum_k lambda_k V_ik^2 =
//                  sum_j Y'_ij Q_ij; the energy in the top-r subspace is that total over all p basis
//                  vectors minus the part of the p - r smallest Ritz pairs,
//                  c_i = sum_j Y'_ij Q_ij - sum_k (Y'_i,win u_k)(Q_i,win u_k).
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

// 1 / sqrt(x) in float64.  The factorisation's critical path runs through this once per column, so
// the chain of dependent float64 operations is kept short: the float32 estimate is first refined
// in float32 (to ~2^-23), then one Newton step in float64 squares that error (~1e-13).  The library
// routine is used outside the float32 range.
__device__ __forceinline__ double rsqrt_f64(double x) {
  if (!(x > 1e-37 && x < 1e37)) return 1.0 / sqrt(x);
  float xf = (float)x;
  float yf = rsqrtf(xf);
  yf = yf * (1.5f - 0.5f * xf * yf * yf);
  double y = (double)yf;
  double e = fma(-0.5 * x * y, y, 0.5);   // (1 - x y^2) / 2
  return fma(y, e, y);
}

// Blocked right-looking Cholesky factorisation of an n x n float64 matrix kept in shared memory as
// 8 x 8 tiles of its lower triangle (tile (I, J <= I) at T + tri_index(I, J) * 64, row-major).
// Per 8-column panel: the diagonal tile is factored by one thread in registers, the tiles below it are solved one
// row per thread, and the trailing tiles take their rank-8 update on the FP64 tensor cores
// (two m8n8k4 instructions per tile); the next panel's diagonal tile is factored while the rest of
// the trailing matrix is still being updated.  Three __syncthreads per panel.
// A pivot below 1e-12 of its original diagonal entry (a numerically dependent direction) is
// clamped there; the next multiplication by G restores the direction.
//   load(i, j)         value of entry (i, j), i >= j
//   store(i, j, v, rd) receives L[i][j] and 1 / L[j][j]
//   T: 64 * nb (nb + 1) / 2 doubles, nb = ceil(n / 8);  aux: 2 * 8 * nb doubles
template <typename Load, typename Store>
__device__ __forceinline__ void cholesky_blocked(int n, double* T, double* aux, Load load, Store store) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  const int nb = (n + 7) >> 3, ntile = nb * (nb + 1) / 2;
  double* d0 = aux;                 // original diagonal
  double* rd = aux + 8 * nb;        // 1 / L[j][j]
  // four entries per thread and trip, so that their global loads overlap
  for (int e0 = tid; e0 < ntile * 64; e0 += 4 * nt) {
    double v[4];
    int ii[4], jj[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int e = e0 + u * nt, I = 0, J = 0;
      if (e < ntile * 64) sub::tri_decode(e >> 6, I, J);
      ii[u] = 8 * I + ((e >> 3) & 7); jj[u] = 8 * J + (e & 7);
      if (e >= ntile * 64) v[u] = 0.0;
      else if (ii[u] < n && jj[u] < n) v[u] = jj[u] <= ii[u] ? load(ii[u], jj[u]) : load(jj[u], ii[u]);
      else v[u] = ii[u] == jj[u] ? 1.0 : 0.0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int e = e0 + u * nt;
      if (e < ntile * 64) {
        T[e] = v[u];
        if (ii[u] == jj[u]) d0[ii[u]] = v[u];
      }
    }
  }
  __syncthreads();
  // factor the diagonal tile (J, J) in registers: one thread; the chain of eight dependent
  // reciprocal square roots is the critical path of the whole factorisation
  auto factor_diag = [&](int J) {
    double* D = T + tri_index(J, J) * 64;
    double a[8][8];
#pragma unroll
    for (int l = 0; l < 8; ++l)
#pragma unroll
      for (int m = 0; m <= l; ++m) a[l][m] = D[l * 8 + m];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      double piv = a[c][c], floor_ = 1e-12 * d0[8 * J + c];
      if (!(piv > floor_)) piv = floor_ > 0.0 ? floor_ : 1.0;
      double rs = rsqrt_f64(piv);
      a[c][c] = piv * rs;
      rd[8 * J + c] = rs;
#pragma unroll
      for (int l = c + 1; l < 8; ++l) a[l][c] *= rs;
#pragma unroll
      for (int l = c + 1; l < 8; ++l)
#pragma unroll
        for (int m = c + 1; m <= l; ++m) a[l][m] -= a[l][c] * a[m][c];
    }
#pragma unroll
    for (int l = 0; l < 8; ++l)
#pragma unroll
      for (int m = 0; m <= l; ++m) D[l * 8 + m] = a[l][m];
  };
  // C(I, K) -= X_I X_K^T for one trailing tile of panel J (rank-8 update, two tensor-core instructions)
  const int fr = lane >> 2, fk = lane & 3;
  auto update_tile = [&](int J, int I, int K) {
    const double* XI = T + tri_index(I, J) * 64 + fr * 8 + fk;
    const double* XK = T + tri_index(K, J) * 64 + fr * 8 + fk;
    double* C = T + tri_index(I, K) * 64 + fr * 8 + 2 * fk;
    double c0 = C[0], c1 = C[1];
    sub::dmma_8x8x4(c0, c1, -XI[0], XK[0]);
    sub::dmma_8x8x4(c0, c1, -XI[4], XK[4]);
    C[0] = c0; C[1] = c1;
  };
  if (tid == 0) factor_diag(0);
  __syncthreads();
  for (int J = 0; J < nb; ++J) {
    const double* D = T + tri_index(J, J) * 64;
    // tiles below the diagonal tile: row i of tile (I, J) <- row * L_JJ^-T
    for (int i = 8 * (J + 1) + tid; i < 8 * nb; i += nt) {
      double* row = T + tri_index(i >> 3, J) * 64 + (i & 7) * 8;
      double x[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) x[c] = row[c];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        double v = x[c];
#pragma unroll
        for (int k = 0; k < c; ++k) v -= x[k] * D[c * 8 + k];
        x[c] = v * rd[8 * J + c];
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) row[c] = x[c];
    }
    __syncthreads();
    if (J + 1 == nb) break;
    // look-ahead: the tiles of column J+1 take their update first ...
    for (int I = J + 1 + warp; I < nb; I += nw) update_tile(J, I, J + 1);
    __syncthreads();
    // ... so that its diagonal tile is factored (warp 0, one thread) while the other warps update
    // the rest of the trailing matrix, tiles (I, K) with J+1 < K <= I
    if (warp == 0) {
      if (lane == 0) factor_diag(J + 1);
      __syncwarp();
    } else {
      const int mrem = nb - J - 2, ntr = mrem * (mrem + 1) / 2;
      for (int q = warp - 1; q < ntr; q += nw - 1) {
        int ii, kk;
        sub::tri_decode(q, ii, kk);
        update_tile(J, J + 2 + ii, J + 2 + kk);
      }
    }
    __syncthreads();
  }
  for (int e = tid; e < ntile * 64; e += nt) {
    int I, J;
    sub::tri_decode(e >> 6, I, J);
    int i = 8 * I + ((e >> 3) & 7), j = 8 * J + (e & 7);
    if (i < n && j <= i) store(i, j, T[e], rd[j]);
  }
}

// Sum of the per-tile partial Gram matrices of a request, in tile order (deterministic).
__device__ __forceinline__ double gram_entry(const ReqPlan& rp, const double* __restrict__ partial,
                                             int i, int j) {
  const int ntile = (rp.m + sub::kTile - 1) / sub::kTile;
  const double* src = partial + (size_t)rp.ptile_off * kTriMax + tri_index(i, j);
  // four independent loads in flight; the summation order is fixed (tile order within each of the
  // four interleaved partial sums, then a fixed combination), so the result is deterministic
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  int t = 0;
  for (; t + 4 <= ntile; t += 4) {
    double a = src[(size_t)t * kTriMax], b = src[(size_t)(t + 1) * kTriMax];
    double c = src[(size_t)(t + 2) * kTriMax], d = src[(size_t)(t + 3) * kTriMax];
    s0 += a; s1 += b; s2 += c; s3 += d;
  }
  for (; t < ntile; ++t) s0 += src[(size_t)t * kTriMax];
  return (s0 + s1) + (s2 + s3);
}

// Bytes of shared memory cholesky_blocked needs for an n x n matrix.
__host__ __device__ inline size_t cholesky_smem_bytes(int n) {
  int nb = (n + 7) / 8;
  return ((size_t)nb * (nb + 1) / 2 * 64 + 16 * nb) * sizeof(double);
}

// One block of 512 threads per request.  Dynamic shared memory: cholesky_smem_bytes(p_max).
__global__ void __launch_bounds__(512)
chol_kernel(const ReqPlan* __restrict__ plan, const double* __restrict__ partial,
            float* __restrict__ lbuf) {
  extern __shared__ double sm_d[];
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  const int p = rp.p, P = (p + 7) & ~7, nb = (p + 7) >> 3;
  float* out = lbuf + (size_t)blockIdx.x * kLbufStride;
  // identity padding of the layout rows / columns p .. P-1 and the entries left of the diagonal
  for (int i = threadIdx.x >> 5; i < P; i += blockDim.x >> 5) {
    int j0 = i & ~3;
    float* row = out + lt_row_offset(i, P) - j0;
    for (int j = j0 + (threadIdx.x & 31); j < P; j += 32)
      if (j < i || i >= p || j >= p) row[j] = (i == j) ? 1.f : 0.f;
  }
  for (int j = p + threadIdx.x; j < P; j += blockDim.x) out[kLtFloats + j] = 1.f;
  auto load = [&](int i, int j) { return gram_entry(rp, partial, i, j); };
  // row j of the layout holds L[i][j] for i >= (j & ~3)
  auto store = [&](int i, int j, double v, double rdj) {
    out[lt_row_offset(j, P) + i - (j & ~3)] = (float)v;
    if (i == j) out[kLtFloats + j] = (float)rdj;
  };
  cholesky_blocked(p, sm_d, sm_d + (size_t)nb * (nb + 1) / 2 * 64, load, store);
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

// Rayleigh-Ritz on the trailing window (see the file comment).  One block of 512 threads per
// request.  Output ub[j * nbot + k]: component j (window coordinates) of the unit eigenvector of
// the k-th smallest Ritz value, k < nbot = p - r.
// Dynamic shared memory: ritz_smem_bytes(win_max).
__global__ void __launch_bounds__(512)
ritz_kernel(const ReqPlan* __restrict__ plan, const double* __restrict__ partial,
            float* __restrict__ ub, int max_sweeps, int* status) {
  extern __shared__ float sm_f[];
  __shared__ float s_scale;
  __shared__ int s_flag;
  ReqPlan rp = plan[blockIdx.x];
  if (!rp.stage2) return;
  const int p = rp.p, w = rp.win, w0 = p - w, nbot = p - rp.r;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int ldc = ritz_ldc(w);
  float* C = sm_f;                                  // columns of the factor: C[c * ldc + row]
  float* sig = C + (size_t)w * ldc;                 // [w] column norms at the end
  for (int e = tid; e < w * ldc; e += nt) C[e] = 0.f;
  if (tid == 0) s_scale = 0.f;
  __syncthreads();
  // scale of the whole problem: sqrt of the largest diagonal entry of B' (~ the largest Ritz value)
  {
    float m = 0.f;
    for (int i = tid; i < p; i += nt) m = fmaxf(m, (float)gram_entry(rp, partial, i, i));
    m = warp_max(m);
    if ((tid & 31) == 0 && m > 0.f) atomicMax(reinterpret_cast<int*>(&s_scale), __float_as_int(m));
  }
  auto load = [&](int i, int j) { return gram_entry(rp, partial, w0 + i, w0 + j); };
  auto store = [&](int i, int j, double v, double) { C[j * ldc + i] = (float)v; };
  {
    const int nbw = (w + 7) >> 3;
    double* Tw = reinterpret_cast<double*>(sm_f + (((size_t)w * ldc + w + 1) & ~(size_t)1));   // 8-byte aligned
    cholesky_blocked(w, Tw, Tw + (size_t)nbw * (nbw + 1) / 2 * 64, load, store);
  }
  __syncthreads();
  const float s1 = sqrtf(s_scale);
  // the rotations run on the first 4 * (pairs per round) threads (whole warps); the rest wait
  const int nact = min(nt, ((((w + 1) >> 1) * 4) + 31) & ~31);
  if (tid == 0) s_flag = 0;
  __syncthreads();
  if (tid < nact) {
    bool converged;
    if (w <= 32) converged = jacobi_sweeps<8>(C, ldc, w, s1, max_sweeps, nact, &s_flag);
    else if (w <= 64) converged = jacobi_sweeps<16>(C, ldc, w, s1, max_sweeps, nact, &s_flag);
    else if (w <= 96) converged = jacobi_sweeps<24>(C, ldc, w, s1, max_sweeps, nact, &s_flag);
    else converged = jacobi_sweeps<(kPMax + 3) / 4>(C, ldc, w, s1, max_sweeps, nact, &s_flag);
    if (!converged && tid == 0) atomicOr(status, kStatusNoConverge);
  }
  __syncthreads();
  // singular values = column norms
  for (int k = tid >> 5; k < w; k += nt >> 5) {
    float s = 0.f;
    for (int row = tid & 31; row < w; row += 32) { float x = C[k * ldc + row]; s += x * x; }
    s = warp_sum(s);
    if ((tid & 31) == 0) sig[k] = sqrtf(s);
  }
  __syncthreads();
  // rank the columns by singular value (ascending, ties by larger index first so that the order is
  // the reverse of the descending one); the nbot smallest become unit vectors ub[j * nbot + rank]
  float* out_u = ub + (size_t)blockIdx.x * kPMax * kPMax;
  for (int k = tid >> 5; k < w; k += nt >> 5) {
    float sk = sig[k];
    int rank = 0;
    for (int q = tid & 31; q < w; q += 32) {
      float sq = sig[q];
      rank += (sq < sk) || (sq == sk && q > k);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
    if (rank < nbot) {
      float scale = sk > 0.f ? 1.f / sk : 0.f;
      for (int j = tid & 31; j < w; j += 32) out_u[j * nbot + rank] = C[k * ldc + j] * scale;
    }
  }
}

// Eq. 15 for the preselected tokens (see the file comment).  grid = (ceil(max M / 64), batch),
// 256 threads, one warp per token.  q / yn: the orthonormal basis Q (rows) and the block Y' = G Q^T,
// float32 [sum M_b, kPMax].  Requests without stage 2 get zeros.
// Dynamic shared memory: win_max * nbot_max floats.
__global__ void __launch_bounds__(256)
energy_kernel(const ReqPlan* __restrict__ plan, const float* __restrict__ q,
              const float* __restrict__ yn, const float* __restrict__ ub, float* __restrict__ energy) {
  extern __shared__ float sm_f[];
  ReqPlan rp = plan[blockIdx.y];
  const int row0 = blockIdx.x * 64;
  if (row0 >= rp.m) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nrows = min(64, rp.m - row0);
  if (!rp.stage2) {
    for (int i = tid; i < nrows; i += blockDim.x) energy[rp.presel_off + row0 + i] = 0.f;
    return;
  }
  const int p = rp.p, w = rp.win, w0 = p - w, nbot = p - rp.r;
  float* us = sm_f;                                     // [w][nbot]
  const float* usrc = ub + (size_t)blockIdx.y * kPMax * kPMax;
  for (int e = tid; e < w * nbot; e += blockDim.x) us[e] = usrc[e];
  __syncthreads();
  __shared__ float rowbuf[8][2 * kPMax];                 // this warp's rows of Y' and Q
  float* ys = rowbuf[warp];
  float* qs = ys + kPMax;
  for (int rr = warp; rr < nrows; rr += 8) {
    const float* yrow = yn + ((size_t)rp.presel_off + row0 + rr) * kPMax;
    const float* qrow = q + ((size_t)rp.presel_off + row0 + rr) * kPMax;
    // total over all p basis vectors; both rows are staged for the window sums
    float total = 0.f;
    __syncwarp();
    for (int c = lane; c < p; c += 32) {
      float yv = yrow[c], qv = qrow[c];
      ys[c] = yv; qs[c] = qv;
      total += yv * qv;
    }
    total = warp_sum(total);
    __syncwarp();
    // discarded Ritz pairs: lanes over k, window components broadcast from shared memory
    float sub_ = 0.f;
    for (int k = lane; k < nbot; k += 32) {
      float ya = 0.f, qa = 0.f;
      for (int j = 0; j < w; ++j) {
        float u = us[j * nbot + k];
        ya += ys[w0 + j] * u;
        qa += qs[w0 + j] * u;
      }
      sub_ += ya * qa;
    }
    sub_ = warp_sum(sub_);
    if (lane == 0) energy[rp.presel_off + row0 + rr] = fmaxf(total - sub_, 0.f);
  }
}

}  // namespace covspec
