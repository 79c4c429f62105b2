// The whole subspace iteration behind Eq. 14-15 in one persistent kernel.
//
// Work items are the 128-row tiles of the stage-2 requests (the same items and per-CTA lists as the
// power step had as a kernel of its own); every CTA walks its list once per multiplication by G.
// What used to be kernel boundaries are per-request counters in global memory:
//   arrive[b]   tiles of request b that have finished a step (their slab of the new block is in the
//               bf16 planes, their float64 partial Gram matrix is in `partial`); step k of a tile may
//               start loading the block once arrive[b] >= tiles(b) * k
//   factor[b]   number of triangular factors published for request b; the epilogue of step k needs
//               factor[b] >= k
//   ritz[b]     1 once the Rayleigh-Ritz vectors of the last block are published
//   last[b]     index of the request's last step: eig_iters on entry; the tile that factors step k
//               lowers it to k + 1 when the Ritz value estimates say that the energies will have
//               settled by then (see team_cholesky).  It only ever decreases and is written before
//               factor[b] = k + 1 is published: the epilogue of step k + 1, which waits for that
//               factor, reads "is this the last step?" with it, and the producer and MMA roles, which
//               only ask "is step s skipped?", can first be affected at step k + 2, whose start
//               every tile's arrival of step k + 1 precedes
//   summed[b]   tiles of request b that have added up their slice of the partial Gram matrices of a
//               step (only when every CTA holds exactly one tile, see spread_sum)
// With SMs to spare the grid carries one more CTA per request that holds no tile and only factors for
// that request (n_servers); otherwise
// the tile that makes arrive[b] reach tiles(b) * (k + 1) (an atomic ticket; nobody waits for it to be
// a particular CTA) sums the partial Gram matrices in tile order and factors the sum right there: a
// Cholesky factorisation after the first steps, the Rayleigh-Ritz solve of the window next to the cut
// after the last one.  All CTAs are resident at the same time (cooperative launch, one CTA per SM),
// every wait is bounded and a CTA that gives up raises a global abort word that ends the others'
// waits too.  After the last step every CTA evaluates the energies (Eq. 15) of its own tiles.
//
// Data that crosses CTAs inside the kernel (partial sums, factors, Ritz vectors, the float32 window
// columns, the bf16 planes the last step re-reads) is read with L1-bypassing loads; the operand
// tiles of the bf16 planes are read by TMA, behind a proxy fence.
#pragma once
#include "eig_kernels.cuh"

namespace covspec {
namespace sub {

constexpr int kSyncStride = 8;           // unsigned words per request: arrive, factor, ritz, last, summed

struct FusedParams {
  const ReqPlan* plan;
  int batch;
  int n_items;              // row tiles over all stage-2 requests
  int tile_rows;            // rows of a tile: 128, or 64 (the MMA still computes 128 rows; the upper half is dropped)
  const int* sched;         // [gridDim.x + 1] offsets, then the item lists of every CTA
  int steps;                // multiplications by G (eig_iters + 1, >= 2)
  float* lbuf;              // [batch][kLbufStride] triangular factor + reciprocal diagonal
  __nv_bfloat16* y_hi[2];   // plane buffers: step k reads [k & 1], writes [(k & 1) ^ 1]
  __nv_bfloat16* y_lo[2];
  int ld;
  float* yf[2];             // [sum M_b, kPMax], window columns only: the orthonormal basis Q of the block
                            // before the last multiplication, and the block after it (Eq. 15)
  double* partial;          // [tiles][kTileDoubles], see tile_offset
  float* ub;                // [batch][kPMax * kPMax] Ritz vectors of the discarded pairs
  float* energy;            // [sum M_b] (out)
  unsigned* sync;           // [batch][kSyncStride] counters (zero on entry), then the abort word
  int spread_sum;           // every CTA holds exactly one tile: the tiles of a request sum the partial matrices together
  int n_tile_ctas;          // CTAs that carry tiles: blockIdx.x < n_tile_ctas
  int n_servers;            // CTAs after those, one per stage-2 request, that only factor (0: the last tile to
                            // finish a step factors)
  int max_sweeps;
  float conv_tol;           // bound on the estimated energy error before NOCONVERGE is raised
  int early_stop;           // 1: requests whose estimate is far below conv_tol stop before `steps`
  int* status;
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() {
  asm volatile("fence.proxy.async;" ::: "memory");
}

constexpr uint32_t kFlagSpinLimit = 1u << 21;       // polls of ~100 ns: gives up after a fraction of a second

// One thread waits until *ctr >= target.  Returns false when the limit expired (raises the global
// abort word) or another CTA gave up.
__device__ __forceinline__ bool flag_wait_ge(const unsigned* ctr, unsigned target, unsigned* gabort,
                                             volatile int* abort_flag) {
  for (uint32_t i = 0; i < kFlagSpinLimit; ++i) {
    if (ld_acquire_u32(ctr) >= target) return true;
    if ((i & 15u) == 15u && (ld_acquire_u32(gabort) != 0u || *abort_flag)) { *abort_flag = 1; return false; }
    __nanosleep(64);
  }
  *abort_flag = 1;
  atomicExch(gabort, 1u);
  return false;
}

// One thread decides whether step `step` (>= 1) of a request runs, and waits until it can: returns
// 1 when every tile has finished step - 1 (run; *last_out = the request's last step as known now),
// 0 when the request's last step is before `step` (skip), -1 when the wait was given up.  `last` is
// examined before `arrive`: after the request's final step arrive reaches the count the skipped
// next step would wait for.
__device__ __forceinline__ int step_decide(const unsigned* sync_b, unsigned nt, int step, unsigned* gabort,
                                           volatile int* abort_flag, int* last_out) {
  for (uint32_t i = 0; i < kFlagSpinLimit; ++i) {
    const unsigned arrived = ld_acquire_u32(sync_b);
    const int last = (int)ld_acquire_u32(sync_b + 3);
    if (last < step) return 0;
    if (arrived >= nt * (unsigned)step) { *last_out = last; return 1; }
    if ((i & 15u) == 15u && (ld_acquire_u32(gabort) != 0u || *abort_flag)) { *abort_flag = 1; return -1; }
    __nanosleep(64);
  }
  *abort_flag = 1;
  atomicExch(gabort, 1u);
  return -1;
}

// Layout of a partial Gram matrix in global memory: the 8 x 8 tiles of the lower triangle, tile
// (I, J <= I) at tri_index(I, J) * 64, row-major inside (diagonal tiles hold all 64 entries) - the
// layout the blocked factorisation works on, so that summing the tiles' partial matrices is an
// element-wise sum of contiguous arrays.
constexpr int kTileDoubles = (kPMax / 8) * (kPMax / 8 + 1) / 2 * 64;      // 13440
__device__ __forceinline__ int tile_offset(int i, int j) {                 // i >= j
  return tri_index(i >> 3, j >> 3) * 64 + (i & 7) * 8 + (j & 7);
}
// One entry summed over the tiles of a request in tile order (L1-bypassing loads, 8 in flight).
__device__ __forceinline__ double gram_entry_cg(int ntile, const double* src) {
  double s = 0.0;
  for (int t0 = 0; t0 < ntile; t0 += 8) {
    double v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = __ldcg(src + (size_t)min(t0 + q, ntile - 1) * kTileDoubles);
#pragma unroll
    for (int q = 0; q < 8; ++q) s += t0 + q < ntile ? v[q] : 0.0;
  }
  return s;
}
// T[0 .. count) = sum over the request's tiles (tile order: deterministic) of their partial
// matrices; count a multiple of 64.  Coalesced 16-byte loads, 32 of them in flight per thread.
__device__ __forceinline__ void team_sum_partials(double* T, const double* pbase, int ntile, int count,
                                                  int tid, int nthreads) {
  const int pairs = count >> 1;
  if (ntile == 1) {
    // one matrix (already summed, or a one-tile request): a plain copy, eight loads in flight per thread
    const double2* src = reinterpret_cast<const double2*>(pbase);
    for (int e0 = tid; e0 < pairs; e0 += 8 * nthreads) {
      double2 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcg(src + min(e0 + u * nthreads, pairs - 1));
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (e0 + u * nthreads < pairs) reinterpret_cast<double2*>(T)[e0 + u * nthreads] = v[u];
    }
    return;
  }
  for (int e0 = tid; e0 < pairs; e0 += 4 * nthreads) {
    int e[4];
    double2 s[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      e[u] = e0 + u * nthreads < pairs ? e0 + u * nthreads : e0;
      s[u] = make_double2(0.0, 0.0);
    }
    for (int t0 = 0; t0 < ntile; t0 += 8) {
      double2 v[4][8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const double2* src = reinterpret_cast<const double2*>(pbase + (size_t)min(t0 + q, ntile - 1) * kTileDoubles);
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u][q] = __ldcg(src + e[u]);
      }
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (t0 + q < ntile) {
#pragma unroll
          for (int u = 0; u < 4; ++u) { s[u].x += v[u][q].x; s[u].y += v[u][q].y; }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (e0 + u * nthreads < pairs) reinterpret_cast<double2*>(T)[e0 + u * nthreads] = s[u];
  }
}

// 1 / sqrt(x) for x > 0 without a range test on the pivot chain: x = m 4^k with m in [1, 4) (integer
// operations on the exponent field), float32 estimate of 1 / sqrt(m) refined in float32 and by one
// Newton step in float64, then scaled by 2^-k.  Subnormal or non-finite x give a meaningless value;
// the caller clamps pivots to a positive floor first.
__device__ __forceinline__ double rsqrt_f64_scaled(double x) {
  const int hi = __double2hiint(x), lo = __double2loint(x);
  const int k = ((((hi >> 20) & 0x7ff) - 1023)) >> 1;
  const double m = __hiloint2double(hi - (k << 21), lo);
  const float xf = (float)m;
  float yf = rsqrtf(xf);
  yf = yf * (1.5f - 0.5f * xf * yf * yf);
  double y = (double)yf;
  const double e = fma(-0.5 * m * y, y, 0.5);
  y = fma(y, e, y);
  return __hiloint2double(__double2hiint(y) - (k << 20), __double2loint(y));
}

// Diagonal 8 x 8 tile, factored by one thread in registers: measured faster than a lane-per-row
// version (64-bit shuffles cost more than the arithmetic they save).  Two columns at a time: for the
// leading 2 x 2 block [[al, be], [be, ga]] the factor is l11 = sqrt(al), l21 = be / l11,
// l22 = sqrt(de / al) with de = al ga - be^2, so the two reciprocal square roots (of al and de) run
// side by side instead of one after the other.  The chain of dependent pivots is the critical path
// of the whole factorisation.  A pivot below 1e-12 of its original diagonal entry (a numerically
// dependent direction) is clamped there; the next multiplication by G restores the direction.
__device__ __forceinline__ void factor_diag_thread(double* D, const double* d0, double* rd) {
  double a[8][8];
#pragma unroll
  for (int l = 0; l < 8; ++l)
#pragma unroll
    for (int m = 0; m <= l; ++m) a[l][m] = D[l * 8 + m];
#pragma unroll
  for (int c = 0; c < 8; c += 2) {
    const double f0 = 1e-12 * d0[c], f1 = 1e-12 * d0[c + 1];
    double al = a[c][c];
    if (!(al > f0)) al = f0 > 0.0 ? f0 : 1.0;
    const double be = a[c + 1][c], ga = a[c + 1][c + 1];
    double de = fma(al, ga, -be * be);                  // al * (second pivot)
    const double fd = f1 * al;
    if (!(de > fd)) de = fd > 0.0 ? fd : al;
    const double ra = rsqrt_f64_scaled(al), rq = rsqrt_f64_scaled(de);
    const double l11 = al * ra, l21 = be * ra, inv22 = rq * l11, l22 = de * rq * ra;
    a[c][c] = l11; a[c + 1][c] = l21; a[c + 1][c + 1] = l22;
    rd[c] = ra; rd[c + 1] = inv22;
#pragma unroll
    for (int l = c + 2; l < 8; ++l) {
      const double x1 = a[l][c] * ra;
      a[l][c + 1] = (a[l][c + 1] - x1 * l21) * inv22;
      a[l][c] = x1;
    }
#pragma unroll
    for (int l = c + 2; l < 8; ++l)
#pragma unroll
      for (int m = c + 2; m <= l; ++m) a[l][m] -= a[l][c] * a[m][c] + a[l][c + 1] * a[m][c + 1];
  }
#pragma unroll
  for (int l = 0; l < 8; ++l)
#pragma unroll
    for (int m = 0; m <= l; ++m) D[l * 8 + m] = a[l][m];
}

// The matrix is already in T (tile layout, see tile_offset); entries beyond n inside the last row of
// tiles are replaced by the identity here.
//   store(I, J, tile, rd)   receives the factor tile (I, J) (64 doubles, row-major) and the array of
//                           reciprocal diagonal entries; called by a whole warp
// kEarlyStore: warp 4 (idle in the panel loop) hands panel J - 1 to store() during iteration J (the
// panel is final since the last barrier) instead of leaving all tiles to the end; the team then has
// at least five warps.
template <bool kEarlyStore = false, typename Store, typename Sync>
__device__ __forceinline__ void cholesky_blocked_team(int n, double* T, double* aux, int tid, int nthreads,
                                                      Store store, Sync sync) {
  const int lane = tid & 31, warp = tid >> 5, nw = nthreads >> 5;
  const int nb = (n + 7) >> 3, ntile = nb * (nb + 1) / 2;
  double* d0 = aux;                 // original diagonal
  double* rd = aux + 8 * nb;        // 1 / L[j][j]
  // identity padding of rows / columns n .. 8 nb - 1 (last row of tiles), then the diagonal
  for (int e = tid; e < nb * 64; e += nthreads) {
    const int J = e >> 6, i = 8 * (nb - 1) + ((e >> 3) & 7), j = 8 * J + (e & 7);
    if (i >= n || j >= n) T[tri_index(nb - 1, J) * 64 + (e & 63)] = (i == j) ? 1.0 : 0.0;
  }
  sync();
  for (int i = tid; i < 8 * nb; i += nthreads) d0[i] = T[tile_offset(i, i)];
  sync();
  const int fr = lane >> 2, fk = lane & 3;
  auto update_tile = [&](int J, int I, int K) {
    const double* XI = T + tri_index(I, J) * 64 + fr * 8 + fk;
    const double* XK = T + tri_index(K, J) * 64 + fr * 8 + fk;
    double* C = T + tri_index(I, K) * 64 + fr * 8 + 2 * fk;
    double c0 = C[0], c1 = C[1];
    dmma_8x8x4(c0, c1, -XI[0], XK[0]);
    dmma_8x8x4(c0, c1, -XI[4], XK[4]);
    C[0] = c0; C[1] = c1;
  };
  // row `i` of the tile (I, J) <- row * L_JJ^-T (forward substitution over the 8 columns)
  auto solve_row = [&](int J, int i) {
    const double* D = T + tri_index(J, J) * 64;
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
  };
  auto update_tile2 = [&](int J, int Ia, int Ka, int Ib, int Kb) {
    const double* XIa = T + tri_index(Ia, J) * 64 + fr * 8 + fk;
    const double* XKa = T + tri_index(Ka, J) * 64 + fr * 8 + fk;
    const double* XIb = T + tri_index(Ib, J) * 64 + fr * 8 + fk;
    const double* XKb = T + tri_index(Kb, J) * 64 + fr * 8 + fk;
    double* Ca = T + tri_index(Ia, Ka) * 64 + fr * 8 + 2 * fk;
    double* Cb = T + tri_index(Ib, Kb) * 64 + fr * 8 + 2 * fk;
    double a0 = Ca[0], a1 = Ca[1], b0 = Cb[0], b1 = Cb[1];
    const double xa0 = -XIa[0], xa4 = -XIa[4], xb0 = -XIb[0], xb4 = -XIb[4];
    const double ka0 = XKa[0], ka4 = XKa[4], kb0 = XKb[0], kb4 = XKb[4];
    dmma_8x8x4(a0, a1, xa0, ka0);
    dmma_8x8x4(b0, b1, xb0, kb0);
    dmma_8x8x4(a0, a1, xa4, ka4);
    dmma_8x8x4(b0, b1, xb4, kb4);
    Ca[0] = a0; Ca[1] = a1; Cb[0] = b0; Cb[1] = b1;
  };
  if (tid == 0) factor_diag_thread(T, d0, rd);
  sync();
  // One barrier of the whole team per 8-column panel.  The chain that bounds the factorisation -
  // panel J's diagonal tile -> tile (J+1, J) -> its update of tile (J+1, J+1) -> that tile's eight
  // dependent pivots - runs on warp 0 alone; the warps of the other three schedulers (the FP64 pipe
  // is per scheduler: warp w issues on scheduler w & 3, so warp 4 stays idle) solve the rest of the
  // panel and update the rest of the trailing matrix meanwhile.  They need tile (J+1, J) for the
  // tiles of column J+1: warp 0 arrives on barrier 4 once it is solved.
  const bool bulk = (warp & 3) != 0;
  const int nbulk = nw - (nw + 3) / 4, me = warp - (warp >> 2) - 1;          // bulk warps, in order
  const int bulk_threads = nbulk * 32, btid = me * 32 + lane;
  for (int J = 0; J + 1 < nb; ++J) {
    if (warp == 0) {
      if (lane < 8) solve_row(J, 8 * (J + 1) + lane);
      __syncwarp();
      asm volatile("bar.arrive 4, %0;" ::"r"(bulk_threads + 32) : "memory");
      update_tile(J, J + 1, J + 1);
      __syncwarp();
      if (lane == 0) factor_diag_thread(T + tri_index(J + 1, J + 1) * 64, d0 + 8 * (J + 1), rd + 8 * (J + 1));
      __syncwarp();
    } else if (bulk) {
      for (int i = 8 * (J + 2) + btid; i < 8 * nb; i += bulk_threads) solve_row(J, i);
      asm volatile("bar.sync 4, %0;" ::"r"(bulk_threads + 32) : "memory");
      // tiles (I, K), J+1 <= K <= I, I >= J+2, dealt one by one to the bulk warps (row-major
      // order); two tiles at a time so that their tensor-core instructions overlap
      int I = J + 2, K = J + 1 + me;
      auto settle = [&]() { while (I < nb && K > I) { K -= I - J; ++I; } };
      settle();
      while (I < nb) {
        const int I1 = I, K1 = K;
        K += nbulk; settle();
        if (I < nb) {
          update_tile2(J, I1, K1, I, K);
          K += nbulk; settle();
        } else {
          update_tile(J, I1, K1);
        }
      }
    } else if (kEarlyStore && warp == 4 && J >= 1) {
      for (int I = J - 1; I < nb; ++I) store(I, J - 1, T + tri_index(I, J - 1) * 64, rd);
    }
    sync();
  }
  if constexpr (kEarlyStore) {
    // the last two panels (or the only one)
    int t = 0;
    for (int J = nb >= 2 ? nb - 2 : 0; J < nb; ++J)
      for (int I = J; I < nb; ++I, ++t)
        if (t % nw == warp) store(I, J, T + tri_index(I, J) * 64, rd);
  } else {
    for (int t = warp; t < ntile; t += nw) {
      int I, J;
      tri_decode(t, I, J);
      store(I, J, T + t * 64, rd);
    }
  }
}

constexpr int kEpiThreads = 256;         // warps 0-7

// Writes the accumulated 8 x 8 tiles of one warp unit (see gram_unit_accumulate) to the tile layout;
// t0 = index of the first tile row / column the unit's coordinates are relative to.
__device__ __forceinline__ void gram_unit_store_tiles(const GramAcc& acc, int ta, int tz, int t0, int lane,
                                                      double* __restrict__ out) {
  const int fr = lane >> 2, fk = lane & 3;
#pragma unroll
  for (int u = 0; u <= kMaxTiles8; ++u) {
    int strip = -1, tb = 0;
    if (u < kMaxTiles8 && u <= ta) { strip = ta; tb = u; }
    else if (u >= 1 && kMaxTiles8 - u <= tz && tz != ta) { strip = tz; tb = kMaxTiles8 - u; }
    if (strip < 0) continue;
    *reinterpret_cast<double2*>(out + tri_index(t0 + strip, t0 + tb) * 64 + fr * 8 + 2 * fk) =
        make_double2(acc.a[u][0], acc.a[u][1]);
  }
}

// 8 x 8 tiles of the partial Gram matrix that do not fit the eight warp units (see the kernel): the
// strips ta = u and tz = nb8 - 1 - u of the units u = 8 .. units - 1, listed strip by strip.
// nb8 <= 20 leaves at most 2 units = 42 tiles, six per warp.
constexpr int kExtraTiles = 6;
__device__ __forceinline__ bool extra_tile(int e, int nb8, int units, int& ta, int& tb) {
  for (int u = 8; u < units; ++u) {
    const int a = u, z = nb8 - 1 - u;
    if (e <= a) { ta = a; tb = e; return true; }
    e -= a + 1;
    if (z != a) {
      if (e <= z) { ta = z; tb = e; return true; }
      e -= z + 1;
    }
  }
  return false;
}


// ---- work of the tile that finishes a step last (all 256 epilogue threads) ----------------------
// Kept out of line: the tile epilogue is register-bound, and these run once per request and step.

// Cholesky factor of the summed Gram matrix, written in the layout the triangular solve reads
// (see lt_row_offset) followed by the reciprocal diagonal.  Tm: cholesky_smem_bytes(p) of scratch.
// Returns (to every thread) whether the next step may be the last one: from the diagonal of
// the summed Gram matrix B = Y'^T Y' (theta_i = sqrt(B_ii) estimates the i-th eigenvalue of G once the
// basis has started to order itself) the energy error after q_final multiplications is predicted as
// max_i 2 (theta_i / theta_1) (theta_min / theta_i)^q_final over the kept directions i < r that the
// cut can tell apart from the discarded ones (theta_i - theta_min > 1e-3 theta_1), the estimate
// team_ritz reports at the end; stop_below is the bound it has to stay under (0: never stop early).
// pad: also write the entries of the layout that no factor touches (the first factorisation of a
// launch does; they stay as they are for the later ones).
__device__ __noinline__ bool team_cholesky(const double* pbase, int nt, int p, int r, float* out, double* Tm,
                                           float* dg, volatile int* s_word, int q_final, float stop_below,
                                           bool pad) {
  const int et = threadIdx.x, warp = et >> 5, lane = et & 31;
  const int P = (p + 7) & ~7, nb = (p + 7) >> 3;
  auto epi_sync = [&]() { named_barrier(1, kEpiThreads); };
  // identity padding of the layout rows / columns p .. P-1 and the entries left of the diagonal
  for (int i = warp; pad && i < P; i += 8) {
    int j0 = i & ~3;
    float* row = out + lt_row_offset(i, P) - j0;
    for (int j = j0 + lane; j < P; j += 32)
      if (j < i || i >= p || j >= p) row[j] = (i == j) ? 1.f : 0.f;
  }
  for (int j = p + et; pad && j < P; j += kEpiThreads) out[kLtFloats + j] = 1.f;
  team_sum_partials(Tm, pbase, nt, nb * (nb + 1) / 2 * 64, et, kEpiThreads);
  epi_sync();
  if (stop_below > 0.f) {
    for (int i = et; i < p; i += kEpiThreads) dg[i] = sqrtf(fmaxf((float)Tm[tile_offset(i, i)], 0.f));
    if (et == 0) *s_word = 0;
    epi_sync();
    if (warp == 0) {
      float tmin = 3.0e38f, tmax = 0.f;
      for (int i = lane; i < p; i += 32) { tmin = fminf(tmin, dg[i]); tmax = fmaxf(tmax, dg[i]); }
      tmin = warp_min(tmin); tmax = warp_max(tmax);
      float worst = 0.f;
      for (int i = lane; i < r; i += 32) {
        float th = dg[i];
        if (th - tmin > 1e-3f * tmax && th > 0.f) worst = fmaxf(worst, 2.f * (th / tmax) * __powf(tmin / th, (float)q_final));
      }
      worst = warp_max(worst);
      if (lane == 0 && tmax > 0.f && worst < stop_below) *s_word = 1;
    }
    epi_sync();
  }
  const bool stop = stop_below > 0.f && *s_word != 0;
  // row j of the layout holds L[i][j] for i >= (j & ~3): lane -> (j, half of the tile's rows), so that
  // a lane's four entries are consecutive floats
  auto store = [&](int I, int J, const double* tile, const double* rd) {
    const int jl = lane >> 2, i0 = (lane & 3) * 2;
    const int j = 8 * J + jl;
    if (j < p) {
      float* dst = out + lt_row_offset(j, P) - (j & ~3);
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int i = 8 * I + i0 + q;
        if (i < p && i >= j) dst[i] = (float)tile[(i0 + q) * 8 + jl];
      }
      if (I == J && (lane & 3) == 0) out[kLtFloats + j] = (float)rd[j];
    }
  };
  cholesky_blocked_team<true>(p, Tm, Tm + (size_t)nb * (nb + 1) / 2 * 64, et, kEpiThreads, store, epi_sync);
  return stop;
}

// Rayleigh-Ritz on the window next to the cut (see eig_kernels.cuh) and the convergence estimate.
// C: ritz_smem_bytes(w) of scratch; dg: p floats of scratch.
__device__ __noinline__ void team_ritz(const double* pbase, int nt, int p, int w, int r, int m, float* out_u,
                                       float* C, float* dg, float* s_scale, int* s_flag, int max_sweeps,
                                       float conv_tol, int steps, int* status) {
  const int et = threadIdx.x, warp = et >> 5, lane = et & 31;
  auto epi_sync = [&]() { named_barrier(1, kEpiThreads); };
  const int w0 = p - w, nbot = p - r;
  const int ldc = ritz_ldc(w);
  float* sig = C + (size_t)w * ldc;
  for (int e = et; e < w * ldc; e += kEpiThreads) C[e] = 0.f;
  if (et == 0) *s_scale = 0.f;
  epi_sync();
  {
    float mx = 0.f;
    for (int i = et; i < p; i += kEpiThreads) {
      float v = (float)gram_entry_cg(nt, pbase + tile_offset(i, i));
      dg[i] = sqrtf(fmaxf(v, 0.f));                      // sqrt of the diagonal of B'
      mx = fmaxf(mx, v);
    }
    mx = warp_max(mx);
    if (lane == 0 && mx > 0.f) atomicMax(reinterpret_cast<int*>(s_scale), __float_as_int(mx));
  }
  {
    // the window block of B' (rows / columns w0 .. p-1), gathered into a tile layout of its own
    const int nbw = (w + 7) >> 3, cnt = nbw * (nbw + 1) / 2 * 64;
    double* Tw = reinterpret_cast<double*>(C + (((size_t)w * ldc + w + 1) & ~(size_t)1));
    for (int e = et; e < cnt; e += kEpiThreads) {
      int I, J;
      tri_decode(e >> 6, I, J);
      int i = 8 * I + ((e >> 3) & 7), j = 8 * J + (e & 7);
      double v = 0.0;
      if (i < w && j < w) v = gram_entry_cg(nt, pbase + tile_offset(w0 + max(i, j), w0 + min(i, j)));
      Tw[e] = v;
    }
    epi_sync();
    auto store = [&](int I, int J, const double* tile, const double*) {
      for (int q = lane; q < 64; q += 32) {
        const int i = 8 * I + (q >> 3), j = 8 * J + (q & 7);
        if (i < w && j <= i) C[j * ldc + i] = (float)tile[q];
      }
    };
    cholesky_blocked_team(w, Tw, Tw + (size_t)cnt, et, kEpiThreads, store, epi_sync);
  }
  epi_sync();
  const float s1 = sqrtf(*s_scale);
  if (conv_tol > 0.f && p < m) {
    // Has the iteration settled?  The basis vectors converge to eigenvectors in order, so
    // theta_k ~ sqrt(B'_kk) estimates the k-th eigenvalue of G and theta_min the first one left
    // out of the basis.  After q multiplications a kept direction k still carries about
    // (theta_min / theta_k)^q of the directions outside the basis, which moves the energies by
    // about 2 theta_k (theta_min / theta_k)^q; relative to the scale theta_1 of the energies, and
    // only for directions that the cut can tell apart from the discarded ones (more than
    // 1e-3 theta_1 above theta_min; closer ones may mix freely, Eq. 15 is not unique there).
    float tmin = 3.0e38f;
    for (int i = lane; i < p; i += 32) tmin = fminf(tmin, dg[i]);
    tmin = warp_min(tmin);
    float worst = 0.f;
    for (int i = et; i < r; i += kEpiThreads) {
      float th = dg[i];
      if (th - tmin > 1e-3f * s1 && th > 0.f)
        worst = fmaxf(worst, 2.f * (th / s1) * __powf(tmin / th, (float)steps));
    }
    worst = warp_max(worst);
    if (lane == 0 && worst > conv_tol) atomicOr(status, kStatusNoConverge);
  }
  const int nact = min(kEpiThreads, ((((w + 1) >> 1) * 4) + 31) & ~31);
  if (et == 0) *s_flag = 0;
  epi_sync();
  if (et < nact) {
    bool converged;
    if (w <= 32) converged = jacobi_sweeps<8>(C, ldc, w, s1, max_sweeps, nact, s_flag);
    else if (w <= 64) converged = jacobi_sweeps<16>(C, ldc, w, s1, max_sweeps, nact, s_flag);
    else if (w <= 96) converged = jacobi_sweeps<24>(C, ldc, w, s1, max_sweeps, nact, s_flag);
    else converged = jacobi_sweeps<(kPMax + 3) / 4>(C, ldc, w, s1, max_sweeps, nact, s_flag);
    if (!converged && et == 0) atomicOr(status, kStatusNoConverge);
  }
  named_barrier(3, kEpiThreads);
  for (int k = warp; k < w; k += 8) {
    float sm = 0.f;
    for (int row = lane; row < w; row += 32) { float x = C[k * ldc + row]; sm += x * x; }
    sm = warp_sum(sm);
    if (lane == 0) sig[k] = sqrtf(sm);
  }
  epi_sync();
  // rank the columns by singular value (ascending, ties by larger index first); the nbot smallest
  // become unit vectors out_u[j * nbot + rank]
  for (int k = warp; k < w; k += 8) {
    float sk = sig[k];
    int rank = 0;
    for (int q = lane; q < w; q += 32) {
      float sq = sig[q];
      rank += (sq < sk) || (sq == sk && q > k);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
    if (rank < nbot) {
      float scale = sk > 0.f ? 1.f / sk : 0.f;
      for (int j = lane; j < w; j += 32) out_u[j * nbot + rank] = C[k * ldc + j] * scale;
    }
  }
}

__global__ void __launch_bounds__(kPowThreads, 1)
subspace_kernel(const __grid_constant__ CUtensorMap map_gh, const __grid_constant__ CUtensorMap map_gl,
                const __grid_constant__ CUtensorMap map_y0h, const __grid_constant__ CUtensorMap map_y0l,
                const __grid_constant__ CUtensorMap map_y1h, const __grid_constant__ CUtensorMap map_y1l,
                const FusedParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  float* xs = reinterpret_cast<float*>(smem);                       // aliases the ring after the MMAs
  float* xq = reinterpret_cast<float*>(smem + kXsBytes);            // previous block (last step)
  float* lt = reinterpret_cast<float*>(smem + kPowRegion);
  float* dinv = lt + kLtFloats;
  uint64_t* bars = reinterpret_cast<uint64_t*>(lt + kLbufStride);
  uint64_t* full = bars;                 // [2]
  uint64_t* empty = bars + 2;            // [2]
  uint64_t* acc_full = bars + 4;
  uint64_t* acc_empty = bars + 5;
  uint64_t* epi_done = bars + 6;         // the region no longer belongs to the epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_word = reinterpret_cast<volatile int*>(tmem_slot + 2);      // [2] broadcast slots of the epilogue
  int* s_flag = reinterpret_cast<int*>(tmem_slot + 4);                        // Jacobi rotation flag
  float* s_scale = reinterpret_cast<float*>(tmem_slot + 5);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned* gabort = prm.sync + (size_t)prm.batch * kSyncStride;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPowStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 128);
    mbar_init(epi_done, kEpiThreads);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(tmem_slot, kPowTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int s_begin = prm.sched[blockIdx.x], s_end = prm.sched[blockIdx.x + 1];
  const int* s_items = prm.sched + gridDim.x + 1;
  const int last_step = prm.steps - 1;
  const int R = prm.tile_rows;
  auto decode = [&](int item, int& b, ReqPlan& rp, int& tile) {
    b = find_request(item, prm.batch, [&](int q) { return prm.plan[q].ptile_off; });
    rp = prm.plan[b];
    tile = item - rp.ptile_off;
  };

  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0, n = 0;
      bool ok = true;
      for (int step = 0; step <= last_step && ok; ++step) {
        const CUtensorMap* myh = (step & 1) ? &map_y1h : &map_y0h;
        const CUtensorMap* myl = (step & 1) ? &map_y1l : &map_y0l;
        for (int si = s_begin; si < s_end && ok; ++si, ++n) {
          const int item = s_items[si];
          int b, tile; ReqPlan rp;
          decode(item, b, rp, tile);
          if (step > 0) {
            // every tile of the request has written its slab of the block this step multiplies,
            // unless the request has already had its last step
            const unsigned nt = (unsigned)((rp.m + R - 1) / R);
            int last_b;
            const int go = step_decide(prm.sync + (size_t)b * kSyncStride, nt, step, gabort, abort_flag, &last_b);
            if (go < 0) { ok = false; break; }
            if (go == 0) { --n; continue; }
            fence_proxy_async_all();
          }
          // the previous item's staged block (and whatever its last tile factored) lives in the
          // ring until its epilogue is done
          if (n > 0 && !(ok = mbar_wait(epi_done, (n - 1) & 1u, abort_flag))) break;
          int k_chunks = (rp.m + kBK - 1) / kBK;
          for (int kc = 0; kc < k_chunks; ++kc, ++it) {
            int s = it % kPowStages;
            if (!(ok = mbar_wait(&empty[s], ((it / kPowStages) & 1u) ^ 1u, abort_flag))) break;
            mbar_expect_tx(&full[s], kPowStageBytes);
            uint32_t dst = smem_u32(smem + s * kPowStageBytes);
            int grow = rp.presel_off + tile * R;
            tma_load_2d(dst, &map_gh, kc * kBK, grow, &full[s]);
            tma_load_2d(dst + kPowBytesA, &map_gl, kc * kBK, grow, &full[s]);
            tma_load_2d(dst + 2 * kPowBytesA, myh, kc * kBK, b * kPMax, &full[s]);
            tma_load_2d(dst + 2 * kPowBytesA + kPowBytesB, myl, kc * kBK, b * kPMax, &full[s]);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, n = 0;
      bool ok = true;
      for (int step = 0; step <= last_step && ok; ++step) {
        for (int si = s_begin; si < s_end && ok; ++si, ++n) {
          const int item = s_items[si];
          int b, tile; ReqPlan rp;
          decode(item, b, rp, tile);
          const uint32_t idesc = umma_idesc(kTile, (rp.p + 15) & ~15);
          if (step > 0) {
            const unsigned nt = (unsigned)((rp.m + R - 1) / R);
            int last_b;
            const int go = step_decide(prm.sync + (size_t)b * kSyncStride, nt, step, gabort, abort_flag, &last_b);
            if (go < 0) { ok = false; break; }
            if (go == 0) { --n; continue; }
          }
          if (!(ok = mbar_wait(acc_empty, (n & 1u) ^ 1u, abort_flag))) break;
          tc_fence_after();
          int k_chunks = (rp.m + kBK - 1) / kBK;
          for (int kc = 0; kc < k_chunks; ++kc, ++it) {
            int s = it % kPowStages;
            if (!(ok = mbar_wait(&full[s], (it / kPowStages) & 1u, abort_flag))) break;
            tc_fence_after();
            uint32_t base = smem_u32(smem + s * kPowStageBytes);
            // T += G_hi Y_hi + G_lo Y_hi + G_hi Y_lo
#pragma unroll
            for (int term = 0; term < 3; ++term) {
              uint64_t adesc = umma_desc(base + (term == 1 ? kPowBytesA : 0));
              uint64_t bdesc = umma_desc(base + 2 * kPowBytesA + (term == 2 ? kPowBytesB : 0));
#pragma unroll
              for (int k = 0; k < kBK / 16; ++k)
                umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (kc | term | k) != 0);
            }
            umma_commit(&empty[s]);
          }
          if (!ok) break;
          umma_commit(acc_full);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue, warps 0-7
    const int et = threadIdx.x;                    // 0 .. 255
    const int r = (warp & 3) * 32 + lane;          // TMEM lane = row of the tile (warps 0-3 solve)
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    auto epi_sync = [&]() { named_barrier(1, kEpiThreads); };
    // thread 0 waits for a counter; everybody learns the outcome
    auto team_wait = [&](const unsigned* ctr, unsigned target) -> bool {
      epi_sync();
      if (et == 0) *s_word = flag_wait_ge(ctr, target, gabort, abort_flag) ? 1 : 0;
      epi_sync();
      return *s_word != 0;
    };
    uint32_t n = 0;
    int cached_b = -1, cached_step = -1;
    bool ok = true;
    // Factors the summed Gram matrix of request b after step `step` (Cholesky, or the Rayleigh-Ritz
    // solve after the last step) and publishes the result; returns whether the next step was
    // declared the last one.  Uses the operand ring as scratch.
    auto factor_request = [&](int b, const ReqPlan& rp, unsigned* sync_b, int step, bool is_last, int last_b,
                              int nt_sum) -> bool {
      __threadfence();
      const int p = rp.p;
      const double* pbase = prm.partial + (size_t)rp.ptile_off * kTileDoubles;
      double* Tm = reinterpret_cast<double*>(smem);        // the region is free: every thread passed the barrier
      bool stop = false;
      if (!is_last) {
        // after the second multiplication and later: may the next step be the last one?  (asked with a
        // margin of 8 under the tolerance, 64 at the first opportunity: the estimate is rough while
        // the basis is still mixing)
        const bool may_stop = prm.early_stop && step >= 1 && step + 1 < last_b && p < rp.m;
        const float margin = step == 1 ? 0.015625f : 0.125f;
        stop = team_cholesky(pbase, nt_sum, p, rp.r, prm.lbuf + (size_t)b * kLbufStride, Tm, dinv,
                             s_word, step + 2, may_stop ? margin * prm.conv_tol : 0.f, step == 0);
        __threadfence();
        epi_sync();
        if (et == 0) {
          if (stop) st_release_u32(sync_b + 3, (unsigned)(step + 1));
          st_release_u32(sync_b + 1, (unsigned)(step + 1));
        }
      } else {
        team_ritz(pbase, nt_sum, p, rp.win, rp.r, rp.m, prm.ub + (size_t)b * kPMax * kPMax, reinterpret_cast<float*>(smem), lt,
                  s_scale, s_flag, prm.max_sweeps, prm.conv_tol, step + 1, prm.status);
        __threadfence();
        epi_sync();
        if (et == 0) st_release_u32(sync_b + 2, 1u);
      }
      return stop;
    };
    if (prm.n_servers > 0 && (int)blockIdx.x >= prm.n_tile_ctas) {
      // ------------------------------------------------------------ factor server
      // This CTA carries no tile.  It factors for one request: on a CTA that also carries a tile the
      // factorisation, which needs the operand ring as scratch, would delay that tile's next
      // multiplication, and with it the request's next step.
      const int mine = (int)blockIdx.x - prm.n_tile_ctas;
      int b = -1, seen = 0;
      for (int q = 0; q < prm.batch && b < 0; ++q)
        if (prm.plan[q].stage2) { if (seen == mine) b = q; ++seen; }
      if (b >= 0) {
        const ReqPlan rp = prm.plan[b];
        unsigned* sync_b = prm.sync + (size_t)b * kSyncStride;
        const unsigned nt = (unsigned)((rp.m + R - 1) / R);
        const bool summed = prm.spread_sum && nt >= 4;      // the tiles have added up the partial matrices
        int last_b = last_step;
        for (int step = 0; step <= last_b; ++step) {
          if (!team_wait(summed ? sync_b + 4 : sync_b, nt * (unsigned)(step + 1))) break;
          if (factor_request(b, rp, sync_b, step, step == last_b, last_b, summed ? 1 : (int)nt)) last_b = step + 1;
        }
      }
    }
    for (int step = 0; step <= last_step; ++step) {
      const bool identity = step == 0;
      __nv_bfloat16* y_hi = prm.y_hi[(step & 1) ^ 1];
      __nv_bfloat16* y_lo = prm.y_lo[(step & 1) ^ 1];
      for (int si = s_begin; si < s_end; ++si, ++n) {
        const int item = s_items[si];
        int b, tile; ReqPlan rp;
        decode(item, b, rp, tile);
        const int p = rp.p, P = (p + 7) & ~7;
        unsigned* sync_b = prm.sync + (size_t)b * kSyncStride;
        const unsigned nt = (unsigned)((rp.m + R - 1) / R);
        // does the request still run this step, and is it its last one?  (one answer for the team)
        int last_b = last_step;
        if (!identity) {
          epi_sync();
          if (et == 0) {
            int lb = last_step;
            const int go = step_decide(sync_b, nt, step, gabort, abort_flag, &lb);
            s_word[0] = go; s_word[1] = lb;
          }
          epi_sync();
          const int go = s_word[0];
          last_b = s_word[1];
          if (go == 0) { --n; continue; }
          if (go < 0) ok = false;
        }
        if (!identity && (b != cached_b || step != cached_step)) {
          // the factor of the previous block, published by whichever tile finished that step last
          ok = team_wait(sync_b + 1, (unsigned)step) && ok;
          if (ok) {
            const float4* src = reinterpret_cast<const float4*>(prm.lbuf + (size_t)b * kLbufStride);
            float4* dst = reinterpret_cast<float4*>(lt);
            int n4 = (lt_row_offset(P, P) + 3) / 4;    // floats used by the P-wide layout
            for (int e = et; e < n4; e += kEpiThreads) dst[e] = __ldcg(src + e);
            const float* dsrc = prm.lbuf + (size_t)b * kLbufStride + kLtFloats;
            for (int e = et; e < P; e += kEpiThreads) dinv[e] = __ldcg(dsrc + e);
          }
          epi_sync();
          cached_b = b; cached_step = step;
        }
        // whether this is the request's last step is known once the previous step's factor has been
        // published: the tile that computed it may have declared this step the last one
        if (!identity) {
          if (et == 0) s_word[1] = (int)ld_acquire_u32(sync_b + 3);
          epi_sync();
          last_b = s_word[1];
          epi_sync();
        }
        const bool is_last = step == last_b;
        float* yf = is_last ? prm.yf[1] : nullptr;
        float* qprev = is_last ? prm.yf[0] : nullptr;
        const int nrows = min(R, rp.m - tile * R);
        // ---- Y_next row = T row * L^-T (forward substitution per row), staged as xs[c][r] ----
        // Between the first and the last step two threads share a row: warps 0-3 own the 32-column
        // super-block S being solved (contributions of the previous super-block and of its own
        // columns), warps 4-7 run one super-block ahead and sum what the columns before that
        // contribute to super-block S + 1 (hs, double-buffered behind the staged block).
        const bool split = !identity && !is_last;
        const int nS = (P + 31) >> 5;
        float* hs = reinterpret_cast<float*>(smem + kXsBytes);          // [2][32][kXsLd]
        if (warp < 4) {
          ok = ok && mbar_wait(acc_full, n & 1u, abort_flag);
          tc_fence_after();
        }
        const bool row_ok = r < nrows;
        // warps whose 32 rows all lie beyond the tile's rows (64-row tiles, ragged last tiles), and
        // their helpers, have nothing to solve; they keep taking part in the barriers.  Their rows
        // of the staged block stay unwritten and are not read below.
        const bool active = (warp & 3) * 32 < nrows;
#pragma unroll 1
        for (int S = 0; S < nS; ++S) {
          if (warp < 4) {
            if (active) {
            float v[32];
            tmem_ld32(t_lane + S * 32, v);
            const float* hcur = hs + (S & 1) * 32 * kXsLd;
#pragma unroll
            for (int sb = 0; sb < 4; ++sb) {
              const int jb = S * 32 + sb * 8;
              if (jb < P) {
                float acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = v[sb * 8 + e];
                if (!identity) {
                  int g0 = 0;
                  if (split && S >= 2) {
                    g0 = 8 * (S - 1);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] += hcur[(sb * 8 + e) * kXsLd + r];
                  }
                  solve_apply_groups(acc, jb, g0, jb >> 2, smem_u32(lt), smem_u32(xs), r, P);
                  solve_inblock8(acc, jb, smem_u32(lt), smem_u32(dinv), P);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) xs[(jb + e) * kXsLd + r] = (row_ok && ok) ? acc[e] : 0.f;
              }
            }
            }
          } else if (active && split && S >= 1 && S + 1 < nS) {
            // minus the contributions of the columns before 32 S to super-block S + 1
            float* hnext = hs + ((S + 1) & 1) * 32 * kXsLd;
#pragma unroll 1
            for (int sb = 0; sb < 4; ++sb) {
              const int jb = (S + 1) * 32 + sb * 8;
              if (jb < P) {
                float acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                solve_apply_groups(acc, jb, 0, 8 * S, smem_u32(lt), smem_u32(xs), r, P);
#pragma unroll
                for (int e = 0; e < 8; ++e) hnext[(sb * 8 + e) * kXsLd + r] = acc[e];
              }
            }
          }
          if (split) epi_sync();
        }
        if (warp < 4) {
          tc_fence_before();
          mbar_arrive(acc_empty);
        } else if (is_last) {
          // ---- last step, warps 4-7: rows of Q = Y L^-T for the previous block Y, in place ----
          ok = ok && mbar_wait(acc_full, n & 1u, abort_flag);      // the ring is no longer read
          const int t4 = et - 128;
          float* qrows = qprev + ((size_t)rp.presel_off + tile * R) * kPMax;
          {
            // the block this step multiplied, row t4 of the tile, from its two bf16 planes
            const __nv_bfloat16* ph = prm.y_hi[step & 1] + (size_t)b * kPMax * prm.ld + tile * R + t4;
            const __nv_bfloat16* pl = prm.y_lo[step & 1] + (size_t)b * kPMax * prm.ld + tile * R + t4;
            const unsigned short* uh = reinterpret_cast<const unsigned short*>(ph);
            const unsigned short* ul = reinterpret_cast<const unsigned short*>(pl);
            const bool have_row = t4 < nrows;
#pragma unroll 1
            for (int c0 = 0; c0 < P; c0 += 8) {
              unsigned short vh[8], vl[8];
#pragma unroll
              for (int u = 0; u < 8; ++u) {
                const bool in = have_row && c0 + u < p;
                vh[u] = in ? __ldcg(uh + (size_t)(c0 + u) * prm.ld) : (unsigned short)0;
                vl[u] = in ? __ldcg(ul + (size_t)(c0 + u) * prm.ld) : (unsigned short)0;
              }
#pragma unroll
              for (int u = 0; u < 8; ++u)
                xq[(c0 + u) * kXsLd + t4] = __uint_as_float((uint32_t)vh[u] << 16) + __uint_as_float((uint32_t)vl[u] << 16);
            }
          }
          named_barrier(2, 128);
          for (int jb = 0; jb < P && active; jb += 8) {
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = xq[(jb + e) * kXsLd + t4];
            solve_apply_groups(acc, jb, 0, jb >> 2, smem_u32(lt), smem_u32(xq), t4, P);
            solve_inblock8(acc, jb, smem_u32(lt), smem_u32(dinv), P);
#pragma unroll
            for (int e = 0; e < 8; ++e) xq[(jb + e) * kXsLd + t4] = acc[e];
          }
          named_barrier(2, 128);
          // only the window columns are read again (second half of Eq. 15)
          for (int c = (p - rp.win) + (t4 & 31); c < p; c += 32)
            for (int rr = t4 >> 5; rr < nrows; rr += 4) qrows[(size_t)rr * kPMax + c] = xq[c * kXsLd + rr];
        }
        epi_sync();                                  // the staged block is complete
        if (is_last && et < nrows) {
          // first half of Eq. 15 while both blocks are on chip: sum_j Y'_ij Q_ij, parked in the
          // energy array until the Ritz vectors of the request are known
          float total = 0.f;
          for (int c = 0; c < p; ++c) total += xs[c * kXsLd + et] * xq[c * kXsLd + et];
          prm.energy[(size_t)rp.presel_off + tile * R + et] = total;
        }
        // the partial Gram below stages its slabs where the previous block (xq) lives: nobody may
        // start on them while a row still reads xq
        if (is_last) epi_sync();
        // ---- bf16 planes of the new block (K-major operand of the next step): 8 positions per thread
        if (!is_last) {
          const int cols = (rp.m + kBK - 1) / kBK * kBK;
          const int cshift = R == 64 ? 3 : 4;          // 8-position chunks per row of the tile: 2^cshift
          for (int wi = et; wi < (p << cshift); wi += kEpiThreads) {
            int c = wi >> cshift, ch = wi & ((1 << cshift) - 1);
            int pos = tile * R + ch * 8;
            if (pos >= cols) continue;
            const float4* xp = reinterpret_cast<const float4*>(xs + c * kXsLd + ch * 8);
            float4 a = xp[0], d = xp[1];
            float f[8] = {a.x, a.y, a.z, a.w, d.x, d.y, d.z, d.w};
            if (ch * 8 + 8 > nrows) {                  // padding positions up to the k-chunk boundary are zero
#pragma unroll
              for (int e = 0; e < 8; ++e)
                if (ch * 8 + e >= nrows) f[e] = 0.f;
            }
            uint32_t ph[4], pl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 hi = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
              ph[e] = *reinterpret_cast<uint32_t*>(&hi);
              pl[e] = pack_bf16(f[2 * e] - __low2float(hi), f[2 * e + 1] - __high2float(hi));
            }
            size_t o = ((size_t)b * kPMax + c) * prm.ld + pos;
            *reinterpret_cast<uint4*>(y_hi + o) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
            *reinterpret_cast<uint4*>(y_lo + o) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
          }
        }
        if (yf != nullptr) {
          // float32 window columns of the final block, one token per row (second half of Eq. 15)
          float* yrows = yf + ((size_t)rp.presel_off + tile * R) * kPMax;
          for (int c = (p - rp.win) + (et & 31); c < p; c += 32)
            for (int rr = et >> 5; rr < nrows; rr += 8) yrows[(size_t)rr * kPMax + c] = xs[c * kXsLd + rr];
        }
        // ---- float64 partial Gram of the tile on the FP64 tensor cores ----
        const int coff = is_last ? ((p - rp.win) & ~7) : 0;
        {
          // The last step only feeds the Rayleigh-Ritz window: the trailing block of columns from
          // coff on, plus the diagonal of the leading columns (the scale of the problem).
          const int pw = p - coff;
          const int nb8 = (pw + 7) >> 3, units = (nb8 + 1) / 2, nslab = (nrows + kSlabRows - 1) / kSlabRows;
          double* slabs = reinterpret_cast<double*>(smem + kXsBytes);
          double* out = prm.partial + (size_t)item * kTileDoubles;
          for (int c = et; c < coff; c += kEpiThreads) {
            double sq = 0.0;
            for (int rr = 0; rr < nrows; ++rr) { double x = (double)xs[c * kXsLd + rr]; sq += x * x; }
            out[tile_offset(c, c)] = sq;
          }
          // Units 0-7 go to the eight warps.  With more than 128 columns one or two units are left
          // over: a second, short pass over the slabs deals their 8 x 8 tiles round-robin to the
          // warps (at most kExtraTiles each) instead of leaving them to one or two warps.
          const int fr = lane >> 2, fk = lane & 3;
          auto fill_slab = [&](double* slab, int sl) {
            for (int e = et; e < nb8 * 8 * kSlabRows; e += kEpiThreads) {
              int c = e >> 4, rr = e & 15;
              slab[c * kSlabLd + rr] = (double)xs[(coff + c) * kXsLd + sl * kSlabRows + rr];
            }
          };
          {
            const bool have = warp < units;
            const int ta = have ? warp : 0, tz = have ? nb8 - 1 - warp : 0;
            GramAcc acc;
#pragma unroll
            for (int u = 0; u <= kMaxTiles8; ++u) { acc.a[u][0] = 0.0; acc.a[u][1] = 0.0; }
            for (int sl = 0; sl < nslab; ++sl) {
              double* slab = slabs + (sl & 1) * (kPMax * kSlabLd);
              fill_slab(slab, sl);
              epi_sync();
              if (have) gram_unit_accumulate(acc, slab, ta, tz, lane);
              // the other buffer is refilled next; this one is reused two slabs later, after the
              // barrier of the next slab
            }
            if (have) gram_unit_store_tiles(acc, ta, tz, coff >> 3, lane, out);
            epi_sync();
          }
          if (units > 8) {
            int xa_t[kExtraTiles], xb_t[kExtraTiles];
            double xacc[kExtraTiles][2];
            int n_extra = 0;
#pragma unroll
            for (int q = 0; q < kExtraTiles; ++q) {
              xacc[q][0] = 0.0; xacc[q][1] = 0.0; xa_t[q] = 0; xb_t[q] = 0;
              if (extra_tile(warp + 8 * q, nb8, units, xa_t[q], xb_t[q])) n_extra = q + 1;
            }
            for (int sl = 0; sl < nslab; ++sl) {
              double* slab = slabs + (sl & 1) * (kPMax * kSlabLd);
              fill_slab(slab, sl);
              epi_sync();
              const double* base = slab + fr * kSlabLd + fk;
#pragma unroll 1
              for (int ks = 0; ks < kSlabRows / 4; ++ks) {
#pragma unroll
                for (int q = 0; q < kExtraTiles; ++q)
                  if (q < n_extra)
                    dmma_8x8x4(xacc[q][0], xacc[q][1], base[xa_t[q] * 8 * kSlabLd + 4 * ks],
                               base[xb_t[q] * 8 * kSlabLd + 4 * ks]);
              }
            }
#pragma unroll
            for (int q = 0; q < kExtraTiles; ++q) {
              if (q < n_extra)
                *reinterpret_cast<double2*>(out + tri_index((coff >> 3) + xa_t[q], (coff >> 3) + xb_t[q]) * 64 +
                                            fr * 8 + 2 * fk) = make_double2(xacc[q][0], xacc[q][1]);
            }
            epi_sync();
          }
        }
        // ---- arrival: this tile's slab and partial sums are published -------------------------
        __threadfence();
        fence_proxy_async_all();
        epi_sync();
        int nt_sum = (int)nt;                        // partial matrices the factoring tile has to add up
        if (prm.spread_sum && nt >= 4) {             // with fewer tiles the extra round trip costs more than it saves
          // Every CTA holds one tile, so all tiles of the request are being worked on at the same
          // time: instead of leaving the sum of the partial matrices to the last tile alone, every
          // tile waits for the others and adds up its own slice of the matrix (in tile order, into
          // the slot of tile 0); the last one to finish its slice factors the summed matrix.
          if (et == 0) atomicAdd(sync_b, 1u);
          ok = team_wait(sync_b, nt * (unsigned)(step + 1)) && ok;
          double* sum0 = prm.partial + (size_t)rp.ptile_off * kTileDoubles;
          const int used = (P >> 3) * ((P >> 3) + 1) / 2 * 64;
          const int chunk = ((used + (int)nt - 1) / (int)nt + 1) & ~1;
          const int e1 = min(used, (tile + 1) * chunk);
          if (ok) {
            for (int e = tile * chunk + 2 * et; e < e1; e += 2 * kEpiThreads) {
              double2 acc = make_double2(0.0, 0.0);
              for (int t0 = 0; t0 < (int)nt; t0 += 8) {
                double2 v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  v[q] = __ldcg(reinterpret_cast<const double2*>(sum0 + (size_t)min(t0 + q, (int)nt - 1) * kTileDoubles + e));
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  if (t0 + q < (int)nt) { acc.x += v[q].x; acc.y += v[q].y; }
              }
              *reinterpret_cast<double2*>(sum0 + e) = acc;
            }
          }
          __threadfence();
          epi_sync();
          if (et == 0) {
            unsigned old = atomicAdd(sync_b + 4, 1u);
            *s_word = (old + 1u == nt * (unsigned)(step + 1) && !*abort_flag) ? 1 : 0;
          }
          nt_sum = 1;
        } else if (et == 0) {
          unsigned old = atomicAdd(sync_b, 1u);
          // one decision for the whole team (a CTA that has given up factors nothing)
          *s_word = (old + 1u == nt * (unsigned)(step + 1) && !*abort_flag) ? 1 : 0;
        }
        epi_sync();
        if (*s_word && prm.n_servers == 0) {
          // ---- the last tile of the request to finish this step factors the summed Gram matrix ----
          factor_request(b, rp, sync_b, step, is_last, last_b, nt_sum);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(epi_done);
      }
    }
    // ------------------------------------------------------------ Eq. 15 for this CTA's tiles
    // c_i = sum_j Y'_ij Q_ij - sum_k (Y'_{i,win} u_k)(Q_{i,win} u_k)  (see eig_kernels.cuh)
    {
      float* us = reinterpret_cast<float*>(smem);                      // [w][nbot]
      int cached_u = -1;
      for (int si = s_begin; si < s_end; ++si) {
        const int item = s_items[si];
        int b, tile; ReqPlan rp;
        decode(item, b, rp, tile);
        const int p = rp.p, w = rp.win, w0 = p - w, nbot = p - rp.r;
        if (b != cached_u) {
          ok = team_wait(prm.sync + (size_t)b * kSyncStride + 2, 1u) && ok;
          const float* usrc = prm.ub + (size_t)b * kPMax * kPMax;
          if (ok) for (int e = et; e < w * nbot; e += kEpiThreads) us[e] = __ldcg(usrc + e);
          epi_sync();
          cached_u = b;
        }
        const int nrows = min(R, rp.m - tile * R);
        // the discarded Ritz pairs take only the window columns of the two blocks: one thread per
        // row, window slices read straight from the float32 blocks
        for (int rr = et; rr < nrows; rr += kEpiThreads) {
          const size_t grow = (size_t)rp.presel_off + tile * R + rr;
          const float* yrow = prm.yf[1] + grow * kPMax + w0;
          const float* qrow = prm.yf[0] + grow * kPMax + w0;
          // projections of the two window slices on every discarded Ritz vector, accumulated over
          // chunks of 32 window columns (all loads of a chunk in flight together)
          float sub_ = 0.f;
          for (int k0 = 0; k0 < nbot; k0 += 8) {
            float ya[8], qa[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) { ya[u] = 0.f; qa[u] = 0.f; }
            for (int j0 = 0; j0 < w; j0 += 32) {
              float yv[32], qv[32];
#pragma unroll
              for (int jj = 0; jj < 32; ++jj) {
                const bool in = ok && j0 + jj < w;
                yv[jj] = in ? __ldcg(yrow + j0 + jj) : 0.f;
                qv[jj] = in ? __ldcg(qrow + j0 + jj) : 0.f;
              }
#pragma unroll
              for (int jj = 0; jj < 32; ++jj) {
                if (j0 + jj < w) {
                  const float* ur = us + (j0 + jj) * nbot + k0;
#pragma unroll
                  for (int u = 0; u < 8; ++u) {
                    const float uu = k0 + u < nbot ? ur[u] : 0.f;
                    ya[u] += yv[jj] * uu; qa[u] += qv[jj] * uu;
                  }
                }
              }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) sub_ += ya[u] * qa[u];
          }
          const float total = ok ? __ldcg(prm.energy + grow) : 0.f;
          prm.energy[grow] = fmaxf(total - sub_, 0.f);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem_base, kPowTmemCols);
  if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, kStatusTimeout);
}

}  // namespace sub
}  // namespace covspec
