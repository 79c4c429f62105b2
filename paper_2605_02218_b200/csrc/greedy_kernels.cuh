// Greedy pivoted low-rank selection, offered as lowrank_mode = 1 next to the truncated-SVD energy of
// Eq. 14-15 (this variant is not in the paper): B_vis times, pick the preselected token whose
// representation has the largest residual energy after projecting out the span of the tokens
// already picked, then update all residuals.  This is the Cholesky factorisation with diagonal
// pivoting of G = Z_M^T Z_M stopped after B_vis columns:
//   p_k = argmax_i e_i (ties: lower index),  c_k = (G[:, p_k] - sum_{j<k} c_j c_j[p_k]) / sqrt(e_{p_k}),
//   e_i <- e_i - c_k[i]^2.
// One block per request; the residuals live in registers (up to 16 per thread), the argmax is a
// warp-shuffle + shared-memory reduction, the factor columns are kept in a workspace array.
// Output: energy[i] = B_vis - k for the k-th pick (k = 0 first), 0 for tokens not picked, so that the
// ordinary final selection (the B_vis largest energies) returns exactly the picked set and the order
// of the picks can be read back.
#pragma once
#include "common.cuh"

namespace covspec {

constexpr int kGreedyThreads = 1024;
constexpr int kGreedyPer = 16;                          // residuals per thread: M <= 16384
constexpr int kGreedyMaxM = kGreedyThreads * kGreedyPer;
constexpr int kGreedyMaxB = 8192;                       // picks per request (row of the factor in shared memory)

__global__ void __launch_bounds__(kGreedyThreads)
greedy_select_kernel(const ReqPlan* __restrict__ plan, const __nv_bfloat16* __restrict__ g_hi,
                     const __nv_bfloat16* __restrict__ g_lo, int ld, float* __restrict__ cbuf,
                     float* __restrict__ energy, int* status) {
  __shared__ float cp[kGreedyMaxB];                     // c_j[p] for the current pivot p, j < k
  __shared__ float red_v[32];
  __shared__ int red_i[32];
  __shared__ float s_ep;
  __shared__ int s_p;
  const ReqPlan rp = plan[blockIdx.x];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int M = rp.m, B = rp.b_vis;
  for (int i = tid; i < M; i += kGreedyThreads) energy[rp.presel_off + i] = 0.f;
  if (!rp.stage2) return;
  auto G = [&](int i, int j) {
    size_t o = ((size_t)rp.presel_off + i) * ld + j;
    return __bfloat162float(g_hi[o]) + __bfloat162float(g_lo[o]);
  };
  float* C = cbuf + rp.c_off;                           // [B][M]
  float e[kGreedyPer];
#pragma unroll
  for (int q = 0; q < kGreedyPer; ++q) {
    int i = tid + q * kGreedyThreads;
    e[q] = i < M ? G(i, i) : -INFINITY;
  }
  bool bad = false;
  for (int k = 0; k < B; ++k) {
    // ---- argmax of the residuals: larger value first, then lower index ----
    // A residual that is not a number (non-finite Gram entries) ranks below every number but
    // above the picked tokens' -inf, so that the pivot is always an unpicked token inside the
    // request; the condition is reported through the status word.
    float bv = -INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int q = 0; q < kGreedyPer; ++q) {
      int i = tid + q * kGreedyThreads;
      if (i < M) {
        float v = e[q];
        if (v != v) { v = -3.0e38f; bad = true; }
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { red_v[warp] = bv; red_i[warp] = bi; }
    __syncthreads();
    if (warp == 0) {
      bv = red_v[lane]; bi = red_i[lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) {
        if (bi >= M) { bi = 0; bv = 0.f; atomicOr(status, kStatusNonFinite); }   // every token picked: cannot happen for B < M
        s_p = bi; s_ep = bv; energy[rp.presel_off + bi] = (float)(B - k);
      }
    }
    __syncthreads();
    const int p = s_p;
    const float ep = s_ep;
    const float rs = ep > 0.f ? rsqrtf(ep) : 0.f;
    for (int j = tid; j < k; j += kGreedyThreads) cp[j] = C[(size_t)j * M + p];
    __syncthreads();
    // ---- new factor column and residual update ----
#pragma unroll
    for (int q = 0; q < kGreedyPer; ++q) {
      int i = tid + q * kGreedyThreads;
      if (i < M) {
        float acc = G(p, i);
        for (int j = 0; j < k; ++j) acc -= C[(size_t)j * M + i] * cp[j];
        float c = acc * rs;
        C[(size_t)k * M + i] = c;
        if (i == p) e[q] = -INFINITY;                   // never picked again
        else if (!(e[q] == -INFINITY)) e[q] -= c * c;
      }
    }
    __syncthreads();
  }
  if (bad) atomicOr(status, kStatusNonFinite);
}

}  // namespace covspec
