// Shared device-side types and helpers of the covspec kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace covspec {

constexpr int kPMax = 160;        // largest subspace-iteration basis (rank + oversampling)
constexpr int kMaxLayers = 17;    // act_layers + 1 snapshots at most

// Device status bits (OR-ed into the context's status word).
constexpr int kStatusNonFinite = 1;
constexpr int kStatusNoConverge = 2;
constexpr int kStatusBounds = 8;      // checked build only (4 is the wait time-out of the tensor-core kernels)

// Checked build (-DCOVSPEC_DEBUG_BOUNDS, libcovspec_debug.so): index-driven global accesses test
// their index first; a bad one raises kStatusBounds in the status word and the access is skipped, so
// the context stays usable and the host reads COVSPEC_ERR_BOUNDS.  The ordinary build compiles the
// test away.
#ifdef COVSPEC_DEBUG_BOUNDS
#define COVSPEC_IN_BOUNDS(idx, limit, status)                                              \
  (((long long)(idx) >= 0 && (long long)(idx) < (long long)(limit))                        \
       ? true                                                                              \
       : ((status) != nullptr ? (atomicOr((status), ::covspec::kStatusBounds), false) : false))
#else
#define COVSPEC_IN_BOUNDS(idx, limit, status) true
#endif

// Per-request launch plan, built on the host from the offset arrays and uploaded once per shape.
struct ReqPlan {
  int vis_off, n;          // rows of X / scores owned by the request
  int txt_off, t;          // rows of Q
  int b_vis, m, r, p;      // keep budget, preselect size, rank, basis size (p = 0: stage 2 skipped)
  int keep_off, presel_off;
  int ldm;                 // m rounded up to a multiple of 4 (row stride of the float32 Gram matrix)
  int stage2;              // 1 when b_vis < m (Eq. 13-15 are evaluated)
  int tile_off;            // first 128-token tile of the request in the tensor-core relevance kernel
  int pair_off;            // first pair of 128-token tiles of the request (two-SM relevance kernel)
  int gram_tile_off;       // first lower-triangle 128 x 256 item of the request's Gram matrix
  int ptile_off;           // first 128-row tile of the request's subspace-iteration block
  int win;                 // basis vectors in the Rayleigh-Ritz window next to the cut at r
  long long g_off;         // float offset of the request's float32 Gram matrix (float32 inputs only)
  long long c_off;         // float offset of the request's factor columns (greedy low-rank mode)
};

// One dense product C[m x n] = A[m x k] * op(B) handled by the tiled SIMT kernel.
struct GemmProb {
  const void* A;
  const void* B;
  void* C;
  int m, n, k;
  int lda, ldb, ldc;
  int tile_start;          // first tile of this problem in the launch's tile list
  int tiles_n;             // tiles along n
};

struct LayerPtrs {
  const void* h[kMaxLayers];
};

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
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Loads 4 consecutive elements as floats (16-byte / 8-byte vector access; caller guarantees
// alignment).
__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
  float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
  uint2 t = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}
__device__ __forceinline__ void load4(const double* p, float (&v)[4]) {
  v[0] = (float)p[0]; v[1] = (float)p[1]; v[2] = (float)p[2]; v[3] = (float)p[3];
}

// Loads 8 consecutive elements (one 16-byte vector for bf16, two for fp32).
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 t = *reinterpret_cast<const uint4*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
  v[4] = __uint_as_float(t.z << 16); v[5] = __uint_as_float(t.z & 0xffff0000u);
  v[6] = __uint_as_float(t.w << 16); v[7] = __uint_as_float(t.w & 0xffff0000u);
}

// Request that owns global row `row` (binary search over the plan's vis_off / presel_off / ...).
template <typename GetOff>
__device__ __forceinline__ int find_request(int row, int batch, GetOff off_of) {
  int lo = 0, hi = batch - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (off_of(mid) <= row) lo = mid; else hi = mid - 1;
  }
  return lo;
}

}  // namespace covspec
