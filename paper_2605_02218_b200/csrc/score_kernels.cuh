// Score kernels: query-element normalisation, cosine-max (Eq. 10), token activity (Eq. 11),
// normalise + fuse (Eq. 12).
#pragma once
#include <float.h>

#include "common.cuh"

namespace covspec {

// Converts every query-element embedding to float32 and scales each head slice to unit length
// (zero slices stay zero, which makes their cosines 0).  One warp per (row, head).
//   src [rows, width_total] of TIn (the projected Qp in float32, or Q itself in identity mode)
//   dst [rows, width_total] float32
template <typename TIn>
__global__ void __launch_bounds__(256)
qnorm_kernel(const TIn* __restrict__ src, float* __restrict__ dst, int rows, int n_heads, int hd) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= rows * n_heads) return;
  size_t base = (size_t)(warp / n_heads) * n_heads * hd + (size_t)(warp % n_heads) * hd;
  float ss = 0.f;
  for (int k = lane; k < hd; k += 32) { float v = to_float(src[base + k]); ss += v * v; }
  ss = warp_sum(ss);
  float inv = ss > FLT_MIN ? rsqrtf(ss) : 0.f;
  // one Newton step on the reciprocal square root for full float32 accuracy
  if (ss > FLT_MIN) inv = inv * (1.5f - 0.5f * ss * inv * inv);
  for (int k = lane; k < hd; k += 32) dst[base + k] = to_float(src[base + k]) * inv;
}

// Eq. 10.  One warp per visual token: for every head, the cosine between the token's embedding
// slice and every (unit-length) query-element slice of the same request; max over (element, head)
// pairs, or mean over heads followed by max over elements.
//   E   [rows, n_heads*hd] embeddings of the tokens first_row .. first_row+rows-1 (float32
//       projection chunk, or X itself in identity mode)
//   Qn  [sum T, n_heads*hd] float32 unit slices
//   s_query[first_row + i]
// Dynamic shared memory: head_mean ? warps_per_block * t_max floats : 0.
template <typename TE>
__global__ void __launch_bounds__(256)
cosmax_kernel(const TE* __restrict__ E, const float* __restrict__ Qn, const ReqPlan* __restrict__ plan,
              int batch, int first_row, int rows, int n_heads, int hd, int head_mean, int t_max,
              float* __restrict__ s_query) {
  extern __shared__ float smem_mean[];
  int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int i = blockIdx.x * (blockDim.x >> 5) + wib;
  if (i >= rows) return;
  int row = first_row + i;
  int b = find_request(row, batch, [&](int q) { return plan[q].vis_off; });
  int t0 = plan[b].txt_off, T = plan[b].t;
  int P = n_heads * hd;
  const TE* e = E + (size_t)i * P;
  float* acc = smem_mean + (size_t)wib * t_max;
  if (head_mean) for (int j = lane; j < T; j += 32) acc[j] = 0.f;
  float best = -FLT_MAX;
  bool nonfinite = false;   // fmaxf drops NaN operands, so non-finite inputs are tracked explicitly
  for (int h = 0; h < n_heads; ++h) {
    const TE* eh = e + (size_t)h * hd;
    float ss = 0.f;
    for (int k = lane * 4; k < hd; k += 128) {
      float v[4]; load4(eh + k, v);
      ss += v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
    }
    ss = warp_sum(ss);
    nonfinite |= !(ss <= FLT_MAX);
    float inv = 0.f;
    if (ss > FLT_MIN) { inv = rsqrtf(ss); inv = inv * (1.5f - 0.5f * ss * inv * inv); }
    for (int j = 0; j < T; ++j) {
      const float* q = Qn + (size_t)(t0 + j) * P + (size_t)h * hd;
      float dot = 0.f;
      for (int k = lane * 4; k < hd; k += 128) {
        float v[4]; load4(eh + k, v);
        float4 w = *reinterpret_cast<const float4*>(q + k);
        dot += v[0] * w.x + v[1] * w.y + v[2] * w.z + v[3] * w.w;
      }
      dot = warp_sum(dot) * inv;
      nonfinite |= dot != dot;
      if (head_mean) { if (lane == 0) acc[j] += dot; }
      else best = fmaxf(best, dot);
    }
  }
  if (head_mean) {
    __syncwarp();
    float m = -FLT_MAX;
    for (int j = lane; j < T; j += 32) m = fmaxf(m, acc[j] / (float)n_heads);
    best = warp_max(m);
  }
  if (lane == 0) s_query[row] = nonfinite ? __int_as_float(0x7fc00000) : best;
}

// Eq. 11.  One warp per token streams the token's row of all act_layers+1 snapshots once, 16 bytes
// per lane per load, and accumulates the squared change of every consecutive pair in registers.
template <typename T, int MAXL>
__global__ void __launch_bounds__(256)
activity_kernel(LayerPtrs hs, int n_layers /* = act_layers */, long long rows, int d,
                float* __restrict__ s_act) {
  long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float acc[MAXL];
#pragma unroll
  for (int l = 0; l < MAXL; ++l) acc[l] = 0.f;
  size_t base = (size_t)row * d;
  for (int k = lane * 8; k < d; k += 256) {
    float prev[8], cur[8];
    load8(reinterpret_cast<const T*>(hs.h[0]) + base + k, prev);
#pragma unroll
    for (int l = 0; l < MAXL; ++l) {
      if (l < n_layers) {
        load8(reinterpret_cast<const T*>(hs.h[l + 1]) + base + k, cur);
#pragma unroll
        for (int e = 0; e < 8; ++e) { float df = cur[e] - prev[e]; acc[l] += df * df; prev[e] = cur[e]; }
      }
    }
  }
  float total = 0.f;
#pragma unroll
  for (int l = 0; l < MAXL; ++l)
    if (l < n_layers) total += sqrtf(warp_sum(acc[l]));
  if (lane == 0) s_act[row] = total / (float)n_layers;
}

// 8 consecutive elements through the streaming path (read once: first to be evicted from L2).
__device__ __forceinline__ void load8_stream(const float* p, float (&v)[8]) {
  float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8_stream(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
  v[4] = __uint_as_float(t.z << 16); v[5] = __uint_as_float(t.z & 0xffff0000u);
  v[6] = __uint_as_float(t.w << 16); v[7] = __uint_as_float(t.w & 0xffff0000u);
}

// Eq. 11 as a background stream: the same arithmetic as activity_kernel, but a small persistent
// grid (one or two blocks per SM, rows handed out round-robin) whose loads bypass L1 and are marked
// evict-first in L2.  Few blocks matter: every resident block reserves 1 KB of the SM's shared
// memory, and the relevance kernel's CTA fits beside at most two of them.  The fused call runs it beside the tensor-core relevance kernel, which leaves
// HBM almost idle and most issue slots free: at a fraction of the HBM rate the whole snapshot stack
// is read before the relevance kernel ends, without evicting the operand tiles that kernel re-reads
// from L2.
template <typename T, int MAXL>
__global__ void __launch_bounds__(512)
activity_stream_kernel(LayerPtrs hs, int n_layers /* = act_layers */, long long rows, int d,
                       float* __restrict__ s_act) {
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); row < rows; row += warps) {
    float acc[MAXL];
#pragma unroll
    for (int l = 0; l < MAXL; ++l) acc[l] = 0.f;
    size_t base = (size_t)row * d;
#pragma unroll 2
    for (int k = lane * 8; k < d; k += 256) {
      float prev[8], cur[8];
      load8_stream(reinterpret_cast<const T*>(hs.h[0]) + base + k, prev);
#pragma unroll
      for (int l = 0; l < MAXL; ++l) {
        if (l < n_layers) {
          load8_stream(reinterpret_cast<const T*>(hs.h[l + 1]) + base + k, cur);
#pragma unroll
          for (int e = 0; e < 8; ++e) { float df = cur[e] - prev[e]; acc[l] += df * df; prev[e] = cur[e]; }
        }
      }
    }
    float total = 0.f;
#pragma unroll
    for (int l = 0; l < MAXL; ++l)
      if (l < n_layers) total += sqrtf(warp_sum(acc[l]));
    if (lane == 0) s_act[row] = total / (float)n_layers;
  }
}

// float32 operands for the bf16 tensor-core kernels.  A float32 row x of width d becomes two bf16
// rows of width 3 dp (dp = d rounded up to 64, padding zero): the "a" form [hi | lo | hi] and the "b"
// form [hi | hi | lo] with hi = bf16(x), lo = bf16(x - hi).  The K-major product of an "a" row and a
// "b" row is hi.hi + lo.hi + hi.lo, the three-term bf16 product (about 2^-17 relative), so the
// kernels written for bf16 inputs run unchanged on a three times longer inner dimension.
struct SplitJob {
  const float* src;            // [rows or more, d] float32
  const int* idx;              // nullptr: row r of src; else row plan[request of r].vis_off + idx[r]
  __nv_bfloat16* out_a;        // [rows, 3 dp] or nullptr
  __nv_bfloat16* out_b;        // [rows, 3 dp] or nullptr
  long long rows;
};
struct SplitJobs { SplitJob j[4]; };

__global__ void __launch_bounds__(256)
split3_kernel(SplitJobs jobs, const ReqPlan* __restrict__ plan, int batch, int d, int dp) {
  const SplitJob job = jobs.j[blockIdx.y];
  for (long long row = blockIdx.x; row < job.rows; row += gridDim.x) {
    long long src_row = row;
    if (job.idx != nullptr) {
      int b = find_request((int)row, batch, [&](int q) { return plan[q].presel_off; });
      src_row = (long long)plan[b].vis_off + job.idx[row];
    }
    const float* x = job.src + (size_t)src_row * d;
    for (int c = threadIdx.x * 4; c < dp; c += blockDim.x * 4) {       // d and dp are multiples of 4
      float4 v = c < d ? *reinterpret_cast<const float4*>(x + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
      __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - __low2float(h0), v.y - __high2float(h0));
      __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - __low2float(h1), v.w - __high2float(h1));
      uint2 hi = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
      uint2 lo = make_uint2(*reinterpret_cast<uint32_t*>(&l0), *reinterpret_cast<uint32_t*>(&l1));
      if (job.out_a != nullptr) {
        __nv_bfloat16* o = job.out_a + (size_t)row * 3 * dp + c;
        *reinterpret_cast<uint2*>(o) = hi;
        *reinterpret_cast<uint2*>(o + dp) = lo;
        *reinterpret_cast<uint2*>(o + 2 * dp) = hi;
      }
      if (job.out_b != nullptr) {
        __nv_bfloat16* o = job.out_b + (size_t)row * 3 * dp + c;
        *reinterpret_cast<uint2*>(o) = hi;
        *reinterpret_cast<uint2*>(o + dp) = hi;
        *reinterpret_cast<uint2*>(o + 2 * dp) = lo;
      }
    }
  }
}

// ---- block-wide reductions used by the fuse kernel (blockDim.x multiple of 32, <= 1024) ----
template <typename Op>
__device__ __forceinline__ float block_reduce(float v, Op op, float identity, float* scratch) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = op(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  v = lane < nw ? scratch[lane] : identity;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = op(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

struct NormParams { float shift, scale; };

// Parameters (shift, scale) such that normalised = (s - shift) * scale, per request.
__device__ __forceinline__ NormParams norm_params(const float* s, int n, int mode, float* scratch,
                                                   int* status) {
  NormParams np{0.f, 1.f};
  if (mode == 2) return np;
  auto fmin2 = [](float a, float b) { return fminf(a, b); };
  auto fmax2 = [](float a, float b) { return fmaxf(a, b); };
  auto fadd2 = [](float a, float b) { return a + b; };
  bool bad = false;
  if (mode == 0) {
    float lo = FLT_MAX, hi = -FLT_MAX;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      float v = s[i];
      bad |= !isfinite(v);
      lo = fminf(lo, v); hi = fmaxf(hi, v);
    }
    lo = block_reduce(lo, fmin2, FLT_MAX, scratch);
    hi = block_reduce(hi, fmax2, -FLT_MAX, scratch);
    np.shift = lo;
    np.scale = hi > lo ? 1.f / (hi - lo) : 0.f;
  } else {
    float sum = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { float v = s[i]; bad |= !isfinite(v); sum += v; }
    float mean = block_reduce(sum, fadd2, 0.f, scratch) / (float)n;
    float sq = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { float df = s[i] - mean; sq += df * df; }
    float var = block_reduce(sq, fadd2, 0.f, scratch) / (float)n;
    np.shift = mean;
    np.scale = var > 0.f ? rsqrtf(var) : 0.f;
  }
  if (bad) atomicOr(status, kStatusNonFinite);
  return np;
}

// Eq. 12 for one request (whole block): normalise both scores to a common scale, fuse with lambda.
// s_act == nullptr (no activity stack): the fused score is the normalised query score.
__device__ __forceinline__ void fuse_request(const ReqPlan& rp, const float* __restrict__ s_query,
                                             const float* __restrict__ s_act, float lambda, int mode,
                                             float* __restrict__ s_fused, float* scratch, int* status) {
  const float* sq = s_query + rp.vis_off;
  NormParams nq = norm_params(sq, rp.n, mode, scratch, status);
  if (s_act == nullptr) {
    for (int i = threadIdx.x; i < rp.n; i += blockDim.x)
      s_fused[rp.vis_off + i] = (sq[i] - nq.shift) * nq.scale;
    return;
  }
  const float* sa = s_act + rp.vis_off;
  NormParams na = norm_params(sa, rp.n, mode, scratch, status);
  for (int i = threadIdx.x; i < rp.n; i += blockDim.x)
    s_fused[rp.vis_off + i] =
        lambda * ((sq[i] - nq.shift) * nq.scale) + (1.f - lambda) * ((sa[i] - na.shift) * na.scale);
}

// Eq. 12.  One block per request.
__global__ void __launch_bounds__(1024)
fuse_kernel(const float* __restrict__ s_query, const float* __restrict__ s_act,
            const ReqPlan* __restrict__ plan, float lambda, int mode, float* __restrict__ s_fused,
            int* status) {
  __shared__ float scratch[32];
  fuse_request(plan[blockIdx.x], s_query, s_act, lambda, mode, s_fused, scratch, status);
}

}  // namespace covspec
