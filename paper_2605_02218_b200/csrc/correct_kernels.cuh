// Device-side gating and correction over the vocabulary (Eq. 2, 4, 5, 6, 16, 17; Sec. III-C.2):
// from the draft logits and the target logits of one position, the draft distribution's top-2 margin
// and gate, the acceptance probability of the drafted token, the residual distribution
// max(p_t - p_d, 0) / mass and a token drawn from it by inverse CDF with a uniform number supplied by
// the caller.
//
// One block per position; HBM-bound.  Both logit rows (2 * W * elem bytes, ~600 KB at W = 152 k in
// 16 bits) are read from HBM once; the second sweep (residual mass) and the short third one (the
// cumulative sum inside the one warp segment that contains the sample) find them in L2.  Each warp
// owns a contiguous segment of the row and reads it with coalesced 16-byte vectors, so the order of
// the cumulative sum is (segment, vector, lane, element).
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"
#include "select_kernels.cuh"

namespace covspec {
namespace corr {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float cvt(float v) { return v; }
__device__ __forceinline__ float cvt(__half v) { return __half2float(v); }
__device__ __forceinline__ float cvt(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> struct Vec;           // 16-byte vector of logits
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<__half> { static constexpr int N = 8; };
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };

constexpr float kLog2e = 1.4426950408889634f;

// 2^x on the special-function unit, results below the normal range flushed to zero (a probability
// under 1e-38): one instruction, where the denormal-preserving form takes four.
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 16 bytes of logits: the largest element and the N values as floats.  Elements at or beyond `w`
// read as -inf (probability zero).  The row base is 16-byte aligned.
__device__ __forceinline__ void unpack(const uint4& raw, float (&v)[4], const float*) {
  v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
  v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
}
__device__ __forceinline__ void unpack(const uint4& raw, float (&v)[8], const __half*) {
  const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
  for (int k = 0; k < 4; ++k) { float2 f = __half22float2(h[k]); v[2 * k] = f.x; v[2 * k + 1] = f.y; }
}
__device__ __forceinline__ void unpack(const uint4& raw, float (&v)[8], const __nv_bfloat16*) {
  const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(u[k] << 16); v[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u); }
}
__device__ __forceinline__ float vec_max(const uint4& raw, const float*) {
  return fmaxf(fmaxf(__uint_as_float(raw.x), __uint_as_float(raw.y)),
               fmaxf(__uint_as_float(raw.z), __uint_as_float(raw.w)));
}
__device__ __forceinline__ float vec_max(const uint4& raw, const __half*) {
  const __half2* h = reinterpret_cast<const __half2*>(&raw);
  __half2 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));       // exact: a maximum rounds nothing
  return __half2float(__hmax(__low2half(m), __high2half(m)));
}
__device__ __forceinline__ float vec_max(const uint4& raw, const __nv_bfloat16*) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
  __nv_bfloat162 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
  return __bfloat162float(__hmax(__low2bfloat16(m), __high2bfloat16(m)));
}

// The N consecutive logits that start at element `i` (a multiple of N) of `row`, as raw bits; the
// tail vector of a row whose length is not a multiple of N is completed with -inf.
template <typename T>
__device__ __forceinline__ uint4 load_raw(const T* __restrict__ row, int i, int w) {
  constexpr int N = Vec<T>::N;
  if (i + N <= w) return *reinterpret_cast<const uint4*>(row + i);
  T e[N];
#pragma unroll
  for (int k = 0; k < N; ++k) e[k] = i + k < w ? row[i + k] : (T)(-INFINITY);
  return *reinterpret_cast<const uint4*>(e);
}
template <typename T>
__device__ __forceinline__ void load_vec(const T* __restrict__ row, int i, int w, float (&v)[Vec<T>::N]) {
  unpack(load_raw(row, i, w), v, (const T*)nullptr);
}

// Running (max, sum of exp(z - max)) pair of a softmax denominator.
struct MaxSum {
  float m, s;
  __device__ __forceinline__ void merge(const MaxSum& o) {
    if (o.m > m) { s = s * __expf(m - o.m) + o.s; m = o.m; }
    else if (o.m > -INFINITY) s += o.s * __expf(o.m - m);
  }
};
__device__ __forceinline__ MaxSum shfl_xor(const MaxSum& a, int o) {
  MaxSum r;
  r.m = __shfl_xor_sync(0xffffffffu, a.m, o);
  r.s = __shfl_xor_sync(0xffffffffu, a.s, o);
  return r;
}

// Probability of one logit: 2^(z log2(e) - c) with c = log2(e) max + log2(sum of exp(z - max)), one
// fused multiply-add and one special-function instruction.  Draft and target rows go through the
// same instructions, so identical rows give a residual of exactly zero.
__device__ __forceinline__ float prob(float z, float neg_c) { return ex2(fmaf(z, kLog2e, neg_c)); }

// Two largest values of a multiset.
struct Top2 {
  float a, b;   // a >= b
  __device__ __forceinline__ void add(float z) {
    if (z > a) { b = a; a = z; } else if (z > b) b = z;
  }
  __device__ __forceinline__ void merge(const Top2& o) { add(o.a); add(o.b); }
};

// rows: positions; w: vocabulary size; ldz: elements between consecutive rows (multiple of 16 bytes).
template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
correct_kernel(const T* __restrict__ zd, const T* __restrict__ zt, long long ldz, int w,
               const int* __restrict__ drafted, const float* __restrict__ uniforms, float gamma,
               float* __restrict__ margin, int* __restrict__ gate, float* __restrict__ accept,
               float* __restrict__ resid_mass, int* __restrict__ token) {
  constexpr int N = Vec<T>::N;
  __shared__ MaxSum sh_d[kWarps], sh_t[kWarps];
  __shared__ Top2 sh_top[kWarps];
  __shared__ float sh_mass[kWarps];
  __shared__ float bc[6];
  __shared__ int sh_token;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* rd = zd + (size_t)row * ldz;
  const T* rt = zt + (size_t)row * ldz;
  const T* const tag = nullptr;
  // contiguous segment of this warp, in whole vectors
  const int nvec = (w + N - 1) / N;
  const int vec_per_warp = (nvec + kWarps - 1) / kWarps;
  const int v0 = warp * vec_per_warp, v1 = min(nvec, v0 + vec_per_warp);

  // ---- sweep 1: softmax denominators of both rows (Eq. 2, 4), two largest draft logits (Eq. 16) ----
  // The sums run relative to the largest logit seen so far by this thread, in the base-2 domain:
  // exp(z - m) = 2^(z log2(e) - m log2(e)).
  MaxSum md{-INFINITY, 0.f}, mt{-INFINITY, 0.f};
  float nd = 0.f, nt = 0.f;                     // -m log2(e) of the two running maxima
  Top2 top{-INFINITY, -INFINITY};
#pragma unroll 2
  for (int v = v0 + lane; v < v1; v += 32) {
    const uint4 ra = load_raw(rd, v * N, w), rb = load_raw(rt, v * N, w);
    // one rescale per vector: every vector holds at least one element of the vocabulary, so its
    // maximum is finite and 2^(-inf) = 0 takes care of the padding
    const float va = vec_max(ra, tag), vb = vec_max(rb, tag);
    if (va > md.m) { md.s *= __expf(md.m - va); md.m = va; nd = -va * kLog2e; }
    if (vb > mt.m) { mt.s *= __expf(mt.m - vb); mt.m = vb; nt = -vb * kLog2e; }
    float a[N], b[N];
    unpack(ra, a, tag);
    unpack(rb, b, tag);
    float sa = 0.f, sb = 0.f;
#pragma unroll
    for (int k = 0; k < N; ++k) {
      sa += ex2(fmaf(a[k], kLog2e, nd));
      sb += ex2(fmaf(b[k], kLog2e, nt));
    }
    md.s += sa;
    mt.s += sb;
    if (va > top.b) {                           // rare once a few vectors have been seen
#pragma unroll
      for (int k = 0; k < N; ++k) top.add(a[k]);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    md.merge(shfl_xor(md, o));
    mt.merge(shfl_xor(mt, o));
    Top2 other{__shfl_xor_sync(0xffffffffu, top.a, o), __shfl_xor_sync(0xffffffffu, top.b, o)};
    top.merge(other);
  }
  if (lane == 0) { sh_d[warp] = md; sh_t[warp] = mt; sh_top[warp] = top; }
  __syncthreads();
  if (warp == 0) {
    if (lane < kWarps) { md = sh_d[lane]; mt = sh_t[lane]; top = sh_top[lane]; }
    else { md = MaxSum{-INFINITY, 0.f}; mt = md; top = Top2{-INFINITY, -INFINITY}; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      md.merge(shfl_xor(md, o));
      mt.merge(shfl_xor(mt, o));
      Top2 other{__shfl_xor_sync(0xffffffffu, top.a, o), __shfl_xor_sync(0xffffffffu, top.b, o)};
      top.merge(other);
    }
    if (lane == 0) {
      // exponent offsets of the two distributions: p = 2^(z log2(e) + bc)
      bc[0] = -(md.m * kLog2e + log2f(md.s));
      bc[1] = -(mt.m * kLog2e + log2f(mt.s));
      float m = (1.f - (top.b > -INFINITY ? __expf(top.b - top.a) : 0.f)) * __expf(top.a - md.m) / md.s;
      margin[row] = m;
      gate[row] = m < gamma ? 1 : 0;                                       // Eq. 17
      if (accept != nullptr) {
        float al = 1.f;
        if (drafted != nullptr) {
          int y = drafted[row];
          float pd = __expf(cvt(rd[y]) - md.m) / md.s, pt = __expf(cvt(rt[y]) - mt.m) / mt.s;
          al = pd > 0.f ? fminf(1.f, pt / pd) : 1.f;                       // Eq. 5
        }
        accept[row] = al;
      }
    }
  }
  __syncthreads();
  const float cd = bc[0], ct = bc[1];

  // ---- sweep 2: residual mass per warp segment (Eq. 6 denominator) ----
  // use_pt: the residual is identically zero (the two distributions coincide): draw from p_t.
  for (int use_pt = 0; use_pt < 2; ++use_pt) {
    float part = 0.f;
    if (!use_pt) {
#pragma unroll 2
      for (int v = v0 + lane; v < v1; v += 32) {
        float a[N], b[N];
        const uint4 ra = load_raw(rd, v * N, w), rb = load_raw(rt, v * N, w);
        unpack(ra, a, tag);
        unpack(rb, b, tag);
        float acc = 0.f;
#pragma unroll
        for (int k = 0; k < N; ++k) acc += fmaxf(prob(b[k], ct) - prob(a[k], cd), 0.f);
        part += acc;
      }
    } else {
      for (int v = v0 + lane; v < v1; v += 32) {
        float b[N];
        load_vec(rt, v * N, w, b);
#pragma unroll
        for (int k = 0; k < N; ++k) part += prob(b[k], ct);
      }
    }
    part = warp_sum(part);
    if (lane == 0) sh_mass[warp] = part;
    __syncthreads();
    float mass = 0.f;
    for (int q = 0; q < kWarps; ++q) mass += sh_mass[q];                  // same order in every thread
    if (!use_pt && tid == 0 && resid_mass != nullptr) resid_mass[row] = mass;
    if (mass > 0.f || use_pt) {
      // ---- sweep 3: the warp whose segment contains x * mass walks it in order ----
      const float target = uniforms[row] * mass;
      float before = 0.f;
      int seg = -1;
      for (int q = 0; q < kWarps; ++q) {
        if (seg < 0 && before + sh_mass[q] > target) seg = q;
        if (seg < 0) before += sh_mass[q];
      }
      if (tid == 0) sh_token = -1;
      __syncthreads();
      float tgt = target;
      if (seg < 0) {
        // rounding left x * mass at or above the total: the last token with positive probability,
        // i.e. the walk below never crosses and reports the last positive entry of this segment
        seg = kWarps - 1;
        while (seg > 0 && !(sh_mass[seg] > 0.f)) --seg;
        tgt = INFINITY;
      }
      if (warp == seg) {
        float run = before;
        int found = -1, last_pos = -1;
        for (int vb = v0; vb < v1; vb += 32) {
          int v = vb + lane;
          float r[N];
          float lsum = 0.f;
          if (v < v1) {
            float a[N], b[N];
            load_vec(rd, v * N, w, a);
            load_vec(rt, v * N, w, b);
#pragma unroll
            for (int k = 0; k < N; ++k) {
              float pt = prob(b[k], ct), pd = prob(a[k], cd);
              r[k] = use_pt ? pt : fmaxf(pt - pd, 0.f);
              lsum += r[k];
            }
          } else {
#pragma unroll
            for (int k = 0; k < N; ++k) r[k] = 0.f;
          }
          // exclusive prefix over lanes
          float inc = lsum;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
          }
          float acc = run + inc - lsum;
          int mine = -1, mylast = -1;
#pragma unroll
          for (int k = 0; k < N; ++k) {
            if (r[k] > 0.f) mylast = v * N + k;
            acc += r[k];
            if (mine < 0 && r[k] > 0.f && acc > tgt) mine = v * N + k;
          }
          // first lane that crossed; last positive element seen so far
          unsigned hit = __ballot_sync(0xffffffffu, mine >= 0);
          unsigned pos = __ballot_sync(0xffffffffu, mylast >= 0);
          if (pos) last_pos = __shfl_sync(0xffffffffu, mylast, 31 - __clz(pos));
          if (hit) { found = __shfl_sync(0xffffffffu, mine, __ffs(hit) - 1); break; }
          run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) sh_token = found >= 0 ? found : last_pos;
      }
      __syncthreads();
      if (tid == 0) {
        int tk = sh_token;
        if (tk < 0) {
          // the chosen segment held no positive entry at all (possible only through rounding):
          // scan back for the last positive probability in the whole row
          for (int i = w - 1; i >= 0 && tk < 0; --i) {
            float pt = prob(cvt(rt[i]), ct), pd = prob(cvt(rd[i]), cd);
            if ((use_pt ? pt : pt - pd) > 0.f) tk = i;
          }
        }
        token[row] = tk;
      }
      break;
    }
    __syncthreads();
  }
}

// Bonus-token candidates of the parallel branching (Sec. III-C.1, Eq. 23): for every position the
// F_j largest draft logits, the token drafted at that position excluded; ties go to the lower
// token id; ids are written in ascending order at cand[cand_offsets[row] ...].  One block per
// position (segmented radix select over the logit row, which stays in L2 between its passes).
template <typename T>
__global__ void __launch_bounds__(1024)
branch_candidates_kernel(const T* __restrict__ zd, long long ldz, int w, const int* __restrict__ drafted,
                         const int* __restrict__ cand_offsets, int* __restrict__ cand) {
  const int row = blockIdx.x;
  const int off = cand_offsets[row], f = cand_offsets[row + 1] - off;
  if (f <= 0) return;
  const T* r = zd + (size_t)row * ldz;
  const int y = drafted != nullptr ? drafted[row] : -1;
  block_topk_by([&](int i) { return i == y ? -INFINITY : cvt(r[i]); }, w, min(f, w), false, nullptr,
                cand + off, nullptr);
}

}  // namespace corr
}  // namespace covspec
