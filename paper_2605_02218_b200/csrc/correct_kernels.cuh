// Device-side gating and correction over the vocabulary (Eq. 2, 4, 5, 6, 16, 17; Sec. III-C.2):
// from the draft logits and the target logits of one position, the draft distribution's top-2 margin
// and gate, the acceptance probability of the drafted token, the residual distribution
// max(p_t - p_d, 0) / mass and a token drawn from it by inverse CDF with a uniform number supplied by
// the caller.
//
// One cluster of two CTAs per position.  Both logit rows (2 * W * elem bytes, ~600 KB at W = 152 k
// in 16 bits) are read from HBM once; the second sweep (residual mass) and the short third one (the
// cumulative sum inside the one warp segment that contains the sample) find them in L2.  Each warp
// owns a contiguous segment of the row and reads it with coalesced 16-byte vectors, so the order of
// the cumulative sum is (segment, vector, lane, element).  The method needs two exponentials per
// vocabulary entry for the denominators and two more for the residual; they run on the
// special-function units (16 per clock per SM), which bound the kernel before HBM does.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"
#include "select_kernels.cuh"

namespace covspec {
namespace corr {

constexpr int kClusterCtas = 2;                       // CTAs that share one position
constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;                         // resident CTAs per SM the register budget allows
constexpr int kSegs = kClusterCtas * kWarps;         // warp segments of a row
constexpr int kMaxChunks = 256;                      // chunks of a segment whose totals fit in shared memory

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

// Branch-free trackers of the two largest logits of the vectors one thread sees.  The 16-bit types
// keep two independent (largest, second) pairs, one per half of a packed register, on the raw bits:
// three packed min / max instructions per two logits, exact because a maximum rounds nothing.
template <typename T> struct Top2Run;
template <> struct Top2Run<float> {
  float a = -INFINITY, b = -INFINITY;
  __device__ __forceinline__ void add(const uint4& raw) {
    const float z[4] = {__uint_as_float(raw.x), __uint_as_float(raw.y), __uint_as_float(raw.z), __uint_as_float(raw.w)};
#pragma unroll
    for (int k = 0; k < 4; ++k) { b = fmaxf(b, fminf(a, z[k])); a = fmaxf(a, z[k]); }
  }
  __device__ __forceinline__ Top2 result() const { return Top2{a, b}; }
};
template <> struct Top2Run<__half> {
  __half2 a = __half2half2(__ushort_as_half((unsigned short)0xfc00)), b = a;       // -inf
  __device__ __forceinline__ void add(const uint4& raw) {
    const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
    for (int k = 0; k < 4; ++k) { b = __hmax2(b, __hmin2(a, h[k])); a = __hmax2(a, h[k]); }
  }
  __device__ __forceinline__ Top2 result() const {
    Top2 t{__low2float(a), __low2float(b)};
    t.add(__high2float(a)); t.add(__high2float(b));
    return t;
  }
};
template <> struct Top2Run<__nv_bfloat16> {
  __nv_bfloat162 a = __bfloat162bfloat162(__ushort_as_bfloat16((unsigned short)0xff80)), b = a;   // -inf
  __device__ __forceinline__ void add(const uint4& raw) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int k = 0; k < 4; ++k) { b = __hmax2(b, __hmin2(a, h[k])); a = __hmax2(a, h[k]); }
  }
  __device__ __forceinline__ Top2 result() const {
    Top2 t{__low2float(a), __low2float(b)};
    t.add(__high2float(a)); t.add(__high2float(b));
    return t;
  }
};

// How far above the reference of a running sum a logit may lie before the sum is moved to a new
// reference: exp(60) ~ 1e26 leaves room for a whole vocabulary of such terms in float32.
constexpr float kRefSlack = 60.f;

// ---- thread-block cluster helpers (a position is shared by the kClusterCtas CTAs of a cluster) ----
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// A float of the shared memory of CTA `cta` of the cluster, at the address `p` has in this CTA.
__device__ __forceinline__ float peer_float(const float* p, unsigned cta) {
  unsigned local = (unsigned)__cvta_generic_to_shared(p), remote;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(cta));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

// rows: positions; w: vocabulary size; ldz: elements between consecutive rows (multiple of 16 bytes).
//
// One cluster of kClusterCtas CTAs per position, two CTAs resident per SM: the sweep that streams
// the rows from HBM in one CTA overlaps the sweeps that re-read them from L2 (special-function
// bound) in the other CTA of the SM, while the positions in flight (one per cluster: 148 x 600 KB)
// still fit in L2 - with one whole position per CTA and two CTAs per SM they would not.  The row is
// cut into kSegs contiguous warp segments in row order (CTA rank, warp); partial results cross the
// cluster through distributed shared memory.
template <typename T>
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kThreads, kCtasPerSm)
correct_kernel(const T* __restrict__ zd, const T* __restrict__ zt, long long ldz, int w,
               const int* __restrict__ drafted, const float* __restrict__ uniforms, float gamma,
               float* __restrict__ margin, int* __restrict__ gate, float* __restrict__ accept,
               float* __restrict__ resid_mass, int* __restrict__ token) {
  constexpr int N = Vec<T>::N;
  __shared__ MaxSum sh_d[kWarps], sh_t[kWarps];
  __shared__ Top2 sh_top[kWarps];
  __shared__ float sh_part[6];                 // this CTA's (max, sum) pairs and two largest draft logits
  __shared__ float sh_mass[2][kWarps];         // this CTA's warp masses (residual pass, p_t pass)
  __shared__ float sh_all[kSegs];              // warp masses of the whole cluster, in row order
  __shared__ float sh_chunk[kMaxChunks];       // totals of the 32-vector chunks of the segment that holds the sample
  __shared__ float bc[2];
  __shared__ int sh_token;
  const unsigned crank = cluster_rank();
  const int row = blockIdx.x / kClusterCtas, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg_id = (int)crank * kWarps + warp;
  const T* rd = zd + (size_t)row * ldz;
  const T* rt = zt + (size_t)row * ldz;
  const T* const tag = nullptr;
  // scalars of the position, requested now so that their latency hides behind the first sweep
  const float x_uniform = __ldg(uniforms + row);
  float zd_y = 0.f, zt_y = 0.f;
  const bool has_y = accept != nullptr && drafted != nullptr;
  if (has_y && tid == 0 && crank == 0) {
    const int y = __ldg(drafted + row);
    zd_y = cvt(rd[y]);
    zt_y = cvt(rt[y]);
  }
  // contiguous segment of this warp, in whole vectors
  const int nvec = (w + N - 1) / N;
  const int vec_per_seg = (nvec + kSegs - 1) / kSegs;
  const int v0 = min(nvec, seg_id * vec_per_seg), v1 = min(nvec, v0 + vec_per_seg);

  // ---- sweep 1: softmax denominators of both rows (Eq. 2, 4), two largest draft logits (Eq. 16) ----
  // The sums run relative to a reference logit of this thread, in the base-2 domain:
  // exp(z - m) = 2^(z log2(e) - m log2(e)).  The reference is the largest logit of the first vector
  // and moves only when a logit lies more than kRefSlack above it (any reference gives the same
  // quotient; the slack keeps the terms inside the float32 range), so the branch is rarely taken.
  MaxSum md{-INFINITY, 0.f}, mt{-INFINITY, 0.f};
  float nd = 0.f, nt = 0.f;                     // -m log2(e) of the two references
  float thr_d = -INFINITY, thr_t = -INFINITY;   // reference + slack
  Top2Run<T> top_run;
  auto sweep1 = [&](const uint4& ra, const uint4& rb) {
    // every vector holds at least one element of the vocabulary; 2^(-inf) = 0 takes care of padding
    const float va = vec_max(ra, tag), vb = vec_max(rb, tag);
    if (va > thr_d) { md.s *= __expf(md.m - va); md.m = va; nd = -va * kLog2e; thr_d = va + kRefSlack; }
    if (vb > thr_t) { mt.s *= __expf(mt.m - vb); mt.m = vb; nt = -vb * kLog2e; thr_t = vb + kRefSlack; }
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
    top_run.add(ra);
  };
  // vectors that lie wholly inside the row, then the one that straddles its end (if any)
  const int nfull = w / N, f1 = min(v1, nfull);
  const bool owns_tail = nfull < nvec && nfull >= v0 && nfull < v1 && ((nfull - v0) & 31) == lane;
  {
    const uint4* pa = reinterpret_cast<const uint4*>(rd) + v0 + lane;
    const uint4* pb = reinterpret_cast<const uint4*>(rt) + v0 + lane;
#pragma unroll 2
    for (int v = v0 + lane; v < f1; v += 32, pa += 32, pb += 32) sweep1(__ldg(pa), __ldg(pb));
    if (owns_tail) sweep1(load_raw(rd, nfull * N, w), load_raw(rt, nfull * N, w));
  }
  Top2 top = top_run.result();
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
      sh_part[0] = md.m; sh_part[1] = md.s; sh_part[2] = mt.m; sh_part[3] = mt.s;
      sh_part[4] = top.a; sh_part[5] = top.b;
    }
  }
  cluster_sync();                               // every CTA's partial results are in its shared memory
  if (warp == 0) {
    // the same merge, in rank order, in every CTA of the cluster
    md = MaxSum{-INFINITY, 0.f}; mt = md; top = Top2{-INFINITY, -INFINITY};
    // lane 6 c + k fetches value k of CTA c; the values are then handed round by shuffles
    float mine = 0.f;
    if (lane < 6 * kClusterCtas) mine = peer_float(&sh_part[lane % 6], (unsigned)(lane / 6));
    for (int c = 0; c < kClusterCtas; ++c) {
      MaxSum od{__shfl_sync(0xffffffffu, mine, 6 * c), __shfl_sync(0xffffffffu, mine, 6 * c + 1)};
      MaxSum ot{__shfl_sync(0xffffffffu, mine, 6 * c + 2), __shfl_sync(0xffffffffu, mine, 6 * c + 3)};
      Top2 otop{__shfl_sync(0xffffffffu, mine, 6 * c + 4), __shfl_sync(0xffffffffu, mine, 6 * c + 5)};
      md.merge(od); mt.merge(ot); top.merge(otop);
    }
    if (lane == 0) {
      // exponent offsets of the two distributions: p = 2^(z log2(e) + bc)
      bc[0] = -(md.m * kLog2e + log2f(md.s));
      bc[1] = -(mt.m * kLog2e + log2f(mt.s));
      if (crank == 0) {
        float m = (1.f - (top.b > -INFINITY ? __expf(top.b - top.a) : 0.f)) * __expf(top.a - md.m) / md.s;
        margin[row] = m;
        gate[row] = m < gamma ? 1 : 0;                                       // Eq. 17
        if (accept != nullptr) {
          float al = 1.f;
          if (has_y) {
            float pd = __expf(zd_y - md.m) / md.s, pt = __expf(zt_y - mt.m) / mt.s;
            al = pd > 0.f ? fminf(1.f, pt / pd) : 1.f;                       // Eq. 5
          }
          accept[row] = al;
        }
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
      auto sweep2 = [&](const uint4& ra, const uint4& rb) {
        float a[N], b[N];
        unpack(ra, a, tag);
        unpack(rb, b, tag);
        float acc = 0.f;
#pragma unroll
        for (int k = 0; k < N; ++k) acc += fmaxf(prob(b[k], ct) - prob(a[k], cd), 0.f);
        part += acc;
      };
      const uint4* pa = reinterpret_cast<const uint4*>(rd) + v0 + lane;
      const uint4* pb = reinterpret_cast<const uint4*>(rt) + v0 + lane;
#pragma unroll 2
      for (int v = v0 + lane; v < f1; v += 32, pa += 32, pb += 32) sweep2(__ldg(pa), __ldg(pb));
      if (owns_tail) sweep2(load_raw(rd, nfull * N, w), load_raw(rt, nfull * N, w));
    } else {
      for (int v = v0 + lane; v < v1; v += 32) {
        float b[N];
        load_vec(rt, v * N, w, b);
#pragma unroll
        for (int k = 0; k < N; ++k) part += prob(b[k], ct);
      }
    }
    part = warp_sum(part);
    if (lane == 0) sh_mass[use_pt][warp] = part;
    cluster_sync();                             // the masses of every CTA are in its shared memory
    if (tid < kSegs) sh_all[tid] = peer_float(&sh_mass[use_pt][tid % kWarps], (unsigned)(tid / kWarps));
    __syncthreads();
    float mass = 0.f;
    for (int q = 0; q < kSegs; ++q) mass += sh_all[q];                    // same order in every thread
    if (!use_pt && crank == 0 && tid == 0 && resid_mass != nullptr) resid_mass[row] = mass;
    if (mass > 0.f || use_pt) {
      // ---- sweep 3: the warp whose segment contains x * mass walks it in order ----
      const float target = x_uniform * mass;
      float before = 0.f;
      int seg = -1;
      for (int q = 0; q < kSegs; ++q) {
        if (seg < 0 && before + sh_all[q] > target) seg = q;
        if (seg < 0) before += sh_all[q];
      }
      if (tid == 0) sh_token = -2;              // -2: the segment belongs to another CTA
      __syncthreads();
      float tgt = target;
      if (seg < 0) {
        // rounding left x * mass at or above the total: the last token with positive probability,
        // i.e. the walk below never crosses and reports the last positive entry of this segment
        seg = kSegs - 1;
        while (seg > 0 && !(sh_all[seg] > 0.f)) --seg;
        tgt = INFINITY;
      }
      // The segment is walked in chunks of 32 vectors.  The warps of the CTA that owns it first
      // sum the chunks in parallel; the walk then starts at the first chunk whose running total
      // passes the target (running totals added up in chunk order, as the walk itself would).
      const int sv0 = min(nvec, seg * vec_per_seg), sv1 = min(nvec, sv0 + vec_per_seg);
      const int nchunks = (sv1 - sv0 + 31) >> 5;
      const bool mine_cta = seg / kWarps == (int)crank;
      const bool skip_ahead = mine_cta && nchunks <= kMaxChunks && tgt != INFINITY;
      auto chunk_values = [&](int v, float (&r)[N]) -> float {
        float lsum = 0.f;
        if (v < sv1) {
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
        return lsum;
      };
      if (skip_ahead) {
        for (int c = warp; c < nchunks; c += kWarps) {
          float r[N];
          float inc = chunk_values(sv0 + 32 * c + lane, r);
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {          // the same inclusive scan the walk uses
            float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
          }
          if (lane == 31) sh_chunk[c] = inc;
        }
      }
      __syncthreads();
      if (seg_id == seg) {
        float run = before;
        int first_chunk = 0;
        if (skip_ahead) {
          while (first_chunk + 1 < nchunks && !(run + sh_chunk[first_chunk] > tgt)) run += sh_chunk[first_chunk++];
        }
        int found = -1, last_pos = -1;
        for (int vb = v0 + 32 * first_chunk; vb < v1; vb += 32) {
          int v = vb + lane;
          float r[N];
          float lsum = chunk_values(v, r);
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
      if (tid == 0 && sh_token != -2) {
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
  cluster_sync();                               // no CTA leaves while its shared memory may be read
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
