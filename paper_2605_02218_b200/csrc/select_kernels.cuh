// Segmented top-k selection (preselect the M best fused scores; keep the B_vis largest energies)
// and the row gather used for Z_M (Eq. 13) and for the compacted output.
#pragma once
#include "common.cuh"
#include "score_kernels.cuh"

namespace covspec {

// Monotone map float -> uint32 (larger float = larger key).  -0 is folded onto +0 so that equal
// values share a key; NaN maps to the smallest key.
__device__ __forceinline__ unsigned order_key(float v) {
  if (v != v) return 0u;
  v += 0.0f;
  unsigned u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Block-wide exclusive scan of a small packed counter (blockDim.x multiple of 32, <= 1024).
// Returns the exclusive prefix; *total receives the block sum.
__device__ __forceinline__ unsigned block_exclusive_scan(unsigned v, unsigned* warp_tot,
                                                         unsigned* total) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  unsigned inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) warp_tot[w] = inc;
  __syncthreads();
  if (w == 0) {
    unsigned t = lane < nw ? warp_tot[lane] : 0u, ti = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned u = __shfl_up_sync(0xffffffffu, ti, o);
      if (lane >= o) ti += u;
    }
    if (lane < nw) warp_tot[lane] = ti - t;   // exclusive warp offsets
    if (lane == 31) warp_tot[32] = ti;        // block total
  }
  __syncthreads();
  *total = warp_tot[32];
  return warp_tot[w] + inc - v;
}

// Top-k of keys[0..n) by an 8-bit-per-pass radix select on the ordered keys, then an ordered
// emission: every element above the k-th value, plus the lowest-index elements equal to it until k
// are taken.  out[0..k) receives the selected positions in ascending order, mapped through `remap`
// when given.  `all_equal` treats every key as equal (selects the first k positions).
constexpr int kRankSelectMax = 1024;   // up to this many keys the selection ranks every key directly
constexpr int kRegKeys = 16;           // keys per thread the radix select keeps in registers

// One digit of the radix select, by the first warp: with `kk` keys still to take among those that
// match the digits fixed so far, the largest digit value d such that the keys with a larger digit
// number fewer than kk (digit 0 when none does); *sel_k = kk minus those keys.  Lane l sums the
// eight histogram bins 8 l .. 8 l + 7; a suffix scan over the lanes finds the lane that holds d.
__device__ __forceinline__ void select_digit(const unsigned* hist, unsigned kk, unsigned prefix, int shift,
                                             unsigned* sel_prefix, unsigned* sel_k) {
  const int lane = threadIdx.x & 31;
  if (kk == 0u) {                             // nothing left to take: no key is above the top digit
    if (lane == 0) { *sel_prefix = prefix | (255u << shift); *sel_k = 0u; }
    return;
  }
  unsigned h[8], mine = 0u;
#pragma unroll
  for (int e = 0; e < 8; ++e) { h[e] = hist[8 * lane + e]; mine += h[e]; }
  unsigned above = mine;                      // inclusive suffix sum over lanes >= this one
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_down_sync(0xffffffffu, above, o);
    if (lane + o < 32) above += t;
  }
  above -= mine;                              // keys in the bins of higher lanes
  const unsigned holds = __ballot_sync(0xffffffffu, above < kk && above + mine >= kk);
  const int owner = holds ? 31 - __clz(holds) : 0;
  if (lane == owner) {
    unsigned c = above;
    int e = 7;
    for (; e > 0; --e) {
      if (c + h[e] >= kk) break;
      c += h[e];
    }
    if (!holds) {                             // fewer matching keys than kk: digit 0 takes the rest
      e = 0;
      c = above + mine - h[0];
    }
    *sel_prefix = prefix | ((unsigned)(8 * lane + e) << shift);
    *sel_k = kk - c;
  }
}

// `load(i)` returns key i as a float; `status` may be nullptr (non-finite keys are then not reported).
template <typename LoadF>
__device__ void block_topk_by(LoadF load, int n, int k, bool all_equal,
                              const int* __restrict__ remap, int* __restrict__ out, int* status) {
  __shared__ unsigned hist[256];
  __shared__ unsigned whist[8][256];
  __shared__ unsigned sel_prefix, sel_k;
  __shared__ unsigned warp_tot[33];
  __shared__ unsigned skeys[kRankSelectMax];
  if (n <= kRankSelectMax) {
    // Small segments: rank of key i = number of keys that precede it in (larger value, lower index)
    // order, counted against the whole segment held in shared memory (every thread reads the same
    // key at the same time: a broadcast); key i is selected when its rank is below k.  Positions
    // are emitted in ascending order through a block scan of the selection flags.
    bool bad = false;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      float v = load(i);
      bad |= !all_equal && !(fabsf(v) <= 3.402823466e38f);
      skeys[i] = all_equal ? 0u : order_key(v);
    }
    if (bad && status != nullptr) atomicOr(status, kStatusNonFinite);
    __syncthreads();
    unsigned run = 0u;
    for (int base = 0; base < n; base += blockDim.x) {
      int i = base + threadIdx.x;
      unsigned sel = 0u;
      if (i < n) {
        unsigned ki = skeys[i];
        int rank = 0;
        for (int j = 0; j < i; ++j) rank += skeys[j] >= ki;       // equal keys with a lower index come first
        for (int j = i + 1; j < n; ++j) rank += skeys[j] > ki;
        sel = rank < k;
      }
      unsigned tot;
      unsigned ex = block_exclusive_scan(sel, warp_tot, &tot);
      if (sel && COVSPEC_IN_BOUNDS(run + ex, k, status)) out[run + ex] = remap ? remap[i] : i;
      run += tot;
    }
    return;
  }
  unsigned prefix = 0u, mask = 0u, kk = (unsigned)k;
  const int per = (n + (int)blockDim.x - 1) / (int)blockDim.x;
  if (per <= kRegKeys) {
    // Medium segments: every thread keeps a contiguous run of `per` keys in registers, so the four
    // digit passes read nothing from memory and the ordered emission needs one block scan.
    unsigned kreg[kRegKeys];
    const int i0 = (int)threadIdx.x * per;
    const int cnt = max(0, min(per, n - i0));
    bool bad = false;
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) {
      kreg[j] = 0u;
      if (j < cnt && !all_equal) {
        float v = load(i0 + j);
        bad |= !(fabsf(v) <= 3.402823466e38f);
        kreg[j] = order_key(v);
      }
    }
    if (bad && status != nullptr) atomicOr(status, kStatusNonFinite);
    if (!all_equal) {
      for (int shift = 24; shift >= 0; shift -= 8) {
        // scores of one request crowd into a few digit values: eight copies of the histogram
        // (one per warp modulo 8) spread the same-address updates
        for (int i = threadIdx.x; i < 8 * 256; i += blockDim.x) (&whist[0][0])[i] = 0u;
        __syncthreads();
        unsigned* myhist = whist[(threadIdx.x >> 5) & 7];
#pragma unroll
        for (int j = 0; j < kRegKeys; ++j)
          if (j < cnt && (kreg[j] & mask) == prefix) atomicAdd(&myhist[(kreg[j] >> shift) & 255u], 1u);
        __syncthreads();
        for (int i = threadIdx.x; i < 256; i += blockDim.x) {
          unsigned c = 0u;
#pragma unroll
          for (int q = 0; q < 8; ++q) c += whist[q][i];
          hist[i] = c;
        }
        __syncthreads();
        if (threadIdx.x < 32) select_digit(hist, kk, prefix, shift, &sel_prefix, &sel_k);
        __syncthreads();
        prefix = sel_prefix;
        kk = sel_k;
        mask |= 255u << shift;
      }
    }
    unsigned gt = 0u, eq = 0u;
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j)
      if (j < cnt) { gt += kreg[j] > prefix; eq += kreg[j] == prefix; }
    unsigned tot;
    unsigned ex = block_exclusive_scan(gt | (eq << 16), warp_tot, &tot);
    unsigned gt_before = ex & 0xffffu, eq_before = ex >> 16;
#pragma unroll
    for (int j = 0; j < kRegKeys; ++j) {
      if (j < cnt) {
        const bool g = kreg[j] > prefix, e = kreg[j] == prefix;
        if ((g || (e && eq_before < kk)) && COVSPEC_IN_BOUNDS(gt_before + min(eq_before, kk), k, status))
          out[gt_before + min(eq_before, kk)] = remap ? remap[i0 + j] : i0 + j;
        gt_before += g;
        eq_before += e;
      }
    }
    return;
  }
  if (!all_equal) {
    bool bad = false;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0u;
      __syncthreads();
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        float v = load(i);
        if (shift == 24) bad |= !(fabsf(v) <= 3.402823466e38f);
        unsigned key = order_key(v);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (threadIdx.x < 32) select_digit(hist, kk, prefix, shift, &sel_prefix, &sel_k);
      __syncthreads();
      prefix = sel_prefix;
      kk = sel_k;
      mask |= 255u << shift;
    }
    if (bad && status != nullptr) atomicOr(status, kStatusNonFinite);
  }
  // Ordered emission.  kk = how many elements equal to the threshold are taken.
  unsigned run_gt = 0u, run_eq = 0u;
  for (int base = 0; base < n; base += blockDim.x) {
    int i = base + threadIdx.x;
    unsigned gt = 0u, eq = 0u;
    if (i < n) {
      if (all_equal) eq = 1u;
      else {
        unsigned key = order_key(load(i));
        gt = key > prefix; eq = key == prefix;
      }
    }
    unsigned tot;
    unsigned ex = block_exclusive_scan(gt | (eq << 16), warp_tot, &tot);
    unsigned gt_before = run_gt + (ex & 0xffffu), eq_before = run_eq + (ex >> 16);
    if (gt || (eq && eq_before < kk)) {
      unsigned pos = gt_before + min(eq_before, kk);
      if (COVSPEC_IN_BOUNDS(pos, k, status)) out[pos] = remap ? remap[i] : i;
    }
    run_gt += tot & 0xffffu;
    run_eq += tot >> 16;
  }
}

__device__ __forceinline__ void block_topk(const float* __restrict__ keys, int n, int k, bool all_equal,
                                           const int* __restrict__ remap, int* __restrict__ out, int* status) {
  block_topk_by([&](int i) { return keys[i]; }, n, k, all_equal, remap, out, status);
}

// Preselection: one block per request, the M best fused scores -> presel (ascending token index).
__global__ void __launch_bounds__(1024)
preselect_kernel(const float* __restrict__ s_fused, const ReqPlan* __restrict__ plan,
                 int* __restrict__ presel, int* status) {
  ReqPlan rp = plan[blockIdx.x];
  block_topk(s_fused + rp.vis_off, rp.n, rp.m, false, nullptr, presel + rp.presel_off, status);
}

// Eq. 12 and the preselection in one launch (the fused call): the block that fused a request's
// scores selects its M best right away.
__global__ void __launch_bounds__(1024)
fuse_preselect_kernel(const float* __restrict__ s_query, const float* __restrict__ s_act,
                      const ReqPlan* __restrict__ plan, float lambda, int mode,
                      float* __restrict__ s_fused, int* __restrict__ presel, int* status) {
  __shared__ float scratch[32];
  ReqPlan rp = plan[blockIdx.x];
  fuse_request(rp, s_query, s_act, lambda, mode, s_fused, scratch, status);
  __syncthreads();                                  // the block's own global writes are visible to it
  block_topk(s_fused + rp.vis_off, rp.n, rp.m, false, nullptr, presel + rp.presel_off, status);
}

// Final selection: one block per request, the B_vis largest energies among the M preselected
// tokens -> keep_idx (token indices, ascending).  Requests whose stage 2 is skipped keep their
// whole preselected set (B_vis == M).
__global__ void __launch_bounds__(1024)
final_select_kernel(const float* __restrict__ energy, const int* __restrict__ presel,
                    const ReqPlan* __restrict__ plan, int* __restrict__ keep_idx, int* status) {
  ReqPlan rp = plan[blockIdx.x];
  block_topk(energy + rp.presel_off, rp.m, rp.b_vis, rp.stage2 == 0, presel + rp.presel_off,
             keep_idx + rp.keep_off, status);
}

// out[row, :] = src[vis_off(b) + idx[row], :] as 16-byte vectors; one warp per output row (its
// first lane looks the request up), four vectors per lane in flight.
// `use_presel` selects which plan offsets delimit the rows of a request (presel_off / keep_off).
constexpr int kGatherWarps = 8;
__global__ void __launch_bounds__(kGatherWarps * 32)
gather_rows_kernel(const uint4* __restrict__ src, const int* __restrict__ idx,
                   const ReqPlan* __restrict__ plan, int batch, int use_presel, int row_vec16, int rows,
                   uint4* __restrict__ dst, int* __restrict__ out_pos, int* status) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kGatherWarps + (threadIdx.x >> 5);
  if (row >= rows) return;
  long long first = 0;
  int tok = 0;
  if (lane == 0) {
    int b = find_request(row, batch, [&](int q) {
      return use_presel ? plan[q].presel_off : plan[q].keep_off;
    });
    tok = idx[row];
    // checked build: a token index outside its request is reported and the row is skipped
    first = COVSPEC_IN_BOUNDS(tok, plan[b].n, status) ? (long long)plan[b].vis_off + tok : -1;
    if (out_pos != nullptr) out_pos[row] = tok;
  }
  first = __shfl_sync(0xffffffffu, first, 0);
  if (first < 0) return;
  const uint4* s = src + (size_t)first * row_vec16;
  uint4* d = dst + (size_t)row * row_vec16;
  int v = lane;
  for (; v + 96 < row_vec16; v += 128) {
    uint4 a = __ldg(s + v), b2 = __ldg(s + v + 32), c = __ldg(s + v + 64), e = __ldg(s + v + 96);
    d[v] = a; d[v + 32] = b2; d[v + 64] = c; d[v + 96] = e;
  }
  for (; v < row_vec16; v += 32) d[v] = __ldg(s + v);
}

inline unsigned gather_grid(long long rows) { return (unsigned)((rows + kGatherWarps - 1) / kGatherWarps); }

}  // namespace covspec
