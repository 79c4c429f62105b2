// Tensor-core pieces of the low-rank redundancy step (Eq. 13-15): the Gram kernel of the stacked
// preselected tokens, and the shared-memory plan, triangular solve and float64 partial-Gram
// routines of the block power step (the step itself is part of the fused kernel in
// subspace_fused.cuh) with which the subspace iteration reaches the top-r eigenspace.
//
// G = Z_M^T Z_M (Eq. 13-14; its eigenpairs are sigma_k^2 and the right singular vectors of Z_M) is
// produced by tcgen05.mma kind::f16 from the gathered bf16 rows, accumulated in float32 in TMEM and
// stored as two bf16 planes G = G_hi + G_lo (16 mantissa bits), which is the operand format of the
// power step.  One power step computes, per 128-row tile of one request,
//     T      = G[tile, :] * Y                    3 MMAs per k-step: hi*hi + lo*hi + hi*lo
//     Y_next = T * L^-T                          forward substitution per row, L = chol(Y^T Y)
//     B_tile = Y_next[tile]^T Y_next[tile]       float64 partial Gram of the new block
// so that orthonormalising the previous block (Y L^-T) never needs its own pass over memory: the
// triangular factor is applied to the product instead (G (Y L^-T) = (G Y) L^-T).
//
// Layouts.  All requests share 2-D arrays so that one tensor map serves the whole batch:
//   G planes   [sum M_b (+pad), ld]  row presel_off(b) + i, column j          (ld = max M rounded to 64)
//   Y planes   [batch * 160, ld]     row b*160 + basis vector, column = token position (K-major B operand)
//   Yf         [sum M_b, 160]        float32 copy of the last block, one token per row
//   partial    [tiles, 13440]        8 x 8 tiles of the lower triangle in float64 (subspace_fused.cuh)
// Columns of G and Y between M_b and the next multiple of 64 are kept finite / zero respectively so
// that whole 64-wide k-chunks can be multiplied.
#pragma once
#include "tc_common.cuh"

namespace covspec {
namespace sub {

using namespace tc;

constexpr int kTile = 128;                 // rows per tile (UMMA M); Gram column tile (UMMA N)
constexpr int kBK = 64;                    // bf16 elements per k-chunk (one 128-byte swizzle row)
constexpr int kTriMax = kPMax * (kPMax + 1) / 2;          // 12880 packed lower-triangle entries
// Triangular factor as the power step reads it: row i holds L[j][i] for j = (i & ~3) .. P-1 so that
// 8-column blocks are two aligned float4 loads.  Largest size (P = 160) and the per-request stride
// (factor followed by the reciprocal diagonal).
constexpr int kLtFloats = kPMax * kPMax - 8 * (kPMax / 4) * (kPMax / 4 - 1);   // 13120
constexpr int kLbufStride = kLtFloats + kPMax;                                  // 13280

__host__ __device__ __forceinline__ int tri_index(int a, int b) { return a * (a + 1) / 2 + b; }
// Offset of row i of the padded upper-triangular layout for width P (a multiple of 4).
__host__ __device__ __forceinline__ int lt_row_offset(int i, int P) {
  int a = i >> 2, b = i & 3;
  return i * P - 8 * a * (a - 1) - 4 * a * b;
}

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Row / column tile of the t-th lower-triangle tile (row-major over (ti, tj <= ti)).
__device__ __forceinline__ void tri_decode(int t, int& ti, int& tj) {
  ti = (int)((sqrtf(8.f * (float)t + 1.f) - 1.f) * 0.5f);
  while ((ti + 1) * (ti + 2) / 2 <= t) ++ti;
  while (ti * (ti + 1) / 2 > t) --ti;
  tj = t - ti * (ti + 1) / 2;
}

// ================================================================================================
// Gram kernel
// ================================================================================================
// Items are 128 x 256 blocks of the lower triangle (row tile ti, pair of column tiles 2 tjp and
// 2 tjp + 1, tjp <= ti / 2): per 64-element k-chunk a 16 KB row tile and a 32 KB column tile feed
// 128 x 256 x 64 products, two thirds of the operand bytes per product a square 128 x 128 item
// needs (the feed from L2 bounds this kernel).  The half of a block that lies above the diagonal
// (ti even, last pair) is computed and dropped.
constexpr int kGramStages = 4;
constexpr int kGramN = 2 * kTile;                         // columns of an item
constexpr int kGramBytesA = kTile * kBK * 2;              // 16 KB
constexpr int kGramStageBytes = kGramBytesA + kGramN * kBK * 2;   // 48 KB
constexpr int kGramSmem = kGramStages * kGramStageBytes + 1024 + 1024;
constexpr int kGramTmemCols = 512;                        // two 256-column accumulators
// Items of a request with nt row tiles, and the decoding of an item index.
__host__ __device__ __forceinline__ int gram_items(int nt) {
  int a = nt >> 1;
  return (nt & 1) ? (a + 1) * (a + 1) : a * (a + 1);
}
__device__ __forceinline__ void gram_decode(int t, int& ti, int& tjp) {
  ti = 0;
  for (int cnt = 1; t >= cnt; cnt = (ti >> 1) + 1) { t -= cnt; ++ti; }
  tjp = t;
}

struct GramParams {
  const ReqPlan* plan;
  int batch;
  int n_items;          // lower-triangle tiles over all stage-2 requests
  int k_chunks;         // ceil(d / 64)
  __nv_bfloat16* g_hi;
  __nv_bfloat16* g_lo;
  int ld;
  int* status;
};

__global__ void __launch_bounds__(192, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap map_z,   // gathered rows [sum M_b, d] bf16, 128-row boxes
               const __grid_constant__ CUtensorMap map_zw,  // the same tensor, 256-row boxes
               const GramParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kGramStages * kGramStageBytes);
  uint64_t* full = bars;                       // [kGramStages]
  uint64_t* empty = bars + kGramStages;        // [kGramStages]
  uint64_t* acc_full = bars + 2 * kGramStages; // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGramStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 128); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(tmem_slot, kGramTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  auto decode = [&](int item, ReqPlan& rp, int& ti, int& tjp) {
    int b = find_request(item, prm.batch, [&](int q) { return prm.plan[q].gram_tile_off; });
    rp = prm.plan[b];
    gram_decode(item - rp.gram_tile_off, ti, tjp);
  };

  if (warp == 4) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x) {
        ReqPlan rp; int ti, tj;
        decode(item, rp, ti, tj);
        for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
          int s = it % kGramStages;
          if (!(ok = mbar_wait(&empty[s], ((it / kGramStages) & 1u) ^ 1u, abort_flag))) break;
          mbar_expect_tx(&full[s], kGramStageBytes);
          uint32_t dst = smem_u32(smem + s * kGramStageBytes);
          tma_load_2d(dst, &map_z, kc * kBK, rp.presel_off + ti * kTile, &full[s]);
          tma_load_2d(dst + kGramBytesA, &map_zw, kc * kBK, rp.presel_off + tj * kGramN, &full[s]);
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(kTile, kGramN);
      uint32_t it = 0, n = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x, ++n) {
        int buf = n & 1;
        if (!(ok = mbar_wait(&acc_empty[buf], ((n >> 1) & 1u) ^ 1u, abort_flag))) break;
        tc_fence_after();
        for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
          int s = it % kGramStages;
          if (!(ok = mbar_wait(&full[s], (it / kGramStages) & 1u, abort_flag))) break;
          tc_fence_after();
          uint32_t a_addr = smem_u32(smem + s * kGramStageBytes);
          uint64_t adesc = umma_desc(a_addr), bdesc = umma_desc(a_addr + kGramBytesA);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16(tmem_base + buf * kGramN, adesc + 2 * k, bdesc + 2 * k, idesc, (kc | k) != 0);
          umma_commit(&empty[s]);
        }
        if (!ok) break;
        umma_commit(&acc_full[buf]);
      }
    }
    __syncwarp();
  } else {
    const int r = warp * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    uint32_t n = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x, ++n) {
      ReqPlan rp; int ti, tj;
      decode(item, rp, ti, tj);
      int buf = n & 1;
      if (!(ok = mbar_wait(&acc_full[buf], (n >> 1) & 1u, abort_flag))) break;
      tc_fence_after();
      const int row = ti * kTile + r;                 // row of G inside the request
      const bool row_ok = row < rp.m;
      const size_t ld = (size_t)prm.ld;
#pragma unroll 1
      for (int c4 = 0; c4 < 8; ++c4) {
        const int tc = 2 * tj + (c4 >> 2);            // column tile of this group of 32 columns
        if (tc > ti) break;                           // above the diagonal: dropped
        float v[32];
        tmem_ld32(t_lane + buf * kGramN + c4 * 32, v);
        const int col0 = tj * kGramN + c4 * 32;
        // entries outside the request's M x M block are stored as zeros: the power step multiplies
        // whole 64-wide k-chunks and must not meet stale non-finite values in the padding
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (col0 + e >= rp.m || !row_ok) v[e] = 0.f;
        uint32_t ph[16], pl[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          __nv_bfloat162 hi = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
          ph[e] = *reinterpret_cast<uint32_t*>(&hi);
          pl[e] = pack_bf16(v[2 * e] - __low2float(hi), v[2 * e + 1] - __high2float(hi));
        }
        if (row_ok && col0 < prm.ld) {
          size_t o = ((size_t)rp.presel_off + row) * ld + col0;
          uint4* dh = reinterpret_cast<uint4*>(prm.g_hi + o);
          uint4* dl = reinterpret_cast<uint4*>(prm.g_lo + o);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            dh[q] = make_uint4(ph[4 * q], ph[4 * q + 1], ph[4 * q + 2], ph[4 * q + 3]);
            dl[q] = make_uint4(pl[4 * q], pl[4 * q + 1], pl[4 * q + 2], pl[4 * q + 3]);
          }
        }
        if (ti != tc && row < prm.ld) {
          // mirrored tile: G[col, row] = G[row, col]; consecutive threads write consecutive columns
          unsigned short* mh = reinterpret_cast<unsigned short*>(prm.g_hi);
          unsigned short* ml = reinterpret_cast<unsigned short*>(prm.g_lo);
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            int mrow = col0 + e;
            if (mrow < rp.m) {
              size_t o = ((size_t)rp.presel_off + mrow) * ld + row;
              uint32_t wh = ph[e >> 1], wl = pl[e >> 1];
              mh[o] = (unsigned short)((e & 1) ? (wh >> 16) : (wh & 0xffffu));
              ml[o] = (unsigned short)((e & 1) ? (wl >> 16) : (wl & 0xffffu));
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem_base, kGramTmemCols);
  if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, kStatusTimeout);
}

// Splits a float32 Gram matrix (CUDA-core path, float32 inputs) into the two bf16 planes.
__global__ void __launch_bounds__(256)
split_planes_kernel(const ReqPlan* __restrict__ plan, const float* __restrict__ G,
                    __nv_bfloat16* __restrict__ g_hi, __nv_bfloat16* __restrict__ g_lo, int ld) {
  ReqPlan rp = plan[blockIdx.y];
  if (!rp.stage2) return;
  int cols = (rp.m + 63) & ~63;
  int total = rp.m * cols;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
    int i = e / cols, j = e % cols;
    float v = j < rp.m ? G[rp.g_off + (size_t)i * rp.ldm + j] : 0.f;
    __nv_bfloat16 hi, lo;
    split_bf16(v, hi, lo);
    size_t o = ((size_t)rp.presel_off + i) * ld + j;
    g_hi[o] = hi; g_lo[o] = lo;
  }
}

// Start block of the subspace iteration: entries uniform in [-1, 1) from a counter hash of
// (request, basis vector, position); zero in the padding columns and in the unused basis rows
// p .. round_up(p, 16) - 1 of both plane buffers (the MMA reads them, nothing else writes them).
// The same launch resets the per-request words of the fused subspace kernel (three counters and the
// index of the last step per request, then the abort word) and writes zero energies for the requests that skip stage 2.
__global__ void __launch_bounds__(256)
basis_init_kernel(const ReqPlan* __restrict__ plan, __nv_bfloat16* __restrict__ y_hi,
                  __nv_bfloat16* __restrict__ y_lo, __nv_bfloat16* __restrict__ y2_hi,
                  __nv_bfloat16* __restrict__ y2_lo, int ld, float* __restrict__ energy,
                  unsigned* __restrict__ sync, int batch, int last_step) {
  ReqPlan rp = plan[blockIdx.y];
  if (blockIdx.x == 0) {
    if (threadIdx.x < 8) sync[blockIdx.y * 8 + threadIdx.x] = threadIdx.x == 3 ? (unsigned)last_step : 0u;
    if (blockIdx.y == 0 && threadIdx.x >= 32 && threadIdx.x < 36) sync[batch * 8 + threadIdx.x - 32] = 0u;
    if (!rp.stage2)
      for (int i = threadIdx.x; i < rp.m; i += blockDim.x) energy[rp.presel_off + i] = 0.f;
  }
  if (!rp.stage2) return;
  int cols = (rp.m + 63) & ~63;
  int rows = (rp.p + 15) & ~15;
  int total = rows * cols;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
    int j = e / cols, i = e % cols;
    float v = 0.f;
    if (j < rp.p && i < rp.m) {
      unsigned h = (unsigned)(j * rp.m + i) * 0x9E3779B1u ^ ((unsigned)blockIdx.y + 1u) * 0x85EBCA77u;
      h ^= h >> 16; h *= 0x7FEB352Du; h ^= h >> 15; h *= 0x846CA68Bu; h ^= h >> 16;
      v = (float)(h >> 8) * (2.0f / 16777216.0f) - 1.0f;
    }
    __nv_bfloat16 hi, lo;
    split_bf16(v, hi, lo);
    size_t o = ((size_t)blockIdx.y * kPMax + j) * ld + i;
    y_hi[o] = hi; y_lo[o] = lo;
    if (j >= rp.p) { y2_hi[o] = hi; y2_lo[o] = lo; }
  }
}

// ================================================================================================
// Power step: shared-memory plan and epilogue routines
// ================================================================================================
constexpr int kPowStages = 2;
constexpr int kPowBytesA = kTile * kBK * 2;              // one plane of the G tile, 16 KB
constexpr int kPowBytesB = kPMax * kBK * 2;              // one plane of the Y tile, 20 KB
constexpr int kPowStageBytes = 2 * kPowBytesA + 2 * kPowBytesB;   // 72 KB
constexpr int kXsLd = kTile + 4;                         // row stride of the staged block (floats)
constexpr int kXsBytes = (kPMax * kXsLd * 4 + 1023) / 1024 * 1024;   // one staged block [kPMax][kXsLd] of float32
// The ring is followed by padding up to two staged blocks: after the MMAs the region holds the new
// block, and either the previous block (last step) or the float64 slabs of the Gram accumulation.
constexpr int kPowRegion = 2 * kXsBytes > kPowStages * kPowStageBytes ? 2 * kXsBytes : kPowStages * kPowStageBytes;
constexpr int kPowSmem = kPowRegion + kLbufStride * 4 + 1024 + 1024;
constexpr int kPowTmemCols = 256;
constexpr int kPowThreads = 320;                         // 8 epilogue warps, TMA producer, MMA issuer
static_assert(kPMax * kXsLd * 4 <= kPowStages * kPowStageBytes, "staged block must fit in the ring");

__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds_v4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

// Four rows i .. i+3 of the triangular layout (two float4 each) and the matching four x_i.
struct SolveGroup {
  float x[4];
  float4 l[4][2];
};
__device__ __forceinline__ void solve_group_load(SolveGroup& g, uint32_t xs_row, uint32_t lt_at, int stride) {
#pragma unroll
  for (int q = 0; q < 4; ++q) g.x[q] = lds_f32(xs_row + q * kXsLd * 4);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    g.l[q][0] = lds_v4(lt_at + q * stride * 4);
    g.l[q][1] = lds_v4(lt_at + q * stride * 4 + 16);
  }
}
__device__ __forceinline__ void solve_group_apply(const SolveGroup& g, float (&acc)[8]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[0] -= g.x[q] * g.l[q][0].x; acc[1] -= g.x[q] * g.l[q][0].y;
    acc[2] -= g.x[q] * g.l[q][0].z; acc[3] -= g.x[q] * g.l[q][0].w;
    acc[4] -= g.x[q] * g.l[q][1].x; acc[5] -= g.x[q] * g.l[q][1].y;
    acc[6] -= g.x[q] * g.l[q][1].z; acc[7] -= g.x[q] * g.l[q][1].w;
  }
}

// acc[0..7] -= sum over the groups g0 .. g1-1 (four solved columns i each; g1 - g0 even) of
// x_i * L[jb + e][i]: the part of the forward substitution for columns jb .. jb+7 that only needs
// x_i already staged in xs[i * kXsLd + r].  The loads of one group are in flight while the previous
// group is applied.
__device__ __forceinline__ void solve_apply_groups(float (&acc)[8], int jb, int g0, int g1, uint32_t lt,
                                                   uint32_t xs, int r, int P) {
  if (g1 <= g0) return;
  uint32_t xr = xs + (r + 4 * g0 * kXsLd) * 4;
  uint32_t at = lt + (4 * g0 * P - 8 * g0 * (g0 - 1) + jb - 4 * g0) * 4;   // row 4 g0 of the layout, column jb
  int stride = P - 4 * g0;                         // rows 4a .. 4a+3 have P - 4a entries
  SolveGroup ga, gb;
  solve_group_load(ga, xr, at, stride);
  for (int g = g0; g < g1; g += 2) {
    xr += 4 * kXsLd * 4; at += (4 * stride - 4) * 4; stride -= 4;
    solve_group_load(gb, xr, at, stride);
    solve_group_apply(ga, acc);
    xr += 4 * kXsLd * 4; at += (4 * stride - 4) * 4; stride -= 4;
    if (g + 2 < g1) solve_group_load(ga, xr, at, stride);
    solve_group_apply(gb, acc);
  }
}
// Triangular solve inside the block of columns jb .. jb+7: acc holds t - (contributions of the
// columns before jb) on entry and x[jb..jb+7] on return.
__device__ __forceinline__ void solve_inblock8(float (&acc)[8], int jb, uint32_t lt, uint32_t dinv, int P) {
#pragma unroll
  for (int jj = 0; jj < 8; ++jj) {
    float x = acc[jj] * lds_f32(dinv + (jb + jj) * 4);
    acc[jj] = x;
    uint32_t lr = lt + (lt_row_offset(jb + jj, P) - (jj & ~3)) * 4;
#pragma unroll
    for (int j2 = jj + 1; j2 < 8; ++j2) acc[j2] -= x * lds_f32(lr + j2 * 4);
  }
}

// C (8x8 float64, two entries per thread) += A (8x4) * B (4x8): one tensor-core instruction.
__device__ __forceinline__ void dmma_8x8x4(double& c0, double& c1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c0), "+d"(c1)
               : "d"(a), "d"(b));
}

// The float64 Gram of the staged block is accumulated from 16-row slabs converted to float64 in
// shared memory (slab[c * kSlabLd + row]); a warp owns two strips of 8x8 tiles, (ta, tb <= ta) and
// (tz = nb8-1-ta, tb <= tz), so that every warp carries nb8 + 1 tiles.
constexpr int kSlabRows = 16;
constexpr int kSlabLd = 20;                      // doubles; conflict-free fragment loads
constexpr int kMaxTiles8 = kPMax / 8;            // 20
static_assert(kXsBytes + 2 * kPMax * kSlabLd * 8 <= kPowRegion, "slabs must fit behind the staged block");

// Accumulator slots of one warp: strip ta (the shorter one) uses slots 0 .. ta for tb = slot,
// strip tz uses slots kMaxTiles8 - tb for tb = 0 .. tz; ta + tz = nb8 - 1 <= 19, so they never meet.
struct GramAcc {
  double a[kMaxTiles8 + 1][2];
};

// The tensor-core instructions sit behind warp-uniform jump tables (switch fall-through), not
// predicates: a predicated-off mma still occupies the FP64 pipe.
#define COVSPEC_GRAM_A(u) case u: dmma_8x8x4(acc.a[u][0], acc.a[u][1], xa, b[u]);
#define COVSPEC_GRAM_Z(t) case t: dmma_8x8x4(acc.a[kMaxTiles8 - t][0], acc.a[kMaxTiles8 - t][1], xz, b[t]);
__device__ __forceinline__ void gram_unit_accumulate(GramAcc& acc, const double* slab, int ta, int tz,
                                                     int lane) {
  const int fr = lane >> 2, fk = lane & 3;
  const double* base = slab + fr * kSlabLd + fk;
#pragma unroll 1
  for (int ks = 0; ks < kSlabRows / 4; ++ks) {
    double b[kMaxTiles8];
#pragma unroll
    for (int t = 0; t < kMaxTiles8; ++t)
      if (t <= tz) b[t] = base[t * 8 * kSlabLd + 4 * ks];
    const double xa = base[ta * 8 * kSlabLd + 4 * ks], xz = base[tz * 8 * kSlabLd + 4 * ks];
    switch (ta) {
      COVSPEC_GRAM_A(19) COVSPEC_GRAM_A(18) COVSPEC_GRAM_A(17) COVSPEC_GRAM_A(16) COVSPEC_GRAM_A(15)
      COVSPEC_GRAM_A(14) COVSPEC_GRAM_A(13) COVSPEC_GRAM_A(12) COVSPEC_GRAM_A(11) COVSPEC_GRAM_A(10)
      COVSPEC_GRAM_A(9) COVSPEC_GRAM_A(8) COVSPEC_GRAM_A(7) COVSPEC_GRAM_A(6) COVSPEC_GRAM_A(5)
      COVSPEC_GRAM_A(4) COVSPEC_GRAM_A(3) COVSPEC_GRAM_A(2) COVSPEC_GRAM_A(1) COVSPEC_GRAM_A(0)
      default: break;
    }
    if (tz != ta) {
      switch (tz) {
        COVSPEC_GRAM_Z(19) COVSPEC_GRAM_Z(18) COVSPEC_GRAM_Z(17) COVSPEC_GRAM_Z(16) COVSPEC_GRAM_Z(15)
        COVSPEC_GRAM_Z(14) COVSPEC_GRAM_Z(13) COVSPEC_GRAM_Z(12) COVSPEC_GRAM_Z(11) COVSPEC_GRAM_Z(10)
        COVSPEC_GRAM_Z(9) COVSPEC_GRAM_Z(8) COVSPEC_GRAM_Z(7) COVSPEC_GRAM_Z(6) COVSPEC_GRAM_Z(5)
        COVSPEC_GRAM_Z(4) COVSPEC_GRAM_Z(3) COVSPEC_GRAM_Z(2) COVSPEC_GRAM_Z(1) COVSPEC_GRAM_Z(0)
        default: break;
      }
    }
  }
}
#undef COVSPEC_GRAM_A
#undef COVSPEC_GRAM_Z

}  // namespace sub
}  // namespace covspec
