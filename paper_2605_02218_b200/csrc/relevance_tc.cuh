// Fused tensor-core kernel for the query-aware score (Eq. 10) with per-head linear embeddings, bf16.
//
// Per work item (one 128-token tile of one request, a group of head pairs) the kernel computes
//   Kp = X_tile * Wk[heads]^T           tcgen05.mma kind::f16, 128 x 256 accumulator in TMEM,
//                                       operands streamed by TMA through a shared-memory ring
//   per token and head: ||Kp||^2        epilogue warps read TMEM, keep the norm in float32 and
//                                       restage Kp, 64 features at a time, as bf16 hi + lo K-major
//                                       tiles in shared memory
//   logits = Kp * Qn[head]^T            second tcgen05.mma against the unit-length query elements,
//                                       as hi*hi + lo*hi + hi*lo so that bf16 staging costs ~2^-16,
//                                       accumulated over the two halves of the head in TMEM
//   S^query = max_j,h logits / ||Kp||   row max in registers, atomic max into the score array
// so the projected embeddings never leave the SM.  MODE 1 reuses the main loop for the query side:
// Qp = Q * Wq^T, normalised per head and written as bf16 for MODE 0 to consume.
//
// Warp roles (192 threads): warps 0-3 epilogue (one TMEM lane = one token each), warp 4 TMA
// producer, warp 5 MMA issuer and TMEM owner.  Every mbarrier wait is bounded; on expiry the CTA
// raises a status bit, leaves its loops, frees TMEM and exits.
#pragma once
#include "tc_common.cuh"

namespace covspec {

namespace tc {

constexpr int kTileM = 128;            // tokens per tile (UMMA M)
constexpr int kTileN = 256;            // projected features per pass: one pair of heads (UMMA N)
constexpr int kHeadDim = 128;
constexpr int kBK = 64;                // bf16 elements per k-chunk = one 128-byte swizzle row
// The ring is bound by how far ahead of their use the loads are issued (2 -> 3 stages: -25 %), so
// the projection is restaged half a head (64 features) at a time: its staging area shrinks from
// 64 KB to 32 KB and a fourth stage fits.
constexpr int kStages = 4;
constexpr int kTT = 64;                // query elements per logits tile (UMMA N of the 2nd product)
constexpr int kHalf = 64;              // features restaged at a time (one 128-byte swizzle row)
constexpr int kLogitSlots = 4;         // logits tiles that accumulate across the two halves
constexpr int kBytesA = kTileM * kBK * 2;          // 16 KB
constexpr int kBytesB = kTileN * kBK * 2;          // 32 KB
constexpr int kBytesStage = kBytesA + kBytesB;
constexpr int kBytesKp = kTileM * kHalf * 2;       // 16 KB: [128 x 64] of one half head; hi and lo
constexpr int kBytesQ = kTT * kHalf * 2;           // 8 KB: [64 x 64] of one half head; hi and lo
// The query sub-tiles (hi + lo = 16 KB) travel through the same ring slots as the main-loop chunks.
// No slack for aligning the base: the dynamic region is declared 1024-byte aligned (the kernel has
// no static shared memory in front of it) and the kernel checks it.  Every resident block reserves
// 1 KB of the SM's 228 KB, so this size leaves room for two small blocks of another kernel beside
// the CTA (the activity stream of the fused call).
constexpr int kSmemBytes = kStages * kBytesStage + 2 * kBytesKp + 1024 /*barriers*/;
constexpr int kTmemCols = 512;
constexpr int kLogitCol = 256;         // logits tiles live at columns 256 + 64 * slot

struct Params {
  const ReqPlan* plan;
  int batch;
  int n_items;          // (tile, group) pairs
  int n_groups;         // head-pair groups per tile
  int hp_per_group;     // head pairs handled by one item
  int n_heads;
  int k_chunks;         // ceil(d / 64)
  int P;                // n_heads * 128
  long long rows_total; // MODE 1: number of query rows
  float* s_query;       // MODE 0 out (pre-filled with -inf)
  __nv_bfloat16* qn_out;// MODE 1 out: hi [rows_total, P] followed by lo at qn_out + qn_lo_off
  long long qn_lo_off;
  float* fill;          // MODE 1: score array to fill with -inf for the MODE 0 launch that follows
  long long fill_n;     //         (nullptr: nothing to fill)
  int* status;
};

template <int MODE>
__global__ void __launch_bounds__(192, 1)
relevance_tc_kernel(const __grid_constant__ CUtensorMap map_a,   // X (MODE 0) or Q (MODE 1): [rows, d]
                    const __grid_constant__ CUtensorMap map_b,   // Wk or Wq: [P, d]
                    const __grid_constant__ CUtensorMap map_q,   // Qn hi: [sum T, P] (MODE 0 only)
                    const __grid_constant__ CUtensorMap map_ql,  // Qn lo
                    const Params prm) {
  extern __shared__ __align__(1024) uint8_t rel_smem_raw[];
  uint8_t* smem = rel_smem_raw;
  if (smem_u32(smem) & 1023u) {          // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicOr(prm.status, kStatusTimeout);
    return;
  }
  uint8_t* stage_base = smem;
  uint8_t* kp_smem = smem + kStages * kBytesStage;       // hi tile, then lo tile
  uint64_t* bars = reinterpret_cast<uint64_t*>(kp_smem + 2 * kBytesKp);
  uint64_t* full = bars;                 // [kStages]
  uint64_t* empty = bars + kStages;      // [kStages]
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 1;
  uint64_t* kp_ready = acc_full + 2;
  uint64_t* kp_free = acc_full + 3;
  uint64_t* logit_full = acc_full + 4;   // [kLogitSlots]
  uint64_t* logit_empty = acc_full + 8;  // [kLogitSlots]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 12);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 128);
    mbar_init(kp_ready, 128);
    mbar_init(kp_free, 1);
    for (int i = 0; i < kLogitSlots; ++i) {
      mbar_init(&logit_full[i], 1); mbar_init(&logit_empty[i], 128);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (MODE == 1 && prm.fill != nullptr) {
    // the visual-side launch combines head groups with an atomic max: its score array starts at -inf
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < prm.fill_n;
         i += (long long)gridDim.x * blockDim.x)
      prm.fill[i] = -INFINITY;
  }

  const int n_hp = (prm.n_heads + 1) >> 1;

  // Work-item decode shared by all roles.
  auto decode = [&](int item, int& row0, int& nrows, int& txt0, int& T, int& hp_begin, int& hp_end) {
    int tile = item / prm.n_groups, g = item % prm.n_groups;
    hp_begin = g * prm.hp_per_group;
    hp_end = min(n_hp, hp_begin + prm.hp_per_group);
    if (MODE == 0) {
      int b = find_request(tile, prm.batch, [&](int q) { return prm.plan[q].tile_off; });
      ReqPlan rp = prm.plan[b];
      int t = tile - rp.tile_off;
      row0 = rp.vis_off + t * kTileM;
      nrows = min(kTileM, rp.n - t * kTileM);
      txt0 = rp.txt_off;
      T = rp.t;
    } else {
      row0 = tile * kTileM;
      long long rem = prm.rows_total - row0;
      nrows = rem < kTileM ? (int)rem : kTileM;
      txt0 = 0; T = 0;
    }
  };

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x) {
        int row0, nrows, txt0, T, hp_begin, hp_end;
        decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
        for (int hp = hp_begin; hp < hp_end && ok; ++hp) {
          for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
            int s = it % kStages;
            uint32_t ph = (it / kStages) & 1u;
            if (!(ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag))) break;
            mbar_expect_tx(&full[s], kBytesStage);
            uint32_t dst = smem_u32(stage_base + s * kBytesStage);
            tma_load_2d(dst, &map_a, kc * kBK, row0, &full[s]);
            tma_load_2d(dst + kBytesA, &map_b, kc * kBK, hp * kTileN, &full[s]);
          }
          if (MODE == 0 && ok) {
            // query sub-tiles of this head pair use the next ring slots, in the order the MMA issuer
            // consumes them: head, group of up to kLogitSlots tiles, half, tile; one slot holds the
            // [64 x 64] hi block followed by the lo block
            int heads = min(2, prm.n_heads - 2 * hp);
            int ntt = (T + kTT - 1) / kTT;
            for (int h = 0; h < heads && ok; ++h)
              for (int g0 = 0; g0 < ntt && ok; g0 += kLogitSlots)
                for (int half = 0; half < 2 && ok; ++half)
                  for (int tt = g0; tt < min(ntt, g0 + kLogitSlots); ++tt, ++it) {
                    int s = it % kStages;
                    uint32_t ph = (it / kStages) & 1u;
                    if (!(ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag))) break;
                    mbar_expect_tx(&full[s], 2 * kBytesQ);
                    uint32_t dst = smem_u32(stage_base + s * kBytesStage);
                    int col = (2 * hp + h) * kHeadDim + half * kHalf, y = txt0 + tt * kTT;
                    tma_load_2d(dst, &map_q, col, y, &full[s]);
                    tma_load_2d(dst + kBytesQ, &map_ql, col, y, &full[s]);
                  }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = umma_idesc(kTileM, kTileN);
      const uint32_t idesc2 = umma_idesc(kTileM, kTT);
      uint32_t it = 0, acc_it = 0, kp_it = 0;
      uint32_t slot_uses[kLogitSlots] = {0u, 0u, 0u, 0u};
      bool ok = true;
      for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x) {
        int row0, nrows, txt0, T, hp_begin, hp_end;
        decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
        for (int hp = hp_begin; hp < hp_end && ok; ++hp, ++acc_it) {
          if (!(ok = mbar_wait(acc_empty, (acc_it & 1u) ^ 1u, abort_flag))) break;
          tc_fence_after();
          for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
            int s = it % kStages;
            uint32_t ph = (it / kStages) & 1u;
            if (!(ok = mbar_wait(&full[s], ph, abort_flag))) break;
            tc_fence_after();
            uint32_t a_addr = smem_u32(stage_base + s * kBytesStage);
            uint64_t adesc = umma_desc(a_addr), bdesc = umma_desc(a_addr + kBytesA);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc1, (kc | k) != 0);
            umma_commit(&empty[s]);
          }
          if (!ok) break;
          umma_commit(acc_full);
          if (MODE == 0) {
            int heads = min(2, prm.n_heads - 2 * hp);
            int ntt = (T + kTT - 1) / kTT;
            for (int h = 0; h < heads && ok; ++h)
              for (int g0 = 0; g0 < ntt && ok; g0 += kLogitSlots) {
                const int ng = min(ntt, g0 + kLogitSlots) - g0;
                for (int half = 0; half < 2 && ok; ++half, ++kp_it) {
                  // the epilogue has restaged features [64 half, 64 half + 64) of this head
                  if (!(ok = mbar_wait(kp_ready, kp_it & 1u, abort_flag))) break;
                  for (int slot = 0; slot < ng; ++slot, ++it) {
                    int s = it % kStages;
                    if (!(ok = mbar_wait(&full[s], (it / kStages) & 1u, abort_flag))) break;
                    if (half == 0 &&
                        !(ok = mbar_wait(&logit_empty[slot], (slot_uses[slot] & 1u) ^ 1u, abort_flag))) break;
                    tc_fence_after();
                    uint32_t kp_addr = smem_u32(kp_smem), q_addr = smem_u32(stage_base + s * kBytesStage);
                    // logits += Kp_hi Qn_hi^T + Kp_lo Qn_hi^T + Kp_hi Qn_lo^T over this half's 64 features
#pragma unroll
                    for (int term = 0; term < 3; ++term) {
                      uint64_t adesc = umma_desc(kp_addr + (term == 1 ? kBytesKp : 0));
                      uint64_t bdesc = umma_desc(q_addr + (term == 2 ? kBytesQ : 0));
#pragma unroll
                      for (int ks = 0; ks < kHalf / 16; ++ks)
                        umma_bf16(tmem_base + kLogitCol + slot * kTT, adesc + 2 * ks, bdesc + 2 * ks, idesc2,
                                  (half | term | ks) != 0);
                    }
                    umma_commit(&empty[s]);
                    if (half == 1) { umma_commit(&logit_full[slot]); ++slot_uses[slot]; }
                  }
                  if (!ok) break;
                  umma_commit(kp_free);
                }
              }
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue (warps 0-3)
    const int r = warp * 32 + lane;                        // token row inside the tile = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    uint32_t acc_it = 0, kp_it = 0;
    uint32_t slot_uses[kLogitSlots] = {0u, 0u, 0u, 0u};
    bool ok = true;
    for (int item = blockIdx.x; item < prm.n_items && ok; item += gridDim.x) {
      int row0, nrows, txt0, T, hp_begin, hp_end;
      decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
      float best = -INFINITY;
      bool nonfinite = false;
      for (int hp = hp_begin; hp < hp_end && ok; ++hp, ++acc_it) {
        if (!(ok = mbar_wait(acc_full, acc_it & 1u, abort_flag))) break;
        tc_fence_after();
        int heads = min(2, prm.n_heads - 2 * hp);
        for (int h = 0; h < heads && ok; ++h) {
          float ss = 0.f;
          if (MODE == 0) {
            const int ntt = (T + kTT - 1) / kTT;
            float inv = 0.f;
            for (int g0 = 0; g0 < ntt && ok; g0 += kLogitSlots) {
              const int ng = min(ntt, g0 + kLogitSlots) - g0;
              for (int half = 0; half < 2 && ok; ++half, ++kp_it) {
                // restage features [64 half, 64 half + 64) of this head as bf16 hi + lo
                if (!(ok = mbar_wait(kp_free, (kp_it & 1u) ^ 1u, abort_flag))) break;
#pragma unroll 1
                for (int c2 = 0; c2 < 2; ++c2) {
                  float v[32];
                  tmem_ld32(t_lane + h * kHeadDim + half * kHalf + c2 * 32, v);
                  uint32_t pk[16], pl[16];
#pragma unroll
                  for (int e = 0; e < 16; ++e) {
                    float a = v[2 * e], b = v[2 * e + 1];
                    if (g0 == 0) ss += a * a + b * b;
                    __nv_bfloat162 hi = __floats2bfloat162_rn(a, b);
                    pk[e] = *reinterpret_cast<uint32_t*>(&hi);
                    pl[e] = pack_bf16(a - __low2float(hi), b - __high2float(hi));
                  }
                  uint8_t* rowp = kp_smem + r * 128;
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    int chunk = (c2 * 4 + q) ^ (r & 7);
                    *reinterpret_cast<uint4*>(rowp + chunk * 16) =
                        make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                    *reinterpret_cast<uint4*>(rowp + kBytesKp + chunk * 16) =
                        make_uint4(pl[4 * q], pl[4 * q + 1], pl[4 * q + 2], pl[4 * q + 3]);
                  }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                tc_fence_before();
                mbar_arrive(kp_ready);
                // the accumulator is fully drained after the last restaging of the last head
                if (h == heads - 1 && half == 1 && g0 + kLogitSlots >= ntt) mbar_arrive(acc_empty);
              }
              if (!ok) break;
              if (g0 == 0) {
                nonfinite |= !(ss <= 3.402823466e38f);
                if (ss > 1.17549435e-38f) { inv = rsqrtf(ss); inv = inv * (1.5f - 0.5f * ss * inv * inv); }
              }
              for (int slot = 0; slot < ng; ++slot) {
                if (!(ok = mbar_wait(&logit_full[slot], slot_uses[slot] & 1u, abort_flag))) break;
                ++slot_uses[slot];
                tc_fence_after();
#pragma unroll 1
                for (int c2 = 0; c2 < 2; ++c2) {
                  float v[32];
                  tmem_ld32(t_lane + kLogitCol + slot * kTT + c2 * 32, v);
                  int jbase = (g0 + slot) * kTT + c2 * 32;
#pragma unroll
                  for (int e = 0; e < 32; ++e)
                    if (jbase + e < T) {
                      nonfinite |= v[e] != v[e];
                      best = fmaxf(best, v[e] * inv);
                    }
                }
                tc_fence_before();
                mbar_arrive(&logit_empty[slot]);
              }
            }
          } else {
            // MODE 1: unit-length bf16 head slice of the projected query element to global memory.
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
              float v[32];
              tmem_ld32(t_lane + h * kHeadDim + c4 * 32, v);
#pragma unroll
              for (int e = 0; e < 32; ++e) ss += v[e] * v[e];
            }
            float inv = 0.f;
            if (ss > 1.17549435e-38f) { inv = rsqrtf(ss); inv = inv * (1.5f - 0.5f * ss * inv * inv); }
            if (!(ss <= 3.402823466e38f)) inv = __int_as_float(0x7fc00000);
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
              float v[32];
              tmem_ld32(t_lane + h * kHeadDim + c4 * 32, v);
              if (r < nrows) {
                __nv_bfloat16* dst = prm.qn_out + (size_t)(row0 + r) * prm.P +
                                     (size_t)(2 * hp + h) * kHeadDim + c4 * 32;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  uint32_t ph[4], pw[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    float a = v[8 * q + 2 * e] * inv, b = v[8 * q + 2 * e + 1] * inv;
                    __nv_bfloat162 hi = __floats2bfloat162_rn(a, b);
                    ph[e] = *reinterpret_cast<uint32_t*>(&hi);
                    pw[e] = pack_bf16(a - __low2float(hi), b - __high2float(hi));
                  }
                  *reinterpret_cast<uint4*>(dst + q * 8) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
                  *reinterpret_cast<uint4*>(dst + prm.qn_lo_off + q * 8) =
                      make_uint4(pw[0], pw[1], pw[2], pw[3]);
                }
              }
            }
            if (h == heads - 1) { tc_fence_before(); mbar_arrive(acc_empty); }
          }
        }
      }
      if (MODE == 0 && ok && r < nrows) {
        if (nonfinite) atomicOr(prm.status, kStatusNonFinite);
        else atomic_max_float(prm.s_query + row0 + r, best);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(kTmemCols)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, kStatusTimeout);
}

}  // namespace tc
}  // namespace covspec
