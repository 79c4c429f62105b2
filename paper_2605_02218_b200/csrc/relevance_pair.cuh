// Fused tensor-core kernel for the query-aware score (Eq. 10) with per-head linear embeddings, bf16:
// the two-SM form.  A cluster of two CTAs owns a pair of neighbouring 128-token tiles of one request
// and works through the head pairs with tcgen05.mma.cta_group::2 (M = 256 across the pair):
//   Kp = X_tile * Wk[heads]^T       every CTA loads its own 128 x 64 token chunk and only HALF of the
//                                   256 x 64 weight chunk (the tensor cores of both SMs read both
//                                   halves): 32 KB of operands per CTA and k-chunk instead of 48 KB,
//                                   which is what bounds the one-CTA form
//   per token and head: ||Kp||^2    epilogue warps of each CTA read their own TMEM lanes, keep the norm
//                                   in float32 and restage Kp, 64 features at a time, as bf16 hi + lo
//                                   K-major tiles in their own shared memory
//   logits = Kp * Qn[head]^T        second pair-wide product against the unit-length query elements
//                                   (both tiles belong to one request, so they share Qn; every CTA loads
//                                   32 of the 64 query rows of a sub-tile), hi*hi + lo*hi + hi*lo
//   S^query = max_j,h logits / ||Kp||
// Loads are plain per-CTA TMA tile loads (no multicast); their completion is counted on the leader
// CTA's barrier.  The MMA issuer of the leader (cluster rank 0) drives both SMs; tcgen05.commit
// signals the barriers of both CTAs.  Barriers the issuer waits on (accumulator drained, projection
// restaged, logits read) live in the leader and are arrived on by the epilogue threads of both CTAs.
// MODE 1 reuses the main loop for the query side: Qp = Q * Wq^T, normalised per head, written as bf16.
//
// Warp roles per CTA (320 threads): warps 0-7 epilogue (two threads per token: warp w and w + 4 read
// the same 32 TMEM lanes and split the columns), warp 8 TMA producer, warp 9 TMEM owner and, in the
// leader, MMA issuer.  The restaged projection is double-buffered, so the epilogue restages the next
// half head while the logits product of the previous one is still running.  Every wait is bounded;
// on expiry the CTA raises a status bit and stops working; both CTAs meet at a cluster barrier
// before exit.
#pragma once
#include "relevance_tc.cuh"

namespace covspec {
namespace tc2 {

using namespace tc;

constexpr int kStages2 = 5;
constexpr int kBytesBh = (kTileN / 2) * kBK * 2;          // 16 KB: this CTA's half of the weight chunk
constexpr int kBytesStage2 = kBytesA + kBytesBh;          // 32 KB
constexpr int kBytesQh = (kTT / 2) * kHalf * 2;           // 4 KB: this CTA's 32 query rows; hi and lo
// No slack for aligning the base (declared 1024-byte aligned, checked in the kernel); the size leaves
// 1 KB of the SM's shared memory for one small block of another kernel (the activity stream).
constexpr int kKpBuffers = 2;                             // restaged half heads in flight
constexpr int kSmemBytes2 = kStages2 * kBytesStage2 + kKpBuffers * 2 * kBytesKp + 2048 /*barriers, norm exchange*/;
constexpr int kPairThreads = 320;
constexpr int kEpiArrivals = 512;                         // epilogue threads of both CTAs

struct PairParams {
  const ReqPlan* plan;
  int batch;
  int n_items;          // (tile pair, head-pair group) pairs
  int n_groups;         // head-pair groups per tile pair
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

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory object in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_at(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load into this CTA's shared memory whose bytes are counted on a barrier of the pair's
// leader CTA (bar_cluster_addr: see map_to_cta).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t smem_dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"((unsigned short)3)
      : "memory");
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
relevance_pair_kernel(const __grid_constant__ CUtensorMap map_a,   // X (MODE 0) or Q (MODE 1): [rows, d], box 128 rows
                      const __grid_constant__ CUtensorMap map_b,   // Wk or Wq: [P, d], box 128 rows
                      const __grid_constant__ CUtensorMap map_q,   // Qn hi: [sum T, P], box 32 rows (MODE 0 only)
                      const __grid_constant__ CUtensorMap map_ql,  // Qn lo
                      const PairParams prm) {
  extern __shared__ __align__(1024) uint8_t pair_smem_raw[];
  uint8_t* smem = pair_smem_raw;
  uint8_t* stage_base = smem;
  uint8_t* kp_smem = smem + kStages2 * kBytesStage2;       // per buffer: hi tile, then lo tile
  uint64_t* bars = reinterpret_cast<uint64_t*>(kp_smem + kKpBuffers * 2 * kBytesKp);
  uint64_t* full = bars;                   // [kStages2]  leader: bytes of both CTAs' loads
  uint64_t* empty = bars + kStages2;       // [kStages2]  both: the MMAs that read the slot are done
  uint64_t* acc_full = bars + 2 * kStages2;       // both: the projection of a head pair is complete
  uint64_t* acc_empty = acc_full + 1;             // leader: both epilogues have drained it (512 arrivals)
  uint64_t* kp_ready = acc_full + 2;              // [kKpBuffers] leader: both CTAs have restaged half a head (512)
  uint64_t* kp_free = acc_full + 4;               // [kKpBuffers] both: the logits MMAs that read the buffer are done
  uint64_t* logit_full = acc_full + 6;            // [kLogitSlots] both
  uint64_t* logit_empty = acc_full + 10;          // [kLogitSlots] leader (512)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 14);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* ss_xchg = reinterpret_cast<float*>(tmem_slot + 4);      // [2][128] partial squared norms

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const bool aligned = (smem_u32(smem) & 1023u) == 0;      // the swizzled tiles need a 1024-byte aligned base

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, kEpiArrivals);
    for (int i = 0; i < kKpBuffers; ++i) { mbar_init(&kp_ready[i], kEpiArrivals); mbar_init(&kp_free[i], 1); }
    for (int i = 0; i < kLogitSlots; ++i) {
      mbar_init(&logit_full[i], 1); mbar_init(&logit_empty[i], kEpiArrivals);
    }
    *abort_flag = aligned ? 0 : 1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                      // both CTAs' barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (MODE == 1 && prm.fill != nullptr) {
    // the visual-side launch combines head groups with an atomic max: its score array starts at -inf
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < prm.fill_n;
         i += (long long)gridDim.x * blockDim.x)
      prm.fill[i] = -INFINITY;
  }

  const int n_hp = (prm.n_heads + 1) >> 1;
  const int n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
  // barriers of the leader, as seen from this CTA
  const uint32_t l_acc_empty = map_to_cta(acc_empty, 0);
  const uint32_t l_kp_ready[kKpBuffers] = {map_to_cta(&kp_ready[0], 0), map_to_cta(&kp_ready[1], 0)};

  // Work-item decode shared by all roles: this CTA's tile of the pair.
  auto decode = [&](int item, int& row0, int& nrows, int& txt0, int& T, int& hp_begin, int& hp_end) {
    int pair = item / prm.n_groups, g = item % prm.n_groups;
    hp_begin = g * prm.hp_per_group;
    hp_end = min(n_hp, hp_begin + prm.hp_per_group);
    if (MODE == 0) {
      int b = find_request(pair, prm.batch, [&](int q) { return prm.plan[q].pair_off; });
      ReqPlan rp = prm.plan[b];
      int t = 2 * (pair - rp.pair_off) + (int)rank;
      row0 = rp.vis_off + t * kTileM;
      nrows = max(0, min(kTileM, rp.n - t * kTileM));
      txt0 = rp.txt_off;
      T = rp.t;
    } else {
      int t = 2 * pair + (int)rank;
      row0 = t * kTileM;
      long long rem = prm.rows_total - row0;
      nrows = rem < 0 ? 0 : (rem < kTileM ? (int)rem : kTileM);
      txt0 = 0; T = 0;
    }
  };

  if (warp == 8) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0 && aligned) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = cluster_id; item < prm.n_items && ok; item += n_clusters) {
        int row0, nrows, txt0, T, hp_begin, hp_end;
        decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
        for (int hp = hp_begin; hp < hp_end && ok; ++hp) {
          for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
            int s = it % kStages2;
            uint32_t ph = (it / kStages2) & 1u;
            if (!(ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag))) break;
            if (leader) mbar_expect_tx(&full[s], 2 * kBytesStage2);
            uint32_t dst = smem_u32(stage_base + s * kBytesStage2);
            uint32_t bar = map_to_cta(&full[s], 0);
            tma_load_2d_pair(dst, &map_a, kc * kBK, row0, bar);
            tma_load_2d_pair(dst + kBytesA, &map_b, kc * kBK, hp * kTileN + (int)rank * (kTileN / 2), bar);
          }
          if (MODE == 0 && ok) {
            // query sub-tiles of this head pair use the next ring slots, in the order the MMA issuer
            // consumes them: head, group of up to kLogitSlots tiles, half, tile; one slot holds this
            // CTA's 32 rows of the [64 x 64] hi block followed by those of the lo block
            int heads = min(2, prm.n_heads - 2 * hp);
            int ntt = (T + kTT - 1) / kTT;
            for (int h = 0; h < heads && ok; ++h)
              for (int g0 = 0; g0 < ntt && ok; g0 += kLogitSlots)
                for (int half = 0; half < 2 && ok; ++half)
                  for (int tt = g0; tt < min(ntt, g0 + kLogitSlots); ++tt, ++it) {
                    int s = it % kStages2;
                    uint32_t ph = (it / kStages2) & 1u;
                    if (!(ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag))) break;
                    if (leader) mbar_expect_tx(&full[s], 4 * kBytesQh);
                    uint32_t dst = smem_u32(stage_base + s * kBytesStage2);
                    uint32_t bar = map_to_cta(&full[s], 0);
                    int col = (2 * hp + h) * kHeadDim + half * kHalf, y = txt0 + tt * kTT + (int)rank * (kTT / 2);
                    tma_load_2d_pair(dst, &map_q, col, y, bar);
                    tma_load_2d_pair(dst + kBytesQh, &map_ql, col, y, bar);
                  }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ---------------------------------------------------------------- MMA issuer (leader only)
    if (lane == 0 && leader && aligned) {
      const uint32_t idesc1 = umma_idesc(2 * kTileM, kTileN);
      const uint32_t idesc2 = umma_idesc(2 * kTileM, kTT);
      uint32_t it = 0, acc_it = 0, kp_it = 0;
      uint32_t slot_uses[kLogitSlots] = {0u, 0u, 0u, 0u};
      bool ok = true;
      for (int item = cluster_id; item < prm.n_items && ok; item += n_clusters) {
        int row0, nrows, txt0, T, hp_begin, hp_end;
        decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
        for (int hp = hp_begin; hp < hp_end && ok; ++hp, ++acc_it) {
          if (!(ok = mbar_wait(acc_empty, (acc_it & 1u) ^ 1u, abort_flag))) break;
          tc_fence_after();
          for (int kc = 0; kc < prm.k_chunks; ++kc, ++it) {
            int s = it % kStages2;
            uint32_t ph = (it / kStages2) & 1u;
            if (!(ok = mbar_wait(&full[s], ph, abort_flag))) break;
            tc_fence_after();
            uint32_t a_addr = smem_u32(stage_base + s * kBytesStage2);
            uint64_t adesc = umma_desc(a_addr), bdesc = umma_desc(a_addr + kBytesA);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16_pair(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc1, (kc | k) != 0);
            umma_commit_pair(&empty[s]);
          }
          if (!ok) break;
          umma_commit_pair(acc_full);
          if (MODE == 0) {
            int heads = min(2, prm.n_heads - 2 * hp);
            int ntt = (T + kTT - 1) / kTT;
            for (int h = 0; h < heads && ok; ++h)
              for (int g0 = 0; g0 < ntt && ok; g0 += kLogitSlots) {
                const int ng = min(ntt, g0 + kLogitSlots) - g0;
                for (int half = 0; half < 2 && ok; ++half, ++kp_it) {
                  // both epilogues have restaged features [64 half, 64 half + 64) of this head
                  const int kb = kp_it & 1u;
                  if (!(ok = mbar_wait(&kp_ready[kb], (kp_it >> 1) & 1u, abort_flag))) break;
                  for (int slot = 0; slot < ng; ++slot, ++it) {
                    int s = it % kStages2;
                    if (!(ok = mbar_wait(&full[s], (it / kStages2) & 1u, abort_flag))) break;
                    if (half == 0 &&
                        !(ok = mbar_wait(&logit_empty[slot], (slot_uses[slot] & 1u) ^ 1u, abort_flag))) break;
                    tc_fence_after();
                    uint32_t kp_addr = smem_u32(kp_smem + kb * 2 * kBytesKp), q_addr = smem_u32(stage_base + s * kBytesStage2);
                    // logits += Kp_hi Qn_hi^T + Kp_lo Qn_hi^T + Kp_hi Qn_lo^T over this half's 64 features
#pragma unroll
                    for (int term = 0; term < 3; ++term) {
                      uint64_t adesc = umma_desc(kp_addr + (term == 1 ? kBytesKp : 0));
                      uint64_t bdesc = umma_desc(q_addr + (term == 2 ? kBytesQh : 0));
#pragma unroll
                      for (int ks = 0; ks < kHalf / 16; ++ks)
                        umma_bf16_pair(tmem_base + kLogitCol + slot * kTT, adesc + 2 * ks, bdesc + 2 * ks, idesc2,
                                       (half | term | ks) != 0);
                    }
                    umma_commit_pair(&empty[s]);
                    if (half == 1) { umma_commit_pair(&logit_full[slot]); ++slot_uses[slot]; }
                  }
                  if (!ok) break;
                  umma_commit_pair(&kp_free[kb]);
                }
              }
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue (warps 0-7, both CTAs)
    const int r = (warp & 3) * 32 + lane;                  // token row inside the tile = TMEM lane
    const int cpart = warp >> 2;                           // which 32 of every 64 columns this thread handles
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    uint32_t l_logit_empty[kLogitSlots];
#pragma unroll
    for (int i = 0; i < kLogitSlots; ++i) l_logit_empty[i] = map_to_cta(&logit_empty[i], 0);
    uint32_t acc_it = 0, kp_it = 0;
    uint32_t slot_uses[kLogitSlots] = {0u, 0u, 0u, 0u};
    bool ok = aligned;
    for (int item = cluster_id; item < prm.n_items; item += n_clusters) {
      int row0, nrows, txt0, T, hp_begin, hp_end;
      decode(item, row0, nrows, txt0, T, hp_begin, hp_end);
      float best = -INFINITY;
      bool nonfinite = false;
      for (int hp = hp_begin; hp < hp_end; ++hp, ++acc_it) {
        ok = ok && mbar_wait(acc_full, acc_it & 1u, abort_flag);
        tc_fence_after();
        int heads = min(2, prm.n_heads - 2 * hp);
        for (int h = 0; h < heads; ++h) {
          float ss = 0.f;
          if (MODE == 0) {
            const int ntt = (T + kTT - 1) / kTT;
            float inv = 0.f;
            for (int g0 = 0; g0 < ntt; g0 += kLogitSlots) {
              const int ng = min(ntt, g0 + kLogitSlots) - g0;
              for (int half = 0; half < 2; ++half, ++kp_it) {
                // restage this thread's 32 of the features [64 half, 64 half + 64) of the head as
                // bf16 hi + lo into the buffer whose previous logits product has finished
                const int kb = kp_it & 1u;
                ok = ok && mbar_wait(&kp_free[kb], ((kp_it >> 1) & 1u) ^ 1u, abort_flag);
                {
                  float v[32];
                  tmem_ld32(t_lane + h * kHeadDim + half * kHalf + cpart * 32, v);
                  uint32_t pk[16], pl[16];
#pragma unroll
                  for (int e = 0; e < 16; ++e) {
                    float a = v[2 * e], b = v[2 * e + 1];
                    if (g0 == 0) ss += a * a + b * b;
                    __nv_bfloat162 hi = __floats2bfloat162_rn(a, b);
                    pk[e] = *reinterpret_cast<uint32_t*>(&hi);
                    pl[e] = pack_bf16(a - __low2float(hi), b - __high2float(hi));
                  }
                  uint8_t* rowp = kp_smem + kb * 2 * kBytesKp + r * 128;
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    int chunk = (cpart * 4 + q) ^ (r & 7);
                    *reinterpret_cast<uint4*>(rowp + chunk * 16) =
                        make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                    *reinterpret_cast<uint4*>(rowp + kBytesKp + chunk * 16) =
                        make_uint4(pl[4 * q], pl[4 * q + 1], pl[4 * q + 2], pl[4 * q + 3]);
                  }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                tc_fence_before();
                mbar_arrive_at(l_kp_ready[kb]);
                // the accumulator is fully drained after the last restaging of the last head
                if (h == heads - 1 && half == 1 && g0 + kLogitSlots >= ntt) mbar_arrive_at(l_acc_empty);
              }
              if (g0 == 0) {
                // the two threads of a token add up their halves of the squared norm
                ss_xchg[cpart * 128 + r] = ss;
                named_barrier(1, 256);
                ss += ss_xchg[(cpart ^ 1) * 128 + r];
                named_barrier(1, 256);
                nonfinite |= !(ss <= 3.402823466e38f);
                if (ss > 1.17549435e-38f) { inv = rsqrtf(ss); inv = inv * (1.5f - 0.5f * ss * inv * inv); }
              }
              for (int slot = 0; slot < ng; ++slot) {
                ok = ok && mbar_wait(&logit_full[slot], slot_uses[slot] & 1u, abort_flag);
                ++slot_uses[slot];
                tc_fence_after();
                {
                  float v[32];
                  tmem_ld32(t_lane + kLogitCol + slot * kTT + cpart * 32, v);
                  int jbase = (g0 + slot) * kTT + cpart * 32;
#pragma unroll
                  for (int e = 0; e < 32; ++e)
                    if (jbase + e < T) {
                      nonfinite |= v[e] != v[e];
                      best = fmaxf(best, v[e] * inv);
                    }
                }
                tc_fence_before();
                mbar_arrive_at(l_logit_empty[slot]);
              }
            }
          } else {
            // MODE 1: unit-length bf16 head slice of the projected query element to global memory;
            // this thread's 64 of the head's 128 features.
#pragma unroll 1
            for (int c4 = 0; c4 < 2; ++c4) {
              float v[32];
              tmem_ld32(t_lane + h * kHeadDim + (cpart * 2 + c4) * 32, v);
#pragma unroll
              for (int e = 0; e < 32; ++e) ss += v[e] * v[e];
            }
            ss_xchg[cpart * 128 + r] = ss;
            named_barrier(1, 256);
            ss += ss_xchg[(cpart ^ 1) * 128 + r];
            named_barrier(1, 256);
            float inv = 0.f;
            if (ss > 1.17549435e-38f) { inv = rsqrtf(ss); inv = inv * (1.5f - 0.5f * ss * inv * inv); }
            if (!(ss <= 3.402823466e38f)) inv = __int_as_float(0x7fc00000);
#pragma unroll 1
            for (int c4 = 0; c4 < 2; ++c4) {
              float v[32];
              tmem_ld32(t_lane + h * kHeadDim + (cpart * 2 + c4) * 32, v);
              if (r < nrows && ok) {
                __nv_bfloat16* dst = prm.qn_out + (size_t)(row0 + r) * prm.P +
                                     (size_t)(2 * hp + h) * kHeadDim + (cpart * 2 + c4) * 32;
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
            if (h == heads - 1) { tc_fence_before(); mbar_arrive_at(l_acc_empty); }
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
  cluster_sync_all();                      // nothing of the peer may still point at this CTA
  if (warp == 9) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, kStatusTimeout);
}

}  // namespace tc2
}  // namespace covspec
