// Host runtime and C ABI of the covspec library: argument validation, budgets, the cached launch
// plan, workspace carving and the kernel sequence of every entry point (see include/covspec.h).
#include "covspec.h"

#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"
#include "correct_kernels.cuh"
#include "eig_kernels.cuh"
#include "gemm_simt.cuh"
#include "greedy_kernels.cuh"
#include "relevance_tc.cuh"
#include "relevance_pair.cuh"
#include "subspace_tc.cuh"
#include "subspace_fused.cuh"
#include "score_kernels.cuh"
#include "select_kernels.cuh"

using namespace covspec;

namespace {

thread_local std::string g_cuda_error;

#define CUDA_TRY(expr)                                                                  \
  do {                                                                                  \
    cudaError_t e_ = (expr);                                                            \
    if (e_ != cudaSuccess) {                                                            \
      g_cuda_error = std::string(#expr) + ": " + cudaGetErrorString(e_);                \
      return COVSPEC_ERR_CUDA;                                                          \
    }                                                                                   \
  } while (0)

inline long long round_up(long long v, long long a) { return (v + a - 1) / a * a; }

// Gemm tables kept on the device (one entry per stage-2 request); only the float32 configuration
// still forms its Gram matrix on the CUDA cores.
enum TableId {
  T_GRAM_G = 0,   // G = Zg Zg^T (float32 operands)
  T_COUNT
};

// Stages reported by the optional event timing.
enum StageId { ST_QEMBED = 0, ST_RELEVANCE, ST_ACTIVITY, ST_FUSE, ST_PRESELECT, ST_GRAM, ST_EIG,
               ST_FINAL, ST_COUNT };
const char* const kStageNames[ST_COUNT] = {"query_embed", "relevance", "activity", "fuse",
                                            "preselect", "gram", "subspace", "final_select_compact"};

struct Plan {
  std::vector<int> vis_off, txt_off, keep;    // key of the cache
  double keep_ratio = 0.0;
  bool has_keep = false;
  std::vector<ReqPlan> req;
  std::vector<int> keep_offsets, presel_offsets;
  int n_stage2 = 0;
  int tiles[T_COUNT] = {0};
  int t_max = 0, p_max = 0, m_max = 0, win_max = 0, nbot_max = 0;
  int n_tiles = 0;                            // 128-token tiles over all requests
  int n_pairs = 0;                            // pairs of neighbouring tiles of one request
  int n_gram_tiles = 0, n_ptiles = 0;         // lower-triangle Gram items / row tiles of the subspace blocks (stage 2)
  int tile_rows = 128;                        // rows of a subspace-block tile: 64 when that still gives every tile a CTA
  int tile_ctas = 0, servers = 0;             // CTAs of the subspace kernel that carry tiles / that only factor
  int pow_grid = 0;                           // CTAs of the power step
  std::vector<int> sched;                     // [pow_grid + 1] offsets + item lists (longest first)
  long long total_vis = 0, total_txt = 0, total_keep = 0, total_presel = 0;
  bool valid = false;
};

}  // namespace

struct covspec_ctx {
  covspec_config cfg;
  int P = 0, hd = 0, heads = 0;          // embedding width, head width, head count (identity: 1 head)
  int esize = 0;
  char* ws = nullptr;                    // device workspace
  long long ws_bytes = 0;
  // carved regions
  int* status = nullptr;
  ReqPlan* d_plan = nullptr;
  int* d_sched = nullptr;                // power-step schedule: [grid + 1] offsets + item lists
  GemmProb* d_tables = nullptr;          // [T_COUNT][max_batch]
  float* Qn = nullptr;
  float* Kp = nullptr;
  long long kp_rows = 0;
  float *sq = nullptr, *sa = nullptr, *sf = nullptr;
  int* presel = nullptr;
  float* energy = nullptr;
  void* Zg = nullptr;
  float* G = nullptr;                    // float32 Gram matrices (float32 inputs only)
  long long g_cap = 0;
  // subspace iteration (see subspace_tc.cuh for the layouts)
  int ld = 0;                            // row stride of the G and Y planes
  long long cap_rows = 0, cap_ptiles = 0;
  __nv_bfloat16 *Ghi = nullptr, *Glo = nullptr;
  __nv_bfloat16* Yp[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // [buffer][hi / lo]
  float* Yf[2] = {nullptr, nullptr};     // float32 blocks before / after the last power step
  double* partial = nullptr;
  float *Lbuf = nullptr, *Ub = nullptr;
  unsigned* sync = nullptr;              // per-request counters of the fused subspace kernel + abort word
  float* Cg = nullptr;                   // factor columns of the greedy low-rank mode
  long long cg_cap = 0;
  CUtensorMap map_zg, map_zgw, map_gh, map_gl, map_y[2][2];
  // float32 inputs on the tensor cores: operands split into bf16 rows three times as wide
  // (split3_kernel); nullptr / 0 when the configuration does not take that route
  bool split_tc = false;
  int dp = 0, d3 = 0;                    // d rounded up to 64; 3 * dp
  __nv_bfloat16 *X3 = nullptr, *Q3 = nullptr, *Wq3 = nullptr, *Wk3 = nullptr, *Za3 = nullptr, *Zb3 = nullptr;
  CUtensorMap map_za3, map_zb3w;
  // pinned staging for the plan upload
  char* h_stage = nullptr;
  long long stage_bytes = 0, stage_sched_off = 0;
  cudaEvent_t stage_free = nullptr;      // the previous upload has been consumed
  // the fused call streams the snapshot stack (Eq. 11) beside the relevance kernel on this stream
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  Plan plan;
  int num_sms = 148;
  bool tc_ready = false;                 // tensor-core relevance kernel configured on this device
  int launches = 0;
  // optional per-stage timing (CUDA events on the call's stream)
  std::vector<cudaEvent_t> prof_events;  // [prof_cap][ST_COUNT][2]
  std::vector<unsigned char> prof_set;
  int prof_cap = 0, prof_calls = 0;
};

namespace {

int budgets_impl(const covspec_config* cfg, int n, int keep, int* b, int* m, int* r) {
  if (n < 1 || keep < 1) return COVSPEC_ERR_ARG;
  int B = keep < n ? keep : n;
  long long want = (long long)ceil((double)cfg->presel_factor * (double)B - 1e-9);
  if (want < B) want = B;
  int M = (int)(want < n ? want : n);
  int R = (int)ceil((double)cfg->rank_frac * (double)B - 1e-9);
  int cap = cfg->rank_cap;
  if (M - 1 < cap) cap = M - 1;
  if (cfg->d - 1 < cap) cap = cfg->d - 1;
  if (R > cap) R = cap;
  if (R < 1) R = 1;
  *b = B; *m = M; *r = R;
  return COVSPEC_OK;
}

int keep_of(const covspec_problem* p, int b, int n) {
  if (p->keep) return p->keep[b];
  int k = (int)ceil(p->keep_ratio * (double)n - 1e-6);
  return k < 1 ? 1 : k;
}

int validate_cfg(const covspec_config* c) {
  if (!c) return COVSPEC_ERR_ARG;
  if (c->dtype != COVSPEC_F32 && c->dtype != COVSPEC_BF16) return COVSPEC_ERR_ARG;
  if (c->d < 8 || c->d % 8) return COVSPEC_ERR_UNSUPPORTED;
  if (c->n_heads < 0) return COVSPEC_ERR_ARG;
  if (c->n_heads > 0 && c->head_dim != 128) return COVSPEC_ERR_UNSUPPORTED;
  if (c->act_layers < 0 || c->act_layers + 1 > kMaxLayers) return COVSPEC_ERR_UNSUPPORTED;
  if (!(c->lambda >= 0.f && c->lambda <= 1.f)) return COVSPEC_ERR_ARG;
  if (c->norm_mode < 0 || c->norm_mode > 2 || c->head_reduce < 0 || c->head_reduce > 1)
    return COVSPEC_ERR_ARG;
  if (!(c->presel_factor >= 1.f) || !(c->rank_frac > 0.f) || c->rank_cap < 1) return COVSPEC_ERR_ARG;
  if (c->eig_iters < 1 || c->eig_oversample < 0) return COVSPEC_ERR_ARG;
  if (c->rank_cap + c->eig_oversample > kPMax) return COVSPEC_ERR_UNSUPPORTED;
  if (c->lowrank_mode < 0 || c->lowrank_mode > 1) return COVSPEC_ERR_ARG;
  if (c->relevance_path < 0 || c->relevance_path > 2) return COVSPEC_ERR_ARG;
  if (c->ritz_window < 0) return COVSPEC_ERR_ARG;
  if (c->activity_overlap < 0 || c->activity_overlap > 2) return COVSPEC_ERR_ARG;
  if (c->eig_iters > 1000 || !(c->conv_tol >= 0.f)) return COVSPEC_ERR_ARG;
  return COVSPEC_OK;
}

int validate_problem(const covspec_config* c, const covspec_problem* p) {
  if (!p || p->batch < 1 || !p->vis_offsets || !p->txt_offsets) return COVSPEC_ERR_ARG;
  if (!p->keep && !(p->keep_ratio > 0.0 && p->keep_ratio <= 1.0)) return COVSPEC_ERR_ARG;
  if (p->vis_offsets[0] != 0 || p->txt_offsets[0] != 0) return COVSPEC_ERR_SHAPE;
  for (int b = 0; b < p->batch; ++b) {
    if (p->vis_offsets[b + 1] <= p->vis_offsets[b]) return COVSPEC_ERR_SHAPE;   // N_b >= 1
    if (p->txt_offsets[b + 1] <= p->txt_offsets[b]) return COVSPEC_ERR_SHAPE;   // T_b >= 1
    if (p->keep && p->keep[b] < 1) return COVSPEC_ERR_SHAPE;
  }
  (void)c;
  return COVSPEC_OK;
}

// Builds (or reuses) the launch plan and uploads it on `stream`.
int get_plan(covspec_ctx* ctx, const covspec_problem* p, cudaStream_t stream) {
  const covspec_config& cfg = ctx->cfg;
  int st = validate_problem(&cfg, p);
  if (st) return st;
  Plan& pl = ctx->plan;
  int B = p->batch;
  bool same = pl.valid && (int)pl.req.size() == B && pl.has_keep == (p->keep != nullptr) &&
              !memcmp(pl.vis_off.data(), p->vis_offsets, sizeof(int) * (B + 1)) &&
              !memcmp(pl.txt_off.data(), p->txt_offsets, sizeof(int) * (B + 1)) &&
              (p->keep ? !memcmp(pl.keep.data(), p->keep, sizeof(int) * B)
                       : pl.keep_ratio == p->keep_ratio);
  if (same) return COVSPEC_OK;
  if (B > cfg.max_batch) return COVSPEC_ERR_WORKSPACE;
  pl.valid = false;
  pl.vis_off.assign(p->vis_offsets, p->vis_offsets + B + 1);
  pl.txt_off.assign(p->txt_offsets, p->txt_offsets + B + 1);
  pl.has_keep = p->keep != nullptr;
  if (p->keep) pl.keep.assign(p->keep, p->keep + B);
  pl.keep_ratio = p->keep_ratio;
  pl.req.assign(B, ReqPlan{});
  pl.keep_offsets.assign(B + 1, 0);
  pl.presel_offsets.assign(B + 1, 0);
  pl.n_stage2 = 0; pl.t_max = 0; pl.p_max = 0; pl.m_max = 0; pl.n_tiles = 0; pl.n_pairs = 0;
  pl.n_gram_tiles = 0; pl.n_ptiles = 0;
  pl.win_max = 0; pl.nbot_max = 0;
  long long g_off = 0, c_off = 0;
  int n_max = 0;
  bool f32 = cfg.dtype == COVSPEC_F32;
  for (int b = 0; b < B; ++b) {
    ReqPlan& r = pl.req[b];
    r.vis_off = p->vis_offsets[b]; r.n = p->vis_offsets[b + 1] - r.vis_off;
    r.txt_off = p->txt_offsets[b]; r.t = p->txt_offsets[b + 1] - r.txt_off;
    st = budgets_impl(&cfg, r.n, keep_of(p, b, r.n), &r.b_vis, &r.m, &r.r);
    if (st) return COVSPEC_ERR_SHAPE;
    r.stage2 = r.b_vis < r.m;
    r.p = 0;
    r.ldm = (int)round_up(r.m, 4);
    r.tile_off = pl.n_tiles;
    pl.n_tiles += (r.n + tc::kTileM - 1) / tc::kTileM;
    r.pair_off = pl.n_pairs;
    pl.n_pairs += ((r.n + tc::kTileM - 1) / tc::kTileM + 1) / 2;
    r.gram_tile_off = pl.n_gram_tiles;
    r.g_off = g_off;
    r.c_off = c_off;
    if (r.stage2) {
      r.p = r.r + cfg.eig_oversample;
      if (r.p > r.m) r.p = r.m;
      ++pl.n_stage2;
      int nt = (r.m + sub::kTile - 1) / sub::kTile;
      pl.n_gram_tiles += sub::gram_items(nt);
      if (f32) g_off += (long long)r.m * r.ldm;
      if (cfg.lowrank_mode == 1) {
        if (r.m > kGreedyMaxM || r.b_vis > kGreedyMaxB) return COVSPEC_ERR_UNSUPPORTED;
        c_off += (long long)r.b_vis * r.m;
      }
      r.win = r.p - r.r + std::min(cfg.ritz_window, r.r);
      if (r.win > r.p) r.win = r.p;
      pl.win_max = std::max(pl.win_max, r.win);
      pl.nbot_max = std::max(pl.nbot_max, r.p - r.r);
    }
    r.keep_off = pl.keep_offsets[b]; r.presel_off = pl.presel_offsets[b];
    pl.keep_offsets[b + 1] = r.keep_off + r.b_vis;
    pl.presel_offsets[b + 1] = r.presel_off + r.m;
    if (r.t > pl.t_max) pl.t_max = r.t;
    if (r.p > pl.p_max) pl.p_max = r.p;
    if (r.m > pl.m_max) pl.m_max = r.m;
    if (r.n > n_max) n_max = r.n;
  }
  pl.total_vis = p->vis_offsets[B]; pl.total_txt = p->txt_offsets[B];
  pl.total_keep = pl.keep_offsets[B]; pl.total_presel = pl.presel_offsets[B];
  if (pl.total_vis > cfg.max_total_vis || pl.total_txt > cfg.max_total_txt ||
      n_max > cfg.max_vis_per_req || g_off > ctx->g_cap || c_off > ctx->cg_cap || pl.m_max > ctx->cfg.max_presel_per_req ||
      pl.total_presel > ctx->cfg.max_total_presel || pl.n_ptiles > ctx->cap_ptiles)
    return COVSPEC_ERR_WORKSPACE;

  // Row tiles of the subspace blocks: 128 rows, or 64 when every 64-row tile still gets a CTA of its
  // own (the per-tile epilogue is the critical path of a step: half the rows, half the time).
  {
    long long n64 = 0;
    for (int b = 0; b < B; ++b)
      if (pl.req[b].stage2) n64 += (pl.req[b].m + 63) / 64;
    pl.tile_rows = (n64 > 0 && n64 <= std::min<long long>(ctx->num_sms, ctx->cap_ptiles)) ? 64 : sub::kTile;
    pl.n_ptiles = 0;
    for (int b = 0; b < B; ++b) {
      pl.req[b].ptile_off = pl.n_ptiles;
      if (pl.req[b].stage2) pl.n_ptiles += (pl.req[b].m + pl.tile_rows - 1) / pl.tile_rows;
    }
    if (pl.n_ptiles > ctx->cap_ptiles) return COVSPEC_ERR_WORKSPACE;
  }

  // Schedule of the subspace kernel.  Its items (row tiles) differ in cost (basis size p, rows
  // in the tile), and every step of a request ends when its slowest tile does.  With more tiles
  // than CTAs, consecutive tiles of one request therefore form groups and a group goes to one CTA
  // as a whole: a CTA that carries several tiles then delays one request instead of several.
  // Groups are handed out longest first, each to the least loaded CTA (with more requests than CTAs
  // every request is one group and the hand-out stacks them).
  // When SMs are left over, one more CTA per stage-2 request does nothing but factor for it (see the
  // kernel): their item lists are empty.
  pl.tile_ctas = std::min(pl.n_ptiles, ctx->num_sms);
  pl.servers = (pl.n_ptiles > 0 && pl.n_ptiles + pl.n_stage2 <= ctx->num_sms) ? pl.n_stage2 : 0;
  pl.pow_grid = pl.tile_ctas + pl.servers;
  pl.sched.assign((size_t)pl.pow_grid + 1 + pl.n_ptiles, 0);
  if (pl.n_ptiles > 0) {
    auto tile_cost = [&](const ReqPlan& r, int t) {
      int rows = std::min(pl.tile_rows, r.m - t * pl.tile_rows);
      double pp = (double)r.p;
      return pp * pp * (1.75 + 0.75 * rows / sub::kTile) + 10.0 * r.m;
    };
    // Every stage-2 request gets CTAs of its own and runs its steps independently of the others, so the
    // call ends with the request whose steps take longest.  A request's tiles are split into g
    // consecutive groups whose sizes differ by at most one, the larger ones last (the last tile may
    // be ragged, hence cheaper); its step time is the cost of its most expensive group.  The number of
    // groups per request (sum = CTAs) minimises the largest step time: the smallest feasible bound
    // is found among the step times every request can have; CTAs that are left then go, one at a
    // time, to the request that is slowest at that moment.  Requests are never mixed inside a group.
    struct Group { double cost; int first, count, req; };
    struct Share { int req, nt, g; };
    std::vector<Group> groups;
    std::vector<Share> shares;
    for (int b = 0; b < B; ++b)
      if (pl.req[b].stage2) shares.push_back(Share{b, (pl.req[b].m + pl.tile_rows - 1) / pl.tile_rows, 1});
    // calls fn(first tile, tile count, cost) for every group of the split into g groups
    auto split = [&](const Share& sh, int g, auto&& fn) {
      const ReqPlan& r = pl.req[sh.req];
      const int small = sh.nt / g, n_large = sh.nt % g;
      for (int i = 0, t = 0; i < g; ++i) {
        const int count = small + (i >= g - n_large ? 1 : 0);
        double cost = 0.0;
        for (int q = 0; q < count; ++q) cost += tile_cost(r, t + q);
        fn(t, count, cost);
        t += count;
      }
    };
    auto step_time = [&](const Share& sh, int g) {
      double worst = 0.0;
      split(sh, g, [&](int, int, double cost) { worst = std::max(worst, cost); });
      return worst;
    };
    if ((int)shares.size() < pl.tile_ctas) {
      // times[i][g - 1]: step time of request i on g groups
      std::vector<std::vector<double>> times(shares.size());
      std::vector<double> cand;
      for (size_t i = 0; i < shares.size(); ++i)
        for (int g = 1; g <= shares[i].nt; ++g) {
          times[i].push_back(step_time(shares[i], g));
          cand.push_back(times[i].back());
        }
      std::sort(cand.begin(), cand.end());
      auto fewest_groups = [&](size_t i, double bound) {       // nt: one tile per group always fits
        for (int g = 1; g < shares[i].nt; ++g)
          if (times[i][g - 1] <= bound) return g;
        return shares[i].nt;
      };
      auto groups_needed = [&](double bound) {
        long long n = 0;
        for (size_t i = 0; i < shares.size(); ++i)
          n += times[i].back() <= bound ? fewest_groups(i, bound) : (long long)1 << 40;
        return n;
      };
      size_t lo = 0, hi = cand.size() - 1;           // the largest candidate needs one group per request
      while (lo < hi) {
        size_t mid = (lo + hi) / 2;
        if (groups_needed(cand[mid]) <= pl.tile_ctas) hi = mid; else lo = mid + 1;
      }
      int used = 0;
      for (size_t i = 0; i < shares.size(); ++i) used += shares[i].g = fewest_groups(i, cand[lo]);
      for (; used < pl.tile_ctas; ++used) {
        int worst = -1;
        for (size_t i = 0; i < shares.size(); ++i)
          if (shares[i].g < shares[i].nt &&
              (worst < 0 || times[i][shares[i].g - 1] > times[worst][shares[worst].g - 1])) worst = (int)i;
        if (worst < 0) break;
        ++shares[worst].g;
      }
    }
    for (const Share& sh : shares)
      split(sh, sh.g, [&](int t, int count, double cost) {
        groups.push_back(Group{cost, pl.req[sh.req].ptile_off + t, count, sh.req});
      });
    std::stable_sort(groups.begin(), groups.end(), [](const Group& a, const Group& b2) { return a.cost > b2.cost; });
    std::vector<double> load(pl.tile_ctas, 0.0);
    std::vector<std::vector<int>> lists(pl.tile_ctas);
    for (const Group& g : groups) {
      int best = 0;
      for (int c = 1; c < pl.tile_ctas; ++c) if (load[c] < load[best]) best = c;
      load[best] += g.cost;
      for (int t = 0; t < g.count; ++t) lists[best].push_back(g.first + t);
    }
    // more groups than CTAs is guaranteed to leave no CTA empty only if groups >= CTAs
    int off = 0;
    int* items_out = pl.sched.data() + pl.pow_grid + 1;
    for (int g = 0; g < pl.pow_grid; ++g) {
      pl.sched[g] = off;
      if (g < pl.tile_ctas)
        for (int v : lists[g]) items_out[off++] = v;
    }
    pl.sched[pl.pow_grid] = off;
  }

  // Stage plan + gemm table in pinned memory and upload.
  if (ctx->stage_free) CUDA_TRY(cudaEventSynchronize(ctx->stage_free));
  ReqPlan* h_plan = reinterpret_cast<ReqPlan*>(ctx->h_stage);
  GemmProb* h_tab = reinterpret_cast<GemmProb*>(ctx->h_stage + round_up(sizeof(ReqPlan) * cfg.max_batch, 256));
  memcpy(h_plan, pl.req.data(), sizeof(ReqPlan) * B);
  int mb = cfg.max_batch;
  for (int t = 0; t < T_COUNT; ++t) pl.tiles[t] = 0;
  int s2 = 0;
  if (f32) {
    char* Zg = reinterpret_cast<char*>(ctx->Zg);
    for (int b = 0; b < B; ++b) {
      const ReqPlan& r = pl.req[b];
      if (!r.stage2) continue;
      GemmProb& g = h_tab[(size_t)T_GRAM_G * mb + s2];
      const void* zg = Zg + (size_t)r.presel_off * cfg.d * ctx->esize;
      g.A = zg; g.B = zg; g.C = ctx->G + r.g_off;
      g.m = r.m; g.n = r.m; g.k = cfg.d; g.lda = cfg.d; g.ldb = cfg.d; g.ldc = r.ldm;
      g.tile_start = pl.tiles[T_GRAM_G];
      g.tiles_n = (r.m + kGemmBN - 1) / kGemmBN;
      pl.tiles[T_GRAM_G] += ((r.m + kGemmBM - 1) / kGemmBM) * g.tiles_n;
      ++s2;
    }
  }
  CUDA_TRY(cudaMemcpyAsync(ctx->d_plan, h_plan, sizeof(ReqPlan) * B, cudaMemcpyHostToDevice, stream));
  if (s2 > 0)
    CUDA_TRY(cudaMemcpyAsync(ctx->d_tables, h_tab, sizeof(GemmProb) * (size_t)T_COUNT * mb,
                             cudaMemcpyHostToDevice, stream));
  if (pl.n_ptiles > 0) {
    int* h_sched = reinterpret_cast<int*>(ctx->h_stage + ctx->stage_sched_off);
    memcpy(h_sched, pl.sched.data(), sizeof(int) * pl.sched.size());
    CUDA_TRY(cudaMemcpyAsync(ctx->d_sched, h_sched, sizeof(int) * pl.sched.size(), cudaMemcpyHostToDevice, stream));
  }
  CUDA_TRY(cudaEventRecord(ctx->stage_free, stream));
  pl.valid = true;
  return COVSPEC_OK;
}

#define LAUNCH_CHECK(ctx)                               \
  do {                                                  \
    ++(ctx)->launches;                                  \
    CUDA_TRY(cudaGetLastError());                       \
  } while (0)

// Records the begin (edge 0) or end (edge 1) event of a stage for the current profiled call.
inline void prof_mark(covspec_ctx* ctx, int stage, int edge, cudaStream_t s) {
  if (ctx->prof_cap == 0 || ctx->prof_calls >= ctx->prof_cap) return;
  size_t i = ((size_t)ctx->prof_calls * ST_COUNT + stage) * 2 + edge;
  if (cudaEventRecord(ctx->prof_events[i], s) == cudaSuccess) ctx->prof_set[i] = 1;
}

template <typename TA, typename TB, typename AccT, typename TC, bool B_KN>
int launch_table(covspec_ctx* ctx, int table, int lower_only, cudaStream_t s) {
  int tiles = ctx->plan.tiles[table];
  if (tiles == 0) return COVSPEC_OK;
  gemm_simt_kernel<TA, TB, AccT, TC, B_KN><<<tiles, 256, 0, s>>>(
      ctx->d_tables + (size_t)table * ctx->cfg.max_batch, ctx->plan.n_stage2, GemmProb{}, lower_only);
  LAUNCH_CHECK(ctx);
  return COVSPEC_OK;
}

template <typename T>
int launch_single_nt(covspec_ctx* ctx, const T* A, const T* B, float* C, int m, int n, int k, int lda,
                     int ldb, int ldc, cudaStream_t s) {
  GemmProb g{};
  g.A = A; g.B = B; g.C = C; g.m = m; g.n = n; g.k = k; g.lda = lda; g.ldb = ldb; g.ldc = ldc;
  g.tile_start = 0;
  g.tiles_n = (n + kGemmBN - 1) / kGemmBN;
  int tiles = ((m + kGemmBM - 1) / kGemmBM) * g.tiles_n;
  gemm_simt_kernel<T, T, float, float, false><<<tiles, 256, 0, s>>>(nullptr, 0, g, 0);
  LAUNCH_CHECK(ctx);
  return COVSPEC_OK;
}

// ---- tensor-core relevance path ----------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      ptr = nullptr;
    return reinterpret_cast<EncodeTiledFn>(ptr);
  }();
  return fn;
}

// Tensor map of a row-major bf16 matrix [rows, cols] with boxes of 64 columns (one 128-byte
// swizzle row) by box_rows rows; out-of-range elements read as zero.
int make_map_bf16(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) { g_cuda_error = "cuTensorMapEncodeTiled is not available"; return COVSPEC_ERR_CUDA; }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)tc::kBK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_cuda_error = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return COVSPEC_ERR_CUDA;
  }
  return COVSPEC_OK;
}

bool tc_supported(const covspec_ctx* ctx) {
  const covspec_config& c = ctx->cfg;
  return ctx->tc_ready && c.relevance_path != 1 && (c.dtype == COVSPEC_BF16 || ctx->split_tc) && c.n_heads > 0 &&
         c.head_dim == tc::kHeadDim && c.head_reduce == 0 && c.d >= tc::kBK;
}

// Eq. 10 on the tensor cores, two-SM form (relevance_pair.cuh): query embedding (MODE 1), -inf fill,
// fused projection + cosine max over pairs of token tiles.
int relevance_pair(covspec_ctx* ctx, const covspec_problem* p, float* s_query, cudaStream_t s) {
  const covspec_config& cfg = ctx->cfg;
  const Plan& pl = ctx->plan;
  int P = ctx->P, d = cfg.d;
  const void *X = p->X, *Q = p->Q, *Wk = p->Wk, *Wq = p->Wq;
  if (ctx->split_tc) { X = ctx->X3; Q = ctx->Q3; Wk = ctx->Wk3; Wq = ctx->Wq3; d = ctx->d3; }
  __nv_bfloat16* qn = reinterpret_cast<__nv_bfloat16*>(ctx->Qn);
  CUtensorMap map_x, map_wk, map_q, map_wq, map_qn, map_qnl;
  long long lo_off = (long long)cfg.max_total_txt * P;   // lo parts follow the hi parts
  int st;
  if ((st = make_map_bf16(&map_x, X, pl.total_vis, d, tc::kTileM))) return st;
  if ((st = make_map_bf16(&map_wk, Wk, P, d, tc::kTileN / 2))) return st;
  if ((st = make_map_bf16(&map_q, Q, pl.total_txt, d, tc::kTileM))) return st;
  if ((st = make_map_bf16(&map_wq, Wq, P, d, tc::kTileN / 2))) return st;
  if ((st = make_map_bf16(&map_qn, qn, pl.total_txt, P, tc::kTT / 2))) return st;
  if ((st = make_map_bf16(&map_qnl, qn + lo_off, pl.total_txt, P, tc::kTT / 2))) return st;
  int n_hp = (cfg.n_heads + 1) / 2;
  tc2::PairParams prm{};
  prm.plan = ctx->d_plan; prm.batch = p->batch;
  prm.n_groups = n_hp; prm.hp_per_group = 1;
  prm.n_heads = cfg.n_heads; prm.k_chunks = (d + tc::kBK - 1) / tc::kBK; prm.P = P;
  prm.status = ctx->status;
  const int max_clusters = ctx->num_sms / 2;
  // query side
  prof_mark(ctx, ST_QEMBED, 0, s);
  prm.rows_total = pl.total_txt;
  prm.n_items = (int)((pl.total_txt + 2 * tc::kTileM - 1) / (2 * tc::kTileM)) * prm.n_groups;
  prm.qn_out = qn; prm.qn_lo_off = lo_off; prm.s_query = nullptr;
  prm.fill = s_query; prm.fill_n = pl.total_vis;          // -inf for the visual-side launch below
  int grid = 2 * std::min(prm.n_items, max_clusters);
  tc2::relevance_pair_kernel<1><<<grid, tc2::kPairThreads, tc2::kSmemBytes2, s>>>(map_q, map_wq, map_qn, map_qnl, prm);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_QEMBED, 1, s);
  // visual side
  prof_mark(ctx, ST_RELEVANCE, 0, s);
  prm.n_items = pl.n_pairs * prm.n_groups;
  prm.qn_out = nullptr; prm.s_query = s_query; prm.fill = nullptr;
  grid = 2 * std::min(prm.n_items, max_clusters);
  tc2::relevance_pair_kernel<0><<<grid, tc2::kPairThreads, tc2::kSmemBytes2, s>>>(map_x, map_wk, map_qn, map_qnl, prm);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_RELEVANCE, 1, s);
  return COVSPEC_OK;
}

// Eq. 10 on the tensor cores: query embedding (MODE 1), -inf fill, fused projection + cosine max.
int relevance_tc(covspec_ctx* ctx, const covspec_problem* p, float* s_query, cudaStream_t s) {
  const covspec_config& cfg = ctx->cfg;
  const Plan& pl = ctx->plan;
  int P = ctx->P, d = cfg.d;
  const void *X = p->X, *Q = p->Q, *Wk = p->Wk, *Wq = p->Wq;
  if (ctx->split_tc) { X = ctx->X3; Q = ctx->Q3; Wk = ctx->Wk3; Wq = ctx->Wq3; d = ctx->d3; }
  __nv_bfloat16* qn = reinterpret_cast<__nv_bfloat16*>(ctx->Qn);
  CUtensorMap map_x, map_wk, map_q, map_wq, map_qn, map_qnl;
  long long lo_off = (long long)cfg.max_total_txt * P;   // lo parts follow the hi parts
  int st;
  if ((st = make_map_bf16(&map_x, X, pl.total_vis, d, tc::kTileM))) return st;
  if ((st = make_map_bf16(&map_wk, Wk, P, d, tc::kTileN))) return st;
  if ((st = make_map_bf16(&map_q, Q, pl.total_txt, d, tc::kTileM))) return st;
  if ((st = make_map_bf16(&map_wq, Wq, P, d, tc::kTileN))) return st;
  if ((st = make_map_bf16(&map_qn, qn, pl.total_txt, P, tc::kTT))) return st;
  if ((st = make_map_bf16(&map_qnl, qn + lo_off, pl.total_txt, P, tc::kTT))) return st;
  int n_hp = (cfg.n_heads + 1) / 2;
  tc::Params prm{};
  prm.plan = ctx->d_plan; prm.batch = p->batch;
  prm.n_groups = n_hp; prm.hp_per_group = 1;
  prm.n_heads = cfg.n_heads; prm.k_chunks = (d + tc::kBK - 1) / tc::kBK; prm.P = P;
  prm.status = ctx->status;
  // query side
  prof_mark(ctx, ST_QEMBED, 0, s);
  prm.rows_total = pl.total_txt;
  prm.n_items = (int)((pl.total_txt + tc::kTileM - 1) / tc::kTileM) * prm.n_groups;
  prm.qn_out = qn; prm.qn_lo_off = lo_off; prm.s_query = nullptr;
  prm.fill = s_query; prm.fill_n = pl.total_vis;          // -inf for the visual-side launch below
  int grid = prm.n_items < ctx->num_sms ? prm.n_items : ctx->num_sms;
  tc::relevance_tc_kernel<1><<<grid, 192, tc::kSmemBytes, s>>>(map_q, map_wq, map_qn, map_qnl, prm);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_QEMBED, 1, s);
  // visual side
  prof_mark(ctx, ST_RELEVANCE, 0, s);
  prm.n_items = pl.n_tiles * prm.n_groups;
  prm.qn_out = nullptr; prm.s_query = s_query; prm.fill = nullptr;
  grid = prm.n_items < ctx->num_sms ? prm.n_items : ctx->num_sms;
  tc::relevance_tc_kernel<0><<<grid, 192, tc::kSmemBytes, s>>>(map_x, map_wk, map_qn, map_qnl, prm);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_RELEVANCE, 1, s);
  return COVSPEC_OK;
}

// ---- Eq. 10-12 -------------------------------------------------------------------------------
// Eq. 11 on `s`: the full-rate kernel, or (background = true) the small persistent grid that runs
// beside the relevance kernel.
template <typename T>
int launch_activity(covspec_ctx* ctx, const covspec_problem* p, float* s_act, bool background,
                    cudaStream_t s) {
  const covspec_config& cfg = ctx->cfg;
  long long rowsX = ctx->plan.total_vis;
  LayerPtrs lp{};
  for (int l = 0; l <= cfg.act_layers; ++l) lp.h[l] = p->Hs[l];
  if (background) {
    // beside the two-SM relevance kernel only one block per SM fits (shared-memory reserve)
    int per_sm = cfg.relevance_path == 2 ? 1 : cfg.activity_overlap;
    unsigned grid = (unsigned)std::min<long long>((rowsX + 15) / 16, (long long)ctx->num_sms * per_sm);
    if (cfg.act_layers <= 4)
      activity_stream_kernel<T, 4><<<grid, 512, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
    else if (cfg.act_layers <= 8)
      activity_stream_kernel<T, 8><<<grid, 512, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
    else
      activity_stream_kernel<T, 16><<<grid, 512, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
  } else {
    unsigned grid = (unsigned)((rowsX + 7) / 8);
    if (cfg.act_layers <= 4)
      activity_kernel<T, 4><<<grid, 256, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
    else if (cfg.act_layers <= 8)
      activity_kernel<T, 8><<<grid, 256, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
    else
      activity_kernel<T, 16><<<grid, 256, 0, s>>>(lp, cfg.act_layers, rowsX, cfg.d, s_act);
  }
  LAUNCH_CHECK(ctx);
  return COVSPEC_OK;
}

template <typename T>
int score_impl(covspec_ctx* ctx, const covspec_problem* p, float* s_query, float* s_act,
               float* s_fused, bool do_fuse, cudaStream_t s) {
  const covspec_config& cfg = ctx->cfg;
  const Plan& pl = ctx->plan;
  int B = p->batch;
  int rowsQ = (int)pl.total_txt;
  long long rowsX = pl.total_vis;
  const T* X = reinterpret_cast<const T*>(p->X);
  const T* Q = reinterpret_cast<const T*>(p->Q);
  int P = ctx->P, hd = ctx->hd, H = ctx->heads;
  if (!s_query) s_query = ctx->sq;
  if (!s_act) s_act = ctx->sa;
  bool identity = cfg.n_heads == 0;
  bool use_tc = tc_supported(ctx);
  // The tensor-core relevance kernel leaves HBM idle: the activity stream runs beside it on the
  // context's side stream (fork here, join before the scores are fused).
  bool overlap = use_tc && cfg.act_layers > 0 && cfg.activity_overlap > 0;
  if (overlap) {
    CUDA_TRY(cudaEventRecord(ctx->ev_fork, s));
    CUDA_TRY(cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    prof_mark(ctx, ST_ACTIVITY, 0, ctx->side);
    int st = launch_activity<T>(ctx, p, s_act, true, ctx->side);
    if (st) return st;
    prof_mark(ctx, ST_ACTIVITY, 1, ctx->side);
    CUDA_TRY(cudaEventRecord(ctx->ev_join, ctx->side));
  }
  if (use_tc) {
    if (ctx->split_tc) {
      // float32 inputs: tokens and queries in the "a" form, the two weight matrices in the "b" form
      SplitJobs jobs{};
      jobs.j[0] = SplitJob{reinterpret_cast<const float*>(p->X), nullptr, ctx->X3, nullptr, rowsX};
      jobs.j[1] = SplitJob{reinterpret_cast<const float*>(p->Q), nullptr, ctx->Q3, nullptr, (long long)rowsQ};
      jobs.j[2] = SplitJob{reinterpret_cast<const float*>(p->Wk), nullptr, nullptr, ctx->Wk3, (long long)P};
      jobs.j[3] = SplitJob{reinterpret_cast<const float*>(p->Wq), nullptr, nullptr, ctx->Wq3, (long long)P};
      long long most = std::max<long long>(std::max<long long>(rowsX, rowsQ), P);
      dim3 grid((unsigned)std::min<long long>(most, 8ll * ctx->num_sms), 4);
      split3_kernel<<<grid, 256, 0, s>>>(jobs, ctx->d_plan, B, cfg.d, ctx->dp);
      LAUNCH_CHECK(ctx);
    }
    int st = cfg.relevance_path == 2 ? relevance_pair(ctx, p, s_query, s) : relevance_tc(ctx, p, s_query, s);
    if (st) return st;
  } else {
  prof_mark(ctx, ST_QEMBED, 0, s);
  if (identity) {
    int warps = rowsQ * H;
    qnorm_kernel<T><<<(warps + 7) / 8, 256, 0, s>>>(Q, ctx->Qn, rowsQ, H, hd);
    LAUNCH_CHECK(ctx);
  } else {
    int st = launch_single_nt<T>(ctx, Q, reinterpret_cast<const T*>(p->Wq), ctx->Qn, rowsQ, P, cfg.d,
                                 cfg.d, cfg.d, P, s);
    if (st) return st;
    int warps = rowsQ * H;
    qnorm_kernel<float><<<(warps + 7) / 8, 256, 0, s>>>(ctx->Qn, ctx->Qn, rowsQ, H, hd);
    LAUNCH_CHECK(ctx);
  }
  prof_mark(ctx, ST_QEMBED, 1, s);
  int mean = cfg.head_reduce == 1;
  size_t smem = mean ? (size_t)8 * pl.t_max * sizeof(float) : 0;
  if (smem > 48 * 1024) return COVSPEC_ERR_UNSUPPORTED;
  prof_mark(ctx, ST_RELEVANCE, 0, s);
  if (identity) {
    cosmax_kernel<T><<<(unsigned)((rowsX + 7) / 8), 256, smem, s>>>(
        X, ctx->Qn, ctx->d_plan, B, 0, (int)rowsX, H, hd, mean, pl.t_max, s_query);
    LAUNCH_CHECK(ctx);
  } else {
    for (long long r0 = 0; r0 < rowsX; r0 += ctx->kp_rows) {
      int rows = (int)((rowsX - r0) < ctx->kp_rows ? (rowsX - r0) : ctx->kp_rows);
      int st = launch_single_nt<T>(ctx, X + (size_t)r0 * cfg.d, reinterpret_cast<const T*>(p->Wk),
                                   ctx->Kp, rows, P, cfg.d, cfg.d, cfg.d, P, s);
      if (st) return st;
      cosmax_kernel<float><<<(rows + 7) / 8, 256, smem, s>>>(ctx->Kp, ctx->Qn, ctx->d_plan, B, (int)r0,
                                                             rows, H, hd, mean, pl.t_max, s_query);
      LAUNCH_CHECK(ctx);
    }
  }
  prof_mark(ctx, ST_RELEVANCE, 1, s);
  }
  if (overlap) {
    CUDA_TRY(cudaStreamWaitEvent(s, ctx->ev_join, 0));
  } else if (cfg.act_layers > 0) {
    prof_mark(ctx, ST_ACTIVITY, 0, s);
    int st = launch_activity<T>(ctx, p, s_act, false, s);
    if (st) return st;
    prof_mark(ctx, ST_ACTIVITY, 1, s);
  }
  if (do_fuse) {
    prof_mark(ctx, ST_FUSE, 0, s);
    fuse_kernel<<<B, 1024, 0, s>>>(s_query, cfg.act_layers > 0 ? s_act : nullptr, ctx->d_plan,
                                   cfg.lambda, cfg.norm_mode, s_fused, ctx->status);
    LAUNCH_CHECK(ctx);
    prof_mark(ctx, ST_FUSE, 1, s);
  }
  return COVSPEC_OK;
}

// ---- preselect, Eq. 13-15, final select ---------------------------------------------------------
template <typename T>
int select_impl(covspec_ctx* ctx, const covspec_problem* p, const float* s_fused, int* keep_idx,
                int* presel_out, float* energy_out, cudaStream_t s, bool presel_done = false) {
  const covspec_config& cfg = ctx->cfg;
  const Plan& pl = ctx->plan;
  int B = p->batch;
  int* presel = presel_out ? presel_out : ctx->presel;
  float* energy = energy_out ? energy_out : ctx->energy;
  if (!presel_done) {
    prof_mark(ctx, ST_PRESELECT, 0, s);
    preselect_kernel<<<B, 1024, 0, s>>>(s_fused, ctx->d_plan, presel, ctx->status);
    LAUNCH_CHECK(ctx);
    prof_mark(ctx, ST_PRESELECT, 1, s);
  }
  if (pl.n_stage2 > 0) {
    prof_mark(ctx, ST_GRAM, 0, s);
    int st;
    dim3 gb(std::min(64, (pl.p_max * pl.m_max + 255) / 256 + 1), B);
    if (ctx->split_tc) {
      // float32 inputs on the tensor cores: the preselected rows are gathered and split in one pass
      SplitJobs jobs{};
      jobs.j[0] = SplitJob{reinterpret_cast<const float*>(p->X), presel, ctx->Za3, ctx->Zb3, pl.total_presel};
      dim3 grid((unsigned)std::min<long long>(pl.total_presel, 8ll * ctx->num_sms), 1);
      split3_kernel<<<grid, 256, 0, s>>>(jobs, ctx->d_plan, B, cfg.d, ctx->dp);
      LAUNCH_CHECK(ctx);
      sub::GramParams gp{};
      gp.plan = ctx->d_plan; gp.batch = B; gp.n_items = pl.n_gram_tiles;
      gp.k_chunks = ctx->d3 / sub::kBK;
      gp.g_hi = ctx->Ghi; gp.g_lo = ctx->Glo; gp.ld = ctx->ld; gp.status = ctx->status;
      int grid_g = std::min(pl.n_gram_tiles, ctx->num_sms);
      sub::gram_tc_kernel<<<grid_g, 192, sub::kGramSmem, s>>>(ctx->map_za3, ctx->map_zb3w, gp);
      LAUNCH_CHECK(ctx);
      prof_mark(ctx, ST_GRAM, 1, s);
    } else {
    int vec16 = cfg.d * ctx->esize / 16;
    gather_rows_kernel<<<gather_grid(pl.total_presel), kGatherWarps * 32, 0, s>>>(
        reinterpret_cast<const uint4*>(p->X), presel, ctx->d_plan, B, 1, vec16, (int)pl.total_presel,
        reinterpret_cast<uint4*>(ctx->Zg), nullptr, ctx->status);
    LAUNCH_CHECK(ctx);
    if (cfg.dtype == COVSPEC_BF16) {
      sub::GramParams gp{};
      gp.plan = ctx->d_plan; gp.batch = B; gp.n_items = pl.n_gram_tiles;
      gp.k_chunks = (cfg.d + sub::kBK - 1) / sub::kBK;
      gp.g_hi = ctx->Ghi; gp.g_lo = ctx->Glo; gp.ld = ctx->ld; gp.status = ctx->status;
      int grid = std::min(pl.n_gram_tiles, ctx->num_sms);
      sub::gram_tc_kernel<<<grid, 192, sub::kGramSmem, s>>>(ctx->map_zg, ctx->map_zgw, gp);
      LAUNCH_CHECK(ctx);
    } else {
      if ((st = launch_table<T, T, float, float, false>(ctx, T_GRAM_G, 1, s))) return st;
      dim3 gs(std::min(64, (pl.m_max * pl.m_max + 255) / 256 + 1), B);
      sub::split_planes_kernel<<<gs, 256, 0, s>>>(ctx->d_plan, ctx->G, ctx->Ghi, ctx->Glo, ctx->ld);
      LAUNCH_CHECK(ctx);
    }
    prof_mark(ctx, ST_GRAM, 1, s);
    }
    prof_mark(ctx, ST_EIG, 0, s);
    if (cfg.lowrank_mode == 1) {
      // greedy pivoted selection instead of the subspace energies; it writes its own `energy`
      greedy_select_kernel<<<B, kGreedyThreads, 0, s>>>(ctx->d_plan, ctx->Ghi, ctx->Glo, ctx->ld, ctx->Cg, energy, ctx->status);
      LAUNCH_CHECK(ctx);
      prof_mark(ctx, ST_EIG, 1, s);
      prof_mark(ctx, ST_FINAL, 0, s);
      final_select_kernel<<<B, 1024, 0, s>>>(energy, presel, ctx->d_plan, keep_idx, ctx->status);
      LAUNCH_CHECK(ctx);
      return COVSPEC_OK;
    }
    sub::basis_init_kernel<<<gb, 256, 0, s>>>(ctx->d_plan, ctx->Yp[0][0], ctx->Yp[0][1], ctx->Yp[1][0],
                                              ctx->Yp[1][1], ctx->ld, energy, ctx->sync, B, cfg.eig_iters);
    LAUNCH_CHECK(ctx);
    // every multiplication by G, the factorisations between them, the Rayleigh-Ritz solve and the
    // energies: one cooperative launch (its CTAs wait on one another through global counters)
    sub::FusedParams fp{};
    fp.plan = ctx->d_plan; fp.batch = B; fp.n_items = pl.n_ptiles; fp.sched = ctx->d_sched;
    fp.tile_rows = pl.tile_rows;
    fp.spread_sum = pl.n_ptiles <= pl.tile_ctas ? 1 : 0;     // one tile per CTA (see the schedule above)
    fp.n_tile_ctas = pl.tile_ctas; fp.n_servers = pl.servers;
    fp.steps = cfg.eig_iters + 1;
    fp.lbuf = ctx->Lbuf;
    for (int i = 0; i < 2; ++i) { fp.y_hi[i] = ctx->Yp[i][0]; fp.y_lo[i] = ctx->Yp[i][1]; fp.yf[i] = ctx->Yf[i]; }
    fp.ld = ctx->ld;
    fp.partial = ctx->partial; fp.ub = ctx->Ub; fp.energy = energy; fp.sync = ctx->sync;
    fp.max_sweeps = 30; fp.conv_tol = cfg.conv_tol; fp.status = ctx->status;
    fp.early_stop = cfg.eig_early_stop && cfg.conv_tol > 0.f;
    void* args[] = {&ctx->map_gh, &ctx->map_gl, &ctx->map_y[0][0], &ctx->map_y[0][1], &ctx->map_y[1][0],
                    &ctx->map_y[1][1], &fp};
    CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(sub::subspace_kernel), dim3(pl.pow_grid),
                                         dim3(sub::kPowThreads), args, sub::kPowSmem, s));
    LAUNCH_CHECK(ctx);
  } else {
    // no request reaches stage 2: the final selection keeps the preselected sets; energies are zero
    dim3 gz(1, B);
    sub::basis_init_kernel<<<gz, 256, 0, s>>>(ctx->d_plan, ctx->Yp[0][0], ctx->Yp[0][1], ctx->Yp[1][0],
                                              ctx->Yp[1][1], ctx->ld, energy, ctx->sync, B, cfg.eig_iters);
    LAUNCH_CHECK(ctx);
  }
  if (pl.n_stage2 > 0) prof_mark(ctx, ST_EIG, 1, s);
  prof_mark(ctx, ST_FINAL, 0, s);
  final_select_kernel<<<B, 1024, 0, s>>>(energy, presel, ctx->d_plan, keep_idx, ctx->status);
  LAUNCH_CHECK(ctx);
  return COVSPEC_OK;
}

int compact_impl(covspec_ctx* ctx, const covspec_problem* p, const int* keep_idx, void* out,
                 int* out_pos, cudaStream_t s) {
  const Plan& pl = ctx->plan;
  int vec16 = ctx->cfg.d * ctx->esize / 16;
  gather_rows_kernel<<<gather_grid(pl.total_keep), kGatherWarps * 32, 0, s>>>(
      reinterpret_cast<const uint4*>(p->X), keep_idx, ctx->d_plan, p->batch, 0, vec16, (int)pl.total_keep,
      reinterpret_cast<uint4*>(out), out_pos, ctx->status);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_FINAL, 1, s);
  return COVSPEC_OK;
}

int check_score_args(const covspec_ctx* ctx, const covspec_problem* p) {
  if (!p->X || !p->Q) return COVSPEC_ERR_ARG;
  if (ctx->cfg.n_heads > 0 && (!p->Wq || !p->Wk)) return COVSPEC_ERR_ARG;
  if (ctx->cfg.act_layers > 0) {
    if (!p->Hs) return COVSPEC_ERR_ARG;
    for (int l = 0; l <= ctx->cfg.act_layers; ++l) if (!p->Hs[l]) return COVSPEC_ERR_ARG;
  }
  return COVSPEC_OK;
}

void copy_offsets(const Plan& pl, int* keep_offsets) {
  if (keep_offsets) memcpy(keep_offsets, pl.keep_offsets.data(), sizeof(int) * pl.keep_offsets.size());
}

}  // namespace

// ================================================================================================
extern "C" {

void covspec_default_config(covspec_config* c) {
  if (!c) return;
  memset(c, 0, sizeof(*c));
  c->dtype = COVSPEC_BF16;
  c->head_dim = 128;
  c->act_layers = 4;
  c->lambda = 0.5f;
  c->norm_mode = 0;
  c->head_reduce = 0;
  c->presel_factor = 2.0f;
  c->rank_frac = 0.5f;
  c->rank_cap = 128;
  c->eig_iters = 5;
  c->eig_oversample = 16;
  c->relevance_path = 0;
  c->lowrank_mode = 0;
  c->ritz_window = 16;
  c->activity_overlap = 1;
  c->conv_tol = 2e-3f;
  c->eig_early_stop = 1;
}

int covspec_budgets(const covspec_config* cfg, int n, int keep, int* b_vis, int* m, int* r) {
  if (!cfg || !b_vis || !m || !r) return COVSPEC_ERR_ARG;
  return budgets_impl(cfg, n, keep, b_vis, m, r);
}

int covspec_plan_sizes(const covspec_config* cfg, const covspec_problem* p, int* keep_offsets,
                       int* presel_offsets) {
  if (!cfg) return COVSPEC_ERR_ARG;
  int st = validate_problem(cfg, p);
  if (st) return st;
  int ko = 0, po = 0;
  if (keep_offsets) keep_offsets[0] = 0;
  if (presel_offsets) presel_offsets[0] = 0;
  for (int b = 0; b < p->batch; ++b) {
    int n = p->vis_offsets[b + 1] - p->vis_offsets[b], B, M, R;
    if (budgets_impl(cfg, n, keep_of(p, b, n), &B, &M, &R)) return COVSPEC_ERR_SHAPE;
    ko += B; po += M;
    if (keep_offsets) keep_offsets[b + 1] = ko;
    if (presel_offsets) presel_offsets[b + 1] = po;
  }
  return COVSPEC_OK;
}

int covspec_prune_init(const covspec_config* cfg, covspec_ctx** out) {
  if (!out) return COVSPEC_ERR_ARG;
  *out = nullptr;
  int st = validate_cfg(cfg);
  if (st) return st;
  if (cfg->max_batch < 1 || cfg->max_total_vis < 1 || cfg->max_total_txt < 1 || cfg->max_vis_per_req < 1)
    return COVSPEC_ERR_ARG;
  covspec_ctx* ctx = new covspec_ctx();
  ctx->cfg = *cfg;
  covspec_config& c = ctx->cfg;
  if (c.max_presel_per_req <= 0) c.max_presel_per_req = c.max_vis_per_req;
  if (c.max_total_presel <= 0) c.max_total_presel = c.max_total_vis;
  ctx->esize = c.dtype == COVSPEC_BF16 ? 2 : 4;
  ctx->heads = c.n_heads > 0 ? c.n_heads : 1;
  ctx->hd = c.n_heads > 0 ? c.head_dim : c.d;
  ctx->P = ctx->heads * ctx->hd;
  // projection chunk: keep the float32 embedding of a chunk within ~64 MB so it stays in L2
  long long rows = (64ll << 20) / ((long long)ctx->P * 4);
  rows = rows < 256 ? 256 : rows / 64 * 64;
  if (rows > c.max_total_vis) rows = round_up(c.max_total_vis, 64);
  ctx->kp_rows = c.n_heads > 0 ? rows : 0;
  bool f32 = c.dtype == COVSPEC_F32;
  long long ldm_max = round_up(c.max_presel_per_req, 4);
  ctx->g_cap = f32 ? (c.max_total_presel + 4ll * c.max_batch) * ldm_max : 0;
  ctx->ld = (int)round_up(c.max_presel_per_req, 64);
  ctx->cap_rows = c.max_total_presel;
  ctx->cap_ptiles = std::max<long long>(c.max_total_presel / sub::kTile + c.max_batch, 192);   // >= one per SM

  long long off = 0;
  auto carve = [&](long long bytes) { long long o = off; off += round_up(bytes, 1024); return o; };
  long long o_status = carve(256);
  long long o_plan = carve(sizeof(ReqPlan) * c.max_batch);
  long long o_tab = carve(sizeof(GemmProb) * (long long)T_COUNT * c.max_batch);
  long long sched_ints = 1024 + ctx->cap_ptiles;   // offsets of up to 1023 CTAs + one entry per tile
  long long o_sched = carve(4 * sched_ints);
  long long o_qn = carve(4ll * c.max_total_txt * ctx->P);
  long long o_kp = carve(4ll * ctx->kp_rows * ctx->P);
  long long o_sq = carve(4ll * c.max_total_vis), o_sa = carve(4ll * c.max_total_vis);
  long long o_sf = carve(4ll * c.max_total_vis);
  long long o_presel = carve(4ll * c.max_total_presel), o_energy = carve(4ll * c.max_total_presel);
  long long o_zg = carve((long long)ctx->esize * c.max_total_presel * c.d);
  long long o_g = carve(4ll * ctx->g_cap);
  long long plane = 2ll * ctx->cap_rows * ctx->ld;
  long long o_gh = carve(plane), o_gl = carve(plane);
  long long yplane = 2ll * c.max_batch * kPMax * ctx->ld;
  long long o_y[2][2];
  for (int i = 0; i < 2; ++i) for (int j = 0; j < 2; ++j) o_y[i][j] = carve(yplane);
  long long o_yf0 = carve(4ll * ctx->cap_rows * kPMax), o_yf1 = carve(4ll * ctx->cap_rows * kPMax);
  long long o_part = carve(8ll * ctx->cap_ptiles * sub::kTileDoubles);
  long long o_lbuf = carve(4ll * c.max_batch * sub::kLbufStride);
  long long o_ub = carve(4ll * c.max_batch * kPMax * kPMax);
  long long o_sync = carve(4ll * (c.max_batch * sub::kSyncStride + 4));
  ctx->cg_cap = c.lowrank_mode == 1 ? (long long)c.max_total_presel * c.max_presel_per_req : 0;
  long long o_cg = carve(4ll * ctx->cg_cap);
  ctx->split_tc = f32 && c.relevance_path != 1 && c.n_heads > 0 && c.head_dim == tc::kHeadDim &&
                  c.head_reduce == 0 && c.d >= tc::kBK && c.d % 4 == 0;
  ctx->dp = (int)round_up(c.d, 64);
  ctx->d3 = 3 * ctx->dp;
  long long o_x3 = 0, o_q3 = 0, o_wq3 = 0, o_wk3 = 0, o_za3 = 0, o_zb3 = 0;
  if (ctx->split_tc) {
    o_x3 = carve(2ll * c.max_total_vis * ctx->d3);
    o_q3 = carve(2ll * c.max_total_txt * ctx->d3);
    o_wq3 = carve(2ll * ctx->P * ctx->d3);
    o_wk3 = carve(2ll * ctx->P * ctx->d3);
    o_za3 = carve(2ll * c.max_total_presel * ctx->d3);
    o_zb3 = carve(2ll * c.max_total_presel * ctx->d3);
  }
  ctx->ws_bytes = off;
  cudaError_t e = cudaMalloc(&ctx->ws, (size_t)off);
  if (e != cudaSuccess) {
    g_cuda_error = std::string("cudaMalloc workspace: ") + cudaGetErrorString(e);
    delete ctx;
    return COVSPEC_ERR_CUDA;
  }
  char* w = ctx->ws;
  ctx->status = reinterpret_cast<int*>(w + o_status);
  ctx->d_plan = reinterpret_cast<ReqPlan*>(w + o_plan);
  ctx->d_tables = reinterpret_cast<GemmProb*>(w + o_tab);
  ctx->d_sched = reinterpret_cast<int*>(w + o_sched);
  ctx->Qn = reinterpret_cast<float*>(w + o_qn);
  ctx->Kp = reinterpret_cast<float*>(w + o_kp);
  ctx->sq = reinterpret_cast<float*>(w + o_sq);
  ctx->sa = reinterpret_cast<float*>(w + o_sa);
  ctx->sf = reinterpret_cast<float*>(w + o_sf);
  ctx->presel = reinterpret_cast<int*>(w + o_presel);
  ctx->energy = reinterpret_cast<float*>(w + o_energy);
  ctx->Zg = w + o_zg;
  ctx->G = reinterpret_cast<float*>(w + o_g);
  ctx->Ghi = reinterpret_cast<__nv_bfloat16*>(w + o_gh);
  ctx->Glo = reinterpret_cast<__nv_bfloat16*>(w + o_gl);
  for (int i = 0; i < 2; ++i)
    for (int j = 0; j < 2; ++j) ctx->Yp[i][j] = reinterpret_cast<__nv_bfloat16*>(w + o_y[i][j]);
  ctx->Yf[0] = reinterpret_cast<float*>(w + o_yf0);
  ctx->Yf[1] = reinterpret_cast<float*>(w + o_yf1);
  ctx->partial = reinterpret_cast<double*>(w + o_part);
  ctx->Lbuf = reinterpret_cast<float*>(w + o_lbuf);
  ctx->Ub = reinterpret_cast<float*>(w + o_ub);
  ctx->sync = reinterpret_cast<unsigned*>(w + o_sync);
  if (ctx->split_tc) {
    ctx->X3 = reinterpret_cast<__nv_bfloat16*>(w + o_x3);
    ctx->Q3 = reinterpret_cast<__nv_bfloat16*>(w + o_q3);
    ctx->Wq3 = reinterpret_cast<__nv_bfloat16*>(w + o_wq3);
    ctx->Wk3 = reinterpret_cast<__nv_bfloat16*>(w + o_wk3);
    ctx->Za3 = reinterpret_cast<__nv_bfloat16*>(w + o_za3);
    ctx->Zb3 = reinterpret_cast<__nv_bfloat16*>(w + o_zb3);
  }
  ctx->Cg = reinterpret_cast<float*>(w + o_cg);
  ctx->stage_bytes = round_up(sizeof(ReqPlan) * c.max_batch, 256) +
                     sizeof(GemmProb) * (long long)T_COUNT * c.max_batch;
  ctx->stage_sched_off = round_up(ctx->stage_bytes, 256);
  ctx->stage_bytes = ctx->stage_sched_off + 4 * sched_ints;
  bool ok = cudaMemset(ctx->status, 0, 256) == cudaSuccess &&
            cudaMallocHost(&ctx->h_stage, (size_t)ctx->stage_bytes) == cudaSuccess &&
            cudaEventCreateWithFlags(&ctx->stage_free, cudaEventDisableTiming) == cudaSuccess &&
            cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) == cudaSuccess;
  // the small dense kernels need more than the default 48 KB of dynamic shared memory
  int dev = 0, cc_major = 0;
  ok = ok && cudaGetDevice(&dev) == cudaSuccess &&
       cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
       cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess;
  if (ok && (cc_major != 10 || encode_tiled_fn() == nullptr)) {
    g_cuda_error = "the library needs a compute capability 10.x device and cuTensorMapEncodeTiled";
    covspec_prune_destroy(ctx);
    return COVSPEC_ERR_UNSUPPORTED;
  }
  if (ok) {
    ctx->tc_ready =
        cudaFuncSetAttribute(tc::relevance_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc::kSmemBytes) == cudaSuccess &&
        cudaFuncSetAttribute(tc::relevance_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc::kSmemBytes) == cudaSuccess &&
        cudaFuncSetAttribute(tc2::relevance_pair_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc2::kSmemBytes2) == cudaSuccess &&
        cudaFuncSetAttribute(tc2::relevance_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc2::kSmemBytes2) == cudaSuccess &&
        cudaFuncSetAttribute(sub::gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sub::kGramSmem) == cudaSuccess &&
        cudaFuncSetAttribute(sub::subspace_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sub::kPowSmem) == cudaSuccess;
    ok = ctx->tc_ready;
  }
  if (ok) {
    // The background activity kernel shares its SMs with the relevance kernel, whose CTA needs the
    // largest shared-memory carve-out: ask for the same split, or the two could not be resident on
    // one SM at the same time (an SM changes its L1 / shared-memory split only when it is idle).
    auto max_shared = [](auto* kernel) {
      return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                  cudaSharedmemCarveoutMaxShared) == cudaSuccess;
    };
    ok = max_shared(activity_stream_kernel<__nv_bfloat16, 4>) && max_shared(activity_stream_kernel<__nv_bfloat16, 8>) &&
         max_shared(activity_stream_kernel<__nv_bfloat16, 16>) && max_shared(activity_stream_kernel<float, 4>) &&
         max_shared(activity_stream_kernel<float, 8>) && max_shared(activity_stream_kernel<float, 16>);
  }
  if (ok) {
    // tensor maps over the workspace arrays of the subspace iteration (fixed for the context)
    int st = COVSPEC_OK;
    if (!f32) st = make_map_bf16(&ctx->map_zg, ctx->Zg, c.max_total_presel, c.d, sub::kTile);
    if (!f32 && !st) st = make_map_bf16(&ctx->map_zgw, ctx->Zg, c.max_total_presel, c.d, sub::kGramN);
    if (ctx->split_tc && !st) st = make_map_bf16(&ctx->map_za3, ctx->Za3, c.max_total_presel, ctx->d3, sub::kTile);
    if (ctx->split_tc && !st) st = make_map_bf16(&ctx->map_zb3w, ctx->Zb3, c.max_total_presel, ctx->d3, sub::kGramN);
    if (!st) st = make_map_bf16(&ctx->map_gh, ctx->Ghi, ctx->cap_rows, ctx->ld, sub::kTile);
    if (!st) st = make_map_bf16(&ctx->map_gl, ctx->Glo, ctx->cap_rows, ctx->ld, sub::kTile);
    for (int i = 0; i < 2 && !st; ++i)
      for (int j = 0; j < 2 && !st; ++j)
        st = make_map_bf16(&ctx->map_y[i][j], ctx->Yp[i][j], (long long)c.max_batch * kPMax, ctx->ld, kPMax);
    if (st) { covspec_prune_destroy(ctx); return st; }
  }
  if (!ok) {
    g_cuda_error = std::string("context set-up: ") + cudaGetErrorString(cudaGetLastError());
    covspec_prune_destroy(ctx);
    return COVSPEC_ERR_CUDA;
  }
  *out = ctx;
  return COVSPEC_OK;
}

int covspec_prune_destroy(covspec_ctx* ctx) {
  if (!ctx) return COVSPEC_ERR_ARG;
  if (ctx->ws) cudaFree(ctx->ws);
  if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
  if (ctx->stage_free) cudaEventDestroy(ctx->stage_free);
  if (ctx->side) cudaStreamDestroy(ctx->side);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  delete ctx;
  return COVSPEC_OK;
}

long long covspec_workspace_bytes(const covspec_ctx* ctx) { return ctx ? ctx->ws_bytes : 0; }

int covspec_score(covspec_ctx* ctx, const covspec_problem* p, float* s_query, float* s_act,
                  float* s_fused, void* stream) {
  if (!ctx || !p || !s_fused) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int st = validate_problem(&ctx->cfg, p);
  if (st) return st;
  if ((st = check_score_args(ctx, p))) return st;
  ctx->launches = 0;
  if ((st = get_plan(ctx, p, s))) return st;
  return ctx->cfg.dtype == COVSPEC_BF16
             ? score_impl<__nv_bfloat16>(ctx, p, s_query, s_act, s_fused, true, s)
             : score_impl<float>(ctx, p, s_query, s_act, s_fused, true, s);
}

int covspec_select(covspec_ctx* ctx, const covspec_problem* p, const float* s_fused, int* keep_idx,
                   int* keep_offsets, int* presel_idx, float* energy, void* stream) {
  if (!ctx || !p || !s_fused || !keep_idx || !p->X) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  int st = get_plan(ctx, p, s);
  if (st) return st;
  copy_offsets(ctx->plan, keep_offsets);
  return ctx->cfg.dtype == COVSPEC_BF16
             ? select_impl<__nv_bfloat16>(ctx, p, s_fused, keep_idx, presel_idx, energy, s)
             : select_impl<float>(ctx, p, s_fused, keep_idx, presel_idx, energy, s);
}

int covspec_compact(covspec_ctx* ctx, const covspec_problem* p, const int* keep_idx,
                    const int* keep_offsets, void* out_hidden, int* out_pos, void* stream) {
  if (!ctx || !p || !keep_idx || !keep_offsets || !out_hidden || !p->X) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  int st = get_plan(ctx, p, s);
  if (st) return st;
  if (memcmp(keep_offsets, ctx->plan.keep_offsets.data(), sizeof(int) * (p->batch + 1)))
    return COVSPEC_ERR_SHAPE;
  return compact_impl(ctx, p, keep_idx, out_hidden, out_pos, s);
}

int covspec_compact_rows(covspec_ctx* ctx, const covspec_problem* p, const int* keep_idx,
                         const int* keep_offsets, const void* src, long long row_bytes, void* out,
                         void* stream) {
  if (!ctx || !p || !keep_idx || !keep_offsets || !src || !out) return COVSPEC_ERR_ARG;
  if (row_bytes < 16 || row_bytes % 16 != 0 || row_bytes / 16 > 0x7fffffffll) return COVSPEC_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(out)) & 15) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  int st = get_plan(ctx, p, s);
  if (st) return st;
  if (memcmp(keep_offsets, ctx->plan.keep_offsets.data(), sizeof(int) * (p->batch + 1)))
    return COVSPEC_ERR_SHAPE;
  gather_rows_kernel<<<gather_grid(ctx->plan.total_keep), kGatherWarps * 32, 0, s>>>(
      reinterpret_cast<const uint4*>(src), keep_idx, ctx->d_plan, p->batch, 0, (int)(row_bytes / 16),
      (int)ctx->plan.total_keep, reinterpret_cast<uint4*>(out), nullptr, ctx->status);
  LAUNCH_CHECK(ctx);
  return COVSPEC_OK;
}

int covspec_prune(covspec_ctx* ctx, const covspec_problem* p, void* out_hidden, int* keep_idx,
                  int* keep_offsets, void* stream) {
  if (!ctx || !p || !out_hidden || !keep_idx) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int st = validate_problem(&ctx->cfg, p);
  if (st) return st;
  if ((st = check_score_args(ctx, p))) return st;
  ctx->launches = 0;
  if ((st = get_plan(ctx, p, s))) return st;
  copy_offsets(ctx->plan, keep_offsets);
  bool bf = ctx->cfg.dtype == COVSPEC_BF16;
  float* fused = ctx->sf;
  st = bf ? score_impl<__nv_bfloat16>(ctx, p, nullptr, nullptr, fused, false, s)
          : score_impl<float>(ctx, p, nullptr, nullptr, fused, false, s);
  if (st) return st;
  // Eq. 12 and the preselection share one launch in the fused call
  prof_mark(ctx, ST_FUSE, 0, s);
  fuse_preselect_kernel<<<p->batch, 1024, 0, s>>>(ctx->sq, ctx->cfg.act_layers > 0 ? ctx->sa : nullptr,
                                                  ctx->d_plan, ctx->cfg.lambda, ctx->cfg.norm_mode, fused,
                                                  ctx->presel, ctx->status);
  LAUNCH_CHECK(ctx);
  prof_mark(ctx, ST_FUSE, 1, s);
  st = bf ? select_impl<__nv_bfloat16>(ctx, p, fused, keep_idx, nullptr, nullptr, s, true)
          : select_impl<float>(ctx, p, fused, keep_idx, nullptr, nullptr, s, true);
  if (st) return st;
  st = compact_impl(ctx, p, keep_idx, out_hidden, nullptr, s);
  if (ctx->prof_cap && ctx->prof_calls < ctx->prof_cap) ++ctx->prof_calls;
  return st;
}

int covspec_profile_begin(covspec_ctx* ctx, int max_calls) {
  if (!ctx || max_calls < 1 || ctx->prof_cap) return COVSPEC_ERR_ARG;
  size_t n = (size_t)max_calls * ST_COUNT * 2;
  ctx->prof_events.assign(n, nullptr);
  ctx->prof_set.assign(n, 0);
  for (size_t i = 0; i < n; ++i) CUDA_TRY(cudaEventCreate(&ctx->prof_events[i]));
  ctx->prof_cap = max_calls;
  ctx->prof_calls = 0;
  return COVSPEC_OK;
}

int covspec_profile_end(covspec_ctx* ctx, double* stage_ms, int n_stages, int* calls) {
  if (!ctx || !ctx->prof_cap) return COVSPEC_ERR_ARG;
  int st = COVSPEC_OK;
  for (int g = 0; g < n_stages; ++g) if (stage_ms) stage_ms[g] = 0.0;
  for (int c = 0; c < ctx->prof_calls; ++c)
    for (int g = 0; g < ST_COUNT; ++g) {
      size_t i = ((size_t)c * ST_COUNT + g) * 2;
      if (!ctx->prof_set[i] || !ctx->prof_set[i + 1]) continue;
      float ms = 0.f;
      if (cudaEventSynchronize(ctx->prof_events[i + 1]) != cudaSuccess ||
          cudaEventElapsedTime(&ms, ctx->prof_events[i], ctx->prof_events[i + 1]) != cudaSuccess) {
        st = COVSPEC_ERR_CUDA;
        continue;
      }
      if (stage_ms && g < n_stages) stage_ms[g] += ms;
    }
  if (calls) *calls = ctx->prof_calls;
  for (cudaEvent_t e : ctx->prof_events) if (e) cudaEventDestroy(e);
  ctx->prof_events.clear();
  ctx->prof_set.clear();
  ctx->prof_cap = ctx->prof_calls = 0;
  return st;
}

int covspec_profile_stage_count(void) { return ST_COUNT; }
const char* covspec_profile_stage_name(int stage) {
  return stage >= 0 && stage < ST_COUNT ? kStageNames[stage] : "";
}

int covspec_get_device_status(covspec_ctx* ctx, void* stream) {
  if (!ctx) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int h = 0;
  CUDA_TRY(cudaMemcpyAsync(&h, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaMemsetAsync(ctx->status, 0, sizeof(int), s));
  CUDA_TRY(cudaStreamSynchronize(s));
  if (h & kStatusBounds) return COVSPEC_ERR_BOUNDS;
  if (h & kStatusTimeout) return COVSPEC_ERR_TIMEOUT;
  if (h & kStatusNonFinite) return COVSPEC_ERR_NONFINITE;
  if (h & kStatusNoConverge) return COVSPEC_ERR_NOCONVERGE;
  return COVSPEC_OK;
}

int covspec_get_iteration_counts(covspec_ctx* ctx, int batch, int* multiplications, void* stream) {
  if (!ctx || !multiplications || batch < 1 || batch > ctx->cfg.max_batch) return COVSPEC_ERR_ARG;
  if (!ctx->plan.valid || (int)ctx->plan.req.size() != batch) return COVSPEC_ERR_SHAPE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  std::vector<unsigned> words((size_t)batch * sub::kSyncStride);
  CUDA_TRY(cudaMemcpyAsync(words.data(), ctx->sync, sizeof(unsigned) * words.size(), cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  for (int b = 0; b < batch; ++b)
    multiplications[b] = ctx->plan.req[b].stage2 ? (int)words[(size_t)b * sub::kSyncStride + 3] + 1 : 0;
  return COVSPEC_OK;
}

int covspec_correct(int logit_dtype, int rows, int vocab, long long ld, const void* z_draft,
                    const void* z_target, const int* drafted, const float* uniforms, float gamma,
                    float* margin, int* gate, float* accept, float* resid_mass, int* token,
                    void* stream) {
  if (!z_draft || !z_target || !uniforms || !margin || !gate || !token) return COVSPEC_ERR_ARG;
  if (logit_dtype != COVSPEC_F32 && logit_dtype != COVSPEC_BF16 && logit_dtype != COVSPEC_F16)
    return COVSPEC_ERR_ARG;
  int esize = logit_dtype == COVSPEC_F32 ? 4 : 2;
  if (rows < 1 || vocab < 2 || ld < vocab || (ld * esize) % 16 != 0) return COVSPEC_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(z_draft) | reinterpret_cast<uintptr_t>(z_target)) & 15) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (logit_dtype == COVSPEC_F32)
    corr::correct_kernel<float><<<rows * corr::kClusterCtas, corr::kThreads, 0, s>>>(
        static_cast<const float*>(z_draft), static_cast<const float*>(z_target), ld, vocab, drafted,
        uniforms, gamma, margin, gate, accept, resid_mass, token);
  else if (logit_dtype == COVSPEC_BF16)
    corr::correct_kernel<__nv_bfloat16><<<rows * corr::kClusterCtas, corr::kThreads, 0, s>>>(
        static_cast<const __nv_bfloat16*>(z_draft), static_cast<const __nv_bfloat16*>(z_target), ld,
        vocab, drafted, uniforms, gamma, margin, gate, accept, resid_mass, token);
  else
    corr::correct_kernel<__half><<<rows * corr::kClusterCtas, corr::kThreads, 0, s>>>(
        static_cast<const __half*>(z_draft), static_cast<const __half*>(z_target), ld, vocab, drafted,
        uniforms, gamma, margin, gate, accept, resid_mass, token);
  CUDA_TRY(cudaGetLastError());
  return COVSPEC_OK;
}

double covspec_uplink_bits(long long n_draft, int b_id, long long n_logit_draft, int b_logit) {
  return (double)n_draft * b_id + (double)n_logit_draft * b_logit;
}

double covspec_downlink_bits(int all_accepted, int b_acc, int b_bonus, int b_rej, long long vocab,
                             int b_logit_tar) {
  return all_accepted ? (double)b_acc + b_bonus : (double)b_rej + (double)vocab * b_logit_tar;
}

double covspec_comm_latency(double bits, double bandwidth_hz, double snr_db) {
  return bits / (bandwidth_hz * log2(1.0 + pow(10.0, snr_db / 10.0)));
}

double covspec_ema_update(double p_hat, double eta, int k, int n_acc) {
  if (n_acc < 0) n_acc = 0;
  if (n_acc > k) n_acc = k;
  for (int i = 0; i < n_acc; ++i) p_hat = (1.0 - eta) * p_hat + eta;
  for (int i = n_acc; i < k; ++i) p_hat = (1.0 - eta) * p_hat;
  return p_hat;
}

int covspec_draft_length(int k, double p_hat, double t_rej, double p_low, double p_up, double t_ref,
                         double s, int k_min, int k_max) {
  if (k < 1 || !(s > 1.0) || k_min > k_max || k_min < 1) return COVSPEC_ERR_ARG;
  int phi = 0;
  if (p_hat <= p_low) phi = -1;
  else if (p_hat >= p_up && t_rej <= t_ref) phi = 1;
  double x = phi < 0 ? (double)k / s : phi > 0 ? (double)k * s : (double)k;
  long long r = (long long)floor(x + 0.5);
  if (r > k_max) r = k_max;
  if (r < k_min) r = k_min;
  return (int)r;
}

int covspec_fanout(int f0, double rho, int j) {
  if (f0 < 0 || j < 0 || !(rho > 0.0 && rho < 1.0)) return COVSPEC_ERR_ARG;
  return (int)ceil((double)f0 * pow(rho, (double)j) - 1e-9);
}

int covspec_branch_candidates(int logit_dtype, int rows, int vocab, long long ld, const void* z_draft,
                              const int* drafted, const int* cand_offsets, int max_fanout, int* cand,
                              void* stream) {
  if (!z_draft || !cand_offsets || !cand) return COVSPEC_ERR_ARG;
  if (logit_dtype != COVSPEC_F32 && logit_dtype != COVSPEC_BF16 && logit_dtype != COVSPEC_F16)
    return COVSPEC_ERR_ARG;
  int esize = logit_dtype == COVSPEC_F32 ? 4 : 2;
  if (rows < 1 || vocab < 2 || ld < vocab || (ld * esize) % 16 != 0) return COVSPEC_ERR_SHAPE;
  if (max_fanout < 0 || max_fanout > vocab - 1) return COVSPEC_ERR_SHAPE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (logit_dtype == COVSPEC_F32)
    corr::branch_candidates_kernel<float><<<rows, 1024, 0, s>>>(static_cast<const float*>(z_draft), ld, vocab,
                                                                drafted, cand_offsets, cand);
  else if (logit_dtype == COVSPEC_BF16)
    corr::branch_candidates_kernel<__nv_bfloat16><<<rows, 1024, 0, s>>>(
        static_cast<const __nv_bfloat16*>(z_draft), ld, vocab, drafted, cand_offsets, cand);
  else
    corr::branch_candidates_kernel<__half><<<rows, 1024, 0, s>>>(static_cast<const __half*>(z_draft), ld, vocab,
                                                                 drafted, cand_offsets, cand);
  CUDA_TRY(cudaGetLastError());
  return COVSPEC_OK;
}

int covspec_selftest_wait_timeout(covspec_ctx* ctx, void* stream) {
  if (!ctx) return COVSPEC_ERR_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  tc::wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(ctx->status, 4096u);
  CUDA_TRY(cudaGetLastError());
  return COVSPEC_OK;
}

int covspec_last_launch_count(const covspec_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* covspec_strerror(int status) {
  switch (status) {
    case COVSPEC_OK: return "ok";
    case COVSPEC_ERR_ARG: return "invalid argument";
    case COVSPEC_ERR_SHAPE: return "invalid shape (offsets, empty request or budget)";
    case COVSPEC_ERR_UNSUPPORTED: return "unsupported configuration";
    case COVSPEC_ERR_WORKSPACE: return "problem exceeds the workspace capacities given at init";
    case COVSPEC_ERR_CUDA: return "CUDA runtime error";
    case COVSPEC_ERR_NONFINITE: return "non-finite score on the device";
    case COVSPEC_ERR_NOCONVERGE: return "small eigen-solve did not converge";
    case COVSPEC_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case COVSPEC_ERR_STATIC_CAPACITY:
      return "problem exceeds the fixed scratch capacity of the allocation-free entry point";
    case COVSPEC_ERR_BOUNDS: return "checked build: an index-driven access was out of range and skipped";
    default: return "unknown status";
  }
}

const char* covspec_last_cuda_error(void) { return g_cuda_error.c_str(); }

int covspec_selftest_fill_workspace(covspec_ctx* ctx, int byte, void* stream) {
  if (!ctx || byte < 0 || byte > 255) return COVSPEC_ERR_ARG;
  // everything behind the per-call plan, schedule and tables: scores, Gram planes, subspace blocks,
  // partial sums, factors, Ritz vectors, synchronisation words
  char* from = reinterpret_cast<char*>(ctx->Qn);
  CUDA_TRY(cudaMemsetAsync(from, byte, (size_t)(ctx->ws + ctx->ws_bytes - from), reinterpret_cast<cudaStream_t>(stream)));
  return COVSPEC_OK;
}

int covspec_build_has_bounds_checks(void) {
#ifdef COVSPEC_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

}  // extern "C"

// ================================================================================================
// Allocation-free query score.  The scratch the cosine kernel needs (the unit-length query
// elements and the per-request plan) lives in this fixed device array instead of a context
// workspace, so the entry point below never calls an allocator.
namespace {

constexpr int kStaticMaxBatch = COVSPEC_STATIC_MAX_BATCH;
constexpr long long kStaticMaxQueryElems = COVSPEC_STATIC_MAX_QUERY_ELEMS;
constexpr size_t kStaticPlanBytes = (sizeof(ReqPlan) * kStaticMaxBatch + 255) / 256 * 256;
constexpr size_t kStaticScratchBytes = kStaticPlanBytes + sizeof(float) * kStaticMaxQueryElems;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kStaticMaxDevices] = {nullptr};

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel can use; the address is looked up once per
// device, with that device current, and cached.
int static_scratch_ptr(unsigned char** out) {
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kStaticMaxDevices) return COVSPEC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_static_scratch));
    g_static_ptr[dev] = ptr;
  }
  *out = reinterpret_cast<unsigned char*>(g_static_ptr[dev]);
  return COVSPEC_OK;
}

// The per-request plan reaches the scratch array as kernel arguments (by value, 64 requests per
// launch), not through a host-to-device copy: nothing of the call keeps pointing at host memory
// after the call has returned.
struct StaticPlanChunk {
  int4 e[64];        // vis_off, n, txt_off, t
  int first, count;
};

__global__ void static_plan_kernel(ReqPlan* __restrict__ plan, const StaticPlanChunk chunk) {
  int i = threadIdx.x;
  if (i >= chunk.count) return;
  ReqPlan rp{};
  rp.vis_off = chunk.e[i].x; rp.n = chunk.e[i].y; rp.txt_off = chunk.e[i].z; rp.t = chunk.e[i].w;
  plan[chunk.first + i] = rp;
}

template <typename T>
int query_score_static_impl(int d, int batch, const int* vis_offsets, const int* txt_offsets,
                            const void* X, const void* Q, float* s_query, cudaStream_t s) {
  unsigned char* scratch = nullptr;
  int st = static_scratch_ptr(&scratch);
  if (st) return st;
  ReqPlan* d_plan = reinterpret_cast<ReqPlan*>(scratch);
  float* Qn = reinterpret_cast<float*>(scratch + kStaticPlanBytes);
  for (int b0 = 0; b0 < batch; b0 += 64) {
    StaticPlanChunk chunk{};
    chunk.first = b0; chunk.count = std::min(64, batch - b0);
    for (int i = 0; i < chunk.count; ++i) {
      int b = b0 + i;
      chunk.e[i] = make_int4(vis_offsets[b], vis_offsets[b + 1] - vis_offsets[b], txt_offsets[b],
                             txt_offsets[b + 1] - txt_offsets[b]);
    }
    static_plan_kernel<<<1, 64, 0, s>>>(d_plan, chunk);
    CUDA_TRY(cudaGetLastError());
  }
  long long rows_x = vis_offsets[batch];
  int rows_q = txt_offsets[batch];
  qnorm_kernel<T><<<(rows_q + 7) / 8, 256, 0, s>>>(reinterpret_cast<const T*>(Q), Qn, rows_q, 1, d);
  CUDA_TRY(cudaGetLastError());
  cosmax_kernel<T><<<(unsigned)((rows_x + 7) / 8), 256, 0, s>>>(
      reinterpret_cast<const T*>(X), Qn, d_plan, batch, 0, (int)rows_x, 1, d, 0, 0, s_query);
  CUDA_TRY(cudaGetLastError());
  return COVSPEC_OK;
}

}  // namespace

extern "C" int covspec_query_score_static(int dtype, int d, int batch, const void* X,
                                          const int* vis_offsets, const void* Q,
                                          const int* txt_offsets, float* s_query, void* stream) {
  if (!X || !Q || !vis_offsets || !txt_offsets || !s_query || batch < 1) return COVSPEC_ERR_ARG;
  if (dtype != COVSPEC_F32 && dtype != COVSPEC_BF16) return COVSPEC_ERR_ARG;
  if (d < 8 || d % 8) return COVSPEC_ERR_UNSUPPORTED;
  if (vis_offsets[0] != 0 || txt_offsets[0] != 0) return COVSPEC_ERR_SHAPE;
  if (batch > kStaticMaxBatch) return COVSPEC_ERR_STATIC_CAPACITY;
  for (int b = 0; b < batch; ++b)
    if (vis_offsets[b + 1] <= vis_offsets[b] || txt_offsets[b + 1] <= txt_offsets[b])
      return COVSPEC_ERR_SHAPE;
  if ((long long)txt_offsets[batch] * d > kStaticMaxQueryElems) return COVSPEC_ERR_STATIC_CAPACITY;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  return dtype == COVSPEC_BF16
             ? query_score_static_impl<__nv_bfloat16>(d, batch, vis_offsets, txt_offsets, X, Q, s_query, s)
             : query_score_static_impl<float>(d, batch, vis_offsets, txt_offsets, X, Q, s_query, s);
}
