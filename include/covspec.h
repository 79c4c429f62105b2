/* covspec.h - C ABI of the B200 (sm_100a) visual-token reduction library.
 *
 * The library computes CoVSpec's training-free visual token selection (Sec. III-A of the paper):
 * query-aware score (Eq. 10), token activity score (Eq. 11), normalise + fuse (Eq. 12), preselect
 * the M best tokens, energy of every preselected token in the top-r singular subspace of the
 * stacked matrix Z_M (Eq. 13-15), keep the B_vis tokens of largest energy, and gather the
 * survivors into a dense buffer (the reduced visual context V-hat that the draft model consumes).
 *
 * Conventions used by every entry point
 *  - "device" pointers are CUDA global-memory addresses on the current device; "host" pointers
 *    are ordinary process memory.  The library never takes ownership of a caller's buffer.
 *  - Matrices are dense row-major.  X, Q and every Hs[l] hold one token per row of `d` elements
 *    of `dtype`; requests are packed back to back and delimited by host offset arrays.
 *  - Wq / Wk are [n_heads*head_dim, d] row-major: one output feature of the embedding map e(.)
 *    per row (the layout of a linear layer's weight).  Head h owns rows [h*head_dim,(h+1)*head_dim).
 *  - Token indices written by the library are request-local (0 .. N_b-1) and ascending inside a
 *    request.
 *  - Every call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *    default stream) except for the small host->device copy of the launch plan, which is issued on
 *    the same stream from a pinned staging buffer owned by the context.
 *  - Return value: COVSPEC_OK or a negative covspec_status.  Argument, shape, capacity and
 *    unsupported-configuration errors are detected on the host before anything is launched.
 *    Conditions only the device can see (non-finite scores) are recorded in a device status word,
 *    read back by covspec_get_device_status(); outputs are then unspecified but in bounds.
 *  - One context serves one stream at a time; calls on one context must not overlap.
 *  - Results are deterministic: the same inputs on the same context give bit-identical outputs
 *    (the only floating-point atomic is a max, which does not depend on order; partial sums are
 *    combined in a fixed order).
 */
#ifndef COVSPEC_H_
#define COVSPEC_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct covspec_ctx covspec_ctx; /* opaque; owns the device workspace and the plan cache */

typedef enum { COVSPEC_F32 = 0, COVSPEC_BF16 = 1 } covspec_dtype;

typedef enum {
  COVSPEC_OK = 0,
  COVSPEC_ERR_ARG = -1,         /* NULL or inconsistent argument                              */
  COVSPEC_ERR_SHAPE = -2,       /* offsets not monotone, empty request, budget out of range   */
  COVSPEC_ERR_UNSUPPORTED = -3, /* configuration outside what the kernels implement           */
  COVSPEC_ERR_WORKSPACE = -4,   /* problem exceeds the capacities given at init               */
  COVSPEC_ERR_CUDA = -5,        /* a CUDA runtime call failed (see covspec_last_cuda_error)   */
  COVSPEC_ERR_NONFINITE = -6,   /* device status: a score was NaN or Inf                      */
  COVSPEC_ERR_NOCONVERGE = -7,  /* device status: the subspace iteration behind Eq. 14 had not
                                   settled within the tolerance after its last step, or the small
                                   eigen-solve hit its sweep limit                             */
  COVSPEC_ERR_TIMEOUT = -8,     /* device status: a bounded wait inside a kernel expired      */
  COVSPEC_ERR_STATIC_CAPACITY = -9, /* covspec_query_score_static: beyond its fixed scratch size */
  COVSPEC_ERR_BOUNDS = -10      /* device status, checked build only: an index was out of range  */
} covspec_status;

/* Static configuration.  Fill with covspec_default_config() and override. */
typedef struct {
  int dtype;           /* covspec_dtype of X, Q, Wq, Wk, Hs and of the compacted output           */
  int d;               /* feature width; must be a multiple of 8                                   */
  int n_heads;         /* 0 = identity embedding e(x)=x (Wq, Wk ignored); else head_dim must be 128 */
  int head_dim;
  int act_layers;      /* K of Eq. 11 (number of late-layer differences); 0 = no activity term     */
  float lambda;        /* lambda of Eq. 12                                                         */
  int norm_mode;       /* "normalize to the same scale": 0 min-max per request, 1 z-score, 2 none  */
  int head_reduce;     /* 0 max over (query element, head) pairs, 1 mean over heads then max       */
  float presel_factor; /* M = min(N, max(B_vis, ceil(presel_factor*B_vis)))                        */
  float rank_frac;     /* r = clamp(ceil(rank_frac*B_vis), 1, min(rank_cap, M-1, d-1))             */
  int rank_cap;
  int eig_iters;       /* Eq. 14 is reached by block subspace iteration on Z_M^T Z_M: eig_iters
                          orthonormalised power steps follow the first multiplication (>= 1)        */
  int eig_oversample;  /* extra basis vectors carried beyond r; rank_cap + eig_oversample <= 160    */
  int max_batch;                 /* capacities the workspace is sized for */
  long long max_total_vis;       /* sum of N_b */
  long long max_total_txt;       /* sum of T_b */
  int max_vis_per_req;           /* max N_b */
  int max_presel_per_req;        /* max M_b   (0: derive from max_vis_per_req) */
  long long max_total_presel;    /* sum of M_b (0: derive from max_total_vis)  */
  int relevance_path;  /* 0: Eq. 10 and the Gram matrix of Eq. 13 on the tensor cores (tcgen05) whenever
                          the configuration allows (128-wide heads, max over heads, d >= 64; float32
                          inputs are first split into three bf16 terms, about 2^-17 relative, which
                          takes workspace for 1.5 times the inputs), else the CUDA-core path;
                          1: always the CUDA-core path; 2: the two-SM form of the tensor-core kernel
                          (tcgen05.mma.cta_group::2 on pairs of token tiles; measured no faster than
                          the one-SM form, kept selectable); other values: COVSPEC_ERR_ARG         */
  int lowrank_mode;    /* 0: energy in the top-r singular subspace (Eq. 14-15, the paper's criterion);
                          1: greedy pivoted selection (not in the paper): pick B_vis times the token with
                             the largest residual energy after projecting out the picked ones; needs
                             M <= 16384 and B_vis <= 8192 per request                              */
  int ritz_window;     /* basis vectors above the cut at r that take part in the final Rayleigh-Ritz
                          step together with the eig_oversample ones below it (default 16; >= p: all) */
  int activity_overlap; /* > 0: while Eq. 10 runs on the tensor cores (which leaves HBM idle), Eq. 11
                          streams the snapshot stack on a second stream of the context with this many
                          512-thread blocks per SM (1 or 2; default 1), joined before Eq. 12; 0: the two
                          scores are computed one after the other on the caller's stream           */
  float conv_tol;      /* the subspace iteration behind Eq. 14 runs a fixed number of steps; after the
                          last one the library estimates, from the Ritz values, how far the energies
                          can still be from those of the exact truncated SVD (relative to the largest
                          energy) and raises COVSPEC_ERR_NOCONVERGE in the device status word when the
                          estimate exceeds conv_tol (default 2e-3; 0 disables the check).  More steps
                          (eig_iters) or more extra vectors (eig_oversample) settle such inputs      */
  int eig_early_stop;  /* 1 (default): a request whose estimate, predicted for the next step from the Ritz
                          value estimates of the running iteration, is below conv_tol / 8 (conv_tol / 64
                          after the second multiplication) makes that step its last instead of running
                          all eig_iters steps; 0: always eig_iters steps                              */
} covspec_config;

/* One batch of requests (Sec. III-A notation in brackets). */
typedef struct {
  int batch;
  const void* X;            /* device [vis_offsets[batch], d]  visual tokens v_i = z_i            */
  const int* vis_offsets;   /* host   [batch+1] first row of each request in X, vis_offsets[0]=0   */
  const void* Q;            /* device [txt_offsets[batch], d]  query elements q_j                  */
  const int* txt_offsets;   /* host   [batch+1]                                                    */
  const void* Wq;           /* device [n_heads*head_dim, d] or NULL when n_heads == 0              */
  const void* Wk;           /* device [n_heads*head_dim, d] or NULL when n_heads == 0              */
  const void* const* Hs;    /* host array of act_layers+1 device pointers h^(L-K) .. h^(L), each
                               laid out like X; NULL when act_layers == 0                          */
  const int* keep;          /* host [batch] B_vis per request, or NULL to use keep_ratio           */
  double keep_ratio;        /* B_vis = max(1, ceil(keep_ratio*N_b - 1e-6)), evaluated in double      */
} covspec_problem;

/* Defaults: lambda 0.5, min-max, head max, presel_factor 2, rank_frac 0.5, rank_cap 128,
 * eig_iters 5, eig_oversample 16, act_layers 4; capacities zero (the caller must set them). */
void covspec_default_config(covspec_config* cfg);

/* Host-only integer logic of the budgets (paper: r < min(M,d), B_vis < M <= N).  `keep` is the
 * requested B_vis (clamped to n).  Writes B_vis, M, r.  Returns COVSPEC_OK or COVSPEC_ERR_ARG. */
int covspec_budgets(const covspec_config* cfg, int n, int keep, int* b_vis, int* m, int* r);

/* Budgets of a whole problem: keep_offsets[batch+1] and presel_offsets[batch+1] (host, either may
 * be NULL) receive the prefix sums of B_vis and M.  Launches nothing. */
int covspec_plan_sizes(const covspec_config* cfg, const covspec_problem* p, int* keep_offsets,
                       int* presel_offsets);

/* Allocates the context and its device workspace for the capacities in cfg (the only allocation
 * the library makes).  *out is NULL on failure.  Must be called with the target device current. */
int covspec_prune_init(const covspec_config* cfg, covspec_ctx** out);
int covspec_prune_destroy(covspec_ctx* ctx);
/* Bytes of device workspace held by the context. */
long long covspec_workspace_bytes(const covspec_ctx* ctx);

/* Eq. 10-12.  Writes float32 device arrays of vis_offsets[batch] elements: s_query (Eq. 10),
 * s_act (Eq. 11), s_fused (Eq. 12).  s_query and s_act may be NULL (kept in the workspace);
 * s_fused is required. */
int covspec_score(covspec_ctx* ctx, const covspec_problem* p, float* s_query, float* s_act,
                  float* s_fused, void* stream);

/* Preselection and low-rank redundancy reduction (Eq. 13-15) from a fused score.
 *  s_fused       device [sum N_b] float32, as written by covspec_score
 *  keep_idx      device [sum B_vis] int32: kept token indices, request-local, ascending
 *  keep_offsets  host   [batch+1] (out, may be NULL): prefix sums of B_vis
 *  presel_idx    device [sum M_b] int32 (out, may be NULL): the M preselected tokens, ascending
 *  energy        device [sum M_b] float32 (out, may be NULL): c_i of Eq. 15 in presel order;
 *                requests whose stage 2 is skipped (B_vis >= M) get zeros
 * Ties in either selection: larger value first, then lower token index. */
int covspec_select(covspec_ctx* ctx, const covspec_problem* p, const float* s_fused, int* keep_idx,
                   int* keep_offsets, int* presel_idx, float* energy, void* stream);

/* Gather of the survivors: out_hidden[keep_offsets[b] + k, :] = X[vis_offsets[b] + keep_idx[..], :]
 * (bit copies, dtype of X), out_pos (device int32, may be NULL) = the same request-local indices.
 * keep_offsets is the host array returned by covspec_select / covspec_plan_sizes. */
int covspec_compact(covspec_ctx* ctx, const covspec_problem* p, const int* keep_idx,
                    const int* keep_offsets, void* out_hidden, int* out_pos, void* stream);

/* The same gather for any other per-token tensor that must follow the kept tokens (the K or V rows of
 * a layer when the pruning is applied after a prefill, position ids, ...): src is laid out like X,
 * one row of row_bytes (a multiple of 16; both bases 16-byte aligned) per visual token;
 * out[keep_offsets[b] + k, :] = src[vis_offsets[b] + keep_idx[..], :], bit copies.  The paper selects
 * before the draft prefill, so its own pipeline has only the hidden states to compact. */
int covspec_compact_rows(covspec_ctx* ctx, const covspec_problem* p, const int* keep_idx,
                         const int* keep_offsets, const void* src, long long row_bytes, void* out,
                         void* stream);

/* The whole path, Eq. 10 through the compacted buffer, in one call.  out_hidden device
 * [sum B_vis, d]; keep_idx device [sum B_vis]; keep_offsets host [batch+1] (may be NULL).
 * The call only enqueues work: on `stream` and on a second stream of the context that forks from it
 * and joins it again; it never waits for the device.  The plan of a batch shape (offsets, budgets)
 * is uploaded by the first call that sees it; later calls with the same offsets copy nothing from
 * the host, so they may be recorded by stream capture and replayed as a CUDA graph (the graph keeps
 * the device pointers of `p` and of the outputs; new contents in the same buffers are fine). */
int covspec_prune(covspec_ctx* ctx, const covspec_problem* p, void* out_hidden, int* keep_idx,
                  int* keep_offsets, void* stream);

/* Synchronises `stream`, returns the device status word (COVSPEC_OK, COVSPEC_ERR_BOUNDS, COVSPEC_ERR_TIMEOUT,
 * COVSPEC_ERR_NONFINITE or COVSPEC_ERR_NOCONVERGE) and clears it. */
int covspec_get_device_status(covspec_ctx* ctx, void* stream);

/* Diagnostics of the subspace iteration behind Eq. 14 for the last covspec_select / covspec_prune call
 * on this context: multiplications[b] (host, [batch]) receives the number of multiplications by the
 * Gram matrix that request b ran (eig_iters + 1 unless it stopped early, see eig_early_stop; 0 for a
 * request that skipped stage 2).  Synchronises `stream`. */
int covspec_get_iteration_counts(covspec_ctx* ctx, int batch, int* multiplications, void* stream);

/* Device-side gating and correction over the vocabulary (Sec. III-B.1 and III-C.2), one call for
 * `rows` decoding positions; needs no context and no workspace.
 *  logit_dtype   COVSPEC_F32, COVSPEC_BF16 or COVSPEC_F16 (the paper sends logits as float16)
 *  z_draft       device [rows, ld] draft logits z_d (Eq. 1); ld >= vocab, ld * element size a
 *                multiple of 16 bytes, base 16-byte aligned
 *  z_target      device [rows, ld] target logits z_t of the position (Eq. 3)
 *  drafted       device [rows] int32 drafted token ids in [0, vocab) or NULL
 *  uniforms      device [rows] float32 in [0, 1): the random numbers of the correction draw
 *  gamma         margin threshold of Eq. 17
 *  margin        device [rows] float32 (out): p_(1) - p_(2) of softmax(z_d)         (Eq. 2, 16)
 *  gate          device [rows] int32   (out): 1 if margin < gamma else 0               (Eq. 17)
 *  accept        device [rows] float32 (out, may be NULL): min(1, p_t(y)/p_d(y))        (Eq. 4, 5);
 *                1 when drafted is NULL
 *  resid_mass    device [rows] float32 (out, may be NULL): sum_w max(p_t(w) - p_d(w), 0)
 *  token         device [rows] int32   (out): the first token whose cumulative residual
 *                probability (Eq. 6, vocabulary order) exceeds uniforms[row]; drawn from p_t when
 *                the residual is identically zero
 * Returns COVSPEC_ERR_ARG / COVSPEC_ERR_SHAPE / COVSPEC_ERR_CUDA on the host before launching. */
#define COVSPEC_F16 2
int covspec_correct(int logit_dtype, int rows, int vocab, long long ld, const void* z_draft,
                    const void* z_target, const int* drafted, const float* uniforms, float gamma,
                    float* margin, int* gate, float* accept, float* resid_mass, int* token,
                    void* stream);

/* Fan-out of the parallel branching, Eq. 23: F_j = ceil(F_0 * rho^j), 0 < rho < 1, evaluated in
 * double (a product within 1e-9 of an integer counts as that integer).  Host only. */
int covspec_fanout(int f0, double rho, int j);

/* Bonus-token candidates (Sec. III-C.1): for every position the F_j largest draft logits, excluding
 * the token drafted at that position; ties go to the lower token id.  No context, no workspace.
 *  z_draft       device [rows, ld], layout and alignment as in covspec_correct
 *  drafted       device [rows] int32 drafted token ids, or NULL (nothing excluded)
 *  cand_offsets  device [rows+1] int32 prefix sums of the fan-outs F_j (built by the caller)
 *  max_fanout    largest F_j (host); must be <= vocab - 1
 *  cand          device [cand_offsets[rows]] int32 (out): candidate token ids, ascending per position */
int covspec_branch_candidates(int logit_dtype, int rows, int vocab, long long ld, const void* z_draft,
                              const int* drafted, const int* cand_offsets, int max_fanout, int* cand,
                              void* stream);

/* Scalar host-side formulas of the link model and the draft-length controller.  No device work.
 *  covspec_uplink_bits       Eq. 7: N_draft * b_id + N_logit_draft * b_logit
 *  covspec_downlink_bits     Eq. 8: b_acc + b_bonus if all drafted tokens were accepted, else
 *                            b_rej + vocab * b_logit_tar
 *  covspec_comm_latency      Eq. 9 / 19: bits / (B log2(1 + 10^(SNR/10))), B in Hz, result in s
 *  covspec_ema_update        Eq. 18: n_acc updates with a = 1, then k - n_acc updates with a = 0
 *  covspec_draft_length      Eq. 20-22: phi from (p_hat, T_rej), k <- clip(round(k s^phi), k_min, k_max),
 *                            halves rounded away from zero; returns the new k (negative status on
 *                            invalid arguments: s <= 1, k_min > k_max, k < 1) */
double covspec_uplink_bits(long long n_draft, int b_id, long long n_logit_draft, int b_logit);
double covspec_downlink_bits(int all_accepted, int b_acc, int b_bonus, int b_rej, long long vocab,
                             int b_logit_tar);
double covspec_comm_latency(double bits, double bandwidth_hz, double snr_db);
double covspec_ema_update(double p_hat, double eta, int k, int n_acc);
int covspec_draft_length(int k, double p_hat, double t_rej, double p_low, double p_up, double t_ref,
                         double s, int k_min, int k_max);

/* Self-test of the kernels' bounded waits (no step of the paper).  Every wait inside the
 * tensor-core kernels gives up after a fixed number of polls, raises COVSPEC_ERR_TIMEOUT in the
 * device status word and lets the kernel return, so that a protocol fault cannot hang the GPU.
 * This call launches one thread that waits, with the same routine and a small limit, on a barrier
 * nothing signals; afterwards covspec_get_device_status() reports COVSPEC_ERR_TIMEOUT (and clears
 * it).  Asynchronous on `stream`; takes well under a millisecond. */
int covspec_selftest_wait_timeout(covspec_ctx* ctx, void* stream);

/* Optional per-stage timing of covspec_prune with CUDA events recorded on the call's stream.
 * covspec_profile_begin reserves events for up to max_calls prune calls; covspec_profile_end
 * waits for them, writes the summed milliseconds of each stage into stage_ms[n_stages] (stage
 * names from covspec_profile_stage_name, count from covspec_profile_stage_count), the number of
 * profiled calls into *calls, and releases the events. */
int covspec_profile_begin(covspec_ctx* ctx, int max_calls);
int covspec_profile_end(covspec_ctx* ctx, double* stage_ms, int n_stages, int* calls);
int covspec_profile_stage_count(void);
const char* covspec_profile_stage_name(int stage);

/* Allocation-free variant of the query-aware score.  (The paper has no counterpart of this entry
 * point: it computes Eq. 10 exactly as covspec_score does with the identity embedding, but is
 * packaged for callers that cannot allocate.)
 *
 * Who needs it: code that runs where device allocation is off limits - inside a serving loop whose
 * memory pool is fully handed out at start-up, in a process whose allocator is owned by another
 * framework and must not see foreign cudaMalloc calls, or in a latency path where an allocation's
 * implicit device synchronisation is unacceptable.  Such callers cannot create a covspec_ctx
 * (covspec_prune_init allocates the workspace).  This entry point needs no context: its scratch
 * (the unit-length query elements and the per-request plan) lives in a fixed device array inside
 * the library, which every GPU that loads the library holds until the process exits.  The call
 * issues no cudaMalloc, cudaFree or other allocating routine.
 *
 *  dtype, d      as in covspec_config (d a multiple of 8); identity embedding, max over elements
 *  X, Q          device, laid out as in covspec_problem; vis_offsets, txt_offsets host [batch+1]
 *  s_query       device [vis_offsets[batch]] float32 (out): Eq. 10 per visual token
 * Limits: batch <= COVSPEC_STATIC_MAX_BATCH and txt_offsets[batch] * d <=
 * COVSPEC_STATIC_MAX_QUERY_ELEMS; larger problems are rejected with COVSPEC_ERR_STATIC_CAPACITY
 * and nothing is launched.
 * The first call on a device looks up the scratch array's device address (once per device, with
 * that device current) and should therefore be made before any stream capture begins.
 * Every call on a device shares the one scratch array and leaves its contents behind.  Nothing in
 * it has to start at zero (each call rewrites the part it reads), but two calls that overlap on
 * the GPU - different streams, or different host threads - race on it: serialise them. */
#define COVSPEC_STATIC_MAX_BATCH 256
#define COVSPEC_STATIC_MAX_QUERY_ELEMS (1 << 20)   /* 4 MiB of float32 scratch */
int covspec_query_score_static(int dtype, int d, int batch, const void* X, const int* vis_offsets,
                               const void* Q, const int* txt_offsets, float* s_query, void* stream);

/* Number of kernels the last call on this context launched. */
int covspec_last_launch_count(const covspec_ctx* ctx);

/* Test aid: fills the context's scratch (scores, Gram planes, subspace blocks, partial sums, factors,
 * Ritz vectors, synchronisation words; not the per-call plan) with `byte` (0..255) on `stream`.  The
 * next call must give the same results whatever the byte (0xFF makes every float and bf16 a NaN):
 * every kernel has to write what it later reads.  Returns COVSPEC_OK, COVSPEC_ERR_ARG or
 * COVSPEC_ERR_CUDA. */
int covspec_selftest_fill_workspace(covspec_ctx* ctx, int byte, void* stream);

/* 1 when the library was built with -DCOVSPEC_DEBUG_BOUNDS (libcovspec_debug.so): the kernels whose
 * global accesses are driven by computed indices (row gathers of Eq. 13 and of the compaction, the
 * ordered emission of the top-k selections) test every such index, raise COVSPEC_ERR_BOUNDS in the
 * device status word and skip the access instead of making it.  0 for the ordinary build, whose
 * kernels carry no such tests.  Host-only, no arguments, cannot fail. */
int covspec_build_has_bounds_checks(void);

/* Text of a covspec_status; for COVSPEC_ERR_CUDA, covspec_last_cuda_error gives the runtime's. */
const char* covspec_strerror(int status);
const char* covspec_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* COVSPEC_H_ */
