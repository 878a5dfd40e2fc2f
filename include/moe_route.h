/*
 * moe_route.h -- C ABI of the B200 (sm_100a) MoE routing and load-control
 * library for ID Balancing (arXiv 2609.39137).
 *
 * One context routes the tokens of L independent router layers per step and
 * runs one bias-controller step for all of them:
 *
 *   logits z = W_r x                         Section 2.2
 *   score  s = sigmoid(z)                    Section 2.2 / Section 4.3
 *   select T(x) = TopK_i (s_i + b_i)         Eq. 2
 *   gates  w_k = s_k / sum_{j in T(x)} s_j   sentence after Eq. 2 (no bias)
 *   loads  n_i += #tokens assigned to i      Algorithm 1 line 4
 *   error  e_i = (nbar - n_i) / nbar         Eq. 3, Algorithm 1 lines 5-7
 *   bias   ID update + centring              Algorithm 1 lines 8-13, Eq. 9-12
 *          fixed-step integral (DeepSeek)    Eq. 5
 *          quantile target (proportional)    Eq. 6-7, EMA variant Section 3
 *   MaxVio / MinVio                          Eq. 13
 *
 * Conventions
 *   - Every tensor pointer is DEVICE memory owned by the caller unless the
 *     parameter name ends in `_host`.  The library allocates no device memory:
 *     its state lives in the caller-provided workspace.  Pointers are borrowed
 *     only for the duration of the enqueued work.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = default stream) and is asynchronous unless stated otherwise.
 *   - Every call returns a MOE_* status; 0 is success.  Argument errors are
 *     found on the host before anything is launched.  Nothing throws, aborts
 *     or prints.  Device-side problems (a bounded wait that expired) are
 *     sticky in the workspace and reported by moe_route_poll.
 *   - A context is thread-compatible: one thread at a time per context.
 *   - Layouts are row-major with the last index fastest:
 *       x        [L][T][H]  bf16        hidden states, T = num_tokens
 *       w        [L][E][H]  bf16        router weights W_r (one row per expert)
 *       topk_idx [L][T][K]  int32       selected experts, by descending biased
 *                                        score, equal scores by ascending index
 *       topk_gate[L][T][K]  float32     combination weights in the same order
 *       logits   [L][T][E]  float32     optional dump of z
 *       alpha    [L][T]     float32     optional (K+1)-th largest biased score
 *       loads    [L][E]     int32
 *       bias, e_prev [L][E] float32
 */
#ifndef MOE_ROUTE_H_
#define MOE_ROUTE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_route_ctx moe_route_ctx; /* opaque, host memory, library-owned */

enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1,
  MOE_ERR_UNSUPPORTED = 2,
  MOE_ERR_CUDA = 3,
  MOE_ERR_STATE = 4,      /* e.g. controller update with no tokens routed */
  MOE_ERR_WORKSPACE = 5,  /* workspace too small or misaligned */
  MOE_ERR_TIMEOUT = 6,    /* a bounded device-side wait expired */
  MOE_ERR_INTERNAL = 7    /* builds with -DMOE_DEBUG only: an index guard inside a kernel tripped (the access
                             was skipped) or a canary between two workspace sections was overwritten */
};

enum {
  MOE_CTRL_ID = 0,         /* Algorithm 1 */
  MOE_CTRL_FIXED_STEP = 1, /* Eq. 5 */
  MOE_CTRL_QUANTILE = 2,   /* Eq. 6-7 */
  MOE_CTRL_FROZEN = 3      /* bias never changes (continued pretraining /
                              inference, Section 4.1); loads and metrics only */
};

typedef struct {
  int32_t struct_size;  /* = sizeof(moe_route_config) */
  int32_t num_layers;   /* L >= 1 */
  int32_t num_experts;  /* E, multiple of 8, K < E <= 1024 (768 is the tuned case) */
  int32_t top_k;        /* K in 1..16 */
  int32_t hidden;       /* H, multiple of 8 */
  int32_t max_tokens;   /* upper bound on num_tokens per call */
  int32_t controller;   /* MOE_CTRL_* */
  float ki, kd;         /* ID gains; paper default 6e-3 each (Section 4) */
  float eta;            /* fixed-step size; paper default 1e-3 (Section 4.1) */
  float qb_ema_rho;     /* 0 <= rho < 1; 0 = plain Quantile Balancing */
  int32_t center;       /* zero-mean centring after the update: 1 on, 0 off,
                           -1 = per-controller default (ID on, others off) */
  int32_t spin_limit;   /* iteration bound of every device-side wait; 0 = default */
  int32_t host_staging; /* 1 = reserve workspace for moe_route_step_host */
  int32_t w_layout;     /* layout of the router weights handed to the step calls:
                           0 = [L][E][H] (W_r in R^{E x d} as Section 2.2 writes it, hidden contiguous),
                           1 = [L][H][E] (expert contiguous); the library then transposes into
                           L*E*H*2 bytes of workspace before every routing launch */
  int32_t chunk_split;  /* scheduling of the 256-expert chunks of a token tile (E > 256 only; results are
                           identical either way): 1 = one CTA pair walks all chunks of its tile and finishes the
                           rows in its epilogue; 2 = the chunks of a tile go to different CTA pairs that run at
                           the same time (the tile is streamed from HBM once) and a merge kernel finishes the
                           rows from L*ceil(E/256)*max_tokens*(K+1)*8 bytes of workspace; 0 = chosen by the
                           library: 2 when the tiles of all resident pairs no longer fit in L2 (hidden > 3072)
                           or when L*ceil(max_tokens/256)*ceil(E/256) <= 64, i.e. every (tile, chunk) gets a
                           CTA pair of its own; else 1 */
  int32_t qb_hist_bins; /* MOE_CTRL_QUANTILE only.  0 = exact quantile of Eq. 7 (radix select over the dump).
                           B > 0 (multiple of 32, 32..2048) = the estimate the footnote to Eq. 7 mentions for use
                           at scale, from a per-expert margin histogram -- the paper fixes neither bins nor
                           rule, this library uses B uniform bins over [-qb_hist_range, qb_hist_range) (margins
                           outside count in the end bins), the same rank r = m - floor(mK/E), and linear
                           interpolation inside the bin that holds the r-th smallest margin:
                           estimate = -range + (k + ((r - below) - 0.5) / count_k) * (2 range / B).
                           |estimate - exact| < 2 range / B while the exact value is inside the range. */
  float qb_hist_range;  /* > 0; default 1.  The margins of an expert are centred at minus the common part of the
                           bias: an uncentred Quantile Balancing bias drifts as a whole, so choose centre = 1 or a
                           range that covers the drift, or every margin ends up in an end bin */
} moe_route_config;

/* Fills *cfg with the paper's defaults (Ki = Kd = 6e-3, eta = 1e-3, rho = 0,
 * centre = -1, ID controller) for the given shape. */
void moe_route_default_config(moe_route_config* cfg, int32_t num_layers, int32_t num_experts,
                              int32_t top_k, int32_t hidden, int32_t max_tokens);

/* Bytes of device workspace a context with this config needs (0 on a bad
 * config).  The caller allocates it (256-byte aligned) and keeps it alive
 * until moe_route_destroy. */
size_t moe_route_workspace_bytes(const moe_route_config* cfg);

/* Creates a context on the current CUDA device.  Clears the workspace (bias,
 * previous error, load accumulators = 0: Algorithm 1 line 1).  Synchronous. */
int moe_route_init(const moe_route_config* cfg, void* dev_workspace, size_t workspace_bytes,
                   moe_route_ctx** out);

/* Routes num_tokens tokens in each of the L layers with the current bias held
 * fixed (Algorithm 1 line 3) and ADDS the selections to the per-expert load
 * accumulators (line 4) -- several calls before a controller update are the
 * microbatch case.  logits_out and alpha_out may be NULL.  With
 * MOE_CTRL_QUANTILE both must be given; they are read again by
 * the next moe_controller_update and must stay valid until then.
 * Alignment: x and w 16 bytes (TMA), logits_out 16 bytes (written with vector
 * stores), topk_idx / topk_gate / alpha_out 4 bytes; anything else returns
 * MOE_ERR_INVALID_ARG before a kernel is launched.
 * w_bf16 is [L][E][H], or [L][H][E] for contexts made with w_layout = 1.
 * Ordering: the kernels are enqueued on cuda_stream and may begin (set-up only)
 * while the work queued before them is still running; they wait for that work
 * before they read x, W_r, the bias or the accumulators, so x and W_r may be
 * produced by the kernel queued just before this call. */
int moe_route_step(moe_route_ctx* ctx, const void* x_bf16, const void* w_bf16, int32_t num_tokens,
                   int32_t* topk_idx, float* topk_gate, float* logits_out, float* alpha_out,
                   void* cuda_stream);

/* Same step with HOST buffers (pinned memory recommended): copies x (and w if
 * w_bf16_host is not NULL; otherwise the weights of the previous call are
 * reused) to the staging area of the workspace, routes, copies indices and
 * gates back.  Needs host_staging = 1.  Asynchronous on the stream. */
int moe_route_step_host(moe_route_ctx* ctx, const void* x_bf16_host, const void* w_bf16_host,
                        int32_t num_tokens, int32_t* topk_idx_host, float* topk_gate_host,
                        void* cuda_stream);

/* One controller step for all layers (Algorithm 1 lines 5-13, or Eq. 5, or
 * Eq. 6-7): consumes the load accumulators, updates bias and previous error,
 * stores loads / MaxVio / MinVio of the consumed step, zeroes the
 * accumulators.  A layer whose accumulators sum to zero is left unchanged and
 * the call reports MOE_ERR_STATE through moe_route_poll. */
int moe_controller_update(moe_route_ctx* ctx, void* cuda_stream);

/* Copies out the loads and MaxVio/MinVio (Eq. 13) of the most recently
 * consumed step and the current bias.  Any pointer may be NULL. */
int moe_load_stats(moe_route_ctx* ctx, int32_t* loads, float* bias, float* maxvio, float* minvio,
                   void* cuda_stream);

/* Number of open derivative gates (g_i = 1, Eq. 11) per layer in the most
 * recent ID update: gate_count [L] int32. */
int moe_gate_stats(moe_route_ctx* ctx, int32_t* gate_count, void* cuda_stream);

/* Diagnostics of the most recent controller update, as plotted in the paper
 * (figure captions of Section 3; Section 4.3): diag [L][4] float32 (device) =
 * { fraction of open worsening gates (Eq. 11), share of all token assignments
 * that went to the busiest 10 % of the experts (round(E/10) experts; 0.10 when
 * balanced), fraction of experts that received no token, mean |bias change| of
 * the update }. */
int moe_load_diagnostics(moe_route_ctx* ctx, float* diag, void* cuda_stream);

/* Mean over the tokens of a routing step of the top-K gating-score entropy
 * H = -sum_k w_k ln w_k (nats, Section 4.3), per layer: topk_gate
 * [L][num_tokens][K] as written by moe_route_step, entropy [L] float32 (device). */
int moe_gate_entropy(moe_route_ctx* ctx, const float* topk_gate, int32_t num_tokens, float* entropy,
                     void* cuda_stream);

/* Statistics of the router's score distribution over a dumped logit matrix
 * (`logits` [L][num_tokens][E] fp32 device, as written by moe_route_step's
 * logits_out), one value per layer, means over the num_tokens tokens:
 *   entropy_biased  [L]  full-pool selection-score entropy (Section 4.3) of the
 *                        bias-controlled score family: p_e = max(sigmoid(z_e) + b_e, 0)
 *                        normalised over the E experts, H = -sum_e p_e ln p_e in nats
 *                        (b = the context's CURRENT bias: call before the controller
 *                        update to get the bias the step was routed with; a token whose
 *                        clamped scores are all zero counts H = 0);
 *   entropy_softmax [L]  the same entropy for p = softmax(z), the auxiliary-loss family;
 *   mean_prob    [L][E]  P_i of Eq. 8: mean softmax probability of expert i;
 *   aux             [L]  sum_i f_i P_i of Eq. 8 with f_i = loads[l][i] / num_tokens (the
 *                        coefficient alpha is left to the caller); needs `loads`
 *                        ([L][E] int32 device, the counts of the SAME tokens, e.g. from
 *                        moe_loads_peek after a single routing step).
 * Every output pointer may be NULL (that quantity is skipped); all are device memory.
 * fp32 arithmetic per token; each warp adds its tokens' values in fp32 (a few
 * hundred to a thousand rows per warp), the per-CTA partial sums are then added
 * in a fixed order in binary64: results are deterministic and agree with the
 * binary64 definition to about 1e-5 relative.
 * Forward statistics only: the gradient side of the auxiliary loss is a training-loop
 * matter.  Errors: MOE_ERR_INVALID_ARG (null logits, logits not
 * 16-byte aligned, num_tokens < 1, aux without loads). */
int moe_score_stats(moe_route_ctx* ctx, const float* logits, int32_t num_tokens, const int32_t* loads,
                    float* entropy_biased, float* entropy_softmax, float* mean_prob, float* aux, void* cuda_stream);

/* Load accumulators not yet consumed: read them, or add external counts.
 * Algorithm 1 line 4 takes n_i over every microbatch and every data-parallel
 * rank of the iteration: a caller that shards tokens across GPUs brings the
 * other ranks' counts in before the controller update. */
int moe_loads_peek(moe_route_ctx* ctx, int32_t* loads, void* cuda_stream);
int moe_loads_add(moe_route_ctx* ctx, const int32_t* loads, void* cuda_stream);

/* Device address of the accumulators themselves ([L][E] int32, inside the
 * workspace), for a caller that sums them over its data-parallel group IN PLACE
 * (one all-reduce(SUM) on this buffer between the last moe_route_step and
 * moe_controller_update, on the same stream, replaces peek + exchange + add).
 * The address stays valid for the life of the context.  Host call, nothing is
 * enqueued. */
int moe_loads_buffer(moe_route_ctx* ctx, int32_t** dev_loads);

/* Controller state of Algorithm 1 for checkpoint / resume: b and e_prev
 * ([L][E] float32, device, either may be NULL) and the number of controller
 * updates this context has enqueued so far (`step_host`, HOST memory, may be
 * NULL; written before the call returns).  Import restores what is given;
 * step = -1 keeps the context's own counter. */
int moe_state_export(moe_route_ctx* ctx, float* bias, float* e_prev, int64_t* step_host, void* cuda_stream);
int moe_state_import(moe_route_ctx* ctx, const float* bias, const float* e_prev, int64_t step, void* cuda_stream);

/* Synchronises the stream of the last call and returns the sticky device
 * status (MOE_OK, MOE_ERR_TIMEOUT, MOE_ERR_STATE, MOE_ERR_CUDA); clears it.
 * After MOE_ERR_TIMEOUT the routing step that gave up is void: its index and
 * gate outputs are incomplete, and this call has cleared the load accumulators
 * (including earlier microbatches of the same iteration), so the next
 * controller update cannot consume a partial histogram.  Bias and previous
 * error are untouched; route the iteration again or skip it. */
int moe_route_poll(moe_route_ctx* ctx);

/* Validation utility for the candidate filter of moe_route_step: sweeps every
 * finite fp32 logit and writes to dev_result[0] (device, one float) the largest
 * absolute difference between the approximate score used for filtering and the
 * exact score of Section 2.2.  The filter is sound while this stays below half
 * of the slack compiled into the kernel (1e-5). */
int moe_debug_score_gap(float* dev_result, void* cuda_stream);

/* Validation utility for the reciprocal inside the score chain (Section 2.2: the
 * score ends in a correctly rounded reciprocal).  The kernels compute it as the
 * hardware approximation plus one Newton step with an exact residual instead of
 * the math library's routine.  Sweeps all 2^32 fp32 bit patterns and writes two
 * counters to dev_result (device, two uint32): [0] logits whose score differs in
 * any bit between the two reciprocals, [1] normal numbers d with |d| in
 * [2^-126, 2^126] whose reciprocal differs.  Both must be 0. */
int moe_debug_rcp_check(uint32_t* dev_result, void* cuda_stream);

/* Validation utility for the gate division (Eq. 3: g = s / sum of the selected
 * s, correctly rounded).  The kernels divide by multiplying with the correctly
 * rounded reciprocal of the denominator and correcting twice with exact
 * residuals.  Compares that with the math library's correctly rounded division
 * for every fp32 denominator in [2^-20, 32] with 48 numerators each (about 1e10
 * pairs) and writes the number of differing pairs to dev_result[0] (device, one
 * uint32).  Must be 0. */
int moe_debug_division_check(uint32_t* dev_result, void* cuda_stream);

/* The same sweep for the quick score (hardware exponential and reciprocal
 * approximations) with which the margin-histogram pass of the quantile
 * controller bins a logit before deciding whether the exact score is needed:
 * dev_result[0] = largest |quick - exact| over every finite fp32 logit.  The
 * pass is exact while this stays below the gap compiled into it (3e-7). */
int moe_debug_quick_score_gap(float* dev_result, void* cuda_stream);

/* Quantile target without any allocation and without a context (the paper has
 * no counterpart for this call; it computes the same Q_j as the quantile
 * controller's update does from its dump).
 *
 * Meant for callers that cannot obtain device memory when they need this
 * result and have no workspace of their own to lend: for instance a serving
 * process that handed all of its device memory to its own pool at start-up, or
 * a latency-critical loop in which the implicit synchronisation and the
 * possible failure of cudaMalloc are not acceptable.  The radix-select scratch
 * (a histogram of 256 bins per expert plus two words per expert) therefore
 * lives in a fixed array inside the library: 1,056,768 bytes, present on every
 * device that loads the library until the process exits.  That caps the call at
 * num_experts <= 1024; more returns MOE_ERR_WORKSPACE and launches nothing.
 * num_tokens is not limited.
 *
 *   logits     [num_tokens][num_experts] float32, device (a dump of moe_route_step)
 *   alpha      [num_tokens] float32, device ((K+1)-th largest biased score per token)
 *   target_out [num_experts] float32, device: Q_j = -(r-th smallest of
 *              sigmoid(logits[i][j]) - alpha[i] over i), r = m - floor(m K / E)
 *
 * The first call on a device looks up the device address of the array and the
 * SM count (nothing is allocated); make that first call with the device current
 * and before any stream capture starts.  Later calls only launch kernels.
 * All calls share the one array and it keeps what the previous call left, so
 * every call first clears what must start at zero -- and two calls whose kernels
 * can overlap on the GPU (different streams, no ordering between them) race on
 * it.  Asynchronous on the stream; returns MOE_OK, MOE_ERR_INVALID_ARG,
 * MOE_ERR_WORKSPACE, MOE_ERR_UNSUPPORTED (device ordinal >= 64) or MOE_ERR_CUDA. */
int moe_quantile_target_static(const float* logits, const float* alpha, int32_t num_tokens,
                               int32_t num_experts, int32_t top_k, float* target_out, void* cuda_stream);

/* Validation utility for the bounded device-side waits: launches one warp that
 * waits, with the same bounded wait the routing kernel uses and the given
 * iteration bound, on a barrier phase that nothing ever completes.  The wait
 * gives up, the kernel returns normally, and the next moe_route_poll reports
 * MOE_ERR_TIMEOUT (wait id 99); the context stays usable. */
int moe_debug_wait_timeout(moe_route_ctx* ctx, int32_t spin_limit, void* cuda_stream);

/* Validation utility for the give-up path of the routing kernel itself: in the
 * NEXT moe_route_step of this context (only that one) every producer warp stops
 * issuing loads after `after_loads` (>= 1) pipeline stages, as if the copies had
 * stalled.  Nothing is left in flight; the consumers' bounded waits run out (use
 * a context with a small spin_limit so that this takes milliseconds), every role
 * of every CTA leaves its loop, tensor memory is released, the kernel returns,
 * and moe_route_poll reports MOE_ERR_TIMEOUT.  Host call; nothing is enqueued. */
int moe_debug_route_stall(moe_route_ctx* ctx, int32_t after_loads);

/* 1 if the library was compiled with -DMOE_DEBUG, else 0.  That build is the stand-in for a memory checker:
 * the routing kernel guards the indices of its shared-memory log, exchange area, output and candidate
 * writes (a bad index is recorded and the access skipped), every workspace section is followed by a
 * 256-byte canary, and moe_route_poll reports either as MOE_ERR_INTERNAL.  Results are identical to the
 * release build's; moe_route_workspace_bytes is larger by the canaries. */
int moe_debug_build(void);

/* Number of kernels this context has launched so far. */
int64_t moe_route_launch_count(const moe_route_ctx* ctx);

/* Text of the last error of this context ("" if none); valid until the next call. */
const char* moe_last_error(const moe_route_ctx* ctx);

int moe_route_destroy(moe_route_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MOE_ROUTE_H_ */
