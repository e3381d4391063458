/*
 * mcce -- cache-conditional MoE decode step for many independent token streams (NVIDIA B200, sm_100a).
 *
 * C ABI of libmcce.so.  Plain pointers and sizes only; every pointer is marked HOST or DEVICE.
 * The method is "Mixture of Cache-Conditional Experts" (arXiv 2412.00099); the citations below name
 * the equation, section or algorithm of that paper which defines each operation.
 *
 * Notation (paper, Sec. 2.1 / 2.2 / 3.3): N = E routed experts per layer, top-K selection, top-J
 * guaranteed experts, cache set C of `cache_capacity` experts per (stream, layer), promotion strength
 * lambda, logit range Delta_avg.  S independent token streams, L MoE layers, hidden size d, expert
 * intermediate size I.  Streams and layers are independent of one another; tokens of one stream are
 * sequential because the cache state carries over.
 *
 * Ownership: the caller owns every buffer, including the workspace, and keeps them alive until
 * mcce_destroy.  The library allocates no device memory and creates no streams (except the three internal
 * streams of the pipelined entry points).  Weights are borrowed.
 * Errors: every call returns 0 on success or a negative MCCE_E* code; nothing throws, aborts or prints.
 * Kernel launches are asynchronous on the given stream unless a function says that it synchronises.
 * A context is not thread-safe; distinct contexts are independent.
 */
#ifndef MCCE_H_
#define MCCE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MCCE_OK = 0,
  MCCE_EINVAL = -1,   /* bad argument or unsupported configuration                      */
  MCCE_ENOSPC = -2,   /* workspace too small                                            */
  MCCE_ESTATE = -3,   /* weights not set, or a counter would overflow (reset needed)    */
  MCCE_ECUDA = -4,    /* a CUDA call failed; see mcce_last_cuda_error                   */
  MCCE_ETIMEOUT = -5, /* a bounded wait inside a kernel gave up: the launch it happened in is incomplete (results,
                         cache state and internal buffers), the CUDA context stays usable; mcce_reset brings the
                         mcce context back to a defined state                                             */
  MCCE_ELIMIT = -6,   /* problem larger than the fixed array of mcce_route_trace_static   */
  MCCE_EINDEX = -7,   /* an expert id outside [0, E) reached the grouping pass (the pair was skipped), or a
                         check of the checked mode failed: a grouping position outside [0, S*K), more than C
                         resident experts, or two resident experts with the same recency key               */
  MCCE_ENONFINITE = -8 /* checked mode: a router logit was NaN or infinite                               */
};

enum { MCCE_F32 = 0, MCCE_BF16 = 1 };
enum { MCCE_DELTA_RUNNING = 0, MCCE_DELTA_FIXED = 1 };
enum { MCCE_FFN_AUTO = 0, MCCE_FFN_SIMT = 1, MCCE_FFN_TENSOR = 2 };
/* How the router's ranking r is changed in favour of cached experts (Sec. 3):
 * CACHE_PRIOR  Eq. 7, the paper's main method: rank by z' = z + lambda*Delta_avg*m~_t;
 * MAX_RANK     Algorithm 1: promote(r[:J]; promote(r[:M] ∩ C; r)) with M = max_rank;
 * CUMSUM       Algorithm 2: the same with M = the smallest number of top-ranked experts whose router
 *              probabilities sum to at least cum_threshold. */
enum { MCCE_RERANK_CACHE_PRIOR = 0, MCCE_RERANK_MAX_RANK = 1, MCCE_RERANK_CUMSUM = 2 };

typedef struct mcce_ctx mcce_ctx; /* opaque; host memory owned by the library */

typedef struct {
  int32_t n_layers;       /* L >= 1                                                              */
  int32_t n_experts;      /* E = N routed experts per layer, 1..256                              */
  int32_t top_k;          /* K, 1..min(E,16)                                                     */
  int32_t top_j;          /* J, 0..K: router's top-J experts are always selected (Sec. 3.3)      */
  int32_t n_shared;       /* always-on experts per layer, weight 1, never cached, >= 0           */
  int32_t d_model;        /* d, multiple of 8                                                    */
  int32_t d_ff;           /* I, multiple of 8                                                    */
  int32_t cache_capacity; /* C >= 1 experts per (stream, layer); C >= E means nothing is evicted */
  int32_t n_streams;      /* S >= 1                                                              */
  float lambda;           /* promotion strength of Eq. 7, finite, >= 0 (paper: [0,1])            */
  int32_t delta_mode;     /* MCCE_DELTA_RUNNING: Delta_avg is the cumulative mean, per (stream,
                             layer), of max(z)-min(z) including the current token (Eq. 8);
                             MCCE_DELTA_FIXED: per-layer constants given to mcce_set_router
                             (appendix "Logit Range Estimation")                                 */
  int32_t renorm;         /* 1: weights renormalised over the K selected experts (Sec. 2.1)      */
  int32_t hidden_dtype;   /* MCCE_F32 or MCCE_BF16                                               */
  int32_t weight_dtype;   /* expert weights; must equal hidden_dtype                             */
  int32_t ffn_impl;       /* MCCE_FFN_AUTO picks the tensor-core path when it applies            */
  int32_t device;         /* CUDA device ordinal                                                 */
  int32_t rerank_mode;    /* MCCE_RERANK_*; lambda / delta_mode only matter for CACHE_PRIOR      */
  int32_t max_rank;       /* M of Algorithm 1, 0..E (MAX_RANK only)                              */
  float cum_threshold;    /* p of Algorithm 2, >= 0 (CUMSUM only)                                */
  int32_t track_lifetime; /* 1: record how long experts stay cached (mcce_lifetime_stats)         */
  int32_t route_impl;     /* MCCE_ROUTE_AUTO (0) picks per launch what was measured faster;
                             MCCE_ROUTE_TWO_KERNELS: logits kernel, then routing tail;
                             MCCE_ROUTE_FUSED: the single cooperative kernel wherever it can run.  That kernel
                             adds the parts of its split reduction of Eq. 3 in the order in which they arrive,
                             so the last bit of a logit (and with it a selection between two experts whose
                             logits are equal to within rounding) can differ between runs; the two-kernel path
                             adds them in a fixed order.  The deterministic and the checked mode never use it */
  int32_t deterministic;  /* 1: repeated runs give identical bits (the paper's runs are deterministic, Sec. 4.1):
                             y = sum_k w_k E_k(x) + shared experts is added in slot order on every path (the
                             tensor-core path then writes one fp32 row per (stream, slot) and sums them in a
                             second pass instead of adding into y with atomics), and the router logits come
                             from the two-kernel path                                                       */
  int32_t checked;        /* 1: checked mode.  Every routing launch is followed by kernels that verify the
                             logits (finite), the cache state (at most C resident experts per (stream,
                             layer), distinct recency keys) and every grouping pass (positions inside
                             [0, S*K)); a violation is recorded and reported by mcce_cache_stats as
                             MCCE_ENONFINITE / MCCE_EINDEX.  Costs a few small launches per call          */
} mcce_config;

typedef struct {
  int64_t steps;       /* (stream, token, layer) routing steps                                   */
  int64_t selections;  /* K * steps, denominator of Eq. 4                                        */
  int64_t misses;      /* selected experts absent from the cache as it was before the token      */
  int64_t cold_misses; /* misses on experts that had never been resident (compulsory misses)     */
} mcce_stats;

/* Bytes of DEVICE workspace mcce_create needs for this configuration (0 if the config is invalid). */
size_t mcce_workspace_bytes(const mcce_config* cfg /*HOST*/);

/* Validates cfg, carves `workspace` (DEVICE, 256-byte aligned, >= mcce_workspace_bytes) into the
 * state arrays, zeroes them (cache empty) and returns a context.  Synchronises the device. */
int mcce_create(const mcce_config* cfg /*HOST*/, void* workspace /*DEVICE*/, size_t workspace_bytes,
                mcce_ctx** out /*HOST*/);
int mcce_destroy(mcce_ctx* ctx);

/* Router G of Eq. 3: z = W_r[l] x.  Wr: DEVICE fp32 [L,E,d], row-major.  fixed_delta: DEVICE fp32 [L],
 * required iff delta_mode == MCCE_DELTA_FIXED, else may be NULL.  Borrowed. */
int mcce_set_router(mcce_ctx* ctx, const float* Wr, const float* fixed_delta);

/* Experts E_i of Eq. 1 as SwiGLU: E_i(x) = W_d (silu(W_g x) * (W_u x)).  DEVICE, weight_dtype,
 * row-major: Wg, Wu [L,E,I,d]; Wd [L,E,d,I]; shared experts shWg, shWu [L,n_shared,I,d],
 * shWd [L,n_shared,d,I] (NULL when n_shared == 0).  Borrowed. */
int mcce_set_experts(mcce_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* shWg,
                     const void* shWu, const void* shWd);

/* Empties every cache, or loads an initial cache content (Sec. 4.8 "Impact of Initial Cache State"):
 * init_order HOST int32 [L,S,C], resident experts most-recently-used first, -1 padding; NULL = empty.
 * These entries count as older than anything touched later.  Counters are zeroed.  The running
 * Delta statistics are kept iff keep_delta_stats != 0, or replaced when delta_sum (HOST fp32 [L,S])
 * is given together with delta_count (tokens it was summed over).  Synchronises. */
int mcce_reset(mcce_ctx* ctx, const int32_t* init_order, int keep_delta_stats, const float* delta_sum,
               int64_t delta_count);

/* n_steps tokens of routing for every (stream, layer): Eq. 3 logits (or given logits), Eq. 8 range
 * statistic, mask m~_t = cache OR top-J, Eq. 7 promotion z' = z + lambda*Delta_avg*m~_t, top-K of z'
 * (ties to the lower expert index), weights = softmax of the UNMODIFIED z over the selected experts
 * (Sec. 3.3), Eq. 4 miss counting against the cache as it was before the token, LRU update in which
 * the selected expert with the higher router weight counts as older (Sec. 4.2).
 *   hidden     DEVICE hidden_dtype [n_steps,L,S,d], or NULL
 *   logits_in  DEVICE fp32 [n_steps,L,S,E], or NULL; exactly one of the two is non-NULL
 *   sel_idx    DEVICE int32 [n_steps,L,S,K] out, rank order of z'
 *   sel_w      DEVICE fp32  [n_steps,L,S,K] out
 *   logits_out DEVICE fp32  [n_steps,L,S,E] out, optional: the logits the decision was taken on
 * When E is a multiple of 4, rows of logits are read and written four floats at a time: logits_in and
 * logits_out must then be 16-byte aligned (MCCE_EINVAL otherwise; 4-byte alignment suffices for other E).
 */
int mcce_route_step(mcce_ctx* ctx, int32_t n_steps, const void* hidden, const float* logits_in,
                    int32_t* sel_idx, float* sel_w, float* logits_out, void* cuda_stream);

/* Eq. 1 for one token of every (stream, layer): groups the (stream, slot) pairs by expert, runs the
 * SwiGLU experts group by group and combines y = sum_k w_k E_sel_k(x) (slot order) + shared experts.
 *   hidden DEVICE hidden_dtype [L,S,d]; sel_idx DEVICE int32 [L,S,K]; sel_w DEVICE fp32 [L,S,K];
 *   y DEVICE fp32 [L,S,d] out.
 * With bf16 weights the intermediate silu(g)*u is rounded to bf16 before the down projection.  On the
 * tensor-core path the K + n_shared terms of a stream are added into y with fp32 atomic adds in no fixed
 * order, so the last bits of y may differ between runs, unless the configuration sets `deterministic`
 * (the fp32-pipe path always sums in slot order).
 * An entry of sel_idx outside [0, E) (padding, an uninitialised buffer) is skipped: the pair contributes
 * nothing to y, and the next mcce_cache_stats reports MCCE_EINDEX. */
int mcce_moe_forward(mcce_ctx* ctx, const void* hidden, const int32_t* sel_idx, const float* sel_w,
                     float* y, void* cuda_stream);

/* One token in sequential-layer mode: the layers are chained through a residual stream instead of being
 * independent, as in a real decoder (the paper changes nothing in the forward pass but the ranking, Sec. 2.2).
 * For l = 0..L-1: route layer l on its input x_l, run its experts, x_{l+1} = x_l + y_l rounded to the hidden
 * dtype (no normalisation layer: the logit scale may drift with depth, which the per-layer Delta_avg absorbs).
 *   x0     DEVICE hidden_dtype [S,d]: input of layer 0        x_out DEVICE hidden_dtype [S,d]: output of layer L-1
 *   sel_idx DEVICE int32 [L,S,K], optional: the selections of every layer
 * Cache state, counters, Delta statistics and the miss trace advance exactly as with mcce_route_step.  Launches
 * L rounds of the single-layer kernels on the stream (asynchronous).  On the tensor-core path the expert
 * outputs are summed with fp32 atomics, so x_{l+1} can differ in its last bit between runs, and with it,
 * rarely, a near-tie routing decision of a later layer. */
int mcce_decode_step_chained(mcce_ctx* ctx, const void* x0, void* x_out, int32_t* sel_idx, void* cuda_stream);

/* One whole decode step from HOST buffers: copies hidden [L,S,d] to the device, routes, runs the
 * experts and copies y [L,S,d] (and, if non-NULL, sel_idx [L,S,K]) back.  Staging lives in the
 * workspace.  hidden_host / y_host should be pinned.  Synchronises the stream before returning. */
int mcce_decode_step_host(mcce_ctx* ctx, const void* hidden_host, float* y_host, int32_t* sel_idx_host,
                          void* cuda_stream);

/* The same decode step, pipelined over successive tokens.  Routing needs only the hidden states of its token and
 * the cache state that the previous token's routing left (Sec. 3.3: the mask m_t is the cache after token t-1),
 * not the previous token's experts; so routing, grouping and the row copy of step t+1 run on an internal stream
 * while the expert kernels of step t, which stream all the weights, still run on cuda_stream.  Two sets of
 * buffers ("slots") alternate.
 *
 * mcce_pipeline_submit_host enqueues, without waiting, the upload of hidden_host [L,S,d] on an internal copy-in
 * stream, the step, and the download of y [L,S,d] (and sel_idx [L,S,K] if non-NULL) on an internal copy-out
 * stream once the step has finished.  A call blocks only if the step submitted two calls earlier has not yet
 * left the device, so the upload of token t+1 and the download of token t-1 also run while token t computes.
 * The host buffers of a submitted step must stay valid, and y_host must not be read, until mcce_pipeline_wait
 * (or the second following submit) returns.  hidden_host / y_host must be pinned for the copies to be
 * asynchronous.
 *
 * mcce_pipeline_submit is its twin for DEVICE buffers: hidden [L,S,d] (hidden_dtype), y [L,S,d] fp32 out, sel_idx
 * [L,S,K] int32 out or NULL.  Nothing is copied.  The library reads `hidden` on its internal stream, which does
 * not wait for cuda_stream: hidden must be complete when the call is made, or hidden_ready (a cudaEvent_t, may be
 * NULL) must mark its completion.  y and sel_idx are complete in cuda_stream order.  y is cleared on the internal
 * stream while the previous step may still compute: consecutive calls must use different y buffers, and neither
 * hidden nor y of a step may be touched by the caller until that step has finished on cuda_stream.
 *
 * The three internal streams and their events are the only CUDA objects the library creates (on the first
 * submit); it still allocates no device memory.  Always use the same cuda_stream per context, and call
 * mcce_pipeline_wait before using any other entry point of the context that routes or runs experts. */
int mcce_pipeline_submit_host(mcce_ctx* ctx, const void* hidden_host, float* y_host, int32_t* sel_idx_host,
                              void* cuda_stream);
int mcce_pipeline_submit(mcce_ctx* ctx, const void* hidden /*DEVICE*/, float* y /*DEVICE*/, int32_t* sel_idx /*DEVICE*/,
                         void* hidden_ready /*cudaEvent_t or NULL*/, void* cuda_stream);
/* Waits until every submitted step has finished (and, for host buffers, has been copied back). */
int mcce_pipeline_wait(mcce_ctx* ctx);

/* Eq. 4 counters, summed over streams: total and per layer (HOST [L], may be NULL).  Synchronises.
 * The counters are always written; the return value also carries what the kernels of this context recorded
 * since the last mcce_reset, in this order of precedence: MCCE_ETIMEOUT (a bounded wait gave up),
 * MCCE_EINDEX (an expert id out of range was skipped, or a check of the checked mode failed),
 * MCCE_ENONFINITE (checked mode: a non-finite logit). */
int mcce_cache_stats(mcce_ctx* ctx, mcce_stats* total /*HOST*/, mcce_stats* per_layer /*HOST*/);

/* Cache lifetimes (the statistic of the paper's Table 2): a lifetime is the number of tokens from the
 * token that loaded an expert into a (stream, layer) cache to the token that evicted it; experts still
 * resident are not counted.  total / per_layer (HOST, [L], may be NULL) receive {evictions, sum of
 * lifetimes, sum of squared lifetimes}; mean = sum/evictions, variance = sumsq/evictions - mean^2.
 * Needs track_lifetime = 1 in the configuration (MCCE_ESTATE otherwise).  Not part of the state that
 * mcce_get_cache_state exports.  Synchronises. */
typedef struct { int64_t evictions, sum, sum_sq; } mcce_lifetime;
int mcce_lifetime_stats(mcce_ctx* ctx, mcce_lifetime* total /*HOST*/, mcce_lifetime* per_layer /*HOST*/);

/* Per-token miss trace (the data behind the paper's hit / miss timelines of Sec. 4.6): while a buffer is set,
 * every routed token writes one word per (layer, stream) whose bit k says that the k-th selected expert was
 * not in the cache.  trace: DEVICE uint32 [capacity_tokens, L, S], caller-owned; tokens beyond the capacity
 * are not recorded; recording restarts at entry 0 when the buffer is set and after mcce_reset.  NULL with
 * capacity 0 turns it off. */
int mcce_set_miss_trace(mcce_ctx* ctx, uint32_t* trace, int64_t capacity_tokens);

/* Logit range from a calibration set (appendix "Logit Range Estimation": Delta_avg estimated once over a
 * calibration set instead of during inference).  After some tokens have been routed in MCCE_DELTA_RUNNING
 * mode, writes for every layer the mean over its streams of the running estimate of Eq. 8,
 *   delta[l] = (1/S) sum_s sum_range[l][s] / tokens,
 * accumulated in double precision and rounded once to fp32: the constants to hand to mcce_set_router of a
 * context in MCCE_DELTA_FIXED mode.  delta HOST fp32 [L].  MCCE_ESTATE if no token has been routed yet.
 * Synchronises. */
int mcce_calibrate_delta(mcce_ctx* ctx, float* delta /*HOST*/);

/* Canonical cache state: order HOST int32 [L,S,C] most-recently-used first, -1 padded; optional
 * ever HOST uint8 [L,S,E]; delta_sum HOST fp32 [L,S] and *delta_count (optional).  Synchronises. */
int mcce_get_cache_state(mcce_ctx* ctx, int32_t* order, uint8_t* ever, float* delta_sum,
                         int64_t* delta_count);

/* Result of the expert-grouping pass of the last mcce_moe_forward (histogram, scan, stable scatter):
 * offsets HOST int32 [L,E+1]; perm HOST int32 [L,S*K], perm[l][pos] = s*K+slot of the pair placed at
 * pos, pairs of one expert contiguous and in increasing (s,slot) order.  Synchronises. */
int mcce_get_grouping(mcce_ctx* ctx, int32_t* offsets, int32_t* perm);

/* Belady's optimal eviction (Sec. 4.8 "Optimal Cache Eviction") replayed on a recorded selection trace: the
 * lossless bound that LRU cannot beat and that the paper's lossy rerouting can.  For every (stream, layer)
 * and every capacity the trace is replayed from an empty cache; on a miss the expert is inserted, and while
 * the cache is over capacity the resident expert whose next use lies farthest ahead is evicted, never one
 * the current token itself selects.  Context-free.
 *   sel_trace  DEVICE int32 [n_tokens, L, S, K]: the sel_idx output of mcce_route_step (K distinct experts)
 *   capacities DEVICE int32 [n_capacities], each >= K
 *   next_use_scratch DEVICE int32 [n_tokens, L, S, K], overwritten
 *   misses     DEVICE int64 [n_capacities, L, S] out
 * Asynchronous on the stream.  Capacities below K are the caller's error (the result is then undefined). */
int mcce_belady_replay(const int32_t* sel_trace, int32_t n_tokens, int32_t n_layers, int32_t n_streams,
                       int32_t n_experts, int32_t top_k, const int32_t* capacities, int32_t n_capacities,
                       int32_t* next_use_scratch, int64_t* misses, void* cuda_stream);

/* Seeded synthetic inputs (counter-based: Philox4x32-10 keyed by (seed, 0), counter = (element
 * block, t, tensor_id), Box-Muller with fixed-order fp32 series); no counterpart in the paper, whose
 * inputs are text corpora.  out DEVICE, dtype MCCE_F32/MCCE_BF16; elements [start, start+count) of the
 * tensor, value = std * n.  start must be a multiple of 4. */
int mcce_gen_normal(void* out, int32_t dtype, uint64_t start, uint64_t count, uint32_t seed,
                    uint32_t tensor_id, uint32_t t, float std, void* cuda_stream);
/* AR(1) hidden states: h <- (t==0 ? n_t : rho*h + c*n_t) on state DEVICE fp32 [count]; emits
 * x = h + offset_scale * n_offset (offset omitted when offset_scale == 0) as dtype.  count % 4 == 0. */
int mcce_gen_hidden_step(float* state, void* x_out, int32_t dtype, uint64_t count, uint32_t seed,
                         uint32_t t, float rho, float c, float offset_scale, void* cuda_stream);
/* Raw Philox words, DEVICE uint32 [n_blocks,4], for checking the generator bit by bit. */
int mcce_gen_philox_words(uint32_t* out, uint64_t start_block, uint64_t n_blocks, uint32_t seed,
                          uint32_t tensor_id, uint32_t t, void* cuda_stream);

/* Per-kernel device time, for measurement (no counterpart in the paper).  When enabled, every launch
 * of this context is bracketed by a pair of CUDA events on its stream; mcce_profile_read waits for the
 * recorded events and returns, per kernel kind, the summed milliseconds and the number of launches
 * (HOST arrays of MCCE_N_KERNELS entries), clearing the sums if reset != 0. */
enum {
  MCCE_K_ROUTE = 0,    /* fused route kernel (with bf16 hidden states: its tail, on the logits of MCCE_K_ROUTE_GEMM) */
  MCCE_K_GROUP = 1,    /* grouping, first pass: histograms of the selected experts per chunk of pairs */
  MCCE_K_GATHER = 2,   /* grouping, second pass: scan, stable scatter, and the activation rows copied into expert
                          order on the way (clears y on the tensor-core path) */
  MCCE_K_FFN_UP = 3,   /* H = silu(X Wg^T) * (X Wu^T), all groups    */
  MCCE_K_FFN_DOWN = 4, /* O = H Wd^T, all groups                     */
  MCCE_K_COMBINE = 5,  /* weighted sum over slots + shared experts (fp32-pipe path; fused into FFN_DOWN otherwise) */
  MCCE_K_ROUTE_GEMM = 6, /* router logits on the tensor cores (bf16 hidden states) */
  MCCE_N_KERNELS = 7
};
int mcce_profile(mcce_ctx* ctx, int enable);
int mcce_profile_read(mcce_ctx* ctx, double* ms /*HOST*/, int64_t* launches /*HOST*/, int reset);

/* Routing with no context, no workspace and no allocation of any kind.  The paper has no counterpart
 * to this call; it exists for callers that cannot allocate device memory where they need routing
 * decisions: a server whose memory pool already owns the whole GPU, a plug-in that only receives input
 * and output buffers, or a latency-critical callback that must not enter the allocator.
 *
 * Routes n_steps tokens of every (stream, layer) with the routing kernels of mcce_route_step, starting from
 * EMPTY caches, zero counters and (running mode) an empty Delta statistic.  From hidden states the logits
 * are formed on the fp32 pipe for both hidden dtypes (a context given bf16 hidden states uses the tensor
 * cores instead, so its logits can differ in the last bits and, at a near tie, so can a selection).  The cache
 * state it needs while it runs lives in a fixed array inside the library image
 * (mcce_route_trace_static_limit() bytes = 4 MiB, resident on every GPU that loads the library until
 * the process exits) instead of in a workspace.  The state needs about L*S*(4*E + 4*ceil(E/32) + 12)
 * bytes; a configuration that does not fit is refused with MCCE_ELIMIT and nothing is launched.
 *   cfg         HOST; n_layers, n_streams, n_experts, top_k, top_j, cache_capacity, lambda, delta_mode,
 *               renorm, hidden_dtype, d_model, rerank_mode, max_rank and cum_threshold are used and checked
 *               as in mcce_create; the rest is ignored
 *               (hidden must be 16-byte aligned, and so must logits_in when E is a multiple of 4)
 *   hidden, Wr  DEVICE [n_steps,L,S,d] (hidden_dtype) and fp32 [L,E,d], or both NULL
 *   logits_in   DEVICE fp32 [n_steps,L,S,E], or NULL; exactly one of hidden / logits_in is given
 *   fixed_delta DEVICE fp32 [L], only for MCCE_DELTA_FIXED
 *   sel_idx, sel_w  DEVICE outputs [n_steps,L,S,K], as in mcce_route_step
 *   totals_host HOST, optional: Eq. 4 counters summed over everything; asking for them makes the call
 *               wait for the stream, otherwise it only enqueues work
 * The device that is current when the call is made is used.  The first call on each device looks up
 * the array's device address and keeps it for the life of the process; make that first call outside any
 * stream capture, and do not call again on a device after cudaDeviceReset (the address is then stale).  The call uses no
 * cudaMalloc / cudaFree and no allocating library routine.  Every call on a device shares the one
 * array and first clears the part it uses, so nothing carries over between calls -- and two calls
 * whose GPU work overlaps (different streams, or different host threads) race on it: serialise them. */
size_t mcce_route_trace_static_limit(void);
int mcce_route_trace_static(const mcce_config* cfg /*HOST*/, int32_t n_steps, const void* hidden, const float* Wr,
                            const float* logits_in, const float* fixed_delta, int32_t* sel_idx, float* sel_w,
                            mcce_stats* totals_host, void* cuda_stream);

/* Self-test of the bounded waits that the tensor-core kernels use (no counterpart in the paper).  Launches
 * a one-CTA kernel that waits on a barrier nothing ever arrives at, with a limit of limit_ns (1..1e9).  The
 * wait must give up and the kernel must return: MCCE_OK then, and the context's error word is set, so that
 * the next mcce_cache_stats reports MCCE_ETIMEOUT until mcce_reset clears it.  The GPU context stays usable.
 * Synchronises. */
int mcce_selftest_wait_timeout(mcce_ctx* ctx, uint64_t limit_ns);

/* 1 if mcce_moe_forward of this context runs the tcgen05/TMA expert kernels, 0 if the fp32-pipe ones. */
int mcce_uses_tensor_path(const mcce_ctx* ctx);

/* Which kernels mcce_route_step runs for a launch of n_tokens tokens from hidden states, once the router is
 * set (Eq. 3 and the routing rule of Sec. 3.3 either way; this is introspection for tests and benchmarks):
 * MCCE_ROUTER_FP32_PIPE      the fused route kernel forms the logits itself on the fp32 pipe (fp32 hidden states);
 * MCCE_ROUTER_GEMM_TAIL      tcgen05 GEMM with the experts as MMA rows, then the routing tail;
 * MCCE_ROUTER_RESIDENT_TAIL  tcgen05 GEMM with the router resident in shared memory, then the routing tail;
 * MCCE_ROUTER_FUSED          the router-resident GEMM and the tail in one cooperative kernel.
 * Negative: an error code. */
enum { MCCE_ROUTE_AUTO = 0, MCCE_ROUTE_TWO_KERNELS = 1, MCCE_ROUTE_FUSED = 2 };
enum { MCCE_ROUTER_FP32_PIPE = 0, MCCE_ROUTER_GEMM_TAIL = 1, MCCE_ROUTER_RESIDENT_TAIL = 2, MCCE_ROUTER_FUSED = 3 };
int mcce_router_kernel_kind(const mcce_ctx* ctx, int32_t n_tokens);

const char* mcce_strerror(int code);
int mcce_last_cuda_error(const mcce_ctx* ctx); /* cudaError_t of the last failed CUDA call */

#ifdef __cplusplus
}
#endif
#endif /* MCCE_H_ */
