// Internal declarations shared by the translation units of libmcce.so.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mcce.h"

namespace mcce {

constexpr int kMaxE = 256;
constexpr int kMaxK = 16;

// Everything the route kernel needs (passed by value).
struct RouteParams {
  int L, S, E, K, J, C, d;
  int n_steps;
  float lambda;
  int delta_mode, renorm;
  int rerank_mode, max_rank;  // MCCE_RERANK_*; M of Algorithm 1
  float cum_threshold;        // p of Algorithm 2
  int hidden_bf16;
  const void* hidden;        // [n_steps,L,S,d] or null
  const float* logits_in;    // [n_steps,L,S,E] or null; n_partials such arrays, partial_stride elements apart,
                             // are summed (the tensor-core router GEMM may split its reduction)
  int n_partials;
  size_t partial_stride;
  const float* Wr;           // [L,E,d]
  const float* fixed_delta;  // [L]
  uint32_t* stamp;           // [L,S,E]   0 = not resident, else recency key
  uint32_t* ever;            // [L,S,EW]  bit e%32 of word e/32
  float* sum_range;          // [L,S]
  uint32_t* miss;            // [L,S]
  uint32_t* cold;            // [L,S]
  uint32_t* load_tok;        // [L,S,E] token that loaded each resident expert, or null (lifetimes not tracked)
  unsigned long long* life;  // [L,S,3]  evictions, sum and sum of squares of cache lifetimes
  uint32_t* miss_trace;      // [trace_avail,L,S] per-token miss bits of this launch's tokens, or null
  int trace_avail;           // tokens of this launch that still fit the trace buffer
  int32_t* sel_idx;          // [n_steps,L,S,K]
  float* sel_w;              // [n_steps,L,S,K]
  float* logits_out;         // [n_steps,L,S,E] or null
  uint32_t tok0;             // tokens already processed since the last reset
  uint32_t cnt0;             // tokens already folded into the running Delta
  uint32_t* err_nonfinite;   // checked mode: set by the kernel that forms its own logits when one is not finite; else null
};

// Bits of the context's index-error word (the second word of its error block; the first is the code of a
// bounded wait that gave up, the third is set when the checked mode meets a non-finite logit).
constexpr uint32_t kErrBadExpertId = 1u;   // sel_idx entry outside [0, E): the pair was skipped
constexpr uint32_t kErrBadPosition = 2u;   // checked mode: offsets not monotone or a position outside [0, S*K)
constexpr uint32_t kErrOverCapacity = 4u;  // checked mode: more than C resident experts in a (stream, layer)
constexpr uint32_t kErrDuplicateKey = 8u;  // checked mode: two resident experts with the same recency key

struct GroupParams {
  int L, S, E, K;
  const int32_t* sel_idx;  // [L,S,K]
  int32_t* offsets;        // [L,E+1]
  int32_t* perm;           // [L,S*K] position -> pair
  int32_t* inv;            // [L,S*K] pair -> position, -1 for a pair whose expert id is out of range
  uint32_t* err_index;     // index-error word of the context
};

// Rows of the activation / intermediate / output buffers: routed pairs first, [l][pos], then the
// shared experts, [l][q][s].
struct FfnParams {
  int L, S, E, K, n_sh, d, I;
  int l0;  // model layer of local layer 0: only the weights are indexed by model layer, everything else is local
  int slot;  // which of the two sets of grouping buffers (and of their tensor maps) this step uses
  int bf16;
  const void* hidden;  // [L,S,d]
  const void *Wg, *Wu, *Wd, *shWg, *shWu, *shWd;
  const int32_t* offsets;  // [L,E+1]
  const int32_t* perm;     // [L,S*K]
  const int32_t* inv;      // [L,S*K]
  const float* sel_w;      // [L,S,K]
  void* Xg;                // [L*S*K, d]   gathered activations, hidden dtype
  void* H;                 // [rows, I]    silu(g)*u, weight dtype
  float* O;                // [rows, d]    expert outputs
  float* y;                // [L,S,d]
};

// Router logits on the tensor cores (route_gemm.cu).  Plain data: lives inside the zero-initialised context.
struct RouterGemmPlan {
  alignas(64) CUtensorMap w, x;
  alignas(64) CUtensorMap w_res, x_res, xt_res;   // router-resident kernel (route_gemm_res.cu)
  const void* hidden_ptr;
  uint64_t hidden_rows;
  const void* hidden_ptr_res;
  uint64_t hidden_rows_res;
  int ready;
  int res_ready, res_parts;   // K parts (= partial logit arrays) of the router-resident kernel
  int res_parts_single;       // the same for a launch of one layer at a time
  int fused_ready, fused_parts;   // the same for the kernel that also runs the routing tail (route_fused.cu)
  int fused_tail_warps;           // tail warps per CTA of that kernel
  int fused_flip;                 // which of its two counter sets the next launch uses
};
bool router_gemm_applicable(const mcce_config& c);
int router_gemm_steps_max();
int router_gemm_plan(const mcce_config& c, const float* Wr, void* terms, RouterGemmPlan* plan, cudaStream_t st);
cudaError_t router_gemm_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps, float* Z,
                               int* k_split, uint32_t* err, cudaStream_t st, int l0 = 0, int n_layers = 0);

bool router_gemm_res_applicable(const mcce_config& c);
int router_gemm_res_parts_max();
int router_gemm_res_plan(const mcce_config& c, void* terms, RouterGemmPlan* plan);
cudaError_t router_gemm_res_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps,
                                   float* Z, int* k_parts, uint32_t* err, cudaStream_t st, int l0 = 0, int n_layers = 0);

int route_fused_plan(const mcce_config& c, RouterGemmPlan* plan);
size_t route_fused_counter_words(int n_layers, int n_steps, int n_streams);
cudaError_t route_fused_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps, float* Z,
                               uint32_t* ready, RouteParams p, uint32_t* err, cudaStream_t st);

cudaError_t launch_wait_timeout_selftest(uint32_t* err, unsigned long long limit_ns, uint32_t* outcome,
                                         cudaStream_t st);
cudaError_t launch_route(const RouteParams& p, cudaStream_t st);   // picks the thread-per-stream kernel where it applies
bool route_thread_applicable(const RouteParams& p);
cudaError_t launch_route_thread(const RouteParams& p, cudaStream_t st);
int group_chunks(int S, int K);   // CTAs per layer of the grouping kernels (= histograms per layer)
cudaError_t launch_group(const GroupParams& p, int* counts /*[L][group_chunks][E]*/, int* tickets /*[L], zero*/,
                         cudaStream_t st);
cudaError_t launch_place(const GroupParams& p, const FfnParams& f, const int* counts, bool zero_y, cudaStream_t st);
cudaError_t launch_ffn_simt_up(const FfnParams& p, cudaStream_t st);
cudaError_t launch_ffn_simt_down(const FfnParams& p, cudaStream_t st);
cudaError_t launch_combine(const FfnParams& p, cudaStream_t st);
cudaError_t launch_residual(const void* x_in, const float* y, void* x_out, size_t n, bool bf16, cudaStream_t st);
cudaError_t launch_stats(const uint32_t* miss, const uint32_t* cold, unsigned long long* out, int L, int S,
                         cudaStream_t st);
cudaError_t launch_check_group(const GroupParams& p, cudaStream_t st);
cudaError_t launch_check_state(const uint32_t* stamp, size_t n_pairs, int E, int C, uint32_t* err_index,
                               cudaStream_t st);
cudaError_t launch_check_finite(const float* z, size_t n, uint32_t* err_nonfinite, cudaStream_t st);
cudaError_t launch_calibrate(const float* sum_range, int L, int S, double count, float* out, cudaStream_t st);

__device__ __forceinline__ float bf16_to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

}  // namespace mcce
