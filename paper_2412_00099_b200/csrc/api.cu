// Host side of libmcce.so: configuration checks, workspace layout, and the entry points of mcce.h.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"
#include "ffn_tc.cuh"

using namespace mcce;

constexpr int kMaxPairs = 1024;
// When MCCE_ROUTE_AUTO takes the single fused kernel: from three tokens per launch.  Measured, fused against two
// kernels, us per launch of 2 / 3 / 4 / 8 tokens: Qwen-shaped 39/37, 46/50, 55/62, 84/100; OLMoE-shaped 55/53,
// 72/74, 84/97, 143/172; DeepSeek-shaped 47/44, 58/58, 69/73, 114/124; Mixtral-shaped 27/34, 33/43, 39/51, 60/85.
constexpr int kFusedMinTokens = 3;

struct mcce_ctx {
  mcce_config cfg;
  int EW;
  size_t rows;  // rows of H / O: L*S*K routed pairs + L*n_sh*S shared
  // workspace pieces (device)
  uint32_t *stamp, *ever, *miss, *cold, *err, *load_tok;
  unsigned long long* life;
  float* sum_range;
  unsigned long long* stats_dev;
  // grouping of a step: bucket offsets, permutation and its inverse, activations in expert order.  Two sets, so
  // that the pipelined entry points can prepare one step while the experts of the previous one still read theirs
  struct GroupBufs {
    int32_t *offsets, *perm, *inv;
    void* Xg;
  } gb[2];
  int last_slot;   // the set the latest forward used (mcce_get_grouping reads it)
  int* group_counts;
  void* H;
  float* O;
  void* stage_hidden;
  int32_t* stage_sel;
  float *stage_w, *stage_y;
  // second staging slot and the host-side machinery of the pipelined host entry point
  void* stage_hidden2;
  int32_t* stage_sel2;
  float *stage_w2, *stage_y2;
  cudaStream_t pipe_in, pipe_out, pipe_prep;   // copy streams and the stream of routing + grouping, created on first use
  cudaEvent_t pipe_h2d[2], pipe_done[2], pipe_compute[2], pipe_prep_done[2], pipe_sync;
  int pipe_ready, pipe_slot, pipe_busy[2], pipe_used[2];
  // borrowed weights
  const float *Wr, *fixed_delta;
  const void *Wg, *Wu, *Wd, *shWg, *shWu, *shWd;
  // optional per-token miss trace (caller's buffer)
  uint32_t* miss_trace;
  int64_t trace_cap, trace_pos;
  // host-side counters
  uint64_t tok, delta_cnt, steps_since_reset;
  int last_cuda;
  int use_tc;
  TcPlan tc;
  int use_tc_router;
  RouterGemmPlan rg;
  void* wr_terms;
  float* z_buf;
  float* z_acc;
  size_t z_acc_bytes;   // the accumulation array and, behind it, the counters of the fused routing kernel
  uint32_t* z_ready;
  // optional per-kernel timing: event pairs recorded around each launch, summed by mcce_profile_read
  int profiling;
  int n_pairs;
  cudaEvent_t ev[kMaxPairs][2];
  int ev_kind[kMaxPairs];
  double prof_ms[MCCE_N_KERNELS];
  int64_t prof_launches[MCCE_N_KERNELS];
};

namespace {

constexpr size_t kAlign = 256;
size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool valid(const mcce_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->n_streams < 1) return false;
  if (c->n_experts < 1 || c->n_experts > kMaxE) return false;
  if (c->top_k < 1 || c->top_k > kMaxK || c->top_k > c->n_experts) return false;
  if (c->top_j < 0 || c->top_j > c->top_k) return false;
  if (c->n_shared < 0 || c->cache_capacity < 1) return false;
  if (c->d_model < 8 || c->d_model % 8 || c->d_ff < 8 || c->d_ff % 8) return false;
  if (!(c->lambda >= 0.f) || !isfinite(c->lambda)) return false;
  if (c->delta_mode != MCCE_DELTA_RUNNING && c->delta_mode != MCCE_DELTA_FIXED) return false;
  if (c->hidden_dtype != MCCE_F32 && c->hidden_dtype != MCCE_BF16) return false;
  if (c->weight_dtype != c->hidden_dtype) return false;
  if (c->ffn_impl < MCCE_FFN_AUTO || c->ffn_impl > MCCE_FFN_TENSOR) return false;
  if (c->ffn_impl == MCCE_FFN_TENSOR && !tc_applicable(*c)) return false;
  if (c->device < 0) return false;
  if (c->rerank_mode < MCCE_RERANK_CACHE_PRIOR || c->rerank_mode > MCCE_RERANK_CUMSUM) return false;
  if (c->rerank_mode == MCCE_RERANK_MAX_RANK && (c->max_rank < 0 || c->max_rank > c->n_experts)) return false;
  if (c->rerank_mode == MCCE_RERANK_CUMSUM && !(c->cum_threshold >= 0.f)) return false;
  if (c->track_lifetime != 0 && c->track_lifetime != 1) return false;
  if (c->route_impl < MCCE_ROUTE_AUTO || c->route_impl > MCCE_ROUTE_FUSED) return false;
  if ((c->deterministic != 0 && c->deterministic != 1) || (c->checked != 0 && c->checked != 1)) return false;
  return true;
}

struct Layout {
  size_t stamp, ever, sum_range, miss, cold, err, stats, offsets, perm, inv, offsets2, perm2, inv2, group_counts, Xg, Xg2, H, O, st_hidden, st_sel, st_w, st_y, st_hidden2, st_sel2, st_w2, st_y2,
      wr_terms, z_buf, z_acc, z_ready, load_tok, life, total;
};

Layout layout_of(const mcce_config& c) {
  const size_t L = c.n_layers, S = c.n_streams, E = c.n_experts, K = c.top_k, d = c.d_model, I = c.d_ff;
  const size_t EW = (E + 31) / 32, esz = c.hidden_dtype == MCCE_BF16 ? 2 : 4;
  const size_t rows = L * S * K + L * (size_t)c.n_shared * S;
  Layout o;
  size_t p = 0;
  auto take = [&](size_t bytes) {
    const size_t at = p;
    p += up(bytes);
    return at;
  };
  o.stamp = take(L * S * E * 4);
  o.ever = take(L * S * EW * 4);
  o.sum_range = take(L * S * 4);
  o.miss = take(L * S * 4);
  o.cold = take(L * S * 4);
  o.err = take(64);
  o.stats = take(L * 2 * 8);
  o.offsets = take(L * (E + 1) * 4);
  o.perm = take(L * S * K * 4);
  o.inv = take(L * S * K * 4);
  o.offsets2 = take(L * (E + 1) * 4);
  o.perm2 = take(L * S * K * 4);
  o.inv2 = take(L * S * K * 4);
  o.group_counts = take((L * (size_t)group_chunks((int)S, (int)K) * E + L) * 4);   // histograms, then a ticket per layer
  o.Xg = take((L * S * K + 256) * d * esz);  // slack rows: tensor-core tiles read past a group's end
  o.Xg2 = take((L * S * K + 256) * d * esz);
  o.H = take((rows + 256) * I * esz);
  // per-pair expert outputs are needed by the fp32-pipe path and by the deterministic mode (otherwise the
  // tensor path combines in its epilogue)
  const bool tensor_ffn = c.ffn_impl != MCCE_FFN_SIMT && tc_applicable(c);
  o.O = take(tensor_ffn && !c.deterministic ? 0 : rows * d * 4);
  o.st_hidden = take(L * S * d * esz);
  o.st_sel = take(L * S * K * 4);
  o.st_w = take(L * S * K * 4);
  o.st_y = take(L * S * d * 4);
  o.st_hidden2 = take(L * S * d * esz);
  o.st_sel2 = take(L * S * K * 4);
  o.st_w2 = take(L * S * K * 4);
  o.st_y2 = take(L * S * d * 4);
  const bool rg = router_gemm_applicable(c);
  o.wr_terms = take(rg ? 3 * L * E * d * 2 : 0);
  // logits of up to router_gemm_steps_max() tokens; the router-resident kernels write one array per K part
  const size_t z_slots = (size_t)router_gemm_steps_max() * (router_gemm_res_applicable(c) ? router_gemm_res_parts_max() : 1);
  o.z_buf = take(rg ? z_slots * L * S * E * 4 : 0);
  // the array the fused kernel accumulates a launch's logits in (zero between launches)
  o.z_acc = take(rg ? (size_t)router_gemm_steps_max() * L * S * E * 4 : 0);
  o.z_ready = take(rg ? route_fused_counter_words((int)L, router_gemm_steps_max(), (int)S) * 4 : 0);   // counters of the fused kernel
  o.load_tok = take(c.track_lifetime ? L * S * E * 4 : 0);
  o.life = take(c.track_lifetime ? L * S * 3 * 8 : 0);
  o.total = p;
  return o;
}

bool use_fused(const mcce_ctx* ctx, int n_tokens) {
  // (the checked mode looks at the logits after the routing pass: the fused kernel does not keep them; its
  // logits are sums in order of arrival, which the deterministic mode rules out)
  if (!ctx->rg.fused_ready || ctx->cfg.route_impl == MCCE_ROUTE_TWO_KERNELS || ctx->cfg.checked || ctx->cfg.deterministic)
    return false;
  if (ctx->cfg.route_impl == MCCE_ROUTE_FUSED) return true;
  return n_tokens >= kFusedMinTokens;
}

int cuda_fail(mcce_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda = (int)e;
  return MCCE_ECUDA;
}
#define CK(call)                                      \
  do {                                                \
    cudaError_t e_ = (call);                          \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_); \
  } while (0)

// Folds the recorded event pairs into the per-kernel sums (synchronises on the last event).
int drain_events(mcce_ctx* ctx) {
  for (int i = 0; i < ctx->n_pairs; ++i) {
    float ms = 0.f;
    CK(cudaEventSynchronize(ctx->ev[i][1]));
    CK(cudaEventElapsedTime(&ms, ctx->ev[i][0], ctx->ev[i][1]));
    ctx->prof_ms[ctx->ev_kind[i]] += ms;
    ctx->prof_launches[ctx->ev_kind[i]] += 1;
  }
  ctx->n_pairs = 0;
  return MCCE_OK;
}

// Runs `launch` between two events on `st` when profiling is on.
template <typename F>
int timed(mcce_ctx* ctx, int kind, cudaStream_t st, F launch) {
  if (!ctx->profiling) {
    CK(launch());
    return MCCE_OK;
  }
  if (ctx->n_pairs == kMaxPairs) {
    const int rc = drain_events(ctx);
    if (rc != MCCE_OK) return rc;
  }
  const int i = ctx->n_pairs;
  CK(cudaEventRecord(ctx->ev[i][0], st));
  CK(launch());
  CK(cudaEventRecord(ctx->ev[i][1], st));
  ctx->ev_kind[i] = kind;
  ctx->n_pairs = i + 1;
  return MCCE_OK;
}
#define TIMED(kind, st, expr)                                   \
  do {                                                          \
    const int rc_ = timed(ctx, kind, st, [&]() { return expr; }); \
    if (rc_ != MCCE_OK) return rc_;                             \
  } while (0)

FfnParams ffn_params(const mcce_ctx* ctx, int slot, const void* hidden, const float* sel_w, float* y) {
  const mcce_config& c = ctx->cfg;
  FfnParams f;
  f.L = c.n_layers, f.S = c.n_streams, f.E = c.n_experts, f.K = c.top_k, f.n_sh = c.n_shared, f.l0 = 0;
  f.d = c.d_model, f.I = c.d_ff, f.bf16 = c.hidden_dtype == MCCE_BF16;
  f.hidden = hidden;
  f.Wg = ctx->Wg, f.Wu = ctx->Wu, f.Wd = ctx->Wd, f.shWg = ctx->shWg, f.shWu = ctx->shWu, f.shWd = ctx->shWd;
  f.slot = slot;
  f.offsets = ctx->gb[slot].offsets, f.perm = ctx->gb[slot].perm, f.inv = ctx->gb[slot].inv, f.sel_w = sel_w;
  f.Xg = ctx->gb[slot].Xg, f.H = ctx->H, f.O = ctx->O, f.y = y;
  return f;
}

// Checked mode, after the routing launches of tokens whose logits lie in z (n floats; null when the route
// kernel formed them itself and checked them on the way): logits finite, cache states consistent.
int check_after_route(mcce_ctx* ctx, const float* z, size_t n, cudaStream_t st) {
  const mcce_config& c = ctx->cfg;
  if (z && n) CK(launch_check_finite(z, n, ctx->err + 2, st));
  CK(launch_check_state(ctx->stamp, (size_t)c.n_layers * c.n_streams, c.n_experts, c.cache_capacity, ctx->err + 1, st));
  return MCCE_OK;
}

}  // namespace

extern "C" size_t mcce_workspace_bytes(const mcce_config* cfg) { return valid(cfg) ? layout_of(*cfg).total : 0; }

extern "C" int mcce_create(const mcce_config* cfg, void* workspace, size_t workspace_bytes, mcce_ctx** out) {
  if (!out) return MCCE_EINVAL;
  *out = nullptr;
  if (!valid(cfg) || !workspace || ((uintptr_t)workspace % kAlign)) return MCCE_EINVAL;
  const Layout lo = layout_of(*cfg);
  if (workspace_bytes < lo.total) return MCCE_ENOSPC;
  mcce_ctx* ctx = new (std::nothrow) mcce_ctx();
  if (!ctx) return MCCE_EINVAL;
  memset(ctx, 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  ctx->EW = (cfg->n_experts + 31) / 32;
  ctx->rows = (size_t)cfg->n_layers * cfg->n_streams * cfg->top_k + (size_t)cfg->n_layers * cfg->n_shared * cfg->n_streams;
  char* w = (char*)workspace;
  ctx->stamp = (uint32_t*)(w + lo.stamp), ctx->ever = (uint32_t*)(w + lo.ever);
  ctx->sum_range = (float*)(w + lo.sum_range);
  ctx->miss = (uint32_t*)(w + lo.miss), ctx->cold = (uint32_t*)(w + lo.cold), ctx->err = (uint32_t*)(w + lo.err);
  ctx->stats_dev = (unsigned long long*)(w + lo.stats);
  ctx->gb[0].offsets = (int32_t*)(w + lo.offsets), ctx->gb[0].perm = (int32_t*)(w + lo.perm);
  ctx->gb[0].inv = (int32_t*)(w + lo.inv), ctx->gb[0].Xg = w + lo.Xg;
  ctx->gb[1].offsets = (int32_t*)(w + lo.offsets2), ctx->gb[1].perm = (int32_t*)(w + lo.perm2);
  ctx->gb[1].inv = (int32_t*)(w + lo.inv2), ctx->gb[1].Xg = w + lo.Xg2;
  ctx->group_counts = (int*)(w + lo.group_counts);
  ctx->H = w + lo.H, ctx->O = (float*)(w + lo.O);
  ctx->stage_hidden = w + lo.st_hidden, ctx->stage_sel = (int32_t*)(w + lo.st_sel);
  ctx->stage_w = (float*)(w + lo.st_w), ctx->stage_y = (float*)(w + lo.st_y);
  ctx->stage_hidden2 = w + lo.st_hidden2, ctx->stage_sel2 = (int32_t*)(w + lo.st_sel2);
  ctx->stage_w2 = (float*)(w + lo.st_w2), ctx->stage_y2 = (float*)(w + lo.st_y2);
  ctx->use_tc = cfg->ffn_impl != MCCE_FFN_SIMT && tc_applicable(*cfg);
  ctx->use_tc_router = router_gemm_applicable(*cfg);
  ctx->wr_terms = w + lo.wr_terms, ctx->z_buf = (float*)(w + lo.z_buf), ctx->z_acc = (float*)(w + lo.z_acc), ctx->z_acc_bytes = lo.load_tok - lo.z_acc, ctx->z_ready = (uint32_t*)(w + lo.z_ready);
  ctx->load_tok = cfg->track_lifetime ? (uint32_t*)(w + lo.load_tok) : nullptr;
  ctx->life = cfg->track_lifetime ? (unsigned long long*)(w + lo.life) : nullptr;
  cudaError_t e = cudaSetDevice(cfg->device);
  // state arrays and the activation buffers start at zero (the slack rows must hold finite values)
  if (e == cudaSuccess) e = cudaMemset(w, 0, lo.O);
  if (e == cudaSuccess && cfg->track_lifetime) e = cudaMemset(w + lo.load_tok, 0, lo.total - lo.load_tok);
  if (e == cudaSuccess && ctx->z_acc_bytes) e = cudaMemset(ctx->z_acc, 0, ctx->z_acc_bytes);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    delete ctx;
    return MCCE_ECUDA;
  }
  *out = ctx;
  return MCCE_OK;
}

extern "C" int mcce_destroy(mcce_ctx* ctx) {
  if (!ctx) return MCCE_EINVAL;
  if (ctx->pipe_ready) {
    mcce_pipeline_wait(ctx);
    cudaStreamSynchronize(ctx->pipe_prep);
    cudaStreamDestroy(ctx->pipe_in);
    cudaStreamDestroy(ctx->pipe_out);
    cudaStreamDestroy(ctx->pipe_prep);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(ctx->pipe_h2d[i]);
      cudaEventDestroy(ctx->pipe_done[i]);
      cudaEventDestroy(ctx->pipe_compute[i]);
      cudaEventDestroy(ctx->pipe_prep_done[i]);
    }
    cudaEventDestroy(ctx->pipe_sync);
  }
  if (ctx->profiling)
    for (int i = 0; i < kMaxPairs; ++i) {
      cudaEventDestroy(ctx->ev[i][0]);
      cudaEventDestroy(ctx->ev[i][1]);
    }
  delete ctx;
  return MCCE_OK;
}

extern "C" int mcce_set_router(mcce_ctx* ctx, const float* Wr, const float* fixed_delta) {
  if (!ctx || !Wr) return MCCE_EINVAL;
  if (ctx->cfg.delta_mode == MCCE_DELTA_FIXED && !fixed_delta) return MCCE_EINVAL;
  if ((uintptr_t)Wr % 16) return MCCE_EINVAL;
  ctx->Wr = Wr;
  ctx->fixed_delta = fixed_delta;
  if (ctx->use_tc_router) {
    CK(cudaSetDevice(ctx->cfg.device));
    const int rc = router_gemm_plan(ctx->cfg, Wr, ctx->wr_terms, &ctx->rg, 0);
    if (rc != MCCE_OK) return rc;
    if (router_gemm_res_applicable(ctx->cfg)) {
      const int rc2 = router_gemm_res_plan(ctx->cfg, ctx->wr_terms, &ctx->rg);
      if (rc2 != MCCE_OK) return rc2;
      const int rc3 = route_fused_plan(ctx->cfg, &ctx->rg);
      if (rc3 != MCCE_OK) return rc3;
    }
    CK(cudaDeviceSynchronize());
  }
  return MCCE_OK;
}

extern "C" int mcce_set_experts(mcce_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* shWg,
                                const void* shWu, const void* shWd) {
  if (!ctx || !Wg || !Wu || !Wd) return MCCE_EINVAL;
  if (ctx->cfg.n_shared > 0 && (!shWg || !shWu || !shWd)) return MCCE_EINVAL;
  const void* all[6] = {Wg, Wu, Wd, shWg, shWu, shWd};
  for (const void* q : all)
    if ((uintptr_t)q % 16) return MCCE_EINVAL;
  ctx->Wg = Wg, ctx->Wu = Wu, ctx->Wd = Wd, ctx->shWg = shWg, ctx->shWu = shWu, ctx->shWd = shWd;
  if (ctx->use_tc) {
    const int rc = tc_plan(ctx->cfg, Wg, Wu, Wd, shWg, shWu, shWd, ctx->gb[0].Xg, ctx->gb[1].Xg, ctx->H, &ctx->tc);
    if (rc != MCCE_OK) return rc;
  }
  return MCCE_OK;
}

extern "C" int mcce_reset(mcce_ctx* ctx, const int32_t* init_order, int keep_delta_stats, const float* delta_sum,
                          int64_t delta_count) {
  if (!ctx) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  const size_t LS = (size_t)c.n_layers * c.n_streams, E = c.n_experts, C = c.cache_capacity, EW = ctx->EW;
  if (delta_sum && delta_count < 0) return MCCE_EINVAL;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  std::vector<uint32_t> stamp(LS * E, 0u), ever(LS * EW, 0u);
  if (init_order) {
    for (size_t p = 0; p < LS; ++p)
      for (size_t r = 0; r < C; ++r) {
        const int32_t e = init_order[p * C + r];
        if (e < 0) continue;
        if ((size_t)e >= E || stamp[p * E + e] != 0u) return MCCE_EINVAL;
        if (r >= E) return MCCE_EINVAL;
        stamp[p * E + e] = (uint32_t)(E - r);  // 1..E, below every later touch (> E); MRU largest
        ever[p * EW + e / 32] |= 1u << (e % 32);
      }
  }
  CK(cudaMemcpy(ctx->stamp, stamp.data(), stamp.size() * 4, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(ctx->ever, ever.data(), ever.size() * 4, cudaMemcpyHostToDevice));
  CK(cudaMemset(ctx->miss, 0, LS * 4));
  CK(cudaMemset(ctx->cold, 0, LS * 4));
  CK(cudaMemset(ctx->err, 0, 64));
  // a fused routing launch that gave up may have left sums and counts behind (the counters follow the sums)
  if (ctx->z_acc_bytes) CK(cudaMemset(ctx->z_acc, 0, ctx->z_acc_bytes));
  if (ctx->load_tok) {
    CK(cudaMemset(ctx->load_tok, 0, LS * E * 4));
    CK(cudaMemset(ctx->life, 0, LS * 3 * 8));
  }
  if (delta_sum) {
    CK(cudaMemcpy(ctx->sum_range, delta_sum, LS * 4, cudaMemcpyHostToDevice));
    ctx->delta_cnt = (uint64_t)delta_count;
  } else if (!keep_delta_stats) {
    CK(cudaMemset(ctx->sum_range, 0, LS * 4));
    ctx->delta_cnt = 0;
  }
  ctx->tok = 0;
  ctx->steps_since_reset = 0;
  ctx->trace_pos = 0;
  CK(cudaDeviceSynchronize());
  return MCCE_OK;
}

extern "C" int mcce_route_step(mcce_ctx* ctx, int32_t n_steps, const void* hidden, const float* logits_in,
                               int32_t* sel_idx, float* sel_w, float* logits_out, void* cuda_stream) {
  if (!ctx || n_steps < 0 || !sel_idx || !sel_w) return MCCE_EINVAL;
  if ((hidden == nullptr) == (logits_in == nullptr)) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  if (hidden && !ctx->Wr) return MCCE_ESTATE;
  if (c.delta_mode == MCCE_DELTA_FIXED && !ctx->fixed_delta) return MCCE_ESTATE;
  // rows of logits are read and written four floats at a time when E is a multiple of 4
  const uintptr_t z_align = (c.n_experts & 3) ? 4 : 16;
  if (((uintptr_t)logits_in % z_align) || ((uintptr_t)logits_out % z_align)) return MCCE_EINVAL;
  if (hidden && ((uintptr_t)hidden % 16)) return MCCE_EINVAL;
  if (n_steps == 0) return MCCE_OK;
  // recency keys and the Delta count are 32-bit on the device
  const uint64_t last_key = (uint64_t)c.n_experts + (ctx->tok + n_steps) * (uint64_t)c.top_k + c.top_k + 1;
  if (last_key >= 0xffffffffull || ctx->delta_cnt + n_steps >= 0xffffffffull) return MCCE_ESTATE;
  RouteParams p;
  p.L = c.n_layers, p.S = c.n_streams, p.E = c.n_experts, p.K = c.top_k, p.J = c.top_j, p.C = c.cache_capacity;
  p.d = c.d_model, p.lambda = c.lambda, p.delta_mode = c.delta_mode, p.renorm = c.renorm;
  p.rerank_mode = c.rerank_mode, p.max_rank = c.max_rank, p.cum_threshold = c.cum_threshold;
  p.hidden_bf16 = c.hidden_dtype == MCCE_BF16;
  p.Wr = ctx->Wr, p.fixed_delta = ctx->fixed_delta;
  p.stamp = ctx->stamp, p.ever = ctx->ever, p.sum_range = ctx->sum_range, p.miss = ctx->miss, p.cold = ctx->cold;
  p.load_tok = ctx->load_tok, p.life = ctx->life;
  p.err_nonfinite = c.checked ? ctx->err + 2 : nullptr;
  const size_t LS_trace = (size_t)c.n_layers * c.n_streams;
  auto trace_at = [&](int t0, int nt) {   // where tokens [t0, t0+nt) of this call go in the trace buffer
    const int64_t pos = ctx->trace_pos + t0;
    const bool on = ctx->miss_trace && pos < ctx->trace_cap;
    p.miss_trace = on ? ctx->miss_trace + (size_t)pos * LS_trace : nullptr;
    p.trace_avail = on ? (int)(ctx->trace_cap - pos < nt ? ctx->trace_cap - pos : nt) : 0;
  };
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (hidden && ctx->use_tc_router && ctx->rg.ready) {
    // logits by the tensor-core GEMM, a few tokens at a time, then the fused tail on those logits
    const size_t LS = (size_t)c.n_layers * c.n_streams, esz = 2;
    for (int t0 = 0; t0 < n_steps; t0 += router_gemm_steps_max()) {
      const int nt = n_steps - t0 < router_gemm_steps_max() ? n_steps - t0 : router_gemm_steps_max();
      const char* h = (const char*)hidden + (size_t)t0 * LS * c.d_model * esz;
      int ks = 1;
      p.tok0 = (uint32_t)(ctx->tok + t0), p.cnt0 = (uint32_t)(ctx->delta_cnt + t0);
      p.sel_idx = sel_idx + (size_t)t0 * LS * c.top_k, p.sel_w = sel_w + (size_t)t0 * LS * c.top_k;
      p.logits_out = logits_out ? logits_out + (size_t)t0 * LS * c.n_experts : nullptr;
      trace_at(t0, nt);
      // GEMM and tail in one kernel once there are a few tokens to overlap them over
      if (use_fused(ctx, nt)) {
        cudaError_t fe = cudaSuccess;
        const int rc_f = timed(ctx, MCCE_K_ROUTE, st, [&]() {
          fe = route_fused_launch(ctx->rg, c, h, nt, ctx->z_acc, ctx->z_ready, p, ctx->err, st);
          return fe == cudaErrorCooperativeLaunchTooLarge ? cudaSuccess : fe;
        });
        if (rc_f != MCCE_OK) return rc_f;
        if (fe == cudaSuccess) continue;
        // the device cannot hold the whole grid at once (it is shared with other work): two kernels from now on
        cudaGetLastError();
        ctx->rg.fused_ready = 0;
      }
      if (ctx->rg.res_ready) {
        TIMED(MCCE_K_ROUTE_GEMM, st, router_gemm_res_launch(ctx->rg, c, h, nt, ctx->z_buf, &ks, ctx->err, st));
      } else {
        TIMED(MCCE_K_ROUTE_GEMM, st, router_gemm_launch(ctx->rg, c, h, nt, ctx->z_buf, &ks, ctx->err, st));
      }
      p.n_steps = nt, p.hidden = nullptr, p.logits_in = ctx->z_buf;
      p.n_partials = ks, p.partial_stride = (size_t)nt * LS * c.n_experts;
      p.sel_idx = sel_idx + (size_t)t0 * LS * c.top_k, p.sel_w = sel_w + (size_t)t0 * LS * c.top_k;
      p.logits_out = logits_out ? logits_out + (size_t)t0 * LS * c.n_experts : nullptr;
      p.tok0 = (uint32_t)(ctx->tok + t0), p.cnt0 = (uint32_t)(ctx->delta_cnt + t0);
      trace_at(t0, nt);
      TIMED(MCCE_K_ROUTE, st, launch_route(p, st));
      if (c.checked) {
        const int rc_c = check_after_route(ctx, ctx->z_buf, (size_t)ks * nt * LS * c.n_experts, st);
        if (rc_c != MCCE_OK) return rc_c;
      }
    }
  } else {
    p.n_steps = n_steps, p.hidden = hidden, p.logits_in = logits_in, p.n_partials = 1, p.partial_stride = 0;
    p.sel_idx = sel_idx, p.sel_w = sel_w, p.logits_out = logits_out;
    p.tok0 = (uint32_t)ctx->tok, p.cnt0 = (uint32_t)ctx->delta_cnt;
    trace_at(0, n_steps);
    TIMED(MCCE_K_ROUTE, st, launch_route(p, st));
    if (c.checked) {
      const int rc_c = check_after_route(ctx, logits_in, logits_in ? (size_t)n_steps * c.n_layers * c.n_streams * c.n_experts : 0, st);
      if (rc_c != MCCE_OK) return rc_c;
    }
  }
  ctx->tok += n_steps;
  ctx->steps_since_reset += n_steps;
  if (ctx->miss_trace) ctx->trace_pos += n_steps;
  if (c.delta_mode == MCCE_DELTA_RUNNING) ctx->delta_cnt += n_steps;
  return MCCE_OK;
}

// Expert forward for model layers [l0, l0 + Ls): hidden, sel_idx, sel_w and y hold those layers only.  The
// grouping, gathered rows and intermediates use the front of the context's buffers (set `slot` of the grouping
// buffers); only the expert weights are addressed by model layer.  Two halves, which the pipelined entry points
// put on different streams: the grouping pass with its row copy, and the expert kernels.
static int group_layers(mcce_ctx* ctx, int slot, int Ls, const void* hidden, const int32_t* sel_idx, float* y,
                        cudaStream_t st) {
  const mcce_config& c = ctx->cfg;
  GroupParams g;
  g.L = Ls, g.S = c.n_streams, g.E = c.n_experts, g.K = c.top_k;
  g.sel_idx = sel_idx, g.offsets = ctx->gb[slot].offsets, g.perm = ctx->gb[slot].perm, g.inv = ctx->gb[slot].inv;
  g.err_index = ctx->err + 1;
  int* tickets = ctx->group_counts + (size_t)c.n_layers * group_chunks(c.n_streams, c.top_k) * c.n_experts;
  TIMED(MCCE_K_GROUP, st, launch_group(g, ctx->group_counts, tickets, st));
  FfnParams f = ffn_params(ctx, slot, hidden, nullptr, y);
  f.L = Ls;
  // on the tensor path the down kernel adds w * E_i(x) into y itself: the grouping pass clears y on the way;
  // in the deterministic mode it stores rows of O instead and the combine pass writes every element of y
  const bool atomic_combine = ctx->use_tc && !c.deterministic;
  TIMED(MCCE_K_GATHER, st, launch_place(g, f, ctx->group_counts, atomic_combine, st));
  if (c.checked) CK(launch_check_group(g, st));
  ctx->last_slot = slot;
  return MCCE_OK;
}

static int expert_layers(mcce_ctx* ctx, int slot, int l0, int Ls, const void* hidden, const float* sel_w, float* y,
                         cudaStream_t st) {
  const mcce_config& c = ctx->cfg;
  FfnParams f = ffn_params(ctx, slot, hidden, sel_w, y);
  f.L = Ls, f.l0 = l0;
  const bool atomic_combine = ctx->use_tc && !c.deterministic;
  if (ctx->use_tc) {
    TIMED(MCCE_K_FFN_UP, st, tc_launch_up(ctx->tc, f, ctx->err, st));
    TIMED(MCCE_K_FFN_DOWN, st, tc_launch_down(ctx->tc, f, !atomic_combine, ctx->err, st));
    if (!atomic_combine) TIMED(MCCE_K_COMBINE, st, launch_combine(f, st));
  } else {
    TIMED(MCCE_K_FFN_UP, st, launch_ffn_simt_up(f, st));
    TIMED(MCCE_K_FFN_DOWN, st, launch_ffn_simt_down(f, st));
    TIMED(MCCE_K_COMBINE, st, launch_combine(f, st));
  }
  return MCCE_OK;
}

static int forward_layers(mcce_ctx* ctx, int l0, int Ls, const void* hidden, const int32_t* sel_idx,
                          const float* sel_w, float* y, cudaStream_t st) {
  const int rc = group_layers(ctx, 0, Ls, hidden, sel_idx, y, st);
  return rc != MCCE_OK ? rc : expert_layers(ctx, 0, l0, Ls, hidden, sel_w, y, st);
}

extern "C" int mcce_moe_forward(mcce_ctx* ctx, const void* hidden, const int32_t* sel_idx, const float* sel_w,
                                float* y, void* cuda_stream) {
  if (!ctx || !hidden || !sel_idx || !sel_w || !y) return MCCE_EINVAL;
  if (!ctx->Wg) return MCCE_ESTATE;
  if (((uintptr_t)hidden % 16) || ((uintptr_t)y % 16)) return MCCE_EINVAL;
  return forward_layers(ctx, 0, ctx->cfg.n_layers, hidden, sel_idx, sel_w, y, (cudaStream_t)cuda_stream);
}

extern "C" int mcce_pipeline_wait(mcce_ctx* ctx);

// ---- sequential-layer mode: the layers of one token chained through a residual stream --------------------
// Routing of model layer l from its input x [S,d]: the same kernels as mcce_route_step, launched for one layer.
static int route_one_layer(mcce_ctx* ctx, int l, const void* x, int32_t* sel, float* w, cudaStream_t st) {
  const mcce_config& c = ctx->cfg;
  const size_t S = c.n_streams, E = c.n_experts, EW = ctx->EW;
  RouteParams p;
  p.L = 1, p.S = c.n_streams, p.E = c.n_experts, p.K = c.top_k, p.J = c.top_j, p.C = c.cache_capacity;
  p.d = c.d_model, p.n_steps = 1, p.lambda = c.lambda, p.delta_mode = c.delta_mode, p.renorm = c.renorm;
  p.rerank_mode = c.rerank_mode, p.max_rank = c.max_rank, p.cum_threshold = c.cum_threshold;
  p.hidden_bf16 = c.hidden_dtype == MCCE_BF16;
  p.Wr = ctx->Wr + (size_t)l * E * c.d_model;
  p.fixed_delta = ctx->fixed_delta ? ctx->fixed_delta + l : nullptr;
  p.stamp = ctx->stamp + (size_t)l * S * E, p.ever = ctx->ever + (size_t)l * S * EW;
  p.sum_range = ctx->sum_range + (size_t)l * S, p.miss = ctx->miss + (size_t)l * S, p.cold = ctx->cold + (size_t)l * S;
  p.load_tok = ctx->load_tok ? ctx->load_tok + (size_t)l * S * E : nullptr;
  p.life = ctx->life ? ctx->life + (size_t)l * S * 3 : nullptr;
  const bool trace = ctx->miss_trace && ctx->trace_pos < ctx->trace_cap;
  p.miss_trace = trace ? ctx->miss_trace + ((size_t)ctx->trace_pos * c.n_layers + l) * S : nullptr;
  p.trace_avail = trace ? 1 : 0;
  p.sel_idx = sel, p.sel_w = w, p.logits_out = nullptr;
  p.tok0 = (uint32_t)ctx->tok, p.cnt0 = (uint32_t)ctx->delta_cnt;
  p.err_nonfinite = c.checked ? ctx->err + 2 : nullptr;
  int ks = 0;
  if (ctx->use_tc_router && ctx->rg.ready) {
    ks = 1;
    // the kernel a one-layer context would launch for this layer
    if (ctx->rg.res_ready)
      TIMED(MCCE_K_ROUTE_GEMM, st, router_gemm_res_launch(ctx->rg, c, x, 1, ctx->z_buf, &ks, ctx->err, st, l, 1));
    else
      TIMED(MCCE_K_ROUTE_GEMM, st, router_gemm_launch(ctx->rg, c, x, 1, ctx->z_buf, &ks, ctx->err, st, l, 1));
    p.hidden = nullptr, p.logits_in = ctx->z_buf, p.n_partials = ks, p.partial_stride = S * E;
  } else {
    p.hidden = x, p.logits_in = nullptr, p.n_partials = 1, p.partial_stride = 0;
  }
  TIMED(MCCE_K_ROUTE, st, launch_route(p, st));
  if (c.checked) {
    if (ks) CK(launch_check_finite(ctx->z_buf, (size_t)ks * S * E, ctx->err + 2, st));
    CK(launch_check_state(p.stamp, S, c.n_experts, c.cache_capacity, ctx->err + 1, st));
  }
  return MCCE_OK;
}

extern "C" int mcce_decode_step_chained(mcce_ctx* ctx, const void* x0, void* x_out, int32_t* sel_idx,
                                        void* cuda_stream) {
  if (!ctx || !x0 || !x_out) return MCCE_EINVAL;
  if (!ctx->Wr || !ctx->Wg) return MCCE_ESTATE;
  if (((uintptr_t)x0 % 16) || ((uintptr_t)x_out % 16)) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  if (c.delta_mode == MCCE_DELTA_FIXED && !ctx->fixed_delta) return MCCE_ESTATE;
  const uint64_t last_key = (uint64_t)c.n_experts + (ctx->tok + 1) * (uint64_t)c.top_k + c.top_k + 1;
  if (last_key >= 0xffffffffull || ctx->delta_cnt + 1 >= 0xffffffffull) return MCCE_ESTATE;
  {
    const int rcw = mcce_pipeline_wait(ctx);   // the staging buffers are used as the residual stream
    if (rcw != MCCE_OK) return rcw;
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t S = c.n_streams, K = c.top_k, n = S * c.d_model;
  const bool bf16 = c.hidden_dtype == MCCE_BF16;
  void* buf[2] = {ctx->stage_hidden, ctx->stage_hidden2};
  const void* x = x0;
  for (int l = 0; l < c.n_layers; ++l) {
    int32_t* sel = ctx->stage_sel + (size_t)l * S * K;
    float* w = ctx->stage_w + (size_t)l * S * K;
    int rc = route_one_layer(ctx, l, x, sel, w, st);
    if (rc != MCCE_OK) return rc;
    rc = forward_layers(ctx, l, 1, x, sel, w, ctx->stage_y, st);
    if (rc != MCCE_OK) return rc;
    void* nxt = l + 1 == c.n_layers ? x_out : buf[l & 1];
    CK(launch_residual(x, ctx->stage_y, nxt, n, bf16, st));
    x = nxt;
  }
  if (sel_idx)
    CK(cudaMemcpyAsync(sel_idx, ctx->stage_sel, (size_t)c.n_layers * S * K * 4, cudaMemcpyDeviceToDevice, st));
  ctx->tok += 1;
  ctx->steps_since_reset += 1;
  if (ctx->miss_trace) ctx->trace_pos += 1;
  if (c.delta_mode == MCCE_DELTA_RUNNING) ctx->delta_cnt += 1;
  return MCCE_OK;
}

extern "C" int mcce_decode_step_host(mcce_ctx* ctx, const void* hidden_host, float* y_host, int32_t* sel_idx_host,
                                     void* cuda_stream) {
  if (!ctx || !hidden_host || !y_host) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t LS = (size_t)c.n_layers * c.n_streams, esz = c.hidden_dtype == MCCE_BF16 ? 2 : 4;
  {  // this call shares the first staging slot with the pipelined entry point: let its steps finish first
    const int rcw = mcce_pipeline_wait(ctx);
    if (rcw != MCCE_OK) return rcw;
  }
  CK(cudaMemcpyAsync(ctx->stage_hidden, hidden_host, LS * c.d_model * esz, cudaMemcpyHostToDevice, st));
  int rc = mcce_route_step(ctx, 1, ctx->stage_hidden, nullptr, ctx->stage_sel, ctx->stage_w, nullptr, cuda_stream);
  if (rc != MCCE_OK) return rc;
  rc = mcce_moe_forward(ctx, ctx->stage_hidden, ctx->stage_sel, ctx->stage_w, ctx->stage_y, cuda_stream);
  if (rc != MCCE_OK) return rc;
  CK(cudaMemcpyAsync(y_host, ctx->stage_y, LS * c.d_model * 4, cudaMemcpyDeviceToHost, st));
  if (sel_idx_host)
    CK(cudaMemcpyAsync(sel_idx_host, ctx->stage_sel, LS * c.top_k * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return MCCE_OK;
}

// ---- pipelined entry points: two slots, routing + grouping of a step on a stream of their own -------------
// Routing needs only the hidden states of its token and the cache state left by the previous token's routing,
// not the previous token's experts.  So a step is split over streams: routing, grouping and the row copy of step
// t + 1 run on the internal stream `pipe_prep` while the expert kernels of step t, which stream all the weights,
// still run on the caller's stream; events order a step's two halves and guard the reuse of a slot's buffers.
static int pipe_setup(mcce_ctx* ctx) {
  if (ctx->pipe_ready) return MCCE_OK;
  CK(cudaSetDevice(ctx->cfg.device));
  CK(cudaStreamCreateWithFlags(&ctx->pipe_in, cudaStreamNonBlocking));
  CK(cudaStreamCreateWithFlags(&ctx->pipe_out, cudaStreamNonBlocking));
  CK(cudaStreamCreateWithFlags(&ctx->pipe_prep, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    CK(cudaEventCreateWithFlags(&ctx->pipe_h2d[i], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&ctx->pipe_done[i], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&ctx->pipe_compute[i], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&ctx->pipe_prep_done[i], cudaEventDisableTiming));
  }
  CK(cudaEventCreateWithFlags(&ctx->pipe_sync, cudaEventDisableTiming));
  ctx->pipe_ready = 1;
  return MCCE_OK;
}

extern "C" int mcce_pipeline_wait(mcce_ctx* ctx) {
  if (!ctx) return MCCE_EINVAL;
  if (!ctx->pipe_ready) return MCCE_OK;
  for (int i = 0; i < 2; ++i)
    if (ctx->pipe_busy[i]) {
      CK(cudaEventSynchronize(ctx->pipe_done[i]));
      ctx->pipe_busy[i] = 0;
    }
  return MCCE_OK;
}

// One step in slot i: routing + grouping of `hidden` on pipe_prep (after `after_event`, if any, and after the
// experts of the step that used the slot before), then the experts on st.  Records pipe_compute[i] on st.
static int pipe_step(mcce_ctx* ctx, int i, const void* hidden, int32_t* sel, float* w, float* y, cudaEvent_t after_event,
                     cudaStream_t st) {
  const mcce_config& c = ctx->cfg;
  if (!ctx->pipe_busy[0] && !ctx->pipe_busy[1]) {
    // the pipeline is empty: whatever the caller's stream did to this context so far comes first
    CK(cudaEventRecord(ctx->pipe_sync, st));
    CK(cudaStreamWaitEvent(ctx->pipe_prep, ctx->pipe_sync, 0));
  }
  if (after_event) CK(cudaStreamWaitEvent(ctx->pipe_prep, after_event, 0));
  if (ctx->pipe_used[i]) CK(cudaStreamWaitEvent(ctx->pipe_prep, ctx->pipe_compute[i], 0));
  int rc = mcce_route_step(ctx, 1, hidden, nullptr, sel, w, nullptr, (void*)ctx->pipe_prep);
  if (rc != MCCE_OK) return rc;
  rc = group_layers(ctx, i, c.n_layers, hidden, sel, y, ctx->pipe_prep);
  if (rc != MCCE_OK) return rc;
  CK(cudaEventRecord(ctx->pipe_prep_done[i], ctx->pipe_prep));
  CK(cudaStreamWaitEvent(st, ctx->pipe_prep_done[i], 0));
  rc = expert_layers(ctx, i, 0, c.n_layers, hidden, w, y, st);
  if (rc != MCCE_OK) return rc;
  CK(cudaEventRecord(ctx->pipe_compute[i], st));
  ctx->pipe_used[i] = 1;
  return MCCE_OK;
}

extern "C" int mcce_pipeline_submit_host(mcce_ctx* ctx, const void* hidden_host, float* y_host, int32_t* sel_idx_host,
                                         void* cuda_stream) {
  if (!ctx || !hidden_host || !y_host) return MCCE_EINVAL;
  if (!ctx->Wr || !ctx->Wg) return MCCE_ESTATE;
  int rc = pipe_setup(ctx);
  if (rc != MCCE_OK) return rc;
  const mcce_config& c = ctx->cfg;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t LS = (size_t)c.n_layers * c.n_streams, esz = c.hidden_dtype == MCCE_BF16 ? 2 : 4;
  const int i = ctx->pipe_slot;
  void* sh = i ? ctx->stage_hidden2 : ctx->stage_hidden;
  int32_t* ss = i ? ctx->stage_sel2 : ctx->stage_sel;
  float* sw = i ? ctx->stage_w2 : ctx->stage_w;
  float* sy = i ? ctx->stage_y2 : ctx->stage_y;
  // the slot's previous step (two submits ago) must have left the device before its buffers are reused
  if (ctx->pipe_busy[i]) {
    CK(cudaEventSynchronize(ctx->pipe_done[i]));
    ctx->pipe_busy[i] = 0;
  }
  CK(cudaMemcpyAsync(sh, hidden_host, LS * c.d_model * esz, cudaMemcpyHostToDevice, ctx->pipe_in));
  CK(cudaEventRecord(ctx->pipe_h2d[i], ctx->pipe_in));
  rc = pipe_step(ctx, i, sh, ss, sw, sy, ctx->pipe_h2d[i], st);
  if (rc != MCCE_OK) return rc;
  CK(cudaStreamWaitEvent(ctx->pipe_out, ctx->pipe_compute[i], 0));
  CK(cudaMemcpyAsync(y_host, sy, LS * c.d_model * 4, cudaMemcpyDeviceToHost, ctx->pipe_out));
  if (sel_idx_host) CK(cudaMemcpyAsync(sel_idx_host, ss, LS * c.top_k * 4, cudaMemcpyDeviceToHost, ctx->pipe_out));
  CK(cudaEventRecord(ctx->pipe_done[i], ctx->pipe_out));
  ctx->pipe_busy[i] = 1;
  ctx->pipe_slot = i ^ 1;
  return MCCE_OK;
}

extern "C" int mcce_pipeline_submit(mcce_ctx* ctx, const void* hidden, float* y, int32_t* sel_idx, void* hidden_ready,
                                    void* cuda_stream) {
  if (!ctx || !hidden || !y) return MCCE_EINVAL;
  if (!ctx->Wr || !ctx->Wg) return MCCE_ESTATE;
  if (((uintptr_t)hidden % 16) || ((uintptr_t)y % 16)) return MCCE_EINVAL;
  int rc = pipe_setup(ctx);
  if (rc != MCCE_OK) return rc;
  const mcce_config& c = ctx->cfg;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t LS = (size_t)c.n_layers * c.n_streams;
  const int i = ctx->pipe_slot;
  int32_t* ss = i ? ctx->stage_sel2 : ctx->stage_sel;
  float* sw = i ? ctx->stage_w2 : ctx->stage_w;
  // steps of the host-buffer entry point that still use the slot's staging buffers come first
  if (ctx->pipe_busy[i]) {
    CK(cudaEventSynchronize(ctx->pipe_done[i]));
    ctx->pipe_busy[i] = 0;
  }
  rc = pipe_step(ctx, i, hidden, ss, sw, y, (cudaEvent_t)hidden_ready, st);
  if (rc != MCCE_OK) return rc;
  if (sel_idx) CK(cudaMemcpyAsync(sel_idx, ss, LS * c.top_k * 4, cudaMemcpyDeviceToDevice, st));
  // "left the device" for this entry point: the step's last work on the caller's stream
  CK(cudaEventRecord(ctx->pipe_done[i], st));
  ctx->pipe_busy[i] = 1;
  ctx->pipe_slot = i ^ 1;
  return MCCE_OK;
}

extern "C" int mcce_cache_stats(mcce_ctx* ctx, mcce_stats* total, mcce_stats* per_layer) {
  if (!ctx || !total) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  CK(launch_stats(ctx->miss, ctx->cold, ctx->stats_dev, c.n_layers, c.n_streams, 0));
  std::vector<unsigned long long> h((size_t)c.n_layers * 2);
  CK(cudaMemcpy(h.data(), ctx->stats_dev, h.size() * 8, cudaMemcpyDeviceToHost));
  uint32_t err[4];
  CK(cudaMemcpy(err, ctx->err, sizeof(err), cudaMemcpyDeviceToHost));
  memset(total, 0, sizeof(*total));
  for (int l = 0; l < c.n_layers; ++l) {
    mcce_stats s;
    s.steps = (int64_t)ctx->steps_since_reset * c.n_streams;
    s.selections = s.steps * c.top_k;
    s.misses = (int64_t)h[2 * l];
    s.cold_misses = (int64_t)h[2 * l + 1];
    if (per_layer) per_layer[l] = s;
    total->steps += s.steps, total->selections += s.selections;
    total->misses += s.misses, total->cold_misses += s.cold_misses;
  }
  return err[0] != 0 ? MCCE_ETIMEOUT : err[1] != 0 ? MCCE_EINDEX : err[2] != 0 ? MCCE_ENONFINITE : MCCE_OK;
}

extern "C" int mcce_calibrate_delta(mcce_ctx* ctx, float* delta) {
  if (!ctx || !delta) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  if (c.delta_mode != MCCE_DELTA_RUNNING || ctx->delta_cnt == 0) return MCCE_ESTATE;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  float* out = (float*)ctx->stats_dev;   // L floats of the per-layer counter scratch (16 bytes per layer)
  CK(launch_calibrate(ctx->sum_range, c.n_layers, c.n_streams, (double)ctx->delta_cnt, out, 0));
  CK(cudaMemcpy(delta, out, (size_t)c.n_layers * 4, cudaMemcpyDeviceToHost));
  return MCCE_OK;
}

extern "C" int mcce_get_cache_state(mcce_ctx* ctx, int32_t* order, uint8_t* ever, float* delta_sum,
                                    int64_t* delta_count) {
  if (!ctx || !order) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  const size_t LS = (size_t)c.n_layers * c.n_streams, E = c.n_experts, C = c.cache_capacity, EW = ctx->EW;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  std::vector<uint32_t> stamp(LS * E), ev(LS * EW);
  CK(cudaMemcpy(stamp.data(), ctx->stamp, stamp.size() * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(ev.data(), ctx->ever, ev.size() * 4, cudaMemcpyDeviceToHost));
  std::vector<std::pair<uint32_t, int32_t>> res;
  for (size_t p = 0; p < LS; ++p) {
    res.clear();
    for (size_t e = 0; e < E; ++e)
      if (stamp[p * E + e]) res.emplace_back(stamp[p * E + e], (int32_t)e);
    // most recent (largest key) first; keys are unique
    for (size_t a = 0; a < res.size(); ++a)
      for (size_t b = a + 1; b < res.size(); ++b)
        if (res[b].first > res[a].first) std::swap(res[a], res[b]);
    for (size_t r = 0; r < C; ++r) order[p * C + r] = r < res.size() ? res[r].second : -1;
    if (ever)
      for (size_t e = 0; e < E; ++e) ever[p * E + e] = (ev[p * EW + e / 32] >> (e % 32)) & 1u;
  }
  if (delta_sum) CK(cudaMemcpy(delta_sum, ctx->sum_range, LS * 4, cudaMemcpyDeviceToHost));
  if (delta_count) *delta_count = (int64_t)ctx->delta_cnt;
  return MCCE_OK;
}

extern "C" int mcce_set_miss_trace(mcce_ctx* ctx, uint32_t* trace, int64_t capacity_tokens) {
  if (!ctx || capacity_tokens < 0 || (trace == nullptr) != (capacity_tokens == 0)) return MCCE_EINVAL;
  ctx->miss_trace = trace;
  ctx->trace_cap = capacity_tokens;
  ctx->trace_pos = 0;
  return MCCE_OK;
}

extern "C" int mcce_lifetime_stats(mcce_ctx* ctx, mcce_lifetime* total, mcce_lifetime* per_layer) {
  if (!ctx || !total) return MCCE_EINVAL;
  if (!ctx->life) return MCCE_ESTATE;
  const mcce_config& c = ctx->cfg;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  std::vector<unsigned long long> h((size_t)c.n_layers * c.n_streams * 3);
  CK(cudaMemcpy(h.data(), ctx->life, h.size() * 8, cudaMemcpyDeviceToHost));
  memset(total, 0, sizeof(*total));
  for (int l = 0; l < c.n_layers; ++l) {
    mcce_lifetime s = {0, 0, 0};
    for (int q = 0; q < c.n_streams; ++q) {
      const unsigned long long* r = &h[((size_t)l * c.n_streams + q) * 3];
      s.evictions += (int64_t)r[0], s.sum += (int64_t)r[1], s.sum_sq += (int64_t)r[2];
    }
    if (per_layer) per_layer[l] = s;
    total->evictions += s.evictions, total->sum += s.sum, total->sum_sq += s.sum_sq;
  }
  return MCCE_OK;
}

extern "C" int mcce_get_grouping(mcce_ctx* ctx, int32_t* offsets, int32_t* perm) {
  if (!ctx || !offsets || !perm) return MCCE_EINVAL;
  const mcce_config& c = ctx->cfg;
  CK(cudaSetDevice(c.device));
  CK(cudaDeviceSynchronize());
  const mcce_ctx::GroupBufs& gb = ctx->gb[ctx->last_slot];
  CK(cudaMemcpy(offsets, gb.offsets, (size_t)c.n_layers * (c.n_experts + 1) * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(perm, gb.perm, (size_t)c.n_layers * c.n_streams * c.top_k * 4, cudaMemcpyDeviceToHost));
  return MCCE_OK;
}

extern "C" int mcce_selftest_wait_timeout(mcce_ctx* ctx, uint64_t limit_ns) {
  if (!ctx || limit_ns == 0 || limit_ns > 1000000000ull) return MCCE_EINVAL;
  CK(cudaSetDevice(ctx->cfg.device));
  uint32_t* outcome = ctx->err + 8;   // a spare word of the error block
  CK(cudaMemset(outcome, 0, 4));
  CK(launch_wait_timeout_selftest(ctx->err, limit_ns, outcome, 0));
  CK(cudaDeviceSynchronize());
  uint32_t h = 0;
  CK(cudaMemcpy(&h, outcome, 4, cudaMemcpyDeviceToHost));
  return h == 2u ? MCCE_OK : MCCE_ESTATE;
}

extern "C" int mcce_uses_tensor_path(const mcce_ctx* ctx) { return ctx ? ctx->use_tc : MCCE_EINVAL; }

extern "C" int mcce_router_kernel_kind(const mcce_ctx* ctx, int32_t n_tokens) {
  if (!ctx || n_tokens < 1) return MCCE_EINVAL;
  if (!ctx->Wr) return MCCE_ESTATE;
  if (!(ctx->use_tc_router && ctx->rg.ready)) return MCCE_ROUTER_FP32_PIPE;
  const int nt = n_tokens < router_gemm_steps_max() ? n_tokens : router_gemm_steps_max();
  if (use_fused(ctx, nt)) return MCCE_ROUTER_FUSED;
  return ctx->rg.res_ready ? MCCE_ROUTER_RESIDENT_TAIL : MCCE_ROUTER_GEMM_TAIL;
}

extern "C" int mcce_profile(mcce_ctx* ctx, int enable) {
  if (!ctx) return MCCE_EINVAL;
  CK(cudaSetDevice(ctx->cfg.device));
  if (enable && !ctx->profiling) {
    for (int i = 0; i < kMaxPairs; ++i) {
      CK(cudaEventCreate(&ctx->ev[i][0]));
      CK(cudaEventCreate(&ctx->ev[i][1]));
    }
    ctx->n_pairs = 0;
  } else if (!enable && ctx->profiling) {
    const int rc = drain_events(ctx);
    if (rc != MCCE_OK) return rc;
    for (int i = 0; i < kMaxPairs; ++i) {
      cudaEventDestroy(ctx->ev[i][0]);
      cudaEventDestroy(ctx->ev[i][1]);
    }
  }
  ctx->profiling = enable != 0;
  return MCCE_OK;
}

extern "C" int mcce_profile_read(mcce_ctx* ctx, double* ms, int64_t* launches, int reset) {
  if (!ctx || !ms || !launches) return MCCE_EINVAL;
  const int rc = drain_events(ctx);
  if (rc != MCCE_OK) return rc;
  for (int k = 0; k < MCCE_N_KERNELS; ++k) {
    ms[k] = ctx->prof_ms[k];
    launches[k] = ctx->prof_launches[k];
    if (reset) ctx->prof_ms[k] = 0.0, ctx->prof_launches[k] = 0;
  }
  return MCCE_OK;
}

extern "C" const char* mcce_strerror(int code) {
  switch (code) {
    case MCCE_OK: return "ok";
    case MCCE_EINVAL: return "invalid argument or unsupported configuration";
    case MCCE_ENOSPC: return "workspace too small";
    case MCCE_ESTATE:
      return "weights not set, a feature not enabled in the configuration, or a 32-bit recency counter would "
             "overflow (call mcce_reset)";
    case MCCE_ECUDA: return "CUDA call failed (see mcce_last_cuda_error)";
    case MCCE_ETIMEOUT: return "a bounded wait inside a kernel gave up";
    case MCCE_EINDEX:
      return "an expert id outside [0, E) was skipped by the grouping pass, or a consistency check of the checked "
             "mode failed (grouping position, cache occupancy or recency keys)";
    case MCCE_ENONFINITE: return "a router logit was NaN or infinite (checked mode)";
    case MCCE_ELIMIT:
      return "the cache state of this configuration exceeds the fixed 4 MiB array of mcce_route_trace_static "
             "(use mcce_create with a workspace instead)";
    default: return "unknown error";
  }
}

extern "C" int mcce_last_cuda_error(const mcce_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }
