// Routing without a context and without any allocation: the fused route kernel run over a trace of
// tokens from an empty cache, with the per-(stream, layer) cache state it needs held in a fixed array
// that is part of the library image instead of in a caller-provided workspace.
//
// Who this is for: code that may not allocate device memory at the point where it needs routing
// decisions -- a serving process whose memory pool already owns the whole GPU (a further cudaMalloc
// fails or fragments the pool), a plug-in that is only handed input and output buffers, or a callback
// on a latency-critical path where the allocator's implicit synchronisation is not acceptable.
#include "common.cuh"

namespace mcce {
namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;  // 4 MiB, held by every GPU that loads the library
constexpr int kMaxDevices = 64;
constexpr int kMaxLayersForTotals = 1024;  // per-layer sums are staged in a host array of this many entries

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device pointer.
static __device__ __align__(256) unsigned char g_route_scratch[kStaticScratchBytes];

// Device address of the array, per device ordinal, resolved on first use and kept for the life of the
// process.  cudaDeviceReset unloads the library image from that device; the address cached here is then
// stale, so a process that resets a device must not call this entry point on it again.
void* g_scratch_ptr[kMaxDevices];

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace
}  // namespace mcce

using namespace mcce;

extern "C" size_t mcce_route_trace_static_limit(void) { return kStaticScratchBytes; }

extern "C" int mcce_route_trace_static(const mcce_config* cfg, int32_t n_steps, const void* hidden, const float* Wr,
                                       const float* logits_in, const float* fixed_delta, int32_t* sel_idx,
                                       float* sel_w, mcce_stats* totals_host, void* cuda_stream) {
  if (!cfg || n_steps < 0 || !sel_idx || !sel_w) return MCCE_EINVAL;
  if ((hidden == nullptr) == (logits_in == nullptr)) return MCCE_EINVAL;
  if (hidden && (!Wr || ((uintptr_t)Wr % 16))) return MCCE_EINVAL;
  if (cfg->n_layers < 1 || cfg->n_streams < 1 || cfg->n_experts < 1 || cfg->n_experts > kMaxE) return MCCE_EINVAL;
  if (cfg->top_k < 1 || cfg->top_k > kMaxK || cfg->top_k > cfg->n_experts) return MCCE_EINVAL;
  if (cfg->top_j < 0 || cfg->top_j > cfg->top_k || cfg->cache_capacity < 1) return MCCE_EINVAL;
  if (!(cfg->lambda >= 0.f) || cfg->lambda > 3.0e38f) return MCCE_EINVAL;
  if (cfg->delta_mode != MCCE_DELTA_RUNNING && cfg->delta_mode != MCCE_DELTA_FIXED) return MCCE_EINVAL;
  if (cfg->delta_mode == MCCE_DELTA_FIXED && !fixed_delta) return MCCE_EINVAL;
  if (cfg->hidden_dtype != MCCE_F32 && cfg->hidden_dtype != MCCE_BF16) return MCCE_EINVAL;
  if (hidden && (cfg->d_model < 8 || cfg->d_model % 8)) return MCCE_EINVAL;
  if (cfg->rerank_mode < MCCE_RERANK_CACHE_PRIOR || cfg->rerank_mode > MCCE_RERANK_CUMSUM) return MCCE_EINVAL;
  if (cfg->rerank_mode == MCCE_RERANK_MAX_RANK && (cfg->max_rank < 0 || cfg->max_rank > cfg->n_experts))
    return MCCE_EINVAL;
  if (cfg->rerank_mode == MCCE_RERANK_CUMSUM && !(cfg->cum_threshold >= 0.f)) return MCCE_EINVAL;
  // four-float accesses to the rows of logits (E a multiple of 4) and to the hidden rows
  if (((uintptr_t)logits_in % ((cfg->n_experts & 3) ? 4 : 16)) || ((uintptr_t)hidden % 16)) return MCCE_EINVAL;
  // refuse before any size is multiplied out: a state of L*S*E words must fit the array at all
  if ((uint64_t)cfg->n_layers * (uint64_t)cfg->n_streams > kStaticScratchBytes / 4) return MCCE_ELIMIT;

  // layout of the state inside the static array; sizes beyond the array are refused
  const size_t LS = (size_t)cfg->n_layers * cfg->n_streams, E = cfg->n_experts, EW = (E + 31) / 32;
  const size_t o_stamp = 0, o_ever = o_stamp + up256(LS * E * 4), o_sum = o_ever + up256(LS * EW * 4);
  const size_t o_miss = o_sum + up256(LS * 4), o_cold = o_miss + up256(LS * 4), o_stats = o_cold + up256(LS * 4);
  const size_t need = o_stats + up256((size_t)cfg->n_layers * 16);
  if (need > kStaticScratchBytes) return MCCE_ELIMIT;
  if (totals_host && cfg->n_layers > kMaxLayersForTotals) return MCCE_ELIMIT;
  const uint64_t last_key = (uint64_t)E + (uint64_t)n_steps * cfg->top_k + cfg->top_k + 1;
  if (last_key >= 0xffffffffull) return MCCE_ESTATE;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MCCE_ECUDA;
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_route_scratch) != cudaSuccess || !ptr) return MCCE_ECUDA;
    g_scratch_ptr[dev] = ptr;
  }
  char* base = (char*)g_scratch_ptr[dev];
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // the array still holds the previous call's state: every cache starts empty, every counter at zero
  if (cudaMemsetAsync(base, 0, need, st) != cudaSuccess) return MCCE_ECUDA;
  if (n_steps == 0) return MCCE_OK;

  RouteParams p;
  p.L = cfg->n_layers, p.S = cfg->n_streams, p.E = cfg->n_experts, p.K = cfg->top_k, p.J = cfg->top_j;
  p.C = cfg->cache_capacity, p.d = cfg->d_model, p.n_steps = n_steps, p.lambda = cfg->lambda;
  p.delta_mode = cfg->delta_mode, p.renorm = cfg->renorm, p.hidden_bf16 = cfg->hidden_dtype == MCCE_BF16;
  p.n_partials = 1, p.partial_stride = 0, p.load_tok = nullptr, p.life = nullptr, p.miss_trace = nullptr, p.trace_avail = 0;
  p.rerank_mode = cfg->rerank_mode, p.max_rank = cfg->max_rank, p.cum_threshold = cfg->cum_threshold;
  p.hidden = hidden, p.logits_in = logits_in, p.Wr = Wr, p.fixed_delta = fixed_delta;
  p.stamp = (uint32_t*)(base + o_stamp), p.ever = (uint32_t*)(base + o_ever);
  p.sum_range = (float*)(base + o_sum), p.miss = (uint32_t*)(base + o_miss), p.cold = (uint32_t*)(base + o_cold);
  p.sel_idx = sel_idx, p.sel_w = sel_w, p.logits_out = nullptr, p.tok0 = 0u, p.cnt0 = 0u;
  p.err_nonfinite = nullptr;
  if (launch_route(p, st) != cudaSuccess) return MCCE_ECUDA;

  if (totals_host) {
    unsigned long long* sums = (unsigned long long*)(base + o_stats);
    if (launch_stats(p.miss, p.cold, sums, p.L, p.S, st) != cudaSuccess) return MCCE_ECUDA;
    unsigned long long h[2 * kMaxLayersForTotals];
    if (cudaMemcpyAsync(h, sums, (size_t)p.L * 16, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MCCE_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MCCE_ECUDA;
    totals_host->steps = (int64_t)n_steps * (int64_t)LS;
    totals_host->selections = totals_host->steps * cfg->top_k;
    totals_host->misses = totals_host->cold_misses = 0;
    for (int l = 0; l < p.L; ++l) {
      totals_host->misses += (int64_t)h[2 * l];
      totals_host->cold_misses += (int64_t)h[2 * l + 1];
    }
  }
  return MCCE_OK;
}
