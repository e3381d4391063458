// Stand-alone routing tail on given logits for the paper's own rule (Cache-Prior, Eq. 7) and up to 64 experts,
// a small group of lanes per (stream, layer): see route_group.cuh.  The warp-per-stream kernel of route.cu
// (one or two experts per lane, two warp-wide reductions per selected expert) remains for the other rules,
// more experts and lifetime tracking.
#include "route_group.cuh"

namespace mcce {

namespace {

constexpr int kThreads = 64;
using rgroup::kPartsMax;

template <int G, int KMAX, bool PF>
__global__ void __launch_bounds__(kThreads) route_group_kernel(const RouteParams p) {
  constexpr int kPerCta = kThreads / G;   // streams per CTA
  const int blocks_per_layer = (p.S + kPerCta - 1) / kPerCta;
  const int l = blockIdx.x / blocks_per_layer;
  const int s_raw = (blockIdx.x % blocks_per_layer) * kPerCta + threadIdx.x / G;
  rgroup::route_group_streams<G, KMAX, PF ? rgroup::kPrefetchAll : rgroup::kLoadDirect, kPartsMax, false, false>(
      p, l, s_raw, threadIdx.x % G, rgroup::AllPresent());
}

template <int G, bool PF>
cudaError_t launch_gp(const RouteParams& p, int grid, cudaStream_t st) {
  if (p.K <= 4)
    route_group_kernel<G, 4, PF><<<grid, kThreads, 0, st>>>(p);
  else if (p.K <= 8)
    route_group_kernel<G, 8, PF><<<grid, kThreads, 0, st>>>(p);
  else
    route_group_kernel<G, 16, PF><<<grid, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(const RouteParams& p, cudaStream_t st) {
  constexpr int kPerCta = kThreads / G;
  const int grid = p.L * ((p.S + kPerCta - 1) / kPerCta);
  // The prefetching instantiation needs about 170 registers per thread: it only pays while every CTA of the
  // grid is resident at once (six CTAs of 64 threads per SM), and there is nothing to prefetch for one token.
  static int sms_of[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!sms_of[dev] && cudaDeviceGetAttribute(&sms_of[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return cudaErrorInvalidDevice;
  const bool pf = p.n_steps > 1 && (p.E & 3) == 0 && p.n_partials <= kPartsMax && grid <= 6 * sms_of[dev];
  return pf ? launch_gp<G, true>(p, grid, st) : launch_gp<G, false>(p, grid, st);
}

}  // namespace

// Logits given (not hidden states), the paper's Cache-Prior rule, no lifetime tracking, E <= 64.
bool route_thread_applicable(const RouteParams& p) {
  return p.hidden == nullptr && p.logits_in != nullptr && p.rerank_mode == MCCE_RERANK_CACHE_PRIOR &&
         p.load_tok == nullptr && p.E <= 64 && p.K <= kMaxK;
}

cudaError_t launch_route_thread(const RouteParams& p, cudaStream_t st) {
  if (p.E <= 8) return launch_g<1>(p, st);
  if (p.E <= 16) return launch_g<2>(p, st);
  if (p.E <= 32) return launch_g<4>(p, st);
  return launch_g<8>(p, st);
}

}  // namespace mcce
