// One kernel for the whole routing step from hidden states (Eq. 3, Eq. 8, Eq. 7, top-K, Eq. 4 and the LRU
// update of Sec. 4.2): the router-resident tensor-core GEMM of route_gemm_res.cuh and the routing tail of
// route_group.cuh run side by side in the same CTAs, so that the tail of one token overlaps the GEMM of the
// next ones instead of following it in a second launch.
//
// A layer belongs to KS CTAs (one K part of the reduction each).  Warps 0-5 of a CTA are the GEMM (TMA
// producer, MMA issuer, four epilogue warps).  An epilogue warp adds the partial logits of its K part for its
// 32 rows of the (token, stream tile) into the launch's logits array (fp32 reductions in L2; the array is zero
// at launch) and, after the last stream tile of a token, notes its progress in shared memory.  Warp 6 publishes:
// once all four epilogue warps are through with a token it issues the device-wide fence and adds the CTA's four
// counts to the counters of the token's pairs.  (A fence takes about 3 us while the device streams hidden
// states; issued by the epilogue warps themselves, tile by tile, it made them, not the tensor core, set the pace:
// 4.8 us per tile instead of 2.7.)  The remaining warps are the
// tail: the S streams of the layer are dealt out to its KS CTAs, a group of lanes per stream as in
// route_group.cuh.  Before a token they wait (bounded) until all KS CTAs of the layer have counted in on the
// tiles they read, then read the sums (L2-coherent loads) and put the zeros back.  The launch is cooperative, so
// every CTA that a tail warp waits for is resident; the GEMM warps and the publisher wait for nothing outside
// their CTA, so the waits cannot form a cycle.
//
// The order in which the KS parts of a logit are added is that of arrival: the last bit of a logit can differ
// from run to run (the two-kernel path adds them in the fixed order 0 .. KS-1).
//
// Measured alternatives (Qwen-shaped, eight tokens per launch): one array per K part, read by the tail when the
// token's turn comes (90 us); the same with the next token's parts held in registers while the current token is
// routed (64 more registers than the 96 a thread has here: spills, 120 us); two more warps per CTA that add the
// parts up ahead of the tail (three more L2 round trips per tile on two latency-bound warps: 164 us).
#include "route_gemm_res.cuh"
#include "route_group.cuh"

namespace mcce {

using namespace rres;

namespace {

constexpr int kGemmWarps = 6;      // TMA producer, MMA issuer, four epilogue warps
constexpr int kFrontWarps = kGemmWarps + 1;   // and the warp that publishes finished pairs
constexpr int kMaxTailWarps = 16;
// Hidden tiles in flight per CTA.  The stand-alone GEMM takes as many ring stages as fit; here a deeper ring
// only lengthens the queues that the tail's loads, the counters and the publisher's fence wait behind (an L2
// round trip takes 3-4 us while 5 stages per SM are in flight): Qwen-shaped, eight tokens, 5 stages 90 us,
// 4 or 3 stages 84 us, 2 stages 95 us.
constexpr int kFusedStages = 4;

struct FusedArgs {
  Geometry g;
  int Sc;               // streams of the layer routed by each of its CTAs
  int tail_warps;
  float* Z;             // [n_steps, L, S, E] logits: zero at launch, the KS parts are added into it, the tail
                        // reads them and puts the zeros back
  uint32_t* part_ready; // [L][n_steps * n_tiles] epilogue warps (4 per K part) whose rows of a tile are added in
  uint32_t* next_ready; // the counters of the next launch (the two sets alternate): cleared by this one
  int counter_words;    // words of a set
  uint32_t* err;
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* q) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(q) : "memory");
  return v;
}

// All lanes of the calling warp wait until *q >= target.  False: the CTA is giving up (this wait ran out of
// time, or another one did).
__device__ __forceinline__ bool wait_count(const uint32_t* q, uint32_t target, volatile uint32_t* abort_flag,
                                           uint32_t* err, uint32_t code) {
  if (__all_sync(kFull, ld_acquire(q) >= target)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    __nanosleep(64);
    if (__all_sync(kFull, ld_acquire(q) >= target)) return true;
    if ((it & 63u) == 0u) {
      bool stop = false;
      if ((threadIdx.x & 31) == 0) {
        if (*abort_flag) {
          stop = true;
        } else if (global_ns() - t0 > kWaitLimitNs) {
          *abort_flag = 1u;
          atomicCAS(err, 0u, code);
          stop = true;
        }
      }
      if (__any_sync(kFull, stop)) return false;
    }
  }
}

// What the tail asks before it reads the partial logits of a token: the counters of the stream tiles that the
// calling warp's streams lie in.
struct TailSync {
  const uint32_t* ready_l;   // part_ready of this layer
  uint32_t target;           // counts of a finished tile: 4 epilogue warps x KS parts
  int n_tiles, tile_lo, tile_hi;
  volatile uint32_t* abort_flag;
  uint32_t* err;
  __device__ __forceinline__ bool wait(int t) const {
    for (int tile = tile_lo; tile <= tile_hi; ++tile)
      if (!wait_count(ready_l + t * n_tiles + tile, target, abort_flag, err, 36u)) return false;
    return true;
  }
  // a warp's streams are adjacent: they lie in one tile or in two
  uint32_t c_lo, c_hi;
  __device__ __forceinline__ void probe(int t) {
    c_lo = ld_acquire(ready_l + t * n_tiles + tile_lo);
    c_hi = ld_acquire(ready_l + t * n_tiles + tile_hi);
  }
  __device__ __forceinline__ bool probed_ok() const { return __all_sync(kFull, c_lo >= target && c_hi >= target); }
};

// TW: tail warps the kernel is compiled for (its register budget follows from the thread count).
template <int G, int KMAX, int TW>
__global__ void __launch_bounds__(32 * (kFrontWarps + TW), 1)
route_fused_kernel(const __grid_constant__ Maps maps, const FusedArgs args, const RouteParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const Geometry& a = args.g;
  const Smem m = carve(smem_raw, a);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ks = blockIdx.x % a.KS, l = blockIdx.x / a.KS;
  const KPart kp = k_part_of(a, ks);
  const int n_pairs = a.n_steps * a.n_tiles;

  if (threadIdx.x == 0) init_barriers(m);
  if (warp == 1) tmem_alloc(smem_u32(m.tmem_slot), kTmemCols);
  for (int w = blockIdx.x * blockDim.x + threadIdx.x; w < args.counter_words; w += gridDim.x * blockDim.x)
    args.next_ready[w] = 0u;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *m.tmem_slot;

  if (warp == 0) {
    if (lane == 0) produce(maps, a, m, l, kp, 0, 1, args.err, 31u);
  } else if (warp == 1) {
    if (lane == 0) issue_mmas(a, m, tmem_base, kp, 0, 1, args.err, 31u);
  } else if (warp < kGemmWarps) {
    const int quad = warp & 3, row = quad * 32 + lane;
    for (int i = 0; i < n_pairs; ++i) {
      const int t = i / a.n_tiles, tile = i % a.n_tiles;
      const size_t grow = (size_t)(t * a.L + l) * a.S + tile * kTileM + row;
      const bool row_ok = tile * kTileM + row < a.S;
      if (!drain_pair<true>(a, m, tmem_base, kp.n_k(i), (uint32_t)i, quad, lane, args.Z + grow * a.E, row_ok, args.err, 35u)) break;
      // Once per token (after its last stream tile; the tail consumes whole tokens): this warp's additions of the
      // token's pairs are ordered before its progress word for the other warps of the CTA.  The fence waits until
      // the reductions have been performed in L2, a round trip of 2-3 us here.
      if (tile == a.n_tiles - 1) {
        asm volatile("fence.acq_rel.cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("fence.acq_rel.cta;" ::: "memory");
          m.drained[quad] = (uint32_t)i + 1u;
        }
      }
    }
  } else if (warp == kGemmWarps) {
    // ---- publisher: pairs that all four epilogue warps have finished are counted in device-wide -------------
    if (lane == 0) {
      uint32_t* cnt = args.part_ready + (size_t)l * n_pairs;
      uint32_t published = 0u;
      unsigned long long last = global_ns();
      for (uint32_t it = 1; published < (uint32_t)n_pairs; ++it) {
        const uint32_t d = min(min(m.drained[0], m.drained[1]), min(m.drained[2], m.drained[3]));
        if (d > published) {
          // acquire on the progress words, release for the counters: the epilogue warps' additions come first
          asm volatile("fence.acq_rel.gpu;" ::: "memory");
          for (uint32_t i = published; i < d; ++i) atomicAdd(cnt + i, 4u);
          published = d;
          last = global_ns();
          continue;
        }
        __nanosleep(100);
        if ((it & 63u) == 0u) {
          if (*m.abort_flag) break;
          if (global_ns() - last > kWaitLimitNs) {
            *m.abort_flag = 1u;
            atomicCAS(args.err, 0u, 37u);
            break;
          }
        }
      }
    }
  } else {
    // ---- routing tail of this CTA's share of the layer's streams -------------------------------------------
    const int tw = warp - kFrontWarps;
    const int idx = (tw * 32 + lane) / G;                      // stream of this CTA
    const int s_raw = idx < args.Sc ? ks * args.Sc + idx : a.S;   // past the share: idle group
    if (tw < args.tail_warps && ks * args.Sc + (tw * 32) / G < a.S) {
      TailSync sync;
      sync.ready_l = args.part_ready + (size_t)l * n_pairs, sync.n_tiles = a.n_tiles, sync.target = 4u * (uint32_t)a.KS;
      sync.tile_lo = min(a.S - 1, ks * args.Sc + (tw * 32) / G) / kTileM;
      sync.tile_hi = min(a.S - 1, ks * args.Sc + min(args.Sc - 1, (tw * 32 + 31) / G)) / kTileM;
      sync.abort_flag = m.abort_flag, sync.err = args.err, sync.c_lo = sync.c_hi = 0u;
      rgroup::route_group_streams<G, KMAX, rgroup::kPrefetchReady, 1, true, true>(p, l, s_raw, lane % G, sync);
    }
  }
  teardown(m, tmem_base, warp, 1);
}

int group_of(int E) { return E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8; }
// (13 tail warps are the most that leave a thread 96 registers: 7 + 13 = 20 warps, five per scheduler)
int tail_bucket(int tail_warps) { return tail_warps <= 8 ? 8 : tail_warps <= 13 ? 13 : 16; }

template <int G, int KMAX, int TW>
cudaError_t launch_one(const Maps& m, const FusedArgs& a, const RouteParams& p, cudaStream_t st) {
  static int cache[64] = {0};
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(route_fused_kernel<G, KMAX, TW>, (size_t)kSmemMax + 1024, cache, &sms);
  if (e0 != cudaSuccess) return e0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(a.g.L * a.g.KS)), cfg.blockDim = dim3((unsigned)(32 * (kFrontWarps + TW)));
  cfg.dynamicSmemBytes = (size_t)kSmemMax + 1024, cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident at once, or the launch fails
  attr[0].val.cooperative = 1;
  cfg.attrs = attr, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, route_fused_kernel<G, KMAX, TW>, m, a, p);
}

// CTAs of this kernel that the device holds at once (0: not launchable).
template <int G, int KMAX, int TW>
int resident_ctas() {
  static int cache[64] = {0};
  int sms = 0, per_sm = 0;
  if (sm_count_and_smem_optin(route_fused_kernel<G, KMAX, TW>, (size_t)kSmemMax + 1024, cache, &sms) != cudaSuccess)
    return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, route_fused_kernel<G, KMAX, TW>, 32 * (kFrontWarps + TW),
                                                    (size_t)kSmemMax + 1024) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return per_sm * sms;
}

// The instantiations: group size by expert count, selections per token, tail warps.
#define MCCE_FUSED_FOR_EACH(X)                                                                             \
  X(1, 4, 8) X(1, 8, 8) X(1, 4, 13) X(1, 8, 13) X(1, 4, 16) X(1, 8, 16)                                      \
  X(2, 4, 8) X(2, 8, 8) X(2, 16, 8) X(2, 4, 13) X(2, 8, 13) X(2, 16, 13) X(2, 4, 16) X(2, 8, 16) X(2, 16, 16) \
  X(4, 4, 8) X(4, 8, 8) X(4, 16, 8) X(4, 4, 13) X(4, 8, 13) X(4, 16, 13) X(4, 4, 16) X(4, 8, 16) X(4, 16, 16) \
  X(8, 4, 8) X(8, 8, 8) X(8, 16, 8) X(8, 4, 13) X(8, 8, 13) X(8, 16, 13) X(8, 4, 16) X(8, 8, 16) X(8, 16, 16)

int k_bucket(int K) { return K <= 4 ? 4 : K <= 8 ? 8 : 16; }

int resident_ctas_of(int G, int K, int TW) {
  const int kb = k_bucket(K);
#define MCCE_X(g, k, tw) if (G == g && kb == k && TW == tw) return resident_ctas<g, k, tw>();
  MCCE_FUSED_FOR_EACH(MCCE_X)
#undef MCCE_X
  return 0;
}

cudaError_t launch_any(int G, int K, int TW, const Maps& m, const FusedArgs& a, const RouteParams& p, cudaStream_t st) {
  const int kb = k_bucket(K);
#define MCCE_X(g, k, tw) if (G == g && kb == k && TW == tw) return launch_one<g, k, tw>(m, a, p, st);
  MCCE_FUSED_FOR_EACH(MCCE_X)
#undef MCCE_X
  return cudaErrorInvalidValue;
}

}  // namespace

// Counter words the kernel needs: one per (layer, token, stream tile), in two sets that alternate from launch to
// launch (a launch clears the set of the next one; both start at zero).
size_t route_fused_counter_words(int n_layers, int n_steps, int n_streams) {
  return 2 * (size_t)n_layers * n_steps * ((n_streams + kTileM - 1) / kTileM);
}

// Fixes the K-split of the fused kernel for this configuration, or leaves plan->fused_ready at 0 when the two-kernel
// path has to be used: other selection rules, lifetime tracking, more than 64 experts or a count that is no multiple
// of 4 (the tail reads rows of logits four at a time), more streams per CTA than its tail warps hold, accumulator
// sets that do not fit TMEM, or so few layers that KS CTAs per layer would leave most SMs idle.
int route_fused_plan(const mcce_config& c, RouterGemmPlan* plan) {
  plan->fused_ready = 0;
  if (!plan->res_ready) return MCCE_OK;
  if (c.rerank_mode != MCCE_RERANK_CACHE_PRIOR || c.track_lifetime || c.n_experts > 64 || (c.n_experts & 3) ||
      c.top_k > kMaxK)
    return MCCE_OK;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MCCE_ECUDA;
  const int Epad = epad_of(c.n_experts), G = group_of(c.n_experts), slabs = c.d_model / kTileK;
  if (G == 1 && c.top_k > 8) return MCCE_OK;
  int best_ks = 0, best_ctas = 0;
  for (int ks = 1; ks <= kPartsMax && ks <= slabs; ++ks) {
    if (res_bytes_of(slabs, ks, Epad) + kMinStages * kStageBytes + kBarBytes > kSmemMax) continue;
    if (!sets_fit(slabs, ks, Epad)) continue;
    const int Sc = (c.n_streams + ks - 1) / ks;
    const int tail_warps = (Sc * G + 31) / 32;
    if (tail_warps > kMaxTailWarps) continue;
    const int ctas = c.n_layers * ks;   // all of them have to be resident together
    if (ctas <= resident_ctas_of(G, c.top_k, tail_bucket(tail_warps)) && ctas > best_ctas)
      best_ctas = ctas, best_ks = ks;
  }
  if (best_ks == 0 || 2 * best_ctas < sms) return MCCE_OK;
  plan->fused_parts = best_ks;
  plan->fused_tail_warps = ((c.n_streams + best_ks - 1) / best_ks * G + 31) / 32;
  plan->fused_ready = 1;
  return MCCE_OK;
}

// The routing step of n_steps tokens of all layers.  p carries the routing parameters and outputs; its logits
// fields are set here.  Z: n_steps*L*S*E floats, zero; counters: route_fused_counter_words() words for the largest
// n_steps, zero before the first launch.
cudaError_t route_fused_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps, float* Z,
                               uint32_t* counters, RouteParams p, uint32_t* err, cudaStream_t st) {
  const uint64_t rows = (uint64_t)n_steps * c.n_layers * c.n_streams;
  cudaError_t e = hidden_maps(plan, hidden, rows, c.d_model, c.n_streams);
  if (e != cudaSuccess) return e;
  FusedArgs args;
  Geometry& a = args.g;
  a.L = c.n_layers, a.l0 = 0, a.L_terms = c.n_layers;
  a.S = c.n_streams, a.E = c.n_experts, a.Epad = epad_of(c.n_experts), a.n_steps = n_steps;
  a.KS = plan.fused_parts, a.slabs = c.d_model / kTileK;
  a.n_tiles = (c.n_streams + kTileM - 1) / kTileM;
  a.res_bytes = res_bytes_of(a.slabs, a.KS, a.Epad);
  a.n_stages = stages_of(a.res_bytes) < kFusedStages ? stages_of(a.res_bytes) : kFusedStages;
  const int G = group_of(c.n_experts);
  args.Sc = (c.n_streams + a.KS - 1) / a.KS;
  args.tail_warps = (args.Sc * G + 31) / 32;
  args.Z = Z, args.err = err;
  // the two counter sets alternate; a set holds the words of the largest launch
  const size_t set_words = route_fused_counter_words(c.n_layers, router_gemm_steps_max(), c.n_streams) / 2;
  args.part_ready = counters + (size_t)(plan.fused_flip & 1) * set_words;
  args.next_ready = counters + (size_t)((plan.fused_flip & 1) ^ 1) * set_words;
  args.counter_words = (int)set_words;
  p.n_steps = n_steps, p.hidden = nullptr, p.logits_in = Z, p.n_partials = 1, p.partial_stride = 0;
  Maps m;
  m.w = plan.w_res, m.x = plan.x_res, m.xt = plan.xt_res;
  e = launch_any(G, c.top_k, tail_bucket(args.tail_warps), m, args, p, st);
  if (e == cudaSuccess) plan.fused_flip ^= 1;
  return e;
}

}  // namespace mcce
