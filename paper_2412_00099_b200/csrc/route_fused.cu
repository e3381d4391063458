// One kernel for the whole routing step from hidden states (Eq. 3, Eq. 8, Eq. 7, top-K, Eq. 4 and the LRU
// update of Sec. 4.2): the router-resident tensor-core GEMM of route_gemm_res.cu and the routing tail of
// route_group.cuh run side by side in the same CTAs, so that the tail of one (token, stream tile) overlaps the
// GEMM of the next ones instead of following it in a second launch.
//
// A layer belongs to KS CTAs (one K part of the reduction each).  Warps 0-5 of a CTA are the GEMM
// (TMA producer, MMA issuer, four epilogue warps); they store the partial logits of their K part and then
// count themselves in on a ready counter of the (layer, token, stream tile).  The remaining warps are the
// tail: the S streams of the layer are dealt out to the KS CTAs, a group of lanes per stream as in
// route_group.cuh; before a token they wait until all 4*KS epilogue warps of the layer have counted in, then
// read the KS partial sums (L2-coherent loads) and route.  The launch is cooperative, so every CTA that a
// tail warp waits for is resident; every wait is bounded in time all the same.
//
// The accumulation is cut into sets of kSetSlabs K-slabs (the tensor core's fp32 accumulate truncates), each
// set with its own TMEM columns; the epilogue adds the sets in round-to-nearest fp32.
#include "route_group.cuh"
#include "tc_common.cuh"

namespace mcce {

using namespace tc;

namespace {

constexpr int kTileM = 128, kTileK = 64, kXBox = 16, kGemmWarps = 6, kMaxStages = 10, kMinStages = 3;
constexpr int kMaxTailWarps = 16, kMaxThreads = 32 * (kGemmWarps + kMaxTailWarps);
constexpr uint32_t kRowBytes = kTileK * 2;
constexpr uint32_t kStageBytes = kTileM * kRowBytes;
constexpr uint32_t kSmemMax = 232448 - 1024;
constexpr uint32_t kBarBytes = 512;
constexpr int kSetSlabs = 8;
constexpr int kBufCols = 256, kTmemCols = 512;
constexpr int kPartsMaxF = 8;

struct FusedArgs {
  int L, S, E, Epad, n_steps;
  int KS, slabs, n_tiles, n_stages;
  int Sc;               // streams of the layer routed by each of its CTAs
  int tail_warps;
  uint32_t res_bytes;
  float* Z;             // [KS][n_steps, L, S, E] partial logits
  size_t z_stride;
  uint32_t* ready;      // [L][n_steps * n_tiles] epilogue warps that have stored their part
  uint32_t* err;
};
struct FusedMaps {
  CUtensorMap w, x, xt;
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* q) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(q) : "memory");
  return v;
}

template <int G, int KMAX>
__global__ void __launch_bounds__(kMaxThreads, 1)
route_fused_kernel(const __grid_constant__ FusedMaps maps, const FusedArgs a, const RouteParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t ring_base = smem_base + a.res_bytes;
  uint64_t* bars = (uint64_t*)(smem_al + (size_t)a.res_bytes + (size_t)a.n_stages * kStageBytes);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kMaxStages;
  const uint32_t bar_tfull = bar_empty + 8 * kMaxStages, bar_tempty = bar_tfull + 16, bar_res = bar_tempty + 16;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * kMaxStages + 5);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const uint32_t kStages = (uint32_t)a.n_stages;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ks = blockIdx.x % a.KS, l = blockIdx.x / a.KS;
  const int k_base = a.slabs / a.KS, k_rem = a.slabs % a.KS;
  const int k_begin = ks * k_base + min(ks, k_rem), n_k = k_base + (ks < k_rem ? 1 : 0);
  const int n_pairs = a.n_steps * a.n_tiles;
  const uint32_t term_bytes = (uint32_t)a.Epad * kRowBytes, slab_bytes = 3u * term_bytes;
  const uint32_t set_cols = 3u * (uint32_t)a.Epad;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 4);
    }
    mbar_init(bar_res, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar_res, (uint32_t)n_k * slab_bytes);
      for (int j = 0; j < n_k; ++j)
#pragma unroll
        for (int q = 0; q < 3; ++q)
          tma_load_3d(smem_base + (uint32_t)j * slab_bytes + q * term_bytes, &maps.w, (k_begin + j) * kTileK, 0,
                      q * a.L + l, bar_res);
      uint32_t stage = 0, phase = 0;
      bool alive = true;
      for (int i = 0; i < n_pairs && alive; ++i) {
        const int t = i / a.n_tiles, tile = i % a.n_tiles;
        const int row0 = (t * a.L + l) * a.S + tile * kTileM;
        const int n_box = (min(kTileM, a.S - tile * kTileM) + kXBox - 1) / kXBox;
        for (int j = 0; j < n_k; ++j) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.err, 31u)) {
            alive = false;
            break;
          }
          const uint32_t sa = ring_base + stage * kStageBytes, full = bar_full + 8 * stage;
          mbar_expect_tx(full, (uint32_t)n_box * kXBox * kRowBytes);
          if (n_box == kTileM / kXBox) {
            tma_load_2d(sa, &maps.xt, (k_begin + j) * kTileK, row0, full);
          } else {
            for (int b = 0; b < n_box; ++b)
              tma_load_2d(sa + b * kXBox * kRowBytes, &maps.x, (k_begin + j) * kTileK, row0 + b * kXBox, full);
          }
          if (++stage == kStages) stage = 0, phase ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      const uint32_t idesc = instr_desc(set_cols);
      bool alive = mbar_wait(bar_res, 0u, abort_flag, a.err, 32u);
      tc_fence_after();
      for (int i = 0; i < n_pairs && alive; ++i) {
        const uint32_t buf = (uint32_t)i & 1u, acc_phase = ((uint32_t)i >> 1) & 1u;
        if (!mbar_wait(bar_tempty + 8 * buf, acc_phase ^ 1u, abort_flag, a.err, 33u)) break;
        tc_fence_after();
        for (int j = 0; j < n_k; ++j) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.err, 34u)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_set = tmem_base + buf * kBufCols + (uint32_t)(j / kSetSlabs) * set_cols;
          const uint32_t sa = ring_base + stage * kStageBytes, sb = smem_base + (uint32_t)j * slab_bytes;
#pragma unroll
          for (int k = 0; k < kTileK / 16; ++k)
            umma_bf16(d_set, smem_desc(sa + k * 32), smem_desc(sb + k * 32), idesc, (j % kSetSlabs == 0 && k == 0) ? 0u : 1u);
          umma_commit(bar_empty + 8 * stage);
          if (++stage == kStages) stage = 0, phase ^= 1u;
        }
        if (alive) umma_commit(bar_tfull + 8 * buf);
      }
    }
  } else if (warp < kGemmWarps) {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int n_sets = (n_k + kSetSlabs - 1) / kSetSlabs;
    float* Zp = a.Z + (size_t)ks * a.z_stride;
    const bool vec4 = (a.E & 3) == 0;
    for (int i = 0; i < n_pairs; ++i) {
      const int t = i / a.n_tiles, tile = i % a.n_tiles;
      const int row0 = (t * a.L + l) * a.S + tile * kTileM;
      const bool row_ok = tile * kTileM + row < a.S;
      const uint32_t buf = (uint32_t)i & 1u, acc_phase = ((uint32_t)i >> 1) & 1u;
      if (!mbar_wait(bar_tfull + 8 * buf, acc_phase, abort_flag, a.err, 35u)) break;
      tc_fence_after();
      const uint32_t t0 = tmem_base + lane_addr + buf * kBufCols;
      float* zrow = Zp + (size_t)(row0 + row) * a.E;
      for (int c = 0; c < a.Epad; c += 16) {
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = 0.f;
        for (int set = 0; set < n_sets; ++set) {
          float hi[16], mid[16], lo[16];
          const uint32_t ts = t0 + (uint32_t)set * set_cols + (uint32_t)c;
          tmem_ld16(ts, hi);
          tmem_ld16(ts + a.Epad, mid);
          tmem_ld16(ts + 2 * a.Epad, lo);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) acc[j] = __fadd_rn(acc[j], __fadd_rn(hi[j], __fadd_rn(mid[j], lo[j])));
        }
        if (row_ok) {
          if (vec4) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              if (c + j < a.E) *(float4*)(zrow + c + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c + j < a.E) zrow[c + j] = acc[j];
          }
        }
      }
      tc_fence_before();
      __threadfence();   // this lane's part of the tile is visible device-wide before the warp counts in
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar_tempty + 8 * buf);
        atomicAdd(a.ready + (size_t)l * n_pairs + i, 1u);
      }
    }
  } else {
    // ---- routing tail of this CTA's share of the layer's streams -------------------------------------------
    const int tw = warp - kGemmWarps;
    const int idx = (tw * 32 + lane) / G;                     // stream of this CTA
    const int s_raw = idx < a.Sc ? ks * a.Sc + idx : a.S;      // past the share: idle group
    const int idx_hi = min(a.Sc - 1, (tw * 32 + 31) / G);
    const int tile_hi = min(a.S - 1, ks * a.Sc + idx_hi) / kTileM;   // last stream tile this warp reads
    const uint32_t target = 4u * (uint32_t)a.KS;
    const uint32_t* ready_l = a.ready + (size_t)l * n_pairs;
    if (tw < a.tail_warps && ks * a.Sc + (tw * 32) / G < a.S) {
      auto wait = [&](int t) -> bool {
        const uint32_t* q = ready_l + t * a.n_tiles + tile_hi;
        // the K parts finish a tile in order, so the last tile's counter covers the earlier ones
        if (__all_sync(kFull, ld_acquire(q) >= target)) return true;
        const unsigned long long t0 = global_ns();
        for (uint32_t it = 1;; ++it) {
          __nanosleep(64);
          if (__all_sync(kFull, ld_acquire(q) >= target)) return true;
          if ((it & 63u) == 0u) {
            bool stop = false;
            if (lane == 0) {
              if (*abort_flag) {
                stop = true;
              } else if (global_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1u;
                atomicCAS(a.err, 0u, 36u);
                stop = true;
              }
            }
            if (__any_sync(kFull, stop)) return false;
          }
        }
      };
      rgroup::route_group_streams<G, KMAX, false, true>(p, l, s_raw, lane % G, wait);
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

int epad_of(int E) { return (E + 15) & ~15; }
int group_of(int E) { return E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8; }

template <int G, int KMAX>
cudaError_t launch_one(const FusedMaps& m, const FusedArgs& a, const RouteParams& p, int threads, cudaStream_t st) {
  static int cache[64] = {0};
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(route_fused_kernel<G, KMAX>, (size_t)kSmemMax + 1024, cache, &sms);
  if (e0 != cudaSuccess) return e0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(a.L * a.KS)), cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = (size_t)kSmemMax + 1024, cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident at once, or the launch fails
  attr[0].val.cooperative = 1;
  cfg.attrs = attr, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, route_fused_kernel<G, KMAX>, m, a, p);
}

template <int G>
cudaError_t launch_g(const FusedMaps& m, const FusedArgs& a, const RouteParams& p, int threads, cudaStream_t st) {
  if (p.K <= 4) return launch_one<G, 4>(m, a, p, threads, st);
  if (p.K <= 8) return launch_one<G, 8>(m, a, p, threads, st);
  return launch_one<G, 16>(m, a, p, threads, st);
}

// CTAs of this kernel that the device holds at once (0: not launchable).
template <int G, int KMAX>
int resident_ctas(int threads) {
  static int cache[64] = {0};
  int sms = 0, per_sm = 0;
  if (sm_count_and_smem_optin(route_fused_kernel<G, KMAX>, (size_t)kSmemMax + 1024, cache, &sms) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, route_fused_kernel<G, KMAX>, threads,
                                                    (size_t)kSmemMax + 1024) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return per_sm * sms;
}
int resident_ctas_of(int G, int K, int threads) {
  const int kb = K <= 4 ? 4 : K <= 8 ? 8 : 16;
#define MCCE_AC(g, k) if (G == g && kb == k) return resident_ctas<g, k>(threads);
  MCCE_AC(1, 4) MCCE_AC(1, 8) MCCE_AC(2, 4) MCCE_AC(2, 8) MCCE_AC(2, 16) MCCE_AC(4, 4) MCCE_AC(4, 8) MCCE_AC(4, 16)
  MCCE_AC(8, 4) MCCE_AC(8, 8) MCCE_AC(8, 16)
#undef MCCE_AC
  return 0;
}

uint32_t res_bytes_of(int slabs, int ks, int Epad) {
  const uint32_t res = (uint32_t)((slabs + ks - 1) / ks) * 3u * (uint32_t)Epad * kRowBytes;
  return (res + 1023u) & ~1023u;
}

}  // namespace

// Fixes the K-split of the fused kernel for this configuration, or leaves plan->fused_ready at 0 when the two-kernel
// path has to be used: other selection rules, lifetime tracking, more than 64 experts, more streams per CTA than
// its tail warps hold, accumulator sets that do not fit TMEM, or so few layers that KS CTAs per layer would leave
// most SMs idle.
int route_fused_plan(const mcce_config& c, RouterGemmPlan* plan) {
  plan->fused_ready = 0;
  if (!plan->res_ready) return MCCE_OK;
  if (c.rerank_mode != MCCE_RERANK_CACHE_PRIOR || c.track_lifetime || c.n_experts > 64 || c.top_k > kMaxK) return MCCE_OK;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MCCE_ECUDA;
  const int Epad = epad_of(c.n_experts), G = group_of(c.n_experts), slabs = c.d_model / kTileK;
  int best_ks = 0, best_ctas = 0;
  for (int ks = 1; ks <= kPartsMaxF && ks <= slabs; ++ks) {
    const int n_k = (slabs + ks - 1) / ks, n_sets = (n_k + kSetSlabs - 1) / kSetSlabs;
    if (res_bytes_of(slabs, ks, Epad) + kMinStages * kStageBytes + kBarBytes > kSmemMax) continue;
    if (n_sets * 3 * Epad > kBufCols) continue;
    const int Sc = (c.n_streams + ks - 1) / ks;
    const int tail_warps = (Sc * G + 31) / 32;
    if (tail_warps > kMaxTailWarps) continue;
    const int ctas = c.n_layers * ks;   // all of them have to be resident together
    if (ctas <= resident_ctas_of(G, c.top_k, 32 * (kGemmWarps + tail_warps)) && ctas > best_ctas)
      best_ctas = ctas, best_ks = ks;
  }
  if (best_ks == 0 || 2 * best_ctas < sms) return MCCE_OK;
  plan->fused_parts = best_ks;
  plan->fused_ready = 1;
  return MCCE_OK;
}

// The routing step of n_steps tokens of all layers.  p carries the routing parameters and outputs; its logits
// fields are set here.  Z: fused_parts arrays of n_steps*L*S*E floats; ready: L*n_steps*ceil(S/128) counters.
cudaError_t route_fused_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps, float* Z,
                               uint32_t* ready, RouteParams p, uint32_t* err, cudaStream_t st) {
  const uint64_t rows = (uint64_t)n_steps * c.n_layers * c.n_streams;
  if (plan.hidden_ptr_res != hidden || plan.hidden_rows_res != rows) {
    EncodeFn fn = encode_fn();
    const cuuint64_t dims[2] = {(cuuint64_t)c.d_model, rows};
    const cuuint64_t strides[1] = {(cuuint64_t)c.d_model * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)kXBox};
    const cuuint32_t box_tile[2] = {(cuuint32_t)kTileK, (cuuint32_t)kTileM};
    const cuuint32_t estr[2] = {1, 1};
    if (!fn || fn(&plan.x_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        fn(&plan.xt_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box_tile,
           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    plan.hidden_ptr_res = hidden;
    plan.hidden_rows_res = rows;
  }
  FusedArgs a;
  a.L = c.n_layers, a.S = c.n_streams, a.E = c.n_experts, a.Epad = epad_of(c.n_experts), a.n_steps = n_steps;
  a.KS = plan.fused_parts, a.slabs = c.d_model / kTileK;
  a.n_tiles = (c.n_streams + kTileM - 1) / kTileM;
  a.res_bytes = res_bytes_of(a.slabs, a.KS, a.Epad);
  const int stages = (int)((kSmemMax - kBarBytes - a.res_bytes) / kStageBytes);
  a.n_stages = stages > kMaxStages ? kMaxStages : stages;
  const int G = group_of(c.n_experts);
  a.Sc = (c.n_streams + a.KS - 1) / a.KS;
  a.tail_warps = (a.Sc * G + 31) / 32;
  a.Z = Z, a.z_stride = (size_t)rows * c.n_experts, a.ready = ready, a.err = err;
  p.n_steps = n_steps, p.hidden = nullptr, p.logits_in = Z, p.n_partials = a.KS, p.partial_stride = a.z_stride;
  cudaError_t e = cudaMemsetAsync(ready, 0, (size_t)a.L * n_steps * a.n_tiles * sizeof(uint32_t), st);
  if (e != cudaSuccess) return e;
  FusedMaps m;
  m.w = plan.w_res, m.x = plan.x_res, m.xt = plan.xt_res;
  const int threads = 32 * (kGemmWarps + a.tail_warps);
  switch (G) {
    case 1: return launch_g<1>(m, a, p, threads, st);
    case 2: return launch_g<2>(m, a, p, threads, st);
    case 4: return launch_g<4>(m, a, p, threads, st);
    default: return launch_g<8>(m, a, p, threads, st);
  }
}

}  // namespace mcce
