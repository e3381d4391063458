// Router logits of Eq. 3 on the tensor cores, router-resident form:
//   Z[(t,l,s), e] = sum_j W_r[l][e][j] x[(t,l,s)][j]   for E <= 80 experts.
//
// What the step has to move is the hidden rows (d bf16 per stream, layer and token); the router of a layer is
// shared by all its streams and tokens.  This kernel therefore keeps the router in shared memory and streams
// only hidden rows:
//   * a CTA owns one layer and one part of the reduction (a range of 64-column K-slabs); the three bf16 terms
//     of W_r (hi + mid + lo, see route_gemm.cu) of that range are loaded once and stay resident;
//   * the streams are the MMA's M (tiles of 128 hidden rows, the A operand), the terms are stacked along N
//     (B operand of 3 x Epad rows), so one tcgen05.mma per 16 columns produces the hi, mid and lo products of
//     128 streams at once, each in its own TMEM columns;
//   * the CTA walks the (token, stream tile) pairs of its layer; the hidden tiles come through a TMA ring;
//   * four epilogue warps (thread = stream row) add hi + (mid + lo) in round-to-nearest fp32 and store the
//     partial logits of this K part; the routing tail sums the parts in a fixed order.
// As in route_gemm.cu an accumulation phase ends every kPhaseSlabs slabs (the tensor core's fp32 accumulate
// truncates), alternating between two TMEM buffers so that the MMA warp never waits for the epilogue.
// Every mbarrier wait is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace mcce {

using namespace tc;

namespace {

constexpr int kTileM = 128, kTileK = 64, kXBox = 16, kThreads = 192, kMaxStages = 10, kMinStages = 3;
constexpr uint32_t kRowBytes = kTileK * 2;               // one 128-byte swizzle row
constexpr uint32_t kStageBytes = kTileM * kRowBytes;     // one hidden tile of one K-slab: 16 KB
constexpr uint32_t kSmemMax = 232448 - 1024;             // opt-in limit less the alignment slack
constexpr uint32_t kBarBytes = 512;
constexpr int kPhaseSlabs = 4;
constexpr int kBufCols = 256, kTmemCols = 512;
constexpr int kEMax = 80, kPartsMax = 8;

struct ResArgs {
  int L, S, E, Epad, n_steps;
  int KS, TG, slabs, n_tiles, n_stages;
  uint32_t res_bytes;   // shared memory reserved for the resident terms (multiple of 1024)
  float* Z;             // [KS][n_steps, L, S, E] partial logits
  size_t z_stride;
  uint32_t* err;
};
struct ResMaps {
  CUtensorMap w;   // 3-D: [3*L][E][d] bf16 terms (term-major), box 1 x Epad x 64
  CUtensorMap x;   // 2-D: [n_steps*L*S][d] hidden rows, box 16 x 64 (ragged last tile of a layer)
  CUtensorMap xt;  // the same rows, box 128 x 64 (full tiles)
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
router_gemm_res_kernel(const __grid_constant__ ResMaps maps, const ResArgs a) {
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
  // this CTA: layer l, K part ks (slabs [k_begin, k_begin + n_k)), pair group g
  const int g = blockIdx.x % a.TG;
  const int ks = (blockIdx.x / a.TG) % a.KS;
  const int l = blockIdx.x / (a.TG * a.KS);
  const int k_base = a.slabs / a.KS, k_rem = a.slabs % a.KS;
  const int k_begin = ks * k_base + min(ks, k_rem), n_k = k_base + (ks < k_rem ? 1 : 0);
  const int n_pairs = a.n_steps * a.n_tiles;
  const uint32_t term_bytes = (uint32_t)a.Epad * kRowBytes, slab_bytes = 3u * term_bytes;

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
      // the resident terms of this (layer, K part), then the hidden tiles of every pair of this CTA
      mbar_expect_tx(bar_res, (uint32_t)n_k * slab_bytes);
      for (int j = 0; j < n_k; ++j)
#pragma unroll
        for (int p = 0; p < 3; ++p)
          tma_load_3d(smem_base + (uint32_t)j * slab_bytes + p * term_bytes, &maps.w, (k_begin + j) * kTileK, 0,
                      p * a.L + l, bar_res);
      uint32_t stage = 0, phase = 0;
      bool alive = true;
      for (int i = g; i < n_pairs && alive; i += a.TG) {
        const int t = i / a.n_tiles, tile = i % a.n_tiles;
        const int row0 = (t * a.L + l) * a.S + tile * kTileM;
        const int n_box = (min(kTileM, a.S - tile * kTileM) + kXBox - 1) / kXBox;
        for (int j = 0; j < n_k; ++j) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.err, 21u)) {
            alive = false;
            break;
          }
          const uint32_t sa = ring_base + stage * kStageBytes, full = bar_full + 8 * stage;
          mbar_expect_tx(full, (uint32_t)n_box * kXBox * kRowBytes);
          if (n_box == kTileM / kXBox) {   // one 16 KB copy: measurably faster than eight of 2 KB
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
      uint32_t stage = 0, phase = 0, acc_iter = 0;
      const uint32_t idesc = instr_desc(3u * (uint32_t)a.Epad);
      bool alive = mbar_wait(bar_res, 0u, abort_flag, a.err, 22u);
      tc_fence_after();
      for (int i = g; i < n_pairs && alive; i += a.TG) {
        for (int k0 = 0; k0 < n_k && alive; k0 += kPhaseSlabs, ++acc_iter) {
          const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
          if (!mbar_wait(bar_tempty + 8 * buf, acc_phase ^ 1u, abort_flag, a.err, 23u)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_buf = tmem_base + buf * kBufCols;
          const int k1 = min(n_k, k0 + kPhaseSlabs);
          for (int j = k0; j < k1; ++j) {
            if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.err, 24u)) {
              alive = false;
              break;
            }
            tc_fence_after();
            const uint32_t sa = ring_base + stage * kStageBytes, sb = smem_base + (uint32_t)j * slab_bytes;
#pragma unroll
            for (int k = 0; k < kTileK / 16; ++k)
              umma_bf16(d_buf, smem_desc(sa + k * 32), smem_desc(sb + k * 32), idesc, (j == k0 && k == 0) ? 0u : 1u);
            umma_commit(bar_empty + 8 * stage);
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
          if (alive) umma_commit(bar_tfull + 8 * buf);
        }
      }
    }
  } else {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t acc_iter = 0;
    bool alive = true;
    float* Zp = a.Z + (size_t)ks * a.z_stride;
    const bool vec4 = (a.E & 3) == 0;
    for (int i = g; i < n_pairs && alive; i += a.TG) {
      const int t = i / a.n_tiles, tile = i % a.n_tiles;
      const int row0 = (t * a.L + l) * a.S + tile * kTileM;
      const bool row_ok = tile * kTileM + row < a.S;
      float zacc[kEMax];
#pragma unroll
      for (int j = 0; j < kEMax; ++j) zacc[j] = 0.f;
      for (int k0 = 0; k0 < n_k && alive; k0 += kPhaseSlabs, ++acc_iter) {
        const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
        if (!mbar_wait(bar_tfull + 8 * buf, acc_phase, abort_flag, a.err, 25u)) {
          alive = false;
          break;
        }
        tc_fence_after();
        const uint32_t t0 = tmem_base + lane_addr + buf * kBufCols;
#pragma unroll
        for (int c = 0; c < kEMax; c += 16) {
          if (c < a.Epad) {
            float hi[16], mid[16], lo[16];
            tmem_ld16(t0 + c, hi);
            tmem_ld16(t0 + a.Epad + c, mid);
            tmem_ld16(t0 + 2 * a.Epad + c, lo);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) zacc[c + j] = __fadd_rn(zacc[c + j], __fadd_rn(hi[j], __fadd_rn(mid[j], lo[j])));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
      }
      if (alive && row_ok) {
        float* zrow = Zp + (size_t)(row0 + row) * a.E;
        if (vec4) {
#pragma unroll
          for (int c = 0; c < kEMax; c += 4)
            if (c < a.E) *(float4*)(zrow + c) = make_float4(zacc[c], zacc[c + 1], zacc[c + 2], zacc[c + 3]);
        } else {
#pragma unroll
          for (int c = 0; c < kEMax; ++c)
            if (c < a.E) zrow[c] = zacc[c];
        }
      }
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

}  // namespace

bool router_gemm_res_applicable(const mcce_config& c) {
  if (!router_gemm_applicable(c) || c.n_experts > kEMax) return false;
  // the resident terms of the deepest split must leave room for the ring
  const int slabs = c.d_model / kTileK, ks = slabs < kPartsMax ? slabs : kPartsMax;
  const uint32_t res = (uint32_t)((slabs + ks - 1) / ks) * 3u * epad_of(c.n_experts) * kRowBytes;
  return res + kMinStages * kStageBytes + kBarBytes <= kSmemMax;
}

int router_gemm_res_parts_max() { return kPartsMax; }

// Describes the term tensor (written by router_gemm_plan) with a box of Epad expert rows, and fixes the
// K-split of this configuration: the fewest parts whose resident terms fit, then as many more as still
// give every part its own SM at one CTA per (layer, part).
int router_gemm_res_plan(const mcce_config& c, void* terms, RouterGemmPlan* plan) {
  EncodeFn fn = encode_fn();
  if (!fn) return MCCE_ECUDA;
  const int Epad = epad_of(c.n_experts);
  const cuuint64_t dims[3] = {(cuuint64_t)c.d_model, (cuuint64_t)c.n_experts, (cuuint64_t)3 * c.n_layers};
  const cuuint64_t strides[2] = {(cuuint64_t)c.d_model * 2, (cuuint64_t)c.d_model * 2 * c.n_experts};
  const cuuint32_t box[3] = {(cuuint32_t)kTileK, (cuuint32_t)Epad, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (fn(&plan->w_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, terms, dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return MCCE_ECUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MCCE_ECUDA;
  const int slabs = c.d_model / kTileK;
  const uint32_t slab_bytes = 3u * Epad * kRowBytes;
  int ks = 1;
  while ((uint32_t)((slabs + ks - 1) / ks) * slab_bytes + kMinStages * kStageBytes + kBarBytes > kSmemMax) ++ks;
  while (ks < kPartsMax && ks < slabs && c.n_layers * (ks + 1) <= sms) ++ks;
  plan->res_parts = ks;
  plan->res_ready = 1;
  return MCCE_OK;
}

// Partial logits of n_steps tokens of all layers: Z holds res_parts arrays of n_steps*L*S*E floats.
cudaError_t router_gemm_res_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps,
                                   float* Z, uint32_t* err, cudaStream_t st) {
  static int cache[64] = {0};
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(router_gemm_res_kernel, (size_t)kSmemMax + 1024, cache, &sms);
  if (e0 != cudaSuccess) return e0;
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
  ResArgs a;
  a.L = c.n_layers, a.S = c.n_streams, a.E = c.n_experts, a.Epad = epad_of(c.n_experts), a.n_steps = n_steps;
  a.KS = plan.res_parts, a.slabs = c.d_model / kTileK;
  a.n_tiles = (c.n_streams + kTileM - 1) / kTileM;
  // more CTAs per (layer, part), each taking every TG-th (token, stream tile) pair, while SMs would idle
  const int pairs = n_steps * a.n_tiles;
  int tg = 1;
  while (tg < pairs && a.L * a.KS * (tg + 1) <= sms) ++tg;
  a.TG = tg;
  const uint32_t res = (uint32_t)((a.slabs + a.KS - 1) / a.KS) * 3u * a.Epad * kRowBytes;
  a.res_bytes = (res + 1023u) & ~1023u;
  int stages = (int)((kSmemMax - kBarBytes - a.res_bytes) / kStageBytes);
  a.n_stages = stages > kMaxStages ? kMaxStages : stages;
  a.Z = Z, a.z_stride = (size_t)rows * c.n_experts, a.err = err;
  ResMaps m;
  m.w = plan.w_res, m.x = plan.x_res, m.xt = plan.xt_res;
  router_gemm_res_kernel<<<a.L * a.KS * a.TG, kThreads, (size_t)kSmemMax + 1024, st>>>(m, a);
  return cudaGetLastError();
}

}  // namespace mcce
