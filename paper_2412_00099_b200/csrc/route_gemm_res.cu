// Router logits of Eq. 3 on the tensor cores, router-resident form, as a kernel of its own: every CTA runs the
// three roles of route_gemm_res.cuh (one layer, one K part, every TG-th (token, stream tile) pair of the layer)
// and stores the partial logits of its K part; the routing tail sums the parts in a fixed order.
#include "route_gemm_res.cuh"

namespace mcce {

using namespace rres;

namespace {

constexpr int kThreads = 192;

struct ResArgs {
  Geometry g;
  int TG;
  float* Z;             // [KS][n_steps, L, S, E] partial logits
  size_t z_stride;
  uint32_t* err;
};

__global__ void __launch_bounds__(kThreads, 1)
router_gemm_res_kernel(const __grid_constant__ Maps maps, const ResArgs args) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const Geometry& a = args.g;
  const Smem m = carve(smem_raw, a);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA: layer l, K part ks, pair group g
  const int g = blockIdx.x % args.TG;
  const int ks = (blockIdx.x / args.TG) % a.KS;
  const int l = blockIdx.x / (args.TG * a.KS);
  const KPart kp = k_part_of(a, ks);
  const int n_pairs = a.n_steps * a.n_tiles;

  if (threadIdx.x == 0) init_barriers(m);
  if (warp == 1) tmem_alloc(smem_u32(m.tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *m.tmem_slot;

  if (warp == 0) {
    if (lane == 0) produce(maps, a, m, l, kp, g, args.TG, args.err, 21u);
  } else if (warp == 1) {
    if (lane == 0) issue_mmas(a, m, tmem_base, kp, g, args.TG, args.err, 21u);
  } else {
    const int quad = warp & 3, row = quad * 32 + lane;
    float* Zp = args.Z + (size_t)ks * args.z_stride;
    uint32_t it = 0;
    for (int i = g; i < n_pairs; i += args.TG, ++it) {
      const int t = i / a.n_tiles, tile = i % a.n_tiles;
      const int row0 = (t * a.L + l) * a.S + tile * kTileM;
      if (!drain_pair<false>(a, m, tmem_base, kp.n_k(i), it, quad, lane, Zp + (size_t)(row0 + row) * a.E, tile * kTileM + row < a.S,
                      args.err, 25u))
        break;
    }
  }
  teardown(m, tmem_base, warp, 1);
}

}  // namespace

bool router_gemm_res_applicable(const mcce_config& c) {
  if (!router_gemm_applicable(c) || c.n_experts > kEMax) return false;
  // the resident terms of the deepest split must leave room for the ring, and its accumulator sets must fit TMEM
  const int slabs = c.d_model / kTileK, ks = slabs < kPartsMax ? slabs : kPartsMax, Epad = epad_of(c.n_experts);
  return res_bytes_of(slabs, ks, Epad) + kMinStages * kStageBytes + kBarBytes <= kSmemMax && sets_fit(slabs, ks, Epad);
}

int router_gemm_res_parts_max() { return kPartsMax; }

// Describes the term tensor (written by router_gemm_plan) with a box of Epad expert rows, and fixes the
// K-split of this configuration: the fewest parts whose resident terms and accumulator sets fit, then as many
// more as still give every part its own SM at one CTA per (layer, part).
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
  int ks = 1;
  while (res_bytes_of(slabs, ks, Epad) + kMinStages * kStageBytes + kBarBytes > kSmemMax || !sets_fit(slabs, ks, Epad)) ++ks;
  const int ks_min = ks;
  while (ks < kPartsMax && ks < slabs && c.n_layers * (ks + 1) <= sms) ++ks;
  plan->res_parts = ks;
  // launches of one layer at a time (sequential-layer mode): the split a one-layer model would get
  int ks1 = ks_min;
  while (ks1 < kPartsMax && ks1 < slabs && ks1 + 1 <= sms) ++ks1;
  plan->res_parts_single = ks1;
  plan->res_ready = 1;
  return MCCE_OK;
}

// Partial logits of n_steps tokens of all layers (or, with n_layers = 1, of model layer l0 alone: hidden and Z
// then hold that layer only): Z receives *k_parts arrays of n_steps*layers*S*E floats.
cudaError_t router_gemm_res_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps,
                                   float* Z, int* k_parts, uint32_t* err, cudaStream_t st, int l0, int n_layers) {
  const int Ls = n_layers > 0 ? n_layers : c.n_layers;
  static int cache[64] = {0};
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(router_gemm_res_kernel, (size_t)kSmemMax + 1024, cache, &sms);
  if (e0 != cudaSuccess) return e0;
  const uint64_t rows = (uint64_t)n_steps * Ls * c.n_streams;
  e0 = hidden_maps(plan, hidden, rows, c.d_model, c.n_streams);
  if (e0 != cudaSuccess) return e0;
  ResArgs args;
  Geometry& a = args.g;
  a.L = Ls, a.l0 = l0, a.L_terms = c.n_layers;
  a.S = c.n_streams, a.E = c.n_experts, a.Epad = epad_of(c.n_experts), a.n_steps = n_steps;
  a.KS = Ls == c.n_layers ? plan.res_parts : plan.res_parts_single, a.slabs = c.d_model / kTileK;
  *k_parts = a.KS;
  a.n_tiles = (c.n_streams + kTileM - 1) / kTileM;
  // more CTAs per (layer, part), each taking every TG-th (token, stream tile) pair, while SMs would idle
  const int pairs = n_steps * a.n_tiles;
  int tg = 1;
  while (tg < pairs && a.L * a.KS * (tg + 1) <= sms) ++tg;
  args.TG = tg;
  a.res_bytes = res_bytes_of(a.slabs, a.KS, a.Epad);
  a.n_stages = stages_of(a.res_bytes);
  args.Z = Z, args.z_stride = (size_t)rows * c.n_experts, args.err = err;
  Maps m;
  m.w = plan.w_res, m.x = plan.x_res, m.xt = plan.xt_res;
  router_gemm_res_kernel<<<a.L * a.KS * tg, kThreads, (size_t)kSmemMax + 1024, st>>>(m, args);
  return cudaGetLastError();
}

}  // namespace mcce
