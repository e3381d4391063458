// Router logits of Eq. 3 on the tensor cores: Z[(t,l,s), e] = sum_j W_r[l][e][j] x[(t,l,s)][j].
//
// Every stream of a layer shares the layer's router matrix, so the S GEMVs of a layer are one GEMM.  The
// routing decision needs near-fp32 logits (ties are resolved at 1e-4), while tcgen05 multiplies bf16:
// the fp32 router is therefore split once, at set-up, into three bf16 terms W = hi + mid + lo (each the
// bf16 rounding of what the previous terms left), and the kernel accumulates the three products in the
// fp32 TMEM accumulators.  The hidden states are bf16 already, so every product is exact.
//
// Accuracy: the tensor core's fp32 accumulate truncates, which over the 3*d/16 accumulate steps of one
// logit would add up to a bias of about 1e-5 relative.  The kernel therefore (i) keeps the large hi
// products and the small mid/lo products in separate accumulators, and (ii) ends an accumulation phase
// every kPhaseSlabs K-slabs: the epilogue warps add each phase's two partial sums into fp32 registers
// with round-to-nearest adds while the MMA warp continues in the other TMEM buffer.
//
// Speed: a tcgen05.mma costs about 110 cycles to issue whatever N <= 128 is, so the kernel is bound by the
// number of MMAs: the stream tile is as wide as TMEM allows with two accumulator buffers (N = 128), and the
// reduction is split over up to eight CTAs per tile so that all SMs have work at one token per launch.
//
// Layout of the work: swapped GEMM as in the expert kernels -- router rows (experts) are MMA M (tiles of
// 128, rows past E zero-filled by TMA at no memory cost), a block of streams is MMA N, the hidden
// dimension is K in 64-column slabs.  Persistent CTAs walk (token, layer, expert tile, stream block)
// items: warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue (TMEM -> fp32 logits in HBM), with
// bounded mbarrier waits throughout.  The fused routing tail then runs on these logits.
#include "common.cuh"
#include "tc_common.cuh"

namespace mcce {

using namespace tc;

namespace {

constexpr int kTileM = 128, kTileK = 64, kNSMax = 128, kXBox = 16, kThreads = 192, kMaxStages = 12;
constexpr uint32_t kRowBytes = kTileK * 2;                 // one 128-byte swizzle row
// The stage ring.  A stage holds the three bf16 terms of a router slab -- only the RA rows that exist
// (E rounded up to 8, at most 128) -- and the stream rows.  The MMA always reads 128 rows from a term's
// start; rows past RA are whatever follows in the ring (finite or not, they only reach accumulator
// rows of experts that do not exist), so the last 16 KB of the ring are never used as a stage start.
constexpr uint32_t kRingBytes = 208 * 1024, kTermReadBytes = kTileM * kRowBytes;
constexpr int kAccSets = 1;                                // independent accumulator sets (alternate k-steps)
constexpr int kAccCols = 2 * kAccSets * kNSMax, kTmemCols = 2 * kAccCols;  // per buffer: sets x {hi, mid/lo}; 2 buffers
constexpr int kPhaseSlabs = 4;                             // K-slabs (of 64) per accumulation phase
constexpr size_t kSmemBytes = (size_t)kRingBytes + 1024 + 256;

struct GemmArgs {
  int L, S, E, d, n_steps, NS;
  int l0, L_terms; // first layer of this launch; layers in the term tensor (stride between the three terms)
  int RA;          // router rows per term tile actually loaded
  int KS, kt_per;  // K-split: partial sums over kt_per slabs each
  int n_stages;
  uint32_t stage_bytes;
  int n_items;
  float* Z;        // [KS][n_steps, L, S, E] partial logits
  size_t z_stride; // elements between partials
  uint32_t* err;
};
struct GemmMaps {
  CUtensorMap w;   // 3-D: [3*L][E][d] bf16 terms (term-major), box 1 x 128 x 64
  CUtensorMap x;   // 2-D: [n_steps*L*S][d] hidden rows, box 16 x 64
};

struct GItem {
  int l, mt, ks, s0, row0;  // layer, expert tile, K part, first stream, first hidden row (t*L + l)*S + s0
};

__device__ __forceinline__ GItem decode(const GemmArgs& a, int w) {
  const int SB = (a.S + a.NS - 1) / a.NS, MT = (a.E + kTileM - 1) / kTileM;
  GItem it;
  const int sb = w % SB;
  it.ks = (w / SB) % a.KS;
  w /= SB * a.KS;
  it.mt = w % MT;
  it.l = (w / MT) % a.L;
  const int t = w / (MT * a.L);
  it.s0 = sb * a.NS;
  it.row0 = (t * a.L + it.l) * a.S + it.s0;
  return it;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
router_gemm_kernel(const __grid_constant__ GemmMaps maps, const GemmArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(smem_al + (size_t)kRingBytes);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kMaxStages;
  const uint32_t bar_tfull = bar_empty + 8 * kMaxStages, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * kMaxStages + 4);
  const uint32_t kStages = (uint32_t)a.n_stages, kStageBytes = a.stage_bytes;
  const uint32_t kABytes = (uint32_t)a.RA * kRowBytes;
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KT = a.kt_per;
  const uint32_t n = (uint32_t)a.NS;   // MMA N: multiple of 16

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 4);
    }
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
      uint32_t stage = 0, phase = 0;
      bool alive = true;
      const uint32_t tx = 3 * kABytes + n * kTileK * 2;
      for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
        const GItem it = decode(a, w);
        for (int kt = it.ks * KT; kt < (it.ks + 1) * KT; ++kt) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.err, 11u)) {
            alive = false;
            break;
          }
          const uint32_t sa = smem_base + stage * kStageBytes, full = bar_full + 8 * stage;
          mbar_expect_tx(full, tx);
#pragma unroll
          for (int p = 0; p < 3; ++p)
            tma_load_3d(sa + p * kABytes, &maps.w, kt * kTileK, it.mt * kTileM, p * a.L_terms + a.l0 + it.l, full);
          const uint32_t sb = sa + 3 * kABytes;
          for (int j = 0; j < a.NS; j += kXBox)
            tma_load_2d(sb + j * kTileK * 2, &maps.x, kt * kTileK, it.row0 + j, full);
          if (++stage == kStages) stage = 0, phase ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, acc_iter = 0;
      bool alive = true;
      const uint32_t idesc = instr_desc(n);
      for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
        for (int k0 = 0; k0 < KT && alive; k0 += kPhaseSlabs, ++acc_iter) {
          const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
          if (!mbar_wait(bar_tempty + 8 * buf, acc_phase ^ 1u, abort_flag, a.err, 12u)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_buf = tmem_base + buf * kAccCols;
          const int k1 = min(KT, k0 + kPhaseSlabs);
          for (int kt = k0; kt < k1; ++kt) {
            if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.err, 13u)) {
              alive = false;
              break;
            }
            tc_fence_after();
            const uint32_t sa = smem_base + stage * kStageBytes, sb = sa + 3 * kABytes;
#pragma unroll
            for (int k = 0; k < kTileK / 16; ++k) {
              const uint64_t bd = smem_desc(sb + k * 32);
              const uint32_t first = (kt == k0 && k < kAccSets) ? 0u : 1u;
              const uint32_t d_hi = d_buf + (k % kAccSets) * 2 * kNSMax, d_lo = d_hi + kNSMax;
              umma_bf16(d_hi, smem_desc(sa + k * 32), bd, idesc, first);
              umma_bf16(d_lo, smem_desc(sa + kABytes + k * 32), bd, idesc, first);
              umma_bf16(d_lo, smem_desc(sa + 2 * kABytes + k * 32), bd, idesc, 1u);
            }
            umma_commit(bar_empty + 8 * stage);
            if (++stage == kStages) stage = 0, phase ^= 1u;
          }
          if (alive) umma_commit(bar_tfull + 8 * buf);
        }
      }
    }
  } else {
    const int quad = warp & 3;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t acc_iter = 0;
    bool alive = true;
    for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
      const GItem it = decode(a, w);
      const int e = it.mt * kTileM + quad * 32 + lane;
      float zacc[kNSMax];
#pragma unroll
      for (int j = 0; j < kNSMax; ++j) zacc[j] = 0.f;
      for (int k0 = 0; k0 < KT && alive; k0 += kPhaseSlabs, ++acc_iter) {
        const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
        if (!mbar_wait(bar_tfull + 8 * buf, acc_phase, abort_flag, a.err, 14u)) {
          alive = false;
          break;
        }
        tc_fence_after();
        const uint32_t t0 = tmem_base + lane_addr + buf * kAccCols;
#pragma unroll
        for (int n0 = 0; n0 < kNSMax; n0 += 16) {
          if (n0 < a.NS) {
            float hi[16], lo[16];
            tmem_ld16(t0 + n0, hi);
            tmem_ld16(t0 + kNSMax + n0, lo);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) zacc[n0 + j] = __fadd_rn(zacc[n0 + j], __fadd_rn(hi[j], lo[j]));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
      }
      if (alive && e < a.E) {
#pragma unroll
        for (int j = 0; j < kNSMax; ++j)
          if (j < a.NS && it.s0 + j < a.S) a.Z[it.ks * a.z_stride + (size_t)(it.row0 + j) * a.E + e] = zacc[j];
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

// Self-test of the bounded wait: one CTA waits on an mbarrier that nothing will ever arrive at; the wait
// must give up after limit_ns, record the error word and let the kernel return normally.
__global__ void wait_timeout_selftest_kernel(uint32_t* err, unsigned long long limit_ns, uint32_t* outcome) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, err, 99u, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0) *outcome = ok ? 1u : 2u;   // 2: the wait gave up, as it must
}

// W (fp32) -> hi, mid, lo (bf16): each term is the bf16 rounding of what the earlier terms left over.
__global__ void split_router_kernel(const float* W, __nv_bfloat16* out, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const float w = W[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
    const float r1 = __fsub_rn(w, __bfloat162float(hi));
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const float r2 = __fsub_rn(r1, __bfloat162float(mid));
    out[i] = hi;
    out[n + i] = mid;
    out[2 * n + i] = __float2bfloat16_rn(r2);
  }
}

}  // namespace

// Router rows loaded per term tile: all 128 of a full tile, else E rounded up to the 8-row swizzle group.
static int term_rows(int E) { return E >= kTileM ? kTileM : (E + 7) & ~7; }

cudaError_t launch_wait_timeout_selftest(uint32_t* err, unsigned long long limit_ns, uint32_t* outcome,
                                         cudaStream_t st) {
  wait_timeout_selftest_kernel<<<1, 64, 0, st>>>(err, limit_ns, outcome);
  return cudaGetLastError();
}

bool router_gemm_applicable(const mcce_config& c) { return c.hidden_dtype == MCCE_BF16 && c.d_model % kTileK == 0; }

int router_gemm_steps_max() { return 8; }

// Splits the router into its bf16 terms (device buffer `terms`, 3*L*E*d bf16) and describes them to TMA.
int router_gemm_plan(const mcce_config& c, const float* Wr, void* terms, RouterGemmPlan* plan, cudaStream_t st) {
  const size_t n = (size_t)c.n_layers * c.n_experts * c.d_model;
  split_router_kernel<<<(unsigned)((n + 255) / 256 > 4096 ? 4096 : (n + 255) / 256), 256, 0, st>>>(
      Wr, (__nv_bfloat16*)terms, n);
  if (cudaGetLastError() != cudaSuccess) return MCCE_ECUDA;
  EncodeFn fn = encode_fn();
  if (!fn) return MCCE_ECUDA;
  const cuuint64_t dims[3] = {(cuuint64_t)c.d_model, (cuuint64_t)c.n_experts, (cuuint64_t)3 * c.n_layers};
  const cuuint64_t strides[2] = {(cuuint64_t)c.d_model * 2, (cuuint64_t)c.d_model * 2 * c.n_experts};
  const cuuint32_t box[3] = {(cuuint32_t)kTileK, (cuuint32_t)term_rows(c.n_experts), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (fn(&plan->w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, terms, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return MCCE_ECUDA;
  plan->hidden_ptr = nullptr;
  plan->hidden_rows = 0;
  plan->ready = 1;
  return MCCE_OK;
}

cudaError_t router_gemm_launch(RouterGemmPlan& plan, const mcce_config& c, const void* hidden, int n_steps, float* Z,
                               int* k_split, uint32_t* err, cudaStream_t st, int l0, int n_layers) {
  const int Ls = n_layers > 0 ? n_layers : c.n_layers;   // layers [l0, l0 + Ls) of the model; hidden holds those only
  static int cache[64] = {0};
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(router_gemm_kernel, kSmemBytes, cache, &sms);
  if (e0 != cudaSuccess) return e0;
  const uint64_t rows = (uint64_t)n_steps * Ls * c.n_streams;
  if (plan.hidden_ptr != hidden || plan.hidden_rows != rows) {
    EncodeFn fn = encode_fn();
    const cuuint64_t dims[2] = {(cuuint64_t)c.d_model, rows};
    const cuuint64_t strides[1] = {(cuuint64_t)c.d_model * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)kXBox};
    const cuuint32_t estr[2] = {1, 1};
    if (!fn || fn(&plan.x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    plan.hidden_ptr = hidden;
    plan.hidden_rows = rows;
  }
  GemmArgs a;
  a.L = Ls, a.S = c.n_streams, a.E = c.n_experts, a.d = c.d_model, a.n_steps = n_steps;
  a.l0 = l0, a.L_terms = c.n_layers;
  // streams per tile: as many as TMEM holds; narrower only when even the deepest K-split would leave most SMs idle
  int ns = c.n_streams >= kNSMax ? kNSMax : (c.n_streams + 15) & ~15;
  const int mt = (c.n_experts + kTileM - 1) / kTileM;
  const int kt = c.d_model / kTileK;
  int ks_max = 1;
  while (ks_max < 8 && kt % (2 * ks_max) == 0 && kt / (2 * ks_max) >= 4 && n_steps * 2 * ks_max <= router_gemm_steps_max())
    ks_max *= 2;
  while (ns > 16 && n_steps * Ls * mt * ((c.n_streams + ns - 1) / ns) * ks_max < sms / 2) ns /= 2;
  ns = (ns + 15) & ~15;
  a.NS = ns;
  // split the reduction over up to eight CTAs per tile while SMs would otherwise idle; the partial
  // logits are summed by the routing tail.  The logits buffer has router_gemm_steps_max() slots.
  const int items = n_steps * Ls * mt * ((c.n_streams + ns - 1) / ns);
  // Cost of a split, from measurements on B200: a round of the persistent grid costs about 1 us per K-slab
  // of its items (twelve MMAs) plus about 5 us of fill and drain, so one round of shorter items wins.
  int ks = 1;
  double best = (double)((items + sms - 1) / sms) * (kt * 1.0 + 5.0);
  for (int cand = 2; cand <= 8; cand *= 2) {
    if (kt % cand || kt / cand < 4 || n_steps * cand > router_gemm_steps_max()) break;
    const double cost = (double)((items * cand + sms - 1) / sms) * (kt / cand * 1.0 + 5.0);
    if (cost < best - 1e-9) best = cost, ks = cand;
  }
  a.KS = ks, a.kt_per = kt / ks;
  a.n_items = items * ks;
  a.RA = term_rows(c.n_experts);
  a.stage_bytes = (uint32_t)(3 * a.RA + ns) * kRowBytes;
  a.n_stages = (int)((kRingBytes - kTermReadBytes) / a.stage_bytes);
  if (a.n_stages > kMaxStages) a.n_stages = kMaxStages;
  a.Z = Z, a.z_stride = (size_t)rows * c.n_experts, a.err = err;
  *k_split = ks;
  GemmMaps m;
  m.w = plan.w, m.x = plan.x;
  const int grid = a.n_items < sms ? a.n_items : sms;
  router_gemm_kernel<<<grid, kThreads, kSmemBytes, st>>>(m, a);
  return cudaGetLastError();
}

}  // namespace mcce
