// Grouped SwiGLU expert FFN of Eq. 1 on the 5th-generation tensor cores: a persistent, warp-specialised
// weight streamer.
//
// At decode batch sizes every expert sees only tens of tokens, so the work is bound by streaming each
// touched expert's weights from HBM exactly once.  The GEMMs are therefore "swapped": the weight rows
// are the MMA M dimension (tiles of 128 rows), the expert's tokens are the N dimension (16..128 per
// instruction), and the reduction runs over the hidden (gate/up) or intermediate (down) dimension:
//
//     up  :  G^T, U^T [128 x N] = Wg, Wu [128 x d] * X_e^T [d x N];   H = bf16(silu(G) * U)
//     down:  O^T      [128 x N] = Wd     [128 x I] * H_e^T [I x N]
//
// One CTA per SM walks a static list of (layer, expert, 128-row tile) items.  Warp 0 issues TMA loads
// (128B-swizzled 64-column slabs of the weight tile and of the token rows) into a ring of shared-memory
// stages, warp 1 issues tcgen05.mma into one of two TMEM accumulator buffers, warps 2-5 drain the other
// buffer with tcgen05.ld and apply the epilogue: SwiGLU and a bf16 store of H (up), or the weighted
// combine of Eq. 1 straight into y with fp32 atomic adds (down; y is zeroed first, and since the order
// of a stream's K + shared addends is not fixed, the last bits of y may differ from run to run).  In the
// deterministic mode the down kernel instead stores one fp32 row per (stream, slot) and a second pass adds
// them in slot order.  Every wait on an mbarrier is bounded: on a timeout the CTA records an error word,
// stops, releases its TMEM and returns.
#include <cuda.h>

#include "ffn_tc.cuh"
#include "tc_common.cuh"

namespace mcce {

using namespace tc;

namespace {

constexpr int kTileM = 128;   // weight rows per tile
constexpr int kTileK = 64;    // reduction slab: 64 bf16 = one 128-byte swizzle row
constexpr int kNMax = 128;    // tokens per pass over a weight tile
constexpr int kXBox = 16;     // token rows per TMA box
constexpr int kThreads = 192;
constexpr uint32_t kABytes = kTileM * kTileK * 2;   // 16 KB
constexpr uint32_t kBBytes = kNMax * kTileK * 2;    // 16 KB

template <bool UP>
struct Cfg {
  // Both kernels stream TWO 128-row weight tiles per stage against one tile of token rows: gate and up
  // rows of the same range (up), or two consecutive row ranges of W_d (down).  The token rows come
  // from L2 but still count against what an SM can take in per microsecond, so sharing them between
  // two weight tiles is worth 10 % on the down kernel.
  static constexpr int kStages = 4;
  static constexpr uint32_t kStageBytes = 2 * kABytes + kBBytes;
  static constexpr int kAccCols = 2 * kNMax;                // TMEM columns per accumulator buffer
  static constexpr int kTmemCols = 2 * kAccCols;            // two buffers: 512
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
};

// The tensor core's fp32 accumulate truncates, which over the hundreds of accumulation steps of a long reduction
// adds up to a relative bias of about 1e-5 -- enough to flip the bf16 rounding of H in a few dozen places per
// token and expert.  A pass over few tokens therefore spreads its K-slabs round-robin over up to four accumulator
// sets (each in its own TMEM columns, as many as fit beside each other), and the epilogue adds the sets in
// round-to-nearest fp32: each accumulator then sees a quarter of the steps.
__host__ __device__ __forceinline__ int acc_sets(int n_pad, int KT) {
  const int s = n_pad <= 32 ? 4 : n_pad <= 64 ? 2 : 1;
  return s < KT ? s : (KT >= 2 ? 2 : 1);
}

struct TcArgs {
  int L, S, E, K, n_sh, d, I;
  int l0;                // model layer of local layer 0 (weights are indexed by model layer)
  int n_items;
  const int32_t* offsets;
  const int32_t* perm;   // [L, S*K] position -> pair, for the fused combine of the down kernel
  const float* sel_w;    // [L, S, K]
  __nv_bfloat16* H;
  float* y;              // [L, S, d], zeroed before the down kernel; receives w * E_i(x) by fp32 atomic adds
  float* O;              // [rows, d] expert outputs per (stream, slot), deterministic mode only
  uint32_t* err;
};

struct TcMaps {
  CUtensorMap w0, w1, sw0, sw1;  // routed / shared weights (w1, sw1 only in the up kernel)
  CUtensorMap x, xs;             // token rows of routed groups / of shared experts
};

// ---- the list of work items ----------------------------------------------------------------------------
// Per layer: one item per (routed expert, 128-row tile), covering all of the expert's tokens (in passes
// of kNMax), then one item per (shared expert, 128-row tile, 128-token pass).  A shared expert sees
// every stream, so its passes are separate, adjacent items: neighbouring CTAs run them at the same
// time and the second read of the weight tile is served by L2 instead of HBM.
struct Item {
  int m;          // tokens this item covers
  int wrow;       // first row of the 128-row weight tile in the weight tensor map
  int xrow;       // first token row in the activation tensor map
  size_t orow;    // first row in H / O
  int col0;       // first output column (= weight row inside the expert) of this tile
  int l;          // layer
  int ntile;      // weight tiles in this item: 2, or 1 for the last odd row range of the down kernel
  bool shared;
};

__host__ __device__ __forceinline__ int items_per_layer(int E, int n_sh, int S, int RT) {
  return E * RT + n_sh * RT * ((S + kNMax - 1) / kNMax);
}

template <bool UP>
__device__ __forceinline__ Item decode(const TcArgs& a, int w) {
  const int rows = UP ? a.I : a.d;
  const int span = UP ? kTileM : 2 * kTileM;   // output features covered by one item
  const int RT = (rows + span - 1) / span, P = a.S * a.K, NC = (a.S + kNMax - 1) / kNMax;
  const int per_layer = items_per_layer(a.E, a.n_sh, a.S, RT);
  const int l = w / per_layer, wl = w % per_layer;
  Item it;
  it.l = l;
  if (wl < a.E * RT) {
    const int g = wl / RT;
    it.col0 = (wl % RT) * span;
    const int o0 = __ldg(a.offsets + (size_t)l * (a.E + 1) + g);
    it.m = min(max(__ldg(a.offsets + (size_t)l * (a.E + 1) + g + 1) - o0, 0), P);   // never beyond a layer's pairs
    it.shared = false;
    it.wrow = ((a.l0 + l) * a.E + g) * rows + it.col0;
    it.xrow = l * P + o0;
    it.orow = (size_t)it.xrow;
  } else {
    const int idx = wl - a.E * RT;
    const int c = idx % NC, rt = (idx / NC) % RT, q = idx / (NC * RT);
    it.col0 = rt * span;
    it.m = min(kNMax, a.S - c * kNMax);
    it.shared = true;
    it.wrow = ((a.l0 + l) * a.n_sh + q) * rows + it.col0;
    it.orow = (size_t)a.L * P + (size_t)(l * a.n_sh + q) * a.S + c * kNMax;
    it.xrow = UP ? l * a.S + c * kNMax : (int)it.orow;   // up: rows of the hidden tensor; down: rows of H
  }
  it.ntile = (UP || it.col0 + 2 * kTileM <= rows) ? 2 : 1;
  return it;
}

// UP: gate/up projection.  Otherwise the down projection, which either adds w * E_i(x) into y (ROWS_OUT
// false) or stores the unweighted expert outputs row by row into O (ROWS_OUT true, deterministic mode).
template <bool UP, bool ROWS_OUT>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using C = Cfg<UP>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(smem_al + (size_t)C::kStages * C::kStageBytes);
  // barrier slots: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2]
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * C::kStages;
  const uint32_t bar_tfull = bar_empty + 8 * C::kStages, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * C::kStages + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int R = UP ? a.d : a.I;       // reduction length
  const int KT = R / kTileK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
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
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---- TMA producer --------------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool alive = true;
      Item nxt = decode<UP>(a, min((int)blockIdx.x, a.n_items - 1));
      for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
        const Item it = nxt;   // the next item's group offsets are fetched while this one streams
        if (w + (int)gridDim.x < a.n_items) nxt = decode<UP>(a, w + gridDim.x);
        const CUtensorMap* mw0 = it.shared ? &maps.sw0 : &maps.w0;
        const CUtensorMap* mw1 = it.shared ? &maps.sw1 : &maps.w1;
        const CUtensorMap* mx = it.shared ? &maps.xs : &maps.x;
        for (int c0 = 0; c0 < it.m && alive; c0 += kNMax) {
          const int n = (min(kNMax, it.m - c0) + 15) & ~15;
          const uint32_t tx = (uint32_t)it.ntile * kABytes + (uint32_t)n * kTileK * 2;
          for (int kt = 0; kt < KT; ++kt) {
            if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.err, 1u)) {
              alive = false;
              break;
            }
            const uint32_t sa = smem_base + stage * C::kStageBytes;
            const uint32_t full = bar_full + 8 * stage;
            mbar_expect_tx(full, tx);
            tma_load_2d(sa, mw0, kt * kTileK, it.wrow, full);
            if (UP) tma_load_2d(sa + kABytes, mw1, kt * kTileK, it.wrow, full);
            else if (it.ntile == 2) tma_load_2d(sa + kABytes, mw0, kt * kTileK, it.wrow + kTileM, full);
            const uint32_t sb = sa + 2 * kABytes;
            for (int j = 0; j < n; j += kXBox)
              tma_load_2d(sb + j * kTileK * 2, mx, kt * kTileK, it.xrow + c0 + j, full);
            if (++stage == C::kStages) stage = 0, phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer ------------------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, acc_iter = 0;
      bool alive = true;
      Item nxt = decode<UP>(a, min((int)blockIdx.x, a.n_items - 1));
      for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
        const Item it = nxt;
        if (w + (int)gridDim.x < a.n_items) nxt = decode<UP>(a, w + gridDim.x);
        for (int c0 = 0; c0 < it.m && alive; c0 += kNMax, ++acc_iter) {
          const uint32_t n = (uint32_t)(min(kNMax, it.m - c0) + 15) & ~15u;
          const uint32_t idesc = instr_desc(n);
          const int sets = acc_sets((int)n, KT);
          const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
          if (!mbar_wait(bar_tempty + 8 * buf, acc_phase ^ 1u, abort_flag, a.err, 2u)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d0 = tmem_base + buf * C::kAccCols;
          for (int kt = 0; kt < KT; ++kt) {
            if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.err, 3u)) {
              alive = false;
              break;
            }
            tc_fence_after();
            const uint32_t sa = smem_base + stage * C::kStageBytes;
            const uint32_t sb = sa + 2 * kABytes;
#pragma unroll
            const uint32_t ds = d0 + (uint32_t)(kt % sets) * n;   // this slab's accumulator set
            for (int k = 0; k < kTileK / 16; ++k) {
              const uint32_t acc = (kt >= sets || k > 0) ? 1u : 0u;
              const uint64_t bd = smem_desc(sb + k * 32);
              umma_bf16(ds, smem_desc(sa + k * 32), bd, idesc, acc);
              if (it.ntile == 2) umma_bf16(ds + kNMax, smem_desc(sa + kABytes + k * 32), bd, idesc, acc);
            }
            umma_commit(bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
            if (++stage == C::kStages) stage = 0, phase ^= 1u;
          }
          if (alive) umma_commit(bar_tfull + 8 * buf);
        }
      }
    }
  } else {
    // ---- epilogue warps: TMEM -> registers -> global ---------------------------------------------------
    const int quad = warp & 3;                         // TMEM lane quadrant this warp may read
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t acc_iter = 0;
    bool alive = true;
    Item nxt = decode<UP>(a, min((int)blockIdx.x, a.n_items - 1));
    for (int w = blockIdx.x; w < a.n_items && alive; w += gridDim.x) {
      const Item it = nxt;
      if (w + (int)gridDim.x < a.n_items) nxt = decode<UP>(a, w + gridDim.x);
      const int col = it.col0 + quad * 32 + lane;      // output feature handled by this thread
      for (int c0 = 0; c0 < it.m && alive; c0 += kNMax, ++acc_iter) {
        const int ntok = min(kNMax, it.m - c0);
        const int n = (ntok + 15) & ~15;
        const uint32_t buf = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
        if (!mbar_wait(bar_tfull + 8 * buf, acc_phase, abort_flag, a.err, 4u)) {
          alive = false;
          break;
        }
        tc_fence_after();
        const uint32_t t0 = tmem_base + lane_addr + buf * C::kAccCols;
        const int sets = acc_sets(n, KT);
        // sum of the accumulator sets of 16 columns starting at column `col0` of the buffer
        auto ld_sets = [&](uint32_t col0, float (&v)[16]) {
          tmem_ld16(t0 + col0, v);
          for (int sidx = 1; sidx < sets; ++sidx) {
            float w[16];
            tmem_ld16(t0 + col0 + (uint32_t)(sidx * n), w);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __fadd_rn(v[j], w[j]);
          }
        };
        for (int n0 = 0; n0 < n; n0 += 16) {
          float g[16];
          ld_sets((uint32_t)n0, g);
          if (UP) {
            float u[16];
            ld_sets((uint32_t)(kNMax + n0), u);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              if (n0 + j < ntok) {
                const float h = __fdividef(g[j], 1.f + __expf(-g[j])) * u[j];
                a.H[(it.orow + c0 + n0 + j) * a.I + col] = __float2bfloat16_rn(h);
              }
            }
          } else if (ROWS_OUT) {
            float g2[16];
            if (it.ntile == 2) ld_sets((uint32_t)(kNMax + n0), g2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              if (n0 + j < ntok) {
                float* o = a.O + (it.orow + c0 + n0 + j) * a.d + col;
                o[0] = g[j];
                if (it.ntile == 2) o[kTileM] = g2[j];
              }
            }
          } else {
            // Eq. 1 combine, fused: y[l, s, :] += w * o.  Lane j looks up the stream and weight of token
            // n0 + j; all lanes then add their column of that token (32 consecutive floats per warp).
            int my_dst = -1;
            float my_w = 0.f;
            if (lane < 16 && n0 + lane < ntok) {
              const size_t r = it.orow + c0 + n0 + lane;
              if (it.shared) {
                my_dst = it.l * a.S + (int)((r - (size_t)a.L * a.S * a.K) % a.S);
                my_w = 1.f;
              } else {
                const int pair = __ldg(a.perm + r);
                my_dst = it.l * a.S + pair / a.K;
                my_w = __ldg(a.sel_w + (size_t)it.l * a.S * a.K + pair);
              }
            }
            float g2[16];
            if (it.ntile == 2) ld_sets((uint32_t)(kNMax + n0), g2);   // second row range: columns col + 128
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int dst = __shfl_sync(0xffffffffu, my_dst, j);
              const float w = __shfl_sync(0xffffffffu, my_w, j);
              if (dst >= 0) {
                atomicAdd(a.y + (size_t)dst * a.d + col, w * g[j]);
                if (it.ntile == 2) atomicAdd(a.y + (size_t)dst * a.d + col + kTileM, w * g2[j]);
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
      }
    }
  }

  // ---- teardown ----------------------------------------------------------------------------------------
  __syncwarp();
  if (*abort_flag) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM are released
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

// ---- host side -------------------------------------------------------------------------------------------
// bf16 matrix [rows, cols] row-major; boxes of [box_rows, 64 columns], 128-byte swizzle, zero fill.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeFn fn = encode_fn();
  if (!fn || !base) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kTileK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool UP, bool ROWS_OUT>
cudaError_t launch(const TcMaps& maps, const FfnParams& p, uint32_t* err, cudaStream_t st) {
  static int cache[64] = {0};   // one per instantiation of this launcher, i.e. per kernel
  int sms = 0;
  cudaError_t e0 = sm_count_and_smem_optin(ffn_tc_kernel<UP, ROWS_OUT>, Cfg<UP>::kSmemBytes, cache, &sms);
  if (e0 != cudaSuccess) return e0;
  TcArgs a;
  a.L = p.L, a.S = p.S, a.E = p.E, a.K = p.K, a.n_sh = p.n_sh, a.d = p.d, a.I = p.I, a.l0 = p.l0;
  a.n_items = p.L * items_per_layer(p.E, p.n_sh, p.S, UP ? p.I / kTileM : (p.d / kTileM + 1) / 2);
  a.offsets = p.offsets, a.perm = p.perm, a.sel_w = p.sel_w, a.H = (__nv_bfloat16*)p.H, a.y = p.y, a.O = p.O;
  a.err = err;
  const int grid = a.n_items < sms ? a.n_items : sms;
  ffn_tc_kernel<UP, ROWS_OUT><<<grid, kThreads, Cfg<UP>::kSmemBytes, st>>>(maps, a);
  return cudaGetLastError();
}

}  // namespace

bool tc_applicable(const mcce_config& c) {
  return c.hidden_dtype == MCCE_BF16 && c.weight_dtype == MCCE_BF16 && c.d_model % kTileM == 0 &&
         c.d_ff % kTileM == 0;
}

int tc_plan(const mcce_config& c, const void* Wg, const void* Wu, const void* Wd, const void* shWg, const void* shWu,
            const void* shWd, void* Xg0, void* Xg1, void* H, TcPlan* plan) {
  const uint64_t L = c.n_layers, E = c.n_experts, S = c.n_streams, K = c.top_k, nsh = c.n_shared;
  const uint64_t d = c.d_model, I = c.d_ff;
  const uint64_t rows = L * S * K + L * nsh * S;
  bool ok = make_map(&plan->w_gate, Wg, L * E * I, d, kTileM) && make_map(&plan->w_up, Wu, L * E * I, d, kTileM) &&
            make_map(&plan->w_down, Wd, L * E * d, I, kTileM);
  if (nsh)
    ok = ok && make_map(&plan->sh_gate, shWg, L * nsh * I, d, kTileM) &&
         make_map(&plan->sh_up, shWu, L * nsh * I, d, kTileM) && make_map(&plan->sh_down, shWd, L * nsh * d, I, kTileM);
  ok = ok && make_map(&plan->x_routed[0], Xg0, L * S * K + 256, d, kXBox) &&
       make_map(&plan->x_routed[1], Xg1, L * S * K + 256, d, kXBox) && make_map(&plan->h_all, H, rows + 256, I, kXBox);
  plan->hidden_ptr[0] = plan->hidden_ptr[1] = nullptr;
  plan->hidden_rows[0] = plan->hidden_rows[1] = 0;
  plan->ready = ok;
  return ok ? MCCE_OK : MCCE_ECUDA;
}

cudaError_t tc_launch_up(TcPlan& plan, const FfnParams& p, uint32_t* err_flag, cudaStream_t st) {
  if (!plan.ready) return cudaErrorNotReady;
  const int sl = p.slot & 1;
  if (p.n_sh && (plan.hidden_ptr[sl] != p.hidden || plan.hidden_rows[sl] != (uint64_t)p.L * p.S)) {
    if (!make_map(&plan.x_hidden[sl], p.hidden, (uint64_t)p.L * p.S, p.d, kXBox)) return cudaErrorInvalidValue;
    plan.hidden_ptr[sl] = p.hidden;
    plan.hidden_rows[sl] = (uint64_t)p.L * p.S;
  }
  TcMaps m;
  m.w0 = plan.w_gate, m.w1 = plan.w_up, m.x = plan.x_routed[sl];
  m.sw0 = p.n_sh ? plan.sh_gate : plan.w_gate, m.sw1 = p.n_sh ? plan.sh_up : plan.w_up;
  m.xs = p.n_sh ? plan.x_hidden[sl] : plan.x_routed[sl];
  return launch<true, false>(m, p, err_flag, st);
}

cudaError_t tc_launch_down(TcPlan& plan, const FfnParams& p, bool rows_out, uint32_t* err_flag, cudaStream_t st) {
  if (!plan.ready) return cudaErrorNotReady;
  TcMaps m;
  m.w0 = plan.w_down, m.w1 = plan.w_down, m.x = plan.h_all, m.xs = plan.h_all;
  m.sw0 = p.n_sh ? plan.sh_down : plan.w_down, m.sw1 = m.sw0;
  return rows_out ? launch<false, true>(m, p, err_flag, st) : launch<false, false>(m, p, err_flag, st);
}

}  // namespace mcce
