// The router-resident tensor-core GEMM of Eq. 3 as device functions: one definition of its shared-memory layout
// and of its three roles (TMA producer, MMA issuer, epilogue), used by the stand-alone logits kernel
// (route_gemm_res.cu) and by the kernel that also routes (route_fused.cu).
//
//   Z[(t,l,s), e] = sum_j W_r[l][e][j] x[(t,l,s)][j]      for E <= 80 experts
//
// A CTA owns one layer and one part of the reduction (a range of 64-column K-slabs).  The three bf16 terms of
// W_r (hi + mid + lo, see route_gemm.cu) of that range are loaded once and stay resident in shared memory; the
// streams are the MMA's M (tiles of 128 hidden rows through a TMA ring), the terms are stacked along N
// (3 x Epad columns), so one tcgen05.mma per 16 hidden columns yields the hi, mid and lo products of 128 streams
// in separate TMEM columns.  The tensor core's fp32 accumulate truncates, so an accumulation never runs over
// more than kSetSlabs slabs: every set of kSetSlabs slabs of a tile has its own TMEM columns, and the epilogue
// (thread = stream row) adds hi + (mid + lo) of the sets in round-to-nearest fp32.  With kSetSlabs = 8 the
// measured error of a logit against an fp64 reference is at most 1.9e-6 (relative to max(1, |z|)) on all four
// model-shaped workloads; the tests bound it at 1e-5.  Two TMEM buffers alternate from tile to tile, so the MMA
// warp never waits for the epilogue.  Every mbarrier wait is bounded.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace mcce {
namespace rres {

using namespace tc;

constexpr int kTileM = 128, kTileK = 64, kXBox = 16, kMaxStages = 10, kMinStages = 3;
constexpr uint32_t kRowBytes = kTileK * 2;               // one 128-byte swizzle row
constexpr uint32_t kStageBytes = kTileM * kRowBytes;     // one hidden tile of one K-slab: 16 KB
constexpr uint32_t kSmemMax = 232448 - 1024;             // opt-in limit less the alignment slack
constexpr uint32_t kBarBytes = 512;
constexpr int kSetSlabs = 8;                             // K-slabs accumulated in one set of TMEM columns
constexpr int kBufCols = 256, kTmemCols = 512;
constexpr int kEMax = 80, kPartsMax = 8;

// What the roles need to know about the problem and this CTA's place in it.
struct Geometry {
  int L, S, E, Epad, n_steps;   // L: layers of this launch (hidden and logits hold those only)
  int l0, L_terms;              // model layer of local layer 0; layers in the term tensor
  int KS, slabs, n_tiles, n_stages;
  uint32_t res_bytes;   // shared memory reserved for the resident terms (multiple of 1024)
};
struct Maps {
  CUtensorMap w;   // 3-D: [3*L][E][d] bf16 terms (term-major), box 1 x Epad x 64
  CUtensorMap x;   // 2-D: [n_steps*L*S][d] hidden rows, box (S mod 128, rounded up to 16) x 64: the ragged last
                   // tile of a layer in one copy (several small copies per slab cost more than the bytes they save)
  CUtensorMap xt;  // the same rows, box 128 x 64 (full tiles)
};

__host__ __device__ inline int epad_of(int E) { return (E + 15) & ~15; }
__host__ __device__ inline uint32_t res_bytes_of(int slabs, int ks, int Epad) {
  const uint32_t res = (uint32_t)((slabs + ks - 1) / ks) * 3u * (uint32_t)Epad * kRowBytes;
  return (res + 1023u) & ~1023u;
}
// TMEM columns of a tile's accumulator sets must fit one buffer.
__host__ __device__ inline bool sets_fit(int slabs, int ks, int Epad) {
  const int n_k = (slabs + ks - 1) / ks;
  return ((n_k + kSetSlabs - 1) / kSetSlabs) * 3 * Epad <= kBufCols;
}
__host__ __device__ inline int stages_of(uint32_t res_bytes) {
  const int stages = (int)((kSmemMax - kBarBytes - res_bytes) / kStageBytes);
  return stages > kMaxStages ? kMaxStages : stages;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// Addresses inside the CTA's dynamic shared memory: resident terms, then the ring, then the barriers.
struct Smem {
  uint32_t base, ring;                                 // resident terms / first ring stage
  uint32_t bar_full, bar_empty, bar_tfull, bar_tempty, bar_res;
  uint32_t* tmem_slot;
  volatile uint32_t* abort_flag;
  volatile uint32_t* drained;   // [4] pairs that each epilogue warp has finished (used by the fused kernel)
};

__device__ __forceinline__ Smem carve(uint8_t* smem_raw, const Geometry& a) {
  Smem m;
  m.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* al = smem_raw + (m.base - smem_u32(smem_raw));
  m.ring = m.base + a.res_bytes;
  uint64_t* bars = (uint64_t*)(al + (size_t)a.res_bytes + (size_t)a.n_stages * kStageBytes);
  m.bar_full = smem_u32(bars), m.bar_empty = m.bar_full + 8 * kMaxStages;
  m.bar_tfull = m.bar_empty + 8 * kMaxStages, m.bar_tempty = m.bar_tfull + 16, m.bar_res = m.bar_tempty + 16;
  m.tmem_slot = (uint32_t*)(bars + 2 * kMaxStages + 5);
  m.abort_flag = m.tmem_slot + 1;
  m.drained = m.tmem_slot + 2;
  return m;
}

// This CTA's K part.  Every part owns slabs / KS slabs of its own, [k_begin, k_begin + n_own).  The slabs % KS
// that are left over (the last ones) are shared: the parts form as many groups as there are left-over slabs, every
// member of a group keeps the group's slab resident beside its own, and for the i-th (token, stream tile) pair of
// the layer the member i mod gsize adds it to its reduction.  Over the pairs every part then does the same work
// to within one slab per gsize pairs (with whole extra slabs per part, 32 slabs over 6 parts are 6,6,5,5,5,5 and
// the parts with six set the pace of their layer).
struct KPart {
  int k_begin, n_own;
  int shared;          // the group's shared slab, or -1
  int gsize, member;   // members of the group, this part's index among them
  __device__ __forceinline__ int n_res() const { return n_own + (shared >= 0 ? 1 : 0); }        // resident slabs
  __device__ __forceinline__ int n_k(int pair) const {                                           // slabs of a pair
    return n_own + (shared >= 0 && pair % gsize == member ? 1 : 0);
  }
  __device__ __forceinline__ int slab(int j) const { return j < n_own ? k_begin + j : shared; }  // j-th of a pair
};
__device__ __forceinline__ KPart k_part_of(const Geometry& a, int ks) {
  const int k_base = a.slabs / a.KS, k_rem = a.slabs % a.KS;
  KPart p;
  p.k_begin = ks * k_base, p.n_own = k_base, p.shared = -1, p.gsize = 1, p.member = 0;
  if (k_rem > 0) {
    const int g = ks * k_rem / a.KS;                                   // groups are runs of consecutive parts
    const int first = (g * a.KS + k_rem - 1) / k_rem, next = ((g + 1) * a.KS + k_rem - 1) / k_rem;
    p.shared = a.KS * k_base + g, p.gsize = next - first, p.member = ks - first;
  }
  return p;
}

// Called by thread 0 before the CTA-wide barrier that precedes the roles.
__device__ __forceinline__ void init_barriers(const Smem& m) {
  for (int s = 0; s < kMaxStages; ++s) {
    mbar_init(m.bar_full + 8 * s, 1);
    mbar_init(m.bar_empty + 8 * s, 1);
  }
  for (int b = 0; b < 2; ++b) {
    mbar_init(m.bar_tfull + 8 * b, 1);
    mbar_init(m.bar_tempty + 8 * b, 4);
  }
  mbar_init(m.bar_res, 1);
  *m.abort_flag = 0u;
  for (int q = 0; q < 4; ++q) m.drained[q] = 0u;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// TMA producer (one thread): the resident terms of this (layer, K part), then the hidden tiles of the (token,
// stream tile) pairs first, first + step, ... of the layer.  code0 .. code0 + 4 name the waits in the error word.
__device__ __forceinline__ void produce(const Maps& maps, const Geometry& a, const Smem& m, int l, KPart kp, int first,
                                        int step, uint32_t* err, uint32_t code0) {
  const uint32_t term_bytes = (uint32_t)a.Epad * kRowBytes, slab_bytes = 3u * term_bytes;
  const int n_pairs = a.n_steps * a.n_tiles;
  mbar_expect_tx(m.bar_res, (uint32_t)kp.n_res() * slab_bytes);
  for (int j = 0; j < kp.n_res(); ++j)
#pragma unroll
    for (int q = 0; q < 3; ++q)
      tma_load_3d(m.base + (uint32_t)j * slab_bytes + q * term_bytes, &maps.w, kp.slab(j) * kTileK, 0,
                  q * a.L_terms + a.l0 + l, m.bar_res);
  uint32_t stage = 0, phase = 0;
  for (int i = first; i < n_pairs; i += step) {
    const int t = i / a.n_tiles, tile = i % a.n_tiles;
    const int row0 = (t * a.L + l) * a.S + tile * kTileM;
    // rows of the copy: a whole tile, or the ragged last tile of the layer rounded up to the box of maps.x
    const int n_box = (min(kTileM, a.S - tile * kTileM) + kXBox - 1) / kXBox;
    const int n_k = kp.n_k(i);
    for (int j = 0; j < n_k; ++j) {
      if (!mbar_wait(m.bar_empty + 8 * stage, phase ^ 1u, m.abort_flag, err, code0)) return;
      const uint32_t sa = m.ring + stage * kStageBytes, full = m.bar_full + 8 * stage;
      mbar_expect_tx(full, (uint32_t)n_box * kXBox * kRowBytes);
      tma_load_2d(sa, n_box == kTileM / kXBox ? &maps.xt : &maps.x, kp.slab(j) * kTileK, row0, full);
      if (++stage == (uint32_t)a.n_stages) stage = 0, phase ^= 1u;
    }
  }
}

// MMA issuer (one thread): per pair, all slabs of this K part into the accumulator sets of one TMEM buffer.
__device__ __forceinline__ void issue_mmas(const Geometry& a, const Smem& m, uint32_t tmem_base, KPart kp, int first,
                                           int step, uint32_t* err, uint32_t code0) {
  const uint32_t slab_bytes = 3u * (uint32_t)a.Epad * kRowBytes, set_cols = 3u * (uint32_t)a.Epad;
  const int n_pairs = a.n_steps * a.n_tiles;
  const uint32_t idesc = instr_desc(set_cols);
  uint32_t stage = 0, phase = 0, it = 0;
  if (!mbar_wait(m.bar_res, 0u, m.abort_flag, err, code0 + 1u)) return;
  tc_fence_after();
  for (int i = first; i < n_pairs; i += step, ++it) {
    const uint32_t buf = it & 1u, acc_phase = (it >> 1) & 1u;
    if (!mbar_wait(m.bar_tempty + 8 * buf, acc_phase ^ 1u, m.abort_flag, err, code0 + 2u)) return;
    tc_fence_after();
    const int n_k = kp.n_k(i);
    for (int j = 0; j < n_k; ++j) {
      if (!mbar_wait(m.bar_full + 8 * stage, phase, m.abort_flag, err, code0 + 3u)) return;
      tc_fence_after();
      const uint32_t d_set = tmem_base + buf * kBufCols + (uint32_t)(j / kSetSlabs) * set_cols;
      const uint32_t sa = m.ring + stage * kStageBytes, sb = m.base + (uint32_t)j * slab_bytes;
#pragma unroll
      for (int k = 0; k < kTileK / 16; ++k)
        umma_bf16(d_set, smem_desc(sa + k * 32), smem_desc(sb + k * 32), idesc, (j % kSetSlabs == 0 && k == 0) ? 0u : 1u);
      umma_commit(m.bar_empty + 8 * stage);
      if (++stage == (uint32_t)a.n_stages) stage = 0, phase ^= 1u;
    }
    umma_commit(m.bar_tfull + 8 * buf);
  }
}

__device__ __forceinline__ void red_add4(float* q, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(q), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Epilogue of one pair for the calling warp (TMEM lane quadrant `quad`, thread = stream row): waits for the
// tile's accumulators, adds the sets and the three terms in round-to-nearest fp32 and stores this K part's
// partial logits of rows row0 + quad*32 + lane (zrow: the row in the part's [rows][E] array); then releases the
// TMEM buffer.  With ADD the partial logits are added to zrow instead (fp32 reductions performed in L2; the K
// parts of a layer then share one array that starts at zero, and the order of the additions is that of arrival).
// Returns false if the CTA is giving up.  it = how many pairs this CTA has finished before; n_k = slabs that
// went into this pair.
template <bool ADD>
__device__ __forceinline__ bool drain_pair(const Geometry& a, const Smem& m, uint32_t tmem_base, int n_k, uint32_t it,
                                           int quad, int lane, float* zrow, bool row_ok, uint32_t* err, uint32_t code) {
  const uint32_t buf = it & 1u, acc_phase = (it >> 1) & 1u;
  if (!mbar_wait(m.bar_tfull + 8 * buf, acc_phase, m.abort_flag, err, code)) return false;
  tc_fence_after();
  const uint32_t set_cols = 3u * (uint32_t)a.Epad;
  const uint32_t t0 = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kBufCols;
  const int n_sets = (n_k + kSetSlabs - 1) / kSetSlabs;
  const bool vec4 = (a.E & 3) == 0;
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
          if (c + j < a.E) {
            if (ADD)
              red_add4(zrow + c + j, acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
            else
              *(float4*)(zrow + c + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
          }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c + j < a.E) {
            if (ADD)
              atomicAdd(zrow + c + j, acc[j]);
            else
              zrow[c + j] = acc[j];
          }
      }
    }
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(m.bar_tempty + 8 * buf);
  return true;
}

// After the roles: lets copies and MMAs in flight land if the CTA gave up, then frees TMEM (warp `alloc_warp`).
__device__ __forceinline__ void teardown(const Smem& m, uint32_t tmem_base, int warp, int alloc_warp) {
  __syncwarp();
  if (*m.abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == alloc_warp) tmem_dealloc(tmem_base, kTmemCols);
}

// Host side: tensor maps over the hidden rows of a launch (rebuilt when the pointer or the row count changes).
inline cudaError_t hidden_maps(RouterGemmPlan& plan, const void* hidden, uint64_t rows, int d_model, int n_streams) {
  if (plan.hidden_ptr_res == hidden && plan.hidden_rows_res == rows) return cudaSuccess;
  EncodeFn fn = encode_fn();
  const cuuint64_t dims[2] = {(cuuint64_t)d_model, rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d_model * 2};
  const int ragged = n_streams % kTileM ? ((n_streams % kTileM + kXBox - 1) / kXBox) * kXBox : kXBox;
  const cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)ragged};
  const cuuint32_t box_tile[2] = {(cuuint32_t)kTileK, (cuuint32_t)kTileM};
  const cuuint32_t estr[2] = {1, 1};
  if (!fn || fn(&plan.x_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
      fn(&plan.xt_res, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box_tile, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  plan.hidden_ptr_res = hidden;
  plan.hidden_rows_res = rows;
  return cudaSuccess;
}

}  // namespace rres
}  // namespace mcce
