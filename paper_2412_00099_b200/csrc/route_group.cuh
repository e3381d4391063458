// Routing tail of a small group of lanes per (stream, layer): the device code shared by the stand-alone
// kernel (route_thread.cu) and the kernel that runs it beside the router GEMM (route_fused.cu).
//
// A stream belongs to G = N/8 adjacent lanes (N = experts rounded up to 8, 16, 32 or 64), each holding eight
// consecutive experts as order-preserving integer keys in registers: a selection is a comparison tree over the
// lane's own eight keys followed by log2(G) butterfly steps inside the group; several streams advance per warp
// instruction.  Recency keys, resident and ever-resident bits stay in registers across the tokens of a launch.
// The state arrays in global memory have the format of route.cu.  Decision arithmetic is the same single IEEE
// fp32 operations in the same order as in route.cu (Eq. 7, Eq. 8, Eq. 4, Sec. 3.3, Sec. 4.2 of the paper).
#pragma once
#include "common.cuh"
#include "warp_select.cuh"

namespace mcce {
namespace rgroup {


constexpr int kNE = 8;        // experts per lane
constexpr int kPartsMax = 8;  // partial logit arrays that the prefetch holds in registers

struct Cand {
  uint32_t k;   // selection key (0 = none)
  int e;        // expert
  uint32_t z;   // key of its unmodified logit
};

// Largest key among the experts of the group not in `taken` (bit i = this lane's i-th expert); equal keys ->
// lowest expert.  Every lane of the group gets the result.
template <int G>
__device__ __forceinline__ Cand group_argmax(const uint32_t (&key)[kNE], const uint32_t (&zk)[kNE], uint32_t taken, int e0) {
  Cand c[kNE];
#pragma unroll
  for (int i = 0; i < kNE; ++i) c[i].k = ((taken >> i) & 1u) ? 0u : key[i], c[i].e = e0 + i, c[i].z = zk[i];
#pragma unroll
  for (int w = kNE / 2; w >= 1; w /= 2)
#pragma unroll
    for (int j = 0; j < w; ++j) {
      // strict comparison: on equal keys the lower expert (left) stays
      const bool gt = c[2 * j + 1].k > c[2 * j].k;
      c[j].k = gt ? c[2 * j + 1].k : c[2 * j].k;
      c[j].e = gt ? c[2 * j + 1].e : c[2 * j].e;
      c[j].z = gt ? c[2 * j + 1].z : c[2 * j].z;
    }
  Cand best = c[0];
  if (G > 1) {
    // largest key of the group by a butterfly on the keys alone; among the lanes that hold it the lowest one
    // has the lowest expert (a lane's experts are consecutive), and hands over its expert and payload
    const int gbase = (threadIdx.x & 31) & ~(G - 1);
    uint32_t m = best.k;
#pragma unroll
    for (int o = 1; o < G; o <<= 1) m = max(m, __shfl_xor_sync(kFull, m, o));
    const unsigned holders = (__ballot_sync(kFull, best.k == m) >> gbase) & ((1u << G) - 1u);
    const int owner = gbase + __ffs(holders) - 1;
    best.e = __shfl_sync(kFull, best.e, owner);
    best.z = __shfl_sync(kFull, best.z, owner);
    best.k = m;
  }
  return best;
}

template <int G>
__device__ __forceinline__ uint32_t group_max(uint32_t v) {
#pragma unroll
  for (int o = 1; o < G; o <<= 1) v = max(v, __shfl_xor_sync(kFull, v, o));
  return v;
}
template <int G>
__device__ __forceinline__ uint32_t group_min(uint32_t v) {
#pragma unroll
  for (int o = 1; o < G; o <<= 1) v = min(v, __shfl_xor_sync(kFull, v, o));
  return v;
}
template <int G>
__device__ __forceinline__ uint32_t group_or(uint32_t v) {
#pragma unroll
  for (int o = 1; o < G; o <<= 1) v |= __shfl_xor_sync(kFull, v, o);
  return v;
}
template <int G>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = 1; o < G; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}


// Loads of logits: through the read-only path when another kernel wrote them, L2-coherent when CTAs of the
// running kernel did (ACCUM below).
template <bool COHERENT>
__device__ __forceinline__ float4 ldz4(const float4* q) { return COHERENT ? __ldcg(q) : __ldg(q); }
template <bool COHERENT>
__device__ __forceinline__ float ldz1(const float* q) { return COHERENT ? __ldcg(q) : __ldg(q); }

// What a token contributes before the cache is consulted: its logits, their maximum, the promotion bias
// lambda * Delta_avg (Eq. 7, Eq. 8) and this lane's bits of the router's own top-J.
struct Pre {
  float z[kNE];
  float zmax, bias;
  uint32_t topj;
};

// How the logits of a token reach the registers.
constexpr int kLoadDirect = 0;     // loaded when the token's turn comes (after sync.wait(t))
constexpr int kPrefetchAll = 1;    // every token is there already: the next token's logits are requested while
                                   // the current one is routed
constexpr int kPrefetchReady = 2;  // tokens appear while the kernel runs: the next token's logits are requested
                                   // half-way through the current one if they are there by then (sync.probe(t + 1)
                                   // before the selection, sync.probed_ok() after it), else after sync.wait(t + 1)

// For callers whose logits are all there before the launch.
struct AllPresent {
  __device__ __forceinline__ bool wait(int) const { return true; }
  __device__ __forceinline__ void probe(int) {}
  __device__ __forceinline__ bool probed_ok() const { return true; }
};

// Routes the p.n_steps tokens of stream s_raw of layer l.  All 32 lanes of a warp must call this together
// (groups past the last stream run on stream 0's data and store nothing).  `sub` is the lane's index in its
// group.  sync.wait(t) is called by every lane before the logits of token t are read and returns false to give
// up; sync.probe(t) starts asking, without waiting, whether they can be read, and sync.probed_ok() has the answer
// (the same one in all lanes of a warp).
//
// ACCUM: the logits are sums that CTAs of the running kernel accumulate in an array that is zero between launches
// (one array: p.n_partials == 1).  They are read L2-coherently, and the lanes that own a row put the zeros back.
//
// A token's work has a part that does not depend on the cache (logits, range statistic, bias, top-J: stage A)
// and a part that does (promotion, top-K, misses, LRU: stage B); only B is a chain from token to token.
// With a prefetching MODE up to NP partial logit arrays of the next token are held in registers.
template <int G, int KMAX, int MODE, int NP, bool COHERENT, bool ACCUM, typename Sync>
__device__ __forceinline__ void route_group_streams(const RouteParams& p, const int l, const int s_raw, const int sub,
                                                    Sync sync) {
  constexpr bool PF = MODE != kLoadDirect;
  static_assert(!ACCUM || (COHERENT && PF && NP == 1), "accumulated logits are one array, cleared where it is prefetched");
  const bool active = s_raw < p.S;
  const int s = active ? s_raw : 0;
  const size_t pair = (size_t)l * p.S + s;
  const int E = p.E, K = p.K;
  const int e0 = sub * kNE;
  const bool vec4 = (E & 3) == 0;

  // ---- state of this (layer, stream) into registers -----------------------------------------------------
  uint32_t st[kNE];
  uint32_t resb = 0u, everb = 0u;   // bit i: this lane's i-th expert is resident / was ever resident
  int resident = 0;
  uint32_t miss_c = 0u, cold_c = 0u;
  float sum_range = 0.f;
  {
    const int EW = (E + 31) >> 5;
    const uint32_t word = e0 < E ? p.ever[pair * EW + (e0 >> 5)] : 0u;
    everb = (word >> (e0 & 31)) & 0xffu;
#pragma unroll
    for (int i = 0; i < kNE; ++i) {
      st[i] = e0 + i < E ? p.stamp[pair * E + e0 + i] : 0u;
      resb |= (st[i] != 0u ? 1u : 0u) << i;
    }
    resident = (int)group_sum<G>((float)__popc(resb));   // exact: at most 64
    miss_c = p.miss[pair], cold_c = p.cold[pair];
  }
  sum_range = p.sum_range[pair];

  // Where this lane's eight logits of token t start in a logits array.
  auto z_at = [&](int t) -> const float* { return p.logits_in + (((size_t)t * p.L + l) * p.S + s) * E + e0; };
  auto load8 = [&](const float* src, float (&v)[kNE]) {
    if (vec4) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e0 + 4 * h < E) u = ldz4<COHERENT>((const float4*)(src + 4 * h));
        v[4 * h] = u.x, v[4 * h + 1] = u.y, v[4 * h + 2] = u.z, v[4 * h + 3] = u.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < kNE; ++i) v[i] = e0 + i < E ? ldz1<COHERENT>(src + i) : 0.f;
    }
  };

  // The partial logits of the next token are requested before the current token is routed, so that their
  // latency (L2, mostly) is off the critical path: up to NP parts of eight logits per lane in flight.
  float raw[PF ? NP : 1][kNE];
  auto request = [&](int t) {
    const float* src = z_at(t);
#pragma unroll
    for (int q = 0; q < (PF ? NP : 1); ++q)
      if (q < p.n_partials) load8(src + (size_t)q * p.partial_stride, raw[q]);
    if (ACCUM && active) {
      // same thread, same addresses: the loads above are ordered before these stores
#pragma unroll
      for (int h = 0; h < 2; ++h)
        if (e0 + 4 * h < E) __stcg((float4*)const_cast<float*>(src + 4 * h), make_float4(0.f, 0.f, 0.f, 0.f));
    }
  };

  // ---- stage A: logits of token t (the K parts of the router GEMM summed in a fixed order), Eq. 8, top-J -------
  auto stage_a = [&](const int t, Pre& o) {
    const size_t row = ((size_t)t * p.L + l) * p.S + s;
    float (&z)[kNE] = o.z;
    if (PF) {
#pragma unroll
      for (int i = 0; i < kNE; ++i) {
        float v = raw[0][i];
#pragma unroll
        for (int q = 1; q < (PF ? NP : 1); ++q)
          if (q < p.n_partials) v = __fadd_rn(v, raw[q][i]);
        z[i] = v;
      }
    } else {
      const float* src = z_at(t);
      load8(src, z);
      for (int q = 1; q < p.n_partials; ++q) {
        float u[kNE];
        load8(src + (size_t)q * p.partial_stride, u);
#pragma unroll
        for (int i = 0; i < kNE; ++i) z[i] = __fadd_rn(z[i], u[i]);
      }
    }
    if (p.logits_out != nullptr && active) {
      float* dst = p.logits_out + row * E + e0;
      if (vec4) {
#pragma unroll
        for (int i = 0; i < kNE; i += 4)
          if (e0 + i < E) *(float4*)(dst + i) = make_float4(z[i], z[i + 1], z[i + 2], z[i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < kNE; ++i)
          if (e0 + i < E) dst[i] = z[i];
      }
    }
    // Eq. 8: range of this token's logits, running mean that includes it
    uint32_t kz[kNE];
    uint32_t kmax_l = 0u, kmin_l = 0xffffffffu;
#pragma unroll
    for (int i = 0; i < kNE; ++i) {
      const bool valid = e0 + i < E;
      kz[i] = valid ? okey(z[i]) : 0u;
      kmax_l = max(kmax_l, kz[i]);
      kmin_l = min(kmin_l, valid ? kz[i] : 0xffffffffu);
    }
    o.zmax = okey_inv(group_max<G>(kmax_l));
    const float zmin = okey_inv(group_min<G>(kmin_l));
    float delta;
    if (p.delta_mode == MCCE_DELTA_RUNNING) {
      sum_range = __fadd_rn(sum_range, __fsub_rn(o.zmax, zmin));
      delta = __fdiv_rn(sum_range, (float)(p.cnt0 + (uint32_t)t + 1u));
    } else {
      delta = __ldg(p.fixed_delta + l);
    }
    o.bias = __fmul_rn(p.lambda, delta);
    // this lane's bits of the router's own top-J
    uint32_t taken = 0u;
    for (int r = 0; r < p.J; ++r) {
      const Cand c = group_argmax<G>(kz, kz, taken, e0);
      if ((c.e >> 3) == sub) taken |= 1u << (c.e & 7);
    }
    o.topj = taken;
  };

  // ---- stage B: Eq. 7, top-K, weights, Eq. 4, LRU ---------------------------------------------------------------------
  auto stage_b = [&](const int t, const Pre& in, auto&& after_selection) {
    const size_t row = ((size_t)t * p.L + l) * p.S + s;
    const float (&z)[kNE] = in.z;
    const float zmax = in.zmax, bias = in.bias;
    // m~_t = cache OR top-J of the router; z' = z + bias on m~_t
    const uint32_t mt = resb | in.topj;
    uint32_t kz[kNE], kp[kNE];
#pragma unroll
    for (int i = 0; i < kNE; ++i) {
      const bool valid = e0 + i < E;
      const float zp = ((mt >> i) & 1u) ? __fadd_rn(z[i], bias) : z[i];
      kz[i] = valid ? okey(z[i]) : 0u;
      kp[i] = valid ? okey(zp) : 0u;
    }

    // top-K of z' in rank order.  Every lane of the group learns all K (expert, unmodified logit) pairs; the work
    // per selected expert that follows (LRU position, weight, output) is dealt out to the lanes: lane `sub`
    // takes the selections r = sub, sub + G, ...
    constexpr int kMine = (KMAX + G - 1) / G;
    int sel_e[KMAX], my_e[kMine];
    uint32_t sel_k[KMAX], my_k[kMine];
    uint32_t miss_bits = 0u, cold_bits = 0u;
#pragma unroll
    for (int j = 0; j < kMine; ++j) my_e[j] = 0, my_k[j] = 0u;
    {
      uint32_t taken = 0u;
#pragma unroll
      for (int r = 0; r < KMAX; ++r) {
        sel_e[r] = 0, sel_k[r] = 0u;
        if (r < K) {
          const Cand c = group_argmax<G>(kp, kz, taken, e0);
          sel_e[r] = c.e, sel_k[r] = c.z;
          if (sub == r % G) my_e[r / G] = c.e, my_k[r / G] = c.z;
          if ((c.e >> 3) == sub) {
            const uint32_t bit = 1u << (c.e & 7);
            taken |= bit;
            // Eq. 4 against the cache before this token (the owner lane knows)
            if (!(resb & bit)) miss_bits |= 1u << r;
            if (!(everb & bit)) cold_bits |= 1u << r;
          }
        }
      }
    }
    after_selection();
    {
      const uint32_t both = group_or<G>(miss_bits | (cold_bits << 16));
      miss_bits = both & 0xffffu, cold_bits = both >> 16;
    }
    miss_c += __popc(miss_bits);
    cold_c += __popc(cold_bits);
    if (p.miss_trace != nullptr && t < p.trace_avail && sub == 0 && active)
      p.miss_trace[((size_t)t * p.L + l) * p.S + s] = miss_bits;

    // my selections: weight (softmax of the unmodified logits) and position in the token's LRU order (the higher
    // router weight is the older one)
    float pe[kMine], loc = 0.f;
    int my_pos[kMine];
#pragma unroll
    for (int j = 0; j < kMine; ++j) {
      const bool mine = sub + j * G < K;
      pe[j] = mine ? expf(okey_inv(my_k[j]) - zmax) : 0.f;
      loc += pe[j];
      int pos = 0;
#pragma unroll
      for (int q = 0; q < KMAX; ++q)
        if (q < K && (sel_k[q] > my_k[j] || (sel_k[q] == my_k[j] && sel_e[q] < my_e[j]))) ++pos;
      my_pos[j] = pos;
    }
    if (!p.renorm) {
      loc = 0.f;
#pragma unroll
      for (int i = 0; i < kNE; ++i)
        if (e0 + i < E) loc += expf(z[i] - zmax);
    }
    const float denom = group_sum<G>(loc);

    // LRU touch by the lane that holds the expert
    const uint32_t base = (uint32_t)E + (p.tok0 + (uint32_t)t) * (uint32_t)K + 1u;
#pragma unroll
    for (int r = 0; r < KMAX; ++r)
      if (r < K) {
        const int pos = G > 1 ? __shfl_sync(kFull, my_pos[r / G], ((threadIdx.x & 31) & ~(G - 1)) + r % G) : my_pos[r / G];
        if ((sel_e[r] >> 3) == sub) {
          const int slot = sel_e[r] & 7;
#pragma unroll
          for (int i = 0; i < kNE; ++i)
            if (i == slot) st[i] = base + (uint32_t)pos;
          resb |= 1u << slot;
          everb |= 1u << slot;
        }
      }
    resident += __popc(miss_bits);
    // evict the resident expert with the smallest recency key until the cache fits (keys of resident experts
    // are distinct); groups that already fit idle through the loop of their warp's other groups
    while (__any_sync(kFull, resident > p.C)) {
      uint32_t lmin = 0xffffffffu;
#pragma unroll
      for (int i = 0; i < kNE; ++i)
        if ((resb >> i) & 1u) lmin = min(lmin, st[i]);
      const uint32_t m = group_min<G>(lmin);
      if (resident > p.C) {
#pragma unroll
        for (int i = 0; i < kNE; ++i)
          if (((resb >> i) & 1u) && st[i] == m) st[i] = 0u, resb &= ~(1u << i);
        --resident;
      }
    }

    // results
    if (active) {
#pragma unroll
      for (int j = 0; j < kMine; ++j) {
        const int r = sub + j * G;
        if (r < K) {
          p.sel_idx[row * K + r] = my_e[j];
          p.sel_w[row * K + r] = pe[j] / denom;
        }
      }
    }
  };

  bool alive = true;
  if (PF) {
    alive = sync.wait(0);
    if (alive) request(0);
  }
  for (int t = 0; t < p.n_steps && alive; ++t) {
    if (!PF && !sync.wait(t)) break;
    Pre pre;
    stage_a(t, pre);            // with PF: consumes the registers that request(t) filled
    bool requested = false;
    const bool more = PF && t + 1 < p.n_steps;
    if (more && MODE == kPrefetchAll) request(t + 1), requested = true;
    if (more && MODE == kPrefetchReady) sync.probe(t + 1);
    stage_b(t, pre, [&]() {
      if (more && MODE == kPrefetchReady) {
        requested = sync.probed_ok();
        if (requested) request(t + 1);
      }
    });
    if (PF && t + 1 < p.n_steps && !requested) {
      alive = sync.wait(t + 1);
      if (alive) request(t + 1);
    }
  }

  // ---- state back to memory ----------------------------------------------------------------------------------------------
  {
    // ever-resident words: four lanes (32 experts) make one word
    uint32_t word = everb << (e0 & 31);
    if (G >= 2) word |= __shfl_xor_sync(kFull, word, 1);
    if (G >= 4) word |= __shfl_xor_sync(kFull, word, 2);
    if (active) {
#pragma unroll
      for (int i = 0; i < kNE; ++i)
        if (e0 + i < E) p.stamp[pair * E + e0 + i] = st[i];
      const int EW = (E + 31) >> 5;
      if ((sub & 3) == 0 && e0 < E) p.ever[pair * EW + (e0 >> 5)] = word;
      if (sub == 0) {
        p.miss[pair] = miss_c;
        p.cold[pair] = cold_c;
      }
    }
  }
  if (active && sub == 0) p.sum_range[pair] = sum_range;
}

}  // namespace rgroup
}  // namespace mcce
