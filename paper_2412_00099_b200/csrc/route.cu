// Fused route kernel: router logits (Eq. 3), logit-range statistic (Eq. 8), Cache-Prior promotion of
// cached logits (Eq. 7), top-K with weights from the unmodified logits (Sec. 3.3), miss counting
// (Eq. 4) and the LRU update (Sec. 4.2) -- one warp per (stream, layer), state in registers across
// the tokens of one launch.
//
// A CTA owns one layer and kWarps consecutive streams.  In hidden-state mode the CTA first forms the
// logits of its streams together: the hidden rows are staged in shared memory once and each router
// row read from L2 is used for all kWarps streams.  The routing tail then runs one warp per stream:
// lane j holds experts j, j+32, ... (NE per lane), every selection is a pair of warp reductions.
#include "common.cuh"
#include "warp_select.cuh"

namespace mcce {

constexpr int kWarps = 8;
constexpr int kDChunkMax = 4096;

// HIDDEN: the kernel forms the logits itself (fp32-pipe front end); otherwise it only reads them, and is
// compiled without that code so that it needs fewer registers and more warps fit on an SM.
template <int NE, bool HIDDEN>
__global__ void __launch_bounds__(kWarps * 32, HIDDEN ? 1 : 4) route_kernel(const RouteParams p, const int dchunk) {
  extern __shared__ __align__(16) float smem[];
  float* xs = smem;                          // [kWarps][dchunk]   hidden rows (fp32)
  float* zs = smem + (size_t)kWarps * dchunk;  // [kWarps][NE*32]   logits of this CTA's streams

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks_per_layer = (p.S + kWarps - 1) / kWarps;
  const int l = blockIdx.x / blocks_per_layer;
  const int s = (blockIdx.x % blocks_per_layer) * kWarps + warp;
  const bool active = s < p.S;
  const size_t pair = (size_t)l * p.S + (active ? s : 0);
  const int E = p.E, K = p.K;
  const int EW = (E + 31) >> 5;

  // ---- state of this (layer, stream) into registers -------------------------------------------
  uint32_t st[NE];
  uint32_t ld[NE];   // token that loaded each resident expert (only when lifetimes are tracked)
  unsigned long long life_n = 0ull, life_sum = 0ull, life_sq = 0ull;
  const bool track = p.load_tok != nullptr;
  uint32_t everb = 0u;
  float sum_range = 0.f;
  uint32_t miss_c = 0u, cold_c = 0u;
  if (active) {
#pragma unroll
    for (int i = 0; i < NE; ++i) {
      const int e = lane + 32 * i;
      st[i] = e < E ? p.stamp[pair * E + e] : 0u;
      ld[i] = (track && e < E) ? p.load_tok[pair * E + e] : 0u;
      if (i < EW) everb |= ((p.ever[pair * EW + i] >> lane) & 1u) << i;
    }
    sum_range = p.sum_range[pair];
    miss_c = p.miss[pair];
    cold_c = p.cold[pair];
  } else {
#pragma unroll
    for (int i = 0; i < NE; ++i) st[i] = ld[i] = 0u;
  }

  for (int t = 0; t < p.n_steps; ++t) {
    const size_t row = ((size_t)t * p.L + l) * p.S + (active ? s : 0);
    float zr[NE];

    if (HIDDEN) {
      // ---- Eq. 3: logits of kWarps streams, router rows shared through the CTA ------------------
      for (int i = lane; i < NE * 32; i += 32) zs[warp * NE * 32 + i] = 0.f;
      const float* Wl = p.Wr + (size_t)l * E * p.d;
      for (int c0 = 0; c0 < p.d; c0 += dchunk) {
        const int dc = min(dchunk, p.d - c0);
        __syncthreads();  // previous chunk fully consumed (and zs zeroed)
        if (active) {
          if (p.hidden_bf16) {
            const __nv_bfloat16* x = (const __nv_bfloat16*)p.hidden + row * p.d + c0;
            for (int k = 2 * lane; k < dc; k += 64) {
              const float2 v = __bfloat1622float2(*(const __nv_bfloat162*)(x + k));
              xs[warp * dchunk + k] = v.x;
              xs[warp * dchunk + k + 1] = v.y;
            }
          } else {
            const float* x = (const float*)p.hidden + row * p.d + c0;
            for (int k = lane; k < dc; k += 32) xs[warp * dchunk + k] = x[k];
          }
        } else {
          for (int k = lane; k < dc; k += 32) xs[warp * dchunk + k] = 0.f;
        }
        __syncthreads();
        for (int e0 = 2 * warp; e0 < E; e0 += 2 * kWarps) {
          const int e1 = min(e0 + 1, E - 1);
          const float* wa = Wl + (size_t)e0 * p.d + c0;
          const float* wb = Wl + (size_t)e1 * p.d + c0;
          float acc_a[kWarps], acc_b[kWarps];
#pragma unroll
          for (int q = 0; q < kWarps; ++q) acc_a[q] = acc_b[q] = 0.f;
          for (int k = 4 * lane; k < dc; k += 128) {
            const float4 a = __ldg((const float4*)(wa + k));
            const float4 b = __ldg((const float4*)(wb + k));
#pragma unroll
            for (int q = 0; q < kWarps; ++q) {
              const float4 x = *(const float4*)(xs + q * dchunk + k);
              acc_a[q] = fmaf(a.x, x.x, fmaf(a.y, x.y, fmaf(a.z, x.z, fmaf(a.w, x.w, acc_a[q]))));
              acc_b[q] = fmaf(b.x, x.x, fmaf(b.y, x.y, fmaf(b.z, x.z, fmaf(b.w, x.w, acc_b[q]))));
            }
          }
#pragma unroll
          for (int q = 0; q < kWarps; ++q) {
            const float ra = warp_sum(acc_a[q]);
            const float rb = warp_sum(acc_b[q]);
            if (lane == q) {
              zs[q * NE * 32 + e0] += ra;
              if (e1 != e0) zs[q * NE * 32 + e1] += rb;
            }
          }
        }
      }
      __syncthreads();
#pragma unroll
      for (int i = 0; i < NE; ++i) zr[i] = zs[warp * NE * 32 + lane + 32 * i];
      __syncthreads();  // zs is rewritten by the next token
    } else {
#pragma unroll
      for (int i = 0; i < NE; ++i) {
        const int e = lane + 32 * i;
        float z = 0.f;
        if (active && e < E) {
          z = __ldg(p.logits_in + row * E + e);
          for (int q = 1; q < p.n_partials; ++q) z = __fadd_rn(z, __ldg(p.logits_in + q * p.partial_stride + row * E + e));
        }
        zr[i] = z;
      }
    }
    if (!active) continue;

    if (HIDDEN && p.err_nonfinite != nullptr) {   // checked mode: these logits exist nowhere else
      bool bad = false;
#pragma unroll
      for (int i = 0; i < NE; ++i) bad |= lane + 32 * i < E && !isfinite(zr[i]);
      if (bad) atomicOr(p.err_nonfinite, 1u);
    }
    if (p.logits_out != nullptr) {
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (lane + 32 * i < E) p.logits_out[row * E + lane + 32 * i] = zr[i];
    }

    // ---- Eq. 8: range of this token's logits, running mean that includes it ----------------------
    uint32_t key[NE];
    uint32_t kmax_l = 0u, kmin_l = 0xffffffffu, resb = 0u;
#pragma unroll
    for (int i = 0; i < NE; ++i) {
      const bool valid = lane + 32 * i < E;
      key[i] = valid ? okey(zr[i]) : 0u;
      if (valid) {
        kmax_l = max(kmax_l, key[i]);
        kmin_l = min(kmin_l, key[i]);
      }
      resb |= (st[i] != 0u ? 1u : 0u) << i;
    }
    const float zmax = okey_inv(__reduce_max_sync(kFull, kmax_l));
    const float zmin = okey_inv(__reduce_min_sync(kFull, kmin_l));
    float delta;
    if (p.delta_mode == MCCE_DELTA_RUNNING) {
      sum_range = __fadd_rn(sum_range, __fsub_rn(zmax, zmin));
      delta = __fdiv_rn(sum_range, (float)(p.cnt0 + (uint32_t)t + 1u));
    } else {
      delta = __ldg(p.fixed_delta + l);
    }
    const float bias = __fmul_rn(p.lambda, delta);

    // ---- m~_t = cache OR top-J of the router; Eq. 7 ------------------------------------------------
    uint32_t mt = resb, taken = 0u;
    for (int r = 0; r < p.J; ++r) {
      const int e = warp_argmax<NE>(key, taken, lane);
      if ((e & 31) == lane) {
        taken |= 1u << (e >> 5);
        mt |= 1u << (e >> 5);
      }
    }
    uint32_t kp[NE];   // selection key of every expert: the K largest are selected, in this order
    if (p.rerank_mode == MCCE_RERANK_CACHE_PRIOR) {
#pragma unroll
      for (int i = 0; i < NE; ++i) {
        const bool valid = lane + 32 * i < E;
        const float zp = ((mt >> i) & 1u) ? __fadd_rn(zr[i], bias) : zr[i];
        kp[i] = valid ? okey(zp) : 0u;
      }
    } else {
      // ---- Algorithms 1 and 2: promote(r[:J]; promote(r[:M] ∩ C; r)) on the router's own ranking r ------
      // rank of every expert in r (value descending, index ascending), by comparison with all others
      uint32_t rk[NE];
#pragma unroll
      for (int i = 0; i < NE; ++i) rk[i] = 0u;
      for (int i2 = 0; i2 < NE; ++i2) {
        for (int src = 0; src < 32; ++src) {
          const int eo = src + 32 * i2;
          if (eo >= E) break;
          const uint32_t ko = __shfl_sync(kFull, key[i2], src);
#pragma unroll
          for (int i = 0; i < NE; ++i) rk[i] += (ko > key[i] || (ko == key[i] && eo < lane + 32 * i)) ? 1u : 0u;
        }
      }
      int M = p.max_rank;
      if (p.rerank_mode == MCCE_RERANK_CUMSUM) {
        // Sec. 3.2 / Algorithm 2: M is the first number of ranks whose router probabilities, added rank by rank
        // in fp32, reach the threshold (all E if they never do)
        float pr[NE], loc = 0.f;
#pragma unroll
        for (int i = 0; i < NE; ++i) {
          pr[i] = lane + 32 * i < E ? expf(zr[i] - zmax) : 0.f;
          loc += pr[i];
        }
        const float inv_all = warp_sum(loc);
        float mass = 0.f;
        for (M = 0; M < E && !(mass >= p.cum_threshold); ++M) {
          // the probability of the expert of rank M sits in exactly one lane
          float wv = 0.f;
          bool own = false;
#pragma unroll
          for (int i = 0; i < NE; ++i)
            if (lane + 32 * i < E && rk[i] == (uint32_t)M) wv = pr[i] / inv_all, own = true;
          mass = __fadd_rn(mass, __shfl_sync(kFull, wv, __ffs(__ballot_sync(kFull, own)) - 1));
        }
      }
#pragma unroll
      for (int i = 0; i < NE; ++i) {
        const bool valid = lane + 32 * i < E;
        const uint32_t cls = rk[i] < (uint32_t)p.J ? 0u : ((rk[i] < (uint32_t)M && ((resb >> i) & 1u)) ? 1u : 2u);
        kp[i] = valid ? 0x7fffffffu - ((cls << 16) | rk[i]) : 0u;
      }
    }

    // ---- top-K of z' (rank order); lane r keeps the r-th selected expert and its unmodified logit ---
    taken = 0u;
    int my_sel = 0;
    float my_z = 0.f;
    for (int r = 0; r < K; ++r) {
      const int e = warp_argmax<NE>(kp, taken, lane);
      const int owner = e & 31, slot = e >> 5;
      float zv = 0.f;
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (i == slot) zv = zr[i];
      zv = __shfl_sync(kFull, zv, owner);
      if (lane == owner) taken |= 1u << slot;
      if (lane == r) {
        my_sel = e;
        my_z = zv;
      }
    }

    // ---- weights: softmax of the unmodified logits ------------------------------------------------
    const float pe = lane < K ? expf(my_z - zmax) : 0.f;
    float denom;
    if (p.renorm) {
      denom = warp_sum(pe);
    } else {
      float loc = 0.f;
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (lane + 32 * i < E) loc += expf(zr[i] - zmax);
      denom = warp_sum(loc);
    }
    const float w = pe / denom;

    // ---- Eq. 4 against the cache before this token -------------------------------------------------
    {
      const uint32_t rb = __shfl_sync(kFull, resb, my_sel & 31);
      const uint32_t eb = __shfl_sync(kFull, everb, my_sel & 31);
      const bool sel_lane = lane < K;
      const uint32_t miss_bits = __ballot_sync(kFull, sel_lane && !((rb >> (my_sel >> 5)) & 1u));
      miss_c += __popc(miss_bits);   // lane k holds the k-th selected expert: bit k = slot k missed
      if (p.miss_trace != nullptr && t < p.trace_avail && lane == 0)
        p.miss_trace[((size_t)t * p.L + l) * p.S + s] = miss_bits;
      cold_c += __popc(__ballot_sync(kFull, sel_lane && !((eb >> (my_sel >> 5)) & 1u)));
    }

    // ---- LRU touch: inside the token the higher router weight is the older one ---------------------
    int pos = 0;
    for (int r = 0; r < K; ++r) {
      const float zo = __shfl_sync(kFull, my_z, r);
      const int eo = __shfl_sync(kFull, my_sel, r);
      if (zo > my_z || (zo == my_z && eo < my_sel)) ++pos;
    }
    const uint32_t base = (uint32_t)E + (p.tok0 + (uint32_t)t) * (uint32_t)K + 1u;
    for (int r = 0; r < K; ++r) {
      const int eo = __shfl_sync(kFull, my_sel, r);
      const int po = __shfl_sync(kFull, pos, r);
      if ((eo & 31) == lane) {
        const int slot = eo >> 5;
#pragma unroll
        for (int i = 0; i < NE; ++i)
          if (i == slot) {
            if (st[i] == 0u) ld[i] = p.tok0 + (uint32_t)t;   // a miss: loaded by this token
            st[i] = base + (uint32_t)po;
          }
        everb |= 1u << slot;
      }
    }
    int resident = 0;
#pragma unroll
    for (int i = 0; i < NE; ++i) resident += st[i] != 0u;
    resident = __reduce_add_sync(kFull, resident);
    while (resident > p.C) {
      uint32_t lmin = 0xffffffffu;
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (st[i] != 0u) lmin = min(lmin, st[i]);
      const uint32_t m = __reduce_min_sync(kFull, lmin);
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (st[i] == m) {
          st[i] = 0u;
          if (track) {   // cache lifetime of the evicted expert, in tokens (Table 2 of the paper)
            const unsigned long long life = (unsigned long long)(p.tok0 + (uint32_t)t - ld[i]);
            life_n += 1ull, life_sum += life, life_sq += life * life;
          }
        }
      --resident;
    }

    if (lane < K) {
      p.sel_idx[row * K + lane] = my_sel;
      p.sel_w[row * K + lane] = w;
    }
  }

  // ---- state back to memory -------------------------------------------------------------------------
  if (active) {
#pragma unroll
    for (int i = 0; i < NE; ++i) {
      const int e = lane + 32 * i;
      if (e < E) p.stamp[pair * E + e] = st[i];
      if (track && e < E) p.load_tok[pair * E + e] = ld[i];
      if (i < EW) {
        const uint32_t word = __ballot_sync(kFull, (everb >> i) & 1u);
        if (lane == 0) p.ever[pair * EW + i] = word;
      }
    }
    if (track) {
      for (int o = 16; o > 0; o >>= 1) {
        life_n += __shfl_xor_sync(kFull, life_n, o);
        life_sum += __shfl_xor_sync(kFull, life_sum, o);
        life_sq += __shfl_xor_sync(kFull, life_sq, o);
      }
      if (lane == 0) {
        p.life[pair * 3 + 0] += life_n;
        p.life[pair * 3 + 1] += life_sum;
        p.life[pair * 3 + 2] += life_sq;
      }
    }
    if (lane == 0) {
      p.sum_range[pair] = sum_range;
      p.miss[pair] = miss_c;
      p.cold[pair] = cold_c;
    }
  }
}

template <int NE>
static cudaError_t launch_ne(const RouteParams& p, cudaStream_t st) {
  if (!p.hidden) {
    const int grid = p.L * ((p.S + kWarps - 1) / kWarps);
    route_kernel<NE, false><<<grid, kWarps * 32, 0, st>>>(p, 0);
    return cudaGetLastError();
  }
  const int dchunk = p.hidden ? min((p.d + 3) & ~3, kDChunkMax) : 0;
  const size_t smem = p.hidden ? ((size_t)kWarps * dchunk + (size_t)kWarps * NE * 32) * sizeof(float) : 0;
  cudaError_t e = cudaFuncSetAttribute(route_kernel<NE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = p.L * ((p.S + kWarps - 1) / kWarps);
  route_kernel<NE, true><<<grid, kWarps * 32, smem, st>>>(p, dchunk);
  return cudaGetLastError();
}

cudaError_t launch_route(const RouteParams& p, cudaStream_t st) {
  if (route_thread_applicable(p)) return launch_route_thread(p, st);
  const int ne = (p.E + 31) / 32;
  if (ne <= 1) return launch_ne<1>(p, st);
  if (ne <= 2) return launch_ne<2>(p, st);
  if (ne <= 4) return launch_ne<4>(p, st);
  return launch_ne<8>(p, st);
}

// Per-layer sums of the miss counters: out[l] = {misses, cold_misses}.
__global__ void stats_kernel(const uint32_t* miss, const uint32_t* cold, unsigned long long* out, int S) {
  const int l = blockIdx.x;
  unsigned long long m = 0, c = 0;
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    m += miss[(size_t)l * S + s];
    c += cold[(size_t)l * S + s];
  }
  __shared__ unsigned long long sm[64];
  for (int o = 16; o > 0; o >>= 1) {
    m += __shfl_xor_sync(kFull, m, o);
    c += __shfl_xor_sync(kFull, c, o);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) {
    sm[warp] = m;
    sm[32 + warp] = c;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long tm = 0, tc = 0;
    for (int i = 0; i < nw; ++i) {
      tm += sm[i];
      tc += sm[32 + i];
    }
    out[2 * l] = tm;
    out[2 * l + 1] = tc;
  }
}

// Logit range from a calibration set (appendix "Logit Range Estimation"): per layer, the mean over the streams
// of the running estimate of Eq. 8, out[l] = (sum_s sum_range[l][s] / S) / count, in double precision (the
// sum of a few hundred fp32 values is exact there, so the order of the additions does not matter), rounded
// once to fp32.  One CTA per layer.
__global__ void calibrate_kernel(const float* sum_range, int S, double count, float* out) {
  __shared__ double part[256];
  const int l = blockIdx.x;
  double acc = 0.0;
  for (int s = threadIdx.x; s < S; s += blockDim.x) acc += (double)sum_range[(size_t)l * S + s];
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int w = blockDim.x / 2; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[l] = (float)(part[0] / (double)S / count);
}

cudaError_t launch_calibrate(const float* sum_range, int L, int S, double count, float* out, cudaStream_t st) {
  calibrate_kernel<<<L, 256, 0, st>>>(sum_range, S, count, out);
  return cudaGetLastError();
}

// Checked mode, after a routing launch: one warp per (layer, stream) verifies that at most C experts are
// resident and that the recency keys of the resident experts are distinct (the LRU order is then total).
__global__ void check_state_kernel(const uint32_t* stamp, size_t n_pairs, int E, int C, uint32_t* err_index) {
  const size_t pair = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pair >= n_pairs) return;
  const int lane = threadIdx.x & 31;
  const uint32_t* st = stamp + pair * E;
  int resident = 0;
  bool dup = false;
  for (int e0 = 0; e0 < E; e0 += 32) {
    const uint32_t mine = e0 + lane < E ? st[e0 + lane] : 0u;
    resident += __popc(__ballot_sync(kFull, mine != 0u));
    // against every expert of this and the later blocks (each unordered pair is visited once)
    for (int f0 = e0; f0 < E; f0 += 32) {
      const uint32_t other = f0 + lane < E ? st[f0 + lane] : 0u;
      for (int j = 0; j < 32; ++j) {
        const uint32_t o = __shfl_sync(kFull, other, j);
        dup |= mine != 0u && o == mine && f0 + j != e0 + lane;
      }
    }
  }
  if (__any_sync(kFull, dup) && lane == 0) atomicOr(err_index, kErrDuplicateKey);
  if (resident > C && lane == 0) atomicOr(err_index, kErrOverCapacity);
}

cudaError_t launch_check_state(const uint32_t* stamp, size_t n_pairs, int E, int C, uint32_t* err_index,
                               cudaStream_t st) {
  const int wpb = 8;
  check_state_kernel<<<(unsigned)((n_pairs + wpb - 1) / wpb), wpb * 32, 0, st>>>(stamp, n_pairs, E, C, err_index);
  return cudaGetLastError();
}

// Checked mode: sets *err_nonfinite when any of the n logits is NaN or infinite.
__global__ void check_finite_kernel(const float* z, size_t n, uint32_t* err_nonfinite) {
  bool bad = false;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    bad |= !isfinite(z[i]);
  if (bad) atomicOr(err_nonfinite, 1u);
}

cudaError_t launch_check_finite(const float* z, size_t n, uint32_t* err_nonfinite, cudaStream_t st) {
  const size_t blocks = (n + 255) / 256;
  check_finite_kernel<<<(unsigned)(blocks > 1184 ? 1184 : blocks), 256, 0, st>>>(z, n, err_nonfinite);
  return cudaGetLastError();
}

cudaError_t launch_stats(const uint32_t* miss, const uint32_t* cold, unsigned long long* out, int L, int S,
                         cudaStream_t st) {
  stats_kernel<<<L, 256, 0, st>>>(miss, cold, out, S);
  return cudaGetLastError();
}

}  // namespace mcce
