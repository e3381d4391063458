// Belady's optimal eviction (Sec. 4.8, "Optimal Cache Eviction") replayed on a recorded routing trace:
// the lossless upper bound on the hit rate that the paper compares its lossy rerouting against.
//
// Input is the selection trace sel[t][l][s][k] of a run (typically original routing, lambda = 0).  A first
// kernel walks every (stream, layer) backwards and records, for each selected expert, the next token at
// which it is selected again.  A second kernel replays the trace forwards once per cache capacity: on a
// miss the expert is inserted, and while the cache is over capacity the resident expert whose next use
// lies farthest ahead is evicted -- never one that the current token itself uses (they are needed now).
// One warp per (stream, layer[, capacity]); lane j holds experts j, j+32, ...
#include "common.cuh"
#include "warp_select.cuh"

namespace mcce {
namespace {

constexpr int kNever = 0x7ffffffe;   // "not selected again"; +1 still fits the arg-max key

template <int NE>
__global__ void next_use_kernel(const int32_t* __restrict__ trace, int32_t* __restrict__ next, int T, int LS, int K) {
  const int pair = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (pair >= LS) return;
  int last[NE];
#pragma unroll
  for (int i = 0; i < NE; ++i) last[i] = kNever;
  for (int t = T - 1; t >= 0; --t) {
    const size_t base = ((size_t)t * LS + pair) * K;
    const int e_k = lane < K ? trace[base + lane] : 0;
    int my_next = kNever;
    for (int k = 0; k < K; ++k) {
      const int e = __shfl_sync(kFull, e_k, k);
      const int owner = e & 31, slot = e >> 5;
      int v = 0;
#pragma unroll
      for (int i = 0; i < NE; ++i)
        if (i == slot) {
          v = last[i];
          if (lane == owner) last[i] = t;
        }
      v = __shfl_sync(kFull, v, owner);
      if (lane == k) my_next = v;
    }
    if (lane < K) next[base + lane] = my_next;
  }
}

template <int NE>
__global__ void belady_kernel(const int32_t* __restrict__ trace, const int32_t* __restrict__ next, int T, int LS, int K,
                              int E, const int32_t* __restrict__ capacities, int n_cap, long long* __restrict__ misses) {
  const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (wid >= LS * n_cap) return;
  const int pair = wid % LS, ci = wid / LS;
  const int C = capacities[ci];
  uint32_t nu[NE];       // next use of every resident expert, as an arg-max key (0 = not a candidate)
  uint32_t resb = 0u;
  long long miss = 0;
#pragma unroll
  for (int i = 0; i < NE; ++i) nu[i] = 0u;
  for (int t = 0; t < T; ++t) {
    const size_t base = ((size_t)t * LS + pair) * K;
    const int e_k = lane < K ? trace[base + lane] : 0;
    const int n_k = lane < K ? next[base + lane] : 0;
    uint32_t pinned = 0u;
    for (int k = 0; k < K; ++k) {
      const int e = __shfl_sync(kFull, e_k, k);
      const int n = __shfl_sync(kFull, n_k, k);
      if ((e & 31) == lane) {
        const int slot = e >> 5;
        if (!((resb >> slot) & 1u)) ++miss;
        resb |= 1u << slot;
        pinned |= 1u << slot;
#pragma unroll
        for (int i = 0; i < NE; ++i)
          if (i == slot) nu[i] = (uint32_t)n + 1u;
      }
    }
    int resident = __reduce_add_sync(kFull, __popc(resb));
    while (resident > C) {
      uint32_t key[NE];
#pragma unroll
      for (int i = 0; i < NE; ++i) key[i] = (((resb & ~pinned) >> i) & 1u) ? nu[i] : 0u;
      const int e = warp_argmax<NE>(key, 0u, lane);   // farthest next use, lowest index among equals
      if ((e & 31) == lane) resb &= ~(1u << (e >> 5));
      --resident;
    }
  }
  miss = __reduce_add_sync(kFull, (unsigned)miss);   // per-lane counts are far below 2^32 / 32
  if (lane == 0) misses[(size_t)ci * LS + pair] = miss;
}

template <int NE>
cudaError_t run(const int32_t* trace, int32_t* next, int T, int LS, int K, int E, const int32_t* caps, int n_cap,
                long long* misses, cudaStream_t st) {
  const int wpb = 4;
  next_use_kernel<NE><<<(LS + wpb - 1) / wpb, wpb * 32, 0, st>>>(trace, next, T, LS, K);
  belady_kernel<NE><<<(LS * n_cap + wpb - 1) / wpb, wpb * 32, 0, st>>>(trace, next, T, LS, K, E, caps, n_cap, misses);
  return cudaGetLastError();
}

}  // namespace
}  // namespace mcce

using namespace mcce;

extern "C" int mcce_belady_replay(const int32_t* sel_trace, int32_t n_tokens, int32_t n_layers, int32_t n_streams,
                                  int32_t n_experts, int32_t top_k, const int32_t* capacities, int32_t n_capacities,
                                  int32_t* next_use_scratch, int64_t* misses, void* cuda_stream) {
  if (!sel_trace || !capacities || !next_use_scratch || !misses) return MCCE_EINVAL;
  if (n_tokens < 0 || n_layers < 1 || n_streams < 1 || n_capacities < 1) return MCCE_EINVAL;
  if (n_experts < 1 || n_experts > kMaxE || top_k < 1 || top_k > kMaxK || top_k > n_experts) return MCCE_EINVAL;
  if ((long long)n_layers * n_streams * n_capacities > (1ll << 26) || n_tokens > kNever / 2) return MCCE_EINVAL;
  const int LS = n_layers * n_streams, ne = (n_experts + 31) / 32;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  cudaError_t e;
  auto* m = reinterpret_cast<long long*>(misses);
  if (ne <= 1) e = run<1>(sel_trace, next_use_scratch, n_tokens, LS, top_k, n_experts, capacities, n_capacities, m, st);
  else if (ne <= 2) e = run<2>(sel_trace, next_use_scratch, n_tokens, LS, top_k, n_experts, capacities, n_capacities, m, st);
  else if (ne <= 4) e = run<4>(sel_trace, next_use_scratch, n_tokens, LS, top_k, n_experts, capacities, n_capacities, m, st);
  else e = run<8>(sel_trace, next_use_scratch, n_tokens, LS, top_k, n_experts, capacities, n_capacities, m, st);
  return e == cudaSuccess ? MCCE_OK : MCCE_ECUDA;
}
