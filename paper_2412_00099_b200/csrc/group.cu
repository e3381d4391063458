// Expert grouping for Eq. 1: the S*K (stream, slot) pairs of a layer are bucketed by expert with a
// histogram, an exclusive scan and a stable scatter, so that each expert's tokens are contiguous.
// One CTA per layer; the order inside a bucket is the pair order (stream-major), which makes the
// result unique.  A second kernel copies the hidden rows into that order.
#include "common.cuh"

namespace mcce {

constexpr int kGroupThreads = 1024;
constexpr int kGroupWarps = kGroupThreads / 32;

__global__ void __launch_bounds__(kGroupThreads) group_kernel(const GroupParams p) {
  __shared__ int hist[kGroupWarps][kMaxE];  // per-warp counts, then per-warp bases
  __shared__ int offs[kMaxE + 1];
  const int l = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int P = p.S * p.K, E = p.E;
  const int32_t* sel = p.sel_idx + (size_t)l * P;
  // contiguous range of pairs per warp, a multiple of 32 so that batches stay aligned
  const int per_warp = ((P + kGroupWarps - 1) / kGroupWarps + 31) & ~31;
  const int begin = min(P, warp * per_warp), end = min(P, begin + per_warp);

  for (int i = threadIdx.x; i < kGroupWarps * kMaxE; i += kGroupThreads) (&hist[0][0])[i] = 0;
  __syncthreads();

  for (int b = begin; b < end; b += 32) {
    const int q = b + lane;
    const bool ok = q < end;
    const int e = ok ? sel[q] : -1;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (ok && lane == __ffs(peers) - 1) hist[warp][e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();

  // per expert: exclusive prefix over warps; then exclusive scan over experts
  for (int e = threadIdx.x; e < E; e += kGroupThreads) {
    int run = 0;
    for (int w = 0; w < kGroupWarps; ++w) {
      const int c = hist[w][e];
      hist[w][e] = run;
      run += c;
    }
    offs[e + 1] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    offs[0] = 0;
    for (int e = 0; e < E; ++e) offs[e + 1] += offs[e];
  }
  __syncthreads();
  for (int e = threadIdx.x; e <= E; e += kGroupThreads) p.offsets[(size_t)l * (E + 1) + e] = offs[e];

  for (int b = begin; b < end; b += 32) {
    const int q = b + lane;
    const bool ok = q < end;
    const int e = ok ? sel[q] : -1;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    int base = 0;
    if (ok) base = hist[warp][e];
    __syncwarp();
    if (ok) {
      const int pos = offs[e] + base + __popc(peers & ((1u << lane) - 1u));
      p.perm[(size_t)l * P + pos] = q;
      p.inv[(size_t)l * P + q] = pos;
      if (lane == __ffs(peers) - 1) hist[warp][e] = base + __popc(peers);
    }
    __syncwarp();
  }
}

cudaError_t launch_group(const GroupParams& p, cudaStream_t st) {
  group_kernel<<<p.L, kGroupThreads, 0, st>>>(p);
  return cudaGetLastError();
}

// Xg[l][pos][:] = hidden[l][perm[l][pos] / K][:]; one warp per row, 16-byte copies.  With zero_y the warp of
// pair (s, k) also clears the k-th of K slices of y[l][s][:], for the expert kernel that accumulates into y.
__global__ void gather_kernel(const FfnParams p, const int zero_y) {
  const int P = p.S * p.K;
  const size_t row = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= (size_t)p.L * P) return;
  const int lane = threadIdx.x & 31;
  const int l = (int)(row / P);
  const int s = p.perm[row] / p.K;
  const size_t bytes = (size_t)p.d * (p.bf16 ? 2 : 4);
  const uint4* src = (const uint4*)((const char*)p.hidden + ((size_t)l * p.S + s) * bytes);
  uint4* dst = (uint4*)((char*)p.Xg + row * bytes);
  for (int i = lane; i < (int)(bytes / 16); i += 32) dst[i] = __ldg(src + i);
  if (zero_y) {
    const int k = p.perm[row] % p.K, n4 = p.d / 4;            // y row: d floats = n4 float4
    const int lo = (int)((long long)n4 * k / p.K), hi = (int)((long long)n4 * (k + 1) / p.K);
    float4* y = (float4*)(p.y + ((size_t)l * p.S + s) * p.d);
    for (int i = lo + lane; i < hi; i += 32) y[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

cudaError_t launch_gather(const FfnParams& p, bool zero_y, cudaStream_t st) {
  const size_t rows = (size_t)p.L * p.S * p.K;
  const int wpb = 8;
  gather_kernel<<<(unsigned)((rows + wpb - 1) / wpb), wpb * 32, 0, st>>>(p, zero_y ? 1 : 0);
  return cudaGetLastError();
}

// Residual stream of the sequential-layer mode: x_out = x_in + y, rounded to the hidden dtype.
__global__ void residual_kernel(const void* x_in, const float* y, void* x_out, size_t n, int bf16) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    if (bf16) {
      const float v = __fadd_rn(__bfloat162float(((const __nv_bfloat16*)x_in)[i]), y[i]);
      ((__nv_bfloat16*)x_out)[i] = __float2bfloat16_rn(v);
    } else {
      ((float*)x_out)[i] = __fadd_rn(((const float*)x_in)[i], y[i]);
    }
  }
}

cudaError_t launch_residual(const void* x_in, const float* y, void* x_out, size_t n, bool bf16, cudaStream_t st) {
  const unsigned grid = (unsigned)((n + 255) / 256 > 2048 ? 2048 : (n + 255) / 256);
  residual_kernel<<<grid, 256, 0, st>>>(x_in, y, x_out, n, bf16 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace mcce
