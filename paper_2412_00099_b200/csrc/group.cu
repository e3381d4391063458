// Expert grouping for Eq. 1: the S*K (stream, slot) pairs of a layer are bucketed by expert with a histogram,
// an exclusive scan and a stable scatter, so that each expert's tokens are contiguous; the order inside a
// bucket is the pair order (stream-major), which makes the result unique.  Two kernels, both spread over the
// whole device:
//   count  one CTA per chunk of kChunk consecutive pairs of a layer: the chunk's histogram over the experts; the
//          CTA that completes a layer turns the histograms into the bucket offsets (exclusive scan over the
//          experts) and, per chunk and expert, the number of pairs that earlier chunks put into the bucket;
//   place  one CTA per chunk again: ranks its pairs behind those of the earlier chunks, writes perm / inv, and
//          copies each pair's hidden row straight to its position in the expert-ordered activation buffer (and
//          clears the pair's slice of y for the expert kernel that accumulates into y) -- grouping and gather are
//          one pass over the rows.
//
// The expert ids come from the caller.  An id outside [0, E) is never used as an index: the pair is left
// out of every bucket (inv = -1, so no later pass touches it) and bit 0 of the context's index-error word
// is set, which mcce_cache_stats reports as MCCE_EINDEX.
#include "common.cuh"

namespace mcce {

constexpr int kChunk = 64;            // pairs per CTA
constexpr int kPlaceThreads = 256;    // two warps rank the chunk's pairs, all eight copy rows
constexpr int kPlaceWarps = kPlaceThreads / 32;
constexpr int kPartVec = 128;         // 16-byte vectors of a row that one CTA moves (column part)

int group_chunks(int S, int K) { return (S * K + kChunk - 1) / kChunk; }

// counts [L][B][E] receives, per layer, the exclusive prefix over the chunks of each expert's per-chunk count (what
// the earlier chunks put into the bucket), and offsets [L][E+1] the bucket offsets: the CTA that finishes a layer's
// last histogram (a ticket per layer, reset for the next launch) turns the histograms into both.
__global__ void __launch_bounds__(kChunk) group_count_kernel(const GroupParams p, int* counts, int* tickets) {
  __shared__ int hist[kMaxE];
  __shared__ int last;
  const int b = blockIdx.x, l = blockIdx.y, B = gridDim.x;
  const int P = p.S * p.K, E = p.E;
  for (int e = threadIdx.x; e < E; e += kChunk) hist[e] = 0;
  __syncthreads();
  const int q = b * kChunk + threadIdx.x;
  if (q < P) {
    const int e = p.sel_idx[(size_t)l * P + q];
    if ((unsigned)e < (unsigned)E) atomicAdd(&hist[e], 1);
    else atomicOr(p.err_index, kErrBadExpertId);
  }
  __syncthreads();
  int* cl = counts + (size_t)l * B * E;
  for (int e = threadIdx.x; e < E; e += kChunk) cl[(size_t)b * E + e] = hist[e];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(&tickets[l], 1) == B - 1;
  __syncthreads();
  if (!last) return;
  __threadfence();
  // every histogram of the layer is in: per expert, running sum over the chunks (eight loads in flight at a time)
  for (int e = threadIdx.x; e < E; e += kChunk) {
    int run = 0;
    for (int b0 = 0; b0 < B; b0 += 8) {
      int n[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) n[i] = b0 + i < B ? __ldcg(cl + (size_t)(b0 + i) * E + e) : 0;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (b0 + i < B) {
          cl[(size_t)(b0 + i) * E + e] = run;
          run += n[i];
        }
    }
    hist[e] = run;   // bucket size
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int* off = p.offsets + (size_t)l * (E + 1);
    int run = 0;
    for (int e = 0; e < E; ++e) {
      off[e] = run;
      run += hist[e];
    }
    off[E] = run;
    tickets[l] = 0;
  }
}

cudaError_t launch_group(const GroupParams& p, int* counts, int* tickets, cudaStream_t st) {
  const int B = group_chunks(p.S, p.K);
  group_count_kernel<<<dim3(B, p.L), kChunk, 0, st>>>(p, counts, tickets);
  return cudaGetLastError();
}

// grid (chunks, layers, column parts): CTA (b, l, c) ranks the pairs of chunk b and moves column part c of their
// rows.  f carries the hidden rows, the activation buffer and y.
__global__ void __launch_bounds__(kPlaceThreads)
group_place_kernel(const GroupParams p, const FfnParams f, const int* counts, const int zero_y) {
  __shared__ int warp_cnt[2][kMaxE];      // pairs of each expert in the chunk's first / second warp
  __shared__ int pos_of[kChunk];          // position of every pair of the chunk, -1: skipped
  const int b = blockIdx.x, l = blockIdx.y, B = gridDim.x, cpart = blockIdx.z, C = gridDim.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int P = p.S * p.K, E = p.E;

  // ---- rank of every pair of the chunk inside its bucket (warps 0 and 1: 32 pairs each, in pair order) --------
  for (int i = threadIdx.x; i < 2 * kMaxE; i += kPlaceThreads) (&warp_cnt[0][0])[i] = 0;
  __syncthreads();
  const int q = b * kChunk + threadIdx.x;
  int e = -1, rank = 0, first = 0;
  bool ok = false;
  if (warp < 2) {
    e = q < P ? p.sel_idx[(size_t)l * P + q] : -1;
    ok = q < P && (unsigned)e < (unsigned)E;
    if (ok) first = p.offsets[(size_t)l * (E + 1) + e] + counts[((size_t)l * B + b) * E + e];
    const unsigned peers = __match_any_sync(0xffffffffu, ok ? e : -1);
    rank = __popc(peers & ((1u << lane) - 1u));
    if (ok && lane == __ffs(peers) - 1) warp_cnt[warp][e] = __popc(peers);
  }
  __syncthreads();
  if (warp < 2) {
    int pos = -1;
    if (ok) pos = first + (warp == 1 ? warp_cnt[0][e] : 0) + rank;
    pos_of[threadIdx.x] = pos;
    if (q < P && cpart == 0) {
      p.inv[(size_t)l * P + q] = pos;
      if (ok) p.perm[(size_t)l * P + pos] = q;
    }
  }
  __syncthreads();

  // ---- rows: Xg[l][pos][:] = hidden[l][s][:], and the pair's slice of y cleared ---------------------------------
  const size_t bytes = (size_t)f.d * (f.bf16 ? 2 : 4);
  const int n16 = (int)(bytes / 16), c_lo = n16 * cpart / C, c_hi = n16 * (cpart + 1) / C;
  const int n4 = f.d / 4, y_lo = n4 * cpart / C, y_hi = n4 * (cpart + 1) / C;
  for (int j = warp; j < kChunk; j += kPlaceWarps) {
    const int qj = b * kChunk + j;
    if (qj >= P) break;
    const int s = qj / p.K, k = qj % p.K;
    if (zero_y) {   // slice k of K of y[l][s], whatever sel_idx held
      const int lo = max(y_lo, (int)((long long)n4 * k / p.K)), hi = min(y_hi, (int)((long long)n4 * (k + 1) / p.K));
      float4* y = (float4*)(f.y + ((size_t)l * f.S + s) * f.d);
      for (int i = lo + lane; i < hi; i += 32) y[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int pos = pos_of[j];
    if (pos < 0) continue;
    const uint4* src = (const uint4*)((const char*)f.hidden + ((size_t)l * f.S + s) * bytes);
    uint4* dst = (uint4*)((char*)f.Xg + ((size_t)l * P + pos) * bytes);
#pragma unroll 4
    for (int i = c_lo + lane; i < c_hi; i += 32) dst[i] = __ldg(src + i);
  }
}

// Column parts per row: no wider than kPartVec vectors (four per lane and row), and more of them while small
// layers would otherwise leave the device idle.
cudaError_t launch_place(const GroupParams& p, const FfnParams& f, const int* counts, bool zero_y, cudaStream_t st) {
  const int B = group_chunks(p.S, p.K);
  const int n16 = (int)((size_t)f.d * (f.bf16 ? 2 : 4) / 16);
  int C = (n16 + kPartVec - 1) / kPartVec;
  while ((long long)B * p.L * C < 592 && n16 / (2 * C) >= 32) C *= 2;
  if (C > 65535) return cudaErrorInvalidValue;
  group_place_kernel<<<dim3(B, p.L, C), kPlaceThreads, 0, st>>>(p, f, counts, zero_y ? 1 : 0);
  return cudaGetLastError();
}

// Checked mode: what the grouping pass wrote is consistent -- offsets start at 0, never decrease and end at
// most at S*K, and every position below the end holds a pair index inside [0, S*K).
__global__ void check_group_kernel(const GroupParams p) {
  const int l = blockIdx.x, P = p.S * p.K;
  const int32_t* off = p.offsets + (size_t)l * (p.E + 1);
  bool bad = false;
  for (int e = threadIdx.x; e <= p.E; e += blockDim.x) {
    const int o = off[e];
    bad |= o < 0 || o > P || (e == 0 && o != 0) || (e > 0 && o < off[e - 1]);
  }
  const int end = min(max(off[p.E], 0), P);
  for (int i = threadIdx.x; i < end; i += blockDim.x) bad |= (unsigned)p.perm[(size_t)l * P + i] >= (unsigned)P;
  if (bad) atomicOr(p.err_index, kErrBadPosition);
}

cudaError_t launch_check_group(const GroupParams& p, cudaStream_t st) {
  check_group_kernel<<<p.L, 256, 0, st>>>(p);
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
