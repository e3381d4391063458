// Expert FFN of Eq. 1 on the plain fp32 pipe: E_i(x) = W_d (silu(W_g x) * (W_u x)), expert by expert
// over the grouped tokens, followed by the weighted combine.  This path handles every shape and both
// dtypes (it is the one used for fp32 weights and for shapes the tensor-core path does not tile); a CTA
// owns 32 output rows of one expert and walks that expert's tokens eight at a time, so each weight
// element fetched is used for eight tokens.
#include "common.cuh"

namespace mcce {

constexpr int kTB = 8;      // tokens per tile (= warps per CTA: warp w stages token w)
constexpr int kRW = 4;      // output rows per warp
constexpr int kKC = 1024;   // reduction chunk staged in shared memory
constexpr unsigned kFull = 0xffffffffu;

template <typename T>
__device__ __forceinline__ float4 load4(const T* p);
template <>
__device__ __forceinline__ float4 load4<float>(const float* p) {
  return __ldg((const float4*)p);
}
template <>
__device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 u = __ldg((const uint2*)p);
  const float2 a = __bfloat1622float2(*(const __nv_bfloat162*)&u.x);
  const float2 b = __bfloat1622float2(*(const __nv_bfloat162*)&u.y);
  return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void store1(float* p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float dot4(const float4 a, const float4 x, float acc) {
  return fmaf(a.x, x.x, fmaf(a.y, x.y, fmaf(a.z, x.z, fmaf(a.w, x.w, acc))));
}

// GATE_UP: in = activations [rows, d], weights Wg/Wu [I, d], out H[rows, I] = silu(g)*u  (type T)
// else   : in = H [rows, I],           weights Wd [d, I],    out O[rows, d]              (fp32)
template <typename T, bool GATE_UP>
__global__ void __launch_bounds__(kTB * 32) ffn_simt_kernel(const FfnParams p) {
  __shared__ __align__(16) float xs[kTB][kKC];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.E + p.n_sh, P = p.S * p.K;
  const int l = blockIdx.y / G, e = blockIdx.y % G;
  const int R = GATE_UP ? p.d : p.I;      // reduction length
  const int NO = GATE_UP ? p.I : p.d;     // output rows of the weight matrix
  const size_t wsz = (size_t)p.I * p.d;

  size_t row0;      // first row of this group in H / O
  int m;            // tokens in the group
  const T *in, *W0, *W1 = nullptr;
  if (e < p.E) {
    const int o0 = p.offsets[(size_t)l * (p.E + 1) + e], o1 = p.offsets[(size_t)l * (p.E + 1) + e + 1];
    row0 = (size_t)l * P + o0;
    m = o1 - o0;
    const size_t wi = (size_t)(p.l0 + l) * p.E + e;
    if (GATE_UP) {
      in = (const T*)p.Xg + row0 * p.d;
      W0 = (const T*)p.Wg + wi * wsz;
      W1 = (const T*)p.Wu + wi * wsz;
    } else {
      in = (const T*)p.H + row0 * p.I;
      W0 = (const T*)p.Wd + wi * wsz;
    }
  } else {
    const int q = e - p.E;
    row0 = (size_t)p.L * P + ((size_t)l * p.n_sh + q) * p.S;
    m = p.S;
    const size_t wi = (size_t)(p.l0 + l) * p.n_sh + q;
    if (GATE_UP) {
      in = (const T*)p.hidden + (size_t)l * p.S * p.d;
      W0 = (const T*)p.shWg + wi * wsz;
      W1 = (const T*)p.shWu + wi * wsz;
    } else {
      in = (const T*)p.H + row0 * p.I;
      W0 = (const T*)p.shWd + wi * wsz;
    }
  }
  if (m == 0) return;

  const int r_base = blockIdx.x * (kTB * kRW) + warp * kRW;
  for (int t0 = 0; t0 < m; t0 += kTB) {
    float acc0[kRW][kTB], acc1[kRW][kTB];
#pragma unroll
    for (int r = 0; r < kRW; ++r)
#pragma unroll
      for (int q = 0; q < kTB; ++q) acc0[r][q] = acc1[r][q] = 0.f;

    for (int c0 = 0; c0 < R; c0 += kKC) {
      const int rc = min(kKC, R - c0);
      __syncthreads();
      {  // warp w stages token t0+w
        const bool ok = t0 + warp < m;
        const T* x = in + (size_t)(t0 + (ok ? warp : 0)) * R + c0;
        for (int k = 4 * lane; k < rc; k += 128) {
          const float4 v = ok ? load4<T>(x + k) : make_float4(0.f, 0.f, 0.f, 0.f);
          *(float4*)&xs[warp][k] = v;
        }
      }
      __syncthreads();
#pragma unroll
      for (int r = 0; r < kRW; ++r) {
        const int ro = min(r_base + r, NO - 1);
        const T* w0 = W0 + (size_t)ro * R + c0;
        const T* w1 = GATE_UP ? W1 + (size_t)ro * R + c0 : nullptr;
        for (int k = 4 * lane; k < rc; k += 128) {
          const float4 a = load4<T>(w0 + k);
          float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
          if (GATE_UP) b = load4<T>(w1 + k);
#pragma unroll
          for (int q = 0; q < kTB; ++q) {
            const float4 x = *(const float4*)&xs[q][k];
            acc0[r][q] = dot4(a, x, acc0[r][q]);
            if (GATE_UP) acc1[r][q] = dot4(b, x, acc1[r][q]);
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kRW; ++r) {
#pragma unroll
      for (int q = 0; q < kTB; ++q) {
        float g = acc0[r][q], u = acc1[r][q];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          g += __shfl_xor_sync(kFull, g, o);
          if (GATE_UP) u += __shfl_xor_sync(kFull, u, o);
        }
        if (lane == q && t0 + q < m && r_base + r < NO) {
          const size_t row = row0 + t0 + q;
          if (GATE_UP) {
            const float h = (g / (1.f + expf(-g))) * u;
            store1((T*)p.H + row * p.I + r_base + r, h);
          } else {
            p.O[row * p.d + r_base + r] = g;
          }
        }
      }
    }
  }
}

cudaError_t launch_ffn_simt_up(const FfnParams& p, cudaStream_t st) {
  const dim3 grid((p.I + kTB * kRW - 1) / (kTB * kRW), p.L * (p.E + p.n_sh));
  if (p.bf16) ffn_simt_kernel<__nv_bfloat16, true><<<grid, kTB * 32, 0, st>>>(p);
  else ffn_simt_kernel<float, true><<<grid, kTB * 32, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_ffn_simt_down(const FfnParams& p, cudaStream_t st) {
  const dim3 grid((p.d + kTB * kRW - 1) / (kTB * kRW), p.L * (p.E + p.n_sh));
  if (p.bf16) ffn_simt_kernel<__nv_bfloat16, false><<<grid, kTB * 32, 0, st>>>(p);
  else ffn_simt_kernel<float, false><<<grid, kTB * 32, 0, st>>>(p);
  return cudaGetLastError();
}

// y[l,s,:] = sum_k w_k O[pair (s,k)] in slot order, then the shared experts with weight 1.
__global__ void combine_kernel(const FfnParams p) {
  const int P = p.S * p.K;
  const size_t ls = blockIdx.x;  // l*S + s
  const int l = (int)(ls / p.S), s = (int)(ls % p.S);
  __shared__ int pos[kMaxK];
  __shared__ float w[kMaxK];
  if (threadIdx.x < p.K) {
    pos[threadIdx.x] = p.inv[(size_t)l * P + s * p.K + threadIdx.x];
    w[threadIdx.x] = p.sel_w[ls * p.K + threadIdx.x];
  }
  __syncthreads();
  for (int j = 4 * threadIdx.x; j < p.d; j += 4 * blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < p.K; ++k) {
      if (pos[k] < 0) continue;   // pair skipped by the grouping pass (expert id out of range)
      const float4 o = __ldg((const float4*)(p.O + ((size_t)l * P + pos[k]) * p.d + j));
      acc.x = fmaf(w[k], o.x, acc.x);
      acc.y = fmaf(w[k], o.y, acc.y);
      acc.z = fmaf(w[k], o.z, acc.z);
      acc.w = fmaf(w[k], o.w, acc.w);
    }
    for (int q = 0; q < p.n_sh; ++q) {
      const size_t row = (size_t)p.L * P + ((size_t)l * p.n_sh + q) * p.S + s;
      const float4 o = __ldg((const float4*)(p.O + row * p.d + j));
      acc.x += o.x;
      acc.y += o.y;
      acc.z += o.z;
      acc.w += o.w;
    }
    *(float4*)(p.y + ls * p.d + j) = acc;
  }
}

cudaError_t launch_combine(const FfnParams& p, cudaStream_t st) {
  combine_kernel<<<p.L * p.S, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace mcce
