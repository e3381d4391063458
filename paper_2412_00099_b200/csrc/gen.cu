// Seeded synthetic inputs on the device.  Counter-based, so any element can be regenerated anywhere:
// Philox4x32-10 (Salmon et al., SC'11) keyed by (seed, 0) with counter (block_lo, block_hi, t,
// tensor_id), block = element index / 4; each call yields four normals by Box-Muller.  ln, sin and cos
// are short series evaluated with single correctly-rounded fp32 operations in a fixed order (no fused
// multiply-add), so a host implementation of the same definition reproduces every bit.
#include "common.cuh"

namespace mcce {

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

// Two standard normals from two 32-bit words.
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& n0, float& n1) {
  // r = sqrt(-2 ln u), u = (k+1) 2^-24 in (0,1]:  ln u = ln m + (e-24) ln 2, m in [1/sqrt2, sqrt2]
  const uint32_t n = (xa >> 8) + 1u;
  int e = 31 - __clz(n);
  float m = __fmul_rn(__uint2float_rn(n), __int_as_float((127 - e) << 23));  // exact, [1,2)
  if (m > 1.41421356237309515f) {
    m = __fmul_rn(m, 0.5f);
    e += 1;
  }
  const float s = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
  const float s2 = __fmul_rn(s, s);
  float poly = (float)(2.0 / 11.0);
  poly = __fadd_rn(__fmul_rn(poly, s2), (float)(2.0 / 9.0));
  poly = __fadd_rn(__fmul_rn(poly, s2), (float)(2.0 / 7.0));
  poly = __fadd_rn(__fmul_rn(poly, s2), (float)(2.0 / 5.0));
  poly = __fadd_rn(__fmul_rn(poly, s2), (float)(2.0 / 3.0));
  poly = __fadd_rn(__fmul_rn(poly, s2), 2.0f);
  const float ln_u = __fadd_rn(__fmul_rn(poly, s), __fmul_rn((float)(e - 24), (float)0.6931471805599453));
  const float r = __fsqrt_rn(__fmul_rn(-2.0f, ln_u));
  // theta = 2 pi k2 2^-24 by octant, angle inside the octant in [0, pi/4]
  const uint32_t k2 = xb >> 8;
  const uint32_t oct = k2 >> 21;
  uint32_t f = k2 & ((1u << 21) - 1u);
  if (oct & 1u) f = (1u << 21) - f;
  const float a = __fmul_rn(__uint2float_rn(f), (float)(0.7853981633974483 / 2097152.0));
  const float a2 = __fmul_rn(a, a);
  float ps = (float)(1.0 / 362880.0);
  ps = __fadd_rn(__fmul_rn(ps, a2), (float)(-1.0 / 5040.0));
  ps = __fadd_rn(__fmul_rn(ps, a2), (float)(1.0 / 120.0));
  ps = __fadd_rn(__fmul_rn(ps, a2), (float)(-1.0 / 6.0));
  ps = __fadd_rn(__fmul_rn(ps, a2), 1.0f);
  const float sin_a = __fmul_rn(ps, a);
  float pc = (float)(-1.0 / 3628800.0);
  pc = __fadd_rn(__fmul_rn(pc, a2), (float)(1.0 / 40320.0));
  pc = __fadd_rn(__fmul_rn(pc, a2), (float)(-1.0 / 720.0));
  pc = __fadd_rn(__fmul_rn(pc, a2), (float)(1.0 / 24.0));
  pc = __fadd_rn(__fmul_rn(pc, a2), -0.5f);
  pc = __fadd_rn(__fmul_rn(pc, a2), 1.0f);
  const bool swap = ((oct + 1u) >> 1) & 1u;
  float cx = swap ? sin_a : pc, sx = swap ? pc : sin_a;
  if (((oct + 2u) >> 2) & 1u) cx = -cx;
  if (oct >= 4u) sx = -sx;
  n0 = __fmul_rn(r, cx);
  n1 = __fmul_rn(r, sx);
}

__device__ __forceinline__ void normals4(uint64_t block, uint32_t t, uint32_t tensor_id, uint32_t seed,
                                         float (&n)[4]) {
  uint32_t x[4];
  philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), t, tensor_id, seed, 0u, x);
  box_muller(x[0], x[1], n[0], n[1]);
  box_muller(x[2], x[3], n[2], n[3]);
}

__device__ __forceinline__ void store4(void* out, int bf16, uint64_t i, const float (&v)[4], uint64_t limit) {
  if (i + 4 <= limit) {
    if (bf16) {
      __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
      uint2 u;
      u.x = *(uint32_t*)&a;
      u.y = *(uint32_t*)&b;
      *(uint2*)((__nv_bfloat16*)out + i) = u;
    } else {
      *(float4*)((float*)out + i) = make_float4(v[0], v[1], v[2], v[3]);
    }
  } else {
    for (int j = 0; j < 4 && i + j < limit; ++j) {
      if (bf16) ((__nv_bfloat16*)out)[i + j] = __float2bfloat16_rn(v[j]);
      else ((float*)out)[i + j] = v[j];
    }
  }
}

__global__ void gen_normal_kernel(void* out, int bf16, uint64_t start_block, uint64_t count, uint32_t seed,
                                  uint32_t tensor_id, uint32_t t, float std) {
  const uint64_t nb = (count + 3) / 4;
  for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nb; b += (uint64_t)gridDim.x * blockDim.x) {
    float n[4];
    normals4(start_block + b, t, tensor_id, seed, n);
#pragma unroll
    for (int j = 0; j < 4; ++j) n[j] = __fmul_rn(n[j], std);
    store4(out, bf16, 4 * b, n, count);
  }
}

constexpr uint32_t kTensorNoise = 8, kTensorOffset = 9;  // ids of the hidden-state streams

__global__ void gen_hidden_kernel(float* state, void* x_out, int bf16, uint64_t count, uint32_t seed, uint32_t t,
                                  float rho, float c, float offset_scale) {
  const uint64_t nb = count / 4;
  for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nb; b += (uint64_t)gridDim.x * blockDim.x) {
    float n[4], h[4];
    normals4(b, t, kTensorNoise, seed, n);
    float4 prev = make_float4(0.f, 0.f, 0.f, 0.f);
    if (t != 0) prev = *(const float4*)(state + 4 * b);
    const float pv[4] = {prev.x, prev.y, prev.z, prev.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) h[j] = t == 0 ? n[j] : __fadd_rn(__fmul_rn(rho, pv[j]), __fmul_rn(c, n[j]));
    *(float4*)(state + 4 * b) = make_float4(h[0], h[1], h[2], h[3]);
    if (offset_scale != 0.f) {
      float o[4];
      normals4(b, 0u, kTensorOffset, seed, o);
#pragma unroll
      for (int j = 0; j < 4; ++j) h[j] = __fadd_rn(h[j], __fmul_rn(o[j], offset_scale));
    }
    store4(x_out, bf16, 4 * b, h, count);
  }
}

__global__ void philox_words_kernel(uint32_t* out, uint64_t start_block, uint64_t n_blocks, uint32_t seed,
                                    uint32_t tensor_id, uint32_t t) {
  for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < n_blocks;
       b += (uint64_t)gridDim.x * blockDim.x) {
    uint32_t x[4];
    const uint64_t blk = start_block + b;
    philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), t, tensor_id, seed, 0u, x);
    *(uint4*)(out + 4 * b) = make_uint4(x[0], x[1], x[2], x[3]);
  }
}

static unsigned grid_for(uint64_t items) {
  const uint64_t g = (items + 255) / 256;
  return (unsigned)(g < 1 ? 1 : (g > 148ull * 32 ? 148ull * 32 : g));
}

}  // namespace mcce

using namespace mcce;

extern "C" int mcce_gen_normal(void* out, int32_t dtype, uint64_t start, uint64_t count, uint32_t seed,
                               uint32_t tensor_id, uint32_t t, float std, void* cuda_stream) {
  if (!out || (start & 3) || (dtype != MCCE_F32 && dtype != MCCE_BF16)) return MCCE_EINVAL;
  if (count == 0) return MCCE_OK;
  gen_normal_kernel<<<grid_for((count + 3) / 4), 256, 0, (cudaStream_t)cuda_stream>>>(
      out, dtype == MCCE_BF16, start / 4, count, seed, tensor_id, t, std);
  return cudaGetLastError() == cudaSuccess ? MCCE_OK : MCCE_ECUDA;
}

extern "C" int mcce_gen_hidden_step(float* state, void* x_out, int32_t dtype, uint64_t count, uint32_t seed,
                                    uint32_t t, float rho, float c, float offset_scale, void* cuda_stream) {
  if (!state || !x_out || (count & 3) || (dtype != MCCE_F32 && dtype != MCCE_BF16)) return MCCE_EINVAL;
  if (count == 0) return MCCE_OK;
  gen_hidden_kernel<<<grid_for(count / 4), 256, 0, (cudaStream_t)cuda_stream>>>(
      state, x_out, dtype == MCCE_BF16, count, seed, t, rho, c, offset_scale);
  return cudaGetLastError() == cudaSuccess ? MCCE_OK : MCCE_ECUDA;
}

extern "C" int mcce_gen_philox_words(uint32_t* out, uint64_t start_block, uint64_t n_blocks, uint32_t seed,
                                     uint32_t tensor_id, uint32_t t, void* cuda_stream) {
  if (!out) return MCCE_EINVAL;
  if (n_blocks == 0) return MCCE_OK;
  philox_words_kernel<<<grid_for(n_blocks), 256, 0, (cudaStream_t)cuda_stream>>>(out, start_block, n_blocks, seed,
                                                                                 tensor_id, t);
  return cudaGetLastError() == cudaSuccess ? MCCE_OK : MCCE_ECUDA;
}
