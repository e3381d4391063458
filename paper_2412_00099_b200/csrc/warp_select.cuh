// Warp-level selection helpers shared by the routing and replay kernels: an order-preserving integer key
// for floats, arg-max over experts spread across the lanes of a warp, and a shuffle sum.
#pragma once
#include <stdint.h>

namespace mcce {

constexpr unsigned kFull = 0xffffffffu;

// Monotone map float -> uint32 (larger float <=> larger key); -0 is folded onto +0 so that equal
// values have equal keys.  Key 0 is reserved for "no candidate".
__device__ __forceinline__ uint32_t okey(float v) {
  uint32_t u = __float_as_uint(v);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float okey_inv(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

// Expert with the largest key among those not taken; equal keys -> lowest expert index.
template <int NE>
__device__ __forceinline__ int warp_argmax(const uint32_t (&key)[NE], uint32_t taken, int lane) {
  uint32_t bk = 0u, bi = 0xffffffffu;
#pragma unroll
  for (int i = 0; i < NE; ++i) {
    const uint32_t k = ((taken >> i) & 1u) ? 0u : key[i];
    if (k > bk) {
      bk = k;
      bi = (uint32_t)(lane + 32 * i);
    }
  }
  const uint32_t m = __reduce_max_sync(kFull, bk);
  return (int)__reduce_min_sync(kFull, bk == m ? bi : 0xffffffffu);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

}  // namespace mcce
