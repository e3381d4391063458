/*
 * Host implementation, in plain C, of the seeded input generator that synth.py defines: the same
 * definition evaluated a few dozen times faster than the numpy code, so that tests and the CPU baseline can
 * regenerate model-sized inputs (hundreds of millions of elements) in seconds.  It holds none of the
 * routing / caching / FFN arithmetic; it only produces inputs.
 *
 * Definition (see synth.py):
 *   integers  Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), key (seed, 0), counter
 *             (block_lo, block_hi, t, tensor_id), block = flat element index / 4;
 *   normals   Box-Muller on two 24-bit uniforms per pair of words; ln, sin and cos are short series of single
 *             fp32 operations in a fixed order -- every operation is correctly rounded by IEEE-754, so this
 *             file, the numpy code and the CUDA generator give identical bits.
 * Build with -ffp-contract=off (no fused multiply-add) and without fast-math.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static void philox4x32_10(uint32_t c[4], uint32_t k0, uint32_t k1) {
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c[0] = n0, c[1] = n1, c[2] = n2, c[3] = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
}

/* Two standard normals from two words. */
static void box_muller(uint32_t xa, uint32_t xb, float* out0, float* out1) {
  /* radius: r = sqrt(-2 ln u), u = n * 2^-24 with n in 1 .. 2^24 */
  const uint32_t n = (xa >> 8) + 1u;
  int ex;
  const double mant = frexp((double)n, &ex); /* n = mant * 2^ex, mant in [0.5, 1) */
  int e = ex - 1;
  float m = (float)(mant * 2.0);             /* exact: n has at most 25 bits */
  if (m > (float)1.4142135623730951) {
    m = m * 0.5f;
    e += 1;
  }
  const float s = (m - 1.0f) / (m + 1.0f);
  const float s2 = s * s;
  float poly = (float)(2.0 / 11.0);
  poly = poly * s2 + (float)(2.0 / 9.0);
  poly = poly * s2 + (float)(2.0 / 7.0);
  poly = poly * s2 + (float)(2.0 / 5.0);
  poly = poly * s2 + (float)(2.0 / 3.0);
  poly = poly * s2 + 2.0f;
  const float ln_u = poly * s + (float)(e - 24) * (float)0.6931471805599453;
  const float r = sqrtf(-2.0f * ln_u);
  /* angle: theta = 2 pi k 2^-24, reduced to an octant */
  const uint32_t k2 = xb >> 8;
  const uint32_t octant = k2 >> 21;
  uint32_t f = k2 & ((1u << 21) - 1u);
  if (octant & 1u) f = (1u << 21) - f;
  const float a = (float)f * (float)(0.7853981633974483 / 2097152.0);
  const float a2 = a * a;
  float ps = (float)(1.0 / 362880.0);
  ps = ps * a2 + (float)(-1.0 / 5040.0);
  ps = ps * a2 + (float)(1.0 / 120.0);
  ps = ps * a2 + (float)(-1.0 / 6.0);
  ps = ps * a2 + 1.0f;
  const float sin_a = ps * a;
  float pc = (float)(-1.0 / 3628800.0);
  pc = pc * a2 + (float)(1.0 / 40320.0);
  pc = pc * a2 + (float)(-1.0 / 720.0);
  pc = pc * a2 + (float)(1.0 / 24.0);
  pc = pc * a2 + -0.5f;
  pc = pc * a2 + 1.0f;
  const float cos_a = pc;
  const int swap = ((octant + 1u) >> 1) & 1u; /* octants 1, 2, 5, 6 */
  float cx = swap ? sin_a : cos_a;
  float sx = swap ? cos_a : sin_a;
  if (((octant + 2u) >> 2) & 1u) cx = -cx;    /* octants 2 .. 5 */
  if (octant >= 4u) sx = -sx;
  *out0 = r * cx;
  *out1 = r * sx;
}

static uint16_t bf16_bits(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

/* Elements [start, start + count) of the tensor: std * n (one fp32 multiplication), stored as fp32
   (as_bf16 == 0) or as bfloat16 bit patterns rounded to nearest even (as_bf16 != 0). */
void synth_fill(uint32_t seed, uint32_t tensor_id, uint32_t t, uint64_t start, uint64_t count, float std,
                int as_bf16, void* out) {
  const uint64_t b0 = start / 4, b1 = (start + count + 3) / 4;
  uint64_t w = 0;
  for (uint64_t b = b0; b < b1; ++b) {
    uint32_t c[4] = {(uint32_t)b, (uint32_t)(b >> 32), t, tensor_id};
    philox4x32_10(c, seed, 0u);
    float v[4];
    box_muller(c[0], c[1], &v[0], &v[1]);
    box_muller(c[2], c[3], &v[2], &v[3]);
    for (int i = 0; i < 4; ++i) {
      const uint64_t idx = 4 * b + (uint64_t)i;
      if (idx < start || idx >= start + count) continue;
      const float x = v[i] * std;
      if (as_bf16) ((uint16_t*)out)[w] = bf16_bits(x);
      else ((float*)out)[w] = x;
      ++w;
    }
  }
}

/* One token of the AR(1) hidden-state recurrence on `count` elements: h <- n (first != 0) or rho*h + c*n (two
   multiplications and one addition, each rounded); emits x = h + off (off may be NULL) as fp32 or bf16 bits. */
void synth_hidden_step(float* h, const float* n, const float* off, uint64_t count, float rho, float c, int first,
                       int as_bf16, void* out) {
  for (uint64_t i = 0; i < count; ++i) {
    const float a = rho * h[i], b = c * n[i];
    const float v = first ? n[i] : a + b;
    h[i] = v;
    const float x = off ? v + off[i] : v;
    if (as_bf16) ((uint16_t*)out)[i] = bf16_bits(x);
    else ((float*)out)[i] = x;
  }
}
