// Elementary functions of the graph VM, fp32, written for a few-ulp relative error so that
// compositions of many operators stay within 1e-5 of an fp64 evaluation.
//
//   sin/cos : two-constant Cody-Waite reduction by pi/2 (fused multiply-adds) up to 2^20, an exact
//             multi-word reduction beyond; odd/even polynomials on [-pi/4, pi/4]
//   exp     : 2^(x*log2 e) with the product held in two parts, the power of two by the hardware approximation
//   tanh    : x*P(x^2)/Q(x^2), argument clamped at 10, result at 1
//   sigmoid : 1/(1+exp(-x))
// Polynomial coefficients are weighted least-squares fits on Chebyshev nodes, iteratively
// re-weighted towards the minimax error (relative errors 4e-9, 1e-10, 3e-9, 3e-9).
//
// The header also compiles for the host so that the accuracy of the polynomials can be swept
// against fp64 without a GPU (the reciprocal is then an exact division).
#pragma once
#include <cmath>
#include <cstdint>
#include <cstring>

#if defined(__CUDACC__)
#define VM_HD __host__ __device__ __forceinline__
#else
#define VM_HD inline
#endif

namespace dragon {
namespace vmmath {

VM_HD float f_rcp(float x) {
#if defined(__CUDA_ARCH__)
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
#else
  return 1.0f / x;
#endif
}

VM_HD float sqrt_f(float x) {
#if defined(__CUDA_ARCH__)
  float r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
#else
  return sqrtf(x);
#endif
}

VM_HD float f_from_bits(uint32_t u) {
#if defined(__CUDA_ARCH__)
  return __uint_as_float(u);
#else
  float f; std::memcpy(&f, &u, 4); return f;
#endif
}
VM_HD uint32_t f_bits(float f) {
#if defined(__CUDA_ARCH__)
  return __float_as_uint(f);
#else
  uint32_t u; std::memcpy(&u, &f, 4); return u;
#endif
}

VM_HD float sin_poly(float r) {
  const float z = r * r;
  float p = fmaf(z, -1.9515285269243e-4f, 8.33216077944338e-3f);
  p = fmaf(z, p, -1.6666654609873324e-1f);
  return fmaf(r * z, p, r);
}
VM_HD float cos_poly(float r) {
  const float z = r * r;
  float p = fmaf(z, 2.4433150705502356e-5f, -1.3887316189460366e-3f);
  p = fmaf(z, p, 4.1666645681363114e-2f);
  return fmaf(z * z, p, fmaf(z, -0.5f, 1.0f));
}

// Reduction of a large finite argument (|x| > 2^20, where the two-constant reduction below starts to
// lose bits) by multiplying with as many bits of 2/pi as the argument's exponent asks for.
// x = m * 2^s with m a 24-bit integer.  Bits of 2/pi whose weight times 2^s is a multiple of 4 only
// move the result by whole periods and are skipped; the next 96 bits are multiplied by m modulo 2^96:
// the top two bits of that product are the quadrant, the 64 bits below them the fraction of a
// quadrant, read as a signed number so that the remainder lies in [-pi/4, pi/4).  The bits left out
// change the fraction by less than 2^-70, so r is exact to the rounding of the final conversion.
// The table is 2/pi = 0x0.A2F9836E4E44... in 32-bit words behind one word of zeros (the integer part),
// which covers every fp32 exponent: the window starts at bit s + 30 <= 134 and is 96 + 31 bits long.
VM_HD float reduce_pio2_large(float x, int* q) {
  const uint32_t two_over_pi[9] = {0x00000000u, 0xA2F9836Eu, 0x4E441529u, 0xFC2757D1u, 0xF534DDC0u,
                                   0xDB629599u, 0x3C439041u, 0xFE5163ABu, 0xDEBBC561u};
  const uint32_t ix = f_bits(x) & 0x7fffffffu;
  const int s = (int)(ix >> 23) - 150;
  const uint32_t m = (ix & 0x7fffffu) | 0x800000u;
  const int start = s + 30, idx = start >> 5, sh = start & 31;
  const uint32_t w0 = two_over_pi[idx], w1 = two_over_pi[idx + 1], w2 = two_over_pi[idx + 2], w3 = two_over_pi[idx + 3];
  const uint32_t h2 = sh ? (w0 << sh) | (w1 >> (32 - sh)) : w0;
  const uint32_t h1 = sh ? (w1 << sh) | (w2 >> (32 - sh)) : w1;
  const uint32_t h0 = sh ? (w2 << sh) | (w3 >> (32 - sh)) : w2;
  const uint64_t p0 = (uint64_t)m * h0;
  const uint64_t p1 = (uint64_t)m * h1 + (p0 >> 32);
  const uint32_t r2 = m * h2 + (uint32_t)(p1 >> 32), r1 = (uint32_t)p1, r0 = (uint32_t)p0;
  int qi = (int)(r2 >> 30);
  const uint64_t frac = ((uint64_t)((r2 << 2) | (r1 >> 30)) << 32) | (uint64_t)((r1 << 2) | (r0 >> 30));
  const int64_t sf = (int64_t)frac;
  if (sf < 0) qi += 1;                                             // nearest quadrant, remainder below zero
  float r = (float)((double)sf * 8.5153039502163865e-20);          // pi/2 * 2^-64
  if (x < 0.0f) { r = -r; qi = -qi; }
  *q = qi & 3;
  return r;
}

// r = x - k*pi/2 with |r| <= pi/4 (approximately), q = k mod 4.  k = round(x*2/pi) is taken
// with the add-a-big-constant trick (1.5*2^23: the sum's low mantissa bits are the integer), which
// costs two fused multiply-adds instead of a round and a float-to-int conversion on the
// quarter-rate pipe; it is exact for |x*2/pi| < 2^22.  Each reduction step is one fused
// multiply-add, so the first difference is exact while k*fl(pi/2) stays within 24 bits of x;
// the part of pi/2 left out is 1.7e-15 per quadrant (1.1e-9 at 2^20), and the rounding of 2/pi moves
// x*2/pi by at most 0.03 there, so |r| stays below 0.84.  Beyond |x| = 2^20 the exact reduction above
// takes over (the rounded 2/pi would put r further and further outside the polynomials' interval);
// inf and NaN give x - x = NaN.
VM_HD float reduce_pio2(float x, int* q) {
  const float big = 12582912.0f;                                  // 1.5 * 2^23
  const float kb = fmaf(x, 0.636619772367581343f, big);
  float k = kb - big;
  float r = fmaf(-k, 1.57079637050628662109375f, x);        // fl(pi/2)
  r = fmaf(-k, -4.371138828673793e-8f, r);                  // fl(pi/2 - c1)
  int qi = (int)f_bits(kb);                                 // low bits = k (two's complement)
  if (!(fabsf(x) <= 1048576.0f)) {
    if ((f_bits(x) & 0x7fffffffu) >= 0x7f800000u) { r = x - x; qi = 0; }
    else r = reduce_pio2_large(x, &qi);
  }
  *q = qi;
  return r;
}

VM_HD void sincos_f(float x, float* s, float* c) {
  int q;
  const float r = reduce_pio2(x, &q);
  const float ps = sin_poly(r), pc = cos_poly(r);
  float ss = (q & 1) ? pc : ps;
  float cc = (q & 1) ? ps : pc;
  if (q & 2) ss = -ss;
  if ((q + 1) & 2) cc = -cc;
  *s = ss;
  *c = cc;
}
VM_HD float sin_f(float x) {
  int q;
  const float r = reduce_pio2(x, &q);
  const float v = (q & 1) ? cos_poly(r) : sin_poly(r);
  return (q & 2) ? -v : v;
}
VM_HD float cos_f(float x) {
  int q;
  const float r = reduce_pio2(x, &q);
  const float v = (q & 1) ? sin_poly(r) : cos_poly(r);
  return ((q + 1) & 2) ? -v : v;
}

// 2^t: the hardware approximation on the device (relative error at most 2^-22 over the whole range, results
// below 2^-126 flushed to zero), exp2f on the host
VM_HD float f_ex2(float t) {
#if defined(__CUDA_ARCH__)
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
  return r;
#else
  return exp2f(t);
#endif
}

// exp for -86 <= x <= 88.7 (callers clamp), where the result is a normal number: e^x = 2^t with t = x * log2(e)
// held as t_hi + e: t_hi the rounded product, e its exact residue (one fused multiply-add) plus x times the part
// of log2(e) that fp32 leaves out; 2^t_hi by f_ex2, times 1 + e * ln 2.  About 2.5e-7 relative on the device.
VM_HD float exp_core(float x) {
  const float l_hi = 1.44269502162933349609375f, l_lo = 1.9259629911266175e-8f;
  const float t = x * l_hi;
  float e = fmaf(x, l_hi, t * -1.0f);
  e = fmaf(x, l_lo, e);
  e = e * 0.693147180559945309f;
  const float p = f_ex2(t);
  return fmaf(p, e, p);
}
// the clamps keep a NaN a NaN, as the kernel's max.NaN / min.NaN do (fminf / fmaxf alone would drop it)
VM_HD float exp_clamped10(float x) { return x != x ? x : exp_core(fminf(fmaxf(x, -10.0f), 10.0f)); }
VM_HD float exp_wide(float x) { return x != x ? x : exp_core(fminf(fmaxf(x, -86.0f), 88.7f)); }

VM_HD float sigmoid_f(float x) { return f_rcp(1.0f + exp_wide(-x)); }

// tanh(x) = x * P(x^2) / Q(x^2): a rational fit on |x| <= 9 (degrees 4 and 4 in x^2, relative error
// 6e-8 in exact arithmetic, about 3e-7 = 5 ulp once the two Horner chains and the reciprocal round).
// From |x| = 9.01 on tanh rounds to 1 in fp32; the fit crosses 1 at 9.07 and keeps growing (1 + 1.9e-6
// at 10), so with the argument clamped at 10 and the result clamped to [-1, 1] a saturated tanh is
// exactly +-1 (a gradient 1 - y^2 behind it is then exactly 0, as in wider arithmetic, instead of one
// rounding step of y blown up by the cancellation).  NaN stays NaN.
VM_HD float tanh_f(float x) {
  if (x != x) return x;
  const float c = fminf(fmaxf(x, -10.0f), 10.0f);
  const float z = c * c;
  float p = fmaf(z, 1.3442309683456469e-08f, 2.0679596671714183e-05f);
  p = fmaf(z, p, 3.5001979607618507e-03f);
  p = fmaf(z, p, 1.3385017810927272e-01f);
  p = fmaf(z, p, 1.0f);
  float q = fmaf(z, 7.814557141497938e-07f, 3.2929435375013785e-04f);
  q = fmaf(z, q, 2.5894861704209737e-02f);
  q = fmaf(z, q, 4.6718338985166813e-01f);
  q = fmaf(z, q, 1.0f);
  const float y = (c * p) * f_rcp(q);
  return fminf(fmaxf(y, -1.0f), 1.0f);
}

VM_HD float divp_f(float a, float b) { return a * f_rcp(1.0f + fabsf(b)); }

// -sgn(b) / (1 + |b|)^2 with sgn(0) = 0
VM_HD float divp_grad_b(float b) {
  const float r = f_rcp(1.0f + fabsf(b));
  const float sg = b > 0.0f ? 1.0f : (b < 0.0f ? -1.0f : 0.0f);
  return -sg * r * r;
}

// float -> bfloat16 (round to nearest even) -> float
VM_HD uint32_t bf16_bits(float f) {
  uint32_t u = f_bits(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x40u;  // quiet NaN
  return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}
VM_HD float round_bf16(float f) { return f_from_bits(bf16_bits(f) << 16); }

}  // namespace vmmath
}  // namespace dragon
