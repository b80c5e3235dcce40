// Element-wise arithmetic of the closed-form recall score (Section 3.3 "Recall": tokens are ranked by
// their theoretical hash collision probability with the query): for a cosine c between a window
// query and a key, the probability that none of K independent Gaussian hyperplanes separates them,
//   (1 - theta / pi)^K,   theta = acos(c).
#pragma once
#include "ptx.cuh"

namespace lkv {

// acos(x) / pi ~= sqrt(1 - x) * P(x) on [0, 1], |error| < 3e-8 (degree 7, the form of Abramowitz &
// Stegun 4.4.46; the coefficients are those of the fit in acos_poly.py beside this file, divided by
// pi). LKV_ACOS_TOP is the leading coefficient, LKV_ACOS_POLY the Horner steps below it.
#define LKV_ACOS_TOP (-4.0197156638e-04f)
#define LKV_ACOS_POLY(STEP) \
  STEP(2.1235386008e-03f) STEP(-5.4398557361e-03f) STEP(9.8335642476e-03f) STEP(-1.5971107888e-02f) \
  STEP(2.8322911244e-02f) STEP(-6.8308920822e-02f) STEP(4.9999999306e-01f)
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// x^KB for two values by repeated squaring (KB a compile-time count of sign bits).
template <int KB>
__device__ __forceinline__ float2 pow_int2(float2 x) {
  float2 r = make_float2(1.f, 1.f), sq = x;
  bool first = true;
#pragma unroll
  for (int b = KB; b > 0; b >>= 1) {
    if (b & 1) { r = first ? sq : __fmul2_rn(r, sq); first = false; }
    if (b > 1) sq = __fmul2_rn(sq, sq);
  }
  return r;
}
// (1 - theta/pi)^K for two cosines: u = acos(-c) / pi = 1 - acos(c)/pi (c >= 0), acos(|c|)/pi (c < 0).
// KB > 0: u^KB by multiplication; KB == 0: any K at run time as 2^(K log2 u). u = 0 gives 0 either way.
template <int KB>
__device__ __forceinline__ float2 collide_pow2(float2 c, float kbits) {
  const float2 x = make_float2(fminf(fabsf(c.x), 1.f), fminf(fabsf(c.y), 1.f));
  float2 p = make_float2(LKV_ACOS_TOP, LKV_ACOS_TOP);            // Horner, highest coefficient first
#define LKV_HORNER(A) p = __ffma2_rn(p, x, make_float2(A, A));
  LKV_ACOS_POLY(LKV_HORNER)
#undef LKV_HORNER
  const float2 om = __ffma2_rn(x, make_float2(-1.f, -1.f), make_float2(1.f, 1.f));   // 1 - x
  const float2 a = __fmul2_rn(make_float2(sqrt_approx(om.x), sqrt_approx(om.y)), p);
  const float2 u = make_float2(c.x >= 0.f ? 1.f - a.x : a.x, c.y >= 0.f ? 1.f - a.y : a.y);
  if (KB > 0) return pow_int2<KB>(u);
  return make_float2(ex2_approx(kbits * lg2_approx(u.x)), ex2_approx(kbits * lg2_approx(u.y)));
}

}  // namespace lkv
