// The router's softmax is defined as a fixed sequence of correctly rounded binary32 operations
// (Eq. 1's gate made bit-reproducible), so that two kernels that evaluate it give the same bits.
#pragma once
#include <cuda_runtime.h>

namespace capmoe {

// exp(x), x <= 0: range reduction x = n ln2 + r with a two-word ln2, a degree-7 Taylor polynomial
// in Horner/fma form, scaling by 2^n through the exponent field.  x < -80 gives exactly 0.
__device__ __forceinline__ float exp_fixed(float x) {
  const float x_in = x;
  x = fmaxf(x, -100.0f);            // keeps n in range; whatever comes out below -80 is replaced by 0
  const float n = rintf(__fmul_rn(x, __uint_as_float(0x3fb8aa3bu)));          // x * log2(e)
  float r = __fmaf_rn(n, -__uint_as_float(0x3f317200u), x);                   // - n * ln2_hi
  r = __fmaf_rn(n, -__uint_as_float(0x35bfbe8eu), r);                         // - n * ln2_lo
  float q = __uint_as_float(0x39500d01u);                                     // 1/7!
  q = __fmaf_rn(q, r, __uint_as_float(0x3ab60b61u));                          // 1/6!
  q = __fmaf_rn(q, r, __uint_as_float(0x3c088889u));                          // 1/5!
  q = __fmaf_rn(q, r, __uint_as_float(0x3d2aaaabu));                          // 1/4!
  q = __fmaf_rn(q, r, __uint_as_float(0x3e2aaaabu));                          // 1/3!
  q = __fmaf_rn(q, r, 0.5f);
  q = __fmaf_rn(q, r, 1.0f);
  q = __fmaf_rn(q, r, 1.0f);
  const int ni = (int)n;
  const float p = __uint_as_float(__float_as_uint(q) + ((unsigned)ni << 23));
  return x_in < -80.0f ? 0.0f : p;
}

// a / b rounded to nearest even, for many numerators over one denominator, without the library
// division's per-call range checks: y = RN(1/b) once, then per numerator the usual pair of
// fma corrections (q0 = a y; q1 = q0 + (a - b q0) y; q = q1 + (a - b q1) y), whose last step rounds
// correctly when the remainders are exact.  Valid for b in [1, 2^20] and a = 0 or a in
// [2^-120, 2^20]: numerators below 2^-60 are scaled by 2^64 first so that no remainder is subnormal,
// and the quotient is scaled back (exactly: it stays normal).
// y = __frcp_rn(b), computed once by the caller.
__device__ __forceinline__ float div_by(float a, float b, float y) {
  const bool tiny = a < __uint_as_float(0x21800000u);                       // 2^-60
  const float as = tiny ? __fmul_rn(a, __uint_as_float(0x5f800000u)) : a;   // * 2^64
  const float q0 = __fmul_rn(as, y);
  const float q1 = __fmaf_rn(__fmaf_rn(-b, q0, as), y, q0);
  const float q2 = __fmaf_rn(__fmaf_rn(-b, q1, as), y, q1);
  return tiny ? __fmul_rn(q2, __uint_as_float(0x1f800000u)) : q2;           // * 2^-64
}

}  // namespace capmoe
