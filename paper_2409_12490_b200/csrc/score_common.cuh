// Device helpers shared by the score kernels (Algorithm 1, lines 9-14 in the log domain): widening of
// the representatives to fp64, and ln(e^a + e^b) through a table of ln(1 + e^-x).
#pragma once
#include <math_constants.h>

#include "cp_common.cuh"

namespace cp {
namespace {

template <typename T> __device__ __forceinline__ double to_f64(T x);
template <> __device__ __forceinline__ double to_f64<float>(float x) { return double(x); }
template <> __device__ __forceinline__ double to_f64<__nv_bfloat16>(__nv_bfloat16 x) { return double(__bfloat162float(x)); }
template <> __device__ __forceinline__ double to_f64<__half>(__half x) { return double(__half2float(x)); }

// ln(1 + e^-x), x >= 0, from piecewise degree-11 polynomials on intervals of width 1/2 (absolute error 1e-15;
// the table and how it is made: gen_softplus_table.py).  The library exp + log pair costs several hundred fp64
// instructions and this function runs once or twice for every element of the score map.
constexpr int kSpIntervals = 80, kSpCoef = 12, kSpStride = 13;   // stride 13: rows of different intervals hit different banks
static __device__ const double kSoftplusTable[kSpIntervals * kSpCoef] = {
#include "softplus_table.inc"
};
__device__ __forceinline__ double softplus_neg(double x, const double* tab) {
  if (!(x < 40.0)) return 0.0;              // e^-40 = 4e-18: below the rounding of whatever it is added to
  const int i = int(x * 2.0);
  const double t = (x - (0.5 * i + 0.25)) * 4.0;
  const double* c = tab + i * kSpStride;
  double p = c[kSpCoef - 1];
#pragma unroll
  for (int k = kSpCoef - 2; k >= 0; --k) p = fma(p, t, c[k]);
  return p;
}
// ln(e^a + e^b) = max + ln(1 + e^-(max - min))
__device__ __forceinline__ double logaddexp(double a, double b, const double* tab) {
  const double hi = fmax(a, b), lo = fmin(a, b);
  const double x = hi - lo;                 // >= 0 (+inf when one term is -inf), or NaN when both are -inf
  if (!(x >= 0.0)) return hi;
  return hi + softplus_neg(x, tab);
}

}  // namespace
}  // namespace cp
