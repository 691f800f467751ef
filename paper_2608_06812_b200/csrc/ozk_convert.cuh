// Shared-exponent integer conversion (Section 4.2): round-to-nearest-even of x * 2^s, done on the integer
// significand so that the scaling is an exact exponent shift for every finite input, subnormals and
// shifts beyond the FP64 exponent range included.
#pragma once

#include <cuda_runtime.h>

namespace ozk {

// Returns the magnitude of round(x * 2^s): at most 2^c when |x| is at most its row or column maximum and s the
// shift for a width of c <= 62 bits (c > 53 only in the extended-capacity mode);
// *neg receives the sign of x.
__device__ __forceinline__ unsigned long long to_integer_magnitude(double x, int s, bool* neg) {
  const unsigned long long bits = (unsigned long long)__double_as_longlong(x);
  *neg = (bits >> 63) != 0;
  const int E = (int)((bits >> 52) & 0x7FF);
  unsigned long long mant = bits & 0x000FFFFFFFFFFFFFull;
  if (E) mant |= 1ull << 52;
  if (mant == 0) return 0;
  const int sh = (E ? E : 1) - 1075 + s;  // x * 2^s = mant * 2^sh
  if (sh >= 0) return sh > 62 ? 0 : mant << sh;  // |x 2^s| <= 2^62 keeps the shifted significand inside 64 bits
  const int d = -sh;
  if (d > 54) return 0;
  const unsigned long long q = mant >> d;
  const unsigned long long rem = mant & ((1ull << d) - 1);
  const unsigned long long half = 1ull << (d - 1);
  return q + ((rem > half) || (rem == half && (q & 1ull)) ? 1ull : 0ull);
}

// The same conversion on the FP64 pipe: round(x * 2^s) with ties to even as a signed 64-bit integer.  Scaling by
// a power of two is exact as long as the product is a normal number, so x * 2^s is formed in two exact steps
// (2^s itself is not a double for s beyond 1023: rows of tiny or huge numbers) and rounded once by the
// conversion instruction.  An intermediate that falls into the subnormal range belongs to an element at least
// 2^900 below its row maximum: its converted value is 0 either way.  Requires |x * 2^s| <= 2^62.
struct ScalePair {
  double f1, f2;  // 2^s = f1 * f2, both normal powers of two
};
__device__ __forceinline__ ScalePair make_scale(int s) {
  const int s1 = max(-1000, min(1000, s));
  ScalePair p;
  p.f1 = __longlong_as_double((long long)(s1 + 1023) << 52);
  p.f2 = __longlong_as_double((long long)(s - s1 + 1023) << 52);
  return p;
}
__device__ __forceinline__ long long to_integer_rne(double x, const ScalePair& p) { return __double2ll_rn(x * p.f1 * p.f2); }

}  // namespace ozk
