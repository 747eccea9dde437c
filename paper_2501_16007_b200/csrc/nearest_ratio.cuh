// nearest_ratio.cuh -- the mean of Algorithm 2's mantissa differences as a correctly rounded
// double, without an fp64 division.
#ifndef TOPLOC_NEAREST_RATIO_CUH_
#define TOPLOC_NEAREST_RATIO_CUH_

#include <stdint.h>

// The double nearest to s / n (ties to even; n > 0) by long division in integers: the same
// value as (double)s / (double)n.  The fp64 division has a latency of microseconds here (5 us
// per chunk were measured at the end of a block that had its SM to itself); this takes a few
// hundred integer instructions.
__device__ __forceinline__ double nearest_ratio(uint32_t s, uint32_t n) {
  if (s == 0) return 0.0;
  const uint32_t whole = s / n;
  unsigned long long r = s - whole * n, m;
  int e, have;
  if (whole) {
    e = 31 - __clz(whole);
    m = whole;
    have = e + 1;
  } else {  // the leading zeros of the fraction
    e = 0;
    do {
      --e;
      r <<= 1;
    } while (r < n);
    r -= n;
    m = 1;
    have = 1;
  }
  for (; have < 54; ++have) {  // 53 bits and a guard bit
    r <<= 1;
    m <<= 1;
    if (r >= n) {
      r -= n;
      m |= 1;
    }
  }
  const bool guard = m & 1ull;
  m >>= 1;
  if (guard && (r != 0 || (m & 1ull))) ++m;
  if (m >> 53) {
    m >>= 1;
    ++e;
  }
  return __longlong_as_double(((long long)(1023 + e) << 52) | (long long)(m & ((1ull << 52) - 1ull)));
}

#endif  // TOPLOC_NEAREST_RATIO_CUH_
