// Exact sums of fp32 values on the device.
//
// Eq. 3 (B^T x) and Eq. 5 (the mean of B alpha - x) are sums over the whole tensor, and the side words
// they produce travel in the stream.  A floating-point sum depends on the order of its terms, and the
// order on a GPU is a property of the launch, not of the method; so the sums here are taken without
// rounding and rounded once, to the nearest double, at the very end.  The result is then a function of
// the multiset of values alone.
//
// Representation ("wide sum"): the integer T = sum / 2^-149 (every fp32 value is a whole multiple of
// 2^-149) held as kAccLimbs digits of 32 bits, T = sum_i limb[i] * 2^(32 i), each digit kept in a
// signed 64-bit word whose carry is propagated only when the sum is read.  Adding to it is therefore a
// handful of independent 64-bit integer atomic adds, which commute: the final digits do not depend on
// the order in which threads and blocks arrive.
//
// Fast path: a thread adds its values into ordinary double accumulators.  That is exact as long as every
// value is a whole multiple of 2^q and the running sum stays below 2^(q+53); with at most
// kFlushElems = 2^6 values between two flushes this holds for all values with
//     2^(q+23) <= |x| < 2^(q+47)   or   x = 0                                   (the WINDOW, 24 octaves)
// (a normal fp32 value of magnitude >= 2^(q+23) has its last mantissa bit at 2^q or above).  The window
// is placed around the magnitudes the data is expected to have; at a flush the accumulator is an integer
// number of units 2^q below 2^53, converted exactly to int64.  Values outside the window (and they may be
// anything: subnormals, 3e38) skip the double accumulators and go straight into the wide sum, mantissa
// and exponent taken apart with integer operations.  Both paths are exact, so where the window sits
// changes the speed, never the result.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "accept_device.cuh"

namespace accept {

constexpr int kAccLimbs = 12;      // 384 bits: 277 for the largest fp32 value in units of 2^-149, the rest for the count
constexpr int kFlushShift = 6;     // a thread adds at most 2^6 values between two flushes
constexpr int kFlushElems = 1 << kFlushShift;
constexpr int kWindowTopBits = 53 - kFlushShift;  // top of the window: 2^(q + 47)
constexpr int kPushFlushes = 32;   // a thread's int64 running sum (below 2^53 per flush) is pushed after this many
                                   // flushes at the latest: 2^58 per lane, 2^63 per warp

// Where the window sits and how accumulators turn into units of 2^q.
struct ExactWindow {
  float top;         // in-window values have |x| < top = 2^(q+47)
  uint32_t ylow;     // 2 * bits(bottom) - 2 with bottom = 2^(q+23): see WindowCheck
  uint32_t top_bits, bottom_bits;
  int pos;           // q + 149: bit position of one unit in the wide sum
  double to_units;   // 2^-q
};

// Window for data whose magnitudes are expected around `scale` (any value; 0, NaN and Inf fall back to 1):
// the top is 2^9 times the binade of scale, the bottom 2^24 below that.
__device__ inline ExactWindow make_window(float scale) {
  // binade of the scale from its exponent field (subnormal scales count as 2^-126)
  int e = 0;
  if (scale > 0.0f && is_finite_bits(scale)) {
    const int field = (int)((__float_as_uint(scale) >> 23) & 0xFFu);
    e = (field ? field : 1) - 127;
  }
  int e_top = e + 9;
  if (e_top > 127) e_top = 127;
  if (e_top < -126 + 24) e_top = -126 + 24;  // keeps the bottom a normal number
  const int q = e_top - kWindowTopBits;
  ExactWindow w;
  w.top_bits = (uint32_t)(e_top + 127) << 23;          // 2^e_top
  w.bottom_bits = (uint32_t)(e_top - 24 + 127) << 23;  // 2^(e_top - 24)
  w.top = __uint_as_float(w.top_bits);
  w.ylow = 2u * w.bottom_bits - 2u;
  w.pos = q + 149;
  w.to_units = __hiloint2double((1023 - q) << 20, 0);  // 2^-q
  return w;
}

// 2 * v - 2 (mod 2^32) as one integer multiply-add, which the FMA pipe takes (the ALU pipe is the busy one)
__device__ __forceinline__ uint32_t twice_minus_two(uint32_t v) {
  uint32_t r;
  asm("mad.lo.u32 %0, %1, 2, 0xFFFFFFFE;" : "=r"(r) : "r"(v));
  return r;
}

struct WindowCheck {
  float amax;
  uint32_t ymin;
  __device__ __forceinline__ void init() { amax = 0.0f; ymin = 0xFFFFFFFFu; }
  __device__ __forceinline__ void add2(float a, float b) {
    amax = max3_nan(amax, fabsf(a), fabsf(b));
    ymin = __vimin3_u32(ymin, twice_minus_two(__float_as_uint(a)), twice_minus_two(__float_as_uint(b)));
  }
  __device__ __forceinline__ bool ok(const ExactWindow& w) const { return amax < w.top && ymin >= w.ylow; }
};

__device__ __forceinline__ bool in_window(const ExactWindow& w, float x) {
  const uint32_t u = __float_as_uint(x) & 0x7FFFFFFFu;
  return u == 0u || (u >= w.bottom_bits && u < w.top_bits);
}

__device__ __forceinline__ void limb_add(long long* limb, long long v) {
  atomicAdd(reinterpret_cast<unsigned long long*>(limb), static_cast<unsigned long long>(v));
}

// limbs += v * 2^pos (units of 2^-149), 0 <= pos < 256, any int64 v: three pieces below 2^33 each.
__device__ __forceinline__ void wide_add_int64(long long* limbs, long long v, int pos) {
  if (v == 0) return;
  const int L = pos >> 5, sh = pos & 31;
  const uint64_t lo = (uint64_t)(uint32_t)v << sh;               // < 2^63
  const long long hi = (long long)(int32_t)(v >> 32) * (1ll << sh);  // |.| < 2^62, weight 2^(32 (L+1))
  limb_add(limbs + L, (long long)(lo & 0xFFFFFFFFull));
  limb_add(limbs + L + 1, (long long)(lo >> 32) + (long long)((uint64_t)hi & 0xFFFFFFFFull));
  limb_add(limbs + L + 2, hi >> 32);
}

// limbs += x (negate: -x), mantissa and exponent taken apart; returns false for NaN/Inf (nothing added).
__device__ __forceinline__ bool wide_add_float(long long* limbs, float x, bool negate) {
  const uint32_t bits = __float_as_uint(x);
  const uint32_t E = (bits >> 23) & 0xFFu, frac = bits & 0x7FFFFFu;
  if (E == 255u) return false;
  const uint32_t m = E ? (frac | 0x800000u) : frac;  // x = m * 2^(E-150), or m * 2^-149 when subnormal
  if (m == 0u) return true;
  const int pos = E ? (int)E - 1 : 0;
  const int L = pos >> 5, sh = pos & 31;
  const uint64_t t = (uint64_t)m << sh;  // < 2^55
  const bool neg = ((bits >> 31) != 0u) != negate;
  const long long p0 = (long long)(t & 0xFFFFFFFFull), p1 = (long long)(t >> 32);
  limb_add(limbs + L, neg ? -p0 : p0);
  if (p1) limb_add(limbs + L + 1, neg ? -p1 : p1);
  return true;
}

// Sum of an int64 over the lanes of a warp (every lane gets it); the caller keeps |v| below 2^58.
__device__ __forceinline__ long long warp_sum_int64(long long v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}

// Carries propagated: digits 0..kAccLimbs-2 end in [0, 2^32), the last one keeps the sign.
__device__ __forceinline__ void wide_normalise(long long (&limbs)[kAccLimbs]) {
  long long carry = 0;
#pragma unroll
  for (int i = 0; i < kAccLimbs - 1; ++i) {
    const long long t = limbs[i] + carry;
    limbs[i] = (long long)((uint64_t)t & 0xFFFFFFFFull);
    carry = t >> 32;  // arithmetic shift: floor division
  }
  limbs[kAccLimbs - 1] += carry;
}

// The wide sum (digits with pending carries) rounded to the nearest double, ties to even.
// d: scratch of kAccLimbs + 1 words that may be indexed by a variable: give it shared memory (an array of
// the thread's own would live in local memory, whose misses cost microseconds in a block that runs alone).
__device__ inline double wide_to_double(const long long* lazy, uint32_t* d) {
  long long limbs[kAccLimbs];
#pragma unroll
  for (int i = 0; i < kAccLimbs; ++i) limbs[i] = lazy[i];
  wide_normalise(limbs);
  const bool negative = limbs[kAccLimbs - 1] < 0;
  if (negative) {
    // magnitude of a two's complement number: complement every digit, add one
    uint64_t carry = 1;
#pragma unroll
    for (int i = 0; i < kAccLimbs - 1; ++i) {
      const uint64_t t = (uint64_t)(~(uint32_t)limbs[i]) + carry;
      d[i] = (uint32_t)t;
      carry = t >> 32;
    }
    d[kAccLimbs - 1] = (uint32_t)((uint64_t)(~limbs[kAccLimbs - 1]) + carry);
  } else {
#pragma unroll
    for (int i = 0; i < kAccLimbs; ++i) d[i] = (uint32_t)limbs[i];
  }
  d[kAccLimbs] = 0u;
  int hi = kAccLimbs - 1;
  while (hi >= 0 && d[hi] == 0u) --hi;
  if (hi < 0) return 0.0;
  const int top = 32 * hi + 31 - __clz((int)d[hi]);  // highest set bit
  double r;
  if (top <= 52) {
    r = ldexp((double)((uint64_t)d[0] | ((uint64_t)d[1] << 32)), -149);
  } else {
    const int low = top - 52;  // mantissa = bits [low, top]
    const int w = low >> 5, off = low & 31;
    // 96 bits starting at digit w, shifted down by off: the low 53 bits are the mantissa
    const uint64_t a = (uint64_t)d[w] | ((uint64_t)d[w + 1] << 32);
    const uint64_t b = (w + 2 <= kAccLimbs) ? (uint64_t)d[w + 2] : 0ull;
    uint64_t mant = off ? ((a >> off) | (b << (64 - off))) : a;
    mant &= (1ull << 53) - 1ull;
    const int g = low - 1;  // guard bit
    const bool guard = (d[g >> 5] >> (g & 31)) & 1u;
    bool sticky = (d[g >> 5] & ((1u << (g & 31)) - 1u)) != 0u;
    for (int i = (g >> 5) - 1; i >= 0; --i) sticky = sticky || d[i] != 0u;
    if (guard && (sticky || (mant & 1ull))) ++mant;  // 2^53 is still exact in a double
    r = ldexp((double)mant, low - 149);
  }
  return negative ? -r : r;
}

}  // namespace accept
