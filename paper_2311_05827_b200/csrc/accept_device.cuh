// Device-side building blocks of the boundary-tensor codec (sm_100a).
//
// Data unit: an OCTET, eight consecutive fp32 values (32 bytes), moved with one 256-bit global
// load or store per thread.  Four neighbouring lanes (a QUAD) hold one pack group of 32 elements.
// Every fp32 operation that decides a code or a reconstructed value is an explicitly rounded
// intrinsic (__fmul_rn, __fadd_rn, __fsub_rn, __fdiv_rn): no FMA contraction, no flush to zero.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace accept {

constexpr int kAbsMax = 0, kMinMax = 1;
constexpr int kNearest = 0, kStochastic = 1;
constexpr int kInterleaved = 0, kBitplane = 1;

constexpr uint32_t kDevNonFinite = 1u, kDevBadHeader = 2u, kDevCopyTimeout = 4u;

// 1.5 * 2^23: adding it to |t| < 2^22 rounds t to an integer (ties to even, the fp32 adder's
// rounding) and leaves that integer in the low mantissa bits.
constexpr float kMagic = 12582912.0f;
constexpr uint32_t kMagicBits = 0x4B400000u;

// ----------------------------------------------------------------------------- memory access

// Every access of the data path to caller memory (input, output, stream, workspace records) goes through
// the helpers below.  In the normal build bounds_ok() is the constant true and they are plain loads and
// stores.  Built with -DACCEPT_BOUNDS_CHECK (a second library that only the tests load, standing in for a
// memory checker) each access is first compared with the byte ranges the host entry point registered for
// the call: one that falls outside, or a write into a read-only range, is COUNTED AND SKIPPED (a load
// returns zeros), never trapped, so the context stays usable and the host can read the tally.
#ifdef ACCEPT_BOUNDS_CHECK
constexpr int kMaxBoundsRanges = 8;
struct BoundsTable {
  unsigned long long lo[kMaxBoundsRanges], hi[kMaxBoundsRanges];  // [lo, hi) in bytes
  unsigned int writable[kMaxBoundsRanges];
  unsigned int n;
};
__device__ BoundsTable g_bounds;
__device__ unsigned int g_bounds_violations;      // accesses skipped since the last report
__device__ unsigned long long g_bounds_first[2];  // the first of them: address, size | write << 32

__device__ __noinline__ bool bounds_ok(const void* p, size_t bytes, bool write) {
  const unsigned long long a = (unsigned long long)p;
  for (unsigned int i = 0; i < g_bounds.n; ++i)
    if (a >= g_bounds.lo[i] && a + bytes <= g_bounds.hi[i] && (!write || g_bounds.writable[i])) return true;
  if (atomicAdd(&g_bounds_violations, 1u) == 0u) {
    g_bounds_first[0] = a;
    g_bounds_first[1] = (unsigned long long)bytes | ((unsigned long long)(write ? 1 : 0) << 32);
  }
  return false;
}
#else
__device__ __forceinline__ constexpr bool bounds_ok(const void*, size_t, bool) { return true; }
#endif

// read-only data (never written by the running kernel)
template <typename T>
__device__ __forceinline__ T ldg_c(const T* p) {
  if (!bounds_ok(p, sizeof(T), false)) return T{};
  return __ldg(p);
}
template <typename T>
__device__ __forceinline__ T ld_c(const T* p) {
  if (!bounds_ok(p, sizeof(T), false)) return T{};
  return *p;
}
template <typename T>
__device__ __forceinline__ void st_c(T* p, T v) {
  if (bounds_ok(p, sizeof(T), true)) *p = v;
}

__device__ __forceinline__ void ld_octet(const float* p, float (&v)[8]) {
  if (!bounds_ok(p, 32, false)) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.0f;
    return;
  }
  asm("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
      : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
      : "l"(p));
}

__device__ __forceinline__ void st_octet(float* p, const float (&v)[8]) {
  if (!bounds_ok(p, 32, true)) return;
  asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]),
               "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
               : "memory");
}

// ----------------------------------------------------------------------------- range statistic

// NaN-propagating max/min: a NaN anywhere in the chunk survives to the result, and so does Inf,
// so one test of the reduced value detects a non-finite chunk.
__device__ __forceinline__ float max_nan(float a, float b) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float min_nan(float a, float b) {
  float r;
  asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float r;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float min3_nan(float a, float b, float c) {
  float r;
  asm("min.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// hi = max|x| (ABSMAX) or max x (MINMAX); lo = min x (MINMAX only).
template <int RANGE>
struct Range {
  float hi, lo;
  __device__ __forceinline__ void init() {
    hi = (RANGE == kAbsMax) ? 0.0f : -__int_as_float(0x7f800000);
    lo = __int_as_float(0x7f800000);
  }
  __device__ __forceinline__ void add(float a) {
    if (RANGE == kAbsMax) {
      hi = max_nan(hi, fabsf(a));
    } else {
      hi = max_nan(hi, a);
      lo = min_nan(lo, a);
    }
  }
  __device__ __forceinline__ void add2(float a, float b) {
    if (RANGE == kAbsMax) {
      hi = max3_nan(hi, fabsf(a), fabsf(b));
    } else {
      hi = max3_nan(hi, a, b);
      lo = min3_nan(lo, a, b);
    }
  }
  __device__ __forceinline__ void merge(float ohi, float olo) {
    hi = max_nan(hi, ohi);
    if (RANGE == kMinMax) lo = min_nan(lo, olo);
  }
  // butterfly over the lanes of a warp; every lane ends with the warp's range
  __device__ __forceinline__ void warp_reduce() {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      float ohi = __shfl_xor_sync(0xffffffffu, hi, d);
      float olo = (RANGE == kMinMax) ? __shfl_xor_sync(0xffffffffu, lo, d) : 0.0f;
      merge(ohi, olo);
    }
  }
};

// Per-chunk quantizer constants derived from the range.
struct Scale {
  float s;     // side word: scaling factor
  float o;     // side word: offset (0 under ABSMAX)
  float inv;   // L / range, or 0 for a degenerate chunk
  float base;  // subtracted before scaling (MINMAX: lo)
  bool nonfinite;
};

__device__ __forceinline__ bool is_finite_bits(float a) {
  return (__float_as_uint(a) & 0x7f800000u) != 0x7f800000u;
}

// L / r rounded toward zero, from the round-to-nearest quotient: that one is above the true quotient
// exactly when q * r - L (one fused operation: the sign is exact) is positive, and the float below a
// positive q is the one with the next lower bit pattern.  q = inf (overflow) is returned as it is.
__device__ __forceinline__ float reciprocal_toward_zero(float L, float r) {
  const float q = __fdiv_rn(L, r);
  const bool above = is_finite_bits(q) && __fmaf_rn(q, r, -L) > 0.0f;
  return __uint_as_float(__float_as_uint(q) - (above ? 1u : 0u));
}

template <int K, int RANGE>
__device__ __forceinline__ Scale make_scale(float hi, float lo) {
  Scale sc;
  if (RANGE == kAbsMax) {
    const float L = (float)((1 << (K - 1)) - 1);
    sc.nonfinite = !is_finite_bits(hi);
    sc.s = __fdiv_rn(hi, L);
    sc.inv = reciprocal_toward_zero(L, hi);  // hi * inv <= L, so |x * inv| <= L and nothing needs a clamp
    sc.base = 0.0f;
    sc.o = 0.0f;
    if (sc.nonfinite || !(hi > 0.0f) || !is_finite_bits(sc.inv)) { sc.s = 0.0f; sc.inv = 0.0f; }
  } else {
    const float L = (float)((1 << K) - 1);
    const float r = __fsub_rn(hi, lo);
    sc.nonfinite = !is_finite_bits(hi) || !is_finite_bits(lo) || !is_finite_bits(r);
    sc.s = __fdiv_rn(r, L);
    sc.inv = reciprocal_toward_zero(L, r);
    sc.base = lo;
    sc.o = (lo == 0.0f) ? 0.0f : lo;  // -0 is written as +0
    if (sc.nonfinite) { sc.s = 0.0f; sc.inv = 0.0f; sc.base = 0.0f; sc.o = 0.0f; }
    else if (!(r > 0.0f) || !is_finite_bits(sc.inv)) { sc.s = 0.0f; sc.inv = 0.0f; }
  }
  return sc;
}

// ----------------------------------------------------------------------------- uniform numbers (Eq. 7)

// 32-bit finaliser of MurmurHash3.
__device__ __forceinline__ uint32_t fmix32(uint32_t h) {
  h ^= h >> 16;
  h *= 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}

// Four neighbouring counters (4j .. 4j+3) share one hash: counter 4j+m takes the hashed word times
// kLaneMul[m] (odd constants, so each is a bijection of the word; m = 0 takes it as it is).  The
// integer hash runs on the half-rate ALU pipe and is what bounds stochastic rounding; shared by
// four elements it costs two ALU instructions per element, the extra products run on the FMA pipe.
__device__ __forceinline__ uint32_t lane_word(uint32_t h, int m) {
  return m == 0 ? h : h * (m == 1 ? 0x9E3779B1u : (m == 2 ? 0x85EBCA77u : 0xC2B2AE3Du));
}

struct Rng {
  uint32_t seed_lo, seed_hi;
  // key for all quads that share the upper 32 bits of their quad index; the constant keeps
  // seed 0 / quad 0 off the fixed point fmix32(0) = 0
  __device__ __forceinline__ uint32_t key(uint32_t quad_hi) const {
    return fmix32(quad_hi ^ seed_lo ^ 0x9E3779B9u) ^ seed_hi;
  }
  // hashed word of a quad
  __device__ __forceinline__ static uint32_t quad_hash(uint32_t quad_lo, uint32_t key) { return fmix32(quad_lo ^ key); }
  // 32 random bits of any counter (the octet path below shares the quad hashes instead)
  __device__ __forceinline__ uint32_t word(uint64_t ctr) const {
    const uint64_t quad = ctr >> 2;
    const uint32_t h = quad_hash((uint32_t)quad, key((uint32_t)(quad >> 32)));
    const int m = (int)(ctr & 3);
    return m == 0 ? h : h * (m == 1 ? 0x9E3779B1u : (m == 2 ? 0x85EBCA77u : 0xC2B2AE3Du));
  }
};

// What a thread works out once for all the octets it quantizes stochastically: the quad index and
// key of its first counter, the counter's position in its quad (the same for every octet, octets
// start 8 apart) and whether the low word of the quad index stays clear of a wrap over the thread's
// whole span.
struct RngThread {
  uint64_t ctr_first;
  uint32_t quad_lo, key;
  int off;    // ctr_first & 3
  bool fast;
  // span = distance, in counters, from the thread's first counter to one past its last
  __device__ __forceinline__ void init(const Rng& rng, uint64_t ctr, uint32_t span) {
    ctr_first = ctr;
    const uint64_t quad = ctr >> 2;
    quad_lo = (uint32_t)quad;
    key = rng.key((uint32_t)(quad >> 32));
    off = (int)(ctr & 3);
    fast = quad_lo <= 0xFFFFFFFFu - (span / 4 + 2);
  }
};

// ----------------------------------------------------------------------------- quantize

// NEAREST.  Returns the fp32 bit pattern of (kMagic + u), u the unsigned stored code: its byte 0 is u.
template <int K, int RANGE>
__device__ __forceinline__ uint32_t quantize_nearest_word(float x, const Scale& sc) {
  constexpr int ZP = (RANGE == kAbsMax) ? (1 << (K - 1)) : 0;
  constexpr float kMagicZ = kMagic + (float)ZP;  // exact; even, so ties still go to even codes
  const float d = (RANGE == kAbsMax) ? x : __fsub_rn(x, sc.base);
  const float t = __fmul_rn(d, sc.inv);
  // |t| <= L (the reciprocal is rounded toward zero): the rounded code cannot leave [zp-L, zp+L], no clamp needed
  return __float_as_uint(__fadd_rn(t, kMagicZ));
}

// STOCHASTIC (Eq. 7) in exact fixed point.  With r = h >> 8 (U = r * 2^-24) and n = floor(t):
//   U < t - n   <=>   r < ceil((t - n) * 2^24)          (r is an integer)
// so  n + [U < t - n] = floor((ceil(t * 2^24) + (2^24 - 1 - r)) / 2^24), and 2^24 - 1 - r = (~h) >> 8.
// Adding zero_point << 24 makes the sum non-negative; byte 3 of the 32-bit sum is the stored code u.
// |t| never exceeds the top level L (the reciprocal is rounded toward zero, see make_scale), so the
// sum stays below 2^32 and the code cannot reach L + 1; the low side cannot pass the lowest code.
template <int K, int RANGE>
__device__ __forceinline__ uint32_t quantize_stochastic_word(float x, const Scale& sc, uint32_t h) {
  constexpr int ZP = (RANGE == kAbsMax) ? (1 << (K - 1)) : 0;
  const float d = (RANGE == kAbsMax) ? x : __fsub_rn(x, sc.base);
  const float t = __fmul_rn(d, sc.inv);  // |t| <= L: inv is rounded toward zero
  const float t24 = __fmul_rn(t, 16777216.0f);  // exact scaling
  const uint32_t tc = (RANGE == kAbsMax) ? (uint32_t)__float2int_ru(t24) : __float2uint_ru(t24);
  return tc + ((uint32_t)ZP << 24) + ((~h) >> 8);
}

// The stored code of one element (any-shape path).
template <int K, int RANGE, int ROUND>
__device__ __forceinline__ uint32_t quantize_code(float x, const Scale& sc, uint32_t h) {
  if (ROUND == kNearest) return quantize_nearest_word<K, RANGE>(x, sc) & 0xFFu;
  return quantize_stochastic_word<K, RANGE>(x, sc, h) >> 24;
}

// byte BYTE of four words -> one word
template <int BYTE>
__device__ __forceinline__ uint32_t pack_bytes(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3) {
  constexpr uint32_t sel = (uint32_t)BYTE | ((uint32_t)(BYTE + 4) << 4);
  const uint32_t p01 = __byte_perm(b0, b1, sel);
  const uint32_t p23 = __byte_perm(b2, b3, sel);
  return __byte_perm(p01, p23, 0x5410);
}

// The same with the COMPLEMENT of the element's random word passed in: (~g) >> 8 is what Eq. 7's fixed
// point form adds, and the complement of a lane word costs nothing extra: ~(h * M) = (-h) * M - 1
// is one multiply-add like h * M itself, so the element is left with one add and one shift-add.
template <int K, int RANGE>
__device__ __forceinline__ uint32_t quantize_stochastic_word_not(float x, const Scale& sc, uint32_t g_not) {
  constexpr int ZP = (RANGE == kAbsMax) ? (1 << (K - 1)) : 0;
  const float d = (RANGE == kAbsMax) ? x : __fsub_rn(x, sc.base);
  const float t = __fmul_rn(d, sc.inv);  // |t| <= L: inv is rounded toward zero
  const float t24 = __fmul_rn(t, 16777216.0f);  // exact scaling
  const uint32_t tc = (RANGE == kAbsMax) ? (uint32_t)__float2int_ru(t24) : __float2uint_ru(t24);
  // (ZP : g_not) >> 8 = (g_not >> 8) + (ZP << 24): the zero point rides in on the funnel shift
  return tc + __funnelshift_r(g_not, (uint32_t)ZP, 8);
}

// ~lane_word(h, m), from h_not = ~h and h_neg = -h
__device__ __forceinline__ uint32_t lane_word_not(uint32_t h_not, uint32_t h_neg, int m) {
  return m == 0 ? h_not : h_neg * (m == 1 ? 0x9E3779B1u : (m == 2 ? 0x85EBCA77u : 0xC2B2AE3Du)) + 0xFFFFFFFFu;
}

// Stochastic codes of an octet whose first counter sits at position OFF of its quad; quad_lo/key
// address that quad.
// (h[p] = hashed word of the p-th quad the octet touches: two quads when OFF = 0, else three)
template <int K, int RANGE, int OFF>
__device__ __forceinline__ void quantize_octet_hashed(const float (&v)[8], const Scale& sc, const uint32_t (&h)[3],
                                                      uint32_t (&b)[8]) {
  constexpr int NQ = (OFF == 0) ? 2 : 3;
  uint32_t h_not[NQ], h_neg[NQ];
#pragma unroll
  for (int p = 0; p < NQ; ++p) {
    h_not[p] = ~h[p];
    h_neg[p] = 0u - h[p];
  }
#pragma unroll
  for (int e = 0; e < 8; ++e)
    b[e] = quantize_stochastic_word_not<K, RANGE>(v[e], sc,
                                                  lane_word_not(h_not[(e + OFF) >> 2], h_neg[(e + OFF) >> 2], (e + OFF) & 3));
}

template <int K, int RANGE, int OFF>
__device__ __forceinline__ void quantize_octet_stochastic(const float (&v)[8], const Scale& sc, uint32_t quad_lo,
                                                          uint32_t key, uint32_t (&b)[8]) {
  constexpr int NQ = (OFF == 0) ? 2 : 3;
  uint32_t h[3] = {0u, 0u, 0u};
#pragma unroll
  for (int p = 0; p < NQ; ++p) h[p] = Rng::quad_hash(quad_lo + p, key);
  quantize_octet_hashed<K, RANGE, OFF>(v, sc, h, b);
}

// Quantizes an octet.  xlo holds the codes of elements 0..3 one per byte, xhi those of 4..7.
// delta = distance of the octet's first counter from the thread's first one (a multiple of 8).
template <int K, int RANGE, int ROUND>
__device__ __forceinline__ void quantize_octet(const float (&v)[8], const Scale& sc, const Rng& rng,
                                               const RngThread& rt, uint32_t delta, uint32_t& xlo, uint32_t& xhi) {
  uint32_t b[8];
  if (ROUND == kStochastic) {
    if (rt.fast) {
      const uint32_t q0 = rt.quad_lo + delta / 4;  // delta is a multiple of 8
      if (rt.off == 0) quantize_octet_stochastic<K, RANGE, 0>(v, sc, q0, rt.key, b);
      else if (rt.off == 1) quantize_octet_stochastic<K, RANGE, 1>(v, sc, q0, rt.key, b);
      else if (rt.off == 2) quantize_octet_stochastic<K, RANGE, 2>(v, sc, q0, rt.key, b);
      else quantize_octet_stochastic<K, RANGE, 3>(v, sc, q0, rt.key, b);
    } else {  // the quad index's low word (or the counter itself) wraps somewhere in this thread's span
#pragma unroll
      for (int e = 0; e < 8; ++e) b[e] = quantize_stochastic_word<K, RANGE>(v[e], sc, rng.word(rt.ctr_first + delta + e));
    }
    xlo = pack_bytes<3>(b[0], b[1], b[2], b[3]);
    xhi = pack_bytes<3>(b[4], b[5], b[6], b[7]);
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) b[e] = quantize_nearest_word<K, RANGE>(v[e], sc);
    xlo = pack_bytes<0>(b[0], b[1], b[2], b[3]);
    xhi = pack_bytes<0>(b[4], b[5], b[6], b[7]);
  }
}

// Quantizes the R octets of a thread; round r starts r * stride counters (a multiple of 8) after the
// thread's first one.  Where a thread's counters sit in their quads, and whether the quad index
// wraps inside the thread's span, is the same for all R octets (and, but for the wrap, for every
// thread of the launch): the case is chosen once here and the octets are coded without further
// branches.  No shuffles inside: threads may take different cases.
template <int K, int RANGE, int R, int OFF>
__device__ __forceinline__ void quantize_rounds_stochastic(const float (&v)[R][8], const Scale& sc, const RngThread& rt,
                                                           uint32_t stride, uint32_t (&xlo)[R], uint32_t (&xhi)[R]) {
#pragma unroll
  for (int r = 0; r < R; ++r) {
    uint32_t b[8];
    quantize_octet_stochastic<K, RANGE, OFF>(v[r], sc, rt.quad_lo + (stride * r) / 4, rt.key, b);
    xlo[r] = pack_bytes<3>(b[0], b[1], b[2], b[3]);
    xhi[r] = pack_bytes<3>(b[4], b[5], b[6], b[7]);
  }
}

template <int K, int RANGE, int ROUND, int R>
__device__ __forceinline__ void quantize_rounds(const float (&v)[R][8], const Scale& sc, const Rng& rng, const RngThread& rt,
                                                uint32_t stride, uint32_t (&xlo)[R], uint32_t (&xhi)[R]) {
  if (ROUND == kNearest) {
#pragma unroll
    for (int r = 0; r < R; ++r) quantize_octet<K, RANGE, kNearest>(v[r], sc, rng, rt, 0u, xlo[r], xhi[r]);
    return;
  }
  switch (rt.fast ? rt.off : 4) {
    case 0: quantize_rounds_stochastic<K, RANGE, R, 0>(v, sc, rt, stride, xlo, xhi); break;
    case 1: quantize_rounds_stochastic<K, RANGE, R, 1>(v, sc, rt, stride, xlo, xhi); break;
    case 2: quantize_rounds_stochastic<K, RANGE, R, 2>(v, sc, rt, stride, xlo, xhi); break;
    case 3: quantize_rounds_stochastic<K, RANGE, R, 3>(v, sc, rt, stride, xlo, xhi); break;
    default:  // the quad index's low word (or the counter itself) wraps somewhere in this thread's span
#pragma unroll
      for (int r = 0; r < R; ++r) {
        uint32_t b[8];
#pragma unroll
        for (int e = 0; e < 8; ++e)
          b[e] = quantize_stochastic_word<K, RANGE>(v[r][e], sc, rng.word(rt.ctr_first + stride * r + e));
        xlo[r] = pack_bytes<3>(b[0], b[1], b[2], b[3]);
        xhi[r] = pack_bytes<3>(b[4], b[5], b[6], b[7]);
      }
      break;
  }
}

// ----------------------------------------------------------------------------- bit permutations

// Exchanges the bits selected by m with the bits s places above them.
__device__ __forceinline__ uint32_t delta_swap(uint32_t x, uint32_t m, int s) {
  const uint32_t t = ((x >> s) ^ x) & m;
  return x ^ t ^ (t << s);
}

// 4 x 8 bit-matrix transpose inside a word, its own inverse.
//   plane form:  bit 8*j + e       = digit j (0..3) of the code of element e (0..7)
//   nibble form: bit 8*b + 4*a + j = digit j of the code of element 4*a + b
// i.e. byte b of the nibble form holds code b in its low and code 4+b in its high nibble.
__device__ __forceinline__ uint32_t planes_nibbles(uint32_t x) {
  x = delta_swap(x, 0x0000CCCCu, 14);  // index bit 4 <-> index bit 1
  x = delta_swap(x, 0x00AA00AAu, 7);   // index bit 3 <-> index bit 0
  return x;
}

// 4 x 4 byte transpose across the four lanes of a quad, its own inverse: before, lane q holds
// bytes [a_q0 a_q1 a_q2 a_q3]; after, lane q holds [a_0q a_1q a_2q a_3q].  All 32 lanes must call.
__device__ __forceinline__ uint32_t quad_transpose(uint32_t v, int lane) {
  uint32_t r = __shfl_xor_sync(0xffffffffu, v, 2);
  v = __byte_perm(v, r, (lane & 2) ? 0x3276 : 0x5410);
  r = __shfl_xor_sync(0xffffffffu, v, 1);
  v = __byte_perm(v, r, (lane & 1) ? 0x3715 : 0x6240);
  return v;
}

// codes 0..3 / 4..7 (one per byte, < 16) -> byte b = code b | code(4+b) << 4
__device__ __forceinline__ uint32_t merge_nibbles(uint32_t xlo, uint32_t xhi) { return xlo | (xhi << 4); }

// ----------------------------------------------------------------------------- dequantize

template <int K, int RANGE>
__device__ __forceinline__ float dequantize_code(uint32_t u, float s, float o) {
  constexpr int ZP = (RANGE == kAbsMax) ? (1 << (K - 1)) : 0;
  // kMagicBits | u is the float kMagic + u; subtracting kMagic + zp leaves the integer u - zp, exactly
  const float g = __fsub_rn(__uint_as_float(kMagicBits | u), kMagic + (float)ZP);
  if (RANGE == kAbsMax) return __fmul_rn(g, s);
  return __fadd_rn(__fmul_rn(g, s), o);
}

}  // namespace accept
