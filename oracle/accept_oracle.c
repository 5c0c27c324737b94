/*
 * accept_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded CPU statement of the AccEPT bit-level compression scheme
 * (Sec. 3.3 "Bit-level Fast Compression Scheme", Sec. 3.4 "Bit-level Fast Decompression Scheme"),
 * written from the paper, sharing no code, header or table with the CUDA library.  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * The method is an encoding, so this file takes the paper's steps in the paper's order, one
 * element at a time, in fp32 (the paper's tensors and side words are 32-bit floats, Sec. 2.2 and
 * "Transmission Data Comparison"); every fp32 operation is rounded on its own (build with
 * -ffp-contract=off, no fast-math).
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *   - one range per chunk of C consecutive values of the vectorised tensor; C >= N is the paper's
 *     per-tensor range ("Backward Quantizer": c = max|g|);
 *   - the division by the scaling factor is computed as a product with inv = L/c rounded toward zero
 *     (one division per chunk; rounded down so that |x * inv| <= L as in exact arithmetic); pinned
 *     against true division in the tests;
 *   - nearest rounding is IEEE round-half-to-even;
 *   - the uniform generator of Eq. 7 is counter based (MurmurHash3's 32-bit finaliser, see oracle_rng_hash below: one hash per four counters); U has 24 bits; pr = t - floor(t) and the test
 *     U < pr are exact;
 *   - bit order in a packed word is LSB first (element t of a group <-> bit t).  The paper's only
 *     worked example, (00110110)_2 = 54, fixes the value of a word, not which element is the MSB:
 *     PARITY UNPINNED for the bit order and for which elements share a word (the figure that
 *     shows it is not in the text);
 *   - a chunk whose range is 0, or so small that inv overflows, is degenerate: s = 0, all codes the
 *     zero point; a chunk with a NaN/Inf (or an overflowing min/max range) is written the same
 *     way and flagged.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAGIC 0x54504341u /* "ACPT" */
#define ORACLE_VERSION 1u

enum { RANGE_ABSMAX = 0, RANGE_MINMAX = 1 };
enum { ROUND_NEAREST = 0, ROUND_STOCHASTIC = 1 };
enum { LAYOUT_INTERLEAVED = 0, LAYOUT_BITPLANE = 1 };

/* ---------------------------------------------------------------- sizes (Eq. 8 and the text around it) */

static uint64_t n_chunks(uint64_t n, uint32_t C) { return (n + C - 1) / C; }

/* Payload starts after the 32-byte header and one {s,o} pair per chunk, rounded up to 16 bytes. */
uint64_t oracle_payload_offset(uint64_t n, uint32_t C) {
  uint64_t off = 32 + 8 * n_chunks(n, C);
  return (off + 15) / 16 * 16;
}

/* k bits per element, elements padded to whole groups of 32 ("ceil(n/8)" of Eq. 8, with words of 32). */
uint64_t oracle_payload_bytes(uint64_t n, uint32_t k) { return 4 * (uint64_t)k * ((n + 31) / 32); }

uint64_t oracle_stream_bytes(uint64_t n, uint32_t C, uint32_t k) {
  return oracle_payload_offset(n, C) + oracle_payload_bytes(n, k);
}

/* ---------------------------------------------------------------- uniform numbers for Eq. 7 */

/* MurmurHash3 32-bit finaliser (public-domain algorithm by A. Appleby), restated. */
static uint32_t fmix32(uint32_t h) {
  h ^= h >> 16;
  h *= 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}

/* 32 random bits for counter ctr under seed.  Counters 4j .. 4j+3 share the hash of their quad
 * index j; counter 4j+m multiplies it by the m-th of four odd constants (1 for m = 0), each a
 * bijection of the 32-bit word. */
uint32_t oracle_rng_hash(uint64_t seed, uint64_t ctr) {
  static const uint32_t lane_mul[4] = {1u, 0x9E3779B1u, 0x85EBCA77u, 0xC2B2AE3Du};
  uint64_t quad = ctr >> 2;
  /* the constant keeps seed 0, quad 0 off the fixed point fmix32(0) = 0 */
  uint32_t inner = fmix32((uint32_t)(quad >> 32) ^ (uint32_t)seed ^ 0x9E3779B9u);
  uint32_t h = fmix32((uint32_t)quad ^ inner ^ (uint32_t)(seed >> 32));
  return h * lane_mul[ctr & 3];
}

/* out[i] = oracle_rng_hash(seed, ctr0 + i): the same words in bulk, for the statistical pins. */
void oracle_rng_fill(uint64_t seed, uint64_t ctr0, uint64_t n, uint32_t* out) {
  for (uint64_t i = 0; i < n; ++i) out[i] = oracle_rng_hash(seed, ctr0 + i);
}

/* U in [0,1) on a grid of 2^-24: the top 24 random bits. */
double oracle_rng_uniform(uint64_t seed, uint64_t ctr) {
  return (double)(oracle_rng_hash(seed, ctr) >> 8) / 16777216.0;
}

/* ---------------------------------------------------------------- quantizer ("Backward Quantizer", Eq. 7) */

/*
 * Quantizes one chunk x[0..valid) to unsigned codes u[0..valid) and writes the side words
 * meta[0] = s (scaling factor), meta[1] = o (offset).  i0 is the index of x[0] in the whole
 * tensor (the random-number counter).  Returns 1 if the chunk was non-finite.
 */
/* L / r rounded TOWARD ZERO (inf if the quotient overflows).  The division by the scaling factor s = r / L
 * is computed as a product with this reciprocal; in the paper's exact arithmetic |g / s| never exceeds L, and
 * rounding the reciprocal down keeps that true in fp32: r * inv <= L, hence fl(d * inv) <= L for every
 * d <= r, so no value has to be clamped back into the code range.  The round-to-nearest quotient is above
 * the true one exactly when its (exact, in double) product with r is above L. */
float oracle_reciprocal_toward_zero(float L, float r) {
  float q = L / r;
  if (isfinite(q) && (double)q * (double)r > (double)L) q = nextafterf(q, 0.0f);
  return q;
}

static int quantize_chunk(const float* x, uint32_t valid, uint32_t k, int range, int round_mode,
                          uint64_t seed, uint64_t rng_offset, uint64_t i0, uint8_t* u,
                          float* meta) {
  int nonfinite = 0;
  float s, o, inv, base;
  int qmin, qmax, zero_point;

  for (uint32_t i = 0; i < valid; ++i)
    if (!isfinite(x[i])) nonfinite = 1;

  if (range == RANGE_ABSMAX) {
    /* c = max|g|, s = c / (2^(k-1) - 1); codes in [-2^(k-1), 2^(k-1)-1], shifted by +2^(k-1). */
    float c = 0.0f;
    for (uint32_t i = 0; i < valid; ++i)
      if (fabsf(x[i]) > c) c = fabsf(x[i]);
    float L = (float)((1 << (k - 1)) - 1);
    s = c / L;
    inv = oracle_reciprocal_toward_zero(L, c);
    base = 0.0f;
    o = 0.0f;
    zero_point = 1 << (k - 1);
    qmin = -(1 << (k - 1));
    qmax = (1 << (k - 1)) - 1;
    if (nonfinite || !(c > 0.0f) || !isfinite(inv)) { s = 0.0f; inv = 0.0f; }
  } else {
    float lo = x[0], hi = x[0];
    for (uint32_t i = 1; i < valid; ++i) {
      if (x[i] < lo) lo = x[i];
      if (x[i] > hi) hi = x[i];
    }
    float L = (float)((1 << k) - 1);
    float r = hi - lo;
    if (!nonfinite && !isfinite(r)) nonfinite = 1; /* range overflow */
    s = r / L;
    inv = oracle_reciprocal_toward_zero(L, r);
    base = lo;
    o = lo + 0.0f; /* -0 becomes +0 */
    zero_point = 0;
    qmin = 0;
    qmax = (1 << k) - 1;
    if (nonfinite) { s = 0.0f; inv = 0.0f; base = 0.0f; o = 0.0f; }
    else if (!(r > 0.0f) || !isfinite(inv)) { s = 0.0f; inv = 0.0f; }
  }
  meta[0] = s;
  meta[1] = o;

  for (uint32_t i = 0; i < valid; ++i) {
    int q;
    if (nonfinite) {
      q = 0;
    } else {
      float d = (range == RANGE_ABSMAX) ? x[i] : (x[i] - base);
      float t = d * inv;
      if (round_mode == ROUND_NEAREST) {
        q = (int)rintf(t); /* default rounding mode: to nearest, ties to even */
      } else {
        /* Eq. 7: floor(t) with probability 1-pr, floor(t)+1 with probability pr = t - floor(t).
         * pr is a real number in the paper: it is held in double here, where the difference of an
         * fp32 value and its floor cannot cross a multiple of 2^-24, so U < pr is decided exactly. */
        double f = floor((double)t);
        double pr = (double)t - f;
        double U = oracle_rng_uniform(seed, rng_offset + i0 + i);
        q = (int)f + ((U < pr) ? 1 : 0);
      }
      if (q < qmin) q = qmin;
      if (q > qmax) q = qmax;
    }
    u[i] = (uint8_t)(q + zero_point);
  }
  return nonfinite;
}

/*
 * Codes and side words of the whole tensor, unpacked: codes[n] (one byte per element),
 * meta[2*M].  Returns 1 if any chunk was non-finite, else 0.
 */
int oracle_quantize(const float* x, uint64_t n, uint32_t C, uint32_t k, int range, int round_mode,
                    uint64_t seed, uint64_t rng_offset, uint8_t* codes, float* meta) {
  int flags = 0;
  uint64_t M = n_chunks(n, C);
  for (uint64_t m = 0; m < M; ++m) {
    uint64_t i0 = m * C;
    uint32_t valid = (uint32_t)((n - i0 < C) ? (n - i0) : C);
    flags |= quantize_chunk(x + i0, valid, k, range, round_mode, seed, rng_offset, i0, codes + i0,
                            meta + 2 * m);
  }
  return flags;
}

/* ---------------------------------------------------------------- encoders */

/*
 * Packs the codes of one chunk into words[0 .. ceil(valid/32)*k), which must be zero on entry.
 * INTERLEAVED ("Backward Encoder": two 4-bit codes per byte; k = 8 sent as is): element t takes
 * bits [k*t, k*t+k) of the chunk's bit string.
 * BITPLANE ("Forward Encoder": the one-bit values of consecutive elements are concatenated,
 * separately for each of the k binary digits): group g of 32 elements owns words g*k .. g*k+k-1;
 * bit t of word g*k+j is digit j of the code of element 32*g+t.
 */
static void pack_chunk(const uint8_t* u, uint32_t valid, uint32_t k, int layout, uint32_t* words) {
  for (uint32_t t = 0; t < valid; ++t) {
    for (uint32_t j = 0; j < k; ++j) {
      uint32_t bit = (u[t] >> j) & 1u;
      uint64_t pos; /* position in the chunk's bit string */
      if (layout == LAYOUT_INTERLEAVED) pos = (uint64_t)k * t + j;
      else pos = 32ull * ((uint64_t)(t / 32) * k + j) + (t % 32);
      words[pos / 32] |= bit << (pos % 32);
    }
  }
}

static void unpack_chunk(const uint32_t* words, uint32_t valid, uint32_t k, int layout,
                         uint8_t* u) {
  for (uint32_t t = 0; t < valid; ++t) {
    uint32_t code = 0;
    for (uint32_t j = 0; j < k; ++j) {
      uint64_t pos;
      if (layout == LAYOUT_INTERLEAVED) pos = (uint64_t)k * t + j;
      else pos = 32ull * ((uint64_t)(t / 32) * k + j) + (t % 32);
      code |= ((words[pos / 32] >> (pos % 32)) & 1u) << j;
    }
    u[t] = (uint8_t)code;
  }
}

/* Packs all chunks; payload must hold oracle_payload_bytes(n,k) bytes. */
void oracle_pack(const uint8_t* codes, uint64_t n, uint32_t C, uint32_t k, int layout,
                 uint32_t* payload) {
  memset(payload, 0, oracle_payload_bytes(n, k));
  uint64_t M = n_chunks(n, C);
  for (uint64_t m = 0; m < M; ++m) {
    uint64_t i0 = m * C;
    uint32_t valid = (uint32_t)((n - i0 < C) ? (n - i0) : C);
    pack_chunk(codes + i0, valid, k, layout, payload + m * ((uint64_t)C * k / 32));
  }
}

void oracle_unpack(const uint32_t* payload, uint64_t n, uint32_t C, uint32_t k, int layout,
                   uint8_t* codes) {
  uint64_t M = n_chunks(n, C);
  for (uint64_t m = 0; m < M; ++m) {
    uint64_t i0 = m * C;
    uint32_t valid = (uint32_t)((n - i0 < C) ? (n - i0) : C);
    unpack_chunk(payload + m * ((uint64_t)C * k / 32), valid, k, layout, codes + i0);
  }
}

/* ---------------------------------------------------------------- dequantizer ("Backward Dequantizer") */

/* ABSMAX: g_hat = g_q * s with g_q = u - 2^(k-1) (the shift by 8 is taken back for k = 4).
 * MINMAX: x_hat = u*s + o, product and sum rounded separately. */
void oracle_dequantize(const uint8_t* codes, const float* meta, uint64_t n, uint32_t C, uint32_t k,
                       int range, float* xhat) {
  for (uint64_t i = 0; i < n; ++i) {
    float s = meta[2 * (i / C)], o = meta[2 * (i / C) + 1];
    if (range == RANGE_ABSMAX) {
      xhat[i] = (float)((int)codes[i] - (1 << (k - 1))) * s;
    } else {
      float prod = (float)codes[i] * s;
      xhat[i] = prod + o;
    }
  }
}

/* ---------------------------------------------------------------- whole stream */

/* Writes header, side words and payload; stream must hold oracle_stream_bytes(n,C,k) bytes.
 * Returns 1 if any chunk was non-finite. */
int oracle_compress(const float* x, uint64_t n, uint32_t C, uint32_t k, int range, int round_mode,
                    int layout, uint64_t seed, uint64_t rng_offset, void* stream) {
  uint8_t* bytes = (uint8_t*)stream;
  uint64_t total = oracle_stream_bytes(n, C, k);
  uint64_t M = n_chunks(n, C);
  memset(bytes, 0, total);

  uint32_t header[8] = {ORACLE_MAGIC, ORACLE_VERSION, (uint32_t)n, (uint32_t)(n >> 32), C, k,
                        (uint32_t)range | ((uint32_t)round_mode << 8) | ((uint32_t)layout << 16), 0u};
  memcpy(bytes, header, 32);

  float* meta = (float*)(bytes + 32);
  uint32_t* payload = (uint32_t*)(bytes + oracle_payload_offset(n, C));
  uint8_t* u = (uint8_t*)malloc(C);
  int flags = 0;
  for (uint64_t m = 0; m < M; ++m) {
    uint64_t i0 = m * C;
    uint32_t valid = (uint32_t)((n - i0 < C) ? (n - i0) : C);
    flags |= quantize_chunk(x + i0, valid, k, range, round_mode, seed, rng_offset, i0, u,
                            meta + 2 * m);
    pack_chunk(u, valid, k, layout, payload + m * ((uint64_t)C * k / 32));
  }
  free(u);
  return flags;
}

/* Reads every parameter from the header (the receiver has only the bytes it got, Sec. 3.4).
 * Returns 0 on success, -1 if the header is invalid or disagrees with n_expected / stream_bytes. */
int oracle_decompress(const void* stream, uint64_t stream_bytes, uint64_t n_expected, float* xhat) {
  const uint8_t* bytes = (const uint8_t*)stream;
  uint32_t header[8];
  if (stream_bytes < 32) return -1;
  memcpy(header, bytes, 32);
  uint64_t n = (uint64_t)header[2] | ((uint64_t)header[3] << 32);
  uint32_t C = header[4], k = header[5];
  int range = header[6] & 0xff, layout = (header[6] >> 16) & 0xff;
  if (header[0] != ORACLE_MAGIC || header[1] != ORACLE_VERSION) return -1;
  if (n != n_expected || n == 0 || C < 32 || C % 32 != 0) return -1;
  if (!(k == 2 || k == 3 || k == 4 || k == 8) || range > 1 || layout > 1) return -1;
  if (k == 3 && layout != LAYOUT_BITPLANE) return -1;
  if (stream_bytes < oracle_stream_bytes(n, C, k)) return -1;

  const float* meta = (const float*)(bytes + 32);
  const uint32_t* payload = (const uint32_t*)(bytes + oracle_payload_offset(n, C));
  uint8_t* u = (uint8_t*)malloc(C);
  uint64_t M = n_chunks(n, C);
  for (uint64_t m = 0; m < M; ++m) {
    uint64_t i0 = m * C;
    uint32_t valid = (uint32_t)((n - i0 < C) ? (n - i0) : C);
    unpack_chunk(payload + m * ((uint64_t)C * k / 32), valid, k, layout, u);
    /* chunk-local dequantize: C passed as valid's chunk so that meta index is 0 */
    oracle_dequantize(u, meta + 2 * m, valid, C, k, range, xhat + i0);
  }
  free(u);
  return 0;
}

/* Bit width schedule: forward starts at 2 and grows by 1 at every learning-rate change up to 4
 * ("Forward Quantizer"); backward is 8 until the first change, then 4 ("Backward Quantizer"). */
int oracle_bitwidth_schedule(int is_backward, int n_lr_changes) {
  if (n_lr_changes < 0) n_lr_changes = 0;
  if (is_backward) return n_lr_changes == 0 ? 8 : 4;
  return (2 + n_lr_changes > 4) ? 4 : 2 + n_lr_changes;
}

/* ============================================================================================
 * Forward quantizer: multi-bit quantization (Sec. 3.3 "Forward Quantizer", Eq. 1-5), its encoder
 * ("Forward Encoder") and the receiver side (Sec. 3.4 "Forward Decoder", "Forward Dequantizer").
 *
 * x_v ~ B_v alpha with B_v in {-1,+1}^(N x k): element i carries k signs b_i0..b_i,k-1, stored as
 * the k-bit code c_i = sum_j [b_ij = +1] << j (a sign of -1 is stored as the bit 0), packed as bit planes
 * (plane j = basis j).  The 2^k possible values (the set P of the paper) are
 *     level(c) = (+-alpha_0) + (+-alpha_1) + ... summed in fp32 in the order j = 0..k-1.
 *
 * Readings:
 *   - batch t >= 1: B^t = nearest element of P^(t-1) for every value (the distances are compared
 *     exactly, whatever the magnitudes of x and the levels; a tie goes to the lower level; codes
 *     whose levels coincide: the smallest code);
 *     then alpha_cur = (B^T B)^-1 B^T x (Eq. 3) and alpha^t = beta alpha^(t-1) + (1-beta) alpha_cur
 *     with beta = min(0.9, (1+t)/(10+t)) (Eq. 4).  B^T B is made of integers; every entry of B^T x is the
 *     exact sum rounded once to double (see "exact sums" below), so neither depends on the order of the
 *     elements; the k x k system is solved in double by Gaussian elimination with partial pivoting and
 *     alpha^t is rounded once to fp32.  If B^T B is singular (a pivot below 1e-9 N) alpha_cur = alpha^(t-1).
 *   - the stream carries alpha^t (the coefficients after the update) and m_q = E[B alpha^t - x]
 *     (Eq. 5), so that the receiver computes B alpha^t - m_q ("Forward Dequantizer").
 *   - batch 0 of an epoch: residue method: r = x; for j = 0..k-1: b_j = sign(r) (+1 for r >= 0),
 *     alpha_j = mean |r|, r <- r - alpha_j b_j (fp32 residues; the mean is the exact sum rounded once to
 *     double, divided by n, rounded to fp32); no Eq. 3/4 update.
 *   - m_q (Eq. 5) = (sum_p alpha_p * (sum of the signs of basis p) - sum of x) / n in double, the sum of x
 *     exact and rounded once.
 * ============================================================================================ */

#define MBQ_MAGIC_KIND 1u /* header word 7 */

uint64_t oracle_mbq_payload_offset(uint32_t k) {
  uint64_t off = 32 + 4 * (uint64_t)(k + 1); /* alpha (k floats) and m_q: the 32(k+1) bits of Eq. 8 */
  return (off + 15) / 16 * 16;
}

uint64_t oracle_mbq_stream_bytes(uint64_t n, uint32_t k) {
  return oracle_mbq_payload_offset(k) + oracle_payload_bytes(n, k);
}

/* The set P: levels[c] for every code c. */
void oracle_mbq_levels(const float* alpha, uint32_t k, float* levels) {
  for (uint32_t c = 0; c < (1u << k); ++c) {
    float v = 0.0f;
    for (uint32_t j = 0; j < k; ++j) {
      float term = ((c >> j) & 1u) ? alpha[j] : -alpha[j];
      v = (j == 0) ? term : v + term;
    }
    levels[c] = v;
  }
}

/* ---- exact sums --------------------------------------------------------------------------------
 * Eq. 3 (B^T x) and Eq. 5 (the mean of B alpha - x) are sums over the whole tensor.  They are taken
 * here as the paper writes them, as sums of real numbers: every fp32 value is an integer multiple of
 * 2^-149, so the sum is held as an integer count of that unit (positive and negative parts apart,
 * 384 bits each: 277 bits for the largest fp32 value and room for 2^64 of them) and rounded ONCE, to
 * the nearest double (ties to even).  The result does not depend on the order of the elements. */

#define EXACT_LIMBS 6
typedef struct { uint64_t pos[EXACT_LIMBS], neg[EXACT_LIMBS]; } exact_sum;

static void exact_clear(exact_sum* a) { memset(a, 0, sizeof(*a)); }

/* acc += v * 2^shift (v < 2^24) */
static void limbs_add_shifted(uint64_t* acc, uint64_t v, unsigned shift) {
  unsigned limb = shift / 64, off = shift % 64;
  uint64_t lo = v << off, hi = off ? (v >> (64 - off)) : 0;
  uint64_t parts[2] = {lo, hi};
  unsigned carry = 0;
  for (unsigned i = limb; i < EXACT_LIMBS; ++i) {
    uint64_t add = (i - limb < 2) ? parts[i - limb] : 0;
    uint64_t before = acc[i];
    uint64_t sum = before + add;
    unsigned c1 = sum < before;
    uint64_t sum2 = sum + carry;
    unsigned c2 = sum2 < sum;
    acc[i] = sum2;
    carry = c1 | c2;
    if (i - limb >= 1 && !carry) break;
  }
}

/* Adds x (or -x when negate != 0).  Non-finite values are skipped: their chunk or tensor is flagged elsewhere. */
static void exact_add(exact_sum* a, float x, int negate) {
  uint32_t bits;
  memcpy(&bits, &x, 4);
  uint32_t E = (bits >> 23) & 0xFFu, frac = bits & 0x7FFFFFu;
  int negative = (int)(bits >> 31) ^ (negate ? 1 : 0);
  if (E == 255u) return;
  /* x = m * 2^(E-150) with the hidden bit in m (E >= 1), or m * 2^-149 (subnormal) */
  uint64_t m = E ? (frac | 0x800000u) : frac;
  unsigned shift = E ? E - 1 : 0;
  if (m) limbs_add_shifted(negative ? a->neg : a->pos, m, shift);
}

static int limbs_compare(const uint64_t* p, const uint64_t* q) {
  for (int i = EXACT_LIMBS - 1; i >= 0; --i)
    if (p[i] != q[i]) return p[i] > q[i] ? 1 : -1;
  return 0;
}

/* The accumulated sum rounded to the nearest double, ties to even. */
static double exact_round(const exact_sum* a) {
  int cmp = limbs_compare(a->pos, a->neg);
  if (cmp == 0) return 0.0;
  const uint64_t* big = cmp > 0 ? a->pos : a->neg;
  const uint64_t* small = cmp > 0 ? a->neg : a->pos;
  uint64_t d[EXACT_LIMBS];
  unsigned borrow = 0;
  for (int i = 0; i < EXACT_LIMBS; ++i) {
    uint64_t t = big[i] - small[i];
    unsigned b1 = big[i] < small[i];
    uint64_t t2 = t - borrow;
    unsigned b2 = t < borrow;
    d[i] = t2;
    borrow = b1 | b2;
  }
  int top = -1; /* index of the highest set bit */
  for (int i = EXACT_LIMBS * 64 - 1; i >= 0; --i)
    if ((d[i / 64] >> (i % 64)) & 1u) { top = i; break; }
  uint64_t mant = 0;
  int low = top > 52 ? top - 52 : 0; /* the mantissa is bits [low, top] */
  for (int i = top; i >= low; --i) mant = (mant << 1) | ((d[i / 64] >> (i % 64)) & 1u);
  if (low > 0) {
    int guard = (int)((d[(low - 1) / 64] >> ((low - 1) % 64)) & 1u), sticky = 0;
    for (int i = low - 2; i >= 0 && !sticky; --i) sticky = (int)((d[i / 64] >> (i % 64)) & 1u);
    if (guard && (sticky || (mant & 1u))) ++mant; /* 2^53 is still exact in a double */
  }
  double r = ldexp((double)mant, low - 149);
  return cmp > 0 ? r : -r;
}

/* Sum of x[0..n), exactly, rounded once to double. */
double oracle_exact_sum(const float* x, uint64_t n) {
  exact_sum a;
  exact_clear(&a);
  for (uint64_t i = 0; i < n; ++i) exact_add(&a, x[i], 0);
  return exact_round(&a);
}

/* Sum of |x[0..n)|, exactly, rounded once to double. */
double oracle_exact_abs_sum(const float* x, uint64_t n) {
  exact_sum a;
  exact_clear(&a);
  for (uint64_t i = 0; i < n; ++i) exact_add(&a, fabsf(x[i]), 0);
  return exact_round(&a);
}

/* (B^T x)_p = sum of +x over the elements whose basis p is +1 and of -x over the others, exactly, rounded once. */
double oracle_exact_signed_sum(const float* x, const uint8_t* codes, uint64_t n, uint32_t p) {
  exact_sum a;
  exact_clear(&a);
  for (uint64_t i = 0; i < n; ++i) exact_add(&a, x[i], !((codes[i] >> p) & 1u));
  return exact_round(&a);
}

/* s + e = a + b exactly (Knuth's two-sum; no overflow for fp32-sized inputs). */
static void two_sum(double a, double b, double* s, double* e) {
  double sum = a + b;
  double bv = sum - a;
  *e = (a - (sum - bv)) + (b - bv);
  *s = sum;
}

/* Sign of 2x - (a + b), exactly.  -(a + b) is held as a two-term non-overlapping expansion and 2x is
 * added to it term by term (smallest first), each step an exact two-sum; the largest non-zero term of
 * the resulting non-overlapping expansion carries the sign of the whole sum. */
static int sign_2x_minus_sum(float x, float a, float b) {
  double s, e, q, h1, h2;
  two_sum(-(double)a, -(double)b, &s, &e);
  two_sum(2.0 * (double)x, e, &q, &h1);
  two_sum(q, s, &q, &h2);
  if (q != 0.0) return q > 0.0 ? 1 : -1;
  if (h2 != 0.0) return h2 > 0.0 ? 1 : -1;
  if (h1 != 0.0) return h1 > 0.0 ? 1 : -1;
  return 0;
}

/* Is level a strictly closer to x than level b?  |x - a| < |x - b| decided without rounding: the
 * differences themselves need up to 277 bits when x and the levels are far apart, so for x strictly
 * between the two levels the test is 2x against a + b; outside, the nearer end wins. */
static int strictly_closer(float x, float a, float b) {
  if (a == b) return 0;
  float lo = a < b ? a : b, hi = a < b ? b : a;
  int lower_wins; /* 1: lo is strictly closer, 0: tie, -1: hi is strictly closer */
  if (x <= lo) lower_wins = 1;
  else if (x >= hi) lower_wins = -1;
  else lower_wins = -sign_2x_minus_sum(x, lo, hi);
  return a < b ? lower_wins > 0 : lower_wins < 0;
}

/* Closest value of P for every element (Sec. 3.3 "Forward Quantizer": each value takes the closest
 * element of P); a tie goes to the lower level, coinciding levels to the smallest code. */
void oracle_mbq_assign_nearest(const float* x, uint64_t n, const float* alpha, uint32_t k, uint8_t* codes) {
  float levels[256];
  oracle_mbq_levels(alpha, k, levels);
  for (uint64_t i = 0; i < n; ++i) {
    uint32_t best = 0;
    for (uint32_t c = 1; c < (1u << k); ++c) {
      int closer = strictly_closer(x[i], levels[c], levels[best]);
      int tie = !closer && !strictly_closer(x[i], levels[best], levels[c]);
      if (closer || (tie && levels[c] < levels[best])) best = c;
    }
    codes[i] = (uint8_t)best;
  }
}

/* Residue-based initialisation: signs of the successive residues and alpha_j = mean |residue|. */
void oracle_mbq_assign_residue(const float* x, uint64_t n, uint32_t k, uint8_t* codes, float* alpha0) {
  float* r = (float*)malloc(sizeof(float) * n);
  memcpy(r, x, sizeof(float) * n);
  memset(codes, 0, n);
  for (uint32_t j = 0; j < k; ++j) {
    double sum = oracle_exact_abs_sum(r, n);
    alpha0[j] = (float)(sum / (double)n);
    for (uint64_t i = 0; i < n; ++i) {
      if (r[i] >= 0.0f) { codes[i] |= (uint8_t)(1u << j); r[i] = r[i] - alpha0[j]; }
      else r[i] = r[i] + alpha0[j];
    }
  }
  free(r);
}

/* Eq. 3: least squares for alpha given the signs; returns 0 and leaves alpha_cur = alpha_prev if singular. */
static int mbq_least_squares(const float* x, const uint8_t* codes, uint64_t n, uint32_t k, const float* alpha_prev,
                             double* alpha_cur) {
  double G[8][8], rhs[8];
  /* B^T B: integers (sums of +-1), exact in double; B^T x: exact sums rounded once */
  for (uint32_t p = 0; p < k; ++p)
    for (uint32_t q = 0; q < k; ++q) {
      int64_t g = 0;
      for (uint64_t i = 0; i < n; ++i) g += (((codes[i] >> p) ^ (codes[i] >> q)) & 1u) ? -1 : 1;
      G[p][q] = (double)g;
    }
  for (uint32_t p = 0; p < k; ++p) rhs[p] = oracle_exact_signed_sum(x, codes, n, p);
  /* Gaussian elimination with partial pivoting */
  for (uint32_t c = 0; c < k; ++c) {
    uint32_t piv = c;
    for (uint32_t r = c + 1; r < k; ++r)
      if (fabs(G[r][c]) > fabs(G[piv][c])) piv = r;
    if (fabs(G[piv][c]) < 1e-9 * (double)n) {
      for (uint32_t p = 0; p < k; ++p) alpha_cur[p] = (double)alpha_prev[p];
      return 0;
    }
    if (piv != c) {
      for (uint32_t q = 0; q < k; ++q) { double t = G[c][q]; G[c][q] = G[piv][q]; G[piv][q] = t; }
      double t = rhs[c]; rhs[c] = rhs[piv]; rhs[piv] = t;
    }
    for (uint32_t r = c + 1; r < k; ++r) {
      double f = G[r][c] / G[c][c];
      for (uint32_t q = c; q < k; ++q) G[r][q] -= f * G[c][q];
      rhs[r] -= f * rhs[c];
    }
  }
  for (int c = (int)k - 1; c >= 0; --c) {
    double s = rhs[c];
    for (uint32_t q = (uint32_t)c + 1; q < k; ++q) s -= G[c][q] * alpha_cur[q];
    alpha_cur[c] = s / G[c][c];
  }
  return 1;
}

/* Eq. 3 + Eq. 4: alpha^t from alpha^(t-1), the signs and the data. */
void oracle_mbq_update_alpha(const float* x, const uint8_t* codes, uint64_t n, uint32_t k, const float* alpha_prev,
                             uint32_t t, float* alpha_next) {
  double cur[8];
  mbq_least_squares(x, codes, n, k, alpha_prev, cur);
  double beta = (1.0 + (double)t) / (10.0 + (double)t);
  if (beta > 0.9) beta = 0.9;
  for (uint32_t p = 0; p < k; ++p) alpha_next[p] = (float)(beta * (double)alpha_prev[p] + (1.0 - beta) * cur[p]);
}

/* Eq. 5: mean of the quantization error of B alpha. */
float oracle_mbq_bias(const float* x, const uint8_t* codes, uint64_t n, uint32_t k, const float* alpha) {
  double sum_x = oracle_exact_sum(x, n), acc = 0.0;
  for (uint32_t p = 0; p < k; ++p) {
    int64_t s = 0; /* sum of the signs of basis p */
    for (uint64_t i = 0; i < n; ++i) s += ((codes[i] >> p) & 1u) ? 1 : -1;
    acc += (double)alpha[p] * (double)s;
  }
  return (float)((acc - sum_x) / (double)n);
}

/* Whole forward compressor for batch t; init != 0 selects the residue method (alpha_prev unused).
 * Writes the stream and alpha_next (= the alpha carried by the stream). */
void oracle_mbq_compress(const float* x, uint64_t n, uint32_t k, uint32_t t, int init, const float* alpha_prev,
                         void* stream, float* alpha_next) {
  uint8_t* bytes = (uint8_t*)stream;
  memset(bytes, 0, oracle_mbq_stream_bytes(n, k));
  uint8_t* codes = (uint8_t*)malloc(n);
  if (init) {
    oracle_mbq_assign_residue(x, n, k, codes, alpha_next);
  } else {
    oracle_mbq_assign_nearest(x, n, alpha_prev, k, codes);
    oracle_mbq_update_alpha(x, codes, n, k, alpha_prev, t, alpha_next);
  }
  float m_q = oracle_mbq_bias(x, codes, n, k, alpha_next);
  uint32_t header[8] = {ORACLE_MAGIC, ORACLE_VERSION, (uint32_t)n, (uint32_t)(n >> 32), 0u, k, 0u, MBQ_MAGIC_KIND};
  memcpy(bytes, header, 32);
  memcpy(bytes + 32, alpha_next, 4 * k);
  memcpy(bytes + 32 + 4 * k, &m_q, 4);
  /* bit planes: plane j of group g = basis j of elements 32g..32g+31, -1 stored as 0 */
  uint32_t* payload = (uint32_t*)(bytes + oracle_mbq_payload_offset(k));
  for (uint64_t i = 0; i < n; ++i)
    for (uint32_t j = 0; j < k; ++j)
      payload[(i / 32) * k + j] |= (uint32_t)((codes[i] >> j) & 1u) << (i % 32);
  free(codes);
}

/* Receiver: decode the planes, x_hat = B alpha - m_q.  Returns -1 on a bad header. */
int oracle_mbq_decompress(const void* stream, uint64_t stream_bytes, uint64_t n_expected, float* xhat) {
  const uint8_t* bytes = (const uint8_t*)stream;
  uint32_t header[8];
  if (stream_bytes < 32) return -1;
  memcpy(header, bytes, 32);
  uint64_t n = (uint64_t)header[2] | ((uint64_t)header[3] << 32);
  uint32_t k = header[5];
  if (header[0] != ORACLE_MAGIC || header[1] != ORACLE_VERSION || header[7] != MBQ_MAGIC_KIND) return -1;
  if (n != n_expected || n == 0 || k < 1 || k > 4) return -1;
  if (stream_bytes < oracle_mbq_stream_bytes(n, k)) return -1;
  float alpha[8], m_q, levels[256];
  memcpy(alpha, bytes + 32, 4 * k);
  memcpy(&m_q, bytes + 32 + 4 * k, 4);
  oracle_mbq_levels(alpha, k, levels);
  const uint32_t* payload = (const uint32_t*)(bytes + oracle_mbq_payload_offset(k));
  for (uint64_t i = 0; i < n; ++i) {
    uint32_t c = 0;
    for (uint32_t j = 0; j < k; ++j) c |= ((payload[(i / 32) * k + j] >> (i % 32)) & 1u) << j;
    xhat[i] = levels[c] - m_q;
  }
  return 0;
}

/* ============================================================================================
 * Grouping along the batch dimension (Sec. 3.3: the encoder works along the batch dimension; "Forward
 * Encoder": consecutive elements along the first dimension share an integer; "Backward Encoder": codes of
 * neighbouring samples are combined into one integer).
 *
 * The tensor is n_b x F (F = w*h*c values per sample, group_stride).  A pack group is made of the
 * 32 batch neighbours (rows 32g .. 32g+31) of one feature f instead of 32 consecutive values:
 * group index G = g*F + f, words G*k .. G*k+k-1, element (row b, feature f) at position t = b % 32.
 * Rows past n_b are zero bits ("ceil(n/8)" of Eq. 8).  Ranges stay per chunk of C consecutive
 * values of the vectorised tensor.  Header word 7 holds F (0 = consecutive grouping).
 * ============================================================================================ */

uint64_t oracle_strided_payload_bytes(uint64_t n, uint32_t k, uint32_t F) {
  uint64_t nb = n / F;
  return 4ull * k * ((nb + 31) / 32) * F;
}

uint64_t oracle_strided_stream_bytes(uint64_t n, uint32_t C, uint32_t k, uint32_t F) {
  return oracle_payload_offset(n, C) + oracle_strided_payload_bytes(n, k, F);
}

/* bit position of digit j of element i in the payload */
static uint64_t strided_bit_position(uint64_t i, uint32_t j, uint32_t k, int layout, uint32_t F) {
  uint64_t b = i / F, f = i % F;
  uint64_t G = (b / 32) * F + f;
  uint32_t t = (uint32_t)(b % 32);
  if (layout == LAYOUT_INTERLEAVED) return 32ull * k * G + (uint64_t)k * t + j;
  return 32ull * (k * G + j) + t;
}

int oracle_compress_strided(const float* x, uint64_t n, uint32_t C, uint32_t k, int range, int round_mode,
                            int layout, uint64_t seed, uint64_t rng_offset, uint32_t F, void* stream) {
  uint8_t* bytes = (uint8_t*)stream;
  memset(bytes, 0, oracle_strided_stream_bytes(n, C, k, F));
  uint32_t header[8] = {ORACLE_MAGIC, ORACLE_VERSION, (uint32_t)n, (uint32_t)(n >> 32), C, k,
                        (uint32_t)range | ((uint32_t)round_mode << 8) | ((uint32_t)layout << 16), F};
  memcpy(bytes, header, 32);
  uint8_t* codes = (uint8_t*)malloc(n);
  int flags = oracle_quantize(x, n, C, k, range, round_mode, seed, rng_offset, codes, (float*)(bytes + 32));
  uint32_t* payload = (uint32_t*)(bytes + oracle_payload_offset(n, C));
  for (uint64_t i = 0; i < n; ++i)
    for (uint32_t j = 0; j < k; ++j) {
      uint64_t pos = strided_bit_position(i, j, k, layout, F);
      payload[pos / 32] |= (uint32_t)((codes[i] >> j) & 1u) << (pos % 32);
    }
  free(codes);
  return flags;
}

int oracle_decompress_strided(const void* stream, uint64_t stream_bytes, uint64_t n_expected, float* xhat) {
  const uint8_t* bytes = (const uint8_t*)stream;
  uint32_t header[8];
  if (stream_bytes < 32) return -1;
  memcpy(header, bytes, 32);
  uint64_t n = (uint64_t)header[2] | ((uint64_t)header[3] << 32);
  uint32_t C = header[4], k = header[5], F = header[7];
  int range = header[6] & 0xff, layout = (header[6] >> 16) & 0xff;
  if (header[0] != ORACLE_MAGIC || header[1] != ORACLE_VERSION) return -1;
  if (n != n_expected || n == 0 || C < 32 || C % 32 != 0 || F == 0 || n % F != 0) return -1;
  if (!(k == 2 || k == 3 || k == 4 || k == 8) || range > 1 || layout > 1) return -1;
  if (stream_bytes < oracle_strided_stream_bytes(n, C, k, F)) return -1;
  const float* meta = (const float*)(bytes + 32);
  const uint32_t* payload = (const uint32_t*)(bytes + oracle_payload_offset(n, C));
  uint8_t* codes = (uint8_t*)malloc(n);
  for (uint64_t i = 0; i < n; ++i) {
    uint32_t c = 0;
    for (uint32_t j = 0; j < k; ++j) {
      uint64_t pos = strided_bit_position(i, j, k, layout, F);
      c |= ((payload[pos / 32] >> (pos % 32)) & 1u) << j;
    }
    codes[i] = (uint8_t)c;
  }
  oracle_dequantize(codes, meta, n, C, k, range, xhat);
  free(codes);
  return 0;
}
