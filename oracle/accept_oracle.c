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
 *   - "dividing by the scaling factor" is computed as a product with inv = L/c (one division per
 *     chunk); pinned against true division in the tests;
 *   - nearest rounding is IEEE round-half-to-even;
 *   - the uniform generator of Eq. 7 is counter based (MurmurHash3's 32-bit finaliser, one hash per
 *     pair of counters, see oracle_rng_hash below); U has 24 bits; pr = t - floor(t) and the test
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

/* 32 random bits for counter ctr under seed.  Counters 2j and 2j+1 share the hash of their pair
 * index j; the odd one multiplies it by an odd constant (a bijection of the 32-bit word). */
uint32_t oracle_rng_hash(uint64_t seed, uint64_t ctr) {
  uint64_t pair = ctr >> 1;
  /* the constant keeps seed 0, pair 0 off the fixed point fmix32(0) = 0 */
  uint32_t inner = fmix32((uint32_t)(pair >> 32) ^ (uint32_t)seed ^ 0x9E3779B9u);
  uint32_t h = fmix32((uint32_t)pair ^ inner ^ (uint32_t)(seed >> 32));
  return (ctr & 1) ? h * 0x9E3779B1u : h;
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
    inv = L / c;
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
    inv = L / r;
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

/* ABSMAX: g_hat = g_q * s with g_q = u - 2^(k-1) ("subtracting each element by 8" for k = 4).
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
