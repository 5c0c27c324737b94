// Pack groups along the batch dimension (Sec. 3.3: the encoder "concatenates the quantized data
// along the batch size dimension"): the tensor is n_b x F, a group is the 32 batch neighbours
// (rows 32g..32g+31) of one feature f, group index G = g*F + f, words G*K .. G*K+K-1.
//
// A thread owns eight consecutive features (one octet column) and eight rows of one batch group: every
// row it reads is a 32-byte load (eight neighbouring threads of the same row block read 256 contiguous
// bytes), the rows are quantized, the 8 x 8 code bytes are transposed in registers (byte permutes) so
// that each feature's eight batch neighbours sit in two words, and those are packed exactly like an
// octet of the consecutive layout.  Ranges stay per chunk of the
// vectorised tensor: the per-chunk constants come from the records the range pass left in the
// workspace (accept_wide.cuh), so this path always runs as range pass + constants + encode.
#pragma once
#include "accept_wide.cuh"

namespace accept {

// 4 x 4 byte transpose in registers: o[c] byte r = a_r byte c.
__device__ __forceinline__ void transpose4x4(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t (&o)[4]) {
  const uint32_t t0 = __byte_perm(a0, a1, 0x5140), t1 = __byte_perm(a2, a3, 0x5140);
  const uint32_t t2 = __byte_perm(a0, a1, 0x7362), t3 = __byte_perm(a2, a3, 0x7362);
  o[0] = __byte_perm(t0, t1, 0x5410);
  o[1] = __byte_perm(t0, t1, 0x7632);
  o[2] = __byte_perm(t2, t3, 0x5410);
  o[3] = __byte_perm(t2, t3, 0x7632);
}

// A thread owns eight consecutive features and EIGHT of the 32 rows of a batch group: the four lanes
// of a quad own the four blocks of eight rows of the same feature octet.  INTERLEAVED words are
// complete per block of eight rows (K = 4: one word, K = 8: two, K = 2: half a word), so a lane
// stores its own piece; BITPLANE words take one byte from each lane of the quad, exchanged with the
// quad byte transpose.  Block = 64 feature octets x 4 row blocks.
constexpr int kStridedOctetsPerBlock = 64;

template <int K, int LAYOUT, int RANGE, int ROUND>
__global__ void __launch_bounds__(256, 4) strided_encode_kernel(const CodecArgs a, const ChunkRecord* rec) {
  grid_dependency_handshake();
  const int tid = threadIdx.x, lane = tid & 31, sub = tid & 3;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    a.header[tid] = header_word(a, tid);
    if ((a.n_chunks & 1) && tid < 2) reinterpret_cast<uint32_t*>(a.meta + a.n_chunks)[tid] = 0u;
  }
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t fo = blockIdx.x * kStridedOctetsPerBlock + (tid >> 2);  // feature octet
  const bool active = (uint64_t)fo * 8 < F;                              // inactive lanes still shuffle
  const uint64_t g = blockIdx.y;
  const uint64_t word0 = (g * F + (uint64_t)fo * 8) * K;  // first word of feature 8*fo of this batch group
  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};

  uint32_t xlo[8], xhi[8];  // per row: codes of features 0..3 / 4..7
  // four rows at a time: 128 bytes in flight per thread at half the registers, so that more blocks
  // stay resident (the kernel waits on memory, not on arithmetic)
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    float v[4][8];
    bool in[4];
    uint4 raw[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const uint64_t row = g * 32 + sub * 8 + half * 4 + r;
      in[r] = active && row < n_rows;
      if (in[r]) {
        const uint64_t i0 = row * F + (uint64_t)fo * 8;
        ld_octet(a.x + i0, v[r]);
        raw[r] = __ldg(reinterpret_cast<const uint4*>(rec + chunk_of(a, i0)));
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int rr = half * 4 + r;
      xlo[rr] = 0; xhi[rr] = 0;
      if (in[r]) {
        const uint64_t i0 = (g * 32 + sub * 8 + rr) * F + (uint64_t)fo * 8;
        Scale sc;
        sc.s = 0.0f; sc.o = 0.0f;
        sc.inv = __uint_as_float(raw[r].z);
        sc.base = __uint_as_float(raw[r].w);
        sc.nonfinite = raw[r].x != 0u;
        if (sc.nonfinite) {
#pragma unroll
          for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
        }
        RngThread rt;
        if (ROUND == kStochastic) rt.init(rng, a.rng_offset + i0, 8u);
        quantize_octet<K, RANGE, ROUND>(v[r], sc, rng, rt, 0u, xlo[rr], xhi[rr]);
      }
    }
  }
  // rows x features -> features x rows
  uint32_t ylo[8], yhi[8];  // per feature: codes of rows 0..3 / 4..7 of this block of eight rows
  {
    uint32_t o[4];
    transpose4x4(xlo[0], xlo[1], xlo[2], xlo[3], o);
#pragma unroll
    for (int e = 0; e < 4; ++e) ylo[e] = o[e];
    transpose4x4(xlo[4], xlo[5], xlo[6], xlo[7], o);
#pragma unroll
    for (int e = 0; e < 4; ++e) yhi[e] = o[e];
    transpose4x4(xhi[0], xhi[1], xhi[2], xhi[3], o);
#pragma unroll
    for (int e = 0; e < 4; ++e) ylo[4 + e] = o[e];
    transpose4x4(xhi[4], xhi[5], xhi[6], xhi[7], o);
#pragma unroll
    for (int e = 0; e < 4; ++e) yhi[4 + e] = o[e];
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    uint32_t* group_words = a.payload + word0 + (uint64_t)e * K;
    if (LAYOUT == kBitplane) {
      // byte j = digit j of my eight rows; after the quad transpose lane q holds digit q of all 32 rows
      const uint32_t w = quad_transpose(planes_nibbles(merge_nibbles(ylo[e], yhi[e])), lane);
      if (active && sub < K) group_words[sub] = w;
    } else if (K == 8) {
      if (active) reinterpret_cast<uint2*>(group_words)[sub] = make_uint2(ylo[e], yhi[e]);
    } else if (K == 4) {
      const uint32_t zlo = ylo[e] | (ylo[e] >> 4), zhi = yhi[e] | (yhi[e] >> 4);
      if (active) group_words[sub] = __byte_perm(zlo, zhi, 0x6420);
    } else {  // K == 2: sixteen bits per eight rows
      uint32_t zlo = ylo[e] | (ylo[e] >> 6), zhi = yhi[e] | (yhi[e] >> 6);
      zlo |= zlo >> 12;
      zhi |= zhi >> 12;
      if (active) reinterpret_cast<uint16_t*>(group_words)[sub] = (uint16_t)__byte_perm(zlo, zhi, 0x0040);
    }
  }
}

template <int K, int LAYOUT, int RANGE>
__global__ void __launch_bounds__(256) strided_decode_kernel(const CodecArgs a) {
  grid_dependency_handshake();
  const int tid = threadIdx.x, lane = tid & 31, sub = tid & 3;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    const uint32_t mask = (tid == 6) ? 0xFFFF00FFu : 0xFFFFFFFFu;
    if ((a.header[tid] & mask) != (header_word(a, tid) & mask)) atomicOr(a.status, kDevBadHeader);
  }
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t fo = blockIdx.x * kStridedOctetsPerBlock + (tid >> 2);
  const bool active = (uint64_t)fo * 8 < F;
  const uint64_t g = blockIdx.y;
  const uint64_t word0 = (g * F + (uint64_t)fo * 8) * K;

  uint32_t ylo[8], yhi[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const uint32_t* group_words = a.payload + word0 + (uint64_t)e * K;
    if (LAYOUT == kBitplane) {
      uint32_t w = 0;
      if (active && sub < K) w = __ldg(group_words + sub);
      const uint32_t nib = planes_nibbles(quad_transpose(w, lane));  // digits of my eight rows
      ylo[e] = nib & 0x0F0F0F0Fu;
      yhi[e] = (nib >> 4) & 0x0F0F0F0Fu;
    } else if (K == 8) {
      uint2 w = make_uint2(0u, 0u);
      if (active) w = __ldg(reinterpret_cast<const uint2*>(group_words) + sub);
      ylo[e] = w.x;
      yhi[e] = w.y;
    } else if (K == 4) {
      uint32_t word = 0;
      if (active) word = __ldg(group_words + sub);
      uint32_t y = __byte_perm(word, 0, 0x4140);
      ylo[e] = (y | (y << 4)) & 0x0F0F0F0Fu;
      y = __byte_perm(word, 0, 0x4342);
      yhi[e] = (y | (y << 4)) & 0x0F0F0F0Fu;
    } else {
      uint32_t half = 0;
      if (active) half = __ldg(reinterpret_cast<const uint16_t*>(group_words) + sub);
      uint32_t y = (half | (half << 12)) & 0x000F000Fu;
      ylo[e] = (y | (y << 6)) & 0x03030303u;
      y = ((half >> 8) | ((half >> 8) << 12)) & 0x000F000Fu;
      yhi[e] = (y | (y << 6)) & 0x03030303u;
    }
  }
  uint32_t xlo[8], xhi[8];
  {
    uint32_t o[4];
    transpose4x4(ylo[0], ylo[1], ylo[2], ylo[3], o);
#pragma unroll
    for (int r = 0; r < 4; ++r) xlo[r] = o[r];
    transpose4x4(yhi[0], yhi[1], yhi[2], yhi[3], o);
#pragma unroll
    for (int r = 0; r < 4; ++r) xlo[4 + r] = o[r];
    transpose4x4(ylo[4], ylo[5], ylo[6], ylo[7], o);
#pragma unroll
    for (int r = 0; r < 4; ++r) xhi[r] = o[r];
    transpose4x4(yhi[4], yhi[5], yhi[6], yhi[7], o);
#pragma unroll
    for (int r = 0; r < 4; ++r) xhi[4 + r] = o[r];
  }
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint64_t row = g * 32 + sub * 8 + r;
    if (active && row < n_rows) {
      const uint64_t i0 = row * F + (uint64_t)fo * 8;
      const float2 so = __ldg(a.meta + chunk_of(a, i0));
      float out[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[i] = dequantize_code<K, RANGE>((xlo[r] >> (8 * i)) & 0xFFu, so.x, so.y);
        out[4 + i] = dequantize_code<K, RANGE>((xhi[r] >> (8 * i)) & 0xFFu, so.x, so.y);
      }
      st_octet(a.xhat + i0, out);
    }
  }
}

}  // namespace accept
