// Pack groups along the batch dimension (Sec. 3.3, "Forward Encoder" / "Backward Encoder": values that share a
// packed integer are neighbours along the first dimension): the tensor is n_b x F, a group is the 32 batch neighbours
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
#include "accept_async.cuh"
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

// The encoder is persistent: a block walks over tiles of 32 rows x 2 KB and stages them in shared
// memory with asynchronous bulk copies (one per row, issued by the lanes of warp 0, completion counted
// in bytes on an mbarrier), so that the bytes in flight per SM are set by shared memory (three resident
// blocks x 64 KB), not by registers, and the next tile streams in while this one is coded.
// A tile is two stages: rows 4h..4h+3 of every block of eight rows form stage h.  Once every thread has
// moved its rows of a stage to registers, the same stage of the next tile is requested.
// The rows of a block of eight are 2 KB apart; each block of eight rows starts 32 bytes further than a
// multiple of 16 KB, which spreads the four lanes of a quad over different banks.
constexpr int kStridedRowBytes = kStridedOctetsPerBlock * 32;
constexpr int kStridedRowBlockPitch = 8 * kStridedRowBytes + 32;
constexpr int kStridedTileBytes = 4 * kStridedRowBlockPitch;
constexpr int kStridedSmemBytes = kStridedTileBytes + 16;  // + two mbarriers

// Transposes a thread's 8 rows x 8 features of codes and stores the words of its eight features.
template <int K, int LAYOUT>
__device__ __forceinline__ void strided_store_tile(const CodecArgs& a, const uint32_t (&xlo)[8], const uint32_t (&xhi)[8],
                                                   uint64_t word0, bool active, int sub, int lane) {
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
    if (LAYOUT == kBitplane && K == 8) {
      // digits 0..3 and 4..7 as two sets of four planes: lane q ends up with digits q and 4 + q of all 32 rows
      const uint32_t lo = merge_nibbles(ylo[e] & 0x0F0F0F0Fu, yhi[e] & 0x0F0F0F0Fu);
      const uint32_t hi = merge_nibbles((ylo[e] >> 4) & 0x0F0F0F0Fu, (yhi[e] >> 4) & 0x0F0F0F0Fu);
      const uint32_t w0 = quad_transpose(planes_nibbles(lo), lane);
      const uint32_t w1 = quad_transpose(planes_nibbles(hi), lane);
      if (active) {
        st_c(group_words + sub, w0);
        st_c(group_words + 4 + sub, w1);
      }
    } else if (LAYOUT == kBitplane) {
      // byte j = digit j of my eight rows; after the quad transpose lane q holds digit q of all 32 rows
      const uint32_t w = quad_transpose(planes_nibbles(merge_nibbles(ylo[e], yhi[e])), lane);
      if (active && sub < K) st_c(group_words + sub, w);
    } else if (K == 8) {
      if (active) st_c(reinterpret_cast<uint2*>(group_words) + sub, make_uint2(ylo[e], yhi[e]));
    } else if (K == 4) {
      const uint32_t zlo = ylo[e] | (ylo[e] >> 4), zhi = yhi[e] | (yhi[e] >> 4);
      if (active) st_c(group_words + sub, __byte_perm(zlo, zhi, 0x6420));
    } else {  // K == 2: sixteen bits per eight rows
      uint32_t zlo = ylo[e] | (ylo[e] >> 6), zhi = yhi[e] | (yhi[e] >> 6);
      zlo |= zlo >> 12;
      zhi |= zhi >> 12;
      if (active) st_c(reinterpret_cast<uint16_t*>(group_words) + sub, (uint16_t)__byte_perm(zlo, zhi, 0x0040));
    }
  }
}

// How the persistent encoder walks the tensor: tiles_x x tiles_y tiles, taken in row-major order with a
// stride of one grid; the stride is given split into whole tile rows and a remainder so that a block
// advances its tile coordinates with an add and a compare.
struct StridedTiling {
  uint32_t tiles_x, tiles_y;
  uint32_t n_rows;           // batch rows of the tensor
  uint32_t step_x, step_y;   // gridDim.x = step_y * tiles_x + step_x
};

// Warp 0 requests stage `half` of tile (bx, g): lane = row of the tile, rows with ((row / 4) & 1) == half.
__device__ __forceinline__ void strided_request_stage(const CodecArgs& a, const StridedTiling& t, uint32_t bx, uint32_t g,
                                                      int half, int lane, uint32_t tile0, uint32_t bar) {
  const uint32_t F = a.group_stride;
  const uint32_t fo0 = bx * kStridedOctetsPerBlock;
  const uint32_t row_bytes = min((uint32_t)kStridedOctetsPerBlock, F / 8 - fo0) * 32;
  const uint32_t rows_left = t.n_rows - g * 32;
  const uint32_t valid = (rows_left >= 32 ? 0xFFFFFFFFu : ((1u << rows_left) - 1u)) & (half ? 0xF0F0F0F0u : 0x0F0F0F0Fu);
  if (lane == 0) mbarrier_expect_bytes(bar, __popc(valid) * row_bytes + kCopyAnnounceExtra);
  __syncwarp();
  if ((valid >> lane) & 1u) {
    const float* src = a.x + (uint64_t)(g * 32 + lane) * F + (uint64_t)fo0 * 8;
    const uint32_t dst = tile0 + (lane >> 3) * kStridedRowBlockPitch + (lane & 7) * kStridedRowBytes;
    if (bounds_ok(src, row_bytes, false)) bulk_copy_to_shared(dst, src, row_bytes, bar);
  }
}

// The encoder's constants of the four rows a thread codes in stage `half` of tile (bx, g): inv (sign
// bit = chunk is non-finite) and, for MINMAX, base.  Rows outside the tensor get in = false.
template <int RANGE>
struct StridedRowConstants {
  float inv[4], base[4];
  bool in[4];
  // ALLFULL: every tile of the launch has all its rows and octets and the chunk size is a power of two
  template <bool ALLFULL>
  __device__ __forceinline__ void fetch(const CodecArgs& a, const ChunkRecord* rec, const StridedTiling& t, uint32_t bx,
                                        uint32_t g, int half, int tid) {
    const uint32_t F = a.group_stride;
    const uint32_t fo = bx * kStridedOctetsPerBlock + (tid >> 2);
    const bool active = fo < F / 8;
    const uint32_t row0 = g * 32 + (tid & 3) * 8 + half * 4;
    uint64_t i0 = (uint64_t)row0 * F + (uint64_t)fo * 8;
#pragma unroll
    for (int r = 0; r < 4; ++r, i0 += F) {
      in[r] = ALLFULL || (active && row0 + r < t.n_rows);
      inv[r] = 0.0f;
      base[r] = 0.0f;
      if (in[r]) {
        const ChunkRecord* c = rec + (ALLFULL ? (i0 >> a.chunk_shift) : chunk_of(a, i0));
        if (RANGE == kAbsMax) {
          inv[r] = ldg_c(&c->inv);
        } else {
          const float2 ib = ldg_c(reinterpret_cast<const float2*>(&c->inv));
          inv[r] = ib.x;
          base[r] = ib.y;
        }
      }
    }
  }
};

template <int K, int LAYOUT, int RANGE, int ROUND, bool ALLFULL>
__device__ __forceinline__ void strided_encode_tiles(const CodecArgs& a, const ChunkRecord* rec, const StridedTiling& t,
                                                     uint8_t* s_tile) {
  const int tid = threadIdx.x, lane = tid & 31, sub = tid & 3;
  const uint32_t F = a.group_stride;
  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  // The eight lanes of a quarter warp read 32 bytes each at {row block 0..3} x {two neighbouring octet columns}; the row
  // blocks are 32 bytes apart modulo 128, so the 16-byte halves of neighbouring columns would meet on the same banks two by
  // two.  Odd columns therefore read their upper half first and hold features 4..7 where the others hold 0..3: codes do not
  // depend on the position (nearest rounding), so the two packed words of a row are exchanged afterwards and nothing else changes.
  const int swapped = (ROUND == kNearest) ? ((tid >> 2) & 1) : 0;

  const uint32_t tile0 = smem_address(s_tile);
  const uint32_t bar[2] = {smem_address(s_tile + kStridedTileBytes), smem_address(s_tile + kStridedTileBytes) + 8u};
  if (tid == 0) {
    mbarrier_init(bar[0], 1);
    mbarrier_init(bar[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  uint32_t bx = blockIdx.x % t.tiles_x, g = blockIdx.x / t.tiles_x;  // this block's tile; g >= tiles_y: none left
  bool pending[2] = {false, false};  // a request of the stage's current phase is in flight
  uint32_t parity[2] = {0u, 0u};     // parity of the stage's current phase
  if (g < t.tiles_y) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      if (tid < 32) strided_request_stage(a, t, bx, g, half, lane, tile0, bar[half]);
      pending[half] = true;
    }
  }
  bool failed = false;
  StridedRowConstants<RANGE> cur, nxt;  // constants are fetched one stage ahead of their use
  if (g < t.tiles_y) cur.template fetch<ALLFULL>(a, rec, t, bx, g, 0, tid);
  while (g < t.tiles_y) {
    uint32_t next_bx = bx + t.step_x, next_g = g + t.step_y;
    if (next_bx >= t.tiles_x) { next_bx -= t.tiles_x; ++next_g; }
    const bool has_next = next_g < t.tiles_y;
    const uint32_t fo = bx * kStridedOctetsPerBlock + (tid >> 2);  // feature octet of this thread
    const bool active = ALLFULL || fo < F / 8;                     // inactive lanes still shuffle
    const uint64_t word0 = ((uint64_t)g * F + (uint64_t)fo * 8) * K;  // first word of feature 8*fo of this batch group

    uint32_t xlo[8], xhi[8];  // per row: codes of features 0..3 / 4..7
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      float v[4][8];
      const bool ok = !failed && mbarrier_wait(bar[half], parity[half]);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float4* src = reinterpret_cast<const float4*>(s_tile + sub * kStridedRowBlockPitch +
                                                            (half * 4 + r) * kStridedRowBytes + (tid >> 2) * 32);
        float4 p0 = make_float4(0.f, 0.f, 0.f, 0.f), p1 = p0;
        if ((ALLFULL || cur.in[r]) && ok) { p0 = src[swapped]; p1 = src[swapped ^ 1]; }
        v[r][0] = p0.x; v[r][1] = p0.y; v[r][2] = p0.z; v[r][3] = p0.w;
        v[r][4] = p1.x; v[r][5] = p1.y; v[r][6] = p1.z; v[r][7] = p1.w;
      }
      // every thread holds its rows of this stage, or some thread gave up (the verdict is the block's)
      if (!failed) {
        if (__syncthreads_and(ok)) {
          pending[half] = false;
          parity[half] ^= 1u;
          if (has_next) {
            if (tid < 32) strided_request_stage(a, t, next_bx, next_g, half, lane, tile0, bar[half]);
            pending[half] = true;
          }
        } else {
          failed = true;
        }
      }
      if (half == 0) nxt.template fetch<ALLFULL>(a, rec, t, bx, g, 1, tid);
      else if (has_next) nxt.template fetch<ALLFULL>(a, rec, t, next_bx, next_g, 0, tid);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int rr = half * 4 + r;
        xlo[rr] = 0; xhi[rr] = 0;
        if ((ALLFULL || cur.in[r]) && !failed) {
          const uint64_t i0 = (uint64_t)(g * 32 + sub * 8 + rr) * F + (uint64_t)fo * 8;
          Scale sc;
          sc.s = 0.0f; sc.o = 0.0f;
          sc.inv = fabsf(cur.inv[r]);
          sc.base = cur.base[r];
          sc.nonfinite = (__float_as_uint(cur.inv[r]) >> 31) != 0u;
          if (sc.nonfinite) {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
          }
          RngThread rt;
          if (ROUND == kStochastic) rt.init(rng, a.rng_offset + i0, 8u);
          quantize_octet<K, RANGE, ROUND>(v[r], sc, rng, rt, 0u, xlo[rr], xhi[rr]);
          if (swapped) { const uint32_t t_lo = xlo[rr]; xlo[rr] = xhi[rr]; xhi[rr] = t_lo; }
        }
      }
      cur = nxt;
    }
    if (failed) break;
    strided_store_tile<K, LAYOUT>(a, xlo, xhi, word0, active, sub, lane);
    bx = next_bx;
    g = next_g;
  }
  if (failed) {
    // a copy did not arrive: report it, give what is still in flight a bounded time to land, and leave
    if (tid == 0) atomicOr(a.status, kDevCopyTimeout);
#pragma unroll
    for (int half = 0; half < 2; ++half)
      if (pending[half]) mbarrier_wait(bar[half], parity[half]);
  }
}

template <int K, int LAYOUT, int RANGE, int ROUND>
__global__ void __launch_bounds__(256, 3) strided_encode_kernel(const CodecArgs a, const ChunkRecord* rec,
                                                                const StridedTiling t) {
  extern __shared__ __align__(128) uint8_t s_tile[];
  grid_dependency_handshake();
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && tid < 8) {
    st_c(a.header + tid, header_word(a, tid));
    if ((a.n_chunks & 1) && tid < 2) st_c(reinterpret_cast<uint32_t*>(a.meta + a.n_chunks) + tid, 0u);
  }
  // the same for every block of the launch: no tile with missing rows or octets, chunk indices by a shift
  const bool all_full = a.chunk_shift >= 0 && t.n_rows % 32 == 0 && (a.group_stride / 8) % kStridedOctetsPerBlock == 0;
  if (all_full) strided_encode_tiles<K, LAYOUT, RANGE, ROUND, true>(a, rec, t, s_tile);
  else strided_encode_tiles<K, LAYOUT, RANGE, ROUND, false>(a, rec, t, s_tile);
}

// Hashed words of three consecutive quads when the low word of the quad index wraps among them (once in
// 2^34 counters): each quad with the key of its own upper word.  Out of line, everything by value.
__device__ __noinline__ uint3 strided_quad_hashes_slowly(Rng rng, uint64_t quad) {
  // (counters wrap at 2^64, so quad indices wrap at 2^62)
  const uint64_t q1 = (quad + 1) & 0x3FFFFFFFFFFFFFFFull, q2 = (quad + 2) & 0x3FFFFFFFFFFFFFFFull;
  uint3 h;
  h.x = Rng::quad_hash((uint32_t)quad, rng.key((uint32_t)(quad >> 32)));
  h.y = Rng::quad_hash((uint32_t)q1, rng.key((uint32_t)(q1 >> 32)));
  h.z = Rng::quad_hash((uint32_t)q2, rng.key((uint32_t)(q2 >> 32)));
  return h;
}

// The same encoder with its rows loaded straight into registers, one tile per block: under STOCHASTIC
// rounding the kernel is bound by instruction issue, not by bytes in flight, and the 32 resident warps
// this form allows (against 24 with a staged tile) are worth more than the staging.
// OFF = position of every octet's first counter in its quad of counters: rows and octets start at
// multiples of eight values, so it is rng_offset & 3 for the whole launch and the host picks the
// instantiation (one copy of the quantizer per row instead of four behind a branch).
// FULL: all 32 rows and all 64 feature octets of the block's tile exist and the chunk size is a power of two
// (decided once per block): no guards, chunk indices by a shift.
template <int K, int LAYOUT, int RANGE, int ROUND, int OFF, bool FULL>
__device__ __forceinline__ void strided_encode_direct_tile(const CodecArgs& a, const ChunkRecord* rec) {
  const int tid = threadIdx.x, lane = tid & 31, sub = tid & 3;
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t fo = blockIdx.x * kStridedOctetsPerBlock + (tid >> 2);  // feature octet
  const bool active = (uint64_t)fo * 8 < F;                              // inactive lanes still shuffle
  const uint64_t g = blockIdx.y;
  const uint64_t word0 = (g * F + (uint64_t)fo * 8) * K;  // first word of feature 8*fo of this batch group
  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  // key of the quads of this thread's first row; a later row almost always shares the upper word of its quad index
  const uint64_t row0 = g * 32 + sub * 8;
  uint32_t key_hi = (uint32_t)((a.rng_offset + row0 * F + (uint64_t)fo * 8) >> 34);
  uint32_t key = rng.key(key_hi);

  uint32_t xlo[8], xhi[8];  // per row: codes of features 0..3 / 4..7
  // four rows at a time: 128 bytes in flight per thread at half the registers, so that more blocks
  // stay resident
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    float v[4][8];
    bool in[4];
    float2 constants[4];  // {inv (its sign bit: the chunk is non-finite), base}
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const uint64_t row = row0 + half * 4 + r;
      in[r] = FULL || (active && row < n_rows);
      if (in[r]) {
        const uint64_t i0 = row * F + (uint64_t)fo * 8;
        ld_octet(a.x + i0, v[r]);
        const uint64_t m = FULL ? (i0 >> a.chunk_shift) : chunk_of(a, i0);
        constants[r] = ldg_c(reinterpret_cast<const float2*>(&rec[m].inv));
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int rr = half * 4 + r;
      xlo[rr] = 0; xhi[rr] = 0;
      if (in[r]) {
        const uint64_t i0 = (row0 + rr) * F + (uint64_t)fo * 8;
        Scale sc;
        sc.s = 0.0f; sc.o = 0.0f;
        sc.inv = fabsf(constants[r].x);
        sc.base = constants[r].y;
        sc.nonfinite = (__float_as_uint(constants[r].x) >> 31) != 0u;
        if (sc.nonfinite) {
#pragma unroll
          for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
        }
        uint32_t b[8];
        if (ROUND == kStochastic) {
          const uint64_t quad = (a.rng_offset + i0) >> 2;
          const uint32_t quad_lo = (uint32_t)quad, quad_hi = (uint32_t)(quad >> 32);
          if (quad_hi != key_hi) { key_hi = quad_hi; key = rng.key(quad_hi); }
          uint32_t h[3];
          if (quad_lo <= 0xFFFFFFFFu - 4u) {
#pragma unroll
            for (int p = 0; p < 3; ++p) h[p] = (p < 2 || OFF != 0) ? Rng::quad_hash(quad_lo + p, key) : 0u;
          } else {
            const uint3 t = strided_quad_hashes_slowly(rng, quad);
            h[0] = t.x; h[1] = t.y; h[2] = t.z;
          }
          quantize_octet_hashed<K, RANGE, OFF>(v[r], sc, h, b);
          xlo[rr] = pack_bytes<3>(b[0], b[1], b[2], b[3]);
          xhi[rr] = pack_bytes<3>(b[4], b[5], b[6], b[7]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) b[e] = quantize_nearest_word<K, RANGE>(v[r][e], sc);
          xlo[rr] = pack_bytes<0>(b[0], b[1], b[2], b[3]);
          xhi[rr] = pack_bytes<0>(b[4], b[5], b[6], b[7]);
        }
      }
    }
  }
  strided_store_tile<K, LAYOUT>(a, xlo, xhi, word0, active, sub, lane);
}

template <int K, int LAYOUT, int RANGE, int ROUND, int OFF>
__global__ void __launch_bounds__(256, 4) strided_encode_direct_kernel(const CodecArgs a, const ChunkRecord* rec) {
  grid_dependency_handshake();
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    st_c(a.header + tid, header_word(a, tid));
    if ((a.n_chunks & 1) && tid < 2) st_c(reinterpret_cast<uint32_t*>(a.meta + a.n_chunks) + tid, 0u);
  }
  const uint64_t n_rows = a.n / a.group_stride;
  const bool full = a.chunk_shift >= 0 && ((uint64_t)blockIdx.y + 1) * 32 <= n_rows &&
                    ((uint64_t)blockIdx.x + 1) * kStridedOctetsPerBlock * 8 <= a.group_stride;
  if (full) strided_encode_direct_tile<K, LAYOUT, RANGE, ROUND, OFF, true>(a, rec);
  else strided_encode_direct_tile<K, LAYOUT, RANGE, ROUND, OFF, false>(a, rec);
}

// FULL: all 32 rows and all 64 feature octets of the block's tile exist and the side words are staged (decided
// once per block): no guards.
template <int K, int LAYOUT, int RANGE, bool FULL>
__device__ __forceinline__ void strided_decode_tile(const CodecArgs& a) {
  const int tid = threadIdx.x, lane = tid & 31, sub = tid & 3;
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t fo = blockIdx.x * kStridedOctetsPerBlock + (tid >> 2);
  const bool active = FULL || (uint64_t)fo * 8 < F;
  const uint64_t g = blockIdx.y;
  const uint64_t word0 = (g * F + (uint64_t)fo * 8) * K;

  // Side words of the block's 32 row segments (512 values each), fetched once per block: with chunks of at
  // least 512 values a segment touches at most two chunks, so 64 threads fetch {first chunk, next chunk} of
  // a row each and everybody reads them from shared memory (instead of eight global loads per thread).
  // s_bound[r] = the octet column of the tile at which row r's second chunk starts (255: none).
  __shared__ float2 s_so[32][2];
  __shared__ __align__(8) uint8_t s_bound[32];
  const bool staged = FULL || a.chunk >= 8u * kStridedOctetsPerBlock;
  if (staged && tid < 64) {
    const int r = tid >> 1, which = tid & 1;
    const uint64_t row = g * 32 + r;
    if (FULL || row < n_rows) {
      const uint64_t first = row * F + (uint64_t)blockIdx.x * kStridedOctetsPerBlock * 8;
      const uint64_t c0 = chunk_of(a, first);
      const uint64_t c = c0 + which < a.n_chunks ? c0 + which : c0;
      s_so[(r & 7) * 4 + (r >> 3)][which] = ldg_c(a.meta + c);  // row 8 b + i at slot 4 i + b: see the read below
      if (which == 0) {
        const uint64_t to_next = (c0 + 1) * a.chunk - first;  // a multiple of 8: chunks are multiples of 32, rows and tiles of 8
        s_bound[r] = to_next < 8u * kStridedOctetsPerBlock ? (uint8_t)(to_next / 8) : (uint8_t)255;
      }
    }
  }

  uint32_t ylo[8], yhi[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const uint32_t* group_words = a.payload + word0 + (uint64_t)e * K;
    if (LAYOUT == kBitplane && K == 8) {
      uint32_t w0 = 0, w1 = 0;
      if (active) { w0 = ldg_c(group_words + sub); w1 = ldg_c(group_words + 4 + sub); }
      const uint32_t lo = planes_nibbles(quad_transpose(w0, lane));  // digits 0..3 of my eight rows
      const uint32_t hi = planes_nibbles(quad_transpose(w1, lane));  // digits 4..7
      ylo[e] = (lo & 0x0F0F0F0Fu) | ((hi & 0x0F0F0F0Fu) << 4);
      yhi[e] = ((lo >> 4) & 0x0F0F0F0Fu) | (hi & 0xF0F0F0F0u);
    } else if (LAYOUT == kBitplane) {
      uint32_t w = 0;
      if (active && sub < K) w = ldg_c(group_words + sub);
      const uint32_t nib = planes_nibbles(quad_transpose(w, lane));  // digits of my eight rows
      ylo[e] = nib & 0x0F0F0F0Fu;
      yhi[e] = (nib >> 4) & 0x0F0F0F0Fu;
    } else if (K == 8) {
      uint2 w = make_uint2(0u, 0u);
      if (active) w = ldg_c(reinterpret_cast<const uint2*>(group_words) + sub);
      ylo[e] = w.x;
      yhi[e] = w.y;
    } else if (K == 4) {
      uint32_t word = 0;
      if (active) word = ldg_c(group_words + sub);
      uint32_t y = __byte_perm(word, 0, 0x4140);
      ylo[e] = (y | (y << 4)) & 0x0F0F0F0Fu;
      y = __byte_perm(word, 0, 0x4342);
      yhi[e] = (y | (y << 4)) & 0x0F0F0F0Fu;
    } else {
      uint32_t half = 0;
      if (active) half = ldg_c(reinterpret_cast<const uint16_t*>(group_words) + sub);
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
  if (staged) __syncthreads();
  uint2 bounds = make_uint2(0u, 0u);  // the boundaries of this thread's eight rows, a byte each
  if (staged) bounds = *reinterpret_cast<const uint2*>(&s_bound[sub * 8]);
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint64_t row = g * 32 + sub * 8 + r;
    if (FULL || (active && row < n_rows)) {
      const uint64_t i0 = row * F + (uint64_t)fo * 8;
      float2 so;
      if (staged) {
        // both candidates in one read that depends on nothing; the boundary decides
        // (the four row blocks of a warp read four neighbouring 16-byte slots: no two on the same banks)
        const float4 both = *reinterpret_cast<const float4*>(&s_so[r * 4 + sub][0]);
        const bool second = (uint32_t)(tid >> 2) >= ((r < 4 ? bounds.x : bounds.y) >> (8 * (r & 3)) & 0xFFu);
        so = second ? make_float2(both.z, both.w) : make_float2(both.x, both.y);
      } else {
        so = ldg_c(a.meta + chunk_of(a, i0));
      }
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

template <int K, int LAYOUT, int RANGE>
__global__ void __launch_bounds__(256) strided_decode_kernel(const CodecArgs a) {
  grid_dependency_handshake();
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    const uint32_t mask = (tid == 6) ? 0xFFFF00FFu : 0xFFFFFFFFu;
    if ((a.header[tid] & mask) != (header_word(a, tid) & mask)) atomicOr(a.status, kDevBadHeader);
  }
  const uint64_t n_rows = a.n / a.group_stride;
  // (measured: the path without guards is faster for bit planes, 41.1 -> 40.3 us on 64 x 802816 at k = 4, and slower
  // for interleaved fields, 40.0 -> 41.7 us, which therefore keep the guarded form for every tile)
  const bool full = LAYOUT == kBitplane && a.chunk >= 8u * kStridedOctetsPerBlock && ((uint64_t)blockIdx.y + 1) * 32 <= n_rows &&
                    ((uint64_t)blockIdx.x + 1) * kStridedOctetsPerBlock * 8 <= a.group_stride;
  if (LAYOUT == kBitplane && full) strided_decode_tile<K, LAYOUT, RANGE, true>(a);
  else strided_decode_tile<K, LAYOUT, RANGE, false>(a);
}

// ----------------------------------------------------------------------------- any shape
//
// Batch groups for any number of values per sample (rows then start at any multiple of four bytes, so there
// are no 32-byte row loads) and for eight bit planes: a thread owns ONE feature and walks down the 32 rows of
// a batch group, so consecutive lanes read consecutive floats of a row (128 bytes per warp instruction,
// whatever the alignment) and a thread ends up with all 32 codes of its group: the k words are formed in the
// thread's own registers and written as one run of k words per lane.  Per element: the chunk's constants from
// the record (neighbouring lanes nearly always share it), one quantizer step, k bit insertions.

constexpr int kStridedAnyBlock = 256;  // features per block

// The codes of rows 8 B .. 8 B + 7 of a thread's group into the group's words.  Bit planes: the eight codes as
// nibbles of one word (two words for eight digits), a 4 x 8 bit-matrix transpose, and byte j of the result is
// digit j of the eight rows: bits 8 B .. 8 B + 7 of word j.  Interleaved: K bits per row at a place fixed by B.
template <int K, int LAYOUT, int B>
__device__ __forceinline__ void strided_any_place(const uint32_t (&u)[8], uint32_t (&word)[K]) {
  if (LAYOUT == kBitplane) {
    uint32_t lo = 0, hi = 0;  // nibble form: byte b = code b in the low, code 4 + b in the high nibble
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      lo |= ((u[b] & 0xFu) | ((u[4 + b] & 0xFu) << 4)) << (8 * b);
      if (K > 4) hi |= ((u[b] >> 4) | ((u[4 + b] >> 4) << 4)) << (8 * b);
    }
    lo = planes_nibbles(lo);
    if (K > 4) hi = planes_nibbles(hi);
#pragma unroll
    for (int j = 0; j < K; ++j) word[j] |= (((j < 4 ? lo : hi) >> (8 * (j & 3))) & 0xFFu) << (8 * B);
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      constexpr int per_word = 32 / K;
      const int r = 8 * B + q;
      word[r / per_word] |= u[q] << (K * (r % per_word));
    }
  }
}

// Chunk of element e; POW2: the chunk size is a power of two (decided once per thread, not per element).
template <bool POW2>
__device__ __forceinline__ uint64_t strided_any_chunk(const CodecArgs& a, uint64_t e) {
  return POW2 ? (e >> a.chunk_shift) : (e / a.chunk);
}

// The random word of counter ctr with the key of its upper word kept from one counter to the next (a thread's
// counters are F apart: the upper 32 bits of the group index change once in 2^34 counters).
struct StridedAnyKey {
  uint32_t hi, key;
};
__device__ __forceinline__ uint32_t strided_any_word(const Rng& rng, StridedAnyKey& k, uint64_t ctr) {
  const uint64_t quad = ctr >> 2;
  const uint32_t hi = (uint32_t)(quad >> 32);
  if (hi != k.hi) { k.hi = hi; k.key = rng.key(hi); }
  const uint32_t h = Rng::quad_hash((uint32_t)quad, k.key);
  const int m = (int)(ctr & 3);
  return m == 0 ? h : h * (m == 1 ? 0x9E3779B1u : (m == 2 ? 0x85EBCA77u : 0xC2B2AE3Du));
}

// Rows 8 B .. 8 B + 7 of the thread's group.  FULL: all eight exist (no guards).
template <int K, int LAYOUT, int RANGE, int ROUND, int B, bool POW2, bool FULL>
__device__ __forceinline__ void strided_any_encode_eight(const CodecArgs& a, const ChunkRecord* rec, const Rng& rng, StridedAnyKey& key,
                                                         uint64_t row0, uint64_t n_rows, uint32_t f, uint32_t (&word)[K]) {
  const uint32_t F = a.group_stride;
  const uint64_t i0 = row0 * F + f;
  float v[8];
  float2 constants[8];  // {inv (its sign bit: the chunk is non-finite), base}
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    v[q] = 0.0f;
    constants[q] = make_float2(0.0f, 0.0f);
    if (FULL || row0 + q < n_rows) {
      const uint64_t i = i0 + (uint64_t)q * F;
      v[q] = ldg_c(a.x + i);
      constants[q] = ldg_c(reinterpret_cast<const float2*>(&rec[strided_any_chunk<POW2>(a, i)].inv));
    }
  }
  uint32_t u[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    u[q] = 0u;
    if (FULL || row0 + q < n_rows) {
      Scale sc;
      sc.s = 0.0f; sc.o = 0.0f;
      sc.inv = fabsf(constants[q].x);
      sc.base = constants[q].y;
      sc.nonfinite = (__float_as_uint(constants[q].x) >> 31) != 0u;
      const float x = sc.nonfinite ? 0.0f : v[q];
      uint32_t h = 0;
      if (ROUND == kStochastic) h = strided_any_word(rng, key, a.rng_offset + i0 + (uint64_t)q * F);
      u[q] = quantize_code<K, RANGE, ROUND>(x, sc, h);
    }
  }
  strided_any_place<K, LAYOUT, B>(u, word);
}

template <int K, int LAYOUT, int RANGE, int ROUND, int B, bool POW2>
__device__ __forceinline__ void strided_any_encode_rows(const CodecArgs& a, const ChunkRecord* rec, const Rng& rng, StridedAnyKey& key,
                                                        uint64_t g, uint64_t n_rows, uint32_t f, uint32_t (&word)[K]) {
  const uint64_t row0 = g * 32 + 8 * B;
  if (row0 >= n_rows) return;  // rows past the last are zero bits
  if (row0 + 8 <= n_rows) strided_any_encode_eight<K, LAYOUT, RANGE, ROUND, B, POW2, true>(a, rec, rng, key, row0, n_rows, f, word);
  else strided_any_encode_eight<K, LAYOUT, RANGE, ROUND, B, POW2, false>(a, rec, rng, key, row0, n_rows, f, word);
}

template <int K, int LAYOUT, int RANGE, int ROUND, bool POW2>
__device__ __forceinline__ void strided_any_encode_group(const CodecArgs& a, const ChunkRecord* rec, const Rng& rng, uint64_t g,
                                                         uint64_t n_rows, uint32_t f, uint32_t (&word)[K]) {
  StridedAnyKey key;
  key.hi = (uint32_t)((a.rng_offset + g * 32 * a.group_stride + f) >> 34);
  key.key = rng.key(key.hi);
  strided_any_encode_rows<K, LAYOUT, RANGE, ROUND, 0, POW2>(a, rec, rng, key, g, n_rows, f, word);
  strided_any_encode_rows<K, LAYOUT, RANGE, ROUND, 1, POW2>(a, rec, rng, key, g, n_rows, f, word);
  strided_any_encode_rows<K, LAYOUT, RANGE, ROUND, 2, POW2>(a, rec, rng, key, g, n_rows, f, word);
  strided_any_encode_rows<K, LAYOUT, RANGE, ROUND, 3, POW2>(a, rec, rng, key, g, n_rows, f, word);
}

template <int K, int LAYOUT, int RANGE, int ROUND>
__global__ void __launch_bounds__(kStridedAnyBlock) strided_encode_any_kernel(const CodecArgs a, const ChunkRecord* rec) {
  grid_dependency_handshake();
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    st_c(a.header + tid, header_word(a, tid));
    if ((a.n_chunks & 1) && tid < 2) st_c(reinterpret_cast<uint32_t*>(a.meta + a.n_chunks) + tid, 0u);
  }
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t f = blockIdx.x * kStridedAnyBlock + tid;
  if (f >= F) return;
  const uint64_t g = blockIdx.y;
  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  uint32_t word[K];
#pragma unroll
  for (int j = 0; j < K; ++j) word[j] = 0u;
  // eight rows at a time: their values and constants are requested together, then coded
  if (a.chunk_shift >= 0) strided_any_encode_group<K, LAYOUT, RANGE, ROUND, true>(a, rec, rng, g, n_rows, f, word);
  else strided_any_encode_group<K, LAYOUT, RANGE, ROUND, false>(a, rec, rng, g, n_rows, f, word);
  // (the payload starts 16-byte aligned and a group is K words: whole groups move as one access where K allows)
  uint32_t* out = a.payload + (g * F + f) * K;
  if (K == 4) {
    st_c(reinterpret_cast<uint4*>(out), make_uint4(word[0], word[1], word[2 % K], word[3 % K]));
  } else if (K == 8) {
    st_c(reinterpret_cast<uint4*>(out), make_uint4(word[0], word[1], word[2 % K], word[3 % K]));
    st_c(reinterpret_cast<uint4*>(out) + 1, make_uint4(word[4 % K], word[5 % K], word[6 % K], word[7 % K]));
  } else if (K == 2) {
    st_c(reinterpret_cast<uint2*>(out), make_uint2(word[0], word[1]));
  } else {
#pragma unroll
    for (int j = 0; j < K; ++j) st_c(out + j, word[j]);
  }
}

// The inverse of strided_any_place: the codes of rows 8 B .. 8 B + 7 out of the group's words.
template <int K, int LAYOUT, int B>
__device__ __forceinline__ void strided_any_take(const uint32_t (&word)[K], uint32_t (&u)[8]) {
  if (LAYOUT == kBitplane) {
    uint32_t lo = 0, hi = 0;  // plane form: byte j = digit j of the eight rows
#pragma unroll
    for (int j = 0; j < K; ++j) {
      const uint32_t byte = (word[j] >> (8 * B)) & 0xFFu;
      if (j < 4) lo |= byte << (8 * j);
      else hi |= byte << (8 * (j - 4));
    }
    lo = planes_nibbles(lo);
    if (K > 4) hi = planes_nibbles(hi);
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      u[b] = (lo >> (8 * b)) & 0xFu;
      u[4 + b] = (lo >> (8 * b + 4)) & 0xFu;
      if (K > 4) {
        u[b] |= ((hi >> (8 * b)) & 0xFu) << 4;
        u[4 + b] |= ((hi >> (8 * b + 4)) & 0xFu) << 4;
      }
    }
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      constexpr int per_word = 32 / K;
      const int r = 8 * B + q;
      u[q] = (word[r / per_word] >> (K * (r % per_word))) & ((1u << K) - 1u);
    }
  }
}

template <int K, int LAYOUT, int RANGE, int B, bool POW2, bool FULL>
__device__ __forceinline__ void strided_any_decode_eight(const CodecArgs& a, uint64_t row0, uint64_t n_rows, uint32_t f,
                                                         const uint32_t (&word)[K]) {
  const uint32_t F = a.group_stride;
  const uint64_t i0 = row0 * F + f;
  float2 so[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    so[q] = make_float2(0.0f, 0.0f);
    if (FULL || row0 + q < n_rows) so[q] = ldg_c(a.meta + strided_any_chunk<POW2>(a, i0 + (uint64_t)q * F));
  }
  uint32_t u[8];
  strided_any_take<K, LAYOUT, B>(word, u);
#pragma unroll
  for (int q = 0; q < 8; ++q)
    if (FULL || row0 + q < n_rows) st_c(a.xhat + i0 + (uint64_t)q * F, dequantize_code<K, RANGE>(u[q], so[q].x, so[q].y));
}

template <int K, int LAYOUT, int RANGE, int B, bool POW2>
__device__ __forceinline__ void strided_any_decode_rows(const CodecArgs& a, uint64_t g, uint64_t n_rows, uint32_t f,
                                                        const uint32_t (&word)[K]) {
  const uint64_t row0 = g * 32 + 8 * B;
  if (row0 >= n_rows) return;
  if (row0 + 8 <= n_rows) strided_any_decode_eight<K, LAYOUT, RANGE, B, POW2, true>(a, row0, n_rows, f, word);
  else strided_any_decode_eight<K, LAYOUT, RANGE, B, POW2, false>(a, row0, n_rows, f, word);
}

template <int K, int LAYOUT, int RANGE, bool POW2>
__device__ __forceinline__ void strided_any_decode_group(const CodecArgs& a, uint64_t g, uint64_t n_rows, uint32_t f,
                                                         const uint32_t (&word)[K]) {
  strided_any_decode_rows<K, LAYOUT, RANGE, 0, POW2>(a, g, n_rows, f, word);
  strided_any_decode_rows<K, LAYOUT, RANGE, 1, POW2>(a, g, n_rows, f, word);
  strided_any_decode_rows<K, LAYOUT, RANGE, 2, POW2>(a, g, n_rows, f, word);
  strided_any_decode_rows<K, LAYOUT, RANGE, 3, POW2>(a, g, n_rows, f, word);
}

template <int K, int LAYOUT, int RANGE>
__global__ void __launch_bounds__(kStridedAnyBlock) strided_decode_any_kernel(const CodecArgs a) {
  grid_dependency_handshake();
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 8) {
    const uint32_t mask = (tid == 6) ? 0xFFFF00FFu : 0xFFFFFFFFu;
    if ((a.header[tid] & mask) != (header_word(a, tid) & mask)) atomicOr(a.status, kDevBadHeader);
  }
  const uint32_t F = a.group_stride;
  const uint64_t n_rows = a.n / F;
  const uint32_t f = blockIdx.x * kStridedAnyBlock + tid;
  if (f >= F) return;
  const uint64_t g = blockIdx.y;
  const uint32_t* in = a.payload + (g * F + f) * K;
  uint32_t word[K];
  if (K == 4) {
    const uint4 w = ldg_c(reinterpret_cast<const uint4*>(in));
    word[0] = w.x; word[1] = w.y; word[2 % K] = w.z; word[3 % K] = w.w;
  } else if (K == 8) {
    const uint4 w = ldg_c(reinterpret_cast<const uint4*>(in)), x = ldg_c(reinterpret_cast<const uint4*>(in) + 1);
    word[0] = w.x; word[1] = w.y; word[2 % K] = w.z; word[3 % K] = w.w;
    word[4 % K] = x.x; word[5 % K] = x.y; word[6 % K] = x.z; word[7 % K] = x.w;
  } else if (K == 2) {
    const uint2 w = ldg_c(reinterpret_cast<const uint2*>(in));
    word[0] = w.x; word[1] = w.y;
  } else {
#pragma unroll
    for (int j = 0; j < K; ++j) word[j] = ldg_c(in + j);
  }
  if (a.chunk_shift >= 0) strided_any_decode_group<K, LAYOUT, RANGE, true>(a, g, n_rows, f, word);
  else strided_any_decode_group<K, LAYOUT, RANGE, false>(a, g, n_rows, f, word);
}

}  // namespace accept
