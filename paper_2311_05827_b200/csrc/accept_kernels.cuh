// Kernels of the boundary-tensor codec: fused range + quantize + pack (compress) and fused
// unpack + dequantize (decompress).  One launch per call; chunks are independent, so no block ever
// waits on another.
#pragma once
#include "accept_device.cuh"

namespace accept {

struct CodecArgs {
  const float* x;         // compress input
  float* xhat;            // decompress output
  uint32_t* header;       // stream + 0
  float2* meta;           // stream + 32
  uint32_t* payload;      // stream + payload offset
  uint32_t* status;       // device status word
  uint64_t n;             // elements
  uint64_t n_chunks;      // M
  uint64_t n_fast_chunks; // leading full chunks coded by the register-resident path
  uint64_t seed, rng_offset;
  uint32_t chunk;         // C
  int chunk_shift;        // log2(C) if C is a power of two, else -1
  uint32_t tpc;           // fast path: threads that share one chunk (C / (8*R))
  int tpc_shift;          // log2(tpc) when a block holds several chunks (tpc divides 256), else unused
  uint32_t chunks_per_block;
  uint32_t fast_blocks;   // blocks of the register-resident path; later blocks take the any-shape coder
  uint32_t header_word6;  // range | round<<8 | layout<<16
  uint32_t k;
  uint32_t group_stride;  // 0, or values per sample when pack groups run along the batch dimension
};

// Word i of the 32-byte stream header.
__device__ __forceinline__ uint32_t header_word(const CodecArgs& a, int i) {
  switch (i) {
    case 0: return 0x54504341u;
    case 1: return 1u;
    case 2: return (uint32_t)a.n;
    case 3: return (uint32_t)(a.n >> 32);
    case 4: return a.chunk;
    case 5: return a.k;
    case 6: return a.header_word6;
    default: return a.group_stride;
  }
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may be
// scheduled while the kernel before it in the stream is still draining.  Every kernel here waits
// for that predecessor (and the visibility of its writes) before it touches memory, and lets its
// own successor be scheduled right away: what overlaps is launch latency and the tail of the grid.
__device__ __forceinline__ void grid_dependency_handshake() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Nothing but the handshake every kernel starts with: what a launch of this library costs (accept_launch_null).
__global__ void null_kernel() { grid_dependency_handshake(); }

constexpr int kFastBlock = 128;     // threads per block when a chunk needs at most 128 threads (finer tail than 256: measured)
constexpr int kGenericBlock = 256;  // threads per block of the any-shape path

// ----------------------------------------------------------------------------- stores of packed codes

// INTERLEAVED: the 8 codes of global octet index oct occupy bits [8*K*oct, 8*K*(oct+1)) of the payload.
template <int K>
__device__ __forceinline__ void store_interleaved(uint32_t* payload, uint64_t oct, uint32_t xlo, uint32_t xhi) {
  if (K == 8) {
    st_c(reinterpret_cast<uint2*>(payload) + oct, make_uint2(xlo, xhi));
  } else if (K == 4) {
    // bytes u0|u1<<4 and u2|u3<<4 sit in bytes 0 and 2 of x | x>>4
    const uint32_t ylo = xlo | (xlo >> 4), yhi = xhi | (xhi >> 4);
    st_c(payload + oct, __byte_perm(ylo, yhi, 0x6420));
  } else {  // K == 2
    uint32_t ylo = xlo | (xlo >> 6), yhi = xhi | (xhi >> 6);
    ylo |= ylo >> 12;
    yhi |= yhi >> 12;
    st_c(reinterpret_cast<uint16_t*>(payload) + oct, (uint16_t)__byte_perm(ylo, yhi, 0x0040));
  }
}

// BITPLANE: lane q of a quad ends with the word of binary digit q (and q+4 for K = 8) of the
// quad's group and stores it.  group = global index of the 32-element group.  All lanes call.
// Returns the word of binary digit q = lane & 3 of the quad's group (K <= 4; 0 for K = 8).
template <int K>
__device__ __forceinline__ uint32_t store_bitplane_guarded(uint32_t* payload, uint64_t group, uint32_t xlo, uint32_t xhi,
                                                           int lane, bool store) {
  const int q = lane & 3;
  if (K <= 4) {
    const uint32_t w = quad_transpose(planes_nibbles(merge_nibbles(xlo, xhi)), lane);
    if (store && q < K) st_c(payload + group * K + q, w);
    return w;
  } else {
    const uint32_t lo = merge_nibbles(xlo & 0x0F0F0F0Fu, xhi & 0x0F0F0F0Fu);
    const uint32_t hi = merge_nibbles((xlo >> 4) & 0x0F0F0F0Fu, (xhi >> 4) & 0x0F0F0F0Fu);
    const uint32_t w0 = quad_transpose(planes_nibbles(lo), lane);
    const uint32_t w1 = quad_transpose(planes_nibbles(hi), lane);
    if (store) {
      st_c(payload + group * 8 + q, w0);
      st_c(payload + group * 8 + 4 + q, w1);
    }
    return 0u;
  }
}

template <int K>
__device__ __forceinline__ void store_bitplane(uint32_t* payload, uint64_t group, uint32_t xlo, uint32_t xhi,
                                               int lane) {
  store_bitplane_guarded<K>(payload, group, xlo, xhi, lane, true);
}

// ----------------------------------------------------------------------------- any-shape chunk coder

// Codes chunk m with the whole block: any C (multiple of 32), partial chunks, any alignment.
// Two passes over the chunk (the second is served by the caches); one element per lane, words
// formed with warp votes.  Used for the partial last chunk and for chunk sizes or alignments the
// register-resident path does not take.
template <int K, int LAYOUT, int RANGE, int ROUND>
__device__ void compress_chunk_generic(const CodecArgs& a, uint64_t m, float* s_hi, float* s_lo) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint64_t i0 = m * a.chunk;
  const uint32_t valid = (uint32_t)min((uint64_t)a.chunk, a.n - i0);
  const float* x = a.x + i0;

  Range<RANGE> rg;
  rg.init();
  for (uint32_t i = tid; i < valid; i += blockDim.x) rg.add(ldg_c(x + i));
  rg.warp_reduce();
  __syncthreads();  // protects s_hi/s_lo against a previous use
  if (lane == 0) { s_hi[warp] = rg.hi; s_lo[warp] = rg.lo; }
  __syncthreads();
  rg.init();
  for (int w = 0; w < nwarps; ++w) rg.merge(s_hi[w], s_lo[w]);

  Scale sc = make_scale<K, RANGE>(rg.hi, rg.lo);
  if (tid == 0) {
    st_c(a.meta + m, make_float2(sc.s, sc.o));
    if (sc.nonfinite) atomicOr(a.status, kDevNonFinite);
  }
  Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  const uint32_t ngroups = (valid + 31) / 32;
  for (uint32_t g = warp; g < ngroups; g += nwarps) {
    const uint32_t t = g * 32 + lane;
    uint32_t u = 0;
    if (t < valid) {
      float v = ldg_c(x + t);
      if (sc.nonfinite) v = 0.0f;
      uint32_t h = 0;
      if (ROUND == kStochastic) h = rng.word(a.rng_offset + i0 + t);
      u = quantize_code<K, RANGE, ROUND>(v, sc, h);
    }
    const uint64_t word0 = (i0 / 32 + g) * K;
#pragma unroll
    for (int w = 0; w < K; ++w) {
      uint32_t bit;
      if (LAYOUT == kBitplane) {
        bit = (u >> w) & 1u;  // word w = binary digit w of the 32 codes
      } else {
        // bit b of word w is bit (32w+b) of the group's string: digit (32w+b)%K of element (32w+b)/K
        const int pos = 32 * w + lane;
        bit = (__shfl_sync(0xffffffffu, u, pos / K) >> (pos % K)) & 1u;
      }
      const uint32_t word = __ballot_sync(0xffffffffu, bit);
      if (lane == w) st_c(a.payload + word0 + w, word);
    }
  }
}

// ----------------------------------------------------------------------------- compress

// Register-resident path.  A chunk of C = 8*R*tpc elements is shared by tpc threads (tpc a multiple
// of 32, the block holds chunks_per_block such groups).  Each thread loads R octets, one per round,
// round r covering elements [8*r*tpc, 8*(r+1)*tpc) of the chunk with consecutive threads on
// consecutive octets; the chunk is read from HBM once and stays in registers between the range
// reduction and the quantizer.  Blocks past the fast chunks code the remaining chunk(s) with the
// any-shape coder.
// BLOCK_MAX is the largest block the instantiation is launched with (256 or 1024); the smaller
// bound lets the compiler keep six (R <= 2) or four (R = 4) blocks resident per SM.
template <int K, int LAYOUT, int RANGE, int ROUND, int R, int BLOCK_MAX>
__global__ void __launch_bounds__(BLOCK_MAX, BLOCK_MAX == 256 ? (R <= 2 ? 6 : 4) : 1) compress_kernel(const CodecArgs a) {
  __shared__ float s_hi[32], s_lo[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  grid_dependency_handshake();

  if (blockIdx.x == 0 && tid < 8) {
    // stream header and the pad between the side words and the payload
    st_c(a.header + tid, header_word(a, tid));
    if ((a.n_chunks & 1) && tid < 2) st_c(reinterpret_cast<uint32_t*>(a.meta + a.n_chunks) + tid, 0u);
  }

  if (blockIdx.x >= a.fast_blocks) {
    compress_chunk_generic<K, LAYOUT, RANGE, ROUND>(a, a.n_fast_chunks + (blockIdx.x - a.fast_blocks), s_hi, s_lo);
    return;
  }

  const uint32_t tpc = a.tpc;
  const uint32_t grp = (a.chunks_per_block > 1) ? (tid >> a.tpc_shift) : 0u, gt = tid - grp * tpc;
  uint64_t m = (uint64_t)blockIdx.x * a.chunks_per_block + grp;
  const bool active = m < a.n_fast_chunks;  // a whole group is active or not; warps never straddle groups
  if (!active) m = a.n_fast_chunks - 1;     // idle groups redo the last chunk's loads, store nothing

  const uint64_t e0 = m * a.chunk;  // first element of the chunk
  float v[R][8];
#pragma unroll
  for (int r = 0; r < R; ++r) ld_octet(a.x + e0 + 8ull * (r * tpc + gt), v[r]);

  Range<RANGE> rg;
  rg.init();
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int e = 0; e < 8; e += 2) rg.add2(v[r][e], v[r][e + 1]);
  }
  rg.warp_reduce();
  if (tpc > 32) {
    if (lane == 0) { s_hi[warp] = rg.hi; s_lo[warp] = rg.lo; }
    __syncthreads();
    // lane w of every warp picks up the partial of the group's warp w; a second butterfly
    // leaves the chunk's range in every lane
    const int w0 = (grp * tpc) >> 5, wn = tpc >> 5;
    rg.init();
    if (lane < wn) { rg.hi = s_hi[w0 + lane]; rg.lo = s_lo[w0 + lane]; }
    rg.warp_reduce();
  }

  Scale sc = make_scale<K, RANGE>(rg.hi, rg.lo);
  if (gt == 0 && active) {
    st_c(a.meta + m, make_float2(sc.s, sc.o));
    if (sc.nonfinite) atomicOr(a.status, kDevNonFinite);
  }
  if (sc.nonfinite) {
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
  }

  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  RngThread rt;
  if (ROUND == kStochastic) rt.init(rng, a.rng_offset + e0 + 8ull * gt, 8u * (R - 1) * tpc + 8u);
  uint32_t xlo[R], xhi[R];
  quantize_rounds<K, RANGE, ROUND, R>(v, sc, rng, rt, 8u * tpc, xlo, xhi);
  // an idle group (whole warps) stores nothing; the bit-plane store shuffles inside a quad, never across warps
  if (!active) return;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint64_t oct = e0 / 8 + (r * tpc + gt);  // global octet index
    if (LAYOUT == kInterleaved) store_interleaved<K>(a.payload, oct, xlo[r], xhi[r]);
    else store_bitplane<K>(a.payload, oct >> 2, xlo[r], xhi[r], lane);
  }
}

// ----------------------------------------------------------------------------- decompress

// What one thread fetches for one octet: its slice of the payload and the chunk's side words.
struct RawOctet {
  uint32_t w0, w1;
  float2 so;
};

template <int K, int LAYOUT>
__device__ __forceinline__ RawOctet load_raw(const CodecArgs& a, uint64_t oct, uint64_t n_oct, uint64_t n_groups,
                                             int lane) {
  RawOctet raw;
  raw.w0 = 0; raw.w1 = 0; raw.so = make_float2(0.0f, 0.0f);
  if (LAYOUT == kInterleaved) {
    if (oct < n_oct) {
      if (K == 8) {
        const uint2 w = ldg_c(reinterpret_cast<const uint2*>(a.payload) + oct);
        raw.w0 = w.x; raw.w1 = w.y;
      } else if (K == 4) {
        raw.w0 = ldg_c(a.payload + oct);
      } else {
        raw.w0 = ldg_c(reinterpret_cast<const uint16_t*>(a.payload) + oct);
      }
    }
  } else {
    // lane q of a quad fetches the word of binary digit q (and q+4) of the quad's group
    const int q = lane & 3;
    const uint64_t group = oct >> 2;
    if (group < n_groups) {
      if (K <= 4) {
        if (q < K) raw.w0 = ldg_c(a.payload + group * K + q);
      } else {
        raw.w0 = ldg_c(a.payload + group * 8 + q);
        raw.w1 = ldg_c(a.payload + group * 8 + 4 + q);
      }
    }
  }
  if (oct < n_oct) {
    const uint64_t e = oct * 8;
    const uint64_t m = (a.chunk_shift >= 0) ? (e >> a.chunk_shift) : (e / a.chunk);
    raw.so = ldg_c(a.meta + m);
  }
  return raw;
}

// Payload slice -> the codes of the octet, one per byte (xlo: elements 0..3, xhi: 4..7).
// BITPLANE shuffles inside a quad: all 32 lanes call.
template <int K, int LAYOUT>
__device__ __forceinline__ void unpack_octet(const RawOctet& raw, int lane, uint32_t& xlo, uint32_t& xhi) {
  if (LAYOUT == kInterleaved) {
    if (K == 8) {
      xlo = raw.w0; xhi = raw.w1;
    } else if (K == 4) {
      uint32_t y = __byte_perm(raw.w0, 0, 0x4140);  // bytes: w.b0, 0, w.b1, 0
      xlo = (y | (y << 4)) & 0x0F0F0F0Fu;           // nibbles -> bytes
      y = __byte_perm(raw.w0, 0, 0x4342);           // bytes: w.b2, 0, w.b3, 0
      xhi = (y | (y << 4)) & 0x0F0F0F0Fu;
    } else {
      const uint32_t w = raw.w0;                    // eight 2-bit fields
      uint32_t y = (w | (w << 12)) & 0x000F000Fu;
      xlo = (y | (y << 6)) & 0x03030303u;
      y = ((w >> 8) | ((w >> 8) << 12)) & 0x000F000Fu;
      xhi = (y | (y << 6)) & 0x03030303u;
    }
  } else {
    // a quad transpose hands every lane the plane bytes of its own octet
    if (K <= 4) {
      const uint32_t nib = planes_nibbles(quad_transpose(raw.w0, lane));
      xlo = nib & 0x0F0F0F0Fu;
      xhi = (nib >> 4) & 0x0F0F0F0Fu;
    } else {
      const uint32_t lo = planes_nibbles(quad_transpose(raw.w0, lane));
      const uint32_t hi = planes_nibbles(quad_transpose(raw.w1, lane));
      xlo = (lo & 0x0F0F0F0Fu) | ((hi & 0x0F0F0F0Fu) << 4);
      xhi = ((lo >> 4) & 0x0F0F0F0Fu) | (hi & 0xF0F0F0F0u);
    }
  }
}

// Decodes and stores the R octets of one tile from the slices fetched earlier.
template <int K, int LAYOUT, int RANGE, int R>
__device__ __forceinline__ void decode_tile(const CodecArgs& a, const RawOctet (&raw)[R], uint64_t first_oct,
                                            uint64_t n_oct, int lane) {
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint64_t oct = first_oct + r * 256;
    uint32_t xlo, xhi;
    unpack_octet<K, LAYOUT>(raw[r], lane, xlo, xhi);
    if (oct < n_oct) {
      const uint64_t e = oct * 8;
      float out[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[i] = dequantize_code<K, RANGE>((xlo >> (8 * i)) & 0xFFu, raw[r].so.x, raw[r].so.y);
        out[4 + i] = dequantize_code<K, RANGE>((xhi >> (8 * i)) & 0xFFu, raw[r].so.x, raw[r].so.y);
      }
      if (e + 8 <= a.n) {
        st_octet(a.xhat + e, out);
      } else {
        for (int i = 0; i < 8; ++i)
          if (e + i < a.n) st_c(a.xhat + e + i, out[i]);
      }
    }
  }
}

// One tile of R*256 octets per block: every thread requests its R payload slices first, then
// decodes and stores them; consecutive threads take consecutive octets, so each store instruction
// of a warp writes 1 KB of contiguous output.  (Grid-stride variants of this kernel that prefetch
// the next tile measured slower than one short-lived block per tile.)
template <int K, int LAYOUT, int RANGE, int R>
__global__ void __launch_bounds__(256, R <= 2 ? 8 : 6) decompress_kernel(const CodecArgs a) {
  const int tid = threadIdx.x, lane = tid & 31;
  grid_dependency_handshake();
  if (blockIdx.x == 0 && tid < 8) {
    // the rounding mode (bits 8..15 of word 6) does not change how a stream is read
    const uint32_t mask = (tid == 6) ? 0xFFFF00FFu : 0xFFFFFFFFu;
    if ((a.header[tid] & mask) != (header_word(a, tid) & mask)) atomicOr(a.status, kDevBadHeader);
  }
  const uint64_t n_oct = (a.n + 7) / 8;       // octets, the last one maybe partial
  const uint64_t n_groups = (a.n + 31) / 32;  // pack groups present in the payload
  const uint64_t first_oct = (uint64_t)blockIdx.x * (R * 256) + tid;
  RawOctet raw[R];
#pragma unroll
  for (int r = 0; r < R; ++r) raw[r] = load_raw<K, LAYOUT>(a, first_oct + r * 256, n_oct, n_groups, lane);
  decode_tile<K, LAYOUT, RANGE, R>(a, raw, first_oct, n_oct, lane);
}

// Scalar any-alignment decoder for output pointers that are not 32-byte aligned.
template <int K, int LAYOUT, int RANGE>
__global__ void __launch_bounds__(256) decompress_unaligned_kernel(const CodecArgs a) {
  grid_dependency_handshake();
  const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n) return;
  uint32_t u = 0;
  if (LAYOUT == kInterleaved) {
    const uint64_t bit = i * K;
    u = (ldg_c(a.payload + (bit >> 5)) >> (bit & 31)) & ((1u << K) - 1);
  } else {
    const uint64_t w0 = (i >> 5) * K;
    for (int j = 0; j < K; ++j) u |= ((ldg_c(a.payload + w0 + j) >> (i & 31)) & 1u) << j;
  }
  const uint64_t m = (a.chunk_shift >= 0) ? (i >> a.chunk_shift) : (i / a.chunk);
  const float2 so = ldg_c(a.meta + m);
  st_c(a.xhat + i, dequantize_code<K, RANGE>(u, so.x, so.y));
}

}  // namespace accept
