// Compress for chunks too large to stay in registers (more than 32768 elements, up to one range
// for the whole tensor, which is the paper's own granularity: "Backward Quantizer", c = max|g|).
// Three launches: ranges of all chunks (one pass over the input), per-chunk constants, then
// quantize + pack (a second pass over the input): 8 + k/8 bytes per element instead of 4 + k/8.
#pragma once
#include "accept_kernels.cuh"

namespace accept {

// One record per chunk in the workspace (after its first 16 bytes).  While ranges are gathered,
// a = largest key of max|x| (ABSMAX: the magnitude bits) or of max x (MINMAX: sortable key),
// b = largest complement of the sortable key of min x (MINMAX); both start at 0, so a cleared
// workspace is the identity.  wide_finalize_kernel replaces them by what the encoder needs.
struct ChunkRecord {
  uint32_t a, b;
  float inv, base;
};

// Monotone map from fp32 order to unsigned order; NaNs land above +Inf or below -Inf, so they
// survive a max (or a min) and are seen as non-finite afterwards.
__device__ __forceinline__ uint32_t sortable_key(float f) {
  const uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float from_sortable_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

template <int RANGE>
__device__ __forceinline__ void merge_into_record(ChunkRecord* rec, float hi, float lo) {
  if (!bounds_ok(rec, sizeof(ChunkRecord), true)) return;
  if (RANGE == kAbsMax) {
    atomicMax(&rec->a, __float_as_uint(hi));  // hi = max|x| >= 0 (or NaN): magnitude bits order as integers
  } else {
    atomicMax(&rec->a, sortable_key(hi));
    atomicMax(&rec->b, ~sortable_key(lo));
  }
}

// Loads octet oct of the input (oct*8 < n).  Elements at or past n read as 0, or as a copy of the
// octet's first element when repeat_first is set (neutral for a range).
__device__ __forceinline__ void ld_octet_guarded(const CodecArgs& a, uint64_t oct, bool repeat_first, float (&v)[8]) {
  const uint64_t e = oct * 8;
  if (e + 8 <= a.n) {
    ld_octet(a.x + e, v);
  } else {
    const float fill = repeat_first ? ldg_c(a.x + e) : 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = (e + i < a.n) ? ldg_c(a.x + e + i) : fill;
  }
}

__device__ __forceinline__ uint64_t chunk_of(const CodecArgs& a, uint64_t e) {
  return (a.chunk_shift >= 0) ? (e >> a.chunk_shift) : (e / a.chunk);
}

// Pass 1.  A block reduces a tile of R*256 octets.  When the tile lies in one chunk (all but the
// blocks that sit on a chunk boundary) it issues one atomic per record word; otherwise every
// octet merges on its own.
template <int RANGE, int R>
__global__ void __launch_bounds__(256) wide_range_kernel(const CodecArgs a, ChunkRecord* rec) {
  grid_dependency_handshake();
  __shared__ float s_hi[8], s_lo[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint64_t n_oct = (a.n + 7) / 8;
  const uint64_t oct0 = (uint64_t)blockIdx.x * (R * 256);
  const uint64_t last_oct = min(oct0 + R * 256, n_oct) - 1;
  const uint64_t m_first = chunk_of(a, oct0 * 8), m_last = chunk_of(a, last_oct * 8);
  float v[R][8];
  bool in[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint64_t oct = oct0 + r * 256 + tid;
    in[r] = oct < n_oct;
    if (in[r]) ld_octet_guarded(a, oct, true, v[r]);
  }
  if (m_first == m_last) {
    Range<RANGE> rg;
    rg.init();
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (in[r]) {
#pragma unroll
        for (int e = 0; e < 8; e += 2) rg.add2(v[r][e], v[r][e + 1]);
      }
    rg.warp_reduce();
    if (lane == 0) { s_hi[warp] = rg.hi; s_lo[warp] = rg.lo; }
    __syncthreads();
    if (tid == 0) {
      rg.init();
      for (int w = 0; w < 8; ++w) rg.merge(s_hi[w], s_lo[w]);
      merge_into_record<RANGE>(rec + m_first, rg.hi, rg.lo);
    }
  } else {
    // the tile spans several chunks: a warp's 32 octets of one round (256 consecutive values) usually
    // still lie in one chunk, then the warp reduces and issues one atomic per record word
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const uint64_t m = chunk_of(a, (oct0 + r * 256 + tid) * 8);
      Range<RANGE> rg;
      rg.init();
      if (in[r]) {
#pragma unroll
        for (int e = 0; e < 8; e += 2) rg.add2(v[r][e], v[r][e + 1]);
      }
      const uint64_t m_lane0 = __shfl_sync(0xffffffffu, m, 0);
      const bool uniform = __all_sync(0xffffffffu, in[r] && m == m_lane0);
      if (uniform) {
        rg.warp_reduce();
        if (lane == 0) merge_into_record<RANGE>(rec + m, rg.hi, rg.lo);
      } else if (in[r]) {
        merge_into_record<RANGE>(rec + m, rg.hi, rg.lo);
      }
    }
  }
}

// The range of chunk m -> its side words (to the stream) and the encoder's constants (to the record: a = 1
// if the chunk is non-finite; the same flag is the sign bit of inv, which is never negative otherwise, for
// readers that fetch only inv and base).
template <int RANGE>
__device__ __forceinline__ void store_chunk_constants(const CodecArgs& a, ChunkRecord* rec, uint64_t m, float hi, float lo) {
  Scale sc;
  switch (a.k) {
    case 2: sc = make_scale<2, RANGE>(hi, lo); break;
    case 3: sc = make_scale<3, RANGE>(hi, lo); break;
    case 4: sc = make_scale<4, RANGE>(hi, lo); break;
    default: sc = make_scale<8, RANGE>(hi, lo); break;
  }
  st_c(a.meta + m, make_float2(sc.s, sc.o));
  if (sc.nonfinite) atomicOr(a.status, kDevNonFinite);
  ChunkRecord constants;
  constants.a = sc.nonfinite ? 1u : 0u;
  constants.b = 0u;
  constants.inv = sc.nonfinite ? -0.0f : sc.inv;
  constants.base = sc.base;
  st_c(rec + m, constants);
}

// Pass 2: one thread per chunk turns the gathered range into the side words (written to the
// stream) and the encoder's constants (written over the record: a = 1 if the chunk is non-finite;
// the same flag is the sign bit of inv, which is never negative otherwise, for readers that fetch
// only inv and base).
template <int RANGE>
__global__ void __launch_bounds__(256) wide_finalize_kernel(const CodecArgs a, ChunkRecord* rec) {
  grid_dependency_handshake();
  const uint64_t m = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= a.n_chunks) return;
  float hi, lo = 0.0f;
  const ChunkRecord gathered = ld_c(rec + m);
  if (RANGE == kAbsMax) {
    hi = __uint_as_float(gathered.a);
  } else {
    hi = from_sortable_key(gathered.a);
    lo = from_sortable_key(~gathered.b);
  }
  store_chunk_constants<RANGE>(a, rec, m, hi, lo);
}

// Passes 1 and 2 in one launch for chunks that a block can hold in registers (the geometry of the
// one-launch coder: a chunk of C = 8*R*tpc elements shared by tpc threads): the block reads its chunk(s),
// reduces the range and writes side words and constants itself -- no atomics, so the records need not be
// cleared, and no pass of its own for the constants.  Blocks past the register-resident chunks take the
// remaining chunk(s) (the ragged last one; all of them when C has no such geometry) with a plain loop.
template <int RANGE, int R, int BLOCK_MAX>
__global__ void __launch_bounds__(BLOCK_MAX, BLOCK_MAX == 256 ? (R <= 2 ? 6 : 4) : 1)
    chunk_constants_kernel(const CodecArgs a, ChunkRecord* rec) {
  __shared__ float s_hi[32], s_lo[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  grid_dependency_handshake();
  Range<RANGE> rg;
  rg.init();
  if (blockIdx.x >= a.fast_blocks) {
    const uint64_t m = a.n_fast_chunks + (blockIdx.x - a.fast_blocks);
    const uint64_t i0 = m * a.chunk;
    const uint32_t valid = (uint32_t)min((uint64_t)a.chunk, a.n - i0);
    for (uint32_t i = tid; i < valid; i += blockDim.x) rg.add(ldg_c(a.x + i0 + i));
    rg.warp_reduce();
    if (lane == 0) { s_hi[warp] = rg.hi; s_lo[warp] = rg.lo; }
    __syncthreads();
    if (tid == 0) {
      rg.init();
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) rg.merge(s_hi[w], s_lo[w]);
      store_chunk_constants<RANGE>(a, rec, m, rg.hi, rg.lo);
    }
    return;
  }
  const uint32_t tpc = a.tpc;
  const uint32_t grp = (a.chunks_per_block > 1) ? (tid >> a.tpc_shift) : 0u, gt = tid - grp * tpc;
  uint64_t m = (uint64_t)blockIdx.x * a.chunks_per_block + grp;
  const bool active = m < a.n_fast_chunks;  // a whole group is active or not; warps never straddle groups
  if (!active) m = a.n_fast_chunks - 1;     // idle groups redo the last chunk's loads, store nothing
  const uint64_t e0 = m * a.chunk;
  float v[R][8];
#pragma unroll
  for (int r = 0; r < R; ++r) ld_octet(a.x + e0 + 8ull * (r * tpc + gt), v[r]);
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int e = 0; e < 8; e += 2) rg.add2(v[r][e], v[r][e + 1]);
  }
  rg.warp_reduce();
  if (tpc > 32) {
    if (lane == 0) { s_hi[warp] = rg.hi; s_lo[warp] = rg.lo; }
    __syncthreads();
    const int w0 = (grp * tpc) >> 5, wn = tpc >> 5;
    rg.init();
    if (lane < wn) { rg.hi = s_hi[w0 + lane]; rg.lo = s_lo[w0 + lane]; }
    rg.warp_reduce();
  }
  if (gt == 0 && active) store_chunk_constants<RANGE>(a, rec, m, rg.hi, rg.lo);
}

// Pass 3: quantize + pack with the constants of each octet's chunk.  A tile that lies inside the
// tensor and inside one chunk (all but the tiles on a chunk boundary and the last one) reads its
// record once and skips the per-octet guards.
__device__ __forceinline__ Scale scale_from_record(const ChunkRecord* rec) {
  const uint4 raw = ldg_c(reinterpret_cast<const uint4*>(rec));
  Scale sc;
  sc.s = 0.0f; sc.o = 0.0f;
  sc.inv = fabsf(__uint_as_float(raw.z));
  sc.base = __uint_as_float(raw.w);
  sc.nonfinite = raw.x != 0u;
  return sc;
}

template <int K, int LAYOUT, int RANGE, int ROUND, int R>
__global__ void __launch_bounds__(256, R <= 2 ? 5 : 4) wide_encode_kernel(const CodecArgs a, const ChunkRecord* rec) {
  grid_dependency_handshake();
  const int tid = threadIdx.x, lane = tid & 31;
  if (blockIdx.x == 0 && tid < 8) {
    st_c(a.header + tid, header_word(a, tid));
    if ((a.n_chunks & 1) && tid < 2) st_c(reinterpret_cast<uint32_t*>(a.meta + a.n_chunks) + tid, 0u);
  }
  const uint64_t n_oct_stored = ((a.n + 31) / 32) * 4;  // whole pack groups are stored
  const uint64_t tile_oct = (uint64_t)blockIdx.x * (R * 256);
  const uint64_t oct0 = tile_oct + tid;
  const Rng rng{(uint32_t)a.seed, (uint32_t)(a.seed >> 32)};
  RngThread rt;
  if (ROUND == kStochastic) rt.init(rng, a.rng_offset + oct0 * 8, 8u * (R - 1) * 256u + 8u);

  const uint64_t tile_first = tile_oct * 8, tile_last = tile_first + (uint64_t)R * 256 * 8 - 1;
  const uint64_t tile_chunk = chunk_of(a, tile_first);
  if (tile_last < a.n && chunk_of(a, tile_last) == tile_chunk) {
    float v[R][8];
#pragma unroll
    for (int r = 0; r < R; ++r) ld_octet(a.x + (oct0 + r * 256) * 8, v[r]);
    const Scale sc = scale_from_record(rec + tile_chunk);
    if (sc.nonfinite) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int i = 0; i < 8; ++i) v[r][i] = 0.0f;
    }
    uint32_t xlo[R], xhi[R];
    quantize_rounds<K, RANGE, ROUND, R>(v, sc, rng, rt, 8u * 256u, xlo, xhi);
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const uint64_t oct = oct0 + r * 256;
      if (LAYOUT == kInterleaved) store_interleaved<K>(a.payload, oct, xlo[r], xhi[r]);
      else store_bitplane<K>(a.payload, oct >> 2, xlo[r], xhi[r], lane);
    }
    return;
  }

  float v[R][8];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint64_t oct = oct0 + r * 256;
    if (oct * 8 < a.n) {
      ld_octet_guarded(a, oct, false, v[r]);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint64_t oct = oct0 + r * 256, e = oct * 8;
    const bool stored = oct < n_oct_stored;
    uint32_t xlo = 0, xhi = 0;
    if (e < a.n) {
      const Scale sc = scale_from_record(rec + chunk_of(a, e));
      if (sc.nonfinite) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[r][i] = 0.0f;
      }
      quantize_octet<K, RANGE, ROUND>(v[r], sc, rng, rt, 8u * r * 256u, xlo, xhi);
      if (e + 8 > a.n) {  // codes of elements past the end are zero bits
        const int valid = (int)(a.n - e);
        const uint64_t keep = (1ull << (8 * valid)) - 1ull;
        xlo &= (uint32_t)keep;
        xhi &= (uint32_t)(keep >> 32);
      }
    }
    if (LAYOUT == kInterleaved) {
      if (stored) store_interleaved<K>(a.payload, oct, xlo, xhi);
    } else {
      // all lanes shuffle; a quad is stored or not as a whole (groups are four octets)
      const uint32_t any = __ballot_sync(0xffffffffu, stored);
      if (any) store_bitplane_guarded<K>(a.payload, oct >> 2, xlo, xhi, lane, stored);
    }
  }
}

}  // namespace accept
