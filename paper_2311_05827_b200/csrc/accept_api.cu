// Host side of the C ABI declared in include/accept.h: argument checks, stream geometry,
// kernel selection and launch.  Nothing here allocates memory or synchronises, except
// accept_last_device_status.
#include "../../include/accept.h"

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <utility>

#include "accept_kernels.cuh"
#include "accept_wide.cuh"
#include "accept_mbq.cuh"
#include "accept_strided.cuh"

namespace {

using accept::CodecArgs;

std::atomic<uint64_t> g_launches{0};

bool is_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

uint64_t n_chunks_of(const accept_params* p) { return (p->n_elems + p->chunk_elems - 1) / p->chunk_elems; }

// Chunks above this size are coded by the three-launch wide path (accept_wide.cuh).
constexpr uint32_t kWideChunk = 32768;

bool is_wide(const accept_params* p) { return p->chunk_elems > kWideChunk; }
bool is_strided(const accept_params* p) { return p->group_stride != 0; }
// pack groups stored in the payload
uint64_t n_groups_of(const accept_params* p) {
  if (!is_strided(p)) return (p->n_elems + 31) / 32;
  return ((p->n_elems / p->group_stride + 31) / 32) * (uint64_t)p->group_stride;
}

// Geometry of the register-resident compress path for chunk size C: rounds R and threads per chunk.
struct FastGeometry { int rounds; uint32_t tpc; };

// Four octets per thread measured fastest (fewest per-thread fixed costs per element); fewer
// rounds serve chunk sizes that four rounds of whole warps do not divide.
FastGeometry fast_geometry(uint32_t C) {
  if (C % 1024 == 0 && C / 32 <= 1024) return {4, C / 32};
  if (C % 512 == 0 && C / 16 <= 1024) return {2, C / 16};
  if (C % 256 == 0 && C / 8 <= 1024) return {1, C / 8};
  return {0, 0};
}

CodecArgs make_args(const accept_params* p, void* d_stream, void* d_ws) {
  CodecArgs a{};
  uint8_t* base = static_cast<uint8_t*>(d_stream);
  a.header = reinterpret_cast<uint32_t*>(base);
  a.meta = reinterpret_cast<float2*>(base + ACCEPT_HEADER_BYTES);
  a.payload = reinterpret_cast<uint32_t*>(base + accept_payload_offset(p));
  a.status = static_cast<uint32_t*>(d_ws);
  a.n = p->n_elems;
  a.n_chunks = n_chunks_of(p);
  a.seed = p->seed;
  a.rng_offset = p->rng_offset;
  a.chunk = p->chunk_elems;
  a.chunk_shift = -1;
  for (int s = 5; s < 32; ++s)
    if (p->chunk_elems == (1u << s)) a.chunk_shift = s;
  a.header_word6 = (uint32_t)p->range | ((uint32_t)p->round << 8) | ((uint32_t)p->layout << 16);
  a.k = p->k;
  a.group_stride = p->group_stride;
  return a;
}

// Launch with programmatic stream serialization: every kernel of this library starts with
// grid_dependency_handshake(), so it may be scheduled while its predecessor in the stream drains.
template <typename... Params, typename... Args>
cudaError_t launch_overlapped_shared(void (*fn)(Params...), dim3 grid, unsigned block, size_t shared_bytes, cudaStream_t s,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = shared_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, fn, std::forward<Args>(args)...);
}

template <typename... Params, typename... Args>
cudaError_t launch_overlapped(void (*fn)(Params...), dim3 grid, unsigned block, cudaStream_t s, Args&&... args) {
  return launch_overlapped_shared(fn, grid, block, 0, s, std::forward<Args>(args)...);
}

// A launch (or any runtime call) that fails ends the entry point at once: later launches of the same call
// are not issued, and only launches that were issued are counted.  The result is the call's own return
// value; cudaGetLastError() is never consulted, so an error left behind by the caller's earlier work is
// neither reported as ours nor cleared.
#define ACCEPT_LAUNCH(call)                                         \
  do {                                                              \
    if ((call) != cudaSuccess) return ACCEPT_ERR_CUDA;              \
    g_launches.fetch_add(1, std::memory_order_relaxed);             \
  } while (0)

// ---- tests-only build: byte ranges the kernels of a call may touch ------------------------------------
#ifdef ACCEPT_BOUNDS_CHECK
// ACCEPT_BOUNDS_TEST_SHRINK=<bytes> in the environment cuts that many bytes off the end of every writable
// range: the test of the checker itself, which shows that the last stores of a call are then counted and
// skipped (nothing is written there, nothing faults).
size_t bounds_test_shrink() {
  const char* text = std::getenv("ACCEPT_BOUNDS_TEST_SHRINK");
  return text ? (size_t)std::strtoull(text, nullptr, 10) : 0;
}

struct BoundsList {
  accept::BoundsTable table{};
  void add(const void* p, size_t bytes, bool writable) {
    if (!p || table.n >= accept::kMaxBoundsRanges) return;
    if (writable) bytes -= bounds_test_shrink() < bytes ? bounds_test_shrink() : bytes;
    table.lo[table.n] = (unsigned long long)p;
    table.hi[table.n] = (unsigned long long)p + bytes;
    table.writable[table.n] = writable ? 1u : 0u;
    ++table.n;
  }
  // ordered with the call's kernels on its stream (the source is pageable host memory: staged before return)
  cudaError_t install(cudaStream_t s) const {
    return cudaMemcpyToSymbolAsync(accept::g_bounds, &table, sizeof(table), 0, cudaMemcpyHostToDevice, s);
  }
};
#define ACCEPT_BOUNDS(stream, ...)                                              \
  do {                                                                          \
    BoundsList bounds_list;                                                     \
    __VA_ARGS__;                                                                \
    if (bounds_list.install(stream) != cudaSuccess) return ACCEPT_ERR_CUDA;     \
  } while (0)
#else
#define ACCEPT_BOUNDS(stream, ...) do { } while (0)
#endif

// ---- kernel tables -------------------------------------------------------------------------

using KernelFn = void (*)(const CodecArgs);

template <int K, int LAYOUT, int RANGE, int ROUND>
KernelFn compress_for_rounds(int rounds, bool small_block) {
  if (small_block) {
    switch (rounds) {
      case 1: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 1, 256>;
      case 4: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 4, 256>;
      default: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 2, 256>;
    }
  }
  switch (rounds) {
    case 1: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 1, 1024>;
    case 4: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 4, 1024>;
    default: return accept::compress_kernel<K, LAYOUT, RANGE, ROUND, 2, 1024>;
  }
}

template <int K, int LAYOUT>
KernelFn compress_for_modes(int range, int round, int rounds, bool sb) {
  if (range == accept::kAbsMax) {
    return round == accept::kNearest ? compress_for_rounds<K, LAYOUT, accept::kAbsMax, accept::kNearest>(rounds, sb)
                                     : compress_for_rounds<K, LAYOUT, accept::kAbsMax, accept::kStochastic>(rounds, sb);
  }
  return round == accept::kNearest ? compress_for_rounds<K, LAYOUT, accept::kMinMax, accept::kNearest>(rounds, sb)
                                   : compress_for_rounds<K, LAYOUT, accept::kMinMax, accept::kStochastic>(rounds, sb);
}

KernelFn select_compress(const accept_params* p, int rounds, bool sb) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? compress_for_modes<2, accept::kBitplane>(p->range, p->round, rounds, sb)
                      : compress_for_modes<2, accept::kInterleaved>(p->range, p->round, rounds, sb);
    case 3: return compress_for_modes<3, accept::kBitplane>(p->range, p->round, rounds, sb);
    case 4: return bp ? compress_for_modes<4, accept::kBitplane>(p->range, p->round, rounds, sb)
                      : compress_for_modes<4, accept::kInterleaved>(p->range, p->round, rounds, sb);
    default: return bp ? compress_for_modes<8, accept::kBitplane>(p->range, p->round, rounds, sb)
                       : compress_for_modes<8, accept::kInterleaved>(p->range, p->round, rounds, sb);
  }
}

template <int K, int LAYOUT, int RANGE>
KernelFn decompress_for_rounds(bool aligned, int rounds) {
  if (!aligned) return accept::decompress_unaligned_kernel<K, LAYOUT, RANGE>;
  (void)rounds;
  return accept::decompress_kernel<K, LAYOUT, RANGE, 2>;
}

template <int K, int LAYOUT>
KernelFn decompress_for_range(int range, bool aligned, int rounds) {
  if (range == accept::kAbsMax) return decompress_for_rounds<K, LAYOUT, accept::kAbsMax>(aligned, rounds);
  return decompress_for_rounds<K, LAYOUT, accept::kMinMax>(aligned, rounds);
}

KernelFn select_decompress(const accept_params* p, bool aligned, int rounds) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? decompress_for_range<2, accept::kBitplane>(p->range, aligned, rounds)
                      : decompress_for_range<2, accept::kInterleaved>(p->range, aligned, rounds);
    case 3: return decompress_for_range<3, accept::kBitplane>(p->range, aligned, rounds);
    case 4: return bp ? decompress_for_range<4, accept::kBitplane>(p->range, aligned, rounds)
                      : decompress_for_range<4, accept::kInterleaved>(p->range, aligned, rounds);
    default: return bp ? decompress_for_range<8, accept::kBitplane>(p->range, aligned, rounds)
                       : decompress_for_range<8, accept::kInterleaved>(p->range, aligned, rounds);
  }
}

// ---- wide chunks: ranges, constants, encode ------------------------------------------------------

// Octets per thread of the encode pass: the stochastic quantizer is instruction bound and amortises its
// per-thread generator set-up over four octets; the nearest one is memory bound and keeps two.
constexpr int kWideOctetsNearest = 2, kWideOctetsStochastic = 4;

template <int K, int LAYOUT, int RANGE>
cudaError_t launch_wide_encode(int round, const CodecArgs& a, const accept::ChunkRecord* rec, uint64_t n_oct_stored, cudaStream_t s) {
  if (round == accept::kNearest) {
    const unsigned grid = (unsigned)((n_oct_stored + kWideOctetsNearest * 256 - 1) / (kWideOctetsNearest * 256));
    return launch_overlapped(accept::wide_encode_kernel<K, LAYOUT, RANGE, accept::kNearest, kWideOctetsNearest>, dim3(grid), 256, s, a, rec);
  }
  const unsigned grid = (unsigned)((n_oct_stored + kWideOctetsStochastic * 256 - 1) / (kWideOctetsStochastic * 256));
  return launch_overlapped(accept::wide_encode_kernel<K, LAYOUT, RANGE, accept::kStochastic, kWideOctetsStochastic>, dim3(grid), 256, s, a, rec);
}

template <int RANGE>
cudaError_t launch_wide_encode_for(const accept_params* p, const CodecArgs& a, const accept::ChunkRecord* rec, uint64_t grid,
                                   cudaStream_t s) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? launch_wide_encode<2, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_wide_encode<2, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    case 3: return launch_wide_encode<3, accept::kBitplane, RANGE>(p->round, a, rec, grid, s);
    case 4: return bp ? launch_wide_encode<4, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_wide_encode<4, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    default: return bp ? launch_wide_encode<8, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                       : launch_wide_encode<8, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
  }
}

// Launch shape of the kernels that hold a chunk in registers (the one-launch coder, the constants pass of the
// batch-group coder): fills the geometry fields of the arguments.  Chunks without such a geometry, the ragged
// last chunk, and everything when the input is not 32-byte aligned get a block of the any-shape path each.
struct ChunkLaunch { unsigned grid, block; int rounds; };

ChunkLaunch chunk_launch(const accept_params* p, CodecArgs& a, bool aligned) {
  const FastGeometry g = fast_geometry(p->chunk_elems);
  const bool fast = g.rounds != 0 && aligned;
  unsigned block = accept::kGenericBlock;
  uint64_t fast_blocks = 0;
  if (fast) {
    a.n_fast_chunks = p->n_elems / p->chunk_elems;  // full chunks
    a.tpc = g.tpc;
    const bool share = g.tpc <= (uint32_t)accept::kFastBlock && accept::kFastBlock % g.tpc == 0;
    block = share ? accept::kFastBlock : g.tpc;
    a.chunks_per_block = share ? accept::kFastBlock / g.tpc : 1;
    a.tpc_shift = 0;
    while ((1u << a.tpc_shift) < g.tpc) ++a.tpc_shift;  // exact when share: tpc is then a power of two
    fast_blocks = (a.n_fast_chunks + a.chunks_per_block - 1) / a.chunks_per_block;
  } else {
    a.n_fast_chunks = 0;
    a.tpc = 32;
    a.chunks_per_block = 1;
  }
  a.fast_blocks = (uint32_t)fast_blocks;
  const uint64_t grid = fast_blocks + (a.n_chunks - a.n_fast_chunks);
  return {(unsigned)grid, block, fast ? g.rounds : 2};
}

// Range pass and constants in one launch (chunks of at most 32768 elements): see chunk_constants_kernel.
template <int RANGE>
cudaError_t launch_chunk_constants(const accept_params* p, CodecArgs& a, accept::ChunkRecord* rec, cudaStream_t s) {
  const ChunkLaunch cl = chunk_launch(p, a, true);
  const dim3 grid(cl.grid);
  if (cl.block > 256) {
    switch (cl.rounds) {
      case 4: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 4, 1024>, grid, cl.block, s, a, rec);
      case 2: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 2, 1024>, grid, cl.block, s, a, rec);
      default: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 1, 1024>, grid, cl.block, s, a, rec);
    }
  }
  switch (cl.rounds) {
    case 4: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 4, 256>, grid, cl.block, s, a, rec);
    case 2: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 2, 256>, grid, cl.block, s, a, rec);
    default: return launch_overlapped(accept::chunk_constants_kernel<RANGE, 1, 256>, grid, cl.block, s, a, rec);
  }
}

// rec_bytes = the workspace past its first 16 bytes: one record per chunk, cleared here.
accept_status launch_wide(const accept_params* p, const CodecArgs& a, uint8_t* rec_bytes, cudaStream_t s) {
  accept::ChunkRecord* rec = reinterpret_cast<accept::ChunkRecord*>(rec_bytes);
  if (cudaMemsetAsync(rec, 0, sizeof(accept::ChunkRecord) * a.n_chunks, s) != cudaSuccess) return ACCEPT_ERR_CUDA;
  const uint64_t n_oct = (p->n_elems + 7) / 8;
  const unsigned range_grid = (unsigned)((n_oct + 4 * 256 - 1) / (4 * 256));
  const unsigned fin_grid = (unsigned)((a.n_chunks + 255) / 256);
  const uint64_t enc_grid = ((p->n_elems + 31) / 32) * 4;  // octets the encode pass stores
  if (p->range == ACCEPT_RANGE_ABSMAX) {
    ACCEPT_LAUNCH(launch_overlapped(accept::wide_range_kernel<accept::kAbsMax, 4>, dim3(range_grid), 256, s, a, rec));
    ACCEPT_LAUNCH(launch_overlapped(accept::wide_finalize_kernel<accept::kAbsMax>, dim3(fin_grid), 256, s, a, rec));
    ACCEPT_LAUNCH(launch_wide_encode_for<accept::kAbsMax>(p, a, rec, enc_grid, s));
  } else {
    ACCEPT_LAUNCH(launch_overlapped(accept::wide_range_kernel<accept::kMinMax, 4>, dim3(range_grid), 256, s, a, rec));
    ACCEPT_LAUNCH(launch_overlapped(accept::wide_finalize_kernel<accept::kMinMax>, dim3(fin_grid), 256, s, a, rec));
    ACCEPT_LAUNCH(launch_wide_encode_for<accept::kMinMax>(p, a, rec, enc_grid, s));
  }
  return ACCEPT_OK;
}

// ---- pack groups along the batch dimension ---------------------------------------------------------

// The encoder is persistent: at most three blocks (64 KB of staged tile each) per SM of a B200.
constexpr unsigned kStridedEncodeBlocks = 3 * 148;

template <int K, int LAYOUT, int RANGE>
cudaError_t launch_strided_encode(int round, const CodecArgs& a, const accept::ChunkRecord* rec, dim3 tiles, cudaStream_t s) {
  if (round != accept::kNearest) {  // instruction bound: one tile per block, rows in registers
    // rows and octets start at multiples of eight values: every octet's first counter sits at the same place in its quad
    switch ((unsigned)(a.rng_offset & 3u)) {
      case 0: return launch_overlapped(accept::strided_encode_direct_kernel<K, LAYOUT, RANGE, accept::kStochastic, 0>, tiles, 256, s, a, rec);
      case 1: return launch_overlapped(accept::strided_encode_direct_kernel<K, LAYOUT, RANGE, accept::kStochastic, 1>, tiles, 256, s, a, rec);
      case 2: return launch_overlapped(accept::strided_encode_direct_kernel<K, LAYOUT, RANGE, accept::kStochastic, 2>, tiles, 256, s, a, rec);
      default: return launch_overlapped(accept::strided_encode_direct_kernel<K, LAYOUT, RANGE, accept::kStochastic, 3>, tiles, 256, s, a, rec);
    }
  }
  // memory bound: persistent blocks with a staged tile, which needs more dynamic shared memory than a
  // kernel gets without opting in (the attribute is per device: set every time)
  auto fn = accept::strided_encode_kernel<K, LAYOUT, RANGE, accept::kNearest>;
  const cudaError_t err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, accept::kStridedSmemBytes);
  if (err != cudaSuccess) return err;
  const uint64_t n_tiles = (uint64_t)tiles.x * tiles.y;
  const unsigned grid = (unsigned)(n_tiles < kStridedEncodeBlocks ? n_tiles : kStridedEncodeBlocks);
  accept::StridedTiling t;
  t.tiles_x = tiles.x;
  t.tiles_y = tiles.y;
  t.n_rows = (uint32_t)(a.n / a.group_stride);
  t.step_x = grid % tiles.x;
  t.step_y = grid / tiles.x;
  return launch_overlapped_shared(fn, dim3(grid), 256, accept::kStridedSmemBytes, s, a, rec, t);
}

template <int RANGE>
cudaError_t launch_strided_encode_for(const accept_params* p, const CodecArgs& a, const accept::ChunkRecord* rec, dim3 grid,
                                      cudaStream_t s) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? launch_strided_encode<2, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_strided_encode<2, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    case 3: return launch_strided_encode<3, accept::kBitplane, RANGE>(p->round, a, rec, grid, s);
    case 4: return bp ? launch_strided_encode<4, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_strided_encode<4, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    default: return bp ? launch_strided_encode<8, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                       : launch_strided_encode<8, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
  }
}

template <int RANGE>
cudaError_t launch_strided_decode_for(const accept_params* p, const CodecArgs& a, dim3 grid, cudaStream_t s) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? launch_overlapped(accept::strided_decode_kernel<2, accept::kBitplane, RANGE>, dim3(grid), 256, s, a)
                      : launch_overlapped(accept::strided_decode_kernel<2, accept::kInterleaved, RANGE>, dim3(grid), 256, s, a);
    case 3: return launch_overlapped(accept::strided_decode_kernel<3, accept::kBitplane, RANGE>, dim3(grid), 256, s, a);
    case 4: return bp ? launch_overlapped(accept::strided_decode_kernel<4, accept::kBitplane, RANGE>, dim3(grid), 256, s, a)
                      : launch_overlapped(accept::strided_decode_kernel<4, accept::kInterleaved, RANGE>, dim3(grid), 256, s, a);
    default: return bp ? launch_overlapped(accept::strided_decode_kernel<8, accept::kBitplane, RANGE>, dim3(grid), 256, s, a)
                       : launch_overlapped(accept::strided_decode_kernel<8, accept::kInterleaved, RANGE>, dim3(grid), 256, s, a);
  }
}

// The octet-per-thread kernels need rows that start on 32-byte boundaries; every other shape goes through the
// feature-per-thread kernels.
bool strided_any_shape(const accept_params* p) { return p->group_stride % 8 != 0; }

dim3 strided_any_grid(const accept_params* p) {
  const unsigned gx = (p->group_stride + accept::kStridedAnyBlock - 1) / accept::kStridedAnyBlock;
  const unsigned gy = (unsigned)((p->n_elems / p->group_stride + 31) / 32);
  return dim3(gx, gy, 1);
}

template <int K, int LAYOUT, int RANGE>
cudaError_t launch_strided_encode_any(int round, const CodecArgs& a, const accept::ChunkRecord* rec, dim3 grid, cudaStream_t s) {
  if (round == accept::kNearest)
    return launch_overlapped(accept::strided_encode_any_kernel<K, LAYOUT, RANGE, accept::kNearest>, grid, accept::kStridedAnyBlock, s, a, rec);
  return launch_overlapped(accept::strided_encode_any_kernel<K, LAYOUT, RANGE, accept::kStochastic>, grid, accept::kStridedAnyBlock, s, a, rec);
}

template <int RANGE>
cudaError_t launch_strided_encode_any_for(const accept_params* p, const CodecArgs& a, const accept::ChunkRecord* rec, dim3 grid,
                                          cudaStream_t s) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  switch (p->k) {
    case 2: return bp ? launch_strided_encode_any<2, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_strided_encode_any<2, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    case 3: return launch_strided_encode_any<3, accept::kBitplane, RANGE>(p->round, a, rec, grid, s);
    case 4: return bp ? launch_strided_encode_any<4, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                      : launch_strided_encode_any<4, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
    default: return bp ? launch_strided_encode_any<8, accept::kBitplane, RANGE>(p->round, a, rec, grid, s)
                       : launch_strided_encode_any<8, accept::kInterleaved, RANGE>(p->round, a, rec, grid, s);
  }
}

template <int RANGE>
cudaError_t launch_strided_decode_any_for(const accept_params* p, const CodecArgs& a, dim3 grid, cudaStream_t s) {
  const bool bp = p->layout == ACCEPT_LAYOUT_BITPLANE;
  const unsigned block = accept::kStridedAnyBlock;
  switch (p->k) {
    case 2: return bp ? launch_overlapped(accept::strided_decode_any_kernel<2, accept::kBitplane, RANGE>, grid, block, s, a)
                      : launch_overlapped(accept::strided_decode_any_kernel<2, accept::kInterleaved, RANGE>, grid, block, s, a);
    case 3: return launch_overlapped(accept::strided_decode_any_kernel<3, accept::kBitplane, RANGE>, grid, block, s, a);
    case 4: return bp ? launch_overlapped(accept::strided_decode_any_kernel<4, accept::kBitplane, RANGE>, grid, block, s, a)
                      : launch_overlapped(accept::strided_decode_any_kernel<4, accept::kInterleaved, RANGE>, grid, block, s, a);
    default: return bp ? launch_overlapped(accept::strided_decode_any_kernel<8, accept::kBitplane, RANGE>, grid, block, s, a)
                       : launch_overlapped(accept::strided_decode_any_kernel<8, accept::kInterleaved, RANGE>, grid, block, s, a);
  }
}

dim3 strided_grid(const accept_params* p) {
  const unsigned gx = (p->group_stride / 8 + accept::kStridedOctetsPerBlock - 1) / accept::kStridedOctetsPerBlock;
  const unsigned gy = (unsigned)((p->n_elems / p->group_stride + 31) / 32);
  return dim3(gx, gy, 1);
}

accept_status launch_strided(const accept_params* p, CodecArgs a, uint8_t* rec_bytes, cudaStream_t s) {
  accept::ChunkRecord* rec = reinterpret_cast<accept::ChunkRecord*>(rec_bytes);
  const bool absmax = p->range == ACCEPT_RANGE_ABSMAX;
  if (!is_wide(p)) {
    // a block holds a chunk: ranges, side words and constants in one launch, nothing to clear
    if (absmax) ACCEPT_LAUNCH(launch_chunk_constants<accept::kAbsMax>(p, a, rec, s));
    else ACCEPT_LAUNCH(launch_chunk_constants<accept::kMinMax>(p, a, rec, s));
  } else {
    if (cudaMemsetAsync(rec, 0, sizeof(accept::ChunkRecord) * a.n_chunks, s) != cudaSuccess) return ACCEPT_ERR_CUDA;
    const uint64_t n_oct = (p->n_elems + 7) / 8;
    const unsigned range_grid = (unsigned)((n_oct + 4 * 256 - 1) / (4 * 256));
    const unsigned fin_grid = (unsigned)((a.n_chunks + 255) / 256);
    if (absmax) {
      ACCEPT_LAUNCH(launch_overlapped(accept::wide_range_kernel<accept::kAbsMax, 4>, dim3(range_grid), 256, s, a, rec));
      ACCEPT_LAUNCH(launch_overlapped(accept::wide_finalize_kernel<accept::kAbsMax>, dim3(fin_grid), 256, s, a, rec));
    } else {
      ACCEPT_LAUNCH(launch_overlapped(accept::wide_range_kernel<accept::kMinMax, 4>, dim3(range_grid), 256, s, a, rec));
      ACCEPT_LAUNCH(launch_overlapped(accept::wide_finalize_kernel<accept::kMinMax>, dim3(fin_grid), 256, s, a, rec));
    }
  }
  const bool any = strided_any_shape(p);
  if (absmax) {
    if (any) ACCEPT_LAUNCH(launch_strided_encode_any_for<accept::kAbsMax>(p, a, rec, strided_any_grid(p), s));
    else ACCEPT_LAUNCH(launch_strided_encode_for<accept::kAbsMax>(p, a, rec, strided_grid(p), s));
  } else {
    if (any) ACCEPT_LAUNCH(launch_strided_encode_any_for<accept::kMinMax>(p, a, rec, strided_any_grid(p), s));
    else ACCEPT_LAUNCH(launch_strided_encode_for<accept::kMinMax>(p, a, rec, strided_grid(p), s));
  }
  return ACCEPT_OK;
}

// ---- multi-bit quantization --------------------------------------------------------------------

uint64_t mbq_tiles(const accept_mbq_params* p) { return (p->n_elems + accept::kMbqTile - 1) / accept::kMbqTile; }

// blocks of the encode pass: one per tile of 256 groups, at most two per SM of a B200 (the blocks are persistent)
uint32_t mbq_blocks(const accept_mbq_params* p) {
  const uint64_t tiles = (p->n_elems + accept::kMbqGroupTile - 1) / accept::kMbqGroupTile;
  return (uint32_t)(tiles < (uint64_t)accept::kMbqMaxBlocks ? tiles : (uint64_t)accept::kMbqMaxBlocks);
}

uint32_t mbq_residue_blocks(const accept_mbq_params* p) {
  const uint64_t tiles = mbq_tiles(p);
  return (uint32_t)(tiles < (uint64_t)accept::kMbqResidueBlocks ? tiles : (uint64_t)accept::kMbqResidueBlocks);
}

accept::MbqArgs mbq_args(const accept_mbq_params* p, void* d_stream, void* d_ws) {
  accept::MbqArgs a{};
  uint8_t* base = static_cast<uint8_t*>(d_stream);
  uint8_t* ws = static_cast<uint8_t*>(d_ws);
  a.header = reinterpret_cast<uint32_t*>(base);
  a.side = reinterpret_cast<float*>(base + ACCEPT_HEADER_BYTES);
  a.payload = reinterpret_cast<uint32_t*>(base + accept_mbq_payload_offset(p));
  a.status = reinterpret_cast<uint32_t*>(ws);
  a.ws = reinterpret_cast<accept::MbqWorkspace*>(ws);
  a.n = p->n_elems;
  a.n_blocks = mbq_blocks(p);
  a.n_residue_blocks = mbq_residue_blocks(p);
  a.n_tiles = mbq_tiles(p);
  a.k = p->k;
  a.batch_index = p->batch_index;
  a.init = p->init ? 1u : 0u;
  return a;
}

template <int K>
accept_status launch_mbq_compress(const accept::MbqArgs& a, cudaStream_t s) {
  const dim3 grid(a.n_blocks);
  // the search grid and the staged tiles need more dynamic shared memory than a kernel gets without opting in
  // (the attribute is per device: set every time)
  if (a.init) {
    const dim3 rgrid(a.n_residue_blocks);
    ACCEPT_LAUNCH(launch_overlapped(accept::mbq_residue_sum_kernel<K, 0>, rgrid, 256, s, a));
    ACCEPT_LAUNCH(launch_overlapped(accept::mbq_residue_sum_kernel<K, 1>, rgrid, 256, s, a));
    if constexpr (K > 2) ACCEPT_LAUNCH(launch_overlapped(accept::mbq_residue_sum_kernel<K, 2>, rgrid, 256, s, a));
    if constexpr (K > 3) ACCEPT_LAUNCH(launch_overlapped(accept::mbq_residue_sum_kernel<K, 3>, rgrid, 256, s, a));
    auto fn = accept::mbq_encode_kernel<K, true>;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, accept::kMbqEncodeSmemBytes) != cudaSuccess)
      return ACCEPT_ERR_CUDA;
    ACCEPT_LAUNCH(launch_overlapped_shared(fn, grid, accept::kMbqEncodeThreads, accept::kMbqEncodeSmemBytes, s, a));
  } else {
    auto fn = accept::mbq_encode_kernel<K, false>;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, accept::kMbqEncodeSmemBytes) != cudaSuccess)
      return ACCEPT_ERR_CUDA;
    ACCEPT_LAUNCH(launch_overlapped_shared(fn, grid, accept::kMbqEncodeThreads, accept::kMbqEncodeSmemBytes, s, a));
  }
  return ACCEPT_OK;
}

// ---- built-in scratch for accept_compress_static ------------------------------------------------
//
// The workspace of callers that cannot allocate.  In host code the name g_static_scratch is only a
// stand-in for the symbol, not a device address: the address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[ACCEPT_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_address[kMaxDevices] = {};

// Device address of the built-in scratch on the current device, or nullptr on a CUDA error.
void* static_scratch_address() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_address[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
    g_scratch_address[dev] = ptr;
  }
  return g_scratch_address[dev];
}

// ws_need: bytes of workspace the call touches (the compress side: accept_workspace_size; the decode side:
// the status word only, whatever the parameters).
accept_status check_buffers(const accept_params* p, const void* d_tensor, const void* d_stream,
                            size_t stream_bytes, const void* d_ws, size_t ws_bytes, bool decode) {
  if (!p || !d_tensor || !d_stream || !d_ws) return ACCEPT_ERR_NULL;
  accept_status st = accept_check_params(p);
  if (st != ACCEPT_OK) return st;
  const size_t ws_need = decode ? 16 : accept_workspace_size(p);
  if (stream_bytes < accept_compressed_size(p) || ws_bytes < ws_need) return ACCEPT_ERR_TOO_SMALL;
  if (!is_aligned(d_tensor, 16) || !is_aligned(d_stream, 16) || !is_aligned(d_ws, 4)) return ACCEPT_ERR_MISALIGNED;
  return ACCEPT_OK;
}

}  // namespace

extern "C" {

accept_status accept_check_params(const accept_params* p) {
  if (!p) return ACCEPT_ERR_NULL;
  if (p->n_elems == 0) return ACCEPT_ERR_BAD_SIZE;
  if (p->chunk_elems < 32 || p->chunk_elems % 32 != 0) return ACCEPT_ERR_BAD_CHUNK;
  if (p->range != ACCEPT_RANGE_ABSMAX && p->range != ACCEPT_RANGE_MINMAX) return ACCEPT_ERR_BAD_ENUM;
  if (p->round != ACCEPT_ROUND_NEAREST && p->round != ACCEPT_ROUND_STOCHASTIC) return ACCEPT_ERR_BAD_ENUM;
  if (p->layout != ACCEPT_LAYOUT_INTERLEAVED && p->layout != ACCEPT_LAYOUT_BITPLANE) return ACCEPT_ERR_BAD_ENUM;
  if (!(p->k == 2 || p->k == 3 || p->k == 4 || p->k == 8)) return ACCEPT_ERR_BAD_K;
  if (p->k == 3 && p->layout != ACCEPT_LAYOUT_BITPLANE) return ACCEPT_ERR_BAD_K;
  if (p->group_stride != 0) {
    if (p->n_elems % p->group_stride != 0) return ACCEPT_ERR_BAD_SIZE;
    if ((p->n_elems / p->group_stride + 31) / 32 > 65535) return ACCEPT_ERR_BAD_SIZE;  // batch groups ride on grid.y
  }
  // one block per chunk / per 4096 elements must fit the grid's x dimension
  if (n_chunks_of(p) > 0x7fffffffull || p->n_elems / 4096 > 0x7ffffff0ull) return ACCEPT_ERR_BAD_SIZE;
  return ACCEPT_OK;
}

size_t accept_payload_offset(const accept_params* p) {
  if (accept_check_params(p) != ACCEPT_OK) return 0;
  const uint64_t off = ACCEPT_HEADER_BYTES + 8 * n_chunks_of(p);
  return (size_t)((off + 15) / 16 * 16);
}

size_t accept_compressed_size(const accept_params* p) {
  if (accept_check_params(p) != ACCEPT_OK) return 0;
  return accept_payload_offset(p) + (size_t)(4ull * p->k * n_groups_of(p));
}

size_t accept_workspace_size(const accept_params* p) {
  if (accept_check_params(p) != ACCEPT_OK) return 0;
  // status word (+ pad); chunks wider than 32768 elements also need one 16-byte record each
  return 16 + ((is_wide(p) || is_strided(p)) ? 16 * (size_t)n_chunks_of(p) : 0);
}

accept_status accept_compress(const accept_params* p, const float* d_x, void* d_stream, size_t stream_bytes,
                              void* d_ws, size_t ws_bytes, void* cuda_stream) {
  accept_status st = check_buffers(p, d_x, d_stream, stream_bytes, d_ws, ws_bytes, false);
  if (st != ACCEPT_OK) return st;
  CodecArgs a = make_args(p, d_stream, d_ws);
  a.x = d_x;
  ACCEPT_BOUNDS(static_cast<cudaStream_t>(cuda_stream), bounds_list.add(d_x, 4 * p->n_elems, false);
                bounds_list.add(d_stream, accept_compressed_size(p), true); bounds_list.add(d_ws, accept_workspace_size(p), true));

  if (is_strided(p)) {
    if (!is_aligned(d_x, 32) || !is_aligned(d_ws, 16)) return ACCEPT_ERR_MISALIGNED;
    return launch_strided(p, a, static_cast<uint8_t*>(d_ws) + 16, static_cast<cudaStream_t>(cuda_stream));
  }
  if (is_wide(p) && is_aligned(d_x, 32)) {
    if (!is_aligned(d_ws, 16)) return ACCEPT_ERR_MISALIGNED;
    return launch_wide(p, a, static_cast<uint8_t*>(d_ws) + 16, static_cast<cudaStream_t>(cuda_stream));
  }

  const ChunkLaunch cl = chunk_launch(p, a, is_aligned(d_x, 32));
  KernelFn fn = select_compress(p, cl.rounds, cl.block <= 256);
  ACCEPT_LAUNCH(launch_overlapped(fn, cl.grid, cl.block, static_cast<cudaStream_t>(cuda_stream), a));
  return ACCEPT_OK;
}

accept_status accept_decompress(const accept_params* p, const void* d_stream, size_t stream_bytes, float* d_xhat,
                                void* d_ws, size_t ws_bytes, void* cuda_stream) {
  accept_status st = check_buffers(p, d_xhat, d_stream, stream_bytes, d_ws, ws_bytes, true);
  if (st != ACCEPT_OK) return st;
  CodecArgs a = make_args(p, const_cast<void*>(d_stream), d_ws);
  a.xhat = d_xhat;
  ACCEPT_BOUNDS(static_cast<cudaStream_t>(cuda_stream), bounds_list.add(d_stream, accept_compressed_size(p), false);
                bounds_list.add(d_xhat, 4 * p->n_elems, true); bounds_list.add(d_ws, 16, true));
  if (is_strided(p)) {
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (strided_any_shape(p)) {
      if (p->range == ACCEPT_RANGE_ABSMAX) ACCEPT_LAUNCH(launch_strided_decode_any_for<accept::kAbsMax>(p, a, strided_any_grid(p), s));
      else ACCEPT_LAUNCH(launch_strided_decode_any_for<accept::kMinMax>(p, a, strided_any_grid(p), s));
      return ACCEPT_OK;
    }
    if (!is_aligned(d_xhat, 32)) return ACCEPT_ERR_MISALIGNED;
    if (p->range == ACCEPT_RANGE_ABSMAX) ACCEPT_LAUNCH(launch_strided_decode_for<accept::kAbsMax>(p, a, strided_grid(p), s));
    else ACCEPT_LAUNCH(launch_strided_decode_for<accept::kMinMax>(p, a, strided_grid(p), s));
    return ACCEPT_OK;
  }
  const bool aligned = is_aligned(d_xhat, 32);
  const int rounds = 2;  // octets per thread
  KernelFn fn = select_decompress(p, aligned, rounds);
  const uint64_t per_block = aligned ? 2048ull * rounds : 256;  // elements per block
  const uint64_t grid = (p->n_elems + per_block - 1) / per_block;
  ACCEPT_LAUNCH(launch_overlapped(fn, (unsigned)grid, 256, static_cast<cudaStream_t>(cuda_stream), a));
  return ACCEPT_OK;
}

accept_status accept_compress_host(const accept_params* p, const float* h_x, void* h_stream, size_t stream_bytes,
                                   float* d_x, void* d_stream, void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!h_x || !h_stream) return ACCEPT_ERR_NULL;
  accept_status st = check_buffers(p, d_x, d_stream, stream_bytes, d_ws, ws_bytes, false);
  if (st != ACCEPT_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(d_x, h_x, p->n_elems * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  st = accept_compress(p, d_x, d_stream, stream_bytes, d_ws, ws_bytes, cuda_stream);
  if (st != ACCEPT_OK) return st;
  if (cudaMemcpyAsync(h_stream, d_stream, accept_compressed_size(p), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  return ACCEPT_OK;
}

accept_status accept_decompress_host(const accept_params* p, const void* h_stream, size_t stream_bytes,
                                     float* h_xhat, void* d_stream, float* d_xhat, void* d_ws, size_t ws_bytes,
                                     void* cuda_stream) {
  if (!h_stream || !h_xhat) return ACCEPT_ERR_NULL;
  accept_status st = check_buffers(p, d_xhat, d_stream, stream_bytes, d_ws, ws_bytes, true);
  if (st != ACCEPT_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(d_stream, h_stream, accept_compressed_size(p), cudaMemcpyHostToDevice, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  st = accept_decompress(p, d_stream, stream_bytes, d_xhat, d_ws, ws_bytes, cuda_stream);
  if (st != ACCEPT_OK) return st;
  if (cudaMemcpyAsync(h_xhat, d_xhat, p->n_elems * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  return ACCEPT_OK;
}

accept_status accept_last_device_status(const void* d_ws, void* cuda_stream, uint32_t* status_bits) {
  if (!d_ws || !status_bits) return ACCEPT_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(status_bits, d_ws, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? ACCEPT_OK : ACCEPT_ERR_CUDA;
}

accept_status accept_parse_header(const void* h_header, accept_params* out) {
  if (!h_header || !out) return ACCEPT_ERR_NULL;
  uint32_t h[8];
  std::memcpy(h, h_header, sizeof(h));
  if (h[0] != ACCEPT_MAGIC || h[1] != ACCEPT_VERSION) return ACCEPT_ERR_BAD_STREAM_HEADER;
  accept_params p{};
  p.n_elems = (uint64_t)h[2] | ((uint64_t)h[3] << 32);
  p.chunk_elems = h[4];
  p.k = h[5];
  p.range = (int32_t)(h[6] & 0xFF);
  p.round = (int32_t)((h[6] >> 8) & 0xFF);
  p.layout = (int32_t)((h[6] >> 16) & 0xFF);
  p.group_stride = h[7];
  if ((h[6] >> 24) != 0 || accept_check_params(&p) != ACCEPT_OK) return ACCEPT_ERR_BAD_STREAM_HEADER;
  *out = p;
  return ACCEPT_OK;
}

int accept_bitwidth_schedule(int is_backward, int n_lr_changes) {
  if (n_lr_changes < 0) n_lr_changes = 0;
  if (is_backward) return n_lr_changes == 0 ? 8 : 4;
  return n_lr_changes >= 2 ? 4 : 2 + n_lr_changes;
}

accept_status accept_mbq_check_params(const accept_mbq_params* p) {
  if (!p) return ACCEPT_ERR_NULL;
  if (p->n_elems == 0) return ACCEPT_ERR_BAD_SIZE;
  if (p->k < 2 || p->k > 4) return ACCEPT_ERR_BAD_K;
  if (p->reserved != 0 || p->init > 1) return ACCEPT_ERR_BAD_ENUM;
  return ACCEPT_OK;
}

size_t accept_mbq_payload_offset(const accept_mbq_params* p) {
  if (accept_mbq_check_params(p) != ACCEPT_OK) return 0;
  return (ACCEPT_HEADER_BYTES + 4 * (size_t)(p->k + 1) + 15) / 16 * 16;
}

size_t accept_mbq_compressed_size(const accept_mbq_params* p) {
  if (accept_mbq_check_params(p) != ACCEPT_OK) return 0;
  return accept_mbq_payload_offset(p) + (size_t)(4ull * p->k * ((p->n_elems + 31) / 32));
}

size_t accept_mbq_workspace_size(const accept_mbq_params* p) {
  if (accept_mbq_check_params(p) != ACCEPT_OK) return 0;
  // status word, residue coefficients, the exact sums (five of 12 digits) and the sign counts
  return sizeof(accept::MbqWorkspace);
}

accept_status accept_mbq_compress(const accept_mbq_params* p, const float* d_x, const float* d_alpha_prev,
                                  float* d_alpha_next, void* d_stream, size_t stream_bytes, void* d_ws,
                                  size_t ws_bytes, void* cuda_stream) {
  if (!p || !d_x || !d_alpha_next || !d_stream || !d_ws) return ACCEPT_ERR_NULL;
  accept_status st = accept_mbq_check_params(p);
  if (st != ACCEPT_OK) return st;
  if (!p->init && !d_alpha_prev) return ACCEPT_ERR_NULL;
  if (stream_bytes < accept_mbq_compressed_size(p) || ws_bytes < accept_mbq_workspace_size(p)) return ACCEPT_ERR_TOO_SMALL;
  if (!is_aligned(d_x, 32) || !is_aligned(d_stream, 16) || !is_aligned(d_ws, 16) || !is_aligned(d_alpha_next, 4) ||
      !is_aligned(d_alpha_prev, 4))
    return ACCEPT_ERR_MISALIGNED;
  accept::MbqArgs a = mbq_args(p, d_stream, d_ws);
  a.x = d_x;
  a.alpha_prev = d_alpha_prev;
  a.alpha_next = d_alpha_next;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  ACCEPT_BOUNDS(s, bounds_list.add(d_x, 4 * p->n_elems, false); bounds_list.add(d_alpha_prev, 4 * p->k, false);
                bounds_list.add(d_alpha_next, 4 * p->k, true); bounds_list.add(d_stream, accept_mbq_compressed_size(p), true);
                bounds_list.add(d_ws, accept_mbq_workspace_size(p), true));
  switch (p->k) {
    case 2: return launch_mbq_compress<2>(a, s);
    case 3: return launch_mbq_compress<3>(a, s);
    default: return launch_mbq_compress<4>(a, s);
  }
}

accept_status accept_mbq_decompress(const accept_mbq_params* p, const void* d_stream, size_t stream_bytes,
                                    float* d_xhat, void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!p || !d_stream || !d_xhat || !d_ws) return ACCEPT_ERR_NULL;
  accept_status st = accept_mbq_check_params(p);
  if (st != ACCEPT_OK) return st;
  if (stream_bytes < accept_mbq_compressed_size(p) || ws_bytes < 16) return ACCEPT_ERR_TOO_SMALL;
  if (!is_aligned(d_xhat, 32) || !is_aligned(d_stream, 16) || !is_aligned(d_ws, 4)) return ACCEPT_ERR_MISALIGNED;
  accept::MbqArgs a = mbq_args(p, const_cast<void*>(d_stream), d_ws);
  a.xhat = d_xhat;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const unsigned grid = (unsigned)((p->n_elems + 4095) / 4096);
  ACCEPT_BOUNDS(s, bounds_list.add(d_stream, accept_mbq_compressed_size(p), false); bounds_list.add(d_xhat, 4 * p->n_elems, true);
                bounds_list.add(d_ws, 16, true));
  switch (p->k) {
    case 2: ACCEPT_LAUNCH(launch_overlapped(accept::mbq_decode_kernel<2>, dim3(grid), 256, s, a)); break;
    case 3: ACCEPT_LAUNCH(launch_overlapped(accept::mbq_decode_kernel<3>, dim3(grid), 256, s, a)); break;
    default: ACCEPT_LAUNCH(launch_overlapped(accept::mbq_decode_kernel<4>, dim3(grid), 256, s, a)); break;
  }
  return ACCEPT_OK;
}

uint64_t accept_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

accept_status accept_launch_null(uint32_t blocks, uint32_t threads, void* cuda_stream) {
  if (blocks == 0 || blocks > 0x7fffffffu || threads < 32 || threads > 1024) return ACCEPT_ERR_BAD_SIZE;
  ACCEPT_LAUNCH(launch_overlapped(accept::null_kernel, dim3(blocks), threads, static_cast<cudaStream_t>(cuda_stream)));
  return ACCEPT_OK;
}

accept_status accept_bounds_check_report(void* cuda_stream, uint32_t* violations, uint64_t* first_address,
                                         uint64_t* first_size_and_kind) {
  if (!violations) return ACCEPT_ERR_NULL;
#ifndef ACCEPT_BOUNDS_CHECK
  (void)cuda_stream;
  *violations = 0;
  if (first_address) *first_address = 0;
  if (first_size_and_kind) *first_size_and_kind = 0;
  return ACCEPT_ERR_UNCHECKED_BUILD;
#else
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long first[2] = {0, 0};
  const unsigned int zero = 0;
  if (cudaStreamSynchronize(s) != cudaSuccess) return ACCEPT_ERR_CUDA;
  if (cudaMemcpyFromSymbol(violations, accept::g_bounds_violations, sizeof(uint32_t)) != cudaSuccess) return ACCEPT_ERR_CUDA;
  if (cudaMemcpyFromSymbol(first, accept::g_bounds_first, sizeof(first)) != cudaSuccess) return ACCEPT_ERR_CUDA;
  if (cudaMemcpyToSymbol(accept::g_bounds_violations, &zero, sizeof(zero)) != cudaSuccess) return ACCEPT_ERR_CUDA;
  if (first_address) *first_address = first[0];
  if (first_size_and_kind) *first_size_and_kind = first[1];
  return ACCEPT_OK;
#endif
}

accept_status accept_compress_static(const accept_params* p, const float* d_x, void* d_stream, size_t stream_bytes,
                                     uint32_t* d_status_out, void* cuda_stream) {
  // everything that can be refused on the host is refused before CUDA is touched
  if (!p || !d_x || !d_stream) return ACCEPT_ERR_NULL;
  accept_status st = accept_check_params(p);
  if (st != ACCEPT_OK) return st;
  if (accept_workspace_size(p) > ACCEPT_STATIC_SCRATCH_BYTES) return ACCEPT_ERR_SCRATCH_LIMIT;
  if (stream_bytes < accept_compressed_size(p)) return ACCEPT_ERR_TOO_SMALL;
  if (!is_aligned(d_x, 16) || !is_aligned(d_stream, 16) || !is_aligned(d_status_out, 4)) return ACCEPT_ERR_MISALIGNED;

  // the built-in array is looked up on the CURRENT device: an input that lives on another one would make the
  // kernel run there with this device's scratch address
  int current = -1;
  cudaPointerAttributes where{};
  if (cudaGetDevice(&current) != cudaSuccess || cudaPointerGetAttributes(&where, d_x) != cudaSuccess) return ACCEPT_ERR_CUDA;
  if (where.type == cudaMemoryTypeDevice && where.device != current) return ACCEPT_ERR_CUDA;
  void* scratch = static_scratch_address();
  if (!scratch) return ACCEPT_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps what the previous call left: the status word must start at zero
  if (cudaMemsetAsync(scratch, 0, 16, s) != cudaSuccess) return ACCEPT_ERR_CUDA;
  st = accept_compress(p, d_x, d_stream, stream_bytes, scratch, ACCEPT_STATIC_SCRATCH_BYTES, cuda_stream);
  if (st != ACCEPT_OK) return st;
  if (d_status_out &&
      cudaMemcpyAsync(d_status_out, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return ACCEPT_ERR_CUDA;
  return ACCEPT_OK;
}

}  // extern "C"
