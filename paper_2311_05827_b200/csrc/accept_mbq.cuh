// Forward quantizer of the paper: multi-bit quantization (Sec. 3.3 "Forward Quantizer", Eq. 1-5),
// "Forward Encoder" (bit planes, -1 stored as 0) and the receiver (Sec. 3.4 "Forward Decoder",
// "Forward Dequantizer").
//
// Element i carries k signs b_i0..b_i,k-1 as the code c_i = sum_j [b_ij = +1] << j; plane j of a
// 32-element group is basis j.  level(c) = (+-alpha_0) + ... + (+-alpha_k-1), summed in fp32 in
// the order j = 0..k-1.  One pass over the input assigns the signs (nearest level through a
// uniform grid over the span of the levels, one shared-memory lookup and one comparison per
// element), writes the planes and gathers what Eq. 3-5 need: counts of +1 per basis, counts of
// differing signs per pair of bases (integers: B^T B exactly), the sum of x over the +1 elements of
// each basis and the sum of x.  The sums of x are EXACT (accept_exact.cuh): integers all the way into
// the workspace, rounded once to double by the single small block that then solves the k x k system,
// applies the moving average and writes the side words.  Nothing depends on the order in which
// threads or blocks add, so the side words are a function of the input alone.
#pragma once
#include "accept_async.cuh"
#include "accept_exact.cuh"
#include "accept_kernels.cuh"

namespace accept {

constexpr int kMbqRounds = 2;                      // octets per thread and tile of a residue pass
constexpr int kMbqTile = kMbqRounds * 256 * 8;     // elements per tile of a residue pass
constexpr int kMbqResidueBlocks = 148 * 3;         // blocks of a residue pass: three resident per SM, each walks over its tiles
constexpr int kMbqSums = 5;                        // wide sums in the workspace: basis 0..3, then the sum of x
constexpr int kMbqFlushTiles = kFlushElems / (kMbqRounds * 8);  // tiles a thread of a residue pass adds between two flushes

// Encode pass: persistent blocks of 256 threads, two per SM.  A thread owns one pack group (32 consecutive
// values, 128 bytes) of each tile; tiles of 256 groups (32 KB) are staged in shared memory with
// asynchronous bulk copies, two stages per block, so a block always has its next tile in flight.
constexpr int kMbqEncodeThreads = 256;
constexpr int kMbqBlocksPerSm = 2;
constexpr int kMbqMaxBlocks = 148 * kMbqBlocksPerSm;
constexpr int kMbqGroupTile = kMbqEncodeThreads * 32;        // elements per tile of the encode pass
constexpr int kMbqTileBytes = kMbqGroupTile * 4;
constexpr int kMbqStages = 2;
constexpr int kMbqCopyBytes = 8192;                          // one bulk copy; a tile is four of them
constexpr int kMbqCells = 256;                               // cells of the uniform search grid
constexpr int kMbqColumns = 8;                               // copies of the grid: one per lane of a quarter warp
constexpr int kMbqGridBytes = kMbqCells * kMbqColumns * 16;  // one 16-byte entry per cell and column: 32 KB
constexpr int kMbqEncodeSmemBytes = kMbqGridBytes + kMbqStages * kMbqTileBytes;
constexpr int kMbqFlushGroups = kFlushElems / 32;            // groups a thread codes between two flushes

// Workspace of the forward quantizer (zeroed once by the caller; every call leaves the sums zeroed again).
struct MbqWorkspace {
  uint32_t status;
  uint32_t pad0[3];
  float alpha_init[4];            // coefficients found by the residue passes (init)
  uint32_t blocks_done;           // blocks of the running pass that have delivered their sums
  uint32_t next_tile;             // encode pass: tiles handed out beyond every block's first two
  uint32_t pad1[6];
  long long wide[kMbqSums][kAccLimbs];  // exact sums, see accept_exact.cuh
  unsigned long long count[4];    // number of +1 per basis
  unsigned long long differ[6];   // pairs (0,1) (0,2) (0,3) (1,2) (1,3) (2,3): elements whose two signs differ
};
static_assert(sizeof(MbqWorkspace) == 64 + 8 * kMbqSums * kAccLimbs + 80, "workspace layout");

struct MbqArgs {
  const float* x;
  float* xhat;
  const float* alpha_prev;  // device, k floats (unused when init)
  float* alpha_next;        // device, k floats
  uint32_t* header;         // stream + 0
  float* side;              // stream + 32: alpha (k floats), m_q
  uint32_t* payload;
  uint32_t* status;
  MbqWorkspace* ws;         // the workspace (its first word is the status word)
  uint64_t n;
  uint64_t n_tiles;         // tiles of kMbqTile elements
  uint32_t n_blocks;        // 256-thread groups of the encode pass that have tiles
  uint32_t n_residue_blocks;  // blocks of a residue pass
  uint32_t k, batch_index, init;
};

__device__ __forceinline__ uint32_t mbq_header_word(const MbqArgs& a, int i) {
  switch (i) {
    case 0: return 0x54504341u;
    case 1: return 1u;
    case 2: return (uint32_t)a.n;
    case 3: return (uint32_t)(a.n >> 32);
    case 5: return a.k;
    case 7: return 1u;  // stream kind: multi-bit quantization
    default: return 0u;
  }
}

// level(c) for the coefficients in alpha[0..K)
template <int K>
__device__ __forceinline__ float mbq_level(const float* alpha, uint32_t c) {
  float v = 0.0f;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    const float term = ((c >> j) & 1u) ? alpha[j] : -alpha[j];
    v = (j == 0) ? term : __fadd_rn(v, term);
  }
  return v;
}

// Search table for the nearest level: thresholds between neighbouring sorted levels and the code
// of each sorted position.  A threshold is the midpoint rounded DOWN to fp32 (the sum and, for
// subnormal levels, the halving too): for an fp32 x, "x > threshold" is then exactly "x is above
// the true midpoint" (a tie goes to the lower level).  Level sums must stay below the fp32 maximum.
// Positions whose levels coincide all map to the smallest code among them.
template <int K>
struct MbqTable {
  float thr[1 << K];     // thr[i], i >= 1: between sorted positions i-1 and i; thr[0] unused
  uint32_t code[1 << K];
};

template <int K>
__device__ void mbq_build_table(const float* alpha_global, MbqTable<K>* t, float* s_level, int tid) {
  constexpr int L = 1 << K;
  __shared__ float s_sorted[16];
  float alpha[K];
#pragma unroll
  for (int j = 0; j < K; ++j) alpha[j] = ldg_c(alpha_global + j);
  if (tid < L) s_level[tid] = mbq_level<K>(alpha, tid);
  __syncthreads();
  if (tid < L) {
    const float mine = s_level[tid];
    int rank = 0;
    uint32_t first = tid;
    for (int d = 0; d < L; ++d) {
      const float other = s_level[d];
      rank += (other < mine || (other == mine && d < tid)) ? 1 : 0;
      if (other == mine && (uint32_t)d < first) first = d;
    }
    s_sorted[rank] = mine;
    t->code[rank] = first;
  }
  __syncthreads();
  if (tid >= 1 && tid < L) t->thr[tid] = __fmul_rd(__fadd_rd(s_sorted[tid - 1], s_sorted[tid]), 0.5f);
  if (tid == 0) t->thr[0] = 0.0f;
  __syncthreads();
}

// Branch-free binary search over the sorted thresholds; the position is kept as a byte offset so
// that every probe is a shared-memory load with an immediate displacement.
template <int K>
__device__ __forceinline__ uint32_t mbq_nearest_code(const MbqTable<K>& t, float x) {
  constexpr int L = 1 << K;
  const char* thr = reinterpret_cast<const char*>(t.thr);
  uint32_t off = 0;
#pragma unroll
  for (int step = L / 2; step >= 1; step >>= 1)
    if (x > *reinterpret_cast<const float*>(thr + off + 4 * step)) off += 4 * step;
  return *reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(t.code) + off);
}

// ---- signs as flag bytes ------------------------------------------------------------------------
//
// Inside the encode pass the k signs of an element travel as a word with one FLAG BYTE per basis:
// byte j = 0x10 when b_j = +1, else 0.  Two things come cheaply from that form:
//  * moved to byte 3 of the high word of a double (low word 0), a flag byte is the number
//    2^-767 (exponent field 0x100) or +0: "add x to the sum of basis j when b_j = +1" becomes one
//    byte permute and one fused multiply-add, acc += x * flag.  Scaling by a power of two is exact
//    (|x| from 2^-149 to 2^128 stays far inside the range of a double), so the sums are the plain
//    ones times 2^-767 and are scaled back exactly at the end;
//  * the plane form of an octet (byte j = the signs of basis j of its 8 elements) is a sum of the
//    eight words times 1, 2, 4, 8: integer multiply-adds instead of byte permutes and bit swaps.
constexpr uint32_t kMbqFlag = 0x10u;

// code (bit j = [b_j = +1]) -> flag bytes
__device__ __forceinline__ uint32_t mbq_flags_of_code(uint32_t c) {
  return ((c * 0x00204081u) & 0x01010101u) << 4;
}

// acc += x * (flag byte J of `flags` as a double: 2^-767 or +0)
template <int J>
__device__ __forceinline__ void mbq_add_flagged(double& acc, double x, uint32_t flags) {
  acc = __fma_rn(x, __hiloint2double((int)__byte_perm(flags, 0u, 0x0444u | ((uint32_t)J << 12)), 0), acc);
}

// flag words of the 8 elements of an octet -> plane form (bit 8*j + e = [b_j of element e = +1])
__device__ __forceinline__ uint32_t mbq_planes_of_flags(const uint32_t (&f)[8]) {
  const uint32_t lo = f[0] + 2u * f[1] + 4u * f[2] + 8u * f[3];  // bits 4..7 of every byte: elements 0..3
  const uint32_t hi = f[4] + 2u * f[5] + 4u * f[6] + 8u * f[7];  // bits 4..7 of every byte: elements 4..7
  return (lo >> 4) | hi;
}

// Nearest level through a uniform grid.  The span of the levels (with a margin) is cut into 256
// cells; mbq_cell() is a non-decreasing function of x, so every x of a cell below the cell of a
// threshold lies below that threshold and every x of a cell above it lies above.  When no cell
// holds more than one threshold, one comparison with "the threshold inside my cell" finishes the
// search: entry = {that threshold (+inf if the cell has none), flag bytes of the code below it,
// flag bytes of the code above it, 0}.  The decisions are the ones of the threshold search, exactly;
// when two thresholds share a cell (coinciding or very close levels), or a level is not finite,
// the grid is marked unusable and the kernel searches the sorted thresholds instead.
//
// The grid is stored eight times, entry (cell, column) at byte 128 * cell + 16 * column, and lane l
// reads column l & 7: a 128-bit shared load is served a quarter warp at a time, and the eight lanes of a
// quarter warp then touch eight different 16-byte columns of the banks whatever cells they ask for: no
// bank conflicts (a single copy cost 8.6 wavefronts per load on post-ReLU data).  32 KB per block.
struct MbqGridInfo {
  float scale;  // 1 / (2 * 1.03125 * largest |level|)
  int usable;
};

// Byte offset of the cell of x inside a column of the grid (128 * cell, cell = 0 .. 255).  Two fused
// multiply-adds on the FMA pipe and one logic operation: the first maps the span onto [0, 1] and saturates
// (NaN goes to 0), the second leaves round(255 * 128 * t) in the low mantissa bits; keeping bits 7..14 of it
// gives 128 * floor(that / 128).  Non-decreasing in x.  (A float-to-integer conversion would do the same in
// one instruction less, but it runs on the conversion unit, which this kernel already keeps busy: measured.)
__device__ __forceinline__ uint32_t mbq_cell_offset(float x, float scale) {
  float t;
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(t) : "f"(x), "f"(scale));
  return __float_as_uint(__fmaf_rn(t, 32640.0f, kMagic)) & 0x7F80u;
}

// Called by all threads of the block.
template <int K>
__device__ void mbq_build_grid(const MbqTable<K>& t, const float* s_level, MbqGridInfo* info, uint4* cells, int tid,
                               int n_threads) {
  constexpr int L = 1 << K;
  __shared__ uint32_t s_cell_of[L];
  __shared__ uint4 s_entry[kMbqCells];
  if (tid == 0) {
    float amax = 0.0f;
    bool finite = true;
    for (int c = 0; c < L; ++c) {
      finite = finite && is_finite_bits(s_level[c]);
      amax = fmaxf(amax, fabsf(s_level[c]));
    }
    const float scale = __fdiv_rn(0.5f, __fmul_rn(amax, 1.03125f));
    info->scale = scale;
    info->usable = (finite && amax > 0.0f && is_finite_bits(scale)) ? 1 : 0;
  }
  __syncthreads();
  if (tid >= 1 && tid < L) s_cell_of[tid] = mbq_cell_offset(t.thr[tid], info->scale) >> 7;
  __syncthreads();
  if (tid < kMbqCells) {
    int below = 0, inside = 0;
    float thr = __int_as_float(0x7f800000);
    for (int m = 1; m < L; ++m) {
      const uint32_t c = s_cell_of[m];
      below += (c < (uint32_t)tid) ? 1 : 0;
      if (c == (uint32_t)tid) { ++inside; thr = t.thr[m]; }
    }
    const uint32_t lo = t.code[below], hi = t.code[below + 1 < L ? below + 1 : L - 1];
    s_entry[tid] = make_uint4(__float_as_uint(thr), mbq_flags_of_code(lo), mbq_flags_of_code(hi), 0u);
    if (inside > 1) info->usable = 0;
  }
  __syncthreads();
  if (info->usable)
    for (int i = tid; i < kMbqCells * kMbqColumns; i += n_threads) cells[i] = s_entry[i / kMbqColumns];
  __syncthreads();
}

// flag bytes of the nearest level's code; column = this lane's copy of the grid (byte address in shared memory)
__device__ __forceinline__ uint32_t mbq_grid_flags(uint32_t column, float scale, float x) {
  uint4 e;
  const uint32_t addr = mbq_cell_offset(x, scale) + column;
  asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(e.x), "=r"(e.y), "=r"(e.z), "=r"(e.w) : "r"(addr));
  return (x > __uint_as_float(e.x)) ? e.z : e.y;
}

// Signs of the successive residues with the given coefficients (residue method): bit j = [r_j >= 0].
// Returns the residue after `upto` steps in *residue.
template <int K>
__device__ __forceinline__ uint32_t mbq_residue_code(const float (&alpha)[K], float x, int upto, float* residue) {
  float r = x;
  uint32_t c = 0;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    if (j < upto) {
      if (r >= 0.0f) { c |= 1u << j; r = __fsub_rn(r, alpha[j]); }
      else r = __fadd_rn(r, alpha[j]);
    }
  }
  *residue = r;
  return c;
}

__device__ __forceinline__ void mbq_ld_octet(const float* x, uint64_t n, uint64_t oct, float (&v)[8]) {
  const uint64_t e = oct * 8;
  if (e + 8 <= n) {
    ld_octet(x + e, v);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = (e + i < n) ? ldg_c(x + e + i) : 0.0f;
  }
}

// ---- exact sums of a block ------------------------------------------------------------------------

// What the threads of a block share for their exact sums: the block's wide sums (slot j = basis j,
// slot kMbqSums - 1 = the sum of x, or the only sum of a residue pass) and the window of the fast path.
struct MbqBlockSums {
  long long wide[kMbqSums][kAccLimbs];
  ExactWindow window;
};

__device__ __forceinline__ void mbq_block_sums_clear(MbqBlockSums* bs, int tid, int n_threads) {
  for (int i = tid; i < kMbqSums * kAccLimbs; i += n_threads) (&bs->wide[0][0])[i] = 0;
}

// A value outside the window: straight into the block's wide sums of `slots` (bit s set: slot s).
__device__ __noinline__ void mbq_wide_add_value(MbqBlockSums* bs, uint32_t* status, float x, uint32_t slots) {
  for (int s = 0; s < kMbqSums; ++s)
    if ((slots >> s) & 1u)
      if (!wide_add_float(bs->wide[s], x, false)) atomicOr(status, kDevNonFinite);
}

// Thread s < kMbqSums hands slot s of the block's wide sums to the workspace: carries propagated first, so
// that each piece is below 2^32 and the 64-bit words of the workspace cannot overflow whatever the grid.
// Call after a __syncthreads() that follows the last addition.
__device__ inline void mbq_block_sums_deliver(MbqBlockSums* bs, MbqWorkspace* ws, int tid) {
  if (tid >= kMbqSums) return;
  long long limbs[kAccLimbs];
  bool any = false;
#pragma unroll
  for (int i = 0; i < kAccLimbs; ++i) { limbs[i] = bs->wide[tid][i]; any = any || limbs[i] != 0; }
  if (!any) return;
  wide_normalise(limbs);
#pragma unroll
  for (int i = 0; i < kAccLimbs; ++i)
    if (limbs[i] != 0) limb_add(&ws->wide[tid][i], limbs[i]);
}

// ---- residue method ---------------------------------------------------------------------------------

// Residue method, step j: alpha_j = mean |r_j| (r_0 = x) with the coefficients found so far.  Every block
// adds the |r_j| of its tiles exactly and hands the sum to the workspace; the block that arrives last
// rounds the total once, divides by n and leaves the workspace clean for the next pass.  No block waits
// for another.
// J = j, the number of coefficients already known (a template parameter: the residue of a value is then J
// straight-line steps).
template <int K, int J>
__global__ void __launch_bounds__(256) mbq_residue_sum_kernel(const MbqArgs a) {
  constexpr int j = J;
  grid_dependency_handshake();
  __shared__ MbqBlockSums s_sums;
  __shared__ float s_amax[8];
  __shared__ uint32_t s_is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int SLOT = kMbqSums - 1;
  float alpha[K];
#pragma unroll
  for (int i = 0; i < K; ++i) alpha[i] = (i < j) ? a.ws->alpha_init[i] : 0.0f;
  const uint64_t n_oct = (a.n + 7) / 8;
  mbq_block_sums_clear(&s_sums, tid, 256);

  // Window of the fast path: around the coefficient of the first basis once it is known; for the first
  // pass around the largest magnitude of the block's first octets.
  float scale = alpha[0];
  if (j == 0) {
    const uint64_t oct = (uint64_t)blockIdx.x * (kMbqRounds * 256) + tid;
    float m = 0.0f;
    if (oct < n_oct) {
      float v[8];
      mbq_ld_octet(a.x, a.n, oct, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) m = fmaxf(m, fabsf(v[e]));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) s_amax[warp] = m;
    __syncthreads();
    scale = 0.0f;
    for (int w = 0; w < 8; ++w) scale = fmaxf(scale, s_amax[w]);
    scale *= 0.125f;  // the top of the window is 2^9 above the binade of the scale
  }
  if (tid == 0) s_sums.window = make_window(scale);
  __syncthreads();
  const ExactWindow win = s_sums.window;

  double acc = 0.0;
  long long irun = 0;
  int since = 0, flushes = 0;
  // |r_j| of one octet into the accumulator; `valid` < 8 only for the octet that holds the end of the tensor
  auto add_octet = [&](const float (&v)[8], int valid) {
    float res[8];
    WindowCheck chk;
    chk.init();
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float rr = v[e];
#pragma unroll
      // a step takes alpha_i towards zero from the side the residue is on.  Only |r| is summed here, and the
      // steps commute with r -> -r, so -0 may go either way: subtracting alpha_i with the residue's sign bit
      // gives the same |r| as the comparison r >= 0 that assigns the signs in the encode pass.
      for (int i = 0; i < J; ++i) rr = __fsub_rn(rr, copysignf(alpha[i], rr));
      res[e] = fabsf(rr);
    }
    if (valid < 8) {  // nothing past the end
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (e >= valid) res[e] = 0.0f;
    }
#pragma unroll
    for (int e = 0; e < 8; e += 2) chk.add2(res[e], res[e + 1]);
    if (!chk.ok(win)) {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (!in_window(win, res[e])) {
          mbq_wide_add_value(&s_sums, a.status, res[e], 1u << SLOT);
          res[e] = 0.0f;
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) acc += (double)res[e];
  };
  auto tile_done = [&]() {
    if (++since == kMbqFlushTiles) {
      since = 0;
      irun += __double2ll_rn(acc * win.to_units);
      acc = 0.0;
      if (++flushes == kPushFlushes) {  // the same for every thread of the block: tiles are the block's
        flushes = 0;
        const long long total = warp_sum_int64(irun);
        if (lane == 0) wide_add_int64(s_sums.wide[SLOT], total, win.pos);
        irun = 0;
      }
    }
  };
  // Full tiles: no guards, and the octets of the block's next tile are in flight while the current ones are
  // added up (two sets of registers used in turn).
  const uint64_t full_tiles = a.n / kMbqTile;
  auto load_tile = [&](uint64_t tile, float (&v)[kMbqRounds][8]) {
    const float* src = a.x + tile * kMbqTile + 8u * tid;
#pragma unroll
    for (int r = 0; r < kMbqRounds; ++r) ld_octet(src + r * (256 * 8), v[r]);
  };
  auto add_tile = [&](const float (&v)[kMbqRounds][8]) {
#pragma unroll
    for (int r = 0; r < kMbqRounds; ++r) add_octet(v[r], 8);
    tile_done();
  };
  {
    float va[kMbqRounds][8], vb[kMbqRounds][8];
    const uint64_t stride = gridDim.x;
    uint64_t tile = blockIdx.x;
    if (tile < full_tiles) load_tile(tile, va);
    while (tile < full_tiles) {
      if (tile + stride < full_tiles) load_tile(tile + stride, vb);
      add_tile(va);
      tile += stride;
      if (tile >= full_tiles) break;
      if (tile + stride < full_tiles) load_tile(tile + stride, va);
      add_tile(vb);
      tile += stride;
    }
  }
  // the ragged last tile, by the block whose turn it is
  if (full_tiles < a.n_tiles && full_tiles % gridDim.x == blockIdx.x) {
#pragma unroll 1
    for (int r = 0; r < kMbqRounds; ++r) {
      const uint64_t oct = full_tiles * (kMbqRounds * 256) + r * 256 + tid;
      if (oct < n_oct) {
        float v[8];
        mbq_ld_octet(a.x, a.n, oct, v);
        const uint64_t left = a.n - oct * 8;
        add_octet(v, left >= 8 ? 8 : (int)left);
      }
    }
  }
  irun += __double2ll_rn(acc * win.to_units);
  {
    const long long total = warp_sum_int64(irun);
    if (lane == 0) wide_add_int64(s_sums.wide[SLOT], total, win.pos);
  }
  __syncthreads();
  if (tid == SLOT) mbq_block_sums_deliver(&s_sums, a.ws, tid);
  // the last block to get here finishes the pass
  if (tid == SLOT) {
    __threadfence();
    const uint32_t ticket = atomicAdd(&a.ws->blocks_done, 1u);
    s_is_last = (ticket == gridDim.x - 1) ? 1u : 0u;
  }
  __syncthreads();
  if (s_is_last && tid == 0) {
    __threadfence();
    long long total[kAccLimbs];
#pragma unroll
    for (int i = 0; i < kAccLimbs; ++i) {
      total[i] = (long long)atomicExch(reinterpret_cast<unsigned long long*>(&a.ws->wide[SLOT][i]), 0ull);
    }
    // (the block's own wide sums have been delivered: their storage serves as scratch)
    a.ws->alpha_init[j] = (float)(wide_to_double(total, reinterpret_cast<uint32_t*>(&s_sums.wide[0][0])) / (double)a.n);
    a.ws->blocks_done = 0u;
  }
}

// How the signs of an element are found.
constexpr int kMbqResidue = 0, kMbqSearch = 1, kMbqGrid = 2;

// Running sums of one thread over all its groups.  plus[] and sum_x hold what the thread added since its
// last flush (plus[] times 2^-767, the flag factor); irun[] the flushed part in units of the window.
template <int K>
struct MbqSums {
  double plus[K], sum_x;
  long long irun[K + 1];   // [K]: the sum of x
  uint32_t count[K];       // +1 signs per basis
  uint32_t differ[6];      // pairs (0,1) (0,2) (0,3) (1,2) (1,3) (2,3): elements whose two signs differ
  __device__ __forceinline__ void clear() {
    sum_x = 0.0;
#pragma unroll
    for (int j = 0; j < K; ++j) { plus[j] = 0.0; count[j] = 0; }
#pragma unroll
    for (int j = 0; j <= K; ++j) irun[j] = 0;
#pragma unroll
    for (int d = 0; d < 6; ++d) differ[d] = 0;
  }
};

// Accumulators -> integer units of the window, exactly (see accept_exact.cuh).
template <int K>
__device__ __forceinline__ void mbq_flush(MbqSums<K>& s, const MbqBlockSums* bs) {
  const double to_units = bs->window.to_units;
  const double flag_to_units = to_units * 0x1p767;  // the flag factor was 2^-767
#pragma unroll
  for (int j = 0; j < K; ++j) {
    s.irun[j] += __double2ll_rn(s.plus[j] * flag_to_units);
    s.plus[j] = 0.0;
  }
  s.irun[K] += __double2ll_rn(s.sum_x * to_units);
  s.sum_x = 0.0;
}

// Running int64 sums of a warp -> the block's wide sums.  All lanes of the warp call.
template <int K>
__device__ __forceinline__ void mbq_push(MbqSums<K>& s, MbqBlockSums* bs, int lane) {
  const int pos = bs->window.pos;
#pragma unroll
  for (int j = 0; j <= K; ++j) {
    const long long total = warp_sum_int64(s.irun[j]);
    if (lane == 0) wide_add_int64(bs->wide[j < K ? j : kMbqSums - 1], total, pos);
    s.irun[j] = 0;
  }
}

// What a thread needs to find the signs of a value.
template <int K>
struct MbqLookup {
  const MbqTable<K>* table;  // sorted thresholds (kMbqSearch)
  uint32_t column;           // shared-memory byte address of this lane's column of the grid (kMbqGrid)
  float scale;               // of the grid
  float alpha[K];            // coefficients of the residue method (kMbqResidue)
};

template <int K, int MODE>
__device__ __forceinline__ uint32_t mbq_flags_of_value(const MbqLookup<K>& lk, float x) {
  if (MODE == kMbqGrid) return mbq_grid_flags(lk.column, lk.scale, x);
  if (MODE == kMbqSearch) return mbq_flags_of_code(mbq_nearest_code<K>(*lk.table, x));
  float res;
  return mbq_flags_of_code(mbq_residue_code<K>(lk.alpha, x, K, &res));
}

// x into the thread's accumulators: the sum of x, and the sum of every basis whose flag byte is set.
template <int K>
__device__ __forceinline__ void mbq_accumulate(MbqSums<K>& sums, float x, uint32_t flags) {
  const double xd = (double)x;
  sums.sum_x += xd;
  mbq_add_flagged<0>(sums.plus[0], xd, flags);
  mbq_add_flagged<1>(sums.plus[1], xd, flags);
  if constexpr (K > 2) mbq_add_flagged<2>(sums.plus[2], xd, flags);
  if constexpr (K > 3) mbq_add_flagged<3>(sums.plus[3], xd, flags);
}

// Four values of a group whose 32 values all lie inside the window: their signs, their share of the
// sums; returns the signs as a word whose byte j holds, in its bits 4..7, basis j of the four values.
template <int K, int MODE>
__device__ __forceinline__ uint32_t mbq_code_four(const MbqLookup<K>& lk, const float4 v, MbqSums<K>& sums) {
  const float w[4] = {v.x, v.y, v.z, v.w};
  uint32_t f[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) f[e] = mbq_flags_of_value<K, MODE>(lk, w[e]);
#pragma unroll
  for (int e = 0; e < 4; ++e) mbq_accumulate<K>(sums, w[e], f[e]);
  return f[0] + 2u * f[1] + 4u * f[2] + 8u * f[3];
}

// One value of a group that holds values outside the window, or fewer than 32 values (the ragged end of
// the tensor): its signs are returned, and the value goes into the block's wide sums (the sum of x, and
// the sum of every basis whose sign is +1) instead of the thread's accumulators -- exact wherever it lies.
// Rare: kept out of line, and everything is passed by value so that the caller's state stays in registers.
template <int K, int MODE>
__device__ __noinline__ uint32_t mbq_code_value_slowly(MbqLookup<K> lk, float x, MbqBlockSums* bs, uint32_t* status) {
  const uint32_t f = mbq_flags_of_value<K, MODE>(lk, x);
  // flag bytes (0x10 per basis) -> slot bits, plus the slot of the sum of x
  const uint32_t slots = ((((f >> 4) * 0x00204081u) >> 21) & 0xFu) | (1u << (kMbqSums - 1));
  mbq_wide_add_value(bs, status, x, slots);
  return f;
}

// The eight sign words of a group (slot c: bits 4..7 of byte j = basis j of values 4c..4c+3) -> the K plane
// words of the group (bit t of word j = basis j of value t), counted and stored.
template <int K>
__device__ __forceinline__ void mbq_finish_group(const MbqArgs& a, const uint32_t (&s4)[8], uint32_t rotate_bits,
                                                 uint64_t group, bool store, MbqSums<K>& sums) {
  // pairs of slots: byte j = basis j of eight values
  uint32_t b[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) b[i] = (s4[2 * i] >> 4) | s4[2 * i + 1];
  // 4 x 4 byte transpose: word j = basis j of all 32 values, in the order of the slots
  const uint32_t t0 = __byte_perm(b[0], b[1], 0x5140), t1 = __byte_perm(b[2], b[3], 0x5140);
  const uint32_t t2 = __byte_perm(b[0], b[1], 0x7362), t3 = __byte_perm(b[2], b[3], 0x7362);
  uint32_t word[4];
  word[0] = __byte_perm(t0, t1, 0x5410);
  word[1] = __byte_perm(t0, t1, 0x7632);
  word[2] = __byte_perm(t2, t3, 0x5410);
  word[3] = __byte_perm(t2, t3, 0x7632);
  // the slots were read in an order rotated by the lane (bank conflicts): turn the words back
#pragma unroll
  for (int j = 0; j < K; ++j) word[j] = __funnelshift_l(word[j], word[j], rotate_bits);
#pragma unroll
  for (int j = 0; j < K; ++j) sums.count[j] += __popc(word[j]);
  {
    int pair = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = i + 1; j < 4; ++j, ++pair)
        if (j < K) sums.differ[pair] += __popc(word[i] ^ word[j]);
  }
  if (store) {
    uint32_t* out = a.payload + group * K;
    if (K == 4) {
      st_c(reinterpret_cast<uint4*>(out), make_uint4(word[0], word[1], word[2], word[3]));
    } else if (K == 2) {
      st_c(reinterpret_cast<uint2*>(out), make_uint2(word[0], word[1]));
    } else {
#pragma unroll
      for (int j = 0; j < K; ++j) st_c(out + j, word[j]);
    }
  }
}

// Scratch of the finalize step, in shared memory: nothing of it is indexed out of a thread's own arrays.
struct MbqFinalScratch {
  long long wide[kMbqSums][kAccLimbs];        // the sums of the workspace
  uint32_t digits[kMbqSums][kAccLimbs + 2];   // wide_to_double's
  unsigned long long cnt[10];
  double val[kMbqSums];                       // [j] = (B^T x)_j, [K] = sum of x
  float alpha_prev[4];
};

// Solves the K x K system G y = rhs by Gaussian elimination with partial pivoting in double, every index a
// compile-time constant (rows are exchanged by conditional moves).  Returns false if a pivot is below
// 1e-9 * N (singular: the caller keeps the previous coefficients).
template <int K>
__device__ __forceinline__ bool mbq_solve(double (&G)[K][K], double (&rhs)[K], double N, double (&y)[K]) {
  bool singular = false;
#pragma unroll
  for (int col = 0; col < K; ++col) {
    // the row, from col down, whose entry in this column is largest in magnitude: the first such row
    int piv = col;
    double best = fabs(G[col][col]);
#pragma unroll
    for (int r = col + 1; r < K; ++r) {
      const double v = fabs(G[r][col]);
      if (v > best) { best = v; piv = r; }
    }
    if (best < 1e-9 * N) singular = true;
#pragma unroll
    for (int r = col + 1; r < K; ++r) {
      if (r == piv) {
#pragma unroll
        for (int q = 0; q < K; ++q) { const double t = G[col][q]; G[col][q] = G[r][q]; G[r][q] = t; }
        const double t = rhs[col]; rhs[col] = rhs[r]; rhs[r] = t;
      }
    }
    if (!singular) {
#pragma unroll
      for (int r = col + 1; r < K; ++r) {
        const double f = G[r][col] / G[col][col];
#pragma unroll
        for (int q = col; q < K; ++q) G[r][q] -= f * G[col][q];
        rhs[r] -= f * rhs[col];
      }
    }
  }
  if (singular) return false;
#pragma unroll
  for (int col = K - 1; col >= 0; --col) {
    double s = rhs[col];
#pragma unroll
    for (int q = col + 1; q < K; ++q) s -= G[col][q] * y[q];
    y[col] = s / G[col][col];
  }
  return true;
}

// The end of the encode pass, run by the block that delivers its sums last (all threads of it call): rounds
// the exact sums once, then Eq. 3 (least squares), Eq. 4 (moving average), Eq. 5 (bias), and writes header,
// side words and alpha_next; leaves the sums of the workspace zeroed for the next call.
template <int K>
__device__ void mbq_finalize(const MbqArgs& a, int tid, MbqFinalScratch* fs) {
  MbqWorkspace* ws = a.ws;
  // one round trip for everything the step reads (the sums were written by other blocks' atomic adds: read
  // them where atomics are performed)
  if (tid < kMbqSums * kAccLimbs) (&fs->wide[0][0])[tid] = __ldcg(&ws->wide[0][0] + tid);
  else if (tid < kMbqSums * kAccLimbs + 4) fs->cnt[tid - kMbqSums * kAccLimbs] = __ldcg(&ws->count[tid - kMbqSums * kAccLimbs]);
  else if (tid < kMbqSums * kAccLimbs + 10) fs->cnt[tid - kMbqSums * kAccLimbs] = __ldcg(&ws->differ[tid - kMbqSums * kAccLimbs - 4]);
  else if (tid < kMbqSums * kAccLimbs + 10 + K && !a.init) fs->alpha_prev[tid - kMbqSums * kAccLimbs - 10] = ldg_c(a.alpha_prev + (tid - kMbqSums * kAccLimbs - 10));
  else if (tid >= 96 && tid < 96 + 8) st_c(a.header + (tid - 96), mbq_header_word(a, tid - 96));
  __syncthreads();
  // the next call starts from zero
  if (tid < kMbqSums * kAccLimbs) (&ws->wide[0][0])[tid] = 0;
  if (tid >= 64 && tid < 68) ws->count[tid - 64] = 0;
  if (tid >= 68 && tid < 74) ws->differ[tid - 68] = 0;
  if (tid == 74) { ws->blocks_done = 0u; ws->next_tile = 0u; }
  if (tid <= K) {
    long long lazy[kAccLimbs];
#pragma unroll
    for (int i = 0; i < kAccLimbs; ++i) {
      const long long sx = fs->wide[kMbqSums - 1][i];
      // sum over the +1 elements minus sum over the -1 elements = 2 * (sum over +1) - (sum of all), digit by digit
      lazy[i] = (tid < K) ? 2 * fs->wide[tid][i] - sx : sx;
    }
    fs->val[tid] = wide_to_double(lazy, fs->digits[tid]);
  }
  __syncthreads();
  if (tid != 0) return;

  const double N = (double)a.n, sum_x = fs->val[K];
  float alpha_next[K];
  if (a.init) {
#pragma unroll
    for (int j = 0; j < K; ++j) alpha_next[j] = ws->alpha_init[j];
  } else {
    double G[K][K], rhs[K], cur[K], prev[K];
    {
      int pair = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = i + 1; j < 4; ++j, ++pair)
          if (j < K) G[i][j] = G[j][i] = N - 2.0 * (double)fs->cnt[4 + pair];
    }
#pragma unroll
    for (int j = 0; j < K; ++j) {
      G[j][j] = N;
      rhs[j] = fs->val[j];
      prev[j] = (double)fs->alpha_prev[j];
      cur[j] = 0.0;
    }
    if (!mbq_solve<K>(G, rhs, N, cur)) {
#pragma unroll
      for (int j = 0; j < K; ++j) cur[j] = prev[j];
    }
    double beta = (1.0 + (double)a.batch_index) / (10.0 + (double)a.batch_index);
    if (beta > 0.9) beta = 0.9;
#pragma unroll
    for (int j = 0; j < K; ++j) alpha_next[j] = (float)(beta * prev[j] + (1.0 - beta) * cur[j]);
  }
  double acc = 0.0;
#pragma unroll
  for (int j = 0; j < K; ++j) acc += (double)alpha_next[j] * (2.0 * (double)fs->cnt[j] - N);
  const float m_q = (float)((acc - sum_x) / N);
#pragma unroll
  for (int j = 0; j < K; ++j) { st_c(a.side + j, alpha_next[j]); st_c(a.alpha_next + j, alpha_next[j]); }
  st_c(a.side + K, m_q);
  // pad up to the payload
  for (uint32_t* w = reinterpret_cast<uint32_t*>(a.side + K + 1); w < a.payload; ++w) st_c(w, 0u);
}

// Shared state of a block of the encode pass besides the dynamic shared memory (grid, then stages).
template <int K>
struct MbqEncodeShared {
  MbqTable<K> table;
  MbqGridInfo grid;
  MbqBlockSums sums;
  float level[16];
  uint32_t cnt[10];
  uint32_t failed;
  uint32_t is_last;
  uint32_t tile[kMbqStages];   // tile each stage holds or is waiting for
  MbqFinalScratch final_step;
  alignas(8) unsigned long long bar[kMbqStages];
};

// Thread 0 asks for a full tile: bulk copies that count their bytes on the stage's mbarrier.
__device__ __forceinline__ void mbq_request_tile(const MbqArgs& a, uint64_t tile, uint8_t* stage, uint32_t bar) {
  mbarrier_expect_bytes(bar, kMbqTileBytes + kCopyAnnounceExtra);
  const uint8_t* src = reinterpret_cast<const uint8_t*>(a.x + tile * kMbqGroupTile);
  const uint32_t dst = smem_address(stage);
#pragma unroll
  for (int part = 0; part < kMbqTileBytes / kMbqCopyBytes; ++part)
    if (bounds_ok(src + part * kMbqCopyBytes, kMbqCopyBytes, false))
      bulk_copy_to_shared(dst + part * kMbqCopyBytes, src + part * kMbqCopyBytes, kMbqCopyBytes, bar);
}

// The tiles of one block.  Full tiles are staged: thread 0 asks for a tile with four bulk copies that
// count their bytes on the stage's mbarrier; when a tile has landed every thread codes its group out of
// shared memory, and after the block has met at a barrier the stage is asked to fetch the tile after next.
// A thread reads its 128 bytes as eight 16-byte slots in an order rotated by its lane, so that the eight
// lanes of a quarter warp, whose groups are 128 bytes apart, hit eight different bank columns.  The ragged
// last tile of the tensor is read from global memory with guards, by the block whose turn it is.
// Returns false if a copy did not arrive in time (reported in the status word; the caller leaves).
template <int K, int MODE>
__device__ __forceinline__ bool mbq_encode_tiles(const MbqArgs& a, const MbqLookup<K>& lk, MbqEncodeShared<K>* sh,
                                                 uint8_t* stages, MbqSums<K>& sums) {
  const int tid = threadIdx.x, lane = tid & 31;
  MbqBlockSums* bs = &sh->sums;
  const float win_top = bs->window.top;
  const uint32_t win_ylow = bs->window.ylow;
  const uint32_t bar[kMbqStages] = {smem_address(&sh->bar[0]), smem_address(&sh->bar[1])};
  const uint64_t full_tiles = a.n / kMbqGroupTile;
  const uint32_t stride = gridDim.x;
  auto request = [&](uint64_t tile, int st) { mbq_request_tile(a, tile, stages + st * kMbqTileBytes, bar[st]); };
  // (the block's first two tiles were asked for before the tables were built; see the kernel)
  bool pending[kMbqStages] = {false, false};  // thread 0: a copy of the stage's current phase is in flight
  if (tid == 0) {
#pragma unroll
    for (int st = 0; st < kMbqStages; ++st) pending[st] = sh->tile[st] < full_tiles;
  }
  // Tiles beyond every block's first two are handed out in the order blocks ask for them, so that the blocks end
  // together.  Thread 0 always holds one ticket in hand: the atomic that fetches the next one has a whole tile's
  // time to come back and never delays a request.
  uint64_t ticket = 0;
  if (tid == 0 && pending[kMbqStages - 1]) ticket = (uint64_t)kMbqStages * stride + atomicAdd(&a.ws->next_tile, 1u);
  const uint32_t rot = (uint32_t)(tid & 7);  // slot c of this thread holds values 4 * ((c + rot) & 7) .. + 3 of its group
  uint32_t slot_offset[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) slot_offset[c] = 16u * ((c + rot) & 7u);
  uint32_t parity[kMbqStages] = {0u, 0u};
  int since_flush = 0, since_push = 0;  // the same in every thread: all code the same number of groups
  for (int st = 0;; st ^= 1) {
    const uint64_t tile = sh->tile[st];  // written before the last barrier
    if (tile >= full_tiles) break;
    if (mbarrier_wait(bar[st], parity[st])) {
      parity[st] ^= 1u;
      if (tid == 0) pending[st] = false;
    } else {
      atomicOr(a.status, kDevCopyTimeout);
      sh->failed = 1u;  // seen by everybody after the barrier below; this tile's values are whatever the stage holds
    }
    const uint8_t* mine = stages + st * kMbqTileBytes + tid * 128;
    // first look: are all 32 values inside the window of the exact sums (or zero)?
    WindowCheck chk;
    chk.init();
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float4 v = *reinterpret_cast<const float4*>(mine + slot_offset[c]);
      chk.add2(v.x, v.y);
      chk.add2(v.z, v.w);
    }
    uint32_t s4[8];
    if (chk.amax < win_top && chk.ymin >= win_ylow) {
#pragma unroll
      for (int c = 0; c < 8; ++c)
        s4[c] = mbq_code_four<K, MODE>(lk, *reinterpret_cast<const float4*>(mine + slot_offset[c]), sums);
    } else {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t word = 0;
#pragma unroll 1
        for (int e = 0; e < 4; ++e)
          word += mbq_code_value_slowly<K, MODE>(lk, *reinterpret_cast<const float*>(mine + slot_offset[c] + 4 * e), bs, a.status) << e;
        s4[c] = word;
      }
    }
    mbq_finish_group<K>(a, s4, 4u * rot, tile * kMbqEncodeThreads + tid, true, sums);
    __syncthreads();  // every thread has taken its values out of the stage
    if (sh->failed) break;
    if (tid == 0) {
      const uint64_t next = ticket;
      sh->tile[st] = next < full_tiles ? (uint32_t)next : 0xFFFFFFFFu;
      if (next < full_tiles) {
        request(next, st);
        pending[st] = true;
        ticket = (uint64_t)kMbqStages * stride + atomicAdd(&a.ws->next_tile, 1u);
      }
    }
    if (++since_flush == kMbqFlushGroups) {
      since_flush = 0;
      mbq_flush<K>(sums, bs);
      if (++since_push == kPushFlushes) {
        since_push = 0;
        mbq_push<K>(sums, bs, lane);
      }
    }
  }
  if (sh->failed) {
    // give what is still in flight a bounded time to land before the block gives its shared memory back
    if (tid == 0) {
#pragma unroll
      for (int st = 0; st < kMbqStages; ++st)
        if (pending[st]) mbarrier_wait(bar[st], parity[st]);
    }
    return false;
  }

  // the ragged last tile, read from global memory by the block whose turn it is
  if (full_tiles * kMbqGroupTile < a.n && full_tiles % stride == blockIdx.x) {
    const uint64_t first = full_tiles * kMbqGroupTile + (uint64_t)tid * 32;  // first value of this thread's group
    const uint64_t n_groups_stored = (a.n + 31) / 32;
    const int valid = first >= a.n ? 0 : (a.n - first >= 32 ? 32 : (int)(a.n - first));
    uint32_t s4[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      uint32_t word = 0;
#pragma unroll 1
      for (int e = 0; e < 4; ++e)
        if (4 * c + e < valid)  // values past the end have no signs and add nothing
          word += mbq_code_value_slowly<K, MODE>(lk, ldg_c(a.x + first + 4 * c + e), bs, a.status) << e;
      s4[c] = word;
    }
    const uint64_t group = full_tiles * kMbqEncodeThreads + tid;
    mbq_finish_group<K>(a, s4, 0u, group, group < n_groups_stored, sums);
  }
  return true;
}

// Assign the signs, write the planes, gather the sums, and (in the block that ends last) solve Eq. 3-5:
// the whole forward quantizer of a batch in one launch.  Persistent blocks of 256 threads, two per SM.
// Dynamic shared memory: the search grid (kMbqGridBytes), then the stages.
template <int K, bool INIT>
__global__ void __launch_bounds__(kMbqEncodeThreads, kMbqBlocksPerSm) mbq_encode_kernel(const MbqArgs a) {
  grid_dependency_handshake();
  extern __shared__ __align__(128) uint8_t s_dyn[];
  __shared__ MbqEncodeShared<K> sh;
  const int tid = threadIdx.x, lane = tid & 31;
  uint4* cells = reinterpret_cast<uint4*>(s_dyn);
  uint8_t* stages = s_dyn + kMbqGridBytes;

  // first of all the block's first two tiles are asked for: they arrive while the tables are built
  if (tid == 0) {
    const uint64_t full_tiles = a.n / kMbqGroupTile;
    mbarrier_init(smem_address(&sh.bar[0]), 1);
    mbarrier_init(smem_address(&sh.bar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    sh.failed = 0u;
    sh.grid.usable = 0;
#pragma unroll
    for (int st = 0; st < kMbqStages; ++st) {
      const uint64_t tile = blockIdx.x + (uint64_t)st * gridDim.x;
      sh.tile[st] = tile < full_tiles ? (uint32_t)tile : 0xFFFFFFFFu;
      if (tile < full_tiles) mbq_request_tile(a, tile, stages + st * kMbqTileBytes, smem_address(&sh.bar[st]));
    }
  }

  MbqLookup<K> lk;
  lk.table = &sh.table;
  lk.column = smem_address(cells) + 16u * (uint32_t)(lane & (kMbqColumns - 1));
  lk.scale = 0.0f;
#pragma unroll
  for (int j = 0; j < K; ++j) lk.alpha[j] = 0.0f;
  mbq_block_sums_clear(&sh.sums, tid, kMbqEncodeThreads);
  if (tid < 10) sh.cnt[tid] = 0;
  __syncthreads();  // sh.grid.usable = 0 is in place before the tables are built
  if (INIT) {
#pragma unroll
    for (int j = 0; j < K; ++j) lk.alpha[j] = a.ws->alpha_init[j];
    // window of the exact sums: around the mean magnitude of the data
    if (tid == 0) sh.sums.window = make_window(lk.alpha[0]);
  } else {
    mbq_build_table<K>(a.alpha_prev, &sh.table, sh.level, tid);
    // (the scratch of the grid builder must not be a stage: copies are landing there)
    mbq_build_grid<K>(sh.table, sh.level, &sh.grid, cells, tid, kMbqEncodeThreads);
    // window of the exact sums: around the largest level (the values the levels were fitted to)
    if (tid == 0) {
      float amax = 0.0f;
      for (int c = 0; c < (1 << K); ++c) amax = fmaxf(amax, fabsf(sh.level[c]));
      sh.sums.window = make_window(amax * 0.125f);
    }
  }
  __syncthreads();
  lk.scale = sh.grid.scale;

  MbqSums<K> sums;
  sums.clear();
  bool ok;
  if (INIT) ok = mbq_encode_tiles<K, kMbqResidue>(a, lk, &sh, stages, sums);
  else if (sh.grid.usable) ok = mbq_encode_tiles<K, kMbqGrid>(a, lk, &sh, stages, sums);
  else ok = mbq_encode_tiles<K, kMbqSearch>(a, lk, &sh, stages, sums);

  if (ok) {
    // what is left in the accumulators, then the warp's total into the block's wide sums
    mbq_flush<K>(sums, &sh.sums);
    mbq_push<K>(sums, &sh.sums, lane);
    // counts: lanes, then warps
#pragma unroll
    for (int j = 0; j < K; ++j) {
      const uint32_t c = __reduce_add_sync(0xffffffffu, sums.count[j]);
      if (lane == 0) atomicAdd(&sh.cnt[j], c);
    }
    int pair = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = i + 1; j < 4; ++j, ++pair) {
        if (j >= K) continue;
        const uint32_t c = __reduce_add_sync(0xffffffffu, sums.differ[pair]);
        if (lane == 0) atomicAdd(&sh.cnt[4 + pair], c);
      }
  }
  __syncthreads();
  if (ok) {
    mbq_block_sums_deliver(&sh.sums, a.ws, tid);
    if (tid >= 32 && tid < 42) {
      const int i = tid - 32;
      const unsigned long long c = sh.cnt[i];
      if (c) atomicAdd(i < 4 ? &a.ws->count[i] : &a.ws->differ[i - 4], c);
    }
  }
  // The block that gets here last finishes the batch (also after a copy that did not arrive: the status word
  // says so, the stream is then meaningless, but the workspace is left clean).  No block waits for another.
  __threadfence();
  __syncthreads();
  if (tid == 0) sh.is_last = (atomicAdd(&a.ws->blocks_done, 1u) == gridDim.x - 1) ? 1u : 0u;
  __syncthreads();
  if (sh.is_last) {
    __threadfence();
    mbq_finalize<K>(a, tid, &sh.final_step);
  }

}

// Receiver: planes -> codes -> level(c) - m_q.
template <int K>
__global__ void __launch_bounds__(256, 8) mbq_decode_kernel(const MbqArgs a) {
  grid_dependency_handshake();
  __shared__ float s_value[1 << K];
  const int tid = threadIdx.x, lane = tid & 31;
  if (blockIdx.x == 0 && tid < 8 && a.header[tid] != mbq_header_word(a, tid)) atomicOr(a.status, kDevBadHeader);
  if (tid < (1 << K)) {
    float alpha[K];
#pragma unroll
    for (int j = 0; j < K; ++j) alpha[j] = ldg_c(a.side + j);
    s_value[tid] = __fsub_rn(mbq_level<K>(alpha, tid), ldg_c(a.side + K));
  }
  __syncthreads();
  const uint64_t n_oct = (a.n + 7) / 8, n_groups = (a.n + 31) / 32;
  const int q = lane & 3;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const uint64_t oct = (uint64_t)blockIdx.x * 512 + r * 256 + tid;
    const uint64_t group = oct >> 2;
    uint32_t w = 0;
    if (group < n_groups && q < K) w = ldg_c(a.payload + group * K + q);
    const uint32_t nib = planes_nibbles(quad_transpose(w, lane));
    if (oct < n_oct) {
      float out[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[i] = s_value[(nib >> (8 * i)) & 0xFu];
        out[4 + i] = s_value[(nib >> (8 * i + 4)) & 0xFu];
      }
      const uint64_t e = oct * 8;
      if (e + 8 <= a.n) {
        st_octet(a.xhat + e, out);
      } else {
        for (int i = 0; i < 8; ++i)
          if (e + i < a.n) st_c(a.xhat + e + i, out[i]);
      }
    }
  }
}

}  // namespace accept
