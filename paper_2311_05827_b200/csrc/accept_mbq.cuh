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
#include "accept_exact.cuh"
#include "accept_kernels.cuh"

namespace accept {

constexpr int kMbqRounds = 2;                      // octets per thread and tile
constexpr int kMbqTile = kMbqRounds * 256 * 8;     // elements per tile
constexpr int kMbqFinalizeThreads = 32;            // threads of the single finalize block
constexpr int kMbqGroups = 2;                      // 256-thread groups per block of the encode pass (one block per SM);
                                                   // 3 groups at 80 registers were slower than 2 at 113 (measured)
constexpr int kMbqEncodeThreads = 256 * kMbqGroups;
constexpr int kMbqMaxBlocks = 148 * kMbqGroups;    // groups of the encode pass
constexpr int kMbqResidueBlocks = 1184;            // blocks of a residue pass
constexpr int kMbqCells = 256;                     // cells of the uniform search grid
constexpr int kMbqGridBytes = kMbqCells * 32 * 16; // one 16-byte entry per cell and lane
constexpr int kMbqSums = 5;                        // wide sums in the workspace: basis 0..3, then the sum of x
constexpr int kMbqFlushTiles = kFlushElems / (kMbqRounds * 8);  // tiles a thread codes between two flushes

// Workspace of the forward quantizer (zeroed once by the caller; every call leaves the sums zeroed again).
struct MbqWorkspace {
  uint32_t status;
  uint32_t pad0[3];
  float alpha_init[4];            // coefficients found by the residue passes (init)
  uint32_t blocks_done;           // blocks of a residue pass that have delivered their sum
  uint32_t pad1[7];
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
// cells; cell_offset() is a non-decreasing function of x, so every x of a cell below the cell of a
// threshold lies below that threshold and every x of a cell above it lies above.  When no cell
// holds more than one threshold, one comparison with "the threshold inside my cell" finishes the
// search: entry = {that threshold (+inf if the cell has none), flag bytes of the code below it,
// flag bytes of the code above it, 0}.  The decisions are the ones of the threshold search, exactly;
// when two thresholds share a cell (coinciding or very close levels), or a level is not finite,
// the grid is marked unusable and the kernel searches the sorted thresholds instead.
//
// The table is stored once per lane, entry (cell, lane) at byte 512 * cell + 16 * lane: whatever
// cells the 32 lanes of a warp ask for, lane l only ever touches its own 16-byte column of the
// banks, so a lookup is one 128-bit shared load without bank conflicts (a single shared copy
// cost 8.6 wavefronts per load on post-ReLU data and bound the pass).  128 KB per block.
struct MbqGridInfo {
  float scale;  // 1 / (2 * span)
  int usable;
};

// Byte offset of entry (cell of x, lane); lane_bytes = 16 * lane.  Two fused multiply-adds on the
// FMA pipe and one logic operation: the first maps the span onto [0, 1] and saturates, the second
// leaves round(255 * 512 * t) in the low mantissa bits; keeping bits 9..16 of it gives
// 512 * floor(that / 512).  NaN goes to cell 0.
__device__ __forceinline__ uint32_t mbq_cell_offset(float x, float scale, uint32_t lane_bytes) {
  float t;
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(t) : "f"(x), "f"(scale));
  return (__float_as_uint(__fmaf_rn(t, 130560.0f, kMagic)) & 0x1FE00u) | lane_bytes;
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
  if (tid >= 1 && tid < L) s_cell_of[tid] = mbq_cell_offset(t.thr[tid], info->scale, 0u) >> 9;
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
    for (int i = tid; i < kMbqCells * 32; i += n_threads) cells[i] = s_entry[i >> 5];
  __syncthreads();
}

// flag bytes of the nearest level's code
__device__ __forceinline__ uint32_t mbq_grid_flags(const uint4* cells, float scale, uint32_t lane_bytes, float x) {
  const uint4 e = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(cells) +
                                                  mbq_cell_offset(x, scale, lane_bytes));
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
  for (int i = 0; i < kAccLimbs; ++i) { limbs[i] = bs->wide[tid][i]; any = any || limbs[i] != 0; }
  if (!any) return;
  wide_normalise(limbs);
  for (int i = 0; i < kAccLimbs; ++i)
    if (limbs[i] != 0) limb_add(&ws->wide[tid][i], limbs[i]);
}

// ---- residue method ---------------------------------------------------------------------------------

// Residue method, step j: alpha_j = mean |r_j| (r_0 = x) with the coefficients found so far.  Every block
// adds the |r_j| of its tiles exactly and hands the sum to the workspace; the block that arrives last
// rounds the total once, divides by n and leaves the workspace clean for the next pass.  No block waits
// for another.
template <int K>
__global__ void __launch_bounds__(256) mbq_residue_sum_kernel(const MbqArgs a, int j) {
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
  for (uint64_t tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
#pragma unroll
    for (int r = 0; r < kMbqRounds; ++r) {
      const uint64_t oct = tile * (kMbqRounds * 256) + r * 256 + tid;
      if (oct < n_oct) {
        float v[8], res[8];
        mbq_ld_octet(a.x, a.n, oct, v);
        WindowCheck chk;
        chk.init();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          mbq_residue_code<K>(alpha, v[e], j, &res[e]);
          res[e] = (oct * 8 + e < a.n) ? fabsf(res[e]) : 0.0f;
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
      }
    }
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
    for (int i = 0; i < kAccLimbs; ++i) {
      total[i] = (long long)atomicExch(reinterpret_cast<unsigned long long*>(&a.ws->wide[SLOT][i]), 0ull);
    }
    a.ws->alpha_init[j] = (float)(wide_to_double(total) / (double)a.n);
    a.ws->blocks_done = 0u;
  }
}

// How the signs of an element are found.
constexpr int kMbqResidue = 0, kMbqSearch = 1, kMbqGrid = 2;

// Running sums of one thread over all its tiles.  plus[] and sum_x hold what the thread added since its
// last flush (plus[] times 2^-767, the flag factor); irun[] the flushed part in units of the window.
template <int K>
struct MbqSums {
  double plus[K], sum_x;
  long long irun[K + 1];      // [K]: the sum of x
  uint32_t count, differ[3];  // of basis q = lane & 3, and of the pairs (q, q ^ d)
  int since, flushes;
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

// The octets of thread tid of a tile: FULL = every element of the tile exists.
template <bool FULL>
__device__ __forceinline__ void mbq_load_tile(const MbqArgs& a, uint64_t tile, int tid, float (&v)[kMbqRounds][8]) {
  const uint64_t oct0 = tile * (kMbqRounds * 256) + tid;
#pragma unroll
  for (int r = 0; r < kMbqRounds; ++r) {
    const uint64_t oct = oct0 + r * 256;
    if (FULL) {
      ld_octet(a.x + oct * 8, v[r]);
    } else if (oct < (a.n + 7) / 8) {
      mbq_ld_octet(a.x, a.n, oct, v[r]);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[r][e] = 0.0f;
    }
  }
}

// A value of the encode pass that may lie outside the window.  If it does, it goes into the block's wide
// sums (the sum of x, and the sum of every basis whose sign is +1) and 0 is returned for the thread's own
// accumulators; otherwise the value itself is returned.
__device__ __noinline__ float mbq_divert_value(MbqBlockSums* bs, uint32_t* status, float x, uint32_t flags) {
  if (in_window(bs->window, x)) return x;
  // flag bytes (0x10 per basis) -> slot bits, plus the slot of the sum of x
  const uint32_t slots = ((((flags >> 4) * 0x00204081u) >> 21) & 0xFu) | (1u << (kMbqSums - 1));
  mbq_wide_add_value(bs, status, x, slots);
  return 0.0f;
}

// One tile of kMbqTile elements, coded by one group of 256 threads (tid = index in the group): assign
// the signs, write the planes, add to the thread's sums.
template <int K, int MODE, bool FULL>
__device__ __forceinline__ void mbq_encode_tile(const MbqArgs& a, uint64_t tile, int tid, int lane,
                                                const float (&v)[kMbqRounds][8], const float (&alpha)[K],
                                                const MbqTable<K>& table, const uint4* cells, float scale,
                                                MbqBlockSums* bs, float win_top, uint32_t win_ylow, MbqSums<K>& sums) {
  const uint64_t n_oct_stored = ((a.n + 31) / 32) * 4;
  const uint64_t oct0 = tile * (kMbqRounds * 256) + tid;
  const int q = lane & 3;
  const uint32_t lane_bytes = 16u * (uint32_t)lane;
#pragma unroll
  for (int r = 0; r < kMbqRounds; ++r) {
    const uint64_t oct = oct0 + r * 256;
    uint32_t f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (MODE == kMbqResidue) {
        float res;
        f[e] = mbq_flags_of_code(mbq_residue_code<K>(alpha, v[r][e], K, &res));
      } else if (MODE == kMbqSearch) {
        f[e] = mbq_flags_of_code(mbq_nearest_code<K>(table, v[r][e]));
      } else {
        f[e] = mbq_grid_flags(cells, scale, lane_bytes, v[r][e]);
      }
    }
    if (!FULL) {
      // elements of this octet that exist; signs past the end are zero bits (their values were loaded as 0)
      const int valid = (oct * 8 + 8 <= a.n) ? 8 : ((oct * 8 < a.n) ? (int)(a.n - oct * 8) : 0);
      if (valid < 8) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (e >= valid) f[e] = 0;
      }
    }
    // the values as the running sums take them: all of them, unless some lie outside the window
    float w[8];
    WindowCheck chk;
    chk.init();
#pragma unroll
    for (int e = 0; e < 8; ++e) w[e] = v[r][e];  // 0 past the end
#pragma unroll
    for (int e = 0; e < 8; e += 2) chk.add2(w[e], w[e + 1]);
    if (!(chk.amax < win_top && chk.ymin >= win_ylow)) {
#pragma unroll
      for (int e = 0; e < 8; ++e) w[e] = mbq_divert_value(bs, a.status, w[e], f[e]);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const double xd = (double)w[e];
      sums.sum_x += xd;
      mbq_add_flagged<0>(sums.plus[0], xd, f[e]);
      mbq_add_flagged<1>(sums.plus[1], xd, f[e]);
      if constexpr (K > 2) mbq_add_flagged<2>(sums.plus[2], xd, f[e]);
      if constexpr (K > 3) mbq_add_flagged<3>(sums.plus[3], xd, f[e]);
    }
    // after the quad transpose lane q holds the 32 signs of basis q of its group: counts of +1 and,
    // against the words of the other three lanes of the quad, counts of differing signs
    const uint32_t word = quad_transpose(mbq_planes_of_flags(f), lane);
    if ((FULL || oct < n_oct_stored) && q < K) st_c(a.payload + (oct >> 2) * K + q, word);
    sums.count += __popc(word);
#pragma unroll
    for (int d = 1; d < 4; ++d) {
      const uint32_t other = __shfl_xor_sync(0xffffffffu, word, d);
      sums.differ[d - 1] += __popc(word ^ other);
    }
  }
  // every thread of the group has coded the same number of tiles: flushes and pushes are taken together
  if (++sums.since == kMbqFlushTiles) {
    sums.since = 0;
    mbq_flush<K>(sums, bs);
    if (++sums.flushes == kPushFlushes) {
      sums.flushes = 0;
      mbq_push<K>(sums, bs, lane);
    }
  }
}

// A group walks over tiles with a stride of the number of groups and keeps its sums in registers: the
// group-level reduction is paid once per group, not once per tile.
// The loads of a group's next tile are in flight while it codes the current one (two register
// buffers, the loop unrolled by two so that both are addressed statically).
template <int K, int MODE>
__device__ __forceinline__ void mbq_encode_tiles(const MbqArgs& a, uint32_t group, int tid, int lane,
                                                 const float (&alpha)[K], const MbqTable<K>& table, const uint4* cells,
                                                 float scale, MbqBlockSums* bs, MbqSums<K>& sums) {
  if (group >= a.n_blocks) return;
  const float win_top = bs->window.top;
  const uint32_t win_ylow = bs->window.ylow;
  const uint64_t full_tiles = a.n / kMbqTile, stride = a.n_blocks;
  float v0[kMbqRounds][8], v1[kMbqRounds][8];
  uint64_t tile = group;
  if (tile < full_tiles) mbq_load_tile<true>(a, tile, tid, v0);
  while (tile < full_tiles) {
    const uint64_t t1 = tile + stride;
    if (t1 < full_tiles) mbq_load_tile<true>(a, t1, tid, v1);
    mbq_encode_tile<K, MODE, true>(a, tile, tid, lane, v0, alpha, table, cells, scale, bs, win_top, win_ylow, sums);
    tile = t1;
    if (t1 >= full_tiles) break;
    const uint64_t t2 = t1 + stride;
    if (t2 < full_tiles) mbq_load_tile<true>(a, t2, tid, v0);
    mbq_encode_tile<K, MODE, true>(a, t1, tid, lane, v1, alpha, table, cells, scale, bs, win_top, win_ylow, sums);
    tile = t2;
  }
  // the ragged last tile of the tensor, if there is one, is the last tile of its group
  if (tile < a.n_tiles) {
    mbq_load_tile<false>(a, tile, tid, v0);
    mbq_encode_tile<K, MODE, false>(a, tile, tid, lane, v0, alpha, table, cells, scale, bs, win_top, win_ylow, sums);
  }
}

// Assign the signs, write the planes, gather the sums.  One block of kMbqGroups groups of 256 threads
// per SM; a group does what a 256-thread block would (its own tiles), the groups of a block share the
// search tables and the block's wide sums.  Dynamic shared memory: the search grid (kMbqGridBytes), not
// needed when INIT.
template <int K, bool INIT>
__global__ void __launch_bounds__(kMbqEncodeThreads, 1) mbq_encode_kernel(const MbqArgs a) {
  grid_dependency_handshake();
  extern __shared__ uint4 s_cells[];
  __shared__ MbqTable<K> s_table;
  __shared__ MbqGridInfo s_grid;
  __shared__ MbqBlockSums s_sums;
  __shared__ float s_level[16];
  __shared__ uint32_t s_cnt[10];
  const int lane = threadIdx.x & 31;
  const int g = threadIdx.x >> 8;            // group in the block
  const int tid = threadIdx.x & 255;         // thread in the group
  const uint32_t group = blockIdx.x * kMbqGroups + g;
  float alpha[K];
  mbq_block_sums_clear(&s_sums, threadIdx.x, kMbqEncodeThreads);
  if (threadIdx.x < 10) s_cnt[threadIdx.x] = 0;
  if (INIT) {
#pragma unroll
    for (int j = 0; j < K; ++j) alpha[j] = a.ws->alpha_init[j];
    // window of the exact sums: around the mean magnitude of the data
    if (threadIdx.x == 0) s_sums.window = make_window(alpha[0]);
  } else {
#pragma unroll
    for (int j = 0; j < K; ++j) alpha[j] = 0.0f;
    mbq_build_table<K>(a.alpha_prev, &s_table, s_level, threadIdx.x);
    mbq_build_grid<K>(s_table, s_level, &s_grid, s_cells, threadIdx.x, kMbqEncodeThreads);
    // window of the exact sums: around the largest level (values the levels were fitted to)
    if (threadIdx.x == 0) {
      float amax = 0.0f;
      for (int c = 0; c < (1 << K); ++c) amax = fmaxf(amax, fabsf(s_level[c]));
      s_sums.window = make_window(amax * 0.125f);
    }
  }
  __syncthreads();

  MbqSums<K> sums;
  sums.sum_x = 0.0;
  sums.count = 0;
  sums.since = 0;
  sums.flushes = 0;
#pragma unroll
  for (int j = 0; j < K; ++j) sums.plus[j] = 0.0;
#pragma unroll
  for (int j = 0; j <= K; ++j) sums.irun[j] = 0;
#pragma unroll
  for (int d = 0; d < 3; ++d) sums.differ[d] = 0;

  if (INIT) mbq_encode_tiles<K, kMbqResidue>(a, group, tid, lane, alpha, s_table, s_cells, 0.0f, &s_sums, sums);
  else if (s_grid.usable) mbq_encode_tiles<K, kMbqGrid>(a, group, tid, lane, alpha, s_table, s_cells, s_grid.scale, &s_sums, sums);
  else mbq_encode_tiles<K, kMbqSearch>(a, group, tid, lane, alpha, s_table, s_cells, 0.0f, &s_sums, sums);

  // what is left in the accumulators, then the warp's total into the block's wide sums
  mbq_flush<K>(sums, &s_sums);
  mbq_push<K>(sums, &s_sums, lane);

  const int q = lane & 3;
  uint32_t my_count = sums.count;
  uint32_t (&my_differ)[3] = sums.differ;
  // lanes with the same q hold partial counts of the same basis / pairs: add over the eight quads
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) {
    my_count += __shfl_xor_sync(0xffffffffu, my_count, d);
#pragma unroll
    for (int i = 0; i < 3; ++i) my_differ[i] += __shfl_xor_sync(0xffffffffu, my_differ[i], d);
  }
  if (lane < 4) {
    atomicAdd(&s_cnt[q], my_count);
#pragma unroll
    for (int d = 1; d < 4; ++d) {
      const int other = q ^ d;
      if (q < other) {  // each pair once; pair index in the order (0,1) (0,2) (0,3) (1,2) (1,3) (2,3)
        const int pair = (q == 0) ? other - 1 : (q == 1 ? other + 1 : 5);
        atomicAdd(&s_cnt[4 + pair], my_differ[d - 1]);
      }
    }
  }
  __syncthreads();
  mbq_block_sums_deliver(&s_sums, a.ws, threadIdx.x);
  if (threadIdx.x >= 32 && threadIdx.x < 42) {
    const int i = threadIdx.x - 32;
    const unsigned long long c = s_cnt[i];
    if (c) atomicAdd(i < 4 ? &a.ws->count[i] : &a.ws->differ[i - 4], c);
  }
}

// Rounds the exact sums once, then Eq. 3 (least squares by Gaussian elimination with partial pivoting, in
// double), Eq. 4 (moving average), Eq. 5 (bias), and writes header, side words and alpha_next; leaves the
// sums of the workspace zeroed for the next call.  One warp.
template <int K>
__global__ void __launch_bounds__(kMbqFinalizeThreads) mbq_finalize_kernel(const MbqArgs a) {
  grid_dependency_handshake();
  __shared__ double s_val[K + 1];  // [j] = (B^T x)_j, [K] = sum of x
  const int tid = threadIdx.x;
  MbqWorkspace* ws = a.ws;
  if (tid <= K) {
    long long lazy[kAccLimbs];
    for (int i = 0; i < kAccLimbs; ++i) {
      const long long sx = ws->wide[kMbqSums - 1][i];
      // sum over the +1 elements minus sum over the -1 elements = 2 * (sum over +1) - (sum of all), digit by digit
      lazy[i] = (tid < K) ? 2 * ws->wide[tid][i] - sx : sx;
    }
    s_val[tid] = wide_to_double(lazy);
  }
  unsigned long long c[10];
#pragma unroll
  for (int j = 0; j < 4; ++j) c[j] = ws->count[j];
#pragma unroll
  for (int j = 0; j < 6; ++j) c[4 + j] = ws->differ[j];
  __syncthreads();
  // the next call starts from zero
  for (int i = tid; i < kMbqSums * kAccLimbs; i += kMbqFinalizeThreads) (&ws->wide[0][0])[i] = 0;
  if (tid < 4) ws->count[tid] = 0;
  if (tid < 6) ws->differ[tid] = 0;
  if (tid != 0) return;

  const double N = (double)a.n, sum_x = s_val[K];
  float alpha_next[K];
  if (a.init) {
#pragma unroll
    for (int j = 0; j < K; ++j) alpha_next[j] = ws->alpha_init[j];
  } else {
    double G[K][K], rhs[K], cur[K], prev[K];
    int pair = 0;
    for (int i = 0; i < 4; ++i)
      for (int j = i + 1; j < 4; ++j, ++pair)
        if (j < K) G[i][j] = G[j][i] = N - 2.0 * (double)c[4 + pair];
    for (int j = 0; j < K; ++j) {
      G[j][j] = N;
      rhs[j] = s_val[j];
      prev[j] = (double)ldg_c(a.alpha_prev + j);
    }
    bool singular = false;
    for (int col = 0; col < K && !singular; ++col) {
      int piv = col;
      for (int r = col + 1; r < K; ++r)
        if (fabs(G[r][col]) > fabs(G[piv][col])) piv = r;
      if (fabs(G[piv][col]) < 1e-9 * N) { singular = true; break; }
      if (piv != col) {
        for (int q = 0; q < K; ++q) { const double t = G[col][q]; G[col][q] = G[piv][q]; G[piv][q] = t; }
        const double t = rhs[col]; rhs[col] = rhs[piv]; rhs[piv] = t;
      }
      for (int r = col + 1; r < K; ++r) {
        const double f = G[r][col] / G[col][col];
        for (int q = col; q < K; ++q) G[r][q] -= f * G[col][q];
        rhs[r] -= f * rhs[col];
      }
    }
    if (singular) {
      for (int j = 0; j < K; ++j) cur[j] = prev[j];
    } else {
      for (int col = K - 1; col >= 0; --col) {
        double s = rhs[col];
        for (int q = col + 1; q < K; ++q) s -= G[col][q] * cur[q];
        cur[col] = s / G[col][col];
      }
    }
    double beta = (1.0 + (double)a.batch_index) / (10.0 + (double)a.batch_index);
    if (beta > 0.9) beta = 0.9;
    for (int j = 0; j < K; ++j) alpha_next[j] = (float)(beta * prev[j] + (1.0 - beta) * cur[j]);
  }
  double acc = 0.0;
  for (int j = 0; j < K; ++j) acc += (double)alpha_next[j] * (2.0 * (double)c[j] - N);
  const float m_q = (float)((acc - sum_x) / N);
  for (int i = 0; i < 8; ++i) st_c(a.header + i, mbq_header_word(a, i));
  for (int j = 0; j < K; ++j) { st_c(a.side + j, alpha_next[j]); st_c(a.alpha_next + j, alpha_next[j]); }
  st_c(a.side + K, m_q);
  // pad up to the payload
  for (uint32_t* w = reinterpret_cast<uint32_t*>(a.side + K + 1); w < a.payload; ++w) st_c(w, 0u);
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
