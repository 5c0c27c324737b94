/*
 * accept.h -- C ABI of the boundary-tensor codec (AccEPT bit-level compression, Sec. 3.3-3.4).
 *
 * The codec turns a flat fp32 tensor x_v (Sec. 3.3, "Forward Quantizer": the boundary tensor is
 * vectorised to N = n*w*h*c values) into k-bit integer codes packed densely into 32-bit words plus
 * fp32 side words, and back.  All compute runs in CUDA kernels built for sm_100a; there is no host
 * fallback.  Every entry point is asynchronous on the stream it is given and allocates nothing.
 *
 * ---------------------------------------------------------------------------------------------
 * Operation (per chunk of chunk_elems consecutive values; the paper's scheme is the case
 * chunk_elems >= n_elems, one range for the whole tensor):
 *
 *   range   ABSMAX (Sec. 3.3 "Backward Quantizer"):  c = max|x|,  L = 2^(k-1)-1,  s = c/L,  o = 0
 *           MINMAX (affine extension):               lo = min x, hi = max x, L = 2^k-1,
 *                                                    s = (hi-lo)/L,  o = lo
 *   scale   inv = L/c  (resp. L/(hi-lo)) rounded toward zero, one IEEE fp32 division per chunk, so that
 *           |x*inv| <= L as in exact arithmetic and no code is clamped.  If the range is 0, or the
 *           quotient overflows, the chunk is degenerate: s = 0, inv = 0, every code is the zero point.
 *   codes   t = x*inv           (MINMAX: t = (x-lo)*inv), each fp32 operation rounded separately
 *           NEAREST:    q = rint(t)                      (ties to even)
 *           STOCHASTIC: q = floor(t) + [U < t-floor(t)]  (Eq. 7), U from the counter-based
 *                       generator described at accept_params.seed; the fraction t-floor(t) and
 *                       the comparison are exact (no rounding of the difference)
 *           ABSMAX: q lies in [-L, L] (inside the paper's [-2^(k-1), 2^(k-1)-1]), stored code
 *           u = q + 2^(k-1)  ("+8" of the "Backward Encoder" for k = 4);  MINMAX: u = q in [0, 2^k-1]
 *   pack    INTERLEAVED ("Backward Encoder"): code of element t of the chunk occupies bits
 *           [k*t, k*t+k) of the chunk's little-endian bit string (k = 8: plain bytes).
 *           BITPLANE ("Forward Encoder"): per group of 32 consecutive elements, k consecutive
 *           32-bit words; bit t of word j is bit j of the code of element t of the group.
 *   decode  ("Backward Decoder/Dequantizer", "Forward Decoder"): unpack u;
 *           ABSMAX: xhat = float(u - 2^(k-1)) * s;   MINMAX: xhat = fl(fl(float(u)*s) + o)
 *
 * Stream layout (little-endian, byte offsets):
 *   [0,32)    header, eight u32: magic 0x54504341 ("ACPT"), version 1, n_elems low, n_elems high,
 *             chunk_elems, k, range | round<<8 | layout<<16, group_stride
 *   [32, 32+8M)   M = ceil(n_elems/chunk_elems) records {float s; float o}, one per chunk
 *   [P, ...)  payload, P = 32+8M rounded up to a multiple of 16.  Chunk m starts at word
 *             m*chunk_elems*k/32 of the payload.  A partial last chunk holds ceil(valid/32)*k
 *             words; codes of padding elements are 0 bits.
 *   total     P + 4*k*ceil(n_elems/32) bytes  (= accept_compressed_size).
 *
 * Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  d_x, d_xhat and d_stream must be
 * 16-byte aligned.  The caller owns every buffer and the stream.
 */
#ifndef ACCEPT_H_
#define ACCEPT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ACCEPT_MAGIC 0x54504341u
#define ACCEPT_VERSION 1u
#define ACCEPT_HEADER_BYTES 32u

/* Return codes of the host entry points (nothing was launched unless ACCEPT_OK). */
typedef enum {
  ACCEPT_OK = 0,
  ACCEPT_ERR_NULL = 1,          /* a required pointer is NULL */
  ACCEPT_ERR_BAD_K = 2,         /* k not in {2,3,4,8}, or k = 3 with INTERLEAVED */
  ACCEPT_ERR_BAD_CHUNK = 3,     /* chunk_elems < 32 or not a multiple of 32 */
  ACCEPT_ERR_BAD_ENUM = 4,      /* range / round / layout out of range */
  ACCEPT_ERR_TOO_SMALL = 5,     /* a buffer is smaller than the size queries say */
  ACCEPT_ERR_BAD_STREAM_HEADER = 6, /* header words do not match the parameters */
  ACCEPT_ERR_CUDA = 7,          /* a CUDA runtime call failed */
  ACCEPT_ERR_NONFINITE = 8,     /* reported through the device status word only */
  ACCEPT_ERR_BAD_SIZE = 9,      /* n_elems = 0 */
  ACCEPT_ERR_MISALIGNED = 10,   /* a device pointer is not 16-byte aligned */
  ACCEPT_ERR_SCRATCH_LIMIT = 11, /* accept_compress_static: the call needs more scratch than the built-in array holds */
  ACCEPT_ERR_UNCHECKED_BUILD = 12 /* accept_bounds_check_report: this library was built without access checks */
} accept_status;

/* Bits of the device status word (word 0 of the workspace); sticky until the caller clears it. */
#define ACCEPT_DEV_NONFINITE 1u   /* some chunk held NaN/Inf (or an overflowing MINMAX range) */
#define ACCEPT_DEV_BAD_HEADER 2u  /* accept_decompress: stream header differs from the parameters */
#define ACCEPT_DEV_COPY_TIMEOUT 4u /* an asynchronous copy inside a kernel did not complete within 0.2 s; output invalid */

typedef enum { ACCEPT_RANGE_ABSMAX = 0, ACCEPT_RANGE_MINMAX = 1 } accept_range;
typedef enum { ACCEPT_ROUND_NEAREST = 0, ACCEPT_ROUND_STOCHASTIC = 1 } accept_round;
typedef enum { ACCEPT_LAYOUT_INTERLEAVED = 0, ACCEPT_LAYOUT_BITPLANE = 1 } accept_layout;

/*
 * Parameters of one call.
 *   n_elems      N >= 1, number of fp32 values.
 *   chunk_elems  C, multiple of 32, >= 32: elements sharing one range.
 *   k            bit width: 2, 3 (BITPLANE only), 4 or 8.
 *   group_stride 0, or F = values per sample (w*h*c): the tensor is (n_elems/F) x F and a pack group is
 *                made of the 32 BATCH neighbours (rows 32g..32g+31) of one feature f: pack groups run
 *                along the batch dimension as in Sec. 3.3, "Forward Encoder" / "Backward Encoder".
 *                Group index G = g*F + f, words G*k .. G*k+k-1 of the payload, element
 *                (row b, feature f) at position t = b % 32 of its group; rows past the last are zero
 *                bits; payload = 4*k*ceil(rows/32)*F bytes.  Ranges stay per chunk of consecutive
 *                values.  Needs n_elems % F == 0 and a 32-byte aligned input; any F >= 1 (the
 *                paper's smallest outputs need not have 8 | w*h*c).  With F % 8 == 0 a thread
 *                codes eight features of eight rows with 32-byte loads;
 *                every other shape takes one feature per thread, slower but for any F.  Runs as
 *                two launches: ranges, side words and constants of every chunk, then the encoder
 *                (workspace: 16 bytes per chunk more, as for chunk_elems > 32768; with such chunks
 *                it is a memset and four launches).  Header word 7 carries F.
 *   seed, rng_offset  STOCHASTIC only.  Element i draws
 *                  U_i = (g >> 8) * 2^-24,
 *                  g   = h * M[ctr & 3] (mod 2^32),  M = {1, 0x9E3779B1, 0x85EBCA77, 0xC2B2AE3D},
 *                  h   = fmix32( lo32(j) ^ fmix32( hi32(j) ^ lo32(seed) ^ 0x9E3779B9 ) ^ hi32(seed) ),
 *                  j   = ctr >> 2,  ctr = rng_offset + i (mod 2^64)
 *                (four neighbouring counters share one hash; each takes it times its own odd constant),
 *                fmix32 = the 32-bit finaliser of MurmurHash3:
 *                  h ^= h>>16; h *= 0x85EBCA6B; h ^= h>>13; h *= 0xC2B2AE35; h ^= h>>16.
 *                The same (seed, rng_offset) reproduces the same stream; advance rng_offset by
 *                n_elems between calls to draw fresh numbers.
 */
typedef struct {
  uint64_t n_elems;
  uint32_t chunk_elems;
  uint32_t k;
  int32_t range;   /* accept_range  */
  int32_t round;   /* accept_round  */
  int32_t layout;  /* accept_layout */
  uint32_t group_stride; /* 0: pack groups of 32 consecutive values; F > 0: see below */
  uint64_t seed;
  uint64_t rng_offset;
} accept_params;

/* Validates p as the compress/decompress entry points do (host only). */
accept_status accept_check_params(const accept_params* p);

/*
 * Size in bytes of the compressed stream for p (layout above); 0 if p is invalid.
 * Sec. 3.3 "Transmission Data Comparison", Eq. 8: payload of k bits per element plus fp32 side words.
 */
size_t accept_compressed_size(const accept_params* p);

/* Byte offset of the payload inside the stream (P above); 0 if p is invalid. */
size_t accept_payload_offset(const accept_params* p);

/*
 * Bytes of device workspace the kernels need: 16, plus 16 per chunk when chunk_elems > 32768 or group_stride != 0
 * (such chunks do not fit on chip: their ranges are gathered in the workspace first, and the input
 * is read twice).  Word 0 is the device status word; the caller zeroes the workspace once (and
 * whenever it wants to clear the status); the workspace must be 16-byte aligned.  0 if p is invalid.
 * This is what accept_compress needs.  accept_decompress touches the status word only: 16 bytes
 * (4-byte aligned) are enough for it, whatever the parameters.
 */
size_t accept_workspace_size(const accept_params* p);

/*
 * Quantizer + encoder (Sec. 3.3): reads n_elems floats at d_x, writes accept_compressed_size(p)
 * bytes at d_stream (header, per-chunk {s,o}, payload), in one kernel launch (three launches and a
 * memset of the workspace records when chunk_elems > 32768, e.g. one range for the whole tensor as
 * in the paper) on cuda_stream
 * (a cudaStream_t, may be NULL for the default stream).  Non-finite input does not fail the call:
 * the chunk is written as degenerate and ACCEPT_DEV_NONFINITE is or-ed into the status word.
 * d_x is only read; d_stream is fully overwritten up to the compressed size.
 */
accept_status accept_compress(const accept_params* p, const float* d_x, void* d_stream,
                              size_t stream_bytes, void* d_ws, size_t ws_bytes, void* cuda_stream);

/*
 * Decoder + dequantizer (Sec. 3.4): reads the stream at d_stream, writes n_elems floats at d_xhat,
 * in one kernel launch.  p carries what the receiver agreed on with the sender (n_elems,
 * chunk_elems, k, range, layout; round/seed are ignored); the kernel compares it with the header
 * words and or-s ACCEPT_DEV_BAD_HEADER into the status word on a mismatch (the output is then
 * unspecified but every access stays inside the buffers as sized by p).  The workspace needs 16 bytes
 * only (the status word), also for wide chunks and batch groups.
 */
accept_status accept_decompress(const accept_params* p, const void* d_stream, size_t stream_bytes,
                                float* d_xhat, void* d_ws, size_t ws_bytes, void* cuda_stream);

/*
 * accept_compress for callers that cannot allocate device memory at all.  (The paper has no counterpart:
 * this is a packaging variant of the quantizer + encoder above, same kernel, same stream.)
 *
 * Who needs it: a pipeline stage on a device whose memory budget is sealed after start-up, or a plug-in
 * living inside a host framework that owns every byte of device memory, has no way to obtain the
 * workspace accept_compress asks for -- cudaMalloc (or the framework's allocator) is off limits to it.
 * Here the workspace is a fixed array of ACCEPT_STATIC_SCRATCH_BYTES (256) bytes that is part of the
 * library image: every GPU that loads the library holds it until the process exits, and the entry point
 * calls no cudaMalloc, cudaFree or any other allocating routine.  The caller still passes the input and
 * the output stream, sized as for accept_compress.
 *
 *   d_status_out  optional DEVICE pointer (4-byte aligned) that receives the ACCEPT_DEV_* status bits of
 *                 THIS call (copied on cuda_stream after the kernel); NULL if not wanted.
 *
 * Limits and rules:
 *   - a call whose workspace need (accept_workspace_size) exceeds ACCEPT_STATIC_SCRATCH_BYTES is rejected
 *     with ACCEPT_ERR_SCRATCH_LIMIT and nothing is launched;
 *   - the first call on each device looks up the array's device address (with that device current); make
 *     that first call before any stream capture begins on that device;
 *   - all calls on a device share the one array.  The status word in it is cleared at the start of every
 *     call (so it does not accumulate across calls as a caller-owned workspace does), and two calls that
 *     overlap on the GPU (different streams) race on it: issue them on one stream, or order them.  Calls
 *     from several host threads must be serialised by the caller even on one stream: a call enqueues a
 *     clear, its kernels and the status copy one after the other, and two threads could interleave them;
 *   - d_x must live on the current device (checked: ACCEPT_ERR_CUDA otherwise), and cuda_stream must
 *     belong to it.
 */
#define ACCEPT_STATIC_SCRATCH_BYTES 256u
accept_status accept_compress_static(const accept_params* p, const float* d_x, void* d_stream,
                                     size_t stream_bytes, uint32_t* d_status_out, void* cuda_stream);

/*
 * Host-buffer variants, for callers whose tensors live in host memory: copy h_x to the staging
 * buffer d_x (host to device), run accept_compress, copy the stream back to h_stream (and the
 * mirror image for decompress), all asynchronously on cuda_stream.  Staging buffers are the
 * caller's; sizes as for the device entry points.  Pinned host memory makes the copies overlap
 * nothing else but avoids a bounce buffer in the driver.
 */
accept_status accept_compress_host(const accept_params* p, const float* h_x, void* h_stream,
                                   size_t stream_bytes, float* d_x, void* d_stream, void* d_ws,
                                   size_t ws_bytes, void* cuda_stream);
accept_status accept_decompress_host(const accept_params* p, const void* h_stream,
                                     size_t stream_bytes, float* h_xhat, void* d_stream,
                                     float* d_xhat, void* d_ws, size_t ws_bytes, void* cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * Forward quantizer of the paper: multi-bit quantization (Sec. 3.3 "Forward Quantizer", Eq. 1-5;
 * "Forward Encoder"; Sec. 3.4 "Forward Decoder", "Forward Dequantizer").
 *
 * x ~ B alpha, B in {-1,+1}^(N x k), alpha in R^k (one alpha per tensor, as in the paper).  Element
 * i carries the code c_i = sum_j [b_ij = +1] << j; level(c) = (+-alpha_0) + ... + (+-alpha_k-1)
 * summed in fp32 in the order j = 0..k-1.
 *   batch_index t >= 1 (init = 0): every value takes the nearest level of alpha_prev (exact
 *     comparison; a tie goes to the lower level; coinciding levels: the smallest code), then
 *     alpha_cur = (B^T B)^-1 B^T x (Eq. 3; kept at alpha_prev if B^T B is singular) and
 *     alpha_next = beta alpha_prev + (1-beta) alpha_cur, beta = min(0.9, (1+t)/(10+t)) (Eq. 4).
 *   init != 0 (batch 0 of an epoch): residue method: r = x; for j = 0..k-1: b_j = [r >= 0],
 *     alpha_j = mean |r|, r <- r - alpha_j b_j; alpha_prev is not read; no Eq. 3/4 update.
 *   The stream carries alpha_next and m_q = mean(B alpha_next - x) (Eq. 5); the receiver
 *     computes xhat = level(c) - m_q.  The sums over the tensor behind Eq. 3 and Eq. 5 (B^T x, the sum
 *     of x, and the mean |r| of the residue method) are taken WITHOUT rounding and rounded once to double:
 *     alpha_next and m_q are a function of the input alone, whatever the order in which threads add (the
 *     k x k system is then solved in double by Gaussian elimination with partial pivoting; a pivot below
 *     1e-9 N counts as singular).  Non-finite input is not supported: ACCEPT_DEV_NONFINITE is set, such
 *     values are left out of the sums and the codes are unspecified.
 * Stream: [0,32) header (magic, version, n low, n high, 0, k, 0, 1), [32, 32+4k) alpha_next,
 *   then m_q, zero pad to a multiple of 16, then bit planes: group g of 32 elements owns words
 *   g*k .. g*k+k-1, bit t of word g*k+j = [b_(32g+t),j = +1] ("-1 replaced by 0").
 * k in {2,3,4} (the paper's forward range); d_alpha_prev / d_alpha_next are DEVICE arrays of k
 * floats (they may be the same array), so successive batches chain without a host round trip.
 * The workspace (accept_mbq_workspace_size bytes = 624, 16-byte aligned, zeroed once by the caller) holds
 * the status word, the residue coefficients and the exact sums (every call leaves them zeroed again; a
 * workspace serves one call at a time).  Launches: 1 (plus k when init).  The encode
 * kernel of a batch >= 1 asks for 128 KB of dynamic shared memory per block (its search table).
 */
typedef struct {
  uint64_t n_elems;
  uint32_t k;
  uint32_t batch_index; /* t of Eq. 4 */
  uint32_t init;        /* 1: residue-based initialisation */
  uint32_t reserved;    /* must be 0 */
} accept_mbq_params;

accept_status accept_mbq_check_params(const accept_mbq_params* p);
size_t accept_mbq_compressed_size(const accept_mbq_params* p); /* 0 if p is invalid */
size_t accept_mbq_payload_offset(const accept_mbq_params* p);
size_t accept_mbq_workspace_size(const accept_mbq_params* p);
accept_status accept_mbq_compress(const accept_mbq_params* p, const float* d_x, const float* d_alpha_prev,
                                  float* d_alpha_next, void* d_stream, size_t stream_bytes, void* d_ws,
                                  size_t ws_bytes, void* cuda_stream);
/* Reads k and n from p; the kernel checks them against the header (ACCEPT_DEV_BAD_HEADER). */
accept_status accept_mbq_decompress(const accept_mbq_params* p, const void* d_stream, size_t stream_bytes,
                                    float* d_xhat, void* d_ws, size_t ws_bytes, void* cuda_stream);

/*
 * Synchronises cuda_stream, copies the status word to the host and returns it in *status_bits
 * (ACCEPT_DEV_* bits).  Returns ACCEPT_ERR_CUDA if the stream reports an error.
 */
accept_status accept_last_device_status(const void* d_ws, void* cuda_stream, uint32_t* status_bits);

/*
 * Parses the 32 header bytes (a HOST copy) into *out; ACCEPT_ERR_BAD_STREAM_HEADER if the magic,
 * version or any field is invalid.  For receivers that know nothing but the bytes they got (Sec. 3.4).
 */
accept_status accept_parse_header(const void* h_header, accept_params* out);

/*
 * Bit width the paper's schedule prescribes after n_lr_changes learning-rate changes:
 * forward (Sec. 3.3 "Forward Quantizer"): starts at 2, +1 per change, at most 4;
 * backward ("Backward Quantizer"): 8 until the first change, then 4.
 */
int accept_bitwidth_schedule(int is_backward, int n_lr_changes);

/* Number of kernels the library has launched in this process (all entry points). */
uint64_t accept_launch_count(void);

/*
 * Launches an EMPTY kernel of `blocks` blocks of `threads` threads on cuda_stream exactly as every kernel of
 * this library is launched (same launch attribute, same first instructions).  It measures what a launch
 * costs where a call is bound by launching rather than by bytes (tensors of a few MB): replayed from a
 * CUDA graph beside the codec's own kernels it gives the floor under their times.  The paper has no
 * counterpart.  blocks in [1, 2^31), threads in [32, 1024].
 */
accept_status accept_launch_null(uint32_t blocks, uint32_t threads, void* cuda_stream);

/*
 * For the checking build of this library (the same sources compiled with -DACCEPT_BOUNDS_CHECK, which the
 * tests load in place of a memory checker): every access of a kernel to caller memory is compared with
 * the byte ranges of the call (input, stream up to accept_compressed_size, workspace up to its size
 * query, output), and one that falls outside -- or a write into the input -- is skipped and counted
 * instead of performed.  This call synchronises cuda_stream, returns the number of skipped accesses since
 * the previous report in *violations and, optionally, the address of the first one and its size (low 32
 * bits) and kind (bit 32: write), then clears the count.  The paper has no counterpart.  In the normal
 * build nothing is checked: *violations = 0 and the result is ACCEPT_ERR_UNCHECKED_BUILD.
 */
accept_status accept_bounds_check_report(void* cuda_stream, uint32_t* violations, uint64_t* first_address,
                                         uint64_t* first_size_and_kind);

#ifdef __cplusplus
}
#endif
#endif /* ACCEPT_H_ */
