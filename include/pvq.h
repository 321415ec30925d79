/*
 * pvq.h - C ABI of the B200 (sm_100a) group-wise Pyramid Vector Quantization codec.
 *
 * A rows x cols matrix (row-major) is cut into groups of N contiguous values
 * along each row, G = cols / N groups per row (Sec. 3.3 Step 0).  Each group is
 * stored as
 *   - one direction code: the Fischer index (Algorithm 2) of the point of the
 *     pyramid P(N,K) = { y in Z^N : sum |y_i| = K } nearest to the group's
 *     direction (Sec. 2.5), an unsigned integer in [0, N(N,K) - 1] kept as W
 *     little-endian 32-bit words, W = ceil(ceil(log2 N(N,K)) / 32);
 *   - one amplitude index of scale_bits bits: the quantile bin of the group's
 *     share of the row energy, u = ||x_g||^2 / ||x_row||^2, under
 *     Beta(N/2, N(G-1)/2) (Sec. 3.4, Sec. 3.3 Step 5);
 * and each row stores its norm ||x_row||_2 once (fp32), which Step 5 says has
 * to be kept for dequantisation.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers owned by the caller; the library
 *     never allocates, frees or keeps them.  Everything else is host memory.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *     return without synchronising; outputs are valid once the stream reaches
 *     that point.  The device current at the call must own all pointers.
 *   - Every function returns a pvq_status; nothing is thrown across the ABI and
 *     no argument error reaches a kernel.
 *   - Inputs must be finite, and so must the fp32 sums taken over them: the l1 norm and
 *     the energy of every group, the energy of every row, and K divided by a group's l1
 *     norm.  NaN or Inf in the input, or a sum that overflows fp32, gives unspecified
 *     codes (the group is then usually treated as having no direction) but never an
 *     out-of-bounds access.
 *
 * Storage formats (also the persistent format of an encoded matrix)
 *   codes      uint32  codes[(r*G + g)*W + w], w = 0 the least significant word.
 *   scale_idx  bytes   one LSB-first bit stream per row: group g occupies bits
 *                      [g*b, (g+1)*b) of the row, b = scale_bits; the row stride
 *                      is pvq_scale_row_stride(G, b) = ceil(G*b/8) rounded up to 4.
 *   row_norm   float   row_norm[r].
 *   count table uint32 pvq_count_table_bytes(N,K) bytes, 16-byte aligned, written by
 *                      pvq_build_count_table.  It opens with the table of the paper,
 *                      table[(n*(K+1) + k)*W + w] = word w of N(n,k) for n = 0..N-1
 *                      (dimensions left after a position) and k = 0..K.  For N <= 256
 *                      and W <= 32 the same numbers follow, rearranged for the kernels
 *                      (each section starts on a 128-byte boundary, in this order):
 *                        N(N,K) as 16 words (64 words when W > 12);
 *                        the decoder's tables, rows by position i (row i = N(N-1-i, .)),
 *                        K+1 rounded up to even entries per row: one with entries of
 *                        1, 2, 4, 6, 8, 12, 16, 20, ... words (the first that holds W), then, when W > 2,
 *                        one with 2-word entries where values from 2^62 up are
 *                        replaced by 2^62, and, when W > 1, one with 1-word entries
 *                        where values from 2^30 up are replaced by 2^30;
 *                        the encoder's tables, rows by position, K+2 entries per row for
 *                        k = -1..K, of the cumulative counts V(n,k) = sum_{j<=k} N(n,j)
 *                        (App. C.2) modulo 2^(32 W): V(n,k) + V(n,k-1), then 2 V(n,k),
 *                        then V(n,k);
 *                        for N <= 64 and W <= 6: the decoder's widest table as doubles
 *                        (values from 2^53 up replaced by 2^53), V(N-1,K) + V(N-1,K-1), and,
 *                        where they fit, the encoder's tables in telescoped form (one read
 *                        per position);
 *                        for W <= 4 and K <= 127, where it fits shared memory: the tables
 *                        of the decoder that finds each coordinate by one threshold
 *                        search (a 16-byte header with N and K, one 16-byte record per
 *                        row, the rows' bucket tables, the thresholds and the
 *                        increments of the running value).
 *                      Callers treat everything after the first section as opaque.
 *   edges      float   2^b - 1 ascending bin edges of u.
 *   levels     float   2^b values sqrt(PPF((q + 1/2) / 2^b)): the factor that
 *                      multiplies row_norm to give the dequantised amplitude.
 */
#ifndef PVQ_H_
#define PVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PVQ_OK = 0,
    PVQ_ERR_INVALID_ARG = 1,     /* null pointer, non-positive size, cols % N != 0, ... */
    PVQ_ERR_UNSUPPORTED = 2,     /* (N, K, W) or G outside what the kernels are built for */
    PVQ_ERR_ALIGNMENT = 3,       /* a pointer or leading dimension breaks the stated alignment */
    PVQ_ERR_TABLE_TOO_SMALL = 4, /* buffer smaller than the size the call needs */
    PVQ_ERR_CUDA = 5             /* a CUDA call failed; see pvq_last_cuda_error() */
} pvq_status;

#define PVQ_DTYPE_F32 0
#define PVQ_DTYPE_BF16 1

/* bit 0 of the decode status word: some code was >= N(N,K) */
#define PVQ_STATUS_INVALID_CODE 1u
/* bit 1: a thread block gave up waiting for its tables to arrive in shared memory and wrote
 * nothing (a bounded wait; not expected to happen).  Decoding reports it in its d_status, the
 * encode-side calls in the word of pvq_encode_status. */
#define PVQ_STATUS_STAGING_TIMEOUT 2u
/* bit 2 of the decode status word: the table given to the call was not built for this (N,K)
 * (its header says so); nothing was decoded. */
#define PVQ_STATUS_TABLE_MISMATCH 4u

typedef void* pvq_stream_t; /* a cudaStream_t */

/* Human-readable name of a status.  Never NULL. */
const char* pvq_strerror(int status);

/* cudaError_t (as int) of the last failed CUDA call made by this library on the
 * calling thread; 0 if none. */
int pvq_last_cuda_error(void);

/* ---- host-side parameter helpers (exact integer arithmetic, no GPU) ---------- */

/* ceil(log2 N(N,K)): bits of one direction code (Sec. 3.3 Step 7).  N >= 1, K >= 0. */
int pvq_index_bits(int N, int K, int* bits_out);

/* Sec. 3.3 Step 2: the largest K with N(N,K) <= 2^index_bits (the comparison is made
 * on the integers).  *K_out = 0 when not even one pulse fits. */
int pvq_max_pulses(int N, int index_bits, int* K_out);

/* W = ceil(pvq_index_bits / 32), at least 1. */
int pvq_code_words(int N, int K, int* W_out);

/* Bytes of the device count table for (N,K), all sections: at least N * (K+1) * W * 4.
 * 0 on bad arguments. */
size_t pvq_count_table_bytes(int N, int K);

/* Row stride in bytes of the packed amplitude indices. */
size_t pvq_scale_row_stride(int64_t G, int scale_bits);

/* ---- set-up kernels (cold path) --------------------------------------------------- */

/* Fill d_table with N(n,k), n = 0..N-1, k = 0..K (Sec. 2.4 recurrence; built a row at a
 * time with a parallel prefix sum over k as in App. C.2 / Algorithm 4, by one thread
 * block).  `bytes` is the size of d_table and must be at least
 * pvq_count_table_bytes(N,K).  Requires 1 <= N <= 256, 1 <= K <= 8191, W <= 32. */
int pvq_build_count_table(int N, int K, uint32_t* d_table, size_t bytes, pvq_stream_t stream);

/* Fill d_edges (2^b - 1 floats) and d_levels (2^b floats) for group size N, G groups per
 * row and b = scale_bits (Sec. 3.4: quantize = floor(CDF * 2^b), dequantize =
 * PPF((q + 1/2) / 2^b), Beta(N/2, N(G-1)/2)).  Computed in fp64 on the device and rounded
 * once to fp32.  Requires N even, G >= 2, 1 <= b <= 8.  Either pointer may be NULL. */
int pvq_build_scale_codebook(int N, int64_t G, int scale_bits, float* d_edges, float* d_levels,
                             pvq_stream_t stream);

/* ---- hot path --------------------------------------------------------------------- */

/* Encode (Sec. 3.3 Steps 3, 4, 5, 7; Algorithms 1 and 2).
 *   d_x        rows x cols values of `dtype`, leading dimension ld (elements); 16-byte
 *              aligned, ld a multiple of 8 (bf16) or 4 (fp32) elements.
 *   N, K       group size (power of two, 8..256) and pulses (up to 8191, codes of up to 32
 *              words); cols % N == 0; 2 <= G <= 4096.  Codes of up to 2, 3, 4, 6 words at
 *              N = 8, 16, 32, 64 run on the kernels with the tables in shared memory.  Wider
 *              codes at N >= 16, and N = 128 and 256, run on slower kernels that keep the
 *              tables in global memory (the paper's grid of group sizes and direction bits,
 *              Sec. 4.1).
 *              Rows of up to 4096 groups are taken by pvq_encode proper (amplitude ||x_g||,
 *              no rotation) for codes of up to 4 words and K <= 127.  Everything else on the
 *              encode side - pvq_roundtrip, pvq_encode_amp with amp_mode 1, the rotating
 *              calls, 5- and 6-word codes, K > 127, the global-table kernels - keeps a whole
 *              row in one thread block and returns PVQ_ERR_UNSUPPORTED for G > 512 (fewer on
 *              the global-table kernels, where a row also has to fit shared memory: about
 *              G <= 256 at N = 128, 192 at N = 256).  Decoding has no such limit.
 *   scale_bits 1..8 (quantile index), or 16 (see pvq_encode_amp).
 *   d_table    from pvq_build_count_table(N, K, ...).
 *   d_edges    2^scale_bits - 1 bin edges.
 *   d_codes    out, rows*G*W words.      d_scale_idx  out, rows * stride bytes.
 *   d_row_norm out, rows floats.
 * Arithmetic: fp32 with one rounding per operation; sums over a group and over the
 * groups of a row use a balanced tree over contiguous halves (row: zero-padded to a
 * power of two).  Amplitude index q = #{ j : u >= edges[j] }.  Direction: scale to the
 * l1 ball of radius K, floor, then hand out the missing pulses one at a time to the
 * largest residual, lowest index first among equals; a group with zero l1 norm maps to
 * (K,0,...,0). */
int pvq_encode(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
               int scale_bits, const uint32_t* d_table, const float* d_edges, uint32_t* d_codes,
               uint8_t* d_scale_idx, float* d_row_norm, pvq_stream_t stream);

/* Decode to bf16 (Algorithm 3; Sec. 2.4 projection on the sphere; Sec. 3.4 dequantize).
 *   out[r][g*N + i] = bf16( y_i * (row_norm[r] * levels[q]) / sqrt(sum y^2) ), rounded to
 *   nearest even, with y the pyramid point of the code.
 *   d_out      rows x cols bf16, leading dimension ld_out (elements, multiple of 8),
 *              16-byte aligned.
 *   d_status   optional device word; PVQ_STATUS_INVALID_CODE is OR-ed into it when a code
 *              is >= N(N,K) (that group decodes to zeros), PVQ_STATUS_TABLE_MISMATCH when
 *              d_table was built for other (N,K) (nothing is written then),
 *              PVQ_STATUS_STAGING_TIMEOUT when a block gave up waiting for its tables.
 *              May be NULL. */
int pvq_decode(const uint32_t* d_codes, const uint8_t* d_scale_idx, const float* d_row_norm,
               int64_t rows, int64_t cols, int N, int K, int scale_bits, const uint32_t* d_table,
               const float* d_levels, void* d_out, int64_t ld_out, uint32_t* d_status,
               pvq_stream_t stream);

/* Fused encode -> decode of activations (Sec. 2.2, Sec. 4.3: on-the-fly quantisation):
 * each group is encoded to its integer code and decoded again inside one kernel, the code
 * living in registers; only d_x is read and d_out written.  Same arguments and arithmetic
 * as pvq_encode followed by pvq_decode. */
int pvq_roundtrip(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                  int scale_bits, const uint32_t* d_table, const float* d_edges,
                  const float* d_levels, void* d_out, int64_t ld_out, pvq_stream_t stream);

/* pvq_encode with a choice of amplitude (Sec. 3.3 Step 4).
 *   amp_mode 0  the amplitude of a group is ||x_g||_2, as in pvq_encode;
 *   amp_mode 1  least squares: the projection of x_g on the chosen direction,
 *               a = (sum_i |y_i| |x_i|) / sqrt(sum_i y_i^2)  (fp32, products rounded, summed by
 *               the balanced tree), and u = a^2 / ||x_row||^2 for the quantile index.
 * Everything else as pvq_encode; decoding does not depend on the mode.
 *
 * scale_bits = 16 (all encode / decode entry points): instead of a quantile index the stream
 * holds the amplitude itself as IEEE binary16, rounded to nearest even, 16 bits per group
 * (Sec. 4.1: 16-bit amplitudes); d_edges / d_levels are then unused and may be NULL, and
 * the row norms are written but not read. */
int pvq_encode_amp(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                   int scale_bits, int amp_mode, const uint32_t* d_table, const float* d_edges,
                   uint32_t* d_codes, uint8_t* d_scale_idx, float* d_row_norm, pvq_stream_t stream);

/* Rotation on the fly (Sec. 2.3 "Hadamard coherence processing", Sec. 3.3 Step 1, along the
 * input dimension; Sec. 4.3 for activations, which have to be rotated at run time): every
 * row is multiplied elementwise by the signs d_signs[col % block] (+-1 as float, `block` of
 * them) and every contiguous run of `block` columns by H_block / sqrt(block), H the
 * Sylvester-Walsh-Hadamard matrix; the rotated row is then encoded (pvq_rotate_encode) or
 * encoded and decoded (pvq_rotate_roundtrip) exactly as by pvq_encode / pvq_roundtrip on fp32
 * input, without the rotated matrix ever being written to memory.
 *   block      a power of two, a multiple of N, dividing cols, at most 16384.
 * Arithmetic: fp32; the sign flip, then butterflies (a, b) -> (a + b, a - b) with strides
 * 1, 2, 4, ..., block/2, one rounding each, then one multiplication by the fp32 nearest to
 * 1/sqrt(block).  The other arguments are those of pvq_encode / pvq_roundtrip; on the kernels
 * with the tables in shared memory the fused form needs K <= 127. */
int pvq_rotate_encode(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int block,
                      const float* d_signs, int N, int K, int scale_bits, const uint32_t* d_table,
                      const float* d_edges, uint32_t* d_codes, uint8_t* d_scale_idx, float* d_row_norm,
                      pvq_stream_t stream);
int pvq_rotate_roundtrip(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int block,
                         const float* d_signs, int N, int K, int scale_bits, const uint32_t* d_table,
                         const float* d_edges, const float* d_levels, void* d_out, int64_t ld_out,
                         pvq_stream_t stream);

/* One matrix of a batched call.  Pointers are device pointers with the meaning and
 * alignment of the corresponding pvq_encode / pvq_decode arguments; d_edges / d_levels
 * belong to this matrix's G. */
typedef struct {
    const void* d_x;      /* encode input (unused by decode) */
    void* d_out;          /* decode output (unused by encode) */
    uint32_t* d_codes;
    uint8_t* d_scale_idx;
    float* d_row_norm;
    const float* d_edges;
    const float* d_levels;
    int64_t rows, cols, ld, ld_out;
} pvq_matrix_desc;

/* Encode / decode `count` matrices (1..32) that share dtype, N, K, scale_bits and the
 * count table with ONE kernel launch (all seven matrices of a decoder layer at once).
 * `descs` is a host array, copied into the launch; it may be freed on return. */
int pvq_encode_batched(const pvq_matrix_desc* descs, int count, int dtype, int N, int K,
                       int scale_bits, const uint32_t* d_table, pvq_stream_t stream);
int pvq_decode_batched(const pvq_matrix_desc* descs, int count, int N, int K, int scale_bits,
                       const uint32_t* d_table, uint32_t* d_status, pvq_stream_t stream);

/* Status word of the encode-side calls (pvq_encode, pvq_encode_amp, pvq_roundtrip, the rotating
 * calls, pvq_encode_batched), which take no status argument: a device word of the caller's into
 * which PVQ_STATUS_STAGING_TIMEOUT is OR-ed when a thread block gave up waiting for its tables
 * (its part of the output is then not written).  Applies to the later calls of the calling
 * thread; NULL (the default) switches reporting off.  (No counterpart in the paper.) */
int pvq_encode_status(uint32_t* d_status);

/* ---- for callers that cannot allocate device memory ---------------------------------- */

/* Size of the count table that is built into the library image (see below). */
#define PVQ_STATIC_TABLE_BYTES (1024u * 1024u)

/* pvq_decode without a caller-provided count table.  (The paper has no counterpart: this
 * is a packaging variant of pvq_decode, with identical results.)
 *
 * For hosts where device allocation is off limits once set-up is over - a plug-in inside
 * an engine that has already planned all of its memory, a control loop whose allocator is
 * frozen, a process whose memory budget is enforced by refusing cudaMalloc - the table
 * N(n,k) is kept in a fixed array inside the library (PVQ_STATIC_TABLE_BYTES per GPU that
 * loads the library, held until the process exits).  This call allocates and frees no
 * device memory; codes, amplitude indices, row norms, levels and the output are still the
 * caller's buffers, with the meaning and alignment they have in pvq_decode.  The first
 * call for an (N,K) in a process also fills small host-side caches (the code width, the
 * kernel's launch geometry), so make it during set-up.
 *
 *   - (N,K) whose table needs more than PVQ_STATIC_TABLE_BYTES (pvq_count_table_bytes
 *     tells) is refused with PVQ_ERR_TABLE_TOO_SMALL.
 *   - The first call on a device looks up the array's device address, creates one event
 *     and fills the table on `stream`; so does (the fill) any later call whose (N,K)
 *     differs from the previous call's on that device.  Make that first call before any
 *     stream capture begins.
 *   - All calls on a device share the one array, which keeps what the last call put
 *     there.  Nothing in it has to start at zero (the fill overwrites every word decode
 *     reads).  A call with the same (N,K) as the previous one only reads the array; if
 *     the fill is still in flight on another stream, the call first makes its stream wait
 *     for it, so such calls may overlap freely.  Two calls with different (N,K) whose
 *     work overlaps on the GPU - different streams, no dependency between them - race on
 *     the array: the second call's fill overwrites what the first call's decode reads. */
int pvq_decode_static_table(const uint32_t* d_codes, const uint8_t* d_scale_idx, const float* d_row_norm,
                            int64_t rows, int64_t cols, int N, int K, int scale_bits,
                            const float* d_levels, void* d_out, int64_t ld_out, uint32_t* d_status,
                            pvq_stream_t stream);

/* ---- bounds-checked build -------------------------------------------------------------- */

/* Bits of the word of pvq_debug_status. */
#define PVQ_DEBUG_TABLE_READ 1u   /* a read outside the staged tables */
#define PVQ_DEBUG_SLOT_WRITE 2u   /* a write outside the thread's output slots */
#define PVQ_DEBUG_SHARED_INDEX 4u /* an index outside one of the encoders' shared arrays */
#define PVQ_DEBUG_GLOBAL_STORE 8u /* a store outside an output buffer */

/* The library built with -DPVQ_DEBUG (`python -m paper_2410_16926_b200.build --debug`,
 * libpvq_b200_debug.so; shared-memory kernels only) checks every table read, slot write,
 * shared-array index and global store of its kernels against the extent it belongs to,
 * skips an access that falls outside and ORs the matching bit into *d_status (a device
 * word of the caller's, zeroed by the caller).  It is the memory-safety evidence of this
 * code base where a memory checker cannot be run; the results are those of the production
 * build.  (The paper has no counterpart.)  This call sets the word for all later calls of
 * the calling thread; NULL switches reporting off.  In the production build it returns
 * PVQ_ERR_UNSUPPORTED. */
int pvq_debug_status(uint32_t* d_status);

#ifdef __cplusplus
}
#endif
#endif /* PVQ_H_ */
