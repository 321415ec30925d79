// Shared declarations of the PVQ library's translation units (host side and
// kernel launch parameters).  Not part of the public interface.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "pvq.h"

namespace pvq {

constexpr int kMaxBatch = 32;     // matrices per launch
constexpr int kMaxWords = 32;     // limbs per code (1024-bit codes)
constexpr int kMaxGroup = 256;    // largest group size; above 64 (or 6 limbs) the tables stay in global memory
constexpr int kMaxPulses = 8191;  // y_i fits 16 bits with room, a_i < 2^23 (up to 1023: one builder thread per k)

// One matrix as the kernels see it.
struct MatrixArgs {
    const void* x;        // encode / round-trip input
    void* out;            // decode / round-trip output (bf16)
    uint32_t* codes;
    uint8_t* scale_idx;
    float* row_norm;
    const float* edges;
    const float* levels;
    long long rows, cols, ld, ld_out;
    int G;                // groups per row
    int sstride;          // bytes per row of scale_idx
    int rows_per_tile;    // encode: rows one thread block covers
    int chunks;           // encode: pieces a row longer than the block is taken in (else 1)
    unsigned tile_begin;  // first tile of this matrix in the launch
};

struct BatchArgs {
    MatrixArgs m[kMaxBatch];
    int count;
    unsigned total_tiles;
    int K;
    int scale_bits;
    int code_words;         // W: 32-bit words of one code in memory (kernels may compute in more)
    const uint32_t* table;  // the blob written by pvq_build_count_table (see TableLayout)
    uint32_t* status;
    int walk_phases;        // decode: which walk tables are staged in shared memory (see walk_tables)
    // The integers 1 and -1 as kernel arguments.  Multiply-adds by a factor the assembler cannot
    // see through stay multiply-adds, which run on the FMA pipe; the walk uses them for plain
    // moves, adds and subtracts to take load off the integer ALU pipe, its bottleneck.
    uint32_t c_one, c_minus_one;
    // rotation in front of the encoder (Sec. 2.3 / Sec. 3.3 Step 1); rot_block = 0: none
    int amp_mode;            // encode: 0 amplitude ||x_g||, 1 least-squares amplitude (Step 4)
    int fused;               // global-table encoder: decode the code just made instead of storing it
    const float* rot_signs;  // +-1, rot_block of them
    int rot_block;           // power of two, a multiple of N, dividing every cols
    uint32_t* debug_status;  // bounds-checked build: where violations are reported (pvq_debug_status); else null
    // decode by threshold search (SearchLayout): the section's place in the blob and its bytes
    uint32_t srch_off, srch_bytes;
    uint32_t srch_t_off;       // where the thresholds T start in the section; they stay in global memory
    uint32_t srch_t_before_e;  // bytes from a row of T to the same row of E
};

// Layout of the table blob.  Section 0 is the count table as the paper defines it,
// [n][k][W] words for n = 0..N-1, k = 0..K.  The other sections are the same numbers
// rearranged for the kernels, so that a thread block can stage them with one flat copy:
//
//   bound       N(N,K) as 16 words, 64 words for codes of more than 12 words (codes are valid
//               below it)
//   walk[0]     rows by position i (row i holds N(N-1-i, .)), `rowlen` entries of
//               `top_words` words each, entry (i, col) = N(N-1-i, col), zero padded
//   walk[1]     same with 2-word entries, values from 2^62 up replaced by 2^62 (present when
//               top_words > 2)
//   walk[2]     same with 1-word entries, values from 2^30 up replaced by 2^30 (present when
//               top_words > 1)
//
// rowlen is K+1 rounded up to an even number: consecutive positions on a diagonal of the
// table, (i, col) and (i+1, col+1), are then an odd number of entries apart, so threads that
// sit on neighbouring diagonals' cells read different shared-memory banks.
//
//   enc[0..2]   for the encoder, rows by position i, K+2 entries of `top_words` words each,
//               entry (i, col+1) for col = -1..K, with V(n,k) = sum_{j<=k} N(n,j), V(n,-1) = 0
//               (App. C.2) and n = N-1-i, all modulo 2^(32 W):
//                 enc[0]  U(n,col) = V(n,col) + V(n,col-1)
//                 enc[1]  2 V(n,col)
//                 enc[2]  V(n,col)
//
// For the kernels that keep their tables in shared memory (N <= 64, W <= 6) three more
// sections follow:
//
//   walkd       the walk table as doubles (8 bytes an entry, same rows and row length as
//               walk[0]), values from 2^53 up replaced by 2^53: the last stretch of the walk,
//               once every remainder is below 2^53, runs in fp64
//   start       U(N-1, K) as `top_words` words (16 bytes reserved): where the encoder's sum starts
//   cenc[0..1]  the encoder's tables in telescoped form (present for codes of up to 4 words and
//               up to 127 pulses when both fit 160 KB), rows by position i, `crow` entries of
//               `top_words` words for k = 0..K (zeros beyond K), crow = 32, 64 or 128, the
//               first that holds K+1, stored word plane by word plane (a row is `top_words`
//               planes of crow words, plane j holding word j of every entry); cenc[1] follows
//               cenc[0] after kCencSkew bytes.  Modulo 2^(32 W):
//                 cenc[0]  U(n-1,k) - U(n,k)      for y_i <= 0
//                 cenc[1]  U(n-1,k) - 2 V(n,k)    for y_i > 0
//               with n = N-1-i and U(-1, .) = 0.  The contribution of position i to the code,
//               U(n,k_i) - U(n,k_{i+1}) or U(n,k_i) - 2 V(n,k_{i+1}) (k_i pulses before it,
//               k_{i+1} after it), then costs one table read: the U(n,k_i) of position i is
//               carried by the entry of position i-1, that of position 0 is `start`.
// words per entry of the widest tables for W-word codes
__host__ __device__ constexpr int top_words_of(int W) {
    return W <= 2 ? W : (W <= 4 ? 4 : (W <= 6 ? 6 : (W <= 8 ? 8 : (W <= 12 ? 12 : ((W + 3) & ~3)))));
}

// words of the blob's copy of N(N,K)
__host__ __device__ constexpr int bound_words_of(int W) { return W <= 12 ? 16 : 64; }

struct TableLayout {
    int rowlen;
    int top_words;
    uint32_t bound_off;
    uint32_t walk_off[3];
    uint32_t walk_bytes[3];
    uint32_t enc_off[3];
    uint32_t enc_bytes;  // of each of the three
    uint32_t walkd_off, walkd_bytes;  // 0 bytes: absent
    uint32_t start_off;
    uint32_t cenc_off[2];
    uint32_t cenc_bytes;  // of each of the two; 0: absent
    int crow;             // entries per row of cenc
    uint32_t total;
};

constexpr uint32_t kCencLimit = 160u * 1024u;  // both telescoped encoder tables have to fit this
// cenc[1] starts half a row of banks (64 bytes) off a multiple of 128 behind cenc[0]: threads of a
// warp that read the same column of the two tables then hit different banks
constexpr uint32_t kCencSkew = 64u;

__host__ __device__ inline TableLayout table_layout(int N, int K, int W) {
    TableLayout L;
    if (N > kMaxGroup || W > kMaxWords) {  // no kernel for these: the blob is the plain count table
        L.rowlen = 0;
        L.top_words = 0;
        L.bound_off = 0;
        for (int p = 0; p < 3; ++p) L.walk_off[p] = L.walk_bytes[p] = L.enc_off[p] = 0;
        L.enc_bytes = 0;
        L.walkd_off = L.walkd_bytes = L.start_off = L.cenc_off[0] = L.cenc_off[1] = L.cenc_bytes = 0;
        L.crow = 0;
        L.total = static_cast<uint32_t>(N) * (K + 1) * W * 4u;
        return L;
    }
    L.rowlen = (K + 2) & ~1;
    L.top_words = top_words_of(W);
    uint32_t off = static_cast<uint32_t>(N) * (K + 1) * W * 4u;
    off = (off + 127u) & ~127u;
    L.bound_off = off;
    off += (static_cast<uint32_t>(bound_words_of(W)) * 4u + 127u) & ~127u;
    const uint32_t entries = static_cast<uint32_t>(N) * L.rowlen;
    const int words[3] = {L.top_words, L.top_words > 2 ? 2 : 0, L.top_words > 1 ? 1 : 0};
    for (int p = 0; p < 3; ++p) {
        L.walk_off[p] = off;
        L.walk_bytes[p] = entries * words[p] * 4u;
        off += (L.walk_bytes[p] + 127u) & ~127u;
    }
    L.enc_bytes = static_cast<uint32_t>(N) * (K + 2) * L.top_words * 4u;
    for (int p = 0; p < 3; ++p) {
        L.enc_off[p] = off;
        off += (L.enc_bytes + 127u) & ~127u;
    }
    L.walkd_off = L.walkd_bytes = L.start_off = L.cenc_off[0] = L.cenc_off[1] = L.cenc_bytes = 0;
    L.crow = 0;
    if (N <= 64 && W <= 6) {
        L.walkd_off = off;
        L.walkd_bytes = entries * 8u;
        off += (L.walkd_bytes + 127u) & ~127u;
        L.start_off = off;
        off += 128u;
        const int crow = K + 1 <= 32 ? 32 : (K + 1 <= 64 ? 64 : 128);
        const uint32_t cb = static_cast<uint32_t>(N) * crow * L.top_words * 4u;
        if (W <= 4 && K + 1 <= 128 && 2u * cb <= kCencLimit) {
            L.crow = crow;
            L.cenc_bytes = cb;
            L.cenc_off[0] = off;
            L.cenc_off[1] = off + cb + kCencSkew;
            off += 2u * cb + 128u;  // cb is a multiple of 128
        }
    }
    L.total = off;
    return L;
}

// ---- tables of the decoder that searches (csrc/pvq_decode_search.cu) ------------------------
//
// With q = N(n+1,k) - r (r the part of the code not yet explained, n dimensions after the
// current position, k pulses left) the coordinate of Algorithm 3 follows from where q falls
// among the thresholds of row n,
//     T_n[2k'] = U(n,k') = V(n,k') + V(n,k'-1),    T_n[2k'+1] = 2 V(n,k'),    k' = 0..K
// (V(n,k) = sum_{j<=k} N(n,j), App. C.2): with m the first index whose threshold is >= q,
// k' = m >> 1 pulses remain after the position, |y| = k - k', y > 0 iff m is odd, and the q of
// the next position is q + E_n[m], E_n[m] = U(n-1,k') - T_n[m] (the encoder's telescoped
// tables).  m is found without a loop.  A key of q (its leading 24 bits as an fp32, see
// search_key) shifted right by a per-row amount numbers a bucket; the shift is chosen (on the
// host, from the exact thresholds) so that no two thresholds of a row share a bucket.  The
// bucket's entry holds m0, the number of thresholds in earlier buckets, and the key bits
// below the shift of the one threshold that can lie in the bucket: q is beyond that threshold
// iff its own low key bits are larger, and only when they are equal and the threshold has more
// than 24 bits (the two agree in their leading 24 bits) does the multi-word compare with
// T_n[m0] have to decide.
//
// Values shrink from row to row (q <= N(n+1,K) at row n), so the rows are narrower towards
// the end of the vector: a row's thresholds and increments are stored, and its arithmetic is
// done, in the fewest words that hold N(n+1,K); rows are classed in aligned blocks of four
// (a block takes the width of its top row), so that the decoder works through four
// positions at a time in one width.
//
// The section follows the sections of TableLayout in the blob (128-byte aligned) and is
// staged as one piece:
//     header    32 bytes: magic, N, K, bytes of the section, then the number of rows whose
//               arithmetic is done in 4, 3, 2 and 1 words (the widest rows are the top ones)
//     records   one 16-byte record per row n: 32 - shift, the byte offsets (from the section's
//               start) of the row of E and of the row's bucket table minus four times its
//               first bucket number, and the shift; the row of T is t_off - e_off from that of E
//     buckets   the rows' tables, one after the other, 4 bytes a bucket: m0 in the low byte,
//               in the top bits the low `shift` key bits of T_n[m0] if T_n[m0] lies in the
//               bucket, else all ones in bits 8..31 (no q of the bucket is beyond T_n[m0]);
//               bit 8 is set when T_n[m0] < 2^24, where equal keys mean equal numbers
//     T, E      rows of `plane` entries (64, 128 or 256: the first that holds the thresholds
//               m = 0..2K; E modulo 2^(32 words)), word by word: a row of w words is w planes
//               of `plane` 32-bit words, plane j holding word j of every entry.  The threads
//               of a warp read entries a few indices apart, which word planes put in
//               different banks (entries of 16 bytes would collide in groups of eight).
constexpr int kSearchMaxRows = 64;
constexpr uint32_t kSearchMagic = 0x53515650u;
constexpr uint32_t kSearchHeader = 32u;
constexpr uint32_t kSearchLimit = 184u * 1024u;  // the section has to leave room for the output slots

__host__ __device__ constexpr int search_plane_of(int K) { return 2 * K + 2 <= 64 ? 64 : (2 * K + 2 <= 128 ? 128 : 256); }

struct SearchRows {  // what the builder needs per row
    uint32_t b_off[kSearchMaxRows];   // of the row's bucket table inside `buckets`
    uint32_t b_len[kSearchMaxRows];   // its entries
    uint32_t te_off[kSearchMaxRows];  // of the row inside T (and inside E)
    uint8_t shift[kSearchMaxRows];    // bucket number = (key >> shift) - (key(1) >> shift)
    uint8_t words[kSearchMaxRows];    // words the row's arithmetic is done in
};

struct SearchLayout {
    bool present;
    int count[5];         // count[w]: rows done in w words
    int plane;            // entries per word plane of a row of T or E
    uint32_t off;         // of the section in the blob
    uint32_t rec_off, b_off, t_off, e_off;  // of its parts, from the section's start
    uint32_t te_bytes;    // of T, and of E
    uint32_t total;       // bytes of the section (a multiple of 128)
    SearchRows rows;
};

// host helpers (pvq_host.cu)
int set_cuda_error(cudaError_t e);  // records e, returns PVQ_ERR_CUDA
int code_words_for(int N, int K);   // W, or 0 when it cannot be computed
bool count_fills_its_words(int N, int K);  // N(N,K) == 2^(32 W) exactly: the one count that needs W + 1 words
// the search section for (N,K), memoised; present == false where the decoder walks instead
const SearchLayout& search_layout_for(int N, int K);
bool is_aligned(const void* p, size_t a);

// What a launcher needs to know about the current device and a kernel at a given block size
// and dynamic shared memory: looked up once, then served from a cache (the queries cost more
// than a small launch).  prepare_kernel also raises the kernel's shared-memory limit.
struct DeviceInfo {
    int sms;
    int smem_max;  // opt-in shared memory per block
};
int device_info(DeviceInfo* out);                                                  // pvq_status
int prepare_kernel(const void* kern, int threads, size_t smem, int* blocks_per_sm);  // pvq_status

// launchers (one per kernel family); all return a pvq_status
int launch_decode(const BatchArgs& args, int N, int W, cudaStream_t stream);
int launch_decode_search(const BatchArgs& args, int N, int W, const SearchLayout& S, cudaStream_t stream);
// large groups / wide codes (N = 128 or more than 6 words): tables in global memory
int launch_big(const BatchArgs& args, int dtype, int N, int W, bool decode, cudaStream_t stream);  // args.fused: round trip
int launch_encode(const BatchArgs& args, int dtype, int N, int W, bool fused, cudaStream_t stream);  // rotates when args.rot_block != 0

// ---------------------------------------------------------------- device bits

#ifdef __CUDACC__

// balanced tree over contiguous halves, each addition rounded to fp32
template <int N>
__device__ __forceinline__ float tree_sum(const float (&v)[N]) {
    float t[N];
#pragma unroll
    for (int i = 0; i < N; ++i) t[i] = v[i];
#pragma unroll
    for (int s = 1; s < N; s <<= 1) {
#pragma unroll
        for (int i = 0; i < N; i += 2 * s) t[i] = __fadd_rn(t[i], t[i + s]);
    }
    return t[0];
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// which matrix does tile t belong to?  (count <= 32: a short scan)
__device__ __forceinline__ int find_matrix(const BatchArgs& a, unsigned tile) {
    int mi = 0;
    for (int i = 1; i < a.count; ++i)
        if (tile >= a.m[i].tile_begin) mi = i;
    return mi;
}

// ---- bounds-checked build (-DPVQ_DEBUG) ---------------------------------------------------
// Every read of a staged table, every write of an output slot, the indices of the encoders'
// shared arrays and the global stores are checked against the extent they belong to; a
// violation ORs a bit into the word given to pvq_debug_status and the access is skipped
// (nothing traps).  The decode walk runs its plain C++ step in this build, so that each of
// its table reads and slot writes passes through the checked helpers; the hand-written
// forms of the production build take the same pointers through the same transitions.
#ifdef PVQ_DEBUG
struct DebugCtx {
    uint32_t tab_lo, tab_hi;                      // shared addresses: the staged tables
    uint32_t slot_base, slot_stride, slot_bytes;  // output slots: thread t owns [base + t * stride, + bytes)
    uint32_t slot_chain, slot_end;                // ... and the same range every slot_chain bytes up to slot_end (0: no)
    uint32_t* status;
};
__shared__ DebugCtx s_debug;

// thread 0 fills the context; the caller's next block-wide barrier publishes it
__device__ __forceinline__ void debug_begin(uint32_t tab_lo, uint32_t tab_hi, uint32_t slot_base, uint32_t slot_stride,
                                            uint32_t slot_bytes, uint32_t* status) {
    if (threadIdx.x == 0) {
        s_debug.tab_lo = tab_lo;
        s_debug.tab_hi = tab_hi;
        s_debug.slot_base = slot_base;
        s_debug.slot_stride = slot_stride;
        s_debug.slot_bytes = slot_bytes;
        s_debug.slot_chain = s_debug.slot_end = 0u;
        s_debug.status = status;
    }
    __syncthreads();
}
__device__ __forceinline__ void debug_flag(uint32_t bit) {
    if (s_debug.status) atomicOr(s_debug.status, bit);
}
__device__ __forceinline__ bool debug_table_ok(uint32_t addr, uint32_t bytes) {
    const bool ok = addr >= s_debug.tab_lo && addr + bytes <= s_debug.tab_hi && (addr & 3u) == 0u;
    if (!ok) debug_flag(PVQ_DEBUG_TABLE_READ);
    return ok;
}
__device__ __forceinline__ bool debug_slot_ok(uint32_t addr, uint32_t bytes) {
    const uint32_t lo = s_debug.slot_base + threadIdx.x * s_debug.slot_stride;
    bool ok = addr >= lo;
    if (s_debug.slot_chain != 0u)
        ok = ok && (addr - lo) % s_debug.slot_chain + bytes <= s_debug.slot_bytes && addr + bytes <= s_debug.slot_end;
    else
        ok = ok && addr + bytes <= lo + s_debug.slot_bytes;
    if (!ok) debug_flag(PVQ_DEBUG_SLOT_WRITE);
    return ok;
}
// index into one of the encoders' shared arrays / a global output
__device__ __forceinline__ bool debug_index_ok(long long idx, long long limit, uint32_t bit) {
    const bool ok = idx >= 0 && idx < limit;
    if (!ok) debug_flag(bit);
    return ok;
}
#define PVQ_DEBUG_INDEX(idx, limit, bit) debug_index_ok((idx), (limit), (bit))
#else
#define PVQ_DEBUG_INDEX(idx, limit, bit) true
#endif

#endif  // __CUDACC__

}  // namespace pvq
