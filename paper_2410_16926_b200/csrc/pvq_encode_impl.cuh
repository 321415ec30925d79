// Encode kernel (and the fused encode -> decode round trip): templates shared by
// the per-group-size translation units.
//
// One thread encodes one group; a thread block covers whole rows (the row norm
// is the only quantity shared between groups).  Steps per group, in the order
// of Sec. 3.3: group norms, row norm, direction (Step 3: l1 scale, floor,
// greedy fix-up), Fischer index (Step 7, Algorithm 2), amplitude index (Step 5).
#pragma once
#include <cuda_fp16.h>

#include <algorithm>

#include "pvq_walk.cuh"

namespace pvq {

// ---- descending sorting network (Batcher's odd-even merge sort), in registers ----
// Written as template recursion so that every index is a compile-time constant: a loop
// nest that the compiler leaves partly rolled would put the array in local memory.
template <int N, int I, int J>
__device__ __forceinline__ void cmp_exchange(float (&v)[N]) {
    const float hi = fmaxf(v[I], v[J]);
    const float lo = fminf(v[I], v[J]);
    v[I] = hi;
    v[J] = lo;
}

// compare-exchange (I, I+R), (I+M, I+M+R), ... while I+R < END
template <int N, int I, int R, int M, int END>
__device__ __forceinline__ void cmp_exchange_row(float (&v)[N]) {
    if constexpr (I + R < END) {
        cmp_exchange<N, I, I + R>(v);
        cmp_exchange_row<N, I + M, R, M, END>(v);
    }
}

// merges the two sorted halves of the LEN elements LO, LO+R, LO+2R, ...
template <int N, int LO, int LEN, int R>
__device__ __forceinline__ void oddeven_merge(float (&v)[N]) {
    constexpr int M = R * 2;
    if constexpr (M < LEN) {
        oddeven_merge<N, LO, LEN, M>(v);
        oddeven_merge<N, LO + R, LEN, M>(v);
        cmp_exchange_row<N, LO + R, R, M, LO + LEN>(v);
    } else {
        cmp_exchange<N, LO, LO + R>(v);
    }
}

template <int N, int LO, int LEN>
__device__ __forceinline__ void oddeven_sort(float (&v)[N]) {
    if constexpr (LEN > 1) {
        oddeven_sort<N, LO, LEN / 2>(v);
        oddeven_sort<N, LO + LEN / 2, LEN / 2>(v);
        oddeven_merge<N, LO, LEN, 1>(v);
    }
}

template <int N>
__device__ __forceinline__ void sort_desc(float (&v)[N]) {
    oddeven_sort<N, 0, N>(v);
}

// v[idx] for a run-time idx in [0, N): a binary tree of selects on the bits of idx.
template <int N>
__device__ __forceinline__ float pick(const float (&v)[N], int idx) {
    float t[N];
#pragma unroll
    for (int i = 0; i < N; ++i) t[i] = v[i];
#pragma unroll
    for (int bit = 0; (1 << bit) < N; ++bit) {
        const int s = 1 << bit;
        const bool hi = (idx >> bit) & 1;
#pragma unroll
        for (int i = 0; i < N; i += 2 * s) t[i] = hi ? t[i + s] : t[i];
    }
    return t[0];
}

// |a| with the sign bit of s
__device__ __forceinline__ float with_sign_of(float a, float s) {
    return __int_as_float(__float_as_int(a) | (__float_as_int(s) & static_cast<int>(0x80000000u)));
}

// Element i of a group held as it sits in memory: N/2 words of two bf16 each, or N fp32 words.
// Widening bf16 is exact.  A group stays in this form for the whole kernel (half the
// registers of N floats for bf16) and its elements are widened where they are used.
template <int N, bool BF16>
__device__ __forceinline__ float raw_value(const uint32_t (&raw)[BF16 ? N / 2 : N], int i) {
    if constexpr (BF16)
        return __uint_as_float((i & 1) ? (raw[i / 2] & 0xffff0000u) : (raw[i / 2] << 16));
    else
        return __uint_as_float(raw[i]);
}

constexpr float kMagic = 8388608.0f;  // 2^23: a + 2^23 rounded down is 2^23 + floor(a) for 0 <= a < 2^23
constexpr int kMagicBits = 0x4B000000;

// Direction of one group (Sec. 2.5 / Algorithm 1 in the floor + greedy reading).
//   a_i = |x_i| * (K / l1), f_i = floor(a_i), e_i = a_i - f_i, d = K - sum f_i.
// The greedy loop "give one pulse to the largest residual, lowest index first among
// equals, d times" touches every element at most once when 0 <= d <= N (after its pulse
// an element's residual is negative, below every untouched one), so its result is: the d
// elements with the largest (e_i, -i) get +1.  v = the d-th largest residual comes from a
// sorting network; every e_i >= v gets a pulse, and when that hands out more than d (equal
// residuals straddle the cut) the elements equal to v with the highest indices give theirs
// back.
//
// Out: mag[i] = 2^23 + |y_i| as a float (the integer sits in the low mantissa bits) with the
// sign bit of x_i.  Returns false for a group without direction (l1 zero or not finite, or
// a scale that overflows): the point is then (K, 0, ..., 0).
template <int N, bool BF16>
__device__ __forceinline__ bool quantize_direction(const uint32_t (&raw)[BF16 ? N / 2 : N], float l1, int K,
                                                   float (&mag)[N]) {
    const float gsc = __fdiv_rn(static_cast<float>(K), l1);
    if (!(l1 > 0.0f) || !(l1 <= 3.4028234e38f) || !(gsc <= 3.4028234e38f)) return false;
    float srt[N];
    float sumf = 0.0f;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float av = __fmul_rn(fabsf(raw_value<N, BF16>(raw, i)), gsc);
        const float t = __fadd_rd(av, kMagic);
        const float f = __fsub_rn(t, kMagic);  // floor(av), exact
        srt[i] = __fsub_rn(av, f);
        sumf = __fadd_rn(sumf, f);             // small integers: exact
    }
    const int d = K - static_cast<int>(sumf);
    if (d < 0 || d > N) return false;  // cannot happen for finite input; keeps the table reads in range
    sort_desc<N>(srt);
    const float v = d > 0 ? pick<N>(srt, d - 1) : 2.0f;  // 2 is above every residual
    // The residuals are computed again rather than kept: N more registers through the sort
    // cost more than the arithmetic.  (The empty asm hides from the compiler that gsc2 == gsc
    // and, by naming v, keeps this second pass from being scheduled into the sort.)
    float gsc2 = gsc;
    asm volatile("" : "+f"(gsc2) : "f"(v));
    float cnt = 0.0f;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float xi = raw_value<N, BF16>(raw, i);
        const float av = __fmul_rn(fabsf(xi), gsc2);
        const float t = __fadd_rd(av, kMagic);
        const float e = __fsub_rn(av, __fsub_rn(t, kMagic));
        const float one = e >= v ? 1.0f : 0.0f;
        mag[i] = with_sign_of(__fadd_rn(t, one), xi);
        cnt = __fadd_rn(cnt, one);
    }
    int excess = static_cast<int>(cnt) - d;
    if (excess > 0) {
        // Residuals equal to v straddle the cut: of the elements equal to v the ones with the
        // highest indices give their pulse back (lowest index first among equals).
        float gsc3 = gsc;
        asm volatile("" : "+f"(gsc3) : "r"(excess));
#pragma unroll
        for (int i = N - 1; i >= 0; --i) {
            const float av = __fmul_rn(fabsf(raw_value<N, BF16>(raw, i)), gsc3);
            const float t = __fadd_rd(av, kMagic);
            const float e = __fsub_rn(av, __fsub_rn(t, kMagic));
            const bool drop = (e == v) && (excess > 0);
            excess -= drop ? 1 : 0;
            mag[i] = __int_as_float(__float_as_int(mag[i]) - (drop ? 1 : 0));  // |y_i| sits in the low bits
        }
    }
    return true;
}

// Algorithm 2 with the cumulative table of App. C.2.  With V(n,k) = sum_{j<=k} N(n,j) the
// contribution of y_i (n = N-1-i dimensions after it, k pulses before it, k' = k - |y_i|
// after it) is
//     U(n,k) - 2 V(n,k')      for y_i > 0        U(n,k) = V(n,k) + V(n,k-1)
//     U(n,k) - U(n,k')        for y_i <= 0       (zero when y_i = 0, as k' = k)
// so every position costs two table reads, one add and one subtract, whatever |y_i| is.
// All arithmetic is modulo 2^(32 W); the total is the code, which is below 2^(32 W).
//   tabU, tab2V   shared addresses of the two tables, rows of `rowbytes` bytes, entry
//                 (i, col + 1) at i * rowbytes + (col + 1) * EB
//   mag[i]        2^23 + |y_i| as float bits, sign bit = sign of y_i (also set for "-0").
//                 As a signed integer it is <= the bits of 2^23 exactly when y_i <= 0, and
//                 times EB (a multiple of 4) the sign bit drops out of the 32-bit product.
template <int N, int W, int EB>
__device__ __forceinline__ mp<W> enumerate_uv(const float (&mag)[N], int K, uint32_t tabU, uint32_t tab2V,
                                              int rowbytes) {
    mp<W> c;
    mp_zero(c);
    // kb = byte offset of column k in a row: (k + 1) * EB.  |y_i| * EB is taken from the float
    // bits of mag[i], whose constant part is folded into `fold`.
    uint32_t kb = (K + 1) * EB;
    const uint32_t fold = static_cast<uint32_t>(kMagicBits) * EB;  // wraps; only differences are used
    uint32_t rowU = tabU;
    const uint32_t delta = tab2V - tabU;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const int mbits = __float_as_int(mag[i]);
        const uint32_t kb2 = kb - (static_cast<uint32_t>(mbits) * EB - fold);
        const bool nonpos = mbits <= kMagicBits;  // y_i <= 0
        const mp<W> u = load_entry<W>(rowU + kb);
        const mp<W> s = load_entry<W>(rowU + kb2 + (nonpos ? 0u : delta));
        mp_add<W>(c, u);
        mp<W> d;
        mp_sub_borrow<W>(d, c, s);
        c = d;
        kb = kb2;
        rowU += rowbytes;
    }
    return c;
}

// The same sum from the single table V (for tables too large to stage twice):
//     V(n,k) + V(n,k-1) - V(n,k') - V(n,k' - [y_i <= 0]).
template <int N, int W, int EB>
__device__ __forceinline__ mp<W> enumerate_v(const float (&mag)[N], int K, uint32_t tabV, int rowbytes) {
    mp<W> c;
    mp_zero(c);
    uint32_t kb = (K + 1) * EB;
    const uint32_t fold = static_cast<uint32_t>(kMagicBits) * EB;
    uint32_t row = tabV;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const int mbits = __float_as_int(mag[i]);
        const uint32_t kb2 = kb - (static_cast<uint32_t>(mbits) * EB - fold);
        const bool nonpos = mbits <= kMagicBits;
        mp_add<W>(c, load_entry<W>(row + kb));
        mp_add<W>(c, load_entry<W>(row + kb - EB));
        mp<W> d;
        mp_sub_borrow<W>(d, c, load_entry<W>(row + kb2));
        mp_sub_borrow<W>(c, d, load_entry<W>(row + kb2 - (nonpos ? static_cast<uint32_t>(EB) : 0u)));
        kb = kb2;
        row += rowbytes;
    }
    return c;
}

// Algorithm 2 as the walk of pvq_walk.cuh run forwards, on the decoder's table: from
// (0, K), a pulse at the current position adds t (its first) or 2t (a further one) and
// goes left, the end of a position adds t when y_i < 0 and goes down; t = N(N-1-i, col).
// N + K steps of the same instructions for every thread.  Used by the fused kernel when
// the cumulative tables do not fit in shared memory beside the decoder's.  y: the thread's
// slots holding the signed point (one spare slot is read past the end).
template <int N, int W, int EB, typename YT>
__device__ __forceinline__ mp<W> enumerate_walk(const YT* y, uint32_t tab0, int rowlen, int K) {
    mp<W> c;
    mp_zero(c);
    const int D = (rowlen + 1) * EB;
    uint32_t p = tab0 + K * EB;
    int yi = y[0];
    int rem = abs(yi);
    int v = 0;
    const int S = N + K;
#pragma unroll 2
    for (int s = 0; s < S; ++s) {
        const mp<W> t = load_entry<W>(p);
        const bool more = rem > 0;
        const bool add1 = more || (yi < 0);
        const bool add2 = more && v > 0;
        mp<W> a1, a2;
#pragma unroll
        for (int w = 0; w < W; ++w) {
            a1.w[w] = add1 ? t.w[w] : 0u;
            a2.w[w] = add2 ? t.w[w] : 0u;
        }
        mp_add<W>(c, a1);
        mp_add<W>(c, a2);
        if (more) {
            rem -= 1;
            v += 1;
        } else {
            ++y;
            yi = *y;
            rem = abs(yi);
            v = 0;
            p += D;
        }
        p -= EB;
    }
    return c;
}

// The N values of one group as they sit in memory, fetched with 16-byte loads.
template <int N, bool BF16>
__device__ __forceinline__ void load_raw(const void* base, size_t elem_off, uint32_t (&r)[BF16 ? N / 2 : N]) {
    constexpr int RW = BF16 ? N / 2 : N;
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(base) + elem_off * (BF16 ? 2 : 4));
#pragma unroll
    for (int v = 0; v < RW / 4; ++v) {
        const uint4 q = p[v];
        r[4 * v] = q.x;
        r[4 * v + 1] = q.y;
        r[4 * v + 2] = q.z;
        r[4 * v + 3] = q.w;
    }
}

// Launch-time geometry of the encode kernels' shared memory (bytes from the start).
struct EncodeSmem {
    uint32_t enc_bytes;   // staged encoder table(s)
    uint32_t walk_bytes;  // fused: staged walk tables
    uint32_t ss_off, edges_off, levels_off, idx_off, wbuf_off;
    int ss_floats;        // per buffer (there are two)
    int idx_words;        // per buffer (there are two)
    int enum_mode;        // 2: U and 2V staged, 1: V only, 0: none (fused: the walk table serves)
    int walk_phases;
    uint32_t signs_off;   // rotation: rot_block floats
    uint32_t xbuf_off;    // rotation across more than a warp: threads * N floats
};

// Random-sign Hadamard rotation of a row tile held one group per thread (Sec. 2.3, Sec. 3.3
// Step 1): x <- (x * s) H_B / sqrt(B) on every block of B = N * T consecutive columns.  The
// Sylvester butterflies (a, b) -> (a + b, a - b) run with strides 1, 2, 4, ...: strides below
// N inside the thread, strides N .. 16 N between threads of a warp by shuffle (T divides G,
// so thread t and its partner t ^ d hold groups of the same block), larger ones through
// shared memory.  Every sum is one fp32 addition, so the result does not depend on which of
// these three ways a stage takes.
// s_signbits: the signs of a block packed N to a word (bit i of word j set: column j*N + i is
// negated; for N = 64 two words per group).
template <int N>
__device__ __forceinline__ void rotate_tile(float (&x)[N], const uint32_t* s_signbits, int block, float scale,
                                            int g, float* xbuf, int tid, int nthreads) {
    const int T0 = block / N;
    const uint32_t* sb = s_signbits + (g & (T0 - 1)) * ((N + 31) / 32);
#pragma unroll
    for (int i = 0; i < N; ++i)  // multiplying by -1 flips the sign bit
        x[i] = __uint_as_float(__float_as_uint(x[i]) ^ ((sb[i / 32] >> (i % 32)) << 31));
#pragma unroll
    for (int h = 1; h < N; h <<= 1) {
#pragma unroll
        for (int j = 0; j < N; ++j) {
            if ((j & h) == 0) {
                const float a = x[j], b2 = x[j + h];
                x[j] = __fadd_rn(a, b2);
                x[j + h] = __fsub_rn(a, b2);
            }
        }
    }
    const int T = block / N;  // threads per rotation block
    // a + b on the thread that holds a, a - b on the one that holds b: other + sgn * own with
    // sgn = +-1 (the product is exact, so this is the one rounding of the sum or difference)
    for (int d = 1; d < T && d < 32; d <<= 1) {
        const float sgn = (tid & d) != 0 ? -1.0f : 1.0f;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const float other = __shfl_xor_sync(kFull, x[i], d);
            x[i] = __fmaf_rn(x[i], sgn, other);
        }
    }
    for (int d = 32; d < T; d <<= 1) {
        __syncthreads();
#pragma unroll
        for (int i = 0; i < N; ++i) xbuf[i * nthreads + tid] = x[i];
        __syncthreads();
        const float sgn = (tid & d) != 0 ? -1.0f : 1.0f;
#pragma unroll
        for (int i = 0; i < N; ++i) x[i] = __fmaf_rn(x[i], sgn, xbuf[i * nthreads + (tid ^ d)]);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) x[i] = __fmul_rn(x[i], scale);
}


// Where a thread works in a tile.
struct TileLoc {
    int mi;          // matrix
    int G, rpt, gp;  // groups per row, rows per tile, G rounded up to a power of two
    int rl, g;       // row within the tile, group within the row
    long long row0;  // first row of the tile
    bool active;     // this thread has a group
};

__device__ __forceinline__ TileLoc locate(const BatchArgs& a, unsigned tile) {
    TileLoc t;
    t.mi = find_matrix(a, tile);
    const MatrixArgs& m = a.m[t.mi];
    t.G = m.G;
    t.rpt = m.rows_per_tile;
    t.gp = 1;
    while (t.gp < t.G) t.gp <<= 1;
    t.rl = threadIdx.x / t.G;
    t.g = threadIdx.x - t.rl * t.G;
    t.row0 = static_cast<long long>(tile - m.tile_begin) * t.rpt;
    t.active = t.rl < t.rpt && t.row0 + t.rl < m.rows;
    return t;
}

// Shared memory: [encoder tables][walk tables (fused)][2 x ss per thread slot, padded rows]
//                [edges][levels (fused)][2 x scale-index words][per-warp slots (fused)]
// The two ss / scale-index buffers alternate between consecutive tiles, and a tile's index
// words are written out behind the next tile's first barrier, which leaves two block-wide
// barriers per tile; the input of the next tile is
// requested as soon as the registers that held this tile's input are free.
//
// ROT: the tile is first rotated (rotate_tile); the kernel then works on the rotated fp32
// values, whatever type the input has.
// LS: the least-squares amplitude of Step 4 (a kernel of its own: its extra live values would
// otherwise cost the common path registers).
template <int N, int W, bool FUSED, typename YT, bool BF16, bool ROT, bool LS>
__global__ void __launch_bounds__(512) encode_kernel(const __grid_constant__ BatchArgs a,
                                                      const __grid_constant__ EncodeSmem sm) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TW = W <= 2 ? W : (W <= 4 ? 4 : 6);
    constexpr int EB = TW * 4;
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    constexpr int RW = BF16 ? N / 2 : N;      // words of a group as loaded
    constexpr bool WBF16 = BF16 && !ROT;       // the form the kernel works on: packed bf16, or fp32
    constexpr int WW = WBF16 ? N / 2 : N;
    const int K = a.K;
    const int b = a.scale_bits;
    const int nedges = b <= 8 ? (1 << b) - 1 : 0;  // 16 bits: the amplitude itself, no codebook
    const TableLayout L = table_layout(N, K, W);
    uint32_t* s_signs = reinterpret_cast<uint32_t*>(smem + sm.signs_off);
    float* s_xbuf = reinterpret_cast<float*>(smem + sm.xbuf_off);
    float rot_scale = 1.0f;
    if constexpr (ROT) {
        constexpr int WPG = (N + 31) / 32;  // sign words per group
        for (int j = threadIdx.x; j < a.rot_block / N * WPG; j += blockDim.x) {
            uint32_t bits = 0;
            const int col = j * (N / WPG);
            for (int i = 0; i < N / WPG; ++i) bits |= (a.rot_signs[col + i] < 0.0f ? 1u : 0u) << i;
            s_signs[j] = bits;
        }
        rot_scale = static_cast<float>(1.0 / sqrt(static_cast<double>(a.rot_block)));
    }
    float* s_ss2 = reinterpret_cast<float*>(smem + sm.ss_off);
    float* s_edges = reinterpret_cast<float*>(smem + sm.edges_off);
    float* s_levels = reinterpret_cast<float*>(smem + sm.levels_off);
    uint32_t* s_idx2 = reinterpret_cast<uint32_t*>(smem + sm.idx_off);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;

    // stage the tables with bulk copies; they land while the first tile's input is requested
    __shared__ uint64_t stage_bar;
    const BulkStage stage = bulk_stage_begin(&stage_bar);
    if (threadIdx.x == 0) {
        const uint8_t* blob = reinterpret_cast<const uint8_t*>(a.table);
        bulk_stage_expect(stage, sm.enc_bytes + (FUSED ? walk_tables_stage_bytes(L, sm.walk_phases) : 0u));
        if (sm.enc_bytes)
            bulk_stage_copy(stage, smem, blob + (sm.enum_mode == 2 ? L.enc_off[0] : L.enc_off[2]), sm.enc_bytes);
        if constexpr (FUSED) walk_tables_stage(stage, smem + sm.enc_bytes, a.table, L, sm.walk_phases);
    }
    for (int i = threadIdx.x; i < 2 * sm.idx_words; i += blockDim.x) s_idx2[i] = 0u;
    const uint32_t tabA = shared_addr(smem);
    const uint32_t tabB = tabA + ((L.enc_bytes + 127u) & ~127u);  // 2V, when two tables are staged
    const int rowbytes = (K + 2) * EB;
    WalkTables wt;
    YT* yslots = nullptr;
    if constexpr (FUSED) {
        wt = walk_tables(L, tabA + sm.enc_bytes, sm.walk_phases, a);
        yslots = reinterpret_cast<YT*>(smem + sm.wbuf_off + threadIdx.x * YS);
    }
    const float* cur_edges = nullptr;

    unsigned tile = blockIdx.x;
    if (tile >= a.total_tiles) return;
    TileLoc loc = locate(a, tile);
    uint32_t pre[RW];  // the group as loaded; filled one tile ahead
#pragma unroll
    for (int i = 0; i < RW; ++i) pre[i] = 0u;
    if (loc.active) {
        const MatrixArgs& m0 = a.m[loc.mi];
        load_raw<N, BF16>(m0.x, static_cast<size_t>(loc.row0 + loc.rl) * m0.ld + static_cast<size_t>(loc.g) * N, pre);
    }
    if (!bulk_stage_wait(stage)) {  // the tables never arrived: report and leave rather than spin
        if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_STAGING_TIMEOUT);
        return;
    }
    __syncthreads();                      // index words cleared
#ifdef PVQ_DEBUG
    debug_begin(tabA, tabA + sm.enc_bytes + (FUSED ? sm.walk_bytes : 0u), tabA + sm.wbuf_off, YS,
                N * static_cast<uint32_t>(sizeof(YT)), a.debug_status);
#endif
    struct {
        bool valid;
        int mi, rpt;
        long long row0;
    } prev = {false, 0, 0, 0};  // the tile whose index words are still to be written out

    for (int buf = 0;; buf ^= 1) {
        const MatrixArgs& m = a.m[loc.mi];
        const int G = loc.G, rpt = loc.rpt, gp = loc.gp, rl = loc.rl, g = loc.g;
        const long long row0 = loc.row0;
        const long long row = row0 + rl;
        const bool active = loc.active;
        const int idx_words = m.sstride >> 2;
        float* s_ss = s_ss2 + buf * sm.ss_floats;
        uint32_t* s_idx = s_idx2 + buf * sm.idx_words;

        uint32_t raw[WW];  // the group the kernel works on
        if constexpr (ROT) {
            float x[N];
#pragma unroll
            for (int i = 0; i < N; ++i) x[i] = raw_value<N, BF16>(pre, i);
            rotate_tile<N>(x, s_signs, a.rot_block, rot_scale, g, s_xbuf, threadIdx.x, blockDim.x);
#pragma unroll
            for (int i = 0; i < N; ++i) raw[i] = __float_as_uint(x[i]);
        } else {
#pragma unroll
            for (int i = 0; i < WW; ++i) raw[i] = pre[i];
        }

        // group norms; an inactive thread holds zeros
        float l1, ss;
        {
            float t[N];
#pragma unroll
            for (int i = 0; i < N; ++i) t[i] = fabsf(raw_value<N, WBF16>(raw, i));
            l1 = tree_sum<N>(t);
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const float xi = raw_value<N, WBF16>(raw, i);
                t[i] = __fmul_rn(xi, xi);
            }
            ss = tree_sum<N>(t);
        }
        if (active && PVQ_DEBUG_INDEX(rl * gp + g, sm.ss_floats, PVQ_DEBUG_SHARED_INDEX)) {
            s_ss[rl * gp + g] = ss;
            if (g < gp - G) s_ss[rl * gp + G + g] = 0.0f;  // zero padding of the row's tree
        }
        __syncthreads();  // (1) group energies of this tile are in s_ss; nobody is in the previous tile

        if (nedges != 0 && cur_edges != m.edges) {  // uniform across the block
            for (int i = threadIdx.x; i < nedges; i += blockDim.x) s_edges[i] = m.edges[i];
            if constexpr (FUSED)
                for (int i = threadIdx.x; i <= nedges; i += blockDim.x) s_levels[i] = m.levels[i];
            cur_edges = m.edges;
        }
        if constexpr (!FUSED) {
            // The previous tile's index words (the other buffer) are complete: every thread added
            // its bits before it came to barrier (1).  Write them out and clear them for the next tile.
            uint32_t* other = s_idx2 + (buf ^ 1) * sm.idx_words;
            if (prev.valid) {
                const MatrixArgs& pm = a.m[prev.mi];
                const int piw = pm.sstride >> 2;
                for (int i = threadIdx.x; i < prev.rpt * piw; i += blockDim.x) {
                    const int r2 = i / piw;
                    const long long row2 = prev.row0 + r2;
                    if (row2 < pm.rows)
                        reinterpret_cast<uint32_t*>(pm.scale_idx + static_cast<size_t>(row2) * pm.sstride)[i - r2 * piw] =
                            other[i];
                }
            }
            for (int i = threadIdx.x; i < sm.idx_words; i += blockDim.x) other[i] = 0u;
        }
        // row energy: balanced tree over the (zero padded) groups of each row, one warp per row
        for (int r = warp; r < rpt; r += nwarps) {
            float* rs = s_ss + r * gp;
            for (int s = 1; s < gp; s <<= 1) {
                for (int j = lane * 2 * s; j < gp; j += 64 * s) rs[j] = __fadd_rn(rs[j], rs[j + s]);
                __syncwarp();
            }
        }

        // direction; nothing here needs the row norm.  mag[i] carries the sign of x_i.
        float mag[N];
        const bool has_dir = quantize_direction<N, WBF16>(raw, l1, K, mag);
        if (!has_dir) {  // (K, 0, ..., 0)
#pragma unroll
            for (int i = 0; i < N; ++i) mag[i] = kMagic;
            mag[0] = __int_as_float(kMagicBits + K);
        }

        // Step 4 as least squares: the amplitude is the projection of x on the chosen direction,
        // a = (sum |y_i| |x_i|) / sqrt(sum y_i^2), the sum of the rounded products by the fixed tree
        float ls_amp = 0.0f;
        if constexpr (LS) {
            float t[N];
            float ssy = 0.0f;
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const float mf = __fsub_rn(fabsf(mag[i]), kMagic);  // |y_i|, exact
                ssy = __fadd_rn(ssy, __fmul_rn(mf, mf));            // integers below 2^24: exact
                t[i] = __fmul_rn(mf, fabsf(raw_value<N, WBF16>(raw, i)));
            }
            ls_amp = __fdiv_rn(tree_sum<N>(t), __fsqrt_rn(ssy));
        }

        // the loaded group is dead: ask for the next tile's input now, it arrives while the index is computed
        const unsigned next_tile = tile + gridDim.x;
        const bool have_next = next_tile < a.total_tiles;
        TileLoc nloc = loc;
        if (have_next) {
            nloc = locate(a, next_tile);
            if (nloc.active) {
                const MatrixArgs& mn = a.m[nloc.mi];
                load_raw<N, BF16>(mn.x, static_cast<size_t>(nloc.row0 + nloc.rl) * mn.ld + static_cast<size_t>(nloc.g) * N,
                                  pre);
            } else {
#pragma unroll
                for (int i = 0; i < RW; ++i) pre[i] = 0u;
            }
        }

        mp<W> c;
        if (sm.enum_mode == 2) {
            c = enumerate_uv<N, W, EB>(mag, K, tabA, tabB, rowbytes);
        } else if (sm.enum_mode == 1) {
            c = enumerate_v<N, W, EB>(mag, K, tabA, rowbytes);
        } else {
            if constexpr (FUSED) {
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    const int mb = __float_as_int(mag[i]);
                    const int mi2 = (mb & 0x7fffffff) - kMagicBits;
                    yslots[i] = static_cast<YT>(mb < 0 ? -mi2 : mi2);
                }
                c = enumerate_walk<N, W, EB, YT>(yslots, wt.tab0, wt.rowlen, K);
            } else {
                mp_zero(c);
            }
        }

        __syncthreads();  // (2) row energies are in s_ss[r * gp]
        float rnorm = 0.0f;
        int q = 0;
        if (active) {
            const float ss_row = s_ss[rl * gp];
            rnorm = __fsqrt_rn(ss_row);
            if (b == 16) {  // the amplitude itself, as binary16
                const float amp16 = LS ? ls_amp : __fsqrt_rn(ss);
                q = __half_as_ushort(__float2half_rn(amp16));
            } else {
                // Step 5: q = floor(CDF(u) 2^b) as the number of bin edges <= u
                const float amp2 = LS ? __fmul_rn(ls_amp, ls_amp) : ss;
                const float u = ss_row > 0.0f ? __fdiv_rn(amp2, ss_row) : 0.0f;
                for (int step = 1 << (b - 1); step >= 1; step >>= 1)
                    if (s_edges[q + step - 1] <= u) q += step;
            }
        }

        if constexpr (!FUSED) {
            if (active) {
                if (g == 0) m.row_norm[row] = rnorm;
                uint32_t* cp = m.codes + (static_cast<size_t>(row) * G + g) * W;
                if (PVQ_DEBUG_INDEX(row * G + g, m.rows * G, PVQ_DEBUG_GLOBAL_STORE)) {
#pragma unroll
                    for (int w = 0; w < W; ++w) cp[w] = c.w[w];
                }
                const unsigned bit = static_cast<unsigned>(g) * b;
                const unsigned sh = bit & 31u;
                atomicOr(&s_idx[rl * idx_words + (bit >> 5)], static_cast<uint32_t>(q) << sh);
                if (sh + b > 32u)
                    atomicOr(&s_idx[rl * idx_words + (bit >> 5) + 1], static_cast<uint32_t>(q) >> (32u - sh));
            }
            prev.valid = true;  // written out after the next tile's first barrier, or after the loop
            prev.mi = loc.mi;
            prev.rpt = rpt;
            prev.row0 = row0;
        } else {
            // decode the code just made (every thread of the warp walks, in lockstep)
            const float amp = !active ? 0.0f
                              : b == 16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(q)))
                                        : __fmul_rn(rnorm, s_levels[q]);
            if (!active) mp_zero(c);
            walk_code<N, W, YT>(c, wt, K, yslots);
            if (active) emit_group<N, YT>(m, yslots, amp, static_cast<unsigned>(row), static_cast<unsigned>(g));
        }

        if (!have_next) {
            if constexpr (!FUSED) {
                __syncthreads();  // the last tile's index words are complete
                for (int i = threadIdx.x; i < rpt * idx_words; i += blockDim.x) {
                    const int r2 = i / idx_words;
                    const long long row2 = row0 + r2;
                    if (row2 < m.rows)
                        reinterpret_cast<uint32_t*>(m.scale_idx + static_cast<size_t>(row2) * m.sstride)[i - r2 * idx_words] =
                            s_idx[i];
                }
            }
            break;
        }
        tile = next_tile;
        loc = nloc;
    }
}

template <int N, int W, bool FUSED, typename YT, bool BF16, bool ROT, bool LS = false>
static int launch_encode_t(BatchArgs& a, cudaStream_t stream) {
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    // Block size: a multiple of 32 that wastes the fewest thread slots over the batch.
    int best_threads = 0;
    long long best_cost = -1;
    for (int threads = 128; threads <= 512; threads += 32) {
        long long cost = 0;
        bool ok = true;
        for (int i = 0; i < a.count; ++i) {
            const int G = a.m[i].G;
            if (G > threads) {
                ok = false;
                break;
            }
            const int rpt = threads / G;
            cost += ((a.m[i].rows + rpt - 1) / rpt) * threads;
        }
        if (!ok) continue;
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && threads == 256)) {
            best_cost = cost;
            best_threads = threads;
        }
    }
    if (best_threads == 0) return PVQ_ERR_UNSUPPORTED;  // a row has more groups than a block has threads
    const int threads = best_threads;
    unsigned tiles = 0;
    int max_idx_words = 1;
    for (int i = 0; i < a.count; ++i) {
        MatrixArgs& m = a.m[i];
        m.rows_per_tile = threads / m.G;
        m.tile_begin = tiles;
        tiles += static_cast<unsigned>((m.rows + m.rows_per_tile - 1) / m.rows_per_tile);
        max_idx_words = std::max(max_idx_words, m.rows_per_tile * (m.sstride / 4));
    }
    // s_ss holds rows_per_tile * (G rounded up to a power of two) floats
    int ss_floats = 0;
    for (int i = 0; i < a.count; ++i) {
        int gp = 1;
        while (gp < a.m[i].G) gp <<= 1;
        ss_floats = std::max(ss_floats, a.m[i].rows_per_tile * gp);
    }
    a.total_tiles = tiles;

    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    const int sms = di.sms, smem_max = di.smem_max;

    const TableLayout L = table_layout(N, a.K, W);
    // rotation: the signs, and an exchange buffer when a rotation block spans more than a warp
    const size_t rot_signs_b = ROT ? static_cast<size_t>(a.rot_block) * 4u : 0;
    const size_t rot_xbuf_b = ROT && a.rot_block / N > 32 ? static_cast<size_t>(threads) * N * 4u : 0;
    const size_t small = (2 * static_cast<size_t>(ss_floats) + 256 + (FUSED ? 256 : 0) + 2 * max_idx_words) * 4u + 64u +
                         rot_signs_b + rot_xbuf_b;
    const size_t wbufs = FUSED ? static_cast<size_t>(threads) * YS : 0;
    const size_t enc_one = (L.enc_bytes + 127u) & ~size_t(127);
    EncodeSmem sm;
    sm.walk_bytes = 0;
    sm.walk_phases = 0;
    size_t walk = 0;
    const size_t cap = static_cast<size_t>(smem_max);
    if (FUSED) {  // the widest walk table has to fit; then as many encoder tables as still do
        sm.enum_mode = -1;
        for (int mode = 2; mode >= 0 && sm.enum_mode < 0; --mode) {
            const size_t fixed = mode * enc_one + small + wbufs;
            if (fixed >= cap) continue;
            const int ph = walk_phases_that_fit(L, cap - fixed);
            if (ph == 0) continue;
            sm.enum_mode = mode;
            sm.walk_phases = ph;
        }
        if (sm.enum_mode < 0) return PVQ_ERR_UNSUPPORTED;
        walk = (walk_tables_bytes(L, sm.walk_phases) + 15u) & ~size_t(15);
        sm.walk_bytes = static_cast<uint32_t>(walk);
    } else {
        sm.enum_mode = 2 * enc_one + small <= cap ? 2 : 1;
        if (sm.enum_mode == 1 && enc_one + small > cap) return PVQ_ERR_UNSUPPORTED;
    }
    sm.enc_bytes = static_cast<uint32_t>(sm.enum_mode * enc_one);
    sm.ss_floats = ss_floats;
    sm.idx_words = max_idx_words;
    sm.ss_off = static_cast<uint32_t>(sm.enc_bytes + walk);
    sm.edges_off = sm.ss_off + 2u * ss_floats * 4u;
    sm.levels_off = sm.edges_off + 256u * 4u;
    sm.idx_off = sm.levels_off + (FUSED ? 256u * 4u : 0u);
    sm.signs_off = (sm.idx_off + 2u * max_idx_words * 4u + 15u) & ~15u;
    sm.xbuf_off = sm.signs_off + static_cast<uint32_t>(rot_signs_b);
    sm.wbuf_off = sm.xbuf_off + static_cast<uint32_t>(rot_xbuf_b);
    const size_t smem = sm.wbuf_off + wbufs;
    if (smem > static_cast<size_t>(smem_max)) return PVQ_ERR_UNSUPPORTED;

    auto kern = encode_kernel<N, W, FUSED, YT, BF16, ROT, LS>;
    int per_sm = 0;
    if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), threads, smem, &per_sm)) != PVQ_OK) return st;
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned grid = std::min<unsigned>(tiles, static_cast<unsigned>(sms * per_sm));
    kern<<<grid, threads, smem, stream>>>(a, sm);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int W, bool BF16>
static int launch_encode_nwb(BatchArgs& a, bool fused, cudaStream_t s) {
    if (a.amp_mode == 1) {  // least squares: the plain encoder only
        if (fused || a.rot_block != 0) return PVQ_ERR_UNSUPPORTED;
        return launch_encode_t<N, W, false, int8_t, BF16, false, true>(a, s);
    }
    if (a.rot_block != 0) {  // rotating kernels are built for byte-sized slots only (K <= 127)
        if (!fused) return launch_encode_t<N, W, false, int8_t, BF16, true>(a, s);
        if (a.K <= 127) return launch_encode_t<N, W, true, int8_t, BF16, true>(a, s);
        return PVQ_ERR_UNSUPPORTED;
    }
    if (!fused) return launch_encode_t<N, W, false, int8_t, BF16, false>(a, s);
    if (a.K <= 127) return launch_encode_t<N, W, true, int8_t, BF16, false>(a, s);
    return launch_encode_t<N, W, true, int16_t, BF16, false>(a, s);
}

template <int N, int W>
static int launch_encode_nw(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return dtype == PVQ_DTYPE_BF16 ? launch_encode_nwb<N, W, true>(a, fused, s)
                                   : launch_encode_nwb<N, W, false>(a, fused, s);
}

}  // namespace pvq
