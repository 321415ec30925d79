// The encode kernel for the plain case (no rotation, amplitude = ||x_g||, codes written out):
// Sec. 3.3 Steps 3, 5, 7 and Algorithms 1, 2 with one thread per group.
//
// What differs from the general kernel of pvq_encode_impl.cuh:
//   - the Fischer index is summed from the telescoped tables (`cenc` of TableLayout): one
//     table read and one multi-word add per position instead of two reads, an add and a
//     subtract.  The tables sit in shared memory with a row length fixed at compile time
//     (CROW entries), so that the row of a position is an immediate offset;
//   - the positions are visited last to first.  The term of position i depends on the pulses
//     before it, k_i, and after it, k_{i+1} = k_i - |y_i|; counted from the back, k_{i+1} is
//     the running sum of the |y_j| already visited, and "of the residuals equal to the cut, the
//     highest indices give their pulse back" becomes a countdown that needs nothing but the
//     number of pulses to take back;
//   - a group is kept as its scaled values a_i = x_i K / l1 (the sign of x_i rides along);
//     floor and residual are taken from them again where needed, on the fp32 pipe, which is
//     idle next to the integer pipe the sorting network and the index arithmetic keep busy;
//   - a row may be longer than a thread block: the block takes it in chunks, keeps the group
//     energies of the row in shared memory and hands out the amplitude indices afterwards;
//   - one block-wide barrier per tile: group energies, bin edges and index words alternate
//     between two buffers, every warp sums the energies of its own rows, and a tile's index
//     words are written out behind the next tile's barrier.
#pragma once
#include <cuda_fp16.h>

#include <algorithm>

#include "pvq_encode_impl.cuh"

namespace pvq {

constexpr int kFastThreadsMax = 256;
constexpr int kFastMaxGroups = 4096;  // groups per row: 128 energies per lane in the row tree

struct FastSmem {
    uint32_t tab_bytes;             // the two telescoped tables, rows of CROW entries
    uint32_t ss_off;                // 2 x ss_floats: group energies of a tile
    uint32_t edges_off, idx_off;    // 2 x 256 floats; 2 x idx_words
    int ss_floats, idx_words;
    // round trip: the decoder's walk tables, 2 x 256 levels, one output slot per thread
    uint32_t walk_off, walk_bytes, levels_off, wbuf_off;
    int walk_phases;
};

// 1.0f where the comparison holds, else 0.0f (one instruction; the flags are then summed or
// multiplied on the fp32 pipe)
__device__ __forceinline__ float flag_ge(float a, float b) {
    float r;
    asm("set.ge.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float flag_eq(float a, float b) {
    float r;
    asm("set.eq.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float flag_gt(float a, float b) {
    float r;
    asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// The N values of one group as they sit in memory, by 16-byte loads that stay where they are
// written (a plain load may be moved down to its first use, which for a request made a tile
// ahead would defeat its purpose).
template <int N, bool BF16>
__device__ __forceinline__ void load_raw_here(const void* base, size_t elem_off, uint32_t (&r)[BF16 ? N / 2 : N]) {
    constexpr int RW = BF16 ? N / 2 : N;
    const uint8_t* p = static_cast<const uint8_t*>(base) + elem_off * (BF16 ? 2 : 4);
#pragma unroll
    for (int v = 0; v < RW / 4; ++v)
        asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(r[4 * v]), "=r"(r[4 * v + 1]), "=r"(r[4 * v + 2]), "=r"(r[4 * v + 3])
                     : "l"(p + 16 * v));
}

// Marks a value as changed without emitting an instruction.  Floor and residual are computed
// from the scaled values three times (for the sort, for the count, for the index sum) rather
// than kept: 64 more live registers through the sorting network would cost far more.  The
// marker keeps the compiler from merging the three computations back into one.
__device__ __forceinline__ void touch(float& x) { asm volatile("" : "+f"(x)); }

// What direction_begin leaves for the later steps.
template <int N>
struct Scaled {
    float avs[N];   // x_i K / l1: magnitude a_i, sign of x_i
    int d;          // pulses the floors leave over
    bool has_dir;
};

// a_i = |x_i| (K / l1) and d = K - sum floor(a_i)  (Sec. 2.5: scale to the l1 ball of radius K)
template <int N, bool BF16>
__device__ __forceinline__ void direction_begin(const uint32_t (&raw)[BF16 ? N / 2 : N], float l1, int K, Scaled<N>& s) {
    const float gsc = __fdiv_rn(static_cast<float>(K), l1);
    // no direction: l1 zero or not finite, or a scale that overflows
    s.has_dir = (l1 > 0.0f) && (l1 <= 3.4028234e38f) && (gsc <= 3.4028234e38f);
    int sumbits = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        s.avs[i] = __fmul_rn(raw_value<N, BF16>(raw, i), gsc);
        const float t = __fadd_rd(fabsf(s.avs[i]), kMagic);  // 2^23 + floor(a_i)
        sumbits += __float_as_int(t) - kMagicBits;           // floor(a_i) sits in the low mantissa bits
    }
    s.d = K - sumbits;
    // 0 <= d <= N for finite input (sum floor(a_i) <= sum a_i < K + 1); anything else is treated
    // as "no direction", which keeps every table read in range
    s.has_dir = s.has_dir && s.d >= 0 && s.d <= N;
    if (!s.has_dir) {  // the point is (K, 0, ..., 0): nothing below may depend on the values
#pragma unroll
        for (int i = 0; i < N; ++i) s.avs[i] = 0.0f;
    }
}

// One position of the index sum, visited from the back.  `one` is 1.0f when the position gets
// a pulse beyond its floor.  A is the shared address of column k_{i+1} of row 0 of cenc[0].
template <int N, int W, int TW, int CROW, int I>
__device__ __forceinline__ void index_step(float avs, float t, float one, uint32_t& A, mp<W>& c) {
    constexpr int EB = TW * 4;
    // 2^23 + |y_i| moved to where one unit in the last place is 1/EB: the low bits of the
    // float are then |y_i| * EB, the bytes to move along the row
    constexpr int SH = 2;  // the rows are stored word plane by word plane: an entry's word 0 is 4 bytes from the next entry's
    constexpr uint32_t kBaseBits = static_cast<uint32_t>(127 + 23 - SH) << 23;   // bits of 2^(23-SH)
    const float tq = __fadd_rn(t, one);                                          // 2^23 + |y_i|
    const float shifted = __fsub_rn(tq, kMagic - static_cast<float>(1 << (23 - SH)));  // 2^(23-SH) + |y_i|, exact
    // y_i > 0 reads cenc[1], N rows and the skew further on.  "|y_i| > 0 and the sign bit of x_i clear" is
    // "|y_i| a_i > 0" with the sign of x_i on a_i: a position with a_i = 0 never gets a pulse
    // (d = sum e_i + (K - sum a_i), the last term far below 1 in magnitude and every e_i below 1,
    // so d does not exceed the number of non-zero residuals), and the point (K, 0, ..., 0) of a
    // group without direction comes in with a_0 = 1.  The choice is made on the fp32 pipe: the
    // flag (1.0f or 0.0f) times the distance between the tables, and its sum with the address,
    // are exact on integers this small held as subnormal floats.
    const float mf = __fsub_rn(tq, kMagic);  // |y_i|
    const float offs = __fmul_rn(flag_gt(__fmul_rn(mf, avs), 0.0f), __int_as_float(N * CROW * EB + static_cast<int>(kCencSkew)));
    const uint32_t addr = __float_as_uint(__fadd_rn(__uint_as_float(A), offs));
    // word w of the entry sits CROW words behind word w - 1 (threads of a warp read
    // neighbouring columns: different banks)
    mp<W> add;
    add.w[0] = load_entry<1, I * CROW * EB>(addr).w[0];
    if constexpr (W > 1) add.w[1] = load_entry<1, I * CROW * EB + CROW * 4>(addr).w[0];
    if constexpr (W > 2) add.w[2] = load_entry<1, I * CROW * EB + 2 * CROW * 4>(addr).w[0];
    if constexpr (W > 3) add.w[3] = load_entry<1, I * CROW * EB + 3 * CROW * 4>(addr).w[0];
    mp_add<W>(c, add);  // modulo 2^(32 W)
    A += __float_as_uint(shifted) - kBaseBits;
}

// Positions I, I-1, ..., 0 of the index sum.
template <int N, int W, int TW, int CROW, int I>
__device__ __forceinline__ void index_steps(Scaled<N>& s, int K, float v, float& excess, uint32_t& A, mp<W>& c) {
    touch(s.avs[I]);
    const float aa = fabsf(s.avs[I]);
    float t = __fadd_rd(aa, kMagic);
    const float e = __fsub_rn(aa, __fsub_rn(t, kMagic));  // exact
    float one = flag_ge(e, v);
    const float drop = fminf(flag_eq(e, v), excess);  // 1 while pulses are left to take back
    excess = __fsub_rn(excess, drop);
    one = __fsub_rn(one, drop);
    float av = s.avs[I];
    if (I == 0 && !s.has_dir) {  // (K, 0, ..., 0)
        t = __int_as_float(kMagicBits + K);
        one = 0.0f;
        av = 1.0f;
    }
    index_step<N, W, TW, CROW, I>(av, t, one, A, c);
    if constexpr (I > 0) index_steps<N, W, TW, CROW, I - 1>(s, K, v, excess, A, c);
}

// The cut of the greedy fix-up: the d largest residuals e_i = a_i - floor(a_i) get one more
// pulse, lowest index first among equals.  v = the d-th largest residual (2 when d = 0: above
// every residual); excess = how many residuals equal to v lie beyond the d-th largest.
template <int N>
__device__ __forceinline__ void direction_cut(const Scaled<N>& s, float& v, float& excess) {
    v = 2.0f;
    excess = 0.0f;
    if (s.has_dir) {
        float srt[N];
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const float aa = fabsf(s.avs[i]);
            srt[i] = __fsub_rn(aa, __fsub_rn(__fadd_rd(aa, kMagic), kMagic));  // exact
        }
        sort_desc<N>(srt);
        if (s.d > 0) v = pick<N>(srt, s.d - 1);
        float cnt = 0.0f;  // how many residuals reach the cut (counted on the sorted copy: the same values)
#pragma unroll
        for (int i = 0; i < N; ++i) cnt = __fadd_rn(cnt, flag_ge(srt[i], v));
        excess = cnt - static_cast<float>(s.d);
    }
}

// The Fischer index (Algorithm 2) of the point the cut defines.
template <int N, int W, int TW, int CROW>
__device__ __forceinline__ mp<W> direction_index(Scaled<N>& s, int K, float v, float excess, uint32_t tab0,
                                                 const mp<W>& start) {
    // A thread may have residuals equal to its cut on both sides of it: coming from the back,
    // the first `excess` of them give their pulse back.  (One loop for all warps: a second,
    // countdown-free copy for warps without such ties cost more in instruction fetch than the
    // four instructions per position it saved.)
    mp<W> c = start;
    uint32_t A = tab0;
    index_steps<N, W, TW, CROW, N - 1>(s, K, v, excess, A, c);
    return c;
}

// Sum of the gp (a power of two, <= 4096) floats at p by the balanced tree over contiguous
// halves, computed by one warp; every lane gets the result.  Lane l takes the gp / 32
// consecutive values that start at l * gp / 32 (zeros beyond gp: adding +0 changes nothing).
__device__ __forceinline__ float warp_tree_sum(const float* p, int gp, int lane) {
    float v = 0.0f;
    if (gp <= 32) {
        v = lane < gp ? p[lane] : 0.0f;
    } else if (gp == 64) {
        const float2 x = reinterpret_cast<const float2*>(p)[lane];
        v = __fadd_rn(x.x, x.y);
    } else if (gp == 128) {
        const float4 x = reinterpret_cast<const float4*>(p)[lane];
        v = __fadd_rn(__fadd_rn(x.x, x.y), __fadd_rn(x.z, x.w));
    } else if (gp == 256) {
        const float4 x = reinterpret_cast<const float4*>(p)[2 * lane], y = reinterpret_cast<const float4*>(p)[2 * lane + 1];
        v = __fadd_rn(__fadd_rn(__fadd_rn(x.x, x.y), __fadd_rn(x.z, x.w)), __fadd_rn(__fadd_rn(y.x, y.y), __fadd_rn(y.z, y.w)));
    } else {
        // 16 Q values per lane, Q = 1, 2, 4 or 8: a tree over each run of 16, then over the runs
        const int Q = gp >> 9;
        float part[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            part[q] = 0.0f;
            if (q < Q) {
                float t[16];
                const float4* src = reinterpret_cast<const float4*>(p + (lane * Q + q) * 16);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 x = src[j];
                    t[4 * j] = x.x, t[4 * j + 1] = x.y, t[4 * j + 2] = x.z, t[4 * j + 3] = x.w;
                }
                part[q] = tree_sum<16>(t);
            }
        }
        v = tree_sum<8>(part);  // the runs beyond Q are zero
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) v = __fadd_rn(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// FUSED: the round trip of pvq_roundtrip.  The code is not stored; once the row energy is known
// the thread walks it back to its point (pvq_walk.cuh) and writes the bf16 values.
template <int N, int W, bool BF16, int CROW, bool FUSED, typename YT>
__global__ void __launch_bounds__(kFastThreadsMax, 2) encode_fast_kernel(const __grid_constant__ BatchArgs a,
                                                                          const __grid_constant__ FastSmem sm) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TW = W <= 2 ? W : 4;
    constexpr int RW = BF16 ? N / 2 : N;
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    const int K = a.K;
    const int b = a.scale_bits;
    const int nedges = b <= 8 ? (1 << b) - 1 : 0;  // 16 bits: the amplitude itself, no codebook
    const TableLayout L = table_layout(N, K, W);
    float* s_ss2 = reinterpret_cast<float*>(smem + sm.ss_off);
    float* s_edges2 = reinterpret_cast<float*>(smem + sm.edges_off);
    uint32_t* s_idx2 = reinterpret_cast<uint32_t*>(smem + sm.idx_off);
    const int tid = threadIdx.x, T = blockDim.x;
    const int lane = tid & 31;

    // the two tables (cenc[0], cenc[1], adjacent in the blob) with one bulk copy; it lands while
    // the first tile's input is requested
    __shared__ uint64_t stage_bar;
    const BulkStage stage = bulk_stage_begin(&stage_bar);
    if (tid == 0) {
        bulk_stage_expect(stage, 2u * L.cenc_bytes + kCencSkew + (FUSED ? walk_tables_stage_bytes(L, sm.walk_phases) : 0u));
        bulk_stage_copy(stage, smem, reinterpret_cast<const uint8_t*>(a.table) + L.cenc_off[0], 2u * L.cenc_bytes + kCencSkew);
        if constexpr (FUSED) walk_tables_stage(stage, smem + sm.walk_off, a.table, L, sm.walk_phases);
    }
    WalkTables wt;
    YT* yslots = nullptr;
    float* s_levels2 = nullptr;
    if constexpr (FUSED) {
        wt = walk_tables(L, shared_addr(smem) + sm.walk_off, sm.walk_phases, a);
        yslots = reinterpret_cast<YT*>(smem + sm.wbuf_off + tid * YS);
        s_levels2 = reinterpret_cast<float*>(smem + sm.levels_off);
    }
    for (int i = tid; i < 2 * sm.idx_words; i += T) s_idx2[i] = 0u;
    const uint32_t tab0 = shared_addr(smem);
    mp<W> start;
#pragma unroll
    for (int w = 0; w < W; ++w) start.w[w] = a.table[L.start_off / 4 + w];
    const float* edges0 = nullptr;  // whose bin edges the two edge buffers hold
    const float* edges1 = nullptr;

    // Where this thread works in the tiles of the current matrix: one group of one of a tile's
    // rows, or (a row longer than the block) one group of every chunk of the tile's single row.
    // Worked out when the matrix changes, not per tile.
    int mi = -1, G = 1, gp = 1, rl = 0, g0 = 0, rpt = 1, chunks = 1, idx_words = 1;
    auto enter_matrix = [&](int i) {
        const MatrixArgs& m = a.m[i];
        mi = i;
        G = m.G;
        rpt = m.rows_per_tile;
        chunks = m.chunks;
        idx_words = m.sstride >> 2;
        gp = 1;
        while (gp < G) gp <<= 1;
        rl = chunks == 1 ? tid / G : 0;
        g0 = chunks == 1 ? tid - rl * G : tid;
    };
    // the group of chunk 0 of `tile` (of the current matrix), or zeros where this thread has none
    auto fetch_first = [&](unsigned tile, uint32_t (&r)[RW]) {
        const MatrixArgs& m = a.m[mi];
        const long long row = static_cast<long long>(tile - m.tile_begin) * rpt + rl;
        if (rl < rpt && row < m.rows && g0 < G) {
            load_raw_here<N, BF16>(m.x, static_cast<size_t>(row) * m.ld + static_cast<size_t>(g0) * N, r);
        } else {
#pragma unroll
            for (int i = 0; i < RW; ++i) r[i] = 0u;
        }
    };
    // index words of a finished tile -> memory; the buffer is cleared for the tile after next
    auto flush_idx = [&](int fmi, unsigned done_tile, uint32_t* s_idx) {
        const MatrixArgs& m = a.m[fmi];
        const int iw = m.sstride >> 2;
        const long long row0 = static_cast<long long>(done_tile - m.tile_begin) * m.rows_per_tile;
        for (int i = tid; i < m.rows_per_tile * iw; i += T) {
            const int r2 = i / iw;
            const long long row2 = row0 + r2;
            if (row2 < m.rows)
                reinterpret_cast<uint32_t*>(m.scale_idx + static_cast<size_t>(row2) * m.sstride)[i - r2 * iw] = s_idx[i];
            s_idx[i] = 0u;
        }
    };

    unsigned tile = blockIdx.x;
    if (tile >= a.total_tiles) return;
    enter_matrix(find_matrix(a, tile));
    uint32_t pre[RW];  // the first chunk's group of the coming tile, requested a tile ahead
    fetch_first(tile, pre);
    if (!bulk_stage_wait(stage)) {  // the tables never arrived: report and leave rather than spin
        if (a.status && tid == 0) atomicOr(a.status, PVQ_STATUS_STAGING_TIMEOUT);
        return;
    }
    __syncthreads();  // index words cleared
#ifdef PVQ_DEBUG
    // tables: the two telescoped ones with the slack behind them, and (round trip) the walk tables
    debug_begin(tab0, tab0 + (FUSED ? sm.walk_off + sm.walk_bytes : sm.tab_bytes), tab0 + sm.wbuf_off, YS,
                N * static_cast<uint32_t>(sizeof(YT)), a.debug_status);
#endif

    int buf = 0, prev_mi = mi;
    for (bool first_tile = true;; buf ^= 1, first_tile = false) {
        const MatrixArgs& m = a.m[mi];
        const long long row0 = static_cast<long long>(tile - m.tile_begin) * rpt;
        const bool row_ok = rl < rpt && row0 + rl < m.rows;
        float* s_ss = s_ss2 + buf * sm.ss_floats;
        float* s_edges = s_edges2 + buf * 256;
        uint32_t* s_idx = s_idx2 + buf * sm.idx_words;
        const unsigned next_tile = tile + gridDim.x;
        const bool have_next = next_tile < a.total_tiles;
        const int cur_mi = mi, cur_G = G, cur_gp = gp, cur_rl = rl, cur_g0 = g0, cur_chunks = chunks, cur_rpt = rpt;
        const int cur_idx_words = idx_words;
        mp<W> kept;  // round trip: this thread's code (one chunk per tile there)
        mp_zero(kept);

        for (int ch = 0; ch < cur_chunks; ++ch) {
            const int g = cur_g0 + ch * T;
            const bool active = row_ok && g < cur_G;
            Scaled<N> sc;
            {
                uint32_t raw[RW];
                if (ch == 0) {
#pragma unroll
                    for (int i = 0; i < RW; ++i) raw[i] = pre[i];
                } else if (active) {
                    load_raw<N, BF16>(m.x, static_cast<size_t>(row0 + cur_rl) * m.ld + static_cast<size_t>(g) * N, raw);
                } else {
#pragma unroll
                    for (int i = 0; i < RW; ++i) raw[i] = 0u;
                }
                float l1, ss;
                float t[N];
#pragma unroll
                for (int i = 0; i < N; ++i) t[i] = fabsf(raw_value<N, BF16>(raw, i));
                l1 = tree_sum<N>(t);
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    const float xi = raw_value<N, BF16>(raw, i);
                    t[i] = __fmul_rn(xi, xi);
                }
                ss = tree_sum<N>(t);
                if (active && PVQ_DEBUG_INDEX(cur_rl * cur_gp + g, sm.ss_floats, PVQ_DEBUG_SHARED_INDEX)) s_ss[cur_rl * cur_gp + g] = ss;
                direction_begin<N, BF16>(raw, l1, K, sc);
            }
            float v, excess;
            direction_cut<N>(sc, v, excess);
            if (ch == cur_chunks - 1 && have_next) {
                // ask for the next tile's first group; it arrives during the index sum
                if (mi + 1 < a.count && next_tile >= a.m[mi + 1].tile_begin) {
                    int ni = mi + 1;
                    while (ni + 1 < a.count && next_tile >= a.m[ni + 1].tile_begin) ++ni;
                    enter_matrix(ni);
                }
                fetch_first(next_tile, pre);
            }
            const mp<W> c = direction_index<N, W, TW, CROW>(sc, K, v, excess, tab0, start);
            if constexpr (FUSED) {
                if (active) kept = c;
            } else if (active) {
                uint32_t* cp = m.codes + (static_cast<size_t>(row0 + cur_rl) * cur_G + g) * W;
                if (PVQ_DEBUG_INDEX((row0 + cur_rl) * cur_G + g, m.rows * cur_G, PVQ_DEBUG_GLOBAL_STORE)) {
#pragma unroll
                    for (int w = 0; w < W; ++w) cp[w] = c.w[w];
                }
            }
        }
        // zero padding of the rows' trees
        if (cur_gp != cur_G)
            for (int j = tid; j < cur_rpt * cur_gp; j += T)
                if ((j & (cur_gp - 1)) >= cur_G && PVQ_DEBUG_INDEX(j, sm.ss_floats, PVQ_DEBUG_SHARED_INDEX)) s_ss[j] = 0.0f;
        if (nedges != 0 && (buf ? edges1 : edges0) != m.edges) {  // uniform across the block
            for (int i = tid; i < nedges; i += T) s_edges[i] = m.edges[i];
            if constexpr (FUSED)
                for (int i = tid; i <= nedges; i += T) s_levels2[buf * 256 + i] = m.levels[i];
            if (buf)
                edges1 = m.edges;
            else
                edges0 = m.edges;
        }
        __syncthreads();  // this tile's energies (and edges) are in place; the previous tile's index words are complete

        if constexpr (!FUSED)
            if (!first_tile) flush_idx(prev_mi, tile - gridDim.x, s_idx2 + (buf ^ 1) * sm.idx_words);

        // Row energies: every warp sums the rows its threads sit in (for a row of 32 k groups that
        // is one row; the same sum is then made by several warps, which costs less than a barrier).
        const int rl_lo = __shfl_sync(kFull, cur_rl, 0);
        const int rl_hi = min(__shfl_sync(kFull, cur_rl, 31), cur_rpt - 1);
        float ss_row = 0.0f;
        for (int r = rl_lo; r <= rl_hi; ++r) {
            const float sum = warp_tree_sum(s_ss + r * cur_gp, cur_gp, lane);
            if (r == cur_rl) ss_row = sum;
        }
        float fused_amp = 0.0f;
        for (int ch = 0; ch < cur_chunks; ++ch) {
            const int g = cur_g0 + ch * T;
            if (!(row_ok && g < cur_G)) continue;
            const float ss = s_ss[cur_rl * cur_gp + g];
            int q = 0;
            if (b == 16) {  // the amplitude itself, as binary16
                q = __half_as_ushort(__float2half_rn(__fsqrt_rn(ss)));
            } else {
                // Step 5: q = floor(CDF(u) 2^b) as the number of bin edges <= u
                const float u = ss_row > 0.0f ? __fdiv_rn(ss, ss_row) : 0.0f;
                for (int step = 1 << (b - 1); step >= 1; step >>= 1)
                    if (s_edges[q + step - 1] <= u) q += step;
            }
            if constexpr (FUSED) {  // the dequantised amplitude, then the walk below
                fused_amp = b == 16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(q)))
                                    : __fmul_rn(__fsqrt_rn(ss_row), s_levels2[buf * 256 + q]);
                continue;
            }
            if (g == 0 && PVQ_DEBUG_INDEX(row0 + cur_rl, m.rows, PVQ_DEBUG_GLOBAL_STORE))
                m.row_norm[row0 + cur_rl] = __fsqrt_rn(ss_row);
            const unsigned bit = static_cast<unsigned>(g) * b;
            const unsigned sh = bit & 31u;
            if (!PVQ_DEBUG_INDEX(cur_rl * cur_idx_words + (bit >> 5) + (sh + b > 32u ? 1 : 0), sm.idx_words, PVQ_DEBUG_SHARED_INDEX))
                continue;
            atomicOr(&s_idx[cur_rl * cur_idx_words + (bit >> 5)], static_cast<uint32_t>(q) << sh);
            if (sh + b > 32u)
                atomicOr(&s_idx[cur_rl * cur_idx_words + (bit >> 5) + 1], static_cast<uint32_t>(q) >> (32u - sh));
        }
        if constexpr (FUSED) {
            // decode the code just made (every thread of the warp walks, in lockstep; a thread
            // without a group walks code 0)
            const bool active = row_ok && cur_g0 < cur_G;
            walk_code<N, W, YT>(kept, wt, K, yslots);
            if (active)
                emit_group<N, YT>(m, yslots, fused_amp, static_cast<unsigned>(row0 + cur_rl), static_cast<unsigned>(cur_g0));
        }
        prev_mi = cur_mi;
        if (!have_next) break;
        tile = next_tile;
    }
    if constexpr (!FUSED) {
        __syncthreads();  // the last tile's index words are complete
        flush_idx(prev_mi, tile, s_idx2 + buf * sm.idx_words);
    }
}

// Geometry and launch.  Returns PVQ_ERR_UNSUPPORTED when the case is not this kernel's (the
// caller then takes the general kernel).
template <int N, int W, bool BF16, int CROW, bool FUSED, typename YT>
static int launch_encode_fast_c(BatchArgs& a, cudaStream_t stream) {
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    constexpr int TW = W <= 2 ? W : 4;
    constexpr int EB = TW * 4;
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;

    // Block size: the multiple of 32 up to 256 that wastes the fewest thread slots over the batch.
    // A row of up to `threads` groups shares a tile with as many whole rows as fit; a longer row
    // is a tile of its own, taken in ceil(G / threads) chunks.
    int best_threads = 0;
    long long best_cost = -1;
    for (int threads = kFastThreadsMax; threads >= 128; threads -= 32) {
        long long cost = 0;
        for (int i = 0; i < a.count; ++i) {
            const int G = a.m[i].G;
            if (G <= threads) {
                const int rpt = threads / G;
                cost += ((a.m[i].rows + rpt - 1) / rpt) * threads;
            } else {
                cost += a.m[i].rows * ((G + threads - 1) / threads) * static_cast<long long>(threads);
            }
        }
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best_threads = threads;
        }
    }
    const int threads = best_threads;
    unsigned tiles = 0;
    int max_idx_words = 1, ss_floats = 4;
    for (int i = 0; i < a.count; ++i) {
        MatrixArgs& m = a.m[i];
        if (m.G > kFastMaxGroups) return PVQ_ERR_UNSUPPORTED;
        if (FUSED && m.G > threads) return PVQ_ERR_UNSUPPORTED;  // the round trip keeps one code per thread
        m.chunks = m.G <= threads ? 1 : (m.G + threads - 1) / threads;
        m.rows_per_tile = m.G <= threads ? threads / m.G : 1;
        m.tile_begin = tiles;
        tiles += static_cast<unsigned>((m.rows + m.rows_per_tile - 1) / m.rows_per_tile);
        max_idx_words = std::max(max_idx_words, m.rows_per_tile * (m.sstride / 4));
        int gp = 1;
        while (gp < m.G) gp <<= 1;
        ss_floats = std::max(ss_floats, m.rows_per_tile * gp);
    }
    a.total_tiles = tiles;

    FastSmem sm;
    // room behind the tables: a column offset is a sum of N small integers that cannot leave
    // [0, K] for finite input; should it ever, the read still falls inside the block's memory
    sm.tab_bytes = static_cast<uint32_t>(2 * N * CROW + N + 2) * EB + kCencSkew;  // == 2 * cenc_bytes + the skew + slack
    sm.ss_off = (sm.tab_bytes + 15u) & ~15u;
    sm.ss_floats = ss_floats;
    sm.edges_off = sm.ss_off + 2u * static_cast<uint32_t>(ss_floats) * 4u;
    sm.idx_off = sm.edges_off + 2u * 256u * 4u;
    sm.idx_words = max_idx_words;
    size_t smem = sm.idx_off + 2u * static_cast<size_t>(max_idx_words) * 4u;
    sm.walk_off = sm.walk_bytes = sm.levels_off = sm.wbuf_off = 0;
    sm.walk_phases = 0;
    if (FUSED) {
        const TableLayout L = table_layout(N, a.K, W);
        sm.levels_off = static_cast<uint32_t>((smem + 15u) & ~size_t(15));
        sm.wbuf_off = sm.levels_off + 2u * 256u * 4u;
        sm.walk_off = (sm.wbuf_off + static_cast<uint32_t>(threads) * YS + 15u) & ~15u;
        if (sm.walk_off >= static_cast<size_t>(di.smem_max)) return PVQ_ERR_UNSUPPORTED;
        sm.walk_phases = walk_phases_that_fit(L, static_cast<size_t>(di.smem_max) - sm.walk_off);
        if (sm.walk_phases == 0) return PVQ_ERR_UNSUPPORTED;
        sm.walk_bytes = (walk_tables_bytes(L, sm.walk_phases) + 15u) & ~15u;
        smem = sm.walk_off + sm.walk_bytes;
    }
    if (smem > static_cast<size_t>(di.smem_max)) return PVQ_ERR_UNSUPPORTED;

    auto kern = encode_fast_kernel<N, W, BF16, CROW, FUSED, YT>;
    int per_sm = 0;
    if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), threads, smem, &per_sm)) != PVQ_OK) return st;
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned grid = std::min<unsigned>(tiles, static_cast<unsigned>(di.sms * per_sm));
    kern<<<grid, threads, smem, stream>>>(a, sm);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int W, bool BF16, bool FUSED, typename YT>
static int launch_encode_fast_t(BatchArgs& a, cudaStream_t stream) {
    if constexpr (W > 4) {
        return PVQ_ERR_UNSUPPORTED;  // entries of 24 bytes: the general kernel
    } else {
        const TableLayout L = table_layout(N, a.K, W);
        if (L.cenc_bytes == 0) return PVQ_ERR_UNSUPPORTED;
        if (L.crow == 32) return launch_encode_fast_c<N, W, BF16, 32, FUSED, YT>(a, stream);
        if (L.crow == 64) return launch_encode_fast_c<N, W, BF16, 64, FUSED, YT>(a, stream);
        if (L.crow == 128) return launch_encode_fast_c<N, W, BF16, 128, FUSED, YT>(a, stream);
        return PVQ_ERR_UNSUPPORTED;
    }
}

// Entry of the per-(N, W) translation units: the plain encode and the round trip go to the
// kernel above when its tables fit (K <= 127 there, so a byte per coordinate), everything else
// (rotation, least-squares amplitude, larger tables) to the general one.
template <int N, int W>
static int launch_encode_any(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    if (a.rot_block == 0 && a.amp_mode == 0) {
        BatchArgs b = a;
        int st;
        if (dtype == PVQ_DTYPE_BF16)
            st = fused ? launch_encode_fast_t<N, W, true, true, int8_t>(b, s) : launch_encode_fast_t<N, W, true, false, int8_t>(b, s);
        else
            st = fused ? launch_encode_fast_t<N, W, false, true, int8_t>(b, s) : launch_encode_fast_t<N, W, false, false, int8_t>(b, s);
        if (st != PVQ_ERR_UNSUPPORTED) return st;
    }
    return launch_encode_nw<N, W>(a, dtype, fused, s);
}

}  // namespace pvq
