// Large groups and wide codes (the paper's weight-only grid of Sec. 4.1: group sizes up to 256,
// 3 and more direction bits per weight, 16-bit amplitudes).  The tables no longer fit in shared
// memory (1.2 MB for N = 128, K = 187) and a group no longer fits in one thread's registers, so
// these kernels keep the tables in global memory (they stay in L2) and each thread's working
// arrays in shared memory, laid out element-major ([i][thread]) so that the threads of a warp
// touch consecutive words.  Same arithmetic, same results as the small-group kernels; one
// thread per group.
//
// A kernel computes in W words.  EXACT: codes are W words in memory.  Otherwise W is the next
// width the kernel is built for and the codes and table entries, a.code_words and top_words
// words long, are zero-extended as they are loaded.
#pragma once
#include <cuda_fp16.h>

#include <algorithm>

#include "pvq_encode_impl.cuh"

namespace pvq {

namespace {

// The low W words of a table entry of TW words in global memory (zero-extended when TW < W).
// Entries of a multiple of 4 words are 16-byte aligned, of an even number 8-byte aligned.
template <int W>
__device__ __forceinline__ mp<W> load_entry_v(const uint8_t* p, int TW) {
    mp<W> t;
    if ((TW & 3) == 0) {
#pragma unroll
        for (int v = 0; v < (W + 3) / 4; ++v) {
            uint4 q = make_uint4(0u, 0u, 0u, 0u);
            if (4 * v < TW) q = __ldg(reinterpret_cast<const uint4*>(p) + v);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (4 * v + u < W) t.w[4 * v + u] = w[u];
        }
    } else if ((TW & 1) == 0) {
#pragma unroll
        for (int v = 0; v < (W + 1) / 2; ++v) {
            uint2 q = make_uint2(0u, 0u);
            if (2 * v < TW) q = __ldg(reinterpret_cast<const uint2*>(p) + v);
            t.w[2 * v] = q.x;
            if (2 * v + 1 < W) t.w[2 * v + 1] = q.y;
        }
    } else {
#pragma unroll
        for (int w = 0; w < W; ++w) t.w[w] = w < TW ? __ldg(reinterpret_cast<const uint32_t*>(p) + w) : 0u;
    }
    return t;
}

// One phase of the decode walk (see pvq_walk.cuh) with the table in global memory, computing
// in PW words on entries of TW words.  The phase ends when every lane can go on in
// next_words words: on a narrow table whose large values are saturated (next_same false:
// the remainder must be two bits below the width), or on this table with fewer words
// (next_same true: the remainder and the entry just read fit next_words words; the entries
// along a path never grow, N(n,k) being monotone in n and k).
template <int PW, int CW, typename YT>
__device__ __forceinline__ int walk_phase_g(mp<CW>& rfull, Walk& st, const uint8_t* tab, int TW, int rowlen,
                                            int K, int s, const int S, const int next_words,
                                            const bool next_same) {
    const int EB = TW * 4;  // bytes per entry
    mp<PW> r, t;
#pragma unroll
    for (int w = 0; w < PW; ++w) {
        r.w[w] = rfull.w[w];
        t.w[w] = 0xffffffffu;  // no entry read yet
    }
    const int D = (rowlen + 1) * EB;
    const int i0 = static_cast<int>(st.y - st.y0) / static_cast<int>(sizeof(YT));
    const uint8_t* p = tab + static_cast<size_t>(i0) * D + (K - s) * EB;
    int v = st.v;
    uint32_t y = st.y;
    for (; s < S; ++s) {
        if (next_words > 0 && (s & 7) == 0) {
            uint32_t hi = 0;
#pragma unroll
            for (int w = 1; w < PW; ++w)
                if (w >= next_words) hi |= next_same ? (r.w[w] | t.w[w]) : r.w[w];
            if (!next_same) {
#pragma unroll
                for (int w = 0; w < PW; ++w)
                    if (w == next_words - 1) hi |= r.w[w] >> 30;
            }
            if (__all_sync(kFull, hi == 0u)) break;
        }
        t = load_entry_v<PW>(p, TW);
        mp<PW> d2, d1;
        const bool lt1 = mp_sub_borrow<PW>(d2, r, t);
        const bool lt2 = mp_sub_borrow<PW>(d1, d2, t);
        const bool placed = v > 0;
        const bool ge1 = !lt1;
        const bool ge2 = ge1 && !lt2 && placed;
        const bool more = ge2 || (ge1 && !placed);
#pragma unroll
        for (int w = 0; w < PW; ++w) r.w[w] = ge2 ? d1.w[w] : (ge1 ? d2.w[w] : r.w[w]);
        store_y<YT>(y, ((ge1 && placed) ? -v : v) + kSlotBias<YT>);
        y += more ? 0u : static_cast<uint32_t>(sizeof(YT));
        p += more ? 0 : D;
        v = more ? v + 1 : 0;
        p -= EB;
    }
#pragma unroll
    for (int w = 0; w < PW; ++w) rfull.w[w] = r.w[w];
    st.v = v;
    st.y = y;
    return s;
}

// The phases on the full-width table: PW words, then 16, 8 and 4 as the remainder shrinks
// (about one bit per step), the last of them handing over to the narrow tables (sat_next).
template <int PW, int CW, typename YT>
__device__ __forceinline__ int walk_wide_phases(mp<CW>& c, Walk& st, const uint8_t* tab, int TW, int rowlen, int K,
                                                int s, const int S, const int sat_next) {
    constexpr int NEXT = PW > 16 ? 16 : (PW > 8 ? 8 : (PW > 4 ? 4 : 0));
    if constexpr (NEXT == 0) {
        return walk_phase_g<PW, CW, YT>(c, st, tab, TW, rowlen, K, s, S, sat_next, false);
    } else {
        s = walk_phase_g<PW, CW, YT>(c, st, tab, TW, rowlen, K, s, S, NEXT, true);
        if (s < S) s = walk_wide_phases<NEXT, CW, YT>(c, st, tab, TW, rowlen, K, s, S, sat_next);
        return s;
    }
}

constexpr int kBigThreads = 256;

// ---- bitonic merge of 32 values in registers (v bitonic on entry), descending or ascending
template <bool DESC, int I, int J>
__device__ __forceinline__ void merge_cx(float (&v)[32]) {
    const float hi = fmaxf(v[I], v[J]), lo = fminf(v[I], v[J]);
    v[I] = DESC ? hi : lo;
    v[J] = DESC ? lo : hi;
}

template <bool DESC, int J, int I>
__device__ __forceinline__ void merge_stage(float (&v)[32]) {  // pairs (i, i + J) for all i with bit J clear
    if constexpr (I < 32) {
        if constexpr ((I & J) == 0) merge_cx<DESC, I, I + J>(v);
        merge_stage<DESC, J, I + 1>(v);
    }
}

template <bool DESC>
__device__ __forceinline__ void merge32(float (&v)[32]) {
    merge_stage<DESC, 16, 0>(v);
    merge_stage<DESC, 8, 0>(v);
    merge_stage<DESC, 4, 0>(v);
    merge_stage<DESC, 2, 0>(v);
    merge_stage<DESC, 1, 0>(v);
}

// Sorts a column of N floats (es[i * T], N up to 32 or a multiple of 64) in descending order: chunks of 32
// in registers (sorting network, then bitonic merges), the strides of 32 and more between
// chunks in shared memory.
template <int N>
__device__ __forceinline__ void sort_column_desc(float* es, int T) {
    if constexpr (N <= 32) {  // one chunk
        float v[N];
#pragma unroll
        for (int i = 0; i < N; ++i) v[i] = es[i * T];
        sort_desc<N>(v);
#pragma unroll
        for (int i = 0; i < N; ++i) es[i * T] = v[i];
        return;
    }
    float v[32];
    for (int q = 0; q < N / 32; ++q) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = es[(q * 32 + i) * T];
        sort_desc<32>(v);
        if (q & 1) {  // odd chunks ascending: neighbours then form bitonic runs of 64
#pragma unroll
            for (int i = 0; i < 32; ++i) es[(q * 32 + i) * T] = v[31 - i];
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) es[(q * 32 + i) * T] = v[i];
        }
    }
    for (int k = 64; k <= N; k <<= 1) {
        for (int j = k >> 1; j >= 32; j >>= 1) {
            for (int p = 0; p < N / 2; ++p) {
                const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));  // the p-th index with bit j clear
                const int l = i | j;
                const float x0 = es[i * T], x1 = es[l * T];
                const bool desc = (i & k) == 0;
                const float hi = fmaxf(x0, x1), lo = fminf(x0, x1);
                es[i * T] = desc ? hi : lo;
                es[l * T] = desc ? lo : hi;
            }
        }
        for (int q = 0; q < N / 32; ++q) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = es[(q * 32 + i) * T];
            if (((q * 32) & k) == 0)
                merge32<true>(v);
            else
                merge32<false>(v);
#pragma unroll
            for (int i = 0; i < 32; ++i) es[(q * 32 + i) * T] = v[i];
        }
    }
}

template <int N, int W, bool EXACT, typename YT>
__global__ void __launch_bounds__(kBigThreads) decode_big_kernel(const __grid_constant__ BatchArgs a) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    const int K = a.K;
    const int Wc = EXACT ? W : a.code_words;
    const TableLayout L = table_layout(N, K, Wc);
    const int TW = EXACT ? top_words_of(W) : L.top_words;
    const uint8_t* blob = reinterpret_cast<const uint8_t*>(a.table);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    YT* yslots = reinterpret_cast<YT*>(smem + threadIdx.x * YS);

    mp<W> bound;
    const uint32_t* bw = a.table + L.bound_off / 4;
#pragma unroll
    for (int w = 0; w < W; ++w) bound.w[w] = w < Wc ? bw[w] : 0u;
    const bool bound_wide = bw[Wc] != 0u;

    const unsigned b = a.scale_bits;
    const int S = N + K;
    const unsigned warps_total = gridDim.x * (blockDim.x >> 5);
    bool bad = false;
    for (unsigned tile = blockIdx.x * (blockDim.x >> 5) + warp; tile < a.total_tiles; tile += warps_total) {
        const int mi = find_matrix(a, tile);
        const MatrixArgs& m = a.m[mi];
        const unsigned G = static_cast<unsigned>(m.G);
        const unsigned ngroups = static_cast<unsigned>(m.rows) * G;
        const unsigned gi = (tile - m.tile_begin) * 32u + lane;
        const bool active = gi < ngroups;
        const unsigned row = gi / G;
        const unsigned g = gi - row * G;

        mp<W> c;
        mp_zero(c);
        float amp = 0.0f;
        if (active) {
            const uint32_t* cp = m.codes + static_cast<size_t>(gi) * Wc;
#pragma unroll
            for (int w = 0; w < W; ++w)
                if (w < Wc) c.w[w] = cp[w];
            mp<W> tmp;
            const bool valid = bound_wide || mp_sub_borrow<W>(tmp, c, bound);
            if (!valid) {
                bad = true;
                mp_zero(c);
            } else {
                const uint8_t* srow = m.scale_idx + static_cast<size_t>(row) * m.sstride;
                const unsigned bit = g * b;
                unsigned bits = srow[bit >> 3];
                if ((bit & 7u) + b > 8u) bits |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
                const unsigned q = (bits >> (bit & 7u)) & ((1u << b) - 1u);
                amp = b == 16u ? __half2float(__ushort_as_half(static_cast<unsigned short>(q)))
                               : __fmul_rn(m.row_norm[row], m.levels[q]);
            }
        }
        Walk st;
        st.v = 0;
        st.y = st.y0 = shared_addr(yslots);
        int s = 0;
        const bool has2 = L.walk_bytes[1] != 0, has1 = L.walk_bytes[2] != 0;
        s = walk_wide_phases<W, W, YT>(c, st, blob + L.walk_off[0], TW, L.rowlen, K, s, S,
                                       has2 ? 2 : (has1 ? 1 : 0));
        if constexpr (W > 2) {
            if (s < S && has2)
                s = walk_phase_g<2, W, YT>(c, st, blob + L.walk_off[1], 2, L.rowlen, K, s, S, has1 ? 1 : 0, false);
        }
        if constexpr (W > 1) {
            if (s < S && has1) s = walk_phase_g<1, W, YT>(c, st, blob + L.walk_off[2], 1, L.rowlen, K, s, S, 0, false);
        }
        if (active) emit_group<N, YT>(m, yslots, amp, row, g);
        __syncwarp();
    }
    if (bad && a.status) atomicOr(a.status, PVQ_STATUS_INVALID_CODE);
}

template <int N, int W, bool EXACT, typename YT>
int launch_decode_big_t(BatchArgs& a, cudaStream_t stream) {
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    unsigned tiles = 0;
    for (int i = 0; i < a.count; ++i) {
        a.m[i].tile_begin = tiles;
        tiles += static_cast<unsigned>((a.m[i].rows * a.m[i].G + 31) / 32);
    }
    a.total_tiles = tiles;
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    const int threads = kBigThreads;
    const size_t smem = static_cast<size_t>(threads) * YS;
    auto kern = decode_big_kernel<N, W, EXACT, YT>;
    int per_sm = 0;
    if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), threads, smem, &per_sm)) != PVQ_OK) return st;
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned wpb = threads / 32;
    const unsigned grid = std::max(1u, std::min<unsigned>((tiles + wpb - 1) / wpb, di.sms * per_sm));
    kern<<<grid, threads, smem, stream>>>(a);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

// ------------------------------------------------------------------------- encode

struct BigSmem {
    uint32_t es_off, ss_off, edges_off, idx_off;
    uint32_t xs_off;  // rotation: a second column per thread for the rotated values
    int ss_floats, idx_words;
};

// element i of this thread's group, from global memory
template <bool BF16>
__device__ __forceinline__ float group_value(const void* gx, int i) {
    if constexpr (BF16)
        return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const unsigned short*>(gx) + i)) << 16);
    else
        return __ldg(static_cast<const float*>(gx) + i);
}

// elements 8j .. 8j+7 of this thread's group with 16-byte loads (groups start 16-byte aligned)
template <bool BF16>
__device__ __forceinline__ void group_values8(const void* gx, int j, float (&x)[8]) {
    if constexpr (BF16) {
        const uint4 q = __ldg(static_cast<const uint4*>(gx) + j);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            x[2 * p] = __uint_as_float(w[p] << 16);
            x[2 * p + 1] = __uint_as_float(w[p] & 0xffff0000u);
        }
    } else {
        const float4 q0 = __ldg(static_cast<const float4*>(gx) + 2 * j);
        const float4 q1 = __ldg(static_cast<const float4*>(gx) + 2 * j + 1);
        x[0] = q0.x, x[1] = q0.y, x[2] = q0.z, x[3] = q0.w;
        x[4] = q1.x, x[5] = q1.y, x[6] = q1.z, x[7] = q1.w;
    }
}


// Encoder for large groups: the steps of encode_kernel with the per-thread arrays (residuals
// to sort, the point) in shared memory columns es[i * T + t], the input re-read
// from global memory where it is needed, and the cumulative tables read from global memory.
template <int N, int W, bool EXACT, bool BF16, bool FUSED, bool ROT>
__global__ void __launch_bounds__(kBigThreads) encode_big_kernel(const __grid_constant__ BatchArgs a,
                                                                  const __grid_constant__ BigSmem sm) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int T = blockDim.x;
    const int t = threadIdx.x;
    float* es = reinterpret_cast<float*>(smem + sm.es_off) + t;         // column of this thread, stride T
    const float* xs = nullptr;  // rotation: the column that holds this thread's rotated group
    // The point lies over the upper half of this thread's es column, two entries to a word: that
    // half is dead once the cut value has been read from the sorted residuals (the least-squares
    // tree uses the lower half).
    auto ms = [&es, T](int i) -> short& {
        return reinterpret_cast<short*>(es + (N / 2 + (i >> 1)) * T)[i & 1];
    };
    float* s_ss = reinterpret_cast<float*>(smem + sm.ss_off);
    float* s_edges = reinterpret_cast<float*>(smem + sm.edges_off);
    uint32_t* s_idx = reinterpret_cast<uint32_t*>(smem + sm.idx_off);
    const int K = a.K;
    const int b = a.scale_bits;
    const int nedges = b <= 8 ? (1 << b) - 1 : 0;
    const int Wc = EXACT ? W : a.code_words;
    const TableLayout L = table_layout(N, K, Wc);
    const int TW = EXACT ? top_words_of(W) : L.top_words;
    const uint8_t* blob = reinterpret_cast<const uint8_t*>(a.table);
    const uint8_t* tabU = blob + L.enc_off[0];
    const uint8_t* tab2V = blob + L.enc_off[1];
    const int lane = t & 31, warp = t >> 5, nwarps = T >> 5;
    const float* cur_edges = nullptr;

    for (unsigned tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x) {
        const TileLoc loc = locate(a, tile);
        const MatrixArgs& m = a.m[loc.mi];
        const int G = loc.G, rpt = loc.rpt, gp = loc.gp, rl = loc.rl, g = loc.g;
        const long long row = loc.row0 + rl;
        const bool active = loc.active;
        const int idx_words = m.sstride >> 2;
        const void* gx = nullptr;
        if (active)
            gx = static_cast<const uint8_t*>(m.x) +
                 (static_cast<size_t>(row) * m.ld + static_cast<size_t>(g) * N) * (BF16 ? 2 : 4);

        __syncthreads();  // previous tile is done with shared memory
        if (nedges != 0 && cur_edges != m.edges) {
            for (int i = t; i < nedges; i += T) s_edges[i] = m.edges[i];
            cur_edges = m.edges;
        }
        for (int i = t; i < rpt * gp; i += T) s_ss[i] = 0.0f;
        for (int i = t; i < rpt * idx_words; i += T) s_idx[i] = 0u;
        __syncthreads();

        // Rotation in front of the encoder (Sec. 2.3 / Sec. 3.3 Step 1, as rotate_tile does it for
        // the small groups): x <- (x * s) H_B / sqrt(B) on every block of B = N * T0 consecutive
        // columns.  The butterflies (a, b) -> (a + b, a - b) run with strides 1, 2, 4, ...: below N
        // inside the thread's column, from N up between the columns of threads t and t ^ d (T0
        // divides G, so both hold groups of the same block), written to the other of two columns
        // with a barrier between stages.  Every sum is one fp32 addition.
        if constexpr (ROT) {
            float* xa = reinterpret_cast<float*>(smem + sm.xs_off) + t;
            float* xb = reinterpret_cast<float*>(smem + sm.es_off) + t;
            const int T0 = a.rot_block / N;
            if (active) {
                const float* sg = a.rot_signs + (g & (T0 - 1)) * N;
                float x[8];
                for (int j = 0; j < N / 8; ++j) {
                    group_values8<BF16>(gx, j, x);
#pragma unroll
                    for (int p = 0; p < 8; ++p) xa[(8 * j + p) * T] = __fmul_rn(x[p], __ldg(sg + 8 * j + p));
                }
                for (int h = 1; h < N; h <<= 1) {
                    for (int q = 0; q < N / 2; ++q) {
                        const int j = ((q & ~(h - 1)) << 1) | (q & (h - 1));  // the q-th index with bit h clear
                        const float u = xa[j * T], w = xa[(j + h) * T];
                        xa[j * T] = __fadd_rn(u, w);
                        xa[(j + h) * T] = __fsub_rn(u, w);
                    }
                }
            }
            for (int d = 1; d < T0; d <<= 1) {
                __syncthreads();
                if (active) {
                    const float sgn = (t & d) != 0 ? -1.0f : 1.0f;  // a + b on the lower thread, a - b on the upper
                    const float* pa = xa + ((t ^ d) - t);           // the partner's column
                    for (int i = 0; i < N; ++i) xb[i * T] = __fmaf_rn(xa[i * T], sgn, pa[i * T]);
                }
                float* tmp = xa;
                xa = xb;
                xb = tmp;
            }
            if (T0 > 1) __syncthreads();  // nobody reads a partner's old column any more
            if (active) {
                const float scale = static_cast<float>(1.0 / sqrt(static_cast<double>(a.rot_block)));
                for (int i = 0; i < N; ++i) xa[i * T] = __fmul_rn(xa[i * T], scale);
            }
            xs = xa;
            es = xb;
        }
        // element i / elements 8j .. 8j+7 of the group the kernel works on
        auto value = [&](int i) -> float { return ROT ? xs[i * T] : group_value<BF16>(gx, i); };
        auto values8 = [&](int j, float (&x)[8]) {
            if constexpr (ROT) {
#pragma unroll
                for (int p = 0; p < 8; ++p) x[p] = xs[(8 * j + p) * T];
            } else {
                group_values8<BF16>(gx, j, x);
            }
        };

        // group norms by the balanced tree, run level by level in the es column
        float l1 = 0.0f, ss = 0.0f;
        if (active) {
            float x[8];
            for (int j = 0; j < N / 8; ++j) {
                values8(j, x);
#pragma unroll
                for (int p = 0; p < 4; ++p) es[(4 * j + p) * T] = __fadd_rn(fabsf(x[2 * p]), fabsf(x[2 * p + 1]));
            }
            for (int len = N / 4; len >= 1; len >>= 1)
                for (int j = 0; j < len; ++j) es[j * T] = __fadd_rn(es[2 * j * T], es[(2 * j + 1) * T]);
            l1 = es[0];
            for (int j = 0; j < N / 8; ++j) {
                values8(j, x);
#pragma unroll
                for (int p = 0; p < 4; ++p)
                    es[(4 * j + p) * T] = __fadd_rn(__fmul_rn(x[2 * p], x[2 * p]), __fmul_rn(x[2 * p + 1], x[2 * p + 1]));
            }
            for (int len = N / 4; len >= 1; len >>= 1)
                for (int j = 0; j < len; ++j) es[j * T] = __fadd_rn(es[2 * j * T], es[(2 * j + 1) * T]);
            ss = es[0];
            s_ss[rl * gp + g] = ss;
        }
        __syncthreads();
        for (int r = warp; r < rpt; r += nwarps) {
            float* rs = s_ss + r * gp;
            for (int s = 1; s < gp; s <<= 1) {
                for (int j = lane * 2 * s; j < gp; j += 64 * s) rs[j] = __fadd_rn(rs[j], rs[j + s]);
                __syncwarp();
            }
        }

        // direction (Sec. 2.5): floor, then the d largest residuals get one more pulse
        mp<W> c;
        mp_zero(c);
        float ls_amp = 0.0f;
        if (active) {
            const float gsc = __fdiv_rn(static_cast<float>(K), l1);
            bool has_dir = (l1 > 0.0f) && (l1 <= 3.4028234e38f) && (gsc <= 3.4028234e38f);
            int d = 0;
            if (has_dir) {
                float sumf = 0.0f;
                float x[8];
                for (int j = 0; j < N / 8; ++j) {
                    values8(j, x);
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        const float av = __fmul_rn(fabsf(x[p]), gsc);
                        const float tt = __fadd_rd(av, kMagic);
                        const float f = __fsub_rn(tt, kMagic);
                        es[(8 * j + p) * T] = __fsub_rn(av, f);
                        sumf = __fadd_rn(sumf, f);
                    }
                }
                d = K - static_cast<int>(sumf);
                has_dir = d >= 0 && d <= N;
            }
            if (has_dir) {
                sort_column_desc<N>(es, T);
                const float v = d > 0 ? es[(d - 1) * T] : 2.0f;
                asm volatile("" ::: "memory");  // the point's column reuses the residuals' memory from here on
                int cnt = 0;
                float x[8];
                for (int j = 0; j < N / 8; ++j) {
                    values8(j, x);
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        const float av = __fmul_rn(fabsf(x[p]), gsc);
                        const float tt = __fadd_rd(av, kMagic);
                        const float e = __fsub_rn(av, __fsub_rn(tt, kMagic));
                        const int one = e >= v ? 1 : 0;
                        const int mi = __float_as_int(tt) - kMagicBits + one;
                        ms(8 * j + p) = static_cast<short>(__float_as_int(x[p]) < 0 ? -mi : mi);
                        cnt += one;
                    }
                }
                int excess = cnt - d;
                for (int i = N - 1; i >= 0 && excess > 0; --i) {  // equal residuals straddle the cut
                    const float xi = value(i);
                    const float av = __fmul_rn(fabsf(xi), gsc);
                    const float tt = __fadd_rd(av, kMagic);
                    if (__fsub_rn(av, __fsub_rn(tt, kMagic)) == v) {
                        ms(i) += __float_as_int(xi) < 0 ? 1 : -1;
                        --excess;
                    }
                }
            } else {
                for (int i = 0; i < N; ++i) ms(i) = 0;
                ms(0) = static_cast<short>(K);
            }

            if (a.amp_mode == 1) {  // least-squares amplitude: tree of |y_i| |x_i| in the es column
                int ssy = 0;  // exact; converted once (it can pass 2^24 when K > 4095)
                float x[8];
                for (int j8 = 0; j8 < N / 8; ++j8) {
                    values8(j8, x);
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const int j = 4 * j8 + p;
                        const int y0 = ms(2 * j), y1 = ms(2 * j + 1);
                        const float m0 = fabsf(static_cast<float>(y0)), m1 = fabsf(static_cast<float>(y1));
                        ssy += y0 * y0 + y1 * y1;
                        es[j * T] = __fadd_rn(__fmul_rn(m0, fabsf(x[2 * p])), __fmul_rn(m1, fabsf(x[2 * p + 1])));
                    }
                }
                for (int len = N / 4; len >= 1; len >>= 1)
                    for (int j = 0; j < len; ++j) es[j * T] = __fadd_rn(es[2 * j * T], es[(2 * j + 1) * T]);
                ls_amp = __fdiv_rn(es[0], __fsqrt_rn(static_cast<float>(ssy)));
            }

            // Algorithm 2 with the cumulative tables (see enumerate_uv)
            mp<W> plus, minus;
            mp_zero(plus);
            mp_zero(minus);
            int k = K;
            const size_t rowwords = static_cast<size_t>(K + 2) * TW;
#pragma unroll 4
            for (int i = 0; i < N; ++i) {
                const int y = ms(i);
                if (y != 0) {  // a zero adds and subtracts the same entry
                    const int k2 = k - abs(y);
                    const uint8_t* ru = tabU + (i * rowwords + static_cast<size_t>(k + 1) * TW) * 4;
                    const uint8_t* rx = (y < 0 ? tabU : tab2V) + (i * rowwords + static_cast<size_t>(k2 + 1) * TW) * 4;
                    mp_add<W>(plus, load_entry_v<W>(ru, TW));
                    mp_add<W>(minus, load_entry_v<W>(rx, TW));
                    k = k2;
                }
            }
            mp_sub_borrow<W>(c, plus, minus);
        }

        __syncthreads();  // row energies are in s_ss[r * gp]
        float amp = 0.0f;     // round trip: the dequantised amplitude
        if (active) {
            const float ss_row = s_ss[rl * gp];
            const float rnorm = __fsqrt_rn(ss_row);
            int q = 0;
            if (b == 16) {
                q = __half_as_ushort(__float2half_rn(a.amp_mode == 1 ? ls_amp : __fsqrt_rn(ss)));
            } else {
                const float amp2 = a.amp_mode == 1 ? __fmul_rn(ls_amp, ls_amp) : ss;
                const float u = ss_row > 0.0f ? __fdiv_rn(amp2, ss_row) : 0.0f;
                for (int step = 1 << (b - 1); step >= 1; step >>= 1)
                    if (s_edges[q + step - 1] <= u) q += step;
            }
            if constexpr (FUSED) {
                amp = b == 16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(q)))
                              : __fmul_rn(rnorm, m.levels[q]);
            } else {
                if (g == 0) m.row_norm[row] = rnorm;
                uint32_t* cp = m.codes + (static_cast<size_t>(row) * G + g) * Wc;
#pragma unroll
                for (int w = 0; w < W; ++w)
                    if (w < Wc) cp[w] = c.w[w];
                const unsigned bit = static_cast<unsigned>(g) * b;
                const unsigned sh = bit & 31u;
                atomicOr(&s_idx[rl * idx_words + (bit >> 5)], static_cast<uint32_t>(q) << sh);
                if (sh + b > 32u)
                    atomicOr(&s_idx[rl * idx_words + (bit >> 5) + 1], static_cast<uint32_t>(q) >> (32u - sh));
            }
        }
        if constexpr (FUSED) {
            // Round trip (activations, Sec. 4.3): decode the code just made.  Every thread is past
            // the enumeration (the barrier above), so the columns are free: each thread collects
            // its point in its own slots there, as decode_big_kernel does.
            constexpr int YS = N * 2 + 4;
            short* yslots = reinterpret_cast<short*>(smem + sm.es_off + static_cast<size_t>(t) * YS);
            Walk st;
            st.v = 0;
            st.y = st.y0 = shared_addr(yslots);
            const int S = N + K;
            int s = 0;
            const bool has2 = L.walk_bytes[1] != 0, has1 = L.walk_bytes[2] != 0;
            s = walk_wide_phases<W, W, short>(c, st, blob + L.walk_off[0], TW, L.rowlen, K, s, S,
                                              has2 ? 2 : (has1 ? 1 : 0));
            if constexpr (W > 2) {
                if (s < S && has2)
                    s = walk_phase_g<2, W, short>(c, st, blob + L.walk_off[1], 2, L.rowlen, K, s, S, has1 ? 1 : 0, false);
            }
            if constexpr (W > 1) {
                if (s < S && has1)
                    s = walk_phase_g<1, W, short>(c, st, blob + L.walk_off[2], 1, L.rowlen, K, s, S, 0, false);
            }
            if (active)
                emit_group<N, short>(m, yslots, amp, static_cast<unsigned>(row), static_cast<unsigned>(g));
            continue;  // the barrier at the top of the loop frees the slots
        }
        __syncthreads();
        for (int i = t; i < rpt * idx_words; i += T) {
            const int r2 = i / idx_words;
            const long long row2 = loc.row0 + r2;
            if (row2 < m.rows)
                reinterpret_cast<uint32_t*>(m.scale_idx + static_cast<size_t>(row2) * m.sstride)[i - r2 * idx_words] = s_idx[i];
        }
    }
}

template <int N, int W, bool EXACT, bool BF16, bool FUSED, bool ROT>
int launch_encode_big_t(BatchArgs& a, cudaStream_t stream) {
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    // a block covers whole rows: the fewest wasted thread slots among multiples of 32 whose
    // columns (one per thread, two when rotating) fit in shared memory
    const unsigned columns = ROT ? 2u : 1u;
    int best = 0;
    long long best_cost = -1;
    for (int threads = 32; threads <= kBigThreads; threads += 32) {
        if (static_cast<size_t>(threads) * N * 4u * columns + 8192u > static_cast<size_t>(di.smem_max)) break;
        long long cost = 0;
        bool ok = true;
        for (int i = 0; i < a.count && ok; ++i) {
            if (a.m[i].G > threads) ok = false;
            else cost += ((a.m[i].rows + threads / a.m[i].G - 1) / (threads / a.m[i].G)) * threads;
        }
        if (ok && (best_cost < 0 || cost < best_cost)) {
            best_cost = cost;
            best = threads;
        }
    }
    if (best == 0) return PVQ_ERR_UNSUPPORTED;
    const int threads = best;
    unsigned tiles = 0;
    int idx_words = 1, ss_floats = 1;
    for (int i = 0; i < a.count; ++i) {
        MatrixArgs& m = a.m[i];
        m.rows_per_tile = threads / m.G;
        m.tile_begin = tiles;
        tiles += static_cast<unsigned>((m.rows + m.rows_per_tile - 1) / m.rows_per_tile);
        idx_words = std::max(idx_words, m.rows_per_tile * (m.sstride / 4));
        int gp = 1;
        while (gp < m.G) gp <<= 1;
        ss_floats = std::max(ss_floats, m.rows_per_tile * gp);
    }
    a.total_tiles = tiles;
    BigSmem sm;
    sm.es_off = 0;
    sm.xs_off = static_cast<uint32_t>(threads) * N * 4u;
    sm.ss_off = sm.xs_off * columns;
    sm.edges_off = sm.ss_off + ss_floats * 4u;
    sm.idx_off = sm.edges_off + 256u * 4u;
    sm.ss_floats = ss_floats;
    sm.idx_words = idx_words;
    const size_t smem = sm.idx_off + idx_words * 4u;
    if (smem > static_cast<size_t>(di.smem_max)) return PVQ_ERR_UNSUPPORTED;
    auto kern = encode_big_kernel<N, W, EXACT, BF16, FUSED, ROT>;
    int per_sm = 0;
    if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), threads, smem, &per_sm)) != PVQ_OK) return st;
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned grid = std::min<unsigned>(tiles, static_cast<unsigned>(di.sms * per_sm));
    kern<<<grid, threads, smem, stream>>>(a, sm);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int W, bool EXACT>
int launch_big_w(BatchArgs& a, int dtype, bool decode, cudaStream_t s) {
    if (decode)
        return a.K <= 127 ? launch_decode_big_t<N, W, EXACT, int8_t>(a, s)
                          : launch_decode_big_t<N, W, EXACT, int16_t>(a, s);
    const bool bf16 = dtype == PVQ_DTYPE_BF16;
    if (a.rot_block != 0) {
        if (a.fused)
            return bf16 ? launch_encode_big_t<N, W, EXACT, true, true, true>(a, s)
                        : launch_encode_big_t<N, W, EXACT, false, true, true>(a, s);
        return bf16 ? launch_encode_big_t<N, W, EXACT, true, false, true>(a, s)
                    : launch_encode_big_t<N, W, EXACT, false, false, true>(a, s);
    }
    if (a.fused)
        return bf16 ? launch_encode_big_t<N, W, EXACT, true, true, false>(a, s)
                    : launch_encode_big_t<N, W, EXACT, false, true, false>(a, s);
    return bf16 ? launch_encode_big_t<N, W, EXACT, true, false, false>(a, s)
                : launch_encode_big_t<N, W, EXACT, false, false, false>(a, s);
}

}  // namespace

// wide codes and the other group sizes (pvq_wide.cu)
int launch_wide(BatchArgs& a, int dtype, int N, int W, bool decode, cudaStream_t stream);

}  // namespace pvq
