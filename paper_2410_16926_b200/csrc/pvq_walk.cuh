// The decode walk (Algorithm 3) shared by the decode kernel and the fused
// encode -> decode kernel.
//
// Algorithm 3 is run as a walk over the cells (i, col) of the count table, i the
// position and col the pulses still to place, from (0, K) to (N, 0).  With r the
// part of the code not yet explained and t = N(N-1-i, col), one step does
//
//   first test at a position:   r >= t   -> r -= t, one pulse here, go left (col-1)
//                               else     -> y_i = 0, go down (i+1)
//   after a pulse at i:         r >= 2t  -> r -= 2t, one more pulse, go left
//                               else     -> y_i = -m if r >= t (then r -= t) else +m, go down
//
// which is Algorithm 3's loop with the test that fails for magnitude m and the
// sign test read from the same table entry.  Every step goes left or down, so
// every group takes exactly N + K steps and at step s sits on the anti-diagonal
// i - col = s - K: the 32 threads of a warp run the same instructions with no
// data-dependent branch, and their table reads fall on neighbouring diagonal
// cells, which the table layout puts in different banks.
//
// r only shrinks.  Once every thread of the warp has r below 2^63 (2^31) the warp
// continues in a copy of the loop that works on two-word (one-word) integers
// and reads a table of that width, whose larger entries are saturated.
#pragma once
#include "mp_uint.cuh"
#include "pvq_internal.cuh"

namespace pvq {

constexpr unsigned kFull = 0xffffffffu;

// Shared-memory accesses of the walk by 32-bit shared-window address.
__device__ __forceinline__ uint32_t shared_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

template <int PW>
__device__ __forceinline__ mp<PW> load_entry(uint32_t addr) {
    mp<PW> t;
    if constexpr (PW == 1) {
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(t.w[0]) : "r"(addr));
    } else if constexpr (PW == 2) {
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(t.w[0]), "=r"(t.w[1]) : "r"(addr));
    } else if constexpr (PW <= 4) {  // 16-byte entries
        uint32_t v[4];
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                     : "r"(addr));
#pragma unroll
        for (int w = 0; w < PW; ++w) t.w[w] = v[w];
    } else {  // 24-byte entries, 8-byte aligned
        uint32_t v[6];
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v[0]), "=r"(v[1]) : "r"(addr));
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+8];" : "=r"(v[2]), "=r"(v[3]) : "r"(addr));
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+16];" : "=r"(v[4]), "=r"(v[5]) : "r"(addr));
#pragma unroll
        for (int w = 0; w < PW; ++w) t.w[w] = v[w];
    }
    return t;
}

template <typename YT>
__device__ __forceinline__ void store_y(uint32_t addr, int val) {
    if constexpr (sizeof(YT) == 1)
        asm volatile("st.shared.u8 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
    else
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
}

// State of one thread's walk.
struct Walk {
    int v;        // pulses placed at the current position so far
    uint32_t y;   // shared address of this thread's slot for the current position
    uint32_t y0;  // ... for position 0
};

// Runs steps s .. S-1 on PW-word integers with the table `tab` (entries of EB bytes),
// leaving early, at a multiple of 8 steps, once every thread's r fits `next_words` words
// with a bit to spare.  Returns the step reached.
template <int PW, int EB, int CW, typename YT>
__device__ __forceinline__ int walk_phase(mp<CW>& rfull, Walk& st, uint32_t tab, int rowlen, int K, int s,
                                          const int S, const int next_words) {
    mp<PW> r;
#pragma unroll
    for (int w = 0; w < PW; ++w) r.w[w] = rfull.w[w];
    const int D = (rowlen + 1) * EB;                   // one step down and one right
    const int i0 = static_cast<int>(st.y - st.y0) / static_cast<int>(sizeof(YT));  // position reached
    uint32_t p = tab + i0 * D + (K - s) * EB;          // entry (i, col) of this step
    int v = st.v;
    uint32_t y = st.y;

    auto step = [&]() {
        const mp<PW> t = load_entry<PW>(p);
        mp<PW> d2, d1;
        const bool lt1 = mp_sub_borrow<PW>(d2, r, t);   // d2 = r - t
        const bool lt2 = mp_sub_borrow<PW>(d1, d2, t);  // d1 = r - 2t
        const bool placed = v > 0;
        const bool ge1 = !lt1;
        const bool ge2 = ge1 && !lt2 && placed;
        const bool more = placed ? ge2 : ge1;  // another pulse at this position
#pragma unroll
        for (int w = 0; w < PW; ++w) r.w[w] = ge2 ? d1.w[w] : (ge1 ? d2.w[w] : r.w[w]);
        if (!more) {
            store_y<YT>(y, (ge1 && placed) ? -v : v);
            y += sizeof(YT);
            p += D;
        }
        v = more ? v + 1 : 0;
        p -= EB;
    };

    while (s + 8 <= S) {
        if (next_words > 0) {
            // does r fit next_words words with the top bit clear?
            uint32_t hi = 0;
#pragma unroll
            for (int w = 2; w < PW; ++w) hi |= r.w[w];
            if constexpr (PW > 1) hi |= next_words == 2 ? (r.w[1] >> 31) : r.w[1];
            if (next_words == 1) hi |= r.w[0] >> 31;
            if (__all_sync(kFull, hi == 0u)) break;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) step();
        s += 8;
    }
    if (next_words == 0 || s + 8 > S) {
        for (; s < S; ++s) step();
    }
#pragma unroll
    for (int w = 0; w < PW; ++w) rfull.w[w] = r.w[w];
    st.v = v;
    st.y = y;
    return s;
}


// The three staged walk tables as shared addresses, and which of them exist.
struct WalkTables {
    uint32_t tab0, tab2, tab1;
    bool has2, has1;
    int rowlen;
};

__device__ __forceinline__ WalkTables walk_tables(const TableLayout& L, uint32_t smem_base, int phases) {
    WalkTables t;
    t.tab0 = smem_base;
    t.tab2 = smem_base + (L.walk_off[1] - L.walk_off[0]);
    t.tab1 = smem_base + (L.walk_off[2] - L.walk_off[0]);
    t.has2 = phases >= 2 && L.walk_bytes[1] != 0;
    t.has1 = phases >= 3;
    t.rowlen = L.rowlen;
    return t;
}

__host__ __device__ inline uint32_t walk_tables_bytes(const TableLayout& L, int phases) {
    return L.walk_off[phases - 1] + L.walk_bytes[phases - 1] - L.walk_off[0];
}

// How many of the walk tables (a prefix of: widest, two-word, one-word) fit in `room` bytes
// of shared memory; 0 when not even the widest does.
inline int walk_phases_that_fit(const TableLayout& L, size_t room) {
    for (int p = 3; p >= 1; --p) {
        if (p > 1 && L.walk_bytes[p - 1] == 0) continue;
        if (((walk_tables_bytes(L, p) + 15u) & ~size_t(15)) <= room) return p;
    }
    return 0;
}

// Code c (destroyed) -> the thread's N slots `yslots` in shared memory.
template <int N, int W, typename YT>
__device__ __forceinline__ void walk_code(mp<W>& c, const WalkTables& t, int K, YT* yslots) {
    constexpr int TW = W <= 2 ? W : (W <= 4 ? 4 : 6);  // words per entry of the widest table
    const int S = N + K;
    Walk st;
    st.v = 0;
    st.y = st.y0 = shared_addr(yslots);
    int s = 0;
    s = walk_phase<W, TW * 4, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, t.has2 ? 2 : (t.has1 ? 1 : 0));
    if constexpr (W > 2) {
        if (s < S && t.has2) s = walk_phase<2, 8, W, YT>(c, st, t.tab2, t.rowlen, K, s, S, t.has1 ? 1 : 0);
    }
    if constexpr (W > 1) {
        if (s < S && t.has1) s = walk_phase<1, 4, W, YT>(c, st, t.tab1, t.rowlen, K, s, S, 0);
    }
}

// After walk_code by all threads of a warp: scale each group's point to the unit sphere
// times `amp` (this thread's group) and write the warp's 32 groups as bf16 with 16-byte
// stores.  wbuf: the warp's slot area (thread l at wbuf + l*YS), wscale: 32 floats.
// Group l of the tile is global group g0 + l of matrix m; groups >= ngroups are skipped.
template <int N, typename YT>
__device__ __forceinline__ void emit_tile(const MatrixArgs& m, uint8_t* wbuf, float* wscale, int lane, float amp,
                                          long long g0, long long ngroups) {
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    const YT* yslots = reinterpret_cast<const YT*>(wbuf + lane * YS);
    int ssy = 0;
    if constexpr (sizeof(YT) == 1) {
        const int* y4 = reinterpret_cast<const int*>(yslots);
#pragma unroll
        for (int v = 0; v < N / 4; ++v) ssy = __dp4a(y4[v], y4[v], ssy);
    } else {
#pragma unroll 8
        for (int v = 0; v < N; ++v) ssy += static_cast<int>(yslots[v]) * static_cast<int>(yslots[v]);
    }
    wscale[lane] = __fdiv_rn(amp, __fsqrt_rn(static_cast<float>(ssy)));
    __syncwarp();

    constexpr int TPG = N / 8;     // threads per group, 16 bytes each
    constexpr int GPI = 32 / TPG;  // groups per iteration
    const int part = lane % TPG;
#pragma unroll 1
    for (int it = 0; it < TPG; ++it) {
        const int gl = it * GPI + lane / TPG;  // group within the tile
        const long long gj = g0 + gl;
        if (gj < ngroups) {
            const YT* ys = reinterpret_cast<const YT*>(wbuf + gl * YS) + part * 8;
            const float sc = wscale[gl];
            float f[8];
            if constexpr (sizeof(YT) == 1) {
                const uint32_t lo = reinterpret_cast<const uint32_t*>(ys)[0];
                const uint32_t hi = reinterpret_cast<const uint32_t*>(ys)[1];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    f[e] = static_cast<float>(static_cast<int>(static_cast<int8_t>(lo >> (8 * e))));
                    f[4 + e] = static_cast<float>(static_cast<int>(static_cast<int8_t>(hi >> (8 * e))));
                }
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = static_cast<float>(static_cast<int>(ys[e]));
            }
            const unsigned row = static_cast<unsigned>(gj) / static_cast<unsigned>(m.G);
            const unsigned g = static_cast<unsigned>(gj) - row * static_cast<unsigned>(m.G);
            uint4 o;
            o.x = pack_bf16x2(__fmul_rn(f[0], sc), __fmul_rn(f[1], sc));
            o.y = pack_bf16x2(__fmul_rn(f[2], sc), __fmul_rn(f[3], sc));
            o.z = pack_bf16x2(__fmul_rn(f[4], sc), __fmul_rn(f[5], sc));
            o.w = pack_bf16x2(__fmul_rn(f[6], sc), __fmul_rn(f[7], sc));
            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.out) +
                                                  static_cast<size_t>(row) * m.ld_out +
                                                  static_cast<size_t>(g) * N + part * 8);
            *dst = o;
        }
    }
    __syncwarp();  // the slots are rewritten by the next tile
}

}  // namespace pvq
