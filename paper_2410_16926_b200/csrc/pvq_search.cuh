// Device pieces shared by the builder of the search section (pvq_tables.cu) and the kernels
// that decode with it (pvq_decode_search.cu, the round trip of pvq_encode_fast.cuh); the
// section is described at SearchLayout.
#pragma once
#include <cstdint>

#include "pvq_walk.cuh"

namespace pvq {

// Key of a W-word integer q >= 1: q truncated to its leading 24 bits, as the bits of an fp32.
// Every conversion and every multiply-add rounds towards zero, and a truncation of a
// truncation is the truncation, so the result is exact whatever the width; it never
// decreases when q grows, which is all the bucket tables need.
__device__ __forceinline__ uint32_t search_key(const uint32_t* q, int W) {
    float x = 0.0f;
    for (int w = W - 1; w >= 0; --w) x = __fmaf_rz(x, 4294967296.0f, __uint2float_rz(q[w]));
    return __float_as_uint(x);
}

template <int W>
__device__ __forceinline__ uint32_t search_key(const uint32_t (&q)[W]) {
    float x = __uint2float_rz(q[W - 1]);
#pragma unroll
    for (int w = W - 2; w >= 0; --w) x = __fmaf_rz(x, 4294967296.0f, __uint2float_rz(q[w]));
    return __float_as_uint(x);
}

constexpr uint32_t kSearchKeyOfOne = 0x3f800000u;  // search_key(1)

__device__ __forceinline__ uint4 load_record(uint32_t addr) {
    uint4 v;
#ifdef PVQ_DEBUG
    if (!debug_table_ok(addr, 16)) return make_uint4(0u, 0u, 0u, 0u);
#endif
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t load_bucket(uint32_t addr) {
    uint32_t v;
#ifdef PVQ_DEBUG
    if (!debug_table_ok(addr, 4)) return 0u;
#endif
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// m0 + (t < q): minus the borrow of t - q, which the last link of the chain leaves as 0 or -1
template <int W>
__device__ __forceinline__ uint32_t bump_if_less(uint32_t m0, const mp<W>& t, const mp<W>& q) {
    uint32_t m;
    if constexpr (W == 1) {
        asm("{\n\t.reg .u32 d;\n\t"
            "sub.cc.u32 d, %2, %3;\n\t"
            "subc.u32 d, 0, 0;\n\t"
            "sub.u32 %0, %1, d;\n\t}"
            : "=r"(m)
            : "r"(m0), "r"(t.w[0]), "r"(q.w[0]));
    } else if constexpr (W == 2) {
        asm("{\n\t.reg .u32 d;\n\t"
            "sub.cc.u32 d, %2, %4;\n\t"
            "subc.cc.u32 d, %3, %5;\n\t"
            "subc.u32 d, 0, 0;\n\t"
            "sub.u32 %0, %1, d;\n\t}"
            : "=r"(m)
            : "r"(m0), "r"(t.w[0]), "r"(t.w[1]), "r"(q.w[0]), "r"(q.w[1]));
    } else if constexpr (W == 3) {
        asm("{\n\t.reg .u32 d;\n\t"
            "sub.cc.u32 d, %2, %5;\n\t"
            "subc.cc.u32 d, %3, %6;\n\t"
            "subc.cc.u32 d, %4, %7;\n\t"
            "subc.u32 d, 0, 0;\n\t"
            "sub.u32 %0, %1, d;\n\t}"
            : "=r"(m)
            : "r"(m0), "r"(t.w[0]), "r"(t.w[1]), "r"(t.w[2]), "r"(q.w[0]), "r"(q.w[1]), "r"(q.w[2]));
    } else {
        static_assert(W == 4, "codes of up to four words");
        asm("{\n\t.reg .u32 d;\n\t"
            "sub.cc.u32 d, %2, %6;\n\t"
            "subc.cc.u32 d, %3, %7;\n\t"
            "subc.cc.u32 d, %4, %8;\n\t"
            "subc.cc.u32 d, %5, %9;\n\t"
            "subc.u32 d, 0, 0;\n\t"
            "sub.u32 %0, %1, d;\n\t}"
            : "=r"(m)
            : "r"(m0), "r"(t.w[0]), "r"(t.w[1]), "r"(t.w[2]), "r"(t.w[3]), "r"(q.w[0]), "r"(q.w[1]), "r"(q.w[2]),
              "r"(q.w[3]));
    }
    return m;
}

// Once the section has arrived in shared memory (at `sec`; `bytes` is its size in the blob): is
// it the section of this (N,K)?  (A table built for another one would send the look-ups
// anywhere.)  If so, the numbers of rows per width go to cnt[1..4] and threads 0..N-1 turn the
// records' offsets into shared addresses; the caller's next block-wide barrier publishes them.
// The thresholds T are not staged (only a 24-bit tie reads one, from global memory): the
// increments E sit where T is in the blob, `t_before_e` bytes lower.
template <int N, int W>
__device__ __forceinline__ bool search_section_begin(uint8_t* sec, uint32_t bytes, uint32_t t_before_e, int K,
                                                     int (&cnt)[5]) {
    const uint32_t* head = reinterpret_cast<const uint32_t*>(sec);
    if (head[0] != kSearchMagic || head[1] != static_cast<uint32_t>(N) || head[2] != static_cast<uint32_t>(K) ||
        head[3] != bytes)
        return false;
    cnt[0] = 0;
#pragma unroll
    for (int w = 1; w <= 4; ++w) cnt[w] = static_cast<int>(head[8 - w]);
    if (cnt[1] + cnt[2] + cnt[3] + cnt[4] != N || ((cnt[1] | cnt[2] | cnt[3] | cnt[4]) & 3) != 0 ||
        (W < 4 && cnt[4] != 0) || (W < 3 && cnt[3] != 0) || (W < 2 && cnt[2] != 0))
        return false;
    if (threadIdx.x < N) {
        uint32_t* rec = reinterpret_cast<uint32_t*>(sec + kSearchHeader) + 4 * threadIdx.x;
        const uint32_t base = shared_addr(sec);
        rec[1] += base - t_before_e;
        rec[2] += base;
    }
    return true;
}

// Entry of PW words of a row stored word plane by word plane (PLANE entries a plane): word w
// sits PLANE words behind word w - 1.  `addr` is the shared address of word 0.
template <int PW, int PLANE>
__device__ __forceinline__ mp<PW> load_planes(uint32_t addr) {
    mp<PW> t;  // the plane offsets go into the loads as immediates
    t.w[0] = load_entry<1, 0>(addr).w[0];
    if constexpr (PW > 1) t.w[1] = load_entry<1, PLANE * 4>(addr).w[0];
    if constexpr (PW > 2) t.w[2] = load_entry<1, 2 * PLANE * 4>(addr).w[0];
    if constexpr (PW > 3) t.w[3] = load_entry<1, 3 * PLANE * 4>(addr).w[0];
    return t;
}

// Four bytes of a thread's slot at once.
__device__ __forceinline__ void store_y4(uint32_t addr, uint32_t val) {
#ifdef PVQ_DEBUG
    if (!debug_slot_ok(addr, 4)) return;
#endif
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
}

// Four positions of GP codes (GP independent chains of dependent table reads, so that one
// thread keeps several reads in flight), in PW-word arithmetic on rows of PW word planes.
// `rec` is the shared address of the record of the first of the four rows (the rows of the
// following positions have the records before it); a record is read once for all chains.
// `t_rows` plus the shared address of a row of E is the global address of the same row of T.
// The four y_i + 128 of chain j go to the word at y + j * ychain.
//
// Per position: the key of q selects a bucket; its entry is m0 and the low key bits of the
// threshold T[m0]; q's own low key bits being larger means q > T[m0], smaller means q <= T[m0]
// (a bucket without a threshold holds all ones there).  Equal bits leave it open: then, and
// that is rare, the threads of the warp whose bits were equal compare q with T[m0] in full.
template <int W, int PW, int GP, int PLANE>
__device__ __forceinline__ void search_block4(mp<W> (&q)[GP], uint32_t (&k)[GP], uint32_t rec, const uint8_t* t_rows,
                                              uint32_t y, uint32_t ychain) {
    uint32_t acc[GP];  // the four threshold indices m, a byte each, first position lowest
    mp<PW> v[GP];      // the low PW words of q: the rest is zero by now
#pragma unroll
    for (int j = 0; j < GP; ++j) {
        acc[j] = 0u;
#pragma unroll
        for (int w = 0; w < PW; ++w) v[j].w[w] = q[j].w[w];
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const uint4 r = load_record(rec - static_cast<uint32_t>(s) * 16u);  // 32 - shift, E row, buckets, shift
        uint32_t key[GP], entry[GP], m[GP];
        mp<PW> e[GP];
        bool open = false;
#pragma unroll
        for (int j = 0; j < GP; ++j) {
            key[j] = search_key<PW>(v[j].w);
            entry[j] = load_bucket(r.z + ((key[j] >> r.w) << 2));
        }
#pragma unroll
        for (int j = 0; j < GP; ++j) {
            const uint32_t x = key[j] << r.x;  // the key bits below the shift, left-aligned like the entry's
            m[j] = (entry[j] & 0xffu) + (x > entry[j] ? 1u : 0u);
            open = open || (entry[j] - x < 256u);
        }
        if (__any_sync(kFull, open)) {
#pragma unroll
            for (int j = 0; j < GP; ++j) {
                const uint32_t m0 = entry[j] & 0xffu;
                if (entry[j] - (key[j] << r.x) < 256u) {
                    // the row of T in global memory lies where the row of E lies in shared memory
                    const uint32_t* tp = reinterpret_cast<const uint32_t*>(t_rows + r.y + m0 * 4u);
                    mp<PW> t;
#pragma unroll
                    for (int w = 0; w < PW; ++w) t.w[w] = tp[w * PLANE];
                    m[j] = bump_if_less<PW>(m0, t, v[j]);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < GP; ++j) e[j] = load_planes<PW, PLANE>(r.y + (m[j] << 2));
#pragma unroll
        for (int j = 0; j < GP; ++j) {
            mp_add<PW>(v[j], e[j]);
            acc[j] = __funnelshift_r(acc[j], m[j], 8);  // the new byte enters at the top
        }
    }
    // From the four indices to the four coordinates, all four bytes of a word at a time:
    // pulses left after a position m >> 1, before it those of the position before (k for the
    // first); their difference is |y|, and y > 0 where m is odd.  No byte borrows from or
    // carries into its neighbour: the pulses left never grow, and |y| <= 127.
#pragma unroll
    for (int j = 0; j < GP; ++j) {
        const uint32_t after = (acc[j] >> 1) & 0x7f7f7f7fu;
        const uint32_t before = (after << 8) | k[j];
        const uint32_t mag = before - after;
        const uint32_t odd = acc[j] & 0x01010101u;
        const uint32_t pos = (odd << 8) - odd;  // 0xff in the bytes with y > 0
        store_y4(y + static_cast<uint32_t>(j) * ychain,
                 ((0x80808080u + mag) & pos) | ((0x80808080u - mag) & ~pos));
        k[j] = after >> 24;
#pragma unroll
        for (int w = 0; w < PW; ++w) q[j].w[w] = v[j].w[w];
    }
}

// The points of GP codes: q = N(N,K) - code on entry.  `recs` is the shared address of the
// row records (absolute shared addresses by now), cnt[w] the number of rows done in w words.
template <int N, int W, int GP, int PLANE>
__device__ __forceinline__ void search_codes(mp<W> (&q)[GP], int K, uint32_t recs, const uint8_t* t_rows,
                                             const int (&cnt)[5], uint32_t y, uint32_t ychain) {
    uint32_t k[GP];
#pragma unroll
    for (int j = 0; j < GP; ++j) k[j] = static_cast<uint32_t>(K);
    uint32_t rec = recs + static_cast<uint32_t>(N - 1) * 16u;
    if constexpr (W >= 4) {
#pragma unroll 1
        for (int b = 0; b < cnt[4]; b += 4, rec -= 64u, y += 4u) search_block4<W, 4, GP, PLANE>(q, k, rec, t_rows, y, ychain);
    }
    if constexpr (W >= 3) {
#pragma unroll 1
        for (int b = 0; b < cnt[3]; b += 4, rec -= 64u, y += 4u) search_block4<W, 3, GP, PLANE>(q, k, rec, t_rows, y, ychain);
    }
    if constexpr (W >= 2) {
#pragma unroll 1
        for (int b = 0; b < cnt[2]; b += 4, rec -= 64u, y += 4u) search_block4<W, 2, GP, PLANE>(q, k, rec, t_rows, y, ychain);
    }
#pragma unroll 1
    for (int b = 0; b < cnt[1]; b += 4, rec -= 64u, y += 4u) search_block4<W, 1, GP, PLANE>(q, k, rec, t_rows, y, ychain);
}

}  // namespace pvq
