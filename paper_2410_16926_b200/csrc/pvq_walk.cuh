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
// r only shrinks, and so do the entries along a path (N(n,k) is monotone in n and k).
// The warp therefore narrows its arithmetic as it goes.  First on the same table: once
// every thread's r and the entry it is about to read leave the two top bits of a narrower
// width free, the steps work on that many words, and with two spare bits the sign of a
// difference tells the comparison.  Then, once every thread has r below 2^62 (2^30), in a
// copy of the loop that works on two-word (one-word) integers and reads a table of that
// width, whose larger entries are replaced by 2^62 (2^30): no r of that phase reaches them.
#pragma once
#include "mp_uint.cuh"
#include "pvq_internal.cuh"

namespace pvq {

constexpr unsigned kFull = 0xffffffffu;

// Shared-memory accesses of the walk by 32-bit shared-window address.
__device__ __forceinline__ uint32_t shared_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Table staging with the bulk-copy engine (TMA, untiled form): thread 0 arms an mbarrier with
// the byte count and issues the copies, global -> shared; the data lands while the block does
// its other set-up, and every thread waits on the barrier before the first table read.
// Source, destination and sizes are multiples of 16 bytes (the table blob's sections are
// 128-byte aligned, the staged region starts the dynamic shared memory).
struct BulkStage {
    uint32_t bar;  // shared address of the mbarrier
};

__device__ __forceinline__ BulkStage bulk_stage_begin(uint64_t* bar_storage) {
    BulkStage st;
    st.bar = shared_addr(bar_storage);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(st.bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    return st;
}

// thread 0 only: announce `total` bytes, then copy the pieces with bulk_stage_copy
__device__ __forceinline__ void bulk_stage_expect(const BulkStage& st, uint32_t total) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(st.bar), "r"(total) : "memory");
}

__device__ __forceinline__ void bulk_stage_copy(const BulkStage& st, void* dst, const void* src, uint32_t bytes) {
    const uint32_t d = shared_addr(dst);
    const uint8_t* s = static_cast<const uint8_t*>(src);
    for (uint32_t off = 0; off < bytes; off += 32768u) {
        const uint32_t n = bytes - off < 32768u ? bytes - off : 32768u;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(d + off),
                     "l"(s + off), "r"(n), "r"(st.bar)
                     : "memory");
    }
}

// every thread: true once the announced bytes have arrived; false if they have not after a
// bounded number of polls (the caller then leaves the kernel instead of spinning)
__device__ __forceinline__ bool bulk_stage_wait(const BulkStage& st) {
    uint32_t done = 0;
    for (int it = 0; it < (1 << 22) && !done; ++it) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(done)
            : "r"(st.bar)
            : "memory");
    }
    return done != 0u;
}

// Entry of PW words at shared address addr + OFF (OFF a compile-time byte offset).
template <int PW, int OFF = 0>
__device__ __forceinline__ mp<PW> load_entry(uint32_t addr) {
    mp<PW> t;
#ifdef PVQ_DEBUG
    {  // checked, word by word (no alignment beyond 4 bytes assumed); an access outside reads as zero
        const bool ok = debug_table_ok(addr + OFF, PW * 4);
#pragma unroll
        for (int w = 0; w < PW; ++w) {
            t.w[w] = 0u;
            if (ok) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(t.w[w]) : "r"(addr + static_cast<uint32_t>(OFF + 4 * w)));
        }
        return t;
    }
#endif
    if constexpr (PW == 1) {
        asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(t.w[0]) : "r"(addr), "n"(OFF));
    } else if constexpr (PW == 2) {
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(t.w[0]), "=r"(t.w[1]) : "r"(addr), "n"(OFF));
    } else if constexpr (PW <= 4) {  // 16-byte entries
        uint32_t v[4];
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4+%5];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                     : "r"(addr), "n"(OFF));
#pragma unroll
        for (int w = 0; w < PW; ++w) t.w[w] = v[w];
    } else {  // 24-byte entries, 8-byte aligned
        uint32_t v[6];
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v[0]), "=r"(v[1]) : "r"(addr), "n"(OFF));
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v[2]), "=r"(v[3]) : "r"(addr), "n"(OFF + 8));
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v[4]), "=r"(v[5]) : "r"(addr), "n"(OFF + 16));
#pragma unroll
        for (int w = 0; w < PW; ++w) t.w[w] = v[w];
    }
    return t;
}

template <typename YT>
__device__ __forceinline__ void store_y(uint32_t addr, int val) {
#ifdef PVQ_DEBUG
    if (!debug_slot_ok(addr, sizeof(YT))) return;
#endif
    if constexpr (sizeof(YT) == 1)
        asm volatile("st.shared.u8 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
    else
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
}

// d = a - b for the narrow phases (1 or 2 words), where the operands leave the two top bits
// free: the sign bit of the top word of d then says whether a < b.
template <int PW>
__device__ __forceinline__ bool sub_negative(mp<PW>& d, const mp<PW>& a, const mp<PW>& b) {
    static_assert(PW == 1 || PW == 2, "narrow phases only");
    if constexpr (PW == 1) {
        d.w[0] = a.w[0] - b.w[0];
    } else {
        asm("sub.cc.u32 %0, %2, %4;\n\t"
            "subc.u32 %1, %3, %5;"
            : "=&r"(d.w[0]), "=&r"(d.w[1])
            : "r"(a.w[0]), "r"(a.w[1]), "r"(b.w[0]), "r"(b.w[1]));
    }
    return static_cast<int>(d.w[PW - 1]) < 0;
}

// State of one thread's walk.
struct Walk {
    int v;        // pulses placed at the current position so far
    uint32_t y;   // shared address of this thread's slot for the current position
    uint32_t y0;  // ... for position 0
};

// What a slot holds for y_i: y_i + 128 in a byte (the store's float conversion then needs no
// sign handling), or y_i itself in 16 bits when K does not fit a byte.
template <typename YT>
constexpr int kSlotBias = sizeof(YT) == 1 ? 128 : 0;

// The two factors of BatchArgs (1 and -1) the walk multiplies by.
struct Factors {
    uint32_t one, minus_one;
};

// One step at the entry U entries to the left of p (the caller moves p left after a block of
// steps; p moves down here when a position ends).  The slot of the current position is
// written at every step; the write of the step that ends the position is the last one.
//
// Generic form (any width, borrow flags), used by the widest phase.
template <int PW, int EB, typename YT, int U>
__device__ __forceinline__ void walk_step_wide(mp<PW>& r, uint32_t& p, int& v, uint32_t& y, const int D) {
    const mp<PW> t = load_entry<PW, -U * EB>(p);
    mp<PW> d2, d1;
    const bool lt1 = mp_sub_borrow<PW>(d2, r, t);   // d2 = r - t
    const bool lt2 = mp_sub_borrow<PW>(d1, d2, t);  // d1 = r - 2t
    const bool placed = v > 0;
    const bool ge1 = !lt1;
    const bool ge2 = ge1 && !lt2 && placed;
    const bool more = ge2 || (ge1 && !placed);  // another pulse at this position
#pragma unroll
    for (int w = 0; w < PW; ++w) r.w[w] = ge2 ? d1.w[w] : (ge1 ? d2.w[w] : r.w[w]);
    store_y<YT>(y, ((ge1 && placed) ? -v : v) + kSlotBias<YT>);
    y += more ? 0u : static_cast<uint32_t>(sizeof(YT));
    p += more ? 0u : static_cast<uint32_t>(D);
    v = more ? v + 1 : 0;
}

// Narrow forms (1 and 2 words, operands below 2^(32 PW - 2) so that the sign of a difference
// is the comparison), written out instruction by instruction.  Moves, the running counters
// and (for one word) the subtractions are multiply-adds by 1 / -1 on the FMA pipe; compares,
// carry chains and predicate logic stay on the integer pipe.
template <int EB, typename YT, int U>
__device__ __forceinline__ void walk_step_1(uint32_t& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                            const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, ng;\n\t"
        ".reg .u32 t, d2, d1, x, val;\n\t"
        "ld.shared.u32 t, [%3+%7];\n\t"
        "mad.lo.u32 d2, t, %5, %0;\n\t"      // r - t
        "mad.lo.u32 d1, t, %5, d2;\n\t"      // r - 2t
        "setp.gt.s32 pl, %1, 0;\n\t"         // a pulse already placed here
        "setp.ge.s32 g1, d2, 0;\n\t"
        "selp.u32 x, d1, d2, pl;\n\t"        // the difference that decides "one more pulse"
        "setp.ge.s32 mo, x, 0;\n\t"
        "and.pred ng, g1, pl;\n\t"           // if the position ends here: negative
        "@g1 mad.lo.u32 %0, d2, %4, 0;\n\t"  // r = d2
        "@mo mad.lo.u32 %0, x, %4, 0;\n\t"   // r = x
        "mad.lo.u32 val, %1, %4, %10;\n\t"     // bias + v
        "@ng mad.lo.u32 val, %1, %5, %10;\n\t" // bias - v
        "st.shared.u%9 [%2], val;\n\t"
        "@!mo add.u32 %2, %2, %8;\n\t"       // next slot
        "@!mo add.u32 %3, %3, %6;\n\t"       // next row
        "mad.lo.u32 %1, %1, %4, %4;\n\t"     // v + 1
        "@!mo mov.u32 %1, 0;\n\t"
        "}"
        : "+r"(r), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * EB), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}

template <int EB, typename YT, int U>
__device__ __forceinline__ void walk_step_2(mp<2>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                            const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, a0, a1, b0, b1, xh, val;\n\t"
        "ld.shared.v2.u32 {t0, t1}, [%4+%8];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"          // d2 = r - t
        "subc.u32 a1, %1, t1;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"          // d1 = r - 2t
        "subc.u32 b1, a1, t1;\n\t"
        "setp.gt.s32 pl, %2, 0;\n\t"
        "setp.ge.s32 g1, a1, 0;\n\t"
        "selp.u32 xh, b1, a1, pl;\n\t"
        "setp.ge.s32 mo, xh, 0;\n\t"
        "and.pred ng, g1, pl;\n\t"
        "and.pred m2, mo, pl;\n\t"
        "@g1 mad.lo.u32 %0, a0, %5, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %5, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %5, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %5, 0;\n\t"
        "mad.lo.u32 val, %2, %5, %11;\n\t"
        "@ng mad.lo.u32 val, %2, %6, %11;\n\t"
        "st.shared.u%10 [%3], val;\n\t"
        "@!mo add.u32 %3, %3, %9;\n\t"
        "@!mo add.u32 %4, %4, %7;\n\t"
        "mad.lo.u32 %2, %2, %5, %5;\n\t"
        "@!mo mov.u32 %2, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * EB), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}

// Widest phase for 3- and 4-word codes (16-byte entries), borrow flags instead of sign bits.
#define PVQ_WIDE_TAIL(R0, NXT)                                                         \
        "setp.gt.s32 pl, %" #R0 ", 0;\n\t"                                            \
        "setp.eq.u32 g1, ab, 0;\n\t"                                                   \
        "or.b32 ob, ab, bb;\n\t"                                                       \
        "selp.u32 ob, ob, ab, pl;\n\t"                                                 \
        "setp.eq.u32 mo, ob, 0;\n\t"                                                   \
        "and.pred ng, g1, pl;\n\t"                                                     \
        "and.pred m2, mo, pl;\n\t"

template <typename YT, int U>
__device__ __forceinline__ void walk_step_w3(mp<3>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                             const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, ab, b0, b1, b2, bb, ob, val;\n\t"
        "ld.shared.v4.u32 {t0, t1, t2, t3}, [%5+%9];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.cc.u32 a2, %2, t2;\n\t"
        "subc.u32 ab, 0, 0;\n\t"               // 0 or -1: r < t
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.cc.u32 b2, a2, t2;\n\t"
        "subc.u32 bb, 0, 0;\n\t"               // r - t < t
        PVQ_WIDE_TAIL(3, 0)
        "@g1 mad.lo.u32 %0, a0, %6, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %6, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %6, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %6, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %6, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %6, 0;\n\t"
        "mad.lo.u32 val, %3, %6, %12;\n\t"
        "@ng mad.lo.u32 val, %3, %7, %12;\n\t"
        "st.shared.u%11 [%4], val;\n\t"
        "@!mo add.u32 %4, %4, %10;\n\t"
        "@!mo add.u32 %5, %5, %8;\n\t"
        "mad.lo.u32 %3, %3, %6, %6;\n\t"
        "@!mo mov.u32 %3, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 16), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}

template <typename YT, int U>
__device__ __forceinline__ void walk_step_w4(mp<4>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                             const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, a3, ab, b0, b1, b2, b3, bb, ob, val;\n\t"
        "ld.shared.v4.u32 {t0, t1, t2, t3}, [%6+%10];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.cc.u32 a2, %2, t2;\n\t"
        "subc.cc.u32 a3, %3, t3;\n\t"
        "subc.u32 ab, 0, 0;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.cc.u32 b2, a2, t2;\n\t"
        "subc.cc.u32 b3, a3, t3;\n\t"
        "subc.u32 bb, 0, 0;\n\t"
        PVQ_WIDE_TAIL(4, 0)
        "@g1 mad.lo.u32 %0, a0, %7, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %7, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %7, 0;\n\t"
        "@g1 mad.lo.u32 %3, a3, %7, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %7, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %7, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %7, 0;\n\t"
        "@m2 mad.lo.u32 %3, b3, %7, 0;\n\t"
        "mad.lo.u32 val, %4, %7, %13;\n\t"
        "@ng mad.lo.u32 val, %4, %8, %13;\n\t"
        "st.shared.u%12 [%5], val;\n\t"
        "@!mo add.u32 %5, %5, %11;\n\t"
        "@!mo add.u32 %6, %6, %9;\n\t"
        "mad.lo.u32 %4, %4, %7, %7;\n\t"
        "@!mo mov.u32 %4, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(r.w[3]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 16), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
// Widest phase for 5- and 6-word codes (24-byte entries; a 5-word code walks with a zero
// sixth word).
template <typename YT, int U>
__device__ __forceinline__ void walk_step_w6(uint32_t (&r)[6], uint32_t& p, int& v, uint32_t& y, const int D,
                                             const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, t4, t5, a0, a1, a2, a3, a4, a5, ab, b0, b1, b2, b3, b4, b5, bb, ob, val;\n\t"
        "ld.shared.v2.u32 {t0, t1}, [%8+%12];\n\t"
        "ld.shared.v2.u32 {t2, t3}, [%8+%13];\n\t"
        "ld.shared.v2.u32 {t4, t5}, [%8+%14];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.cc.u32 a2, %2, t2;\n\t"
        "subc.cc.u32 a3, %3, t3;\n\t"
        "subc.cc.u32 a4, %4, t4;\n\t"
        "subc.cc.u32 a5, %5, t5;\n\t"
        "subc.u32 ab, 0, 0;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.cc.u32 b2, a2, t2;\n\t"
        "subc.cc.u32 b3, a3, t3;\n\t"
        "subc.cc.u32 b4, a4, t4;\n\t"
        "subc.cc.u32 b5, a5, t5;\n\t"
        "subc.u32 bb, 0, 0;\n\t"
        PVQ_WIDE_TAIL(6, 0)
        "@g1 mad.lo.u32 %0, a0, %9, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %9, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %9, 0;\n\t"
        "@g1 mad.lo.u32 %3, a3, %9, 0;\n\t"
        "@g1 mad.lo.u32 %4, a4, %9, 0;\n\t"
        "@g1 mad.lo.u32 %5, a5, %9, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %9, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %9, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %9, 0;\n\t"
        "@m2 mad.lo.u32 %3, b3, %9, 0;\n\t"
        "@m2 mad.lo.u32 %4, b4, %9, 0;\n\t"
        "@m2 mad.lo.u32 %5, b5, %9, 0;\n\t"
        "mad.lo.u32 val, %6, %9, %17;\n\t"
        "@ng mad.lo.u32 val, %6, %10, %17;\n\t"
        "st.shared.u%16 [%7], val;\n\t"
        "@!mo add.u32 %7, %7, %15;\n\t"
        "@!mo add.u32 %8, %8, %11;\n\t"
        "mad.lo.u32 %6, %6, %9, %9;\n\t"
        "@!mo mov.u32 %6, 0;\n\t"
        "}"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 24), "n"(-U * 24 + 8), "n"(-U * 24 + 16), "n"(SZ),
          "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
// Middle phases for 5- and 6-word codes: once every r of the warp and the entry it is about to
// read are below 2^(32 M - 2) the steps work on M = 5, 4, then 3 words (sign-bit compares),
// reading the low words of the 24-byte entries.  The entries along a path never grow (N(n,k)
// is monotone in n and k), so every later entry fits as well.
template <typename YT, int U>
__device__ __forceinline__ void walk_step_4of6(mp<4>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                               const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, a3, b0, b1, b2, b3, xh, val;\n\t"
        "ld.shared.v2.u32 {t0, t1}, [%6+%10];\n\t"
        "ld.shared.v2.u32 {t2, t3}, [%6+%11];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.cc.u32 a2, %2, t2;\n\t"
        "subc.u32 a3, %3, t3;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.cc.u32 b2, a2, t2;\n\t"
        "subc.u32 b3, a3, t3;\n\t"
        "setp.gt.s32 pl, %4, 0;\n\t"
        "setp.ge.s32 g1, a3, 0;\n\t"
        "selp.u32 xh, b3, a3, pl;\n\t"
        "setp.ge.and.s32 mo, xh, 0, g1;\n\t"
        "and.pred ng, g1, pl;\n\t"
        "and.pred m2, mo, pl;\n\t"
        "@g1 mad.lo.u32 %0, a0, %7, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %7, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %7, 0;\n\t"
        "@g1 mad.lo.u32 %3, a3, %7, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %7, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %7, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %7, 0;\n\t"
        "@m2 mad.lo.u32 %3, b3, %7, 0;\n\t"
        "mad.lo.u32 val, %4, %7, %15;\n\t"
        "@ng mad.lo.u32 val, %4, %8, %15;\n\t"
        "st.shared.u%14 [%5], val;\n\t"
        "@!mo add.u32 %5, %5, %13;\n\t"
        "@!mo add.u32 %6, %6, %9;\n\t"
        "mad.lo.u32 %4, %4, %7, %7;\n\t"
        "@!mo mov.u32 %4, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(r.w[3]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 24), "n"(-U * 24 + 8), "n"(-U * 24 + 16), "n"(SZ),
          "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
template <typename YT, int U>
__device__ __forceinline__ void walk_step_5of6(mp<5>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                               const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, t4, t5, a0, a1, a2, a3, a4, b0, b1, b2, b3, b4, xh, val;\n\t"
        "ld.shared.v2.u32 {t0, t1}, [%7+%11];\n\t"
        "ld.shared.v2.u32 {t2, t3}, [%7+%12];\n\t"
        "ld.shared.v2.u32 {t4, t5}, [%7+%13];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.cc.u32 a2, %2, t2;\n\t"
        "subc.cc.u32 a3, %3, t3;\n\t"
        "subc.u32 a4, %4, t4;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.cc.u32 b2, a2, t2;\n\t"
        "subc.cc.u32 b3, a3, t3;\n\t"
        "subc.u32 b4, a4, t4;\n\t"
        "setp.gt.s32 pl, %5, 0;\n\t"
        "setp.ge.s32 g1, a4, 0;\n\t"
        "selp.u32 xh, b4, a4, pl;\n\t"
        "setp.ge.and.s32 mo, xh, 0, g1;\n\t"
        "and.pred ng, g1, pl;\n\t"
        "and.pred m2, mo, pl;\n\t"
        "@g1 mad.lo.u32 %0, a0, %8, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %8, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %8, 0;\n\t"
        "@g1 mad.lo.u32 %3, a3, %8, 0;\n\t"
        "@g1 mad.lo.u32 %4, a4, %8, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %8, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %8, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %8, 0;\n\t"
        "@m2 mad.lo.u32 %3, b3, %8, 0;\n\t"
        "@m2 mad.lo.u32 %4, b4, %8, 0;\n\t"
        "mad.lo.u32 val, %5, %8, %16;\n\t"
        "@ng mad.lo.u32 val, %5, %9, %16;\n\t"
        "st.shared.u%15 [%6], val;\n\t"
        "@!mo add.u32 %6, %6, %14;\n\t"
        "@!mo add.u32 %7, %7, %10;\n\t"
        "mad.lo.u32 %5, %5, %8, %8;\n\t"
        "@!mo mov.u32 %5, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(r.w[3]), "+r"(r.w[4]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 24), "n"(-U * 24 + 8), "n"(-U * 24 + 16), "n"(SZ),
          "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
template <typename YT, int U>
__device__ __forceinline__ void walk_step_3of6(mp<3>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                               const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, b0, b1, b2, xh, val;\n\t"
        "ld.shared.v2.u32 {t0, t1}, [%5+%9];\n\t"
        "ld.shared.v2.u32 {t2, t3}, [%5+%10];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.u32 a2, %2, t2;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.u32 b2, a2, t2;\n\t"
        "setp.gt.s32 pl, %3, 0;\n\t"
        "setp.ge.s32 g1, a2, 0;\n\t"
        "selp.u32 xh, b2, a2, pl;\n\t"
        "setp.ge.and.s32 mo, xh, 0, g1;\n\t"
        "and.pred ng, g1, pl;\n\t"
        "and.pred m2, mo, pl;\n\t"
        "@g1 mad.lo.u32 %0, a0, %6, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %6, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %6, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %6, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %6, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %6, 0;\n\t"
        "mad.lo.u32 val, %3, %6, %14;\n\t"
        "@ng mad.lo.u32 val, %3, %7, %14;\n\t"
        "st.shared.u%13 [%4], val;\n\t"
        "@!mo add.u32 %4, %4, %12;\n\t"
        "@!mo add.u32 %5, %5, %8;\n\t"
        "mad.lo.u32 %3, %3, %6, %6;\n\t"
        "@!mo mov.u32 %3, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 24), "n"(-U * 24 + 8), "n"(-U * 24 + 16), "n"(SZ),
          "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
// The same for 3- and 4-word codes (16-byte entries): three words with sign-bit compares once
// r and the coming entry are below 2^94.
template <typename YT, int U>
__device__ __forceinline__ void walk_step_3of4(mp<3>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                               const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred pl, g1, mo, m2, ng;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, b0, b1, b2, xh, val;\n\t"
        "ld.shared.v4.u32 {t0, t1, t2, t3}, [%5+%9];\n\t"
        "sub.cc.u32 a0, %0, t0;\n\t"
        "subc.cc.u32 a1, %1, t1;\n\t"
        "subc.u32 a2, %2, t2;\n\t"
        "sub.cc.u32 b0, a0, t0;\n\t"
        "subc.cc.u32 b1, a1, t1;\n\t"
        "subc.u32 b2, a2, t2;\n\t"
        "setp.gt.s32 pl, %3, 0;\n\t"
        "setp.ge.s32 g1, a2, 0;\n\t"
        "selp.u32 xh, b2, a2, pl;\n\t"
        "setp.ge.and.s32 mo, xh, 0, g1;\n\t"
        "and.pred ng, g1, pl;\n\t"
        "and.pred m2, mo, pl;\n\t"
        "@g1 mad.lo.u32 %0, a0, %6, 0;\n\t"
        "@g1 mad.lo.u32 %1, a1, %6, 0;\n\t"
        "@g1 mad.lo.u32 %2, a2, %6, 0;\n\t"
        "@m2 mad.lo.u32 %0, b0, %6, 0;\n\t"
        "@m2 mad.lo.u32 %1, b1, %6, 0;\n\t"
        "@m2 mad.lo.u32 %2, b2, %6, 0;\n\t"
        "mad.lo.u32 val, %3, %6, %14;\n\t"
        "@ng mad.lo.u32 val, %3, %7, %14;\n\t"
        "st.shared.u%13 [%4], val;\n\t"
        "@!mo add.u32 %4, %4, %12;\n\t"
        "@!mo add.u32 %5, %5, %8;\n\t"
        "mad.lo.u32 %3, %3, %6, %6;\n\t"
        "@!mo mov.u32 %3, 0;\n\t"
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(-U * 16), "n"(-U * 16 + 8), "n"(-U * 16 + 16), "n"(SZ),
          "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_WIDE_TAIL

// Eight consecutive steps in one asm statement, for the sign-bit forms.  Whether a pulse has
// already been placed at the current position (v > 0) is, from the second step on, the previous
// step's "one more pulse" predicate, so only the first step tests v.  Step u reads the entry
// u entries to the left of p; the caller moves p left by eight entries afterwards.
#define PVQ_STEP_1(OFF, PL, MO) \
    "ld.shared.u32 t, [%3+" #OFF "];\n\t"     \
    "mad.lo.u32 d2, t, %5, %0;\n\t"           \
    "mad.lo.u32 d1, t, %5, d2;\n\t"           \
    "setp.ge.s32 g1, d2, 0;\n\t"              \
    "selp.u32 x, d1, d2, " #PL ";\n\t"        \
    "setp.ge.s32 " #MO ", x, 0;\n\t"          \
    "and.pred ng, g1, " #PL ";\n\t"           \
    "@g1 mad.lo.u32 %0, d2, %4, 0;\n\t"       \
    "@" #MO " mad.lo.u32 %0, x, %4, 0;\n\t"   \
    "mad.lo.u32 val, %1, %4, %9;\n\t"         \
    "@ng mad.lo.u32 val, %1, %5, %9;\n\t"     \
    "st.shared.u%8 [%2], val;\n\t"            \
    "@!" #MO " add.u32 %2, %2, %7;\n\t"       \
    "@!" #MO " add.u32 %3, %3, %6;\n\t"       \
    "mad.lo.u32 %1, %1, %4, %4;\n\t"          \
    "@!" #MO " mov.u32 %1, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_1(uint32_t& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t, d2, d1, x, val;\n\t"
        "setp.gt.s32 pl0, %1, 0;\n\t"
        PVQ_STEP_1(0, pl0, mo0)
        PVQ_STEP_1(-4, mo0, mo1)
        PVQ_STEP_1(-8, mo1, mo2)
        PVQ_STEP_1(-12, mo2, mo3)
        PVQ_STEP_1(-16, mo3, mo4)
        PVQ_STEP_1(-20, mo4, mo5)
        PVQ_STEP_1(-24, mo5, mo6)
        PVQ_STEP_1(-28, mo6, mo7)
        "}"
        : "+r"(r), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_1

#define PVQ_STEP_2(OFF, PL, MO) \
    "ld.shared.v2.u32 {t0, t1}, [%4+" #OFF "];\n\t"   \
    "sub.cc.u32 a0, %0, t0;\n\t"                      \
    "subc.u32 a1, %1, t1;\n\t"                        \
    "sub.cc.u32 b0, a0, t0;\n\t"                      \
    "subc.u32 b1, a1, t1;\n\t"                        \
    "setp.ge.s32 g1, a1, 0;\n\t"                      \
    "selp.u32 xh, b1, a1, " #PL ";\n\t"               \
    "setp.ge.and.s32 " #MO ", xh, 0, g1;\n\t"         \
    "and.pred ng, g1, " #PL ";\n\t"                   \
    "and.pred m2, " #MO ", " #PL ";\n\t"              \
    "@g1 mad.lo.u32 %0, a0, %5, 0;\n\t"               \
    "@g1 mad.lo.u32 %1, a1, %5, 0;\n\t"               \
    "@m2 mad.lo.u32 %0, b0, %5, 0;\n\t"               \
    "@m2 mad.lo.u32 %1, b1, %5, 0;\n\t"               \
    "mad.lo.u32 val, %2, %5, %10;\n\t"                \
    "@ng mad.lo.u32 val, %2, %6, %10;\n\t"            \
    "st.shared.u%9 [%3], val;\n\t"                    \
    "@!" #MO " add.u32 %3, %3, %8;\n\t"               \
    "@!" #MO " add.u32 %4, %4, %7;\n\t"               \
    "mad.lo.u32 %2, %2, %5, %5;\n\t"                  \
    "@!" #MO " mov.u32 %2, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_2(mp<2>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t0, t1, a0, a1, b0, b1, xh, val;\n\t"
        "setp.gt.s32 pl0, %2, 0;\n\t"
        PVQ_STEP_2(0, pl0, mo0)
        PVQ_STEP_2(-8, mo0, mo1)
        PVQ_STEP_2(-16, mo1, mo2)
        PVQ_STEP_2(-24, mo2, mo3)
        PVQ_STEP_2(-32, mo3, mo4)
        PVQ_STEP_2(-40, mo4, mo5)
        PVQ_STEP_2(-48, mo5, mo6)
        PVQ_STEP_2(-56, mo6, mo7)
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_2

#define PVQ_STEP_3OF4(OFF, PL, MO) \
    "ld.shared.v4.u32 {t0, t1, t2, t3}, [%5+" #OFF "];\n\t"   \
    "sub.cc.u32 a0, %0, t0;\n\t"                              \
    "subc.cc.u32 a1, %1, t1;\n\t"                             \
    "subc.u32 a2, %2, t2;\n\t"                                \
    "sub.cc.u32 b0, a0, t0;\n\t"                              \
    "subc.cc.u32 b1, a1, t1;\n\t"                             \
    "subc.u32 b2, a2, t2;\n\t"                                \
    "setp.ge.s32 g1, a2, 0;\n\t"                              \
    "selp.u32 xh, b2, a2, " #PL ";\n\t"                       \
    "setp.ge.and.s32 " #MO ", xh, 0, g1;\n\t"                 \
    "and.pred ng, g1, " #PL ";\n\t"                           \
    "and.pred m2, " #MO ", " #PL ";\n\t"                      \
    "@g1 mad.lo.u32 %0, a0, %6, 0;\n\t"                       \
    "@g1 mad.lo.u32 %1, a1, %6, 0;\n\t"                       \
    "@g1 mad.lo.u32 %2, a2, %6, 0;\n\t"                       \
    "@m2 mad.lo.u32 %0, b0, %6, 0;\n\t"                       \
    "@m2 mad.lo.u32 %1, b1, %6, 0;\n\t"                       \
    "@m2 mad.lo.u32 %2, b2, %6, 0;\n\t"                       \
    "mad.lo.u32 val, %3, %6, %11;\n\t"                        \
    "@ng mad.lo.u32 val, %3, %7, %11;\n\t"                    \
    "st.shared.u%10 [%4], val;\n\t"                           \
    "@!" #MO " add.u32 %4, %4, %9;\n\t"                       \
    "@!" #MO " add.u32 %5, %5, %8;\n\t"                       \
    "mad.lo.u32 %3, %3, %6, %6;\n\t"                          \
    "@!" #MO " mov.u32 %3, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_3of4(mp<3>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t0, t1, t2, t3, a0, a1, a2, b0, b1, b2, xh, val;\n\t"
        "setp.gt.s32 pl0, %3, 0;\n\t"
        PVQ_STEP_3OF4(0, pl0, mo0)
        PVQ_STEP_3OF4(-16, mo0, mo1)
        PVQ_STEP_3OF4(-32, mo1, mo2)
        PVQ_STEP_3OF4(-48, mo2, mo3)
        PVQ_STEP_3OF4(-64, mo3, mo4)
        PVQ_STEP_3OF4(-80, mo4, mo5)
        PVQ_STEP_3OF4(-96, mo5, mo6)
        PVQ_STEP_3OF4(-112, mo6, mo7)
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_3OF4

#define PVQ_STEP_3OF6(OFF, OFF8, OFF16, PL, MO) \
    "ld.shared.v2.u32 {t0, t1}, [%5+" #OFF "];\n\t"    \
    "ld.shared.v2.u32 {t2, t3}, [%5+" #OFF8 "];\n\t"   \
    "sub.cc.u32 a0, %0, t0;\n\t"                       \
    "subc.cc.u32 a1, %1, t1;\n\t"                      \
    "subc.u32 a2, %2, t2;\n\t"                         \
    "sub.cc.u32 b0, a0, t0;\n\t"                       \
    "subc.cc.u32 b1, a1, t1;\n\t"                      \
    "subc.u32 b2, a2, t2;\n\t"                         \
    "setp.ge.s32 g1, a2, 0;\n\t"                       \
    "selp.u32 xh, b2, a2, " #PL ";\n\t"                \
    "setp.ge.and.s32 " #MO ", xh, 0, g1;\n\t"          \
    "and.pred ng, g1, " #PL ";\n\t"                    \
    "and.pred m2, " #MO ", " #PL ";\n\t"               \
    "@g1 mad.lo.u32 %0, a0, %6, 0;\n\t"                \
    "@g1 mad.lo.u32 %1, a1, %6, 0;\n\t"                \
    "@g1 mad.lo.u32 %2, a2, %6, 0;\n\t"                \
    "@m2 mad.lo.u32 %0, b0, %6, 0;\n\t"                \
    "@m2 mad.lo.u32 %1, b1, %6, 0;\n\t"                \
    "@m2 mad.lo.u32 %2, b2, %6, 0;\n\t"                \
    "mad.lo.u32 val, %3, %6, %11;\n\t"                 \
    "@ng mad.lo.u32 val, %3, %7, %11;\n\t"             \
    "st.shared.u%10 [%4], val;\n\t"                    \
    "@!" #MO " add.u32 %4, %4, %9;\n\t"                \
    "@!" #MO " add.u32 %5, %5, %8;\n\t"                \
    "mad.lo.u32 %3, %3, %6, %6;\n\t"                   \
    "@!" #MO " mov.u32 %3, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_3of6(mp<3>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t0, t1, t2, t3, t4, t5, a0, a1, a2, b0, b1, b2, xh, val;\n\t"
        "setp.gt.s32 pl0, %3, 0;\n\t"
        PVQ_STEP_3OF6(0, 8, 16, pl0, mo0)
        PVQ_STEP_3OF6(-24, -16, -8, mo0, mo1)
        PVQ_STEP_3OF6(-48, -40, -32, mo1, mo2)
        PVQ_STEP_3OF6(-72, -64, -56, mo2, mo3)
        PVQ_STEP_3OF6(-96, -88, -80, mo3, mo4)
        PVQ_STEP_3OF6(-120, -112, -104, mo4, mo5)
        PVQ_STEP_3OF6(-144, -136, -128, mo5, mo6)
        PVQ_STEP_3OF6(-168, -160, -152, mo6, mo7)
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_3OF6

#define PVQ_STEP_4OF6(OFF, OFF8, OFF16, PL, MO) \
    "ld.shared.v2.u32 {t0, t1}, [%6+" #OFF "];\n\t"    \
    "ld.shared.v2.u32 {t2, t3}, [%6+" #OFF8 "];\n\t"   \
    "sub.cc.u32 a0, %0, t0;\n\t"                       \
    "subc.cc.u32 a1, %1, t1;\n\t"                      \
    "subc.cc.u32 a2, %2, t2;\n\t"                      \
    "subc.u32 a3, %3, t3;\n\t"                         \
    "sub.cc.u32 b0, a0, t0;\n\t"                       \
    "subc.cc.u32 b1, a1, t1;\n\t"                      \
    "subc.cc.u32 b2, a2, t2;\n\t"                      \
    "subc.u32 b3, a3, t3;\n\t"                         \
    "setp.ge.s32 g1, a3, 0;\n\t"                       \
    "selp.u32 xh, b3, a3, " #PL ";\n\t"                \
    "setp.ge.and.s32 " #MO ", xh, 0, g1;\n\t"          \
    "and.pred ng, g1, " #PL ";\n\t"                    \
    "and.pred m2, " #MO ", " #PL ";\n\t"               \
    "@g1 mad.lo.u32 %0, a0, %7, 0;\n\t"                \
    "@g1 mad.lo.u32 %1, a1, %7, 0;\n\t"                \
    "@g1 mad.lo.u32 %2, a2, %7, 0;\n\t"                \
    "@g1 mad.lo.u32 %3, a3, %7, 0;\n\t"                \
    "@m2 mad.lo.u32 %0, b0, %7, 0;\n\t"                \
    "@m2 mad.lo.u32 %1, b1, %7, 0;\n\t"                \
    "@m2 mad.lo.u32 %2, b2, %7, 0;\n\t"                \
    "@m2 mad.lo.u32 %3, b3, %7, 0;\n\t"                \
    "mad.lo.u32 val, %4, %7, %12;\n\t"                 \
    "@ng mad.lo.u32 val, %4, %8, %12;\n\t"             \
    "st.shared.u%11 [%5], val;\n\t"                    \
    "@!" #MO " add.u32 %5, %5, %10;\n\t"               \
    "@!" #MO " add.u32 %6, %6, %9;\n\t"                \
    "mad.lo.u32 %4, %4, %7, %7;\n\t"                   \
    "@!" #MO " mov.u32 %4, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_4of6(mp<4>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t0, t1, t2, t3, t4, t5, a0, a1, a2, a3, b0, b1, b2, b3, xh, val;\n\t"
        "setp.gt.s32 pl0, %4, 0;\n\t"
        PVQ_STEP_4OF6(0, 8, 16, pl0, mo0)
        PVQ_STEP_4OF6(-24, -16, -8, mo0, mo1)
        PVQ_STEP_4OF6(-48, -40, -32, mo1, mo2)
        PVQ_STEP_4OF6(-72, -64, -56, mo2, mo3)
        PVQ_STEP_4OF6(-96, -88, -80, mo3, mo4)
        PVQ_STEP_4OF6(-120, -112, -104, mo4, mo5)
        PVQ_STEP_4OF6(-144, -136, -128, mo5, mo6)
        PVQ_STEP_4OF6(-168, -160, -152, mo6, mo7)
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(r.w[3]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_4OF6

#define PVQ_STEP_5OF6(OFF, OFF8, OFF16, PL, MO) \
    "ld.shared.v2.u32 {t0, t1}, [%7+" #OFF "];\n\t"     \
    "ld.shared.v2.u32 {t2, t3}, [%7+" #OFF8 "];\n\t"    \
    "ld.shared.v2.u32 {t4, t5}, [%7+" #OFF16 "];\n\t"   \
    "sub.cc.u32 a0, %0, t0;\n\t"                        \
    "subc.cc.u32 a1, %1, t1;\n\t"                       \
    "subc.cc.u32 a2, %2, t2;\n\t"                       \
    "subc.cc.u32 a3, %3, t3;\n\t"                       \
    "subc.u32 a4, %4, t4;\n\t"                          \
    "sub.cc.u32 b0, a0, t0;\n\t"                        \
    "subc.cc.u32 b1, a1, t1;\n\t"                       \
    "subc.cc.u32 b2, a2, t2;\n\t"                       \
    "subc.cc.u32 b3, a3, t3;\n\t"                       \
    "subc.u32 b4, a4, t4;\n\t"                          \
    "setp.ge.s32 g1, a4, 0;\n\t"                        \
    "selp.u32 xh, b4, a4, " #PL ";\n\t"                 \
    "setp.ge.and.s32 " #MO ", xh, 0, g1;\n\t"           \
    "and.pred ng, g1, " #PL ";\n\t"                     \
    "and.pred m2, " #MO ", " #PL ";\n\t"                \
    "@g1 mad.lo.u32 %0, a0, %8, 0;\n\t"                 \
    "@g1 mad.lo.u32 %1, a1, %8, 0;\n\t"                 \
    "@g1 mad.lo.u32 %2, a2, %8, 0;\n\t"                 \
    "@g1 mad.lo.u32 %3, a3, %8, 0;\n\t"                 \
    "@g1 mad.lo.u32 %4, a4, %8, 0;\n\t"                 \
    "@m2 mad.lo.u32 %0, b0, %8, 0;\n\t"                 \
    "@m2 mad.lo.u32 %1, b1, %8, 0;\n\t"                 \
    "@m2 mad.lo.u32 %2, b2, %8, 0;\n\t"                 \
    "@m2 mad.lo.u32 %3, b3, %8, 0;\n\t"                 \
    "@m2 mad.lo.u32 %4, b4, %8, 0;\n\t"                 \
    "mad.lo.u32 val, %5, %8, %13;\n\t"                  \
    "@ng mad.lo.u32 val, %5, %9, %13;\n\t"              \
    "st.shared.u%12 [%6], val;\n\t"                     \
    "@!" #MO " add.u32 %6, %6, %11;\n\t"                \
    "@!" #MO " add.u32 %7, %7, %10;\n\t"                \
    "mad.lo.u32 %5, %5, %8, %8;\n\t"                    \
    "@!" #MO " mov.u32 %5, 0;\n\t"
template <typename YT>
__device__ __forceinline__ void walk_block8_5of6(mp<5>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                                const Factors f) {
    constexpr int SZ = static_cast<int>(sizeof(YT));
    asm volatile(
        "{\n\t"
        ".reg .pred g1, m2, ng, pl0, mo0, mo1, mo2, mo3, mo4, mo5, mo6, mo7;\n\t"
        ".reg .u32 t0, t1, t2, t3, t4, t5, a0, a1, a2, a3, a4, b0, b1, b2, b3, b4, xh, val;\n\t"
        "setp.gt.s32 pl0, %5, 0;\n\t"
        PVQ_STEP_5OF6(0, 8, 16, pl0, mo0)
        PVQ_STEP_5OF6(-24, -16, -8, mo0, mo1)
        PVQ_STEP_5OF6(-48, -40, -32, mo1, mo2)
        PVQ_STEP_5OF6(-72, -64, -56, mo2, mo3)
        PVQ_STEP_5OF6(-96, -88, -80, mo3, mo4)
        PVQ_STEP_5OF6(-120, -112, -104, mo4, mo5)
        PVQ_STEP_5OF6(-144, -136, -128, mo5, mo6)
        PVQ_STEP_5OF6(-168, -160, -152, mo6, mo7)
        "}"
        : "+r"(r.w[0]), "+r"(r.w[1]), "+r"(r.w[2]), "+r"(r.w[3]), "+r"(r.w[4]), "+r"(v), "+r"(y), "+r"(p)
        : "r"(f.one), "r"(f.minus_one), "r"(D), "n"(SZ), "n"(SZ * 8), "n"(kSlotBias<YT>)
        : "memory");
}
#undef PVQ_STEP_5OF6

template <int PW, int EB, bool HEADROOM, typename YT, int U>
__device__ __forceinline__ void walk_step(mp<PW>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                          const Factors f) {
#ifdef PVQ_DEBUG
    walk_step_wide<PW, EB, YT, U>(r, p, v, y, D);  // the plain step: every access through the checked helpers
    return;
#endif
    if constexpr (HEADROOM && PW == 1)
        walk_step_1<EB, YT, U>(r.w[0], p, v, y, D, f);
    else if constexpr (HEADROOM && PW == 2)
        walk_step_2<EB, YT, U>(r, p, v, y, D, f);
    else if constexpr (HEADROOM && PW == 5 && EB == 24)
        walk_step_5of6<YT, U>(r, p, v, y, D, f);
    else if constexpr (HEADROOM && PW == 4 && EB == 24)
        walk_step_4of6<YT, U>(r, p, v, y, D, f);
    else if constexpr (HEADROOM && PW == 3 && EB == 24)
        walk_step_3of6<YT, U>(r, p, v, y, D, f);
    else if constexpr (HEADROOM && PW == 3 && EB == 16)
        walk_step_3of4<YT, U>(r, p, v, y, D, f);
    else if constexpr (!HEADROOM && PW == 3)
        walk_step_w3<YT, U>(r, p, v, y, D, f);
    else if constexpr (!HEADROOM && PW == 4)
        walk_step_w4<YT, U>(r, p, v, y, D, f);
    else if constexpr (!HEADROOM && PW == 6)
        walk_step_w6<YT, U>(r.w, p, v, y, D, f);
    else if constexpr (!HEADROOM && PW == 5) {
        uint32_t r6[6] = {r.w[0], r.w[1], r.w[2], r.w[3], r.w[4], 0u};
        walk_step_w6<YT, U>(r6, p, v, y, D, f);
#pragma unroll
        for (int w = 0; w < 5; ++w) r.w[w] = r6[w];
    } else
        walk_step_wide<PW, EB, YT, U>(r, p, v, y, D);
}

// Eight steps: one block where the form has one, else eight single steps.
template <int PW, int EB, bool HEADROOM, typename YT>
__device__ __forceinline__ void walk_block8(mp<PW>& r, uint32_t& p, int& v, uint32_t& y, const int D,
                                            const Factors f) {
#ifdef PVQ_DEBUG
    if constexpr (true) {
        walk_step<PW, EB, HEADROOM, YT, 0>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 1>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 2>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 3>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 4>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 5>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 6>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 7>(r, p, v, y, D, f);
        return;
    }
#endif
    if constexpr (HEADROOM && PW == 1) {
        walk_block8_1<YT>(r.w[0], p, v, y, D, f);
    } else if constexpr (HEADROOM && PW == 2 && EB == 8) {
        walk_block8_2<YT>(r, p, v, y, D, f);
    } else if constexpr (HEADROOM && PW == 3 && EB == 16) {
        walk_block8_3of4<YT>(r, p, v, y, D, f);
    } else if constexpr (HEADROOM && PW == 3 && EB == 24) {
        walk_block8_3of6<YT>(r, p, v, y, D, f);
    } else if constexpr (HEADROOM && PW == 4 && EB == 24) {
        walk_block8_4of6<YT>(r, p, v, y, D, f);
    } else if constexpr (HEADROOM && PW == 5 && EB == 24) {
        walk_block8_5of6<YT>(r, p, v, y, D, f);
    } else {
        walk_step<PW, EB, HEADROOM, YT, 0>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 1>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 2>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 3>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 4>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 5>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 6>(r, p, v, y, D, f);
        walk_step<PW, EB, HEADROOM, YT, 7>(r, p, v, y, D, f);
    }
}

// Runs steps s .. S-1 on PW-word integers with the table `tab` (entries of EB bytes),
// leaving early, at a multiple of 8 steps, once every thread can go on in `next_words` words.
// Returns the step reached.
template <int PW, int EB, bool HEADROOM, bool NEXT_SAME, int CW, typename YT>
__device__ __forceinline__ int walk_phase(mp<CW>& rfull, Walk& st, uint32_t tab, int rowlen, int K, int s,
                                          const int S, const int next_words, const Factors f) {
    mp<PW> r;
#pragma unroll
    for (int w = 0; w < PW; ++w) r.w[w] = rfull.w[w];
    const int D = (rowlen + 1) * EB;                   // one step down and one right
    const int i0 = static_cast<int>(st.y - st.y0) / static_cast<int>(sizeof(YT));  // position reached
    uint32_t p = tab + i0 * D + (K - s) * EB;          // entry (i, col) of this step
    int v = st.v;
    uint32_t y = st.y;

    while (s + 8 <= S) {
        if (next_words > 0) {
            // can every thread go on in next_words words?  On a narrow table with its large values
            // saturated: when r has the two top bits of that width clear.  NEXT_SAME, on this
            // table with sign-bit compares: when r and the entry of the coming step have them clear.
            uint32_t hi = 0;
            if constexpr (NEXT_SAME) {
                const mp<EB / 4> t = load_entry<EB / 4, 0>(p);
#pragma unroll
                for (int w = 0; w < EB / 4; ++w) {
                    const uint32_t rw = w < PW ? r.w[w < PW ? w : 0] : 0u;
                    if (w >= next_words) hi |= rw | t.w[w];
                    if (w == next_words - 1) hi |= (rw | t.w[w]) >> 30;
                }
            } else {
#pragma unroll
                for (int w = 2; w < PW; ++w) hi |= r.w[w];
                if constexpr (PW > 1) hi |= next_words == 2 ? (r.w[1] >> 30) : r.w[1];
                if (next_words == 1) hi |= r.w[0] >> 30;
            }
            if (__all_sync(kFull, hi == 0u)) break;
        }
        walk_block8<PW, EB, HEADROOM, YT>(r, p, v, y, D, f);
        p -= 8 * EB;
        s += 8;
    }
    if (next_words == 0 || s + 8 > S) {
        for (; s < S; ++s) {
            walk_step<PW, EB, HEADROOM, YT, 0>(r, p, v, y, D, f);
            p -= EB;
        }
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
    Factors f;
};

// `phases`: how many of the walk tables are staged, in the blob's order (widest, two-word,
// one-word): 1, 2 or 3; or 4 = the widest and the one-word table only, the one-word table
// directly behind the widest (when the two-word table does not fit beside them).
__device__ __forceinline__ WalkTables walk_tables(const TableLayout& L, uint32_t smem_base, int phases,
                                                  const BatchArgs& a) {
    WalkTables t;
    t.tab0 = smem_base;
    t.tab2 = smem_base + (L.walk_off[1] - L.walk_off[0]);
    t.tab1 = phases == 4 ? smem_base + ((L.walk_bytes[0] + 127u) & ~127u) : smem_base + (L.walk_off[2] - L.walk_off[0]);
    t.has2 = (phases == 2 || phases == 3) && L.walk_bytes[1] != 0;
    t.has1 = phases >= 3;
    t.rowlen = L.rowlen;
    t.f.one = a.c_one;
    t.f.minus_one = a.c_minus_one;
    return t;
}

__host__ __device__ inline uint32_t walk_tables_bytes(const TableLayout& L, int phases) {
    if (phases == 4) return ((L.walk_bytes[0] + 127u) & ~127u) + L.walk_bytes[2];
    return L.walk_off[phases - 1] + L.walk_bytes[phases - 1] - L.walk_off[0];
}

// Which walk tables fit in `room` bytes of shared memory (see walk_tables for the codes): all
// three, the widest two, the widest and the one-word one, the widest alone; 0 when not even that.
inline int walk_phases_that_fit(const TableLayout& L, size_t room) {
    const int order[4] = {3, 2, 4, 1};
    for (int p : order) {
        if (p == 3 && L.walk_bytes[2] == 0) continue;  // one-word codes: the widest table is all there is
        if (p == 2 && L.walk_bytes[1] == 0) continue;  // no two-word copy (codes of one or two words)
        if (p == 4 && (L.walk_bytes[1] == 0 || L.walk_bytes[2] == 0)) continue;  // 3 covers these
        if (((walk_tables_bytes(L, p) + 15u) & ~size_t(15)) <= room) return p;
    }
    return 0;
}

// Stages the chosen walk tables at `dst` (thread 0 only, between bulk_stage_expect and the wait).
__device__ __forceinline__ void walk_tables_stage(const BulkStage& st, void* dst, const uint32_t* blob,
                                                  const TableLayout& L, int phases) {
    const uint8_t* src = reinterpret_cast<const uint8_t*>(blob);
    if (phases == 4) {
        bulk_stage_copy(st, dst, src + L.walk_off[0], L.walk_bytes[0]);
        bulk_stage_copy(st, static_cast<uint8_t*>(dst) + ((L.walk_bytes[0] + 127u) & ~127u), src + L.walk_off[2],
                        L.walk_bytes[2]);
    } else {
        bulk_stage_copy(st, dst, src + L.walk_off[0], walk_tables_bytes(L, phases));
    }
}
__host__ __device__ inline uint32_t walk_tables_stage_bytes(const TableLayout& L, int phases) {
    return phases == 4 ? L.walk_bytes[0] + L.walk_bytes[2] : walk_tables_bytes(L, phases);
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
    const int narrow = t.has2 ? 2 : (t.has1 ? 1 : 0);
    // widest phase, then fewer words (or, for two-word codes, the same two) with sign-bit
    // compares on the same table as r shrinks
    constexpr int kSame = W > 5 ? 5 : (W > 4 ? 4 : (W > 2 ? 3 : (W == 2 ? 2 : 0)));
    if constexpr (kSame > 0)
        s = walk_phase<W, TW * 4, false, true, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, kSame, t.f);
    else
        s = walk_phase<W, TW * 4, false, false, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, narrow, t.f);
    if constexpr (W == 2) {
        if (s < S) s = walk_phase<2, 8, true, false, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, narrow, t.f);
    }
    if constexpr (W == 3 || W == 4) {
        if (s < S) s = walk_phase<3, 16, true, false, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, narrow, t.f);
    }
    if constexpr (W > 4) {
        if constexpr (W > 5) {
            if (s < S) s = walk_phase<5, 24, true, true, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, 4, t.f);
        }
        if (s < S) s = walk_phase<4, 24, true, true, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, 3, t.f);
        if (s < S) s = walk_phase<3, 24, true, false, W, YT>(c, st, t.tab0, t.rowlen, K, s, S, narrow, t.f);
    }
    if constexpr (W > 2) {
        if (s < S && t.has2) s = walk_phase<2, 8, true, false, W, YT>(c, st, t.tab2, t.rowlen, K, s, S, t.has1 ? 1 : 0, t.f);
    }
    if constexpr (W > 1) {
        if (s < S && t.has1) s = walk_phase<1, 4, true, false, W, YT>(c, st, t.tab1, t.rowlen, K, s, S, 0, t.f);
    }
}

// After walk_code: scale this thread's point to the unit sphere times `amp` and write its N
// values as bf16 with 16-byte stores (row `row`, group `g` of matrix m).  Each thread writes
// its own N*2 contiguous bytes; the threads of a warp hold consecutive groups, so a warp
// fills a contiguous stretch of the row.
template <int N, typename YT>
__device__ __forceinline__ void emit_group(const MatrixArgs& m, const YT* yslots, float amp, unsigned row,
                                           unsigned g) {
    const uint32_t* y4 = reinterpret_cast<const uint32_t*>(yslots);
    int ssy = 0;
    if constexpr (sizeof(YT) == 1) {
        // slots hold b = y + 128:  sum y^2 = sum b^2 - 256 sum b + 128^2 N
        unsigned sq = 0, su = 0;
#pragma unroll
        for (int v = 0; v < N / 4; ++v) {
            sq = __dp4a(y4[v], y4[v], sq);
            su = __dp4a(y4[v], 0x01010101u, su);
        }
        ssy = static_cast<int>(sq) - 256 * static_cast<int>(su) + 16384 * N;
    } else {
#pragma unroll 8
        for (int v = 0; v < N; ++v) ssy += static_cast<int>(yslots[v]) * static_cast<int>(yslots[v]);
    }
    const float sc = __fdiv_rn(amp, __fsqrt_rn(static_cast<float>(ssy)));
    if (!PVQ_DEBUG_INDEX(static_cast<long long>(row), m.rows, PVQ_DEBUG_GLOBAL_STORE) ||
        !PVQ_DEBUG_INDEX(static_cast<long long>(g + 1) * N - 1, m.cols, PVQ_DEBUG_GLOBAL_STORE))
        return;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.out) + static_cast<size_t>(row) * m.ld_out +
                                          static_cast<size_t>(g) * N);
#pragma unroll
    for (int q = 0; q < N / 8; ++q) {
        float f[8];
        if constexpr (sizeof(YT) == 1) {
            // byte b into the low mantissa bits of 2^23: the float 2^23 + b, then minus 2^23 + 128
            const uint32_t lo = y4[2 * q], hi = y4[2 * q + 1];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                f[e] = __fsub_rn(__uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7540u + e)), 8388736.0f);
                f[4 + e] = __fsub_rn(__uint_as_float(__byte_perm(hi, 0x4B000000u, 0x7540u + e)), 8388736.0f);
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = static_cast<float>(static_cast<int>(yslots[8 * q + e]));
        }
        uint4 o;
        o.x = pack_bf16x2(__fmul_rn(f[0], sc), __fmul_rn(f[1], sc));
        o.y = pack_bf16x2(__fmul_rn(f[2], sc), __fmul_rn(f[3], sc));
        o.z = pack_bf16x2(__fmul_rn(f[4], sc), __fmul_rn(f[5], sc));
        o.w = pack_bf16x2(__fmul_rn(f[6], sc), __fmul_rn(f[7], sc));
        dst[q] = o;
    }
}

}  // namespace pvq
