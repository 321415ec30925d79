// Decode kernel for codes of up to four words and up to 127 pulses: direction code ->
// pyramid point (Algorithm 3) -> unit sphere times dequantised amplitude -> bf16
// (Sec. 2.4, Sec. 3.4), one thread per group, N steps per group instead of the N + K of
// the lockstep walk (pvq_walk.cuh).
//
// Algorithm 3 finds the coordinate of a position by subtracting N(n,k), 2 N(n,k-1),
// 2 N(n,k-2), ... from the remainder r until it no longer fits.  Written with the cumulative
// counts of App. C.2 and q = N(n+1,k) - r, that loop is a search for q among the sorted
// thresholds of row n, which do not depend on k (SearchLayout in pvq_internal.cuh): the first
// threshold index m with T_n[m] >= q gives the pulses left after the position (m >> 1) and
// the sign (m odd: positive), and q + E_n[m] is the q of the next position.  The search is one
// table look-up and one multi-word compare: the leading bits of q, as an fp32 key shifted
// by a per-row amount, select a bucket whose byte entry is the first index that can be
// right, and the buckets are fine enough that the only other candidate is the next index.
//
// All threads of a warp are at the same position, so nothing diverges; table reads of a warp
// go to one row (neighbouring entries for similar q).  Threads collect their point in shared
// memory, then scale it and write N bf16 values with 16-byte stores (emit_group).
#include <algorithm>
#include <cmath>

#include <cuda_fp16.h>

#include "pvq_search.cuh"
#include "pvq_walk.cuh"

namespace pvq {

namespace {

constexpr int kSearchThreads = 1024;

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

// Four bytes of a thread's slot at once.
__device__ __forceinline__ void store_y4(uint32_t addr, uint32_t val) {
#ifdef PVQ_DEBUG
    if (!debug_slot_ok(addr, 4)) return;
#endif
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(val) : "memory");
}

// Four positions of GP codes (GP independent chains of dependent table reads, so that one
// thread keeps several reads in flight), in PW-word arithmetic on rows stored PW words wide.
// `rec` is the shared address of the record of the first of the four rows (the rows of the
// following positions have the records before it); a record is read once for all chains.
// The four y_i + 128 of chain j go to the word at y + j * ychain.
//
// Per position: the key of q selects a bucket; its entry is m0 and the low key bits of the
// threshold T[m0]; q's own low key bits being larger means q > T[m0], smaller means q <= T[m0]
// (a bucket without a threshold holds all ones there).  Equal bits leave it open: then, and
// that is rare, the threads of the warp whose bits were equal compare q with T[m0] in full.
template <int W, int PW, int GP>
__device__ __forceinline__ void search_block4(mp<W> (&q)[GP], uint32_t (&k)[GP], uint32_t rec, uint32_t t_before_e,
                                              uint32_t y, uint32_t ychain) {
    constexpr int EB = search_entry_words(PW) * 4;  // bytes of an entry of T and E
    uint32_t acc[GP];
    mp<PW> v[GP];  // the low PW words of q: the rest is zero by now
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
                if (entry[j] - (key[j] << r.x) < 256u)
                    m[j] = bump_if_less<PW>(m0, load_entry<PW>(r.y - t_before_e + m0 * EB), v[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < GP; ++j) e[j] = load_entry<PW>(r.y + m[j] * EB);
#pragma unroll
        for (int j = 0; j < GP; ++j) {
            mp_add<PW>(v[j], e[j]);
            const uint32_t kp = m[j] >> 1;  // pulses left after this position
            const int mag = static_cast<int>(k[j] - kp);
            const uint32_t val = static_cast<uint32_t>((m[j] & 1u) ? 128 + mag : 128 - mag);
            acc[j] = __funnelshift_r(acc[j], val, 8);  // the new byte enters at the top
            k[j] = kp;
        }
    }
#pragma unroll
    for (int j = 0; j < GP; ++j) {
        store_y4(y + static_cast<uint32_t>(j) * ychain, acc[j]);
#pragma unroll
        for (int w = 0; w < PW; ++w) q[j].w[w] = v[j].w[w];
    }
}

// The points of GP codes: q = N(N,K) - code on entry.  `recs` is the shared address of the
// row records (absolute shared addresses by now), cnt[w] the number of rows done in w words.
template <int N, int W, int GP>
__device__ __forceinline__ void search_codes(mp<W> (&q)[GP], int K, uint32_t recs, uint32_t t_before_e,
                                             const int (&cnt)[5], uint32_t y, uint32_t ychain) {
    uint32_t k[GP];
#pragma unroll
    for (int j = 0; j < GP; ++j) k[j] = static_cast<uint32_t>(K);
    uint32_t rec = recs + static_cast<uint32_t>(N - 1) * 16u;
    if constexpr (W >= 4) {
#pragma unroll 1
        for (int b = 0; b < cnt[4]; b += 4, rec -= 64u, y += 4u) search_block4<W, 4, GP>(q, k, rec, t_before_e, y, ychain);
    }
    if constexpr (W >= 3) {
#pragma unroll 1
        for (int b = 0; b < cnt[3]; b += 4, rec -= 64u, y += 4u) search_block4<W, 3, GP>(q, k, rec, t_before_e, y, ychain);
    }
    if constexpr (W >= 2) {
#pragma unroll 1
        for (int b = 0; b < cnt[2]; b += 4, rec -= 64u, y += 4u) search_block4<W, 2, GP>(q, k, rec, t_before_e, y, ychain);
    }
#pragma unroll 1
    for (int b = 0; b < cnt[1]; b += 4, rec -= 64u, y += 4u) search_block4<W, 1, GP>(q, k, rec, t_before_e, y, ychain);
}

// GP groups per thread: a warp takes GP consecutive tiles of 32 groups in one pass.
template <int N, int W, int GP>
__global__ void __launch_bounds__(kSearchThreads / (GP > 2 ? 2 : 1), 1)
    decode_search_kernel(const __grid_constant__ BatchArgs a) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int YS = N + 4;  // bytes between two threads' slots (an odd number of words)
    const int K = a.K;
    const TableLayout L = table_layout(N, K, W);
    const uint32_t sbase = shared_addr(smem);

    // stage the search section with the bulk-copy engine; waited for below
    __shared__ uint64_t stage_bar;
    const BulkStage stage = bulk_stage_begin(&stage_bar);
    if (threadIdx.x == 0) {
        bulk_stage_expect(stage, a.srch_bytes);
        bulk_stage_copy(stage, smem, reinterpret_cast<const uint8_t*>(a.table) + a.srch_off, a.srch_bytes);
    }

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // slots: chain j of thread t at (j * blockDim.x + t) * YS behind the tables (srch_bytes is a
    // multiple of 128)
    uint8_t* yslots = smem + a.srch_bytes + threadIdx.x * YS;
    const uint32_t ychain = blockDim.x * YS;

    // N(N,K): codes at or above it are invalid
    mp<W> bound;
    const uint32_t* bw = a.table + L.bound_off / 4;
#pragma unroll
    for (int w = 0; w < W; ++w) bound.w[w] = bw[w];
    if (!bulk_stage_wait(stage)) {  // the tables never arrived: report and leave
        if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_STAGING_TIMEOUT);
        return;
    }
    {  // a table built for another (N,K) would send the look-ups anywhere: refuse it
        const uint32_t* head = reinterpret_cast<const uint32_t*>(smem);
        if (head[0] != kSearchMagic || head[1] != static_cast<uint32_t>(N) || head[2] != static_cast<uint32_t>(K) ||
            head[3] != a.srch_bytes) {
            if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_TABLE_MISMATCH);
            return;
        }
    }
    int cnt[5];
#pragma unroll
    for (int w = 1; w <= 4; ++w) cnt[w] = static_cast<int>(reinterpret_cast<const uint32_t*>(smem)[8 - w]);
    cnt[0] = 0;
    if (cnt[1] + cnt[2] + cnt[3] + cnt[4] != N || ((cnt[1] | cnt[2] | cnt[3] | cnt[4]) & 3) != 0 ||
        (W < 4 && cnt[4] != 0) || (W < 3 && cnt[3] != 0) || (W < 2 && cnt[2] != 0)) {
        if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_TABLE_MISMATCH);
        return;
    }
    if (threadIdx.x < N) {  // the records' offsets become shared addresses
        uint32_t* rec = reinterpret_cast<uint32_t*>(smem + kSearchHeader) + 4 * threadIdx.x;
        rec[1] += sbase;
        rec[2] += sbase;
    }
#ifdef PVQ_DEBUG
    debug_begin(sbase, sbase + a.srch_bytes, sbase + a.srch_bytes, YS, N, a.debug_status);
    if (threadIdx.x == 0) {
        s_debug.slot_chain = ychain;
        s_debug.slot_end = sbase + a.srch_bytes + GP * ychain;
    }
#endif
    __syncthreads();
    const uint32_t recs = sbase + kSearchHeader;

    const unsigned b = a.scale_bits;
    const unsigned warps_total = gridDim.x * (blockDim.x >> 5);
    bool bad = false;

    int mi = 0;  // the matrices follow one another: a tile's matrix only ever moves on
    for (unsigned tile0 = (blockIdx.x * (blockDim.x >> 5) + warp) * GP; tile0 < a.total_tiles;
         tile0 += warps_total * GP) {
        while (mi + 1 < a.count && tile0 >= a.m[mi + 1].tile_begin) ++mi;
        int mj[GP];
        unsigned row[GP], g[GP];
        float amp[GP];
        bool active[GP];
        mp<W> q[GP];
        int mcur = mi;
#pragma unroll
        for (int j = 0; j < GP; ++j) {
            const unsigned tile = tile0 + j;
            while (mcur + 1 < a.count && tile >= a.m[mcur + 1].tile_begin) ++mcur;
            mj[j] = mcur;
            const MatrixArgs& m = a.m[mcur];
            const unsigned G = static_cast<unsigned>(m.G);
            const unsigned ngroups = static_cast<unsigned>(m.rows) * G;  // below 2^31 (checked by the host)
            const unsigned g0 = (tile - m.tile_begin) * 32u;             // first group of the tile
            const unsigned gi = g0 + lane;
            active[j] = tile < a.total_tiles && gi < ngroups;
            // row and group-in-row: one division per tile, the threads follow from the first group
            row[j] = g0 / G;
            g[j] = g0 - row[j] * G + lane;
            if (g[j] >= G) {
                g[j] -= G;
                row[j] += 1;
                if (g[j] >= G) {  // rows shorter than a tile
                    const unsigned qq = g[j] / G;
                    row[j] += qq;
                    g[j] -= qq * G;
                }
            }
            mp<W> c;
            mp_zero(c);
            amp[j] = 0.0f;
            if (active[j]) {
                c = mp_load<W>(m.codes + static_cast<size_t>(gi) * W);
                mp<W> tmp;
                const bool valid = mp_sub_borrow<W>(tmp, c, bound);
                if (!valid) {  // decodes to zeros: search code 0, whose point has no negative entry
                    bad = true;
                    mp_zero(c);
                } else {
                    // amplitude index: bits [g*b, g*b + b) of the row's LSB-first stream
                    const uint8_t* srow = m.scale_idx + static_cast<size_t>(row[j]) * m.sstride;
                    const unsigned bit = g[j] * b;
                    unsigned bits = srow[bit >> 3];
                    if ((bit & 7u) + b > 8u) bits |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
                    const unsigned qi = (bits >> (bit & 7u)) & ((1u << b) - 1u);
                    // 16 bits: the amplitude itself as binary16; else the quantile level times the row norm
                    amp[j] = b == 16u ? __half2float(__ushort_as_half(static_cast<unsigned short>(qi)))
                                      : __fmul_rn(m.row_norm[row[j]], m.levels[qi]);
                }
            }
            mp_sub_borrow<W>(q[j], bound, c);  // 1 <= q <= N(N,K)
        }
        search_codes<N, W, GP>(q, K, recs, a.srch_t_before_e, cnt, shared_addr(yslots), ychain);
#pragma unroll
        for (int j = 0; j < GP; ++j)
            if (active[j])
                emit_group<N, int8_t>(a.m[mj[j]], reinterpret_cast<const int8_t*>(yslots + j * ychain), amp[j], row[j],
                                      g[j]);
    }
    if (bad && a.status) atomicOr(a.status, PVQ_STATUS_INVALID_CODE);
}

template <int N, int W, int GP>
int launch_search_t(BatchArgs& a, const SearchLayout& S, cudaStream_t stream) {
    constexpr int YS = N + 4;
    constexpr int kMaxThreads = kSearchThreads / (GP > 2 ? 2 : 1);
    unsigned tiles = 0;
    for (int i = 0; i < a.count; ++i) {
        a.m[i].tile_begin = tiles;
        const long long ngroups = a.m[i].rows * a.m[i].G;
        tiles += static_cast<unsigned>((ngroups + 31) / 32);
    }
    a.total_tiles = tiles;
    a.srch_off = S.off;
    a.srch_bytes = S.total;
    a.srch_t_before_e = S.e_off - S.t_off;
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    // One block per SM.  Every tile costs the same, so the launch runs in rounds of GP tiles
    // per resident warp; among the block sizes that fit, take the one whose rounds are
    // fullest, with a preference for more warps (they hide the latency of the dependent
    // table reads).
    auto kern = decode_search_kernel<N, W, GP>;
    int threads = 0;
    size_t smem = 0;
    double best_score = -1.0;
    for (int t = kMaxThreads; t >= kMaxThreads / 2; t -= 32) {
        const size_t bytes = static_cast<size_t>(S.total) + static_cast<size_t>(t) * YS * GP;
        if (bytes > static_cast<size_t>(di.smem_max)) continue;
        const double slots = static_cast<double>(di.sms) * (t / 32) * GP;
        const double rounds = std::ceil(tiles / slots);
        const double score = tiles / (rounds * slots) * (1.0 - 0.004 * (kMaxThreads - t) / 32);
        if (score > best_score) {
            best_score = score;
            threads = t;
            smem = bytes;
        }
    }
    if (threads == 0) return PVQ_ERR_UNSUPPORTED;
    int per_sm = 0;
    if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), threads, smem, &per_sm)) != PVQ_OK) return st;
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned warps_per_block = threads / 32;
    const unsigned blocks_needed = (tiles + warps_per_block * GP - 1) / (warps_per_block * GP);
    const unsigned grid = std::max(1u, std::min<unsigned>(blocks_needed, static_cast<unsigned>(di.sms * per_sm)));
    kern<<<grid, threads, smem, stream>>>(a);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

// Two groups per thread: enough independent chains to cover the latency of the dependent
// table reads with the warps one SM holds (one group: 389 us on the decoder-layer workload,
// two: 333 us, four at half the threads: 455 us).
template <int N, int W>
int launch_search_g(BatchArgs& a, const SearchLayout& S, cudaStream_t stream) {
    return launch_search_t<N, W, 2>(a, S, stream);
}

template <int N, int WMAX>
int launch_search_n(BatchArgs& a, int W, const SearchLayout& S, cudaStream_t stream) {
    if (W > WMAX) return PVQ_ERR_UNSUPPORTED;
    switch (W) {
        case 1: return launch_search_g<N, 1>(a, S, stream);
        case 2: if constexpr (WMAX >= 2) return launch_search_g<N, 2>(a, S, stream);
        case 3: if constexpr (WMAX >= 3) return launch_search_g<N, 3>(a, S, stream);
        case 4: if constexpr (WMAX >= 4) return launch_search_g<N, 4>(a, S, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace

// PVQ_ERR_UNSUPPORTED: no kernel of this family for (N, W); the caller walks instead
int launch_decode_search(const BatchArgs& args, int N, int W, const SearchLayout& S, cudaStream_t stream) {
    if (!S.present || W > 4 || args.K > 127) return PVQ_ERR_UNSUPPORTED;
    BatchArgs a = args;
    switch (N) {
        case 8: return launch_search_n<8, 2>(a, W, S, stream);
        case 16: return launch_search_n<16, 3>(a, W, S, stream);
        case 32: return launch_search_n<32, 4>(a, W, S, stream);
        case 64: return launch_search_n<64, 4>(a, W, S, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
