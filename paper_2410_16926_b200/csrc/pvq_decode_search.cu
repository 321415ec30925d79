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

// GP groups per thread: a warp takes GP consecutive tiles of 32 groups in one pass.
template <int N, int W, int GP, int PLANE>
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
    // (records and bucket tables, then the increments E where the blob has the thresholds T)
    const uint8_t* section = reinterpret_cast<const uint8_t*>(a.table) + a.srch_off;
    const uint32_t staged = a.srch_bytes - a.srch_t_before_e;
    if (threadIdx.x == 0) {
        bulk_stage_expect(stage, staged);
        bulk_stage_copy(stage, smem, section, a.srch_t_off);
        bulk_stage_copy(stage, smem + a.srch_t_off, section + a.srch_t_off + a.srch_t_before_e, staged - a.srch_t_off);
    }
    // global address of a row of T = t_rows + shared address of the row of E
    const uint8_t* t_rows = section - sbase;

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // slots: chain j of thread t at (j * blockDim.x + t) * YS behind the tables (a multiple of 16 bytes)
    uint8_t* yslots = smem + staged + threadIdx.x * YS;
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
    int cnt[5];
    if (!search_section_begin<N, W>(smem, a.srch_bytes, a.srch_t_before_e, K, cnt)) {  // not the table of this (N,K): refuse it
        if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_TABLE_MISMATCH);
        return;
    }
#ifdef PVQ_DEBUG
    debug_begin(sbase, sbase + staged, sbase + staged, YS, N, a.debug_status);
    if (threadIdx.x == 0) {
        s_debug.slot_chain = ychain;
        s_debug.slot_end = sbase + staged + GP * ychain;
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
        float rnorm[GP];
        unsigned sbits[GP];
        bool active[GP], active_valid[GP];
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
            active_valid[j] = active[j];
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
            sbits[j] = 0u;
            rnorm[j] = 0.0f;
            if (active[j]) {
                c = mp_load<W>(m.codes + static_cast<size_t>(gi) * W);
                // the bytes that hold the amplitude index, bits [g*b, g*b + b) of the row's LSB-first
                // stream, and the row norm: asked for now, used after the search
                const uint8_t* srow = m.scale_idx + static_cast<size_t>(row[j]) * m.sstride;
                const unsigned bit = g[j] * b;
                sbits[j] = srow[bit >> 3];
                if ((bit & 7u) + b > 8u) sbits[j] |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
                if (b != 16u) rnorm[j] = m.row_norm[row[j]];
                mp<W> tmp;
                if (!mp_sub_borrow<W>(tmp, c, bound)) {  // invalid: decodes to zeros (search code 0, whose point has no negative entry)
                    bad = true;
                    active_valid[j] = false;
                    mp_zero(c);
                }
            }
            mp_sub_borrow<W>(q[j], bound, c);  // 1 <= q <= N(N,K)
        }
        search_codes<N, W, GP, PLANE>(q, K, recs, t_rows, cnt, shared_addr(yslots), ychain);
#pragma unroll
        for (int j = 0; j < GP; ++j)
            if (active[j]) {
                const MatrixArgs& m = a.m[mj[j]];
                float amp = 0.0f;  // an invalid code decodes to zeros
                if (active_valid[j]) {
                    const unsigned qi = (sbits[j] >> ((g[j] * b) & 7u)) & ((1u << b) - 1u);
                    // 16 bits: the amplitude itself as binary16; else the quantile level times the row norm
                    amp = b == 16u ? __half2float(__ushort_as_half(static_cast<unsigned short>(qi)))
                                   : __fmul_rn(rnorm[j], m.levels[qi]);
                }
                emit_group<N, int8_t>(m, reinterpret_cast<const int8_t*>(yslots + j * ychain), amp, row[j], g[j]);
            }
    }
    if (bad && a.status) atomicOr(a.status, PVQ_STATUS_INVALID_CODE);
}

template <int N, int W, int GP, int PLANE>
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
    a.srch_t_off = S.t_off;
    a.srch_t_before_e = S.e_off - S.t_off;
    const size_t staged = S.total - (S.e_off - S.t_off);
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    // One block per SM.  Every tile costs the same, so the launch runs in rounds of GP tiles
    // per resident warp; among the block sizes that fit, take the one whose rounds are
    // fullest, with a preference for more warps (they hide the latency of the dependent
    // table reads).
    auto kern = decode_search_kernel<N, W, GP, PLANE>;
    int threads = 0;
    size_t smem = 0;
    double best_score = -1.0;
    for (int t = kMaxThreads; t >= 128; t -= 32) {
        const size_t bytes = staged + static_cast<size_t>(t) * YS * GP;
        if (bytes > static_cast<size_t>(di.smem_max)) continue;
        const double slots = static_cast<double>(di.sms) * (t / 32) * GP;
        const double rounds = std::ceil(tiles / slots);
        // a launch of one round: the smallest block that still makes it one round (the work
        // spreads over more SMs); otherwise the fullest rounds among the larger blocks
        if (rounds > 1.0 && t < kMaxThreads / 2) break;
        const double score = rounds > 1.0 ? tiles / (rounds * slots) * (1.0 - 0.004 * (kMaxThreads - t) / 32)
                                          : 2.0 + (kMaxThreads - t);
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
    switch (S.plane) {  // entries per word plane of the section's rows
        case 64: return launch_search_t<N, W, 2, 64>(a, S, stream);
        case 128: return launch_search_t<N, W, 2, 128>(a, S, stream);
        case 256: return launch_search_t<N, W, 2, 256>(a, S, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
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
