// Decode kernel: direction code -> pyramid point (Algorithm 3) -> unit sphere
// times dequantised amplitude -> bf16 (Sec. 2.4, Sec. 3.4).
//
// One thread decodes one group; a warp takes 32 consecutive groups and walks their
// codes in lockstep (pvq_walk.cuh), each thread collecting its point in shared
// memory, from where it scales it and writes its N bf16 values with 16-byte stores.
#include <algorithm>
#include <cmath>

#include <cuda_fp16.h>

#include "pvq_walk.cuh"

namespace pvq {

namespace {

constexpr int kDecThreads = 768;

template <int N, int W, typename YT>
__global__ void __launch_bounds__(kDecThreads, 1) decode_kernel(const __grid_constant__ BatchArgs a) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;  // bytes between two threads' slots
    const int K = a.K;
    const TableLayout L = table_layout(N, K, W);
    const uint32_t tab_bytes = walk_tables_bytes(L, a.walk_phases);

    // stage the walk tables with the bulk-copy engine; waited for below
    __shared__ uint64_t stage_bar;
    const BulkStage stage = bulk_stage_begin(&stage_bar);
    if (threadIdx.x == 0) {
        bulk_stage_expect(stage, walk_tables_stage_bytes(L, a.walk_phases));
        walk_tables_stage(stage, smem, a.table, L, a.walk_phases);
    }
    const WalkTables wt = walk_tables(L, shared_addr(smem), a.walk_phases, a);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    YT* yslots = reinterpret_cast<YT*>(smem + ((tab_bytes + 15u) & ~15u) + threadIdx.x * YS);

    // N(N,K): codes at or above it are invalid
    mp<W> bound;
    const uint32_t* bw = a.table + L.bound_off / 4;
#pragma unroll
    for (int w = 0; w < W; ++w) bound.w[w] = bw[w];
    const bool bound_wide = bw[W] != 0u;  // N(N,K) = 2^(32W) exactly: every W-word code is valid
    if (!bulk_stage_wait(stage)) {  // the tables never arrived: report and leave
        if (a.status && threadIdx.x == 0) atomicOr(a.status, PVQ_STATUS_STAGING_TIMEOUT);
        return;
    }
#ifdef PVQ_DEBUG
    debug_begin(shared_addr(smem), shared_addr(smem) + tab_bytes, shared_addr(smem) + ((tab_bytes + 15u) & ~15u), YS,
                N * static_cast<uint32_t>(sizeof(YT)), a.debug_status);
#endif

    const unsigned b = a.scale_bits;
    const unsigned warps_total = gridDim.x * (blockDim.x >> 5);
    bool bad = false;

    int mi = 0;  // the matrices follow one another: the tile's matrix only ever moves on
    for (unsigned tile = blockIdx.x * (blockDim.x >> 5) + warp; tile < a.total_tiles; tile += warps_total) {
        while (mi + 1 < a.count && tile >= a.m[mi + 1].tile_begin) ++mi;
        const MatrixArgs& m = a.m[mi];
        const unsigned G = static_cast<unsigned>(m.G);
        const unsigned ngroups = static_cast<unsigned>(m.rows) * G;  // below 2^31 (checked by the host)
        const unsigned g0 = (tile - m.tile_begin) * 32u;             // first group of the tile
        const unsigned gi = g0 + lane;
        const bool active = gi < ngroups;
        // row and group-in-row: one division per tile, the threads follow from the first group
        unsigned row = g0 / G;
        unsigned g = g0 - row * G + lane;
        if (g >= G) {
            g -= G;
            row += 1;
            if (g >= G) {  // rows shorter than a tile
                const unsigned q = g / G;
                row += q;
                g -= q * G;
            }
        }

        mp<W> c;
        mp_zero(c);
        unsigned sbits = 0u;
        float rnorm = 0.0f;
        bool valid = false;
        if (active) {
            c = mp_load<W>(m.codes + static_cast<size_t>(gi) * W);
            // the bytes that hold the amplitude index, bits [g*b, g*b + b) of the row's LSB-first
            // stream, and the row norm: asked for now, used after the walk
            const uint8_t* srow = m.scale_idx + static_cast<size_t>(row) * m.sstride;
            const unsigned bit = g * b;
            sbits = srow[bit >> 3];
            if ((bit & 7u) + b > 8u) sbits |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
            if (b != 16u) rnorm = m.row_norm[row];
            mp<W> tmp;
            valid = bound_wide || mp_sub_borrow<W>(tmp, c, bound);
            if (!valid) {  // decodes to zeros: walk code 0, whose point has no negative entry
                bad = true;
                mp_zero(c);
            }
        }
        walk_code<N, W, YT>(c, wt, K, yslots);
        if (active) {
            float amp = 0.0f;
            if (valid) {
                const unsigned q = (sbits >> ((g * b) & 7u)) & ((1u << b) - 1u);
                // 16 bits: the amplitude itself as binary16; else the quantile level times the row norm
                amp = b == 16u ? __half2float(__ushort_as_half(static_cast<unsigned short>(q)))
                               : __fmul_rn(rnorm, m.levels[q]);
            }
            emit_group<N, YT>(m, yslots, amp, row, g);
        }
    }
    if (bad && a.status) atomicOr(a.status, PVQ_STATUS_INVALID_CODE);
}

template <int N, int W, typename YT>
int launch_decode_t(BatchArgs& a, cudaStream_t stream) {
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;
    unsigned tiles = 0;
    for (int i = 0; i < a.count; ++i) {
        a.m[i].tile_begin = tiles;
        const long long ngroups = a.m[i].rows * a.m[i].G;
        tiles += static_cast<unsigned>((ngroups + 31) / 32);
    }
    a.total_tiles = tiles;
    const TableLayout L = table_layout(N, a.K, W);
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    const int sms = di.sms, smem_max = di.smem_max;
    // Block size: every tile costs the same, so the launch runs in rounds of one tile per
    // resident warp and the last round is only partly filled.  Among block sizes of 12..16
    // warps take the one that wastes the fewest warp slots over the rounds (with a small
    // preference for more warps, which hide latency better); smaller blocks only when the
    // tables leave no room for more output slots.  With each size go as many of the narrower
    // walk tables as fit beside the widest one.
    auto kern = decode_kernel<N, W, YT>;
    int threads = 0, phases = 0, per_sm = 0;
    size_t smem = 0;
    double best_score = -1.0;
    for (int t = kDecThreads; t >= 128; t -= 32) {
        if (t < 384 && threads != 0) break;
        const size_t wbufs = static_cast<size_t>(t) * YS;
        if (wbufs >= static_cast<size_t>(smem_max)) continue;
        const int ph = walk_phases_that_fit(L, static_cast<size_t>(smem_max) - wbufs);
        if (ph == 0) continue;
        const size_t sm_bytes = ((walk_tables_bytes(L, ph) + 15u) & ~size_t(15)) + wbufs;
        int bps = 0;
        if ((st = prepare_kernel(reinterpret_cast<const void*>(kern), t, sm_bytes, &bps)) != PVQ_OK) return st;
        if (bps < 1) continue;
        const double slots = static_cast<double>(sms) * bps * (t / 32);
        const double rounds = std::ceil(tiles / slots);
        const double score = tiles / (rounds * slots) * (1.0 - 0.01 * (kDecThreads - t) / 32);
        if (score > best_score) {
            best_score = score;
            threads = t;
            phases = ph;
            per_sm = bps;
            smem = sm_bytes;
        }
    }
    if (threads == 0) return PVQ_ERR_UNSUPPORTED;
    a.walk_phases = phases;
    const unsigned warps_per_block = threads / 32;
    const unsigned blocks_needed = (tiles + warps_per_block - 1) / warps_per_block;
    const unsigned grid = std::max(1u, std::min<unsigned>(blocks_needed, static_cast<unsigned>(sms * per_sm)));
    kern<<<grid, threads, smem, stream>>>(a);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int W>
int launch_decode_nw(BatchArgs& a, cudaStream_t stream) {
    if (a.K <= 127) return launch_decode_t<N, W, int8_t>(a, stream);
    return launch_decode_t<N, W, int16_t>(a, stream);
}

template <int N, int WMAX>
int launch_decode_n(BatchArgs& a, int W, cudaStream_t stream) {
    if (W > WMAX) return PVQ_ERR_UNSUPPORTED;
    switch (W) {
        case 1: return launch_decode_nw<N, 1>(a, stream);
        case 2: if constexpr (WMAX >= 2) return launch_decode_nw<N, 2>(a, stream);
        case 3: if constexpr (WMAX >= 3) return launch_decode_nw<N, 3>(a, stream);
        case 4: if constexpr (WMAX >= 4) return launch_decode_nw<N, 4>(a, stream);
        case 5: if constexpr (WMAX >= 5) return launch_decode_nw<N, 5>(a, stream);
        case 6: if constexpr (WMAX >= 6) return launch_decode_nw<N, 6>(a, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace

int launch_decode(const BatchArgs& args, int N, int W, cudaStream_t stream) {
    // codes of up to four words and 127 pulses: one threshold search per position, where
    // the tables for it are part of the blob; everything else walks
    if (W <= 4 && args.K <= 127) {
        const SearchLayout& S = search_layout_for(N, args.K);
        if (S.present) {
            const int st = launch_decode_search(args, N, W, S, stream);
            if (st != PVQ_ERR_UNSUPPORTED) return st;
        }
    }
    BatchArgs a = args;
    switch (N) {
        case 8: return launch_decode_n<8, 2>(a, W, stream);
        case 16: return launch_decode_n<16, 3>(a, W, stream);
        case 32: return launch_decode_n<32, 4>(a, W, stream);
        case 64: return launch_decode_n<64, 6>(a, W, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
