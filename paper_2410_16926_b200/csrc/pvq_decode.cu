// Decode kernel: direction code -> pyramid point (Algorithm 3) -> unit sphere
// times dequantised amplitude -> bf16 (Sec. 2.4, Sec. 3.4).
//
// One thread decodes one group; a warp takes 32 consecutive groups.  Algorithm 3
// is run as a walk over the cells (i, col) of the count table, i the position
// and col the pulses still to place, from (0, K) to (N, 0).  With r the part of
// the code not yet explained and t = N(N-1-i, col), one step does
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
#include <algorithm>

#include "mp_uint.cuh"
#include "pvq_internal.cuh"

namespace pvq {

namespace {

constexpr int kDecThreads = 512;
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

template <int N, int W, typename YT>
__global__ void __launch_bounds__(kDecThreads, 1) decode_kernel(const __grid_constant__ BatchArgs a) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TW = W <= 2 ? W : (W <= 4 ? 4 : 6);  // words per entry of the widest table
    constexpr int YS = N * static_cast<int>(sizeof(YT)) + 4;  // bytes between two threads' slots
    const int K = a.K;
    const TableLayout L = table_layout(N, K, W);
    const int phases = a.walk_phases;
    const uint32_t tab_bytes = L.walk_off[phases - 1] + L.walk_bytes[phases - 1] - L.walk_off[0];

    {   // stage the walk tables: one flat copy
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a.table) + L.walk_off[0]);
        uint4* dst = reinterpret_cast<uint4*>(smem);
        for (uint32_t q = threadIdx.x; q < tab_bytes / 16; q += blockDim.x) dst[q] = src[q];
    }
    const uint32_t tab0 = shared_addr(smem);
    const uint32_t tab2 = tab0 + (L.walk_off[1] - L.walk_off[0]);
    const uint32_t tab1 = tab0 + (L.walk_off[2] - L.walk_off[0]);
    const bool has2 = phases >= 2 && L.walk_bytes[1] != 0;
    const bool has1 = phases >= 3;

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    uint8_t* wbuf = smem + ((tab_bytes + 15u) & ~15u) + warp * (32 * YS + 128);
    YT* yslots = reinterpret_cast<YT*>(wbuf + lane * YS);
    float* wscale = reinterpret_cast<float*>(wbuf + 32 * YS);

    // N(N,K): codes at or above it are invalid
    mp<W> bound;
    const uint32_t* bw = a.table + L.bound_off / 4;
#pragma unroll
    for (int w = 0; w < W; ++w) bound.w[w] = bw[w];
    const bool bound_wide = bw[W] != 0u;  // N(N,K) = 2^(32W) exactly: every W-word code is valid
    __syncthreads();

    const int b = a.scale_bits;
    const int S = N + K;
    const unsigned warps_total = gridDim.x * (blockDim.x >> 5);
    bool bad = false;

    for (unsigned tile = blockIdx.x * (blockDim.x >> 5) + warp; tile < a.total_tiles; tile += warps_total) {
        const int mi = find_matrix(a, tile);
        const MatrixArgs& m = a.m[mi];
        const long long g0 = static_cast<long long>(tile - m.tile_begin) * 32;  // first group of the tile
        const long long ngroups = m.rows * m.G;
        const long long gi = g0 + lane;
        const bool active = gi < ngroups;

        mp<W> c;
        mp_zero(c);
        float amp = 0.0f;
        if (active) {
            c = mp_load<W>(m.codes + gi * W);
            mp<W> tmp;
            const bool valid = bound_wide || mp_sub_borrow<W>(tmp, c, bound);
            if (!valid) {  // decodes to zeros: walk code 0, whose point has no negative entry
                bad = true;
                mp_zero(c);
            } else {
                const unsigned row = static_cast<unsigned>(gi) / static_cast<unsigned>(m.G);
                const unsigned g = static_cast<unsigned>(gi) - row * static_cast<unsigned>(m.G);
                // amplitude index: bits [g*b, g*b + b) of the row's LSB-first stream
                const uint8_t* srow = m.scale_idx + static_cast<size_t>(row) * m.sstride;
                const unsigned bit = g * b;
                unsigned bits = srow[bit >> 3];
                if ((bit & 7u) + b > 8u) bits |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
                const unsigned q = (bits >> (bit & 7u)) & ((1u << b) - 1u);
                amp = __fmul_rn(m.row_norm[row], m.levels[q]);
            }
        }

        // ---- the walk
        Walk st;
        st.v = 0;
        st.y = st.y0 = shared_addr(yslots);
        int s = 0;
        s = walk_phase<W, TW * 4, W, YT>(c, st, tab0, L.rowlen, K, s, S, has2 ? 2 : (has1 ? 1 : 0));
        if constexpr (W > 2) {
            if (s < S && has2) s = walk_phase<2, 8, W, YT>(c, st, tab2, L.rowlen, K, s, S, has1 ? 1 : 0);
        }
        if constexpr (W > 1) {
            if (s < S && has1) s = walk_phase<1, 4, W, YT>(c, st, tab1, L.rowlen, K, s, S, 0);
        }

        // ---- scale: point on the unit sphere times the amplitude
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

        // ---- coalesced stores: N/8 threads per group, 16 bytes each
        constexpr int TPG = N / 8;       // threads per group
        constexpr int GPI = 32 / TPG;    // groups per iteration
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
    int dev = 0, sms = 0, smem_max = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return set_cuda_error(e);
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return set_cuda_error(e);
    if ((e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
        return set_cuda_error(e);
    // As many of the narrower walk tables as fit beside the widest one; fewer threads if even
    // that leaves no room for their output slots.
    int threads = kDecThreads;
    int phases = 0;
    size_t smem = 0;
    for (; threads >= 128 && phases == 0; threads /= 2) {
        const size_t wbufs = static_cast<size_t>(threads / 32) * (32 * YS + 128);
        for (int p = 3; p >= 1; --p) {
            if (p > 1 && L.walk_bytes[p - 1] == 0) continue;
            const size_t tab = L.walk_off[p - 1] + L.walk_bytes[p - 1] - L.walk_off[0];
            const size_t need = ((tab + 15) & ~size_t(15)) + wbufs;
            if (need <= static_cast<size_t>(smem_max)) {
                phases = p;
                smem = need;
                break;
            }
        }
        if (phases) break;
    }
    if (phases == 0) return PVQ_ERR_UNSUPPORTED;
    a.walk_phases = phases;
    auto kern = decode_kernel<N, W, YT>;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem))) !=
        cudaSuccess)
        return set_cuda_error(e);
    int per_sm = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem)) != cudaSuccess)
        return set_cuda_error(e);
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned warps_per_block = threads / 32;
    const unsigned blocks_needed = (tiles + warps_per_block - 1) / warps_per_block;
    const unsigned grid = std::max(1u, std::min<unsigned>(blocks_needed, static_cast<unsigned>(sms * per_sm)));
    kern<<<grid, threads, smem, stream>>>(a);
    e = cudaGetLastError();
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
