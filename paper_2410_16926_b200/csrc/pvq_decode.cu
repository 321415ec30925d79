// Decode kernel: direction code -> pyramid point (Algorithm 3) -> unit sphere
// times dequantised amplitude -> bf16 (Sec. 2.4, Sec. 3.4).
//
// One thread decodes one group.  The count table lives in shared memory for
// the life of the block; a block walks over tiles of blockDim.x consecutive
// groups.  The walk over the N positions is unrolled so that the decoded
// point stays in registers.
#include <algorithm>

#include "mp_uint.cuh"
#include "pvq_internal.cuh"

namespace pvq {

// Walk of Algorithm 3 with r = c - z (the part of the code not yet explained):
//   r <  N(n,k)            -> y_i = 0
//   else r -= N(n,k); while r >= 2 N(n,k-j): r -= 2 N(n,k-j), j += 1
//        r <  N(n,k-j)     -> y_i = +j
//        else                 y_i = -j, r -= N(n,k-j)
// n = N-1-i dimensions remain after position i; k pulses remain.
// Returns true when the code was valid (r == 0 and k == 0 at the end).
template <int N, int W>
__device__ __forceinline__ bool deenumerate(mp<W> r, int K, const uint32_t* __restrict__ tab, int (&y)[N]) {
    int k = K;
    const int rowstride = (K + 1) * W;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        y[i] = 0;
        if (k > 0) {
            const uint32_t* row = tab + (N - 1 - i) * rowstride;
            mp<W> t = mp_load<W>(row + k * W);
            if (mp_sub_if_ge<W>(r, t)) {
                int j = 1;
                t = mp_load<W>(row + (k - 1) * W);
                while (j < k) {
                    mp<W> d = t;
                    mp_dbl<W>(d);
                    if (!mp_sub_if_ge<W>(r, d)) break;
                    ++j;
                    t = mp_load<W>(row + (k - j) * W);
                }
                const bool neg = mp_sub_if_ge<W>(r, t);
                y[i] = neg ? -j : j;
                k -= j;
            }
        }
    }
    return k == 0 && mp_is_zero<W>(r);
}

template <int N, int W>
__global__ void __launch_bounds__(256) decode_kernel(const __grid_constant__ BatchArgs a) {
    extern __shared__ __align__(16) uint32_t smem_tab[];
    const int K = a.K;
    const int tab_words = N * (K + 1) * W;
    for (int i = threadIdx.x; i < tab_words; i += blockDim.x) smem_tab[i] = a.table[i];
    __syncthreads();

    const int b = a.scale_bits;
    bool bad = false;
    for (unsigned tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x) {
        const int mi = find_matrix(a, tile);
        const MatrixArgs& m = a.m[mi];
        const long long gi = static_cast<long long>(tile - m.tile_begin) * blockDim.x + threadIdx.x;
        const long long ngroups = m.rows * m.G;
        if (gi >= ngroups) continue;
        const unsigned row = static_cast<unsigned>(gi) / static_cast<unsigned>(m.G);
        const unsigned g = static_cast<unsigned>(gi) - row * static_cast<unsigned>(m.G);

        mp<W> c = mp_load<W>(m.codes + gi * W);
        int y[N];
        const bool ok = deenumerate<N, W>(c, K, smem_tab, y);
        bad |= !ok;

        // amplitude index: bits [g*b, g*b + b) of the row's LSB-first stream
        const uint8_t* srow = m.scale_idx + static_cast<size_t>(row) * m.sstride;
        const unsigned bit = g * b;
        unsigned bits = srow[bit >> 3];
        if ((bit & 7u) + b > 8u) bits |= static_cast<unsigned>(srow[(bit >> 3) + 1]) << 8;
        const unsigned q = (bits >> (bit & 7u)) & ((1u << b) - 1u);

        int ssy = 0;
#pragma unroll
        for (int i = 0; i < N; ++i) ssy += y[i] * y[i];
        const float amp = __fmul_rn(m.row_norm[row], m.levels[q]);
        float s = __fdiv_rn(amp, __fsqrt_rn(static_cast<float>(ssy)));
        if (!ok) s = 0.0f;

        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.out) +
                                              static_cast<size_t>(row) * m.ld_out + static_cast<size_t>(g) * N);
#pragma unroll
        for (int v = 0; v < N / 8; ++v) {
            uint4 o;
            uint32_t p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float lo = __fmul_rn(static_cast<float>(y[v * 8 + 2 * e]), s);
                float hi = __fmul_rn(static_cast<float>(y[v * 8 + 2 * e + 1]), s);
                if (!ok) lo = hi = 0.0f;  // +0 rather than the sign of y
                p[e] = pack_bf16x2(lo, hi);
            }
            o.x = p[0];
            o.y = p[1];
            o.z = p[2];
            o.w = p[3];
            dst[v] = o;
        }
    }
    if (bad && a.status) atomicOr(a.status, PVQ_STATUS_INVALID_CODE);
}

template <int N, int W>
static int launch_decode_nw(BatchArgs& a, cudaStream_t stream) {
    const int threads = 256;
    unsigned tiles = 0;
    for (int i = 0; i < a.count; ++i) {
        a.m[i].tile_begin = tiles;
        const long long ngroups = a.m[i].rows * a.m[i].G;
        tiles += static_cast<unsigned>((ngroups + threads - 1) / threads);
    }
    a.total_tiles = tiles;
    const size_t smem = static_cast<size_t>(N) * (a.K + 1) * W * sizeof(uint32_t);
    if (smem > 200 * 1024) return PVQ_ERR_UNSUPPORTED;
    auto kern = decode_kernel<N, W>;
    cudaError_t e;
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return set_cuda_error(e);
    }
    int dev = 0, sms = 0, per_sm = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return set_cuda_error(e);
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return set_cuda_error(e);
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem)) != cudaSuccess)
        return set_cuda_error(e);
    if (per_sm < 1) return PVQ_ERR_UNSUPPORTED;
    const unsigned grid = std::min<unsigned>(tiles, static_cast<unsigned>(sms * per_sm));
    kern<<<grid, threads, smem, stream>>>(a);
    e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int WMAX>
static int launch_decode_n(BatchArgs& a, int W, cudaStream_t stream) {
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
