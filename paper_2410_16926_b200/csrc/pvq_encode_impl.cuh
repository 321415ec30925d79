// Encode kernel (and the fused encode -> decode round trip): templates shared by
// the per-group-size translation units.
//
// One thread encodes one group; a thread block covers whole rows (the row norm
// is the only quantity shared between groups).  Steps per group, in the order
// of Sec. 3.3: group norms, row norm, amplitude index (Step 5), direction
// (Step 3: l1 scale, floor, greedy fix-up), Fischer index (Step 7, Algorithm 2).
#pragma once
#include <algorithm>

#include "mp_uint.cuh"
#include "pvq_internal.cuh"

namespace pvq {

// ---- descending sorting network (Batcher odd-even merge sort), in registers ----
template <int N>
__device__ __forceinline__ void sort_desc(float (&v)[N]) {
#pragma unroll
    for (int p = 1; p < N; p <<= 1) {
#pragma unroll
        for (int k = p; k >= 1; k >>= 1) {
#pragma unroll
            for (int j = k % p; j + k < N; j += 2 * k) {
#pragma unroll
                for (int i = 0; i < k; ++i) {
                    if (i + j + k < N && (i + j) / (2 * p) == (i + j + k) / (2 * p)) {
                        const float hi = fmaxf(v[i + j], v[i + j + k]);
                        const float lo = fminf(v[i + j], v[i + j + k]);
                        v[i + j] = hi;
                        v[i + j + k] = lo;
                    }
                }
            }
        }
    }
}

// Direction of one group (Sec. 2.5 / Algorithm 1 in the floor + greedy reading).
//   a_i = |x_i| * (K / l1), m_i = floor(a_i), e_i = a_i - m_i, d = K - sum m_i.
// The greedy loop "give one pulse to the largest residual, lowest index first
// among equals, d times" touches every element at most once when 0 <= d <= N
// (after its pulse an element's residual is negative, below every untouched
// one), so its result is: the d elements with the largest (e_i, -i) get +1.
// They are found with a sorting network on the residuals: v = d-th largest
// value; everything above v gets a pulse, and the elements equal to v share
// what is left, lowest index first.
template <int N>
__device__ __forceinline__ void quantize_direction(const float (&x)[N], float l1, int K, int (&m)[N]) {
    const float gsc = __fdiv_rn(static_cast<float>(K), l1);
    if (!(l1 > 0.0f) || isinf(gsc)) {  // no direction: (K, 0, ..., 0)
#pragma unroll
        for (int i = 0; i < N; ++i) m[i] = 0;
        m[0] = K;
        return;
    }
    float e[N], srt[N];
    int sum = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float av = __fmul_rn(fabsf(x[i]), gsc);
        const float f = floorf(av);
        m[i] = static_cast<int>(f);
        e[i] = __fsub_rn(av, f);
        srt[i] = e[i];
        sum += m[i];
    }
    int d = K - sum;
    d = max(0, min(d, N));  // finite input keeps d in [0, N]; the clamp is for NaN / Inf only
    sort_desc<N>(srt);
    float v = 2.0f;  // above every residual: d == 0 adds nothing
#pragma unroll
    for (int i = 0; i < N; ++i)
        if (i == d - 1) v = srt[i];
    int above = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) above += (e[i] > v) ? 1 : 0;
    int ties = d - above;  // pulses for the elements equal to v
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const bool eq = (e[i] == v) && (ties > 0);
        ties -= eq ? 1 : 0;
        m[i] += ((e[i] > v) || eq) ? 1 : 0;
    }
#pragma unroll
    for (int i = 0; i < N; ++i)
        if (signbit(x[i])) m[i] = -m[i];
}

// Algorithm 2: c = sum over non-zero positions of
//   N(n,k) + 2 sum_{j=1}^{|y_i|-1} N(n,k-j) + [y_i < 0] N(n,k-|y_i|),  n = N-1-i.
template <int N, int W>
__device__ __forceinline__ mp<W> enumerate(const int (&y)[N], int K, const uint32_t* __restrict__ tab) {
    mp<W> c;
    mp_zero(c);
    int k = K;
    const int rowstride = (K + 1) * W;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const int mag = abs(y[i]);
        if (mag > 0) {
            const uint32_t* row = tab + (N - 1 - i) * rowstride;
            mp_add<W>(c, mp_load<W>(row + k * W));
            for (int j = 1; j < mag; ++j) {
                mp<W> t = mp_load<W>(row + (k - j) * W);
                mp_dbl<W>(t);
                mp_add<W>(c, t);
            }
            if (y[i] < 0) mp_add<W>(c, mp_load<W>(row + (k - mag) * W));
            k -= mag;
        }
    }
    return c;
}

template <int N, int W>
__device__ __forceinline__ bool deenumerate_rt(mp<W> r, int K, const uint32_t* __restrict__ tab, int (&y)[N]) {
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

template <int N>
__device__ __forceinline__ void load_group(const void* base, size_t elem_off, bool bf16, float (&x)[N]) {
    if (bf16) {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(base) + elem_off);
#pragma unroll
        for (int v = 0; v < N / 8; ++v) {
            const uint4 q = p[v];
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                x[v * 8 + 2 * e] = __uint_as_float(w[e] << 16);
                x[v * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
        }
    } else {
        const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem_off);
#pragma unroll
        for (int v = 0; v < N / 4; ++v) {
            const float4 q = p[v];
            x[v * 4] = q.x;
            x[v * 4 + 1] = q.y;
            x[v * 4 + 2] = q.z;
            x[v * 4 + 3] = q.w;
        }
    }
}

// Shared memory: [count table][ss per thread slot, padded rows][edges][scale-index words]
template <int N, int W, bool FUSED>
__global__ void __launch_bounds__(512) encode_kernel(const __grid_constant__ BatchArgs a, int ss_floats,
                                                      int bf16) {
    extern __shared__ __align__(16) uint32_t smem[];
    const int K = a.K;
    const int b = a.scale_bits;
    const int nedges = (1 << b) - 1;
    const int tab_words = N * (K + 1) * W;
    uint32_t* s_tab = smem;
    float* s_ss = reinterpret_cast<float*>(smem + tab_words);                   // ss_floats
    float* s_edges = s_ss + ss_floats;                                   // 256
    float* s_levels = s_edges + 256;                                            // 256 (fused only)
    uint32_t* s_idx = reinterpret_cast<uint32_t*>(s_levels + (FUSED ? 256 : 0));  // max_rpt * words per row

    for (int i = threadIdx.x; i < tab_words; i += blockDim.x) s_tab[i] = a.table[i];
    const float* cur_edges = nullptr;

    for (unsigned tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x) {
        const int mi = find_matrix(a, tile);
        const MatrixArgs& m = a.m[mi];
        const int G = m.G;
        const int rpt = m.rows_per_tile;
        int gp = 1;
        while (gp < G) gp <<= 1;
        const int idx_words = m.sstride >> 2;

        __syncthreads();  // previous tile is done with shared memory
        if (cur_edges != m.edges) {  // uniform across the block
            for (int i = threadIdx.x; i < nedges; i += blockDim.x) s_edges[i] = m.edges[i];
            if constexpr (FUSED)
                for (int i = threadIdx.x; i <= nedges; i += blockDim.x) s_levels[i] = m.levels[i];
            cur_edges = m.edges;
        }
        for (int i = threadIdx.x; i < rpt * gp; i += blockDim.x) s_ss[i] = 0.0f;  // zero padding of the tree
        if constexpr (!FUSED)
            for (int i = threadIdx.x; i < rpt * idx_words; i += blockDim.x) s_idx[i] = 0u;
        __syncthreads();

        const int rl = threadIdx.x / G;       // row within the tile
        const int g = threadIdx.x - rl * G;   // group within the row
        const long long row = static_cast<long long>(tile - m.tile_begin) * rpt + rl;
        const bool active = rl < rpt && row < m.rows;

        float x[N];
        float l1 = 0.0f, ss = 0.0f;
        if (active) {
            load_group<N>(m.x, static_cast<size_t>(row) * m.ld + static_cast<size_t>(g) * N, bf16 != 0, x);
            float t[N];
#pragma unroll
            for (int i = 0; i < N; ++i) t[i] = fabsf(x[i]);
            l1 = tree_sum<N>(t);
#pragma unroll
            for (int i = 0; i < N; ++i) t[i] = __fmul_rn(x[i], x[i]);
            ss = tree_sum<N>(t);
            s_ss[rl * gp + g] = ss;
        }
        __syncthreads();
        // row energy: balanced tree over the (zero padded) groups of each row
        for (int s = 1; s < gp; s <<= 1) {
            for (int i = threadIdx.x; i < rpt * gp; i += blockDim.x) {
                const int gg = i & (gp - 1);
                if ((gg & (2 * s - 1)) == 0) s_ss[i] = __fadd_rn(s_ss[i], s_ss[i + s]);
            }
            __syncthreads();
        }
        if (active) {
            const float ss_row = s_ss[rl * gp];
            const float rnorm = __fsqrt_rn(ss_row);
            // Step 5: q = floor(CDF(u) 2^b) as the number of bin edges <= u
            const float u = ss_row > 0.0f ? __fdiv_rn(ss, ss_row) : 0.0f;
            int q = 0;
            for (int step = 1 << (b - 1); step >= 1; step >>= 1)
                if (s_edges[q + step - 1] <= u) q += step;

            int y[N];
            quantize_direction<N>(x, l1, K, y);
            const mp<W> c = enumerate<N, W>(y, K, s_tab);

            if constexpr (!FUSED) {
                if (g == 0) m.row_norm[row] = rnorm;
                uint32_t* cp = m.codes + (static_cast<size_t>(row) * G + g) * W;
#pragma unroll
                for (int w = 0; w < W; ++w) cp[w] = c.w[w];
                const unsigned bit = static_cast<unsigned>(g) * b;
                const unsigned sh = bit & 31u;
                atomicOr(&s_idx[rl * idx_words + (bit >> 5)], static_cast<uint32_t>(q) << sh);
                if (sh + b > 32u) atomicOr(&s_idx[rl * idx_words + (bit >> 5) + 1], static_cast<uint32_t>(q) >> (32u - sh));
            } else {
                int yd[N];
                const bool ok = deenumerate_rt<N, W>(c, K, s_tab, yd);
                int ssy = 0;
#pragma unroll
                for (int i = 0; i < N; ++i) ssy += yd[i] * yd[i];
                const float amp = __fmul_rn(rnorm, s_levels[q]);
                float sc = __fdiv_rn(amp, __fsqrt_rn(static_cast<float>(ssy)));
                if (!ok) sc = 0.0f;
                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.out) +
                                                      static_cast<size_t>(row) * m.ld_out +
                                                      static_cast<size_t>(g) * N);
#pragma unroll
                for (int v = 0; v < N / 8; ++v) {
                    uint32_t p[4];
#pragma unroll
                    for (int e2 = 0; e2 < 4; ++e2) {
                        const float lo = __fmul_rn(static_cast<float>(yd[v * 8 + 2 * e2]), sc);
                        const float hi = __fmul_rn(static_cast<float>(yd[v * 8 + 2 * e2 + 1]), sc);
                        p[e2] = pack_bf16x2(lo, hi);
                    }
                    dst[v] = make_uint4(p[0], p[1], p[2], p[3]);
                }
            }
        }
        if constexpr (!FUSED) {
            __syncthreads();
            for (int i = threadIdx.x; i < rpt * idx_words; i += blockDim.x) {
                const int r2 = i / idx_words;
                const long long row2 = static_cast<long long>(tile - m.tile_begin) * rpt + r2;
                if (row2 < m.rows)
                    reinterpret_cast<uint32_t*>(m.scale_idx + static_cast<size_t>(row2) * m.sstride)[i - r2 * idx_words] =
                        s_idx[i];
            }
        }
    }
}

template <int N, int W, bool FUSED>
static int launch_encode_t(BatchArgs& a, int dtype, cudaStream_t stream) {
    // Block size: a multiple of 32 that wastes the fewest thread slots over the batch.
    int best_threads = 0;
    long long best_cost = -1;
    for (int threads = 128; threads <= 512; threads += 32) {
        long long cost = 0;
        bool ok = true;
        for (int i = 0; i < a.count; ++i) {
            const int G = a.m[i].G;
            if (G > threads) {
                ok = false;
                break;
            }
            const int rpt = threads / G;
            cost += ((a.m[i].rows + rpt - 1) / rpt) * threads;
        }
        if (!ok) continue;
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && threads == 256)) {
            best_cost = cost;
            best_threads = threads;
        }
    }
    if (best_threads == 0) return PVQ_ERR_UNSUPPORTED;  // a row has more groups than a block has threads
    const int threads = best_threads;
    unsigned tiles = 0;
    int max_idx_words = 1;
    for (int i = 0; i < a.count; ++i) {
        MatrixArgs& m = a.m[i];
        m.rows_per_tile = threads / m.G;
        m.tile_begin = tiles;
        tiles += static_cast<unsigned>((m.rows + m.rows_per_tile - 1) / m.rows_per_tile);
        max_idx_words = std::max(max_idx_words, m.rows_per_tile * (m.sstride / 4));
    }
    // s_ss holds rows_per_tile * (G rounded up to a power of two) floats
    int ss_floats = 0;
    for (int i = 0; i < a.count; ++i) {
        int gp = 1;
        while (gp < a.m[i].G) gp <<= 1;
        ss_floats = std::max(ss_floats, a.m[i].rows_per_tile * gp);
    }
    a.total_tiles = tiles;
    const size_t smem = (static_cast<size_t>(N) * (a.K + 1) * W + ss_floats + 256 + (FUSED ? 256 : 0) +
                         max_idx_words) * 4u;
    if (smem > 200 * 1024) return PVQ_ERR_UNSUPPORTED;
    auto kern = encode_kernel<N, W, FUSED>;
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
    kern<<<grid, threads, smem, stream>>>(a, ss_floats, dtype == PVQ_DTYPE_BF16 ? 1 : 0);
    e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int N, int W>
static int launch_encode_nw(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return fused ? launch_encode_t<N, W, true>(a, dtype, s) : launch_encode_t<N, W, false>(a, dtype, s);
}

}  // namespace pvq
