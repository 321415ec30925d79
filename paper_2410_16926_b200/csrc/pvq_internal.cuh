// Shared declarations of the PVQ library's translation units (host side and
// kernel launch parameters).  Not part of the public interface.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "pvq.h"

namespace pvq {

constexpr int kMaxBatch = 32;     // matrices per launch
constexpr int kMaxWords = 12;     // limbs per code the kernels are instantiated for
constexpr int kMaxPulses = 1023;  // table builder: one thread per k

// One matrix as the kernels see it.
struct MatrixArgs {
    const void* x;        // encode / round-trip input
    void* out;            // decode / round-trip output (bf16)
    uint32_t* codes;
    uint8_t* scale_idx;
    float* row_norm;
    const float* edges;
    const float* levels;
    long long rows, cols, ld, ld_out;
    int G;                // groups per row
    int sstride;          // bytes per row of scale_idx
    int rows_per_tile;    // encode: rows one thread block covers
    unsigned tile_begin;  // first tile of this matrix in the launch
};

struct BatchArgs {
    MatrixArgs m[kMaxBatch];
    int count;
    unsigned total_tiles;
    int K;
    int scale_bits;
    const uint32_t* table;
    uint32_t* status;
};

// host helpers (pvq_host.cu)
int set_cuda_error(cudaError_t e);  // records e, returns PVQ_ERR_CUDA
int code_words_for(int N, int K);   // W, or 0 when it cannot be computed
bool is_aligned(const void* p, size_t a);

// launchers (one per kernel family); all return a pvq_status
int launch_decode(const BatchArgs& args, int N, int W, cudaStream_t stream);
int launch_encode(const BatchArgs& args, int dtype, int N, int W, bool fused, cudaStream_t stream);

// ---------------------------------------------------------------- device bits

#ifdef __CUDACC__

// balanced tree over contiguous halves, each addition rounded to fp32
template <int N>
__device__ __forceinline__ float tree_sum(const float (&v)[N]) {
    float t[N];
#pragma unroll
    for (int i = 0; i < N; ++i) t[i] = v[i];
#pragma unroll
    for (int s = 1; s < N; s <<= 1) {
#pragma unroll
        for (int i = 0; i < N; i += 2 * s) t[i] = __fadd_rn(t[i], t[i + s]);
    }
    return t[0];
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// which matrix does tile t belong to?  (count <= 32: a short scan)
__device__ __forceinline__ int find_matrix(const BatchArgs& a, unsigned tile) {
    int mi = 0;
    for (int i = 1; i < a.count; ++i)
        if (tile >= a.m[i].tile_begin) mi = i;
    return mi;
}

#endif  // __CUDACC__

}  // namespace pvq
