/* The codec from plain C: build the tables, encode a matrix, decode it, report the error.
 *
 *   gcc -std=c99 -I include -I /usr/local/cuda/include roundtrip.c \
 *       -L paper_2410_16926_b200 -lpvq_b200 -L /usr/local/cuda/lib64 -lcudart -lm -o roundtrip
 *
 * Group-wise PVQ as in Sec. 3.3: groups of N values along each row, one direction code and one
 * amplitude index per group, one norm per row.  Exit status 0 when the round trip is a valid
 * quantisation (no invalid code; relative error of the order that the bit rate allows). */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "pvq.h"

#define CHECK_PVQ(call)                                                                  \
    do {                                                                                 \
        int st_ = (call);                                                                \
        if (st_ != PVQ_OK) {                                                             \
            fprintf(stderr, "%s -> %s (cuda error %d)\n", #call, pvq_strerror(st_),      \
                    pvq_last_cuda_error());                                              \
            return 2;                                                                    \
        }                                                                                \
    } while (0)

#define CHECK_CUDA(call)                                                     \
    do {                                                                     \
        cudaError_t e_ = (call);                                             \
        if (e_ != cudaSuccess) {                                             \
            fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_));    \
            return 3;                                                        \
        }                                                                    \
    } while (0)

static float bf16_to_float(uint16_t h) {
    union {
        uint32_t u;
        float f;
    } v;
    v.u = (uint32_t)h << 16;
    return v.f;
}

int main(void) {
    const int N = 32, index_bits = 96, scale_bits = 4;
    const int64_t rows = 64, cols = 1024, G = cols / N;
    int K = 0, W = 0;
    CHECK_PVQ(pvq_max_pulses(N, index_bits, &K));
    CHECK_PVQ(pvq_code_words(N, K, &W));
    const size_t table_bytes = pvq_count_table_bytes(N, K);
    const size_t stride = pvq_scale_row_stride(G, scale_bits);
    printf("N=%d K=%d W=%d table %zu bytes, %zu index bytes per row\n", N, K, W, table_bytes, stride);

    /* a Gaussian matrix (Box-Muller on a small LCG) */
    float* x = (float*)malloc(sizeof(float) * rows * cols);
    uint16_t* y = (uint16_t*)malloc(sizeof(uint16_t) * rows * cols);
    if (!x || !y) return 1;
    uint64_t s = 12345;
    for (int64_t i = 0; i < rows * cols; i += 2) {
        s = s * 6364136223846793005ull + 1442695040888963407ull;
        const double u1 = ((s >> 11) + 1.0) / 9007199254740993.0;
        s = s * 6364136223846793005ull + 1442695040888963407ull;
        const double u2 = (s >> 11) / 9007199254740992.0;
        const double r = sqrt(-2.0 * log(u1));
        x[i] = (float)(0.02 * r * cos(6.283185307179586 * u2));
        x[i + 1] = (float)(0.02 * r * sin(6.283185307179586 * u2));
    }

    uint32_t *d_table = NULL, *d_codes = NULL, *d_status = NULL;
    float *d_x = NULL, *d_edges = NULL, *d_levels = NULL, *d_rnorm = NULL;
    uint8_t* d_sidx = NULL;
    void* d_out = NULL;
    CHECK_CUDA(cudaMalloc((void**)&d_table, table_bytes));
    CHECK_CUDA(cudaMalloc((void**)&d_x, sizeof(float) * rows * cols));
    CHECK_CUDA(cudaMalloc((void**)&d_edges, sizeof(float) * ((1 << scale_bits) - 1)));
    CHECK_CUDA(cudaMalloc((void**)&d_levels, sizeof(float) * (1 << scale_bits)));
    CHECK_CUDA(cudaMalloc((void**)&d_codes, sizeof(uint32_t) * rows * G * W));
    CHECK_CUDA(cudaMalloc((void**)&d_sidx, stride * rows));
    CHECK_CUDA(cudaMalloc((void**)&d_rnorm, sizeof(float) * rows));
    CHECK_CUDA(cudaMalloc(&d_out, sizeof(uint16_t) * rows * cols));
    CHECK_CUDA(cudaMalloc((void**)&d_status, sizeof(uint32_t)));
    CHECK_CUDA(cudaMemset(d_status, 0, sizeof(uint32_t)));
    CHECK_CUDA(cudaMemcpy(d_x, x, sizeof(float) * rows * cols, cudaMemcpyHostToDevice));

    CHECK_PVQ(pvq_build_count_table(N, K, d_table, table_bytes, NULL));
    CHECK_PVQ(pvq_build_scale_codebook(N, G, scale_bits, d_edges, d_levels, NULL));
    CHECK_PVQ(pvq_encode(d_x, PVQ_DTYPE_F32, rows, cols, cols, N, K, scale_bits, d_table, d_edges, d_codes, d_sidx,
                         d_rnorm, NULL));
    CHECK_PVQ(pvq_decode(d_codes, d_sidx, d_rnorm, rows, cols, N, K, scale_bits, d_table, d_levels, d_out, cols,
                         d_status, NULL));
    uint32_t status = 0;
    CHECK_CUDA(cudaMemcpy(y, d_out, sizeof(uint16_t) * rows * cols, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(&status, d_status, sizeof status, cudaMemcpyDeviceToHost));

    double err = 0.0, ref = 0.0;
    for (int64_t i = 0; i < rows * cols; ++i) {
        const double d = (double)bf16_to_float(y[i]) - x[i];
        err += d * d;
        ref += (double)x[i] * x[i];
    }
    const double qsnr = 10.0 * log10(ref / err);
    printf("status %u, QSNR %.2f dB at %.3f bits per value\n", status,
           qsnr, (double)index_bits / N + (double)scale_bits / N + 32.0 / cols);
    return (status == 0 && qsnr > 10.0 && qsnr < 30.0) ? 0 : 4;
}
