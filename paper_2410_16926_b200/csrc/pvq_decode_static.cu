// pvq_decode_static_table: decode for callers that may not allocate device memory.
//
// pvq_decode reads the count table N(n,k) from a device buffer that the caller
// allocated and filled with pvq_build_count_table.  Some callers cannot do
// that: a plug-in that runs inside somebody else's inference engine after the
// engine has handed out all of its memory plan, a real-time loop whose
// allocator is frozen once it starts, a process that runs under a memory
// budget enforced by refusing cudaMalloc.  For them the table lives here, in
// a fixed array that is part of the library image: every GPU that loads the
// library holds kStaticTableBytes for it until the process exits, whether or
// not this entry point is ever called.
//
// The array's name is only a handle in host code; the device address is asked
// for once per device with cudaGetSymbolAddress and that pointer is what the
// kernels get.
#include <mutex>

#include "pvq_internal.cuh"

namespace pvq {

constexpr size_t kStaticTableBytes = PVQ_STATIC_TABLE_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) uint32_t g_static_table[kStaticTableBytes / sizeof(uint32_t)];

namespace {

struct DeviceSlot {
    uint32_t* ptr = nullptr;      // device address of g_static_table on this device
    cudaEvent_t filled = nullptr; // recorded behind the last fill, on the stream that ran it
    int N = 0, K = 0;             // the table it was last filled for (0: never)
};

std::mutex g_mu;
DeviceSlot g_slots[kMaxDevices];

}  // namespace
}  // namespace pvq

using namespace pvq;

extern "C" int pvq_decode_static_table(const uint32_t* d_codes, const uint8_t* d_scale_idx,
                                       const float* d_row_norm, int64_t rows, int64_t cols, int N, int K,
                                       int scale_bits, const float* d_levels, void* d_out, int64_t ld_out,
                                       uint32_t* d_status, pvq_stream_t stream) {
    if (N < 1 || K < 1) return PVQ_ERR_INVALID_ARG;
    const size_t need = pvq_count_table_bytes(N, K);
    if (need == 0) return PVQ_ERR_INVALID_ARG;
    if (need > kStaticTableBytes) return PVQ_ERR_TABLE_TOO_SMALL;  // (N,K) too large for the built-in table

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return PVQ_ERR_UNSUPPORTED;

    std::lock_guard<std::mutex> lock(g_mu);
    DeviceSlot& slot = g_slots[dev];
    if (!slot.ptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_table);
        if (e != cudaSuccess) return set_cuda_error(e);
        cudaEvent_t ev = nullptr;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) return set_cuda_error(e);
        slot.ptr = static_cast<uint32_t*>(p);
        slot.filled = ev;
    }
    const cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (slot.N != N || slot.K != K) {
        // Every word the decode kernel reads for (N,K) is written by the builder, so the
        // array needs no clearing between different (N,K).
        slot.N = slot.K = 0;
        const int st = pvq_build_count_table(N, K, slot.ptr, kStaticTableBytes, stream);
        if (st != PVQ_OK) return st;
        e = cudaEventRecord(slot.filled, cs);
        if (e != cudaSuccess) return set_cuda_error(e);
        slot.N = N;
        slot.K = K;
    } else if (cudaEventQuery(slot.filled) != cudaSuccess) {
        // Same (N,K), but the fill may still be in flight on another stream: order this call's
        // decode behind it.  Once the fill has completed no wait is enqueued any more.
        (void)cudaGetLastError();  // cudaErrorNotReady from the query is not an error
        e = cudaStreamWaitEvent(cs, slot.filled, 0);
        if (e != cudaSuccess) return set_cuda_error(e);
    }
    return pvq_decode(d_codes, d_scale_idx, d_row_norm, rows, cols, N, K, scale_bits, slot.ptr, d_levels,
                      d_out, ld_out, d_status, stream);
}
