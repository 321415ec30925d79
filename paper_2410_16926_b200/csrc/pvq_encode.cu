// Dispatch of the encode launch to the translation unit of its (group size, code words).
#include "pvq_internal.cuh"

namespace pvq {

int launch_encode_n8_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n8_w2(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n16_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n16_w2(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n16_w3(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n32_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n32_w2(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n32_w3(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n32_w4(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w2(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w3(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w4(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w5(BatchArgs& a, int dtype, bool fused, cudaStream_t s);
int launch_encode_n64_w6(BatchArgs& a, int dtype, bool fused, cudaStream_t s);

int launch_encode(const BatchArgs& args, int dtype, int N, int W, bool fused, cudaStream_t stream) {
    BatchArgs a = args;
    switch (N * 100 + W) {
        case 801: return launch_encode_n8_w1(a, dtype, fused, stream);
        case 802: return launch_encode_n8_w2(a, dtype, fused, stream);
        case 1601: return launch_encode_n16_w1(a, dtype, fused, stream);
        case 1602: return launch_encode_n16_w2(a, dtype, fused, stream);
        case 1603: return launch_encode_n16_w3(a, dtype, fused, stream);
        case 3201: return launch_encode_n32_w1(a, dtype, fused, stream);
        case 3202: return launch_encode_n32_w2(a, dtype, fused, stream);
        case 3203: return launch_encode_n32_w3(a, dtype, fused, stream);
        case 3204: return launch_encode_n32_w4(a, dtype, fused, stream);
        case 6401: return launch_encode_n64_w1(a, dtype, fused, stream);
        case 6402: return launch_encode_n64_w2(a, dtype, fused, stream);
        case 6403: return launch_encode_n64_w3(a, dtype, fused, stream);
        case 6404: return launch_encode_n64_w4(a, dtype, fused, stream);
        case 6405: return launch_encode_n64_w5(a, dtype, fused, stream);
        case 6406: return launch_encode_n64_w6(a, dtype, fused, stream);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
