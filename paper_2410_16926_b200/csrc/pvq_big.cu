// Group size 128 with codes of up to 12 words (the paper's setting at 3 bits per weight,
// Sec. 4.1): kernels that compute in exactly the code's width.
#include "pvq_big_impl.cuh"

namespace pvq {

namespace {

int launch_big_128(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s) {
    switch (W) {
        case 1: return launch_big_w<128, 1, true>(a, dtype, decode, s);
        case 2: return launch_big_w<128, 2, true>(a, dtype, decode, s);
        case 3: return launch_big_w<128, 3, true>(a, dtype, decode, s);
        case 4: return launch_big_w<128, 4, true>(a, dtype, decode, s);
        case 5: return launch_big_w<128, 5, true>(a, dtype, decode, s);
        case 6: return launch_big_w<128, 6, true>(a, dtype, decode, s);
        case 7: return launch_big_w<128, 7, true>(a, dtype, decode, s);
        case 8: return launch_big_w<128, 8, true>(a, dtype, decode, s);
        case 9: return launch_big_w<128, 9, true>(a, dtype, decode, s);
        case 10: return launch_big_w<128, 10, true>(a, dtype, decode, s);
        case 11: return launch_big_w<128, 11, true>(a, dtype, decode, s);
        case 12: return launch_big_w<128, 12, true>(a, dtype, decode, s);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace

int launch_big(const BatchArgs& args, int dtype, int N, int W, bool decode, cudaStream_t stream) {
    BatchArgs a = args;
    if (N == 128 && W <= 12) return launch_big_128(a, dtype, W, decode, stream);
    return launch_wide(a, dtype, N, W, decode, stream);
}

}  // namespace pvq
