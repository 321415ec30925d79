// Group size 128, codes of 9 to 10 words: kernels that compute in exactly the code's width
// (one of the translation units the instantiations are spread over, to build in parallel).
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_big_128_w9_10(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s) {
    switch (W) {
        case 9: return launch_big_w<128, 9, true>(a, dtype, decode, s);
        case 10: return launch_big_w<128, 10, true>(a, dtype, decode, s);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
