// Group size 128, codes of 1 to 4 words: kernels that compute in exactly the code's width
// (one of the translation units the instantiations are spread over, to build in parallel).
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_big_128_w1_4(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s) {
    switch (W) {
        case 1: return launch_big_w<128, 1, true>(a, dtype, decode, s);
        case 2: return launch_big_w<128, 2, true>(a, dtype, decode, s);
        case 3: return launch_big_w<128, 3, true>(a, dtype, decode, s);
        case 4: return launch_big_w<128, 4, true>(a, dtype, decode, s);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
