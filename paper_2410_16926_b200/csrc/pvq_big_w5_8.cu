// Group size 128, codes of 5 to 8 words: kernels that compute in exactly the code's width
// (one of the translation units the instantiations are spread over, to build in parallel).
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_big_128_w5_8(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s) {
    switch (W) {
        case 5: return launch_big_w<128, 5, true>(a, dtype, decode, s);
        case 6: return launch_big_w<128, 6, true>(a, dtype, decode, s);
        case 7: return launch_big_w<128, 7, true>(a, dtype, decode, s);
        case 8: return launch_big_w<128, 8, true>(a, dtype, decode, s);
        default: return PVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace pvq
