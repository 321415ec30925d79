// Encode kernels for group size 8, 1-word codes.
#include "pvq_encode_fast.cuh"

namespace pvq {
int launch_encode_n8_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return launch_encode_any<8, 1>(a, dtype, fused, s);
}
}  // namespace pvq
