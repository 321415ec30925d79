// Encode kernels for group size 64, 1-word codes.
#include "pvq_encode_fast.cuh"

namespace pvq {
int launch_encode_n64_w1(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return launch_encode_any<64, 1>(a, dtype, fused, s);
}
}  // namespace pvq
