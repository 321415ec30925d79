// Encode kernels for group size 16, 2-word codes.
#include "pvq_encode_fast.cuh"

namespace pvq {
int launch_encode_n16_w2(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return launch_encode_any<16, 2>(a, dtype, fused, s);
}
}  // namespace pvq
