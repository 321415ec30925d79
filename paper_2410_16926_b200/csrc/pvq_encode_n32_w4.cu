// Encode kernels for group size 32, 4-word codes.
#include "pvq_encode_fast.cuh"

namespace pvq {
int launch_encode_n32_w4(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return launch_encode_any<32, 4>(a, dtype, fused, s);
}
}  // namespace pvq
