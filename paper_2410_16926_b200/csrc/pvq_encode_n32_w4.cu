// Encode kernels for group size 32, 4-word codes.
#include "pvq_encode_impl.cuh"

namespace pvq {
int launch_encode_n32_w4(BatchArgs& a, int dtype, bool fused, cudaStream_t s) {
    return launch_encode_nw<32, 4>(a, dtype, fused, s);
}
}  // namespace pvq
