// Group size 128 with codes of more than 12 words, computed in 16 or 32 words (see pvq_wide.cu).
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_wide_128(BatchArgs& a, int dtype, int WB, bool decode, cudaStream_t s) {
    if (WB <= 16) return launch_big_w<128, 16, false>(a, dtype, decode, s);
    return launch_big_w<128, 32, false>(a, dtype, decode, s);
}

}  // namespace pvq
