// Group size 256, computed in 8, 16 or 32 words (see pvq_wide.cu).
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_wide_256(BatchArgs& a, int dtype, int WB, bool decode, cudaStream_t s) {
    if (WB == 8) return launch_big_w<256, 8, false>(a, dtype, decode, s);
    if (WB == 16) return launch_big_w<256, 16, false>(a, dtype, decode, s);
    return launch_big_w<256, 32, false>(a, dtype, decode, s);
}

}  // namespace pvq
