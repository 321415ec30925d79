// Codes wider than the shared-memory kernels take (group sizes 16 to 64) or than 12 words
// (group size 128), and group size 256: the global-table kernels computing in the next of
// 8, 16 or 32 words (the paper's grid of group sizes and direction bits, Sec. 4.1).  Group
// sizes 16 to 64 are instantiated here, 128 and 256 in pvq_wide_n128.cu and pvq_wide_n256.cu.
#include "pvq_big_impl.cuh"

namespace pvq {

int launch_wide_128(BatchArgs& a, int dtype, int WB, bool decode, cudaStream_t s);
int launch_wide_256(BatchArgs& a, int dtype, int WB, bool decode, cudaStream_t s);

int launch_wide(BatchArgs& a, int dtype, int N, int W, bool decode, cudaStream_t s) {
    const int WB = W <= 8 ? 8 : (W <= 16 ? 16 : 32);
    switch (N) {
        case 16:
            if (WB == 8) return launch_big_w<16, 8, false>(a, dtype, decode, s);
            break;
        case 32:
            if (WB == 8) return launch_big_w<32, 8, false>(a, dtype, decode, s);
            break;
        case 64:
            if (WB == 8) return launch_big_w<64, 8, false>(a, dtype, decode, s);
            if (WB == 16) return launch_big_w<64, 16, false>(a, dtype, decode, s);
            break;
        case 128: return launch_wide_128(a, dtype, WB, decode, s);
        case 256: return launch_wide_256(a, dtype, WB, decode, s);
        default: break;
    }
    return PVQ_ERR_UNSUPPORTED;
}

}  // namespace pvq
