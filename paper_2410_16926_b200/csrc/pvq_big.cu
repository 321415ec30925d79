// Group size 128 with codes of up to 12 words (the paper's setting at 3 bits per weight,
// Sec. 4.1): kernels that compute in exactly the code's width, instantiated in
// pvq_big_w*.cu; everything else goes to the kernels of pvq_wide*.cu.
#include "pvq_internal.cuh"

namespace pvq {

int launch_big_128_w1_4(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s);
int launch_big_128_w5_8(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s);
int launch_big_128_w9_10(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s);
int launch_big_128_w11_12(BatchArgs& a, int dtype, int W, bool decode, cudaStream_t s);
int launch_wide(BatchArgs& a, int dtype, int N, int W, bool decode, cudaStream_t stream);

int launch_big(const BatchArgs& args, int dtype, int N, int W, bool decode, cudaStream_t stream) {
    BatchArgs a = args;
    if (N == 128 && W <= 12) {
        if (W <= 4) return launch_big_128_w1_4(a, dtype, W, decode, stream);
        if (W <= 8) return launch_big_128_w5_8(a, dtype, W, decode, stream);
        if (W <= 10) return launch_big_128_w9_10(a, dtype, W, decode, stream);
        return launch_big_128_w11_12(a, dtype, W, decode, stream);
    }
    return launch_wide(a, dtype, N, W, decode, stream);
}

}  // namespace pvq
