// Device pieces shared by the builder of the search section (pvq_tables.cu) and the decoder
// that uses it (pvq_decode_search.cu); the section is described at SearchLayout.
#pragma once
#include <cstdint>

namespace pvq {

// Key of a W-word integer q >= 1: q truncated to its leading 24 bits, as the bits of an fp32.
// Every conversion and every multiply-add rounds towards zero, and a truncation of a
// truncation is the truncation, so the result is exact whatever the width; it never
// decreases when q grows, which is all the bucket tables need.
__device__ __forceinline__ uint32_t search_key(const uint32_t* q, int W) {
    float x = 0.0f;
    for (int w = W - 1; w >= 0; --w) x = __fmaf_rz(x, 4294967296.0f, __uint2float_rz(q[w]));
    return __float_as_uint(x);
}

template <int W>
__device__ __forceinline__ uint32_t search_key(const uint32_t (&q)[W]) {
    float x = __uint2float_rz(q[W - 1]);
#pragma unroll
    for (int w = W - 2; w >= 0; --w) x = __fmaf_rz(x, 4294967296.0f, __uint2float_rz(q[w]));
    return __float_as_uint(x);
}

constexpr uint32_t kSearchKeyOfOne = 0x3f800000u;  // search_key(1)

}  // namespace pvq
