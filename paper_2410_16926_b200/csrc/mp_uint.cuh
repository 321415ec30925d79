// Multi-word unsigned integers for the Fischer enumeration (Sec. 4.5: integer
// codes wider than any native type, handled with the carry flag of the 32-bit
// add / subtract instructions).  A number is W little-endian 32-bit limbs held
// in registers.  Every add or subtract is ONE asm statement holding the whole
// carry chain, so nothing can be scheduled between two links of it.
#pragma once
#include <cstdint>

namespace pvq {

template <int W>
struct mp {
    uint32_t w[W];
};

// a += b (the caller knows the sum fits W limbs).  Widths 1..12 are specialised below; wider
// numbers take this plain form, whose carries the compiler turns into the same chain.
template <int W>
__device__ __forceinline__ void mp_add(mp<W>& a, const mp<W>& b) {
    uint64_t c = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
        const uint64_t s = static_cast<uint64_t>(a.w[w]) + b.w[w] + c;
        a.w[w] = static_cast<uint32_t>(s);
        c = s >> 32;
    }
}

// d = a - b; returns true when a < b (a borrow leaves the top limb)
template <int W>
__device__ __forceinline__ bool mp_sub_borrow(mp<W>& d, const mp<W>& a, const mp<W>& b) {
    uint64_t brw = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
        const uint64_t s = static_cast<uint64_t>(a.w[w]) - b.w[w] - brw;
        d.w[w] = static_cast<uint32_t>(s);
        brw = (s >> 32) & 1u;
    }
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<1>(mp<1>& a, const mp<1>& b) {
    a.w[0] += b.w[0];
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<1>(mp<1>& d, const mp<1>& a, const mp<1>& b) {
    d.w[0] = a.w[0] - b.w[0];
    return a.w[0] < b.w[0];
}

template <>
__device__ __forceinline__ void mp_add<2>(mp<2>& a, const mp<2>& b) {
    asm("add.cc.u32 %0, %0, %2;\n\t"
        "addc.u32 %1, %1, %3;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1])
        : "r"(b.w[0]), "r"(b.w[1]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<2>(mp<2>& d, const mp<2>& a, const mp<2>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %3, %5;\n\t"
        "subc.cc.u32 %1, %4, %6;\n\t"
        "subc.u32 %2, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(b.w[0]), "r"(b.w[1]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<3>(mp<3>& a, const mp<3>& b) {
    asm("add.cc.u32 %0, %0, %3;\n\t"
        "addc.cc.u32 %1, %1, %4;\n\t"
        "addc.u32 %2, %2, %5;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<3>(mp<3>& d, const mp<3>& a, const mp<3>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %4, %7;\n\t"
        "subc.cc.u32 %1, %5, %8;\n\t"
        "subc.cc.u32 %2, %6, %9;\n\t"
        "subc.u32 %3, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<4>(mp<4>& a, const mp<4>& b) {
    asm("add.cc.u32 %0, %0, %4;\n\t"
        "addc.cc.u32 %1, %1, %5;\n\t"
        "addc.cc.u32 %2, %2, %6;\n\t"
        "addc.u32 %3, %3, %7;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<4>(mp<4>& d, const mp<4>& a, const mp<4>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %5, %9;\n\t"
        "subc.cc.u32 %1, %6, %10;\n\t"
        "subc.cc.u32 %2, %7, %11;\n\t"
        "subc.cc.u32 %3, %8, %12;\n\t"
        "subc.u32 %4, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<5>(mp<5>& a, const mp<5>& b) {
    asm("add.cc.u32 %0, %0, %5;\n\t"
        "addc.cc.u32 %1, %1, %6;\n\t"
        "addc.cc.u32 %2, %2, %7;\n\t"
        "addc.cc.u32 %3, %3, %8;\n\t"
        "addc.u32 %4, %4, %9;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<5>(mp<5>& d, const mp<5>& a, const mp<5>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %6, %11;\n\t"
        "subc.cc.u32 %1, %7, %12;\n\t"
        "subc.cc.u32 %2, %8, %13;\n\t"
        "subc.cc.u32 %3, %9, %14;\n\t"
        "subc.cc.u32 %4, %10, %15;\n\t"
        "subc.u32 %5, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<6>(mp<6>& a, const mp<6>& b) {
    asm("add.cc.u32 %0, %0, %6;\n\t"
        "addc.cc.u32 %1, %1, %7;\n\t"
        "addc.cc.u32 %2, %2, %8;\n\t"
        "addc.cc.u32 %3, %3, %9;\n\t"
        "addc.cc.u32 %4, %4, %10;\n\t"
        "addc.u32 %5, %5, %11;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<6>(mp<6>& d, const mp<6>& a, const mp<6>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %7, %13;\n\t"
        "subc.cc.u32 %1, %8, %14;\n\t"
        "subc.cc.u32 %2, %9, %15;\n\t"
        "subc.cc.u32 %3, %10, %16;\n\t"
        "subc.cc.u32 %4, %11, %17;\n\t"
        "subc.cc.u32 %5, %12, %18;\n\t"
        "subc.u32 %6, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<7>(mp<7>& a, const mp<7>& b) {
    asm("add.cc.u32 %0, %0, %7;\n\t"
        "addc.cc.u32 %1, %1, %8;\n\t"
        "addc.cc.u32 %2, %2, %9;\n\t"
        "addc.cc.u32 %3, %3, %10;\n\t"
        "addc.cc.u32 %4, %4, %11;\n\t"
        "addc.cc.u32 %5, %5, %12;\n\t"
        "addc.u32 %6, %6, %13;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<7>(mp<7>& d, const mp<7>& a, const mp<7>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %8, %15;\n\t"
        "subc.cc.u32 %1, %9, %16;\n\t"
        "subc.cc.u32 %2, %10, %17;\n\t"
        "subc.cc.u32 %3, %11, %18;\n\t"
        "subc.cc.u32 %4, %12, %19;\n\t"
        "subc.cc.u32 %5, %13, %20;\n\t"
        "subc.cc.u32 %6, %14, %21;\n\t"
        "subc.u32 %7, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<8>(mp<8>& a, const mp<8>& b) {
    asm("add.cc.u32 %0, %0, %8;\n\t"
        "addc.cc.u32 %1, %1, %9;\n\t"
        "addc.cc.u32 %2, %2, %10;\n\t"
        "addc.cc.u32 %3, %3, %11;\n\t"
        "addc.cc.u32 %4, %4, %12;\n\t"
        "addc.cc.u32 %5, %5, %13;\n\t"
        "addc.cc.u32 %6, %6, %14;\n\t"
        "addc.u32 %7, %7, %15;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6]), "+&r"(a.w[7])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<8>(mp<8>& d, const mp<8>& a, const mp<8>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %9, %17;\n\t"
        "subc.cc.u32 %1, %10, %18;\n\t"
        "subc.cc.u32 %2, %11, %19;\n\t"
        "subc.cc.u32 %3, %12, %20;\n\t"
        "subc.cc.u32 %4, %13, %21;\n\t"
        "subc.cc.u32 %5, %14, %22;\n\t"
        "subc.cc.u32 %6, %15, %23;\n\t"
        "subc.cc.u32 %7, %16, %24;\n\t"
        "subc.u32 %8, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(d.w[7]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(a.w[7]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<9>(mp<9>& a, const mp<9>& b) {
    asm("add.cc.u32 %0, %0, %9;\n\t"
        "addc.cc.u32 %1, %1, %10;\n\t"
        "addc.cc.u32 %2, %2, %11;\n\t"
        "addc.cc.u32 %3, %3, %12;\n\t"
        "addc.cc.u32 %4, %4, %13;\n\t"
        "addc.cc.u32 %5, %5, %14;\n\t"
        "addc.cc.u32 %6, %6, %15;\n\t"
        "addc.cc.u32 %7, %7, %16;\n\t"
        "addc.u32 %8, %8, %17;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6]), "+&r"(a.w[7]), "+&r"(a.w[8])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<9>(mp<9>& d, const mp<9>& a, const mp<9>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %10, %19;\n\t"
        "subc.cc.u32 %1, %11, %20;\n\t"
        "subc.cc.u32 %2, %12, %21;\n\t"
        "subc.cc.u32 %3, %13, %22;\n\t"
        "subc.cc.u32 %4, %14, %23;\n\t"
        "subc.cc.u32 %5, %15, %24;\n\t"
        "subc.cc.u32 %6, %16, %25;\n\t"
        "subc.cc.u32 %7, %17, %26;\n\t"
        "subc.cc.u32 %8, %18, %27;\n\t"
        "subc.u32 %9, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(d.w[7]), "=&r"(d.w[8]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(a.w[7]), "r"(a.w[8]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<10>(mp<10>& a, const mp<10>& b) {
    asm("add.cc.u32 %0, %0, %10;\n\t"
        "addc.cc.u32 %1, %1, %11;\n\t"
        "addc.cc.u32 %2, %2, %12;\n\t"
        "addc.cc.u32 %3, %3, %13;\n\t"
        "addc.cc.u32 %4, %4, %14;\n\t"
        "addc.cc.u32 %5, %5, %15;\n\t"
        "addc.cc.u32 %6, %6, %16;\n\t"
        "addc.cc.u32 %7, %7, %17;\n\t"
        "addc.cc.u32 %8, %8, %18;\n\t"
        "addc.u32 %9, %9, %19;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6]), "+&r"(a.w[7]), "+&r"(a.w[8]), "+&r"(a.w[9])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<10>(mp<10>& d, const mp<10>& a, const mp<10>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %11, %21;\n\t"
        "subc.cc.u32 %1, %12, %22;\n\t"
        "subc.cc.u32 %2, %13, %23;\n\t"
        "subc.cc.u32 %3, %14, %24;\n\t"
        "subc.cc.u32 %4, %15, %25;\n\t"
        "subc.cc.u32 %5, %16, %26;\n\t"
        "subc.cc.u32 %6, %17, %27;\n\t"
        "subc.cc.u32 %7, %18, %28;\n\t"
        "subc.cc.u32 %8, %19, %29;\n\t"
        "subc.cc.u32 %9, %20, %30;\n\t"
        "subc.u32 %10, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(d.w[7]), "=&r"(d.w[8]), "=&r"(d.w[9]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(a.w[7]), "r"(a.w[8]), "r"(a.w[9]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<11>(mp<11>& a, const mp<11>& b) {
    asm("add.cc.u32 %0, %0, %11;\n\t"
        "addc.cc.u32 %1, %1, %12;\n\t"
        "addc.cc.u32 %2, %2, %13;\n\t"
        "addc.cc.u32 %3, %3, %14;\n\t"
        "addc.cc.u32 %4, %4, %15;\n\t"
        "addc.cc.u32 %5, %5, %16;\n\t"
        "addc.cc.u32 %6, %6, %17;\n\t"
        "addc.cc.u32 %7, %7, %18;\n\t"
        "addc.cc.u32 %8, %8, %19;\n\t"
        "addc.cc.u32 %9, %9, %20;\n\t"
        "addc.u32 %10, %10, %21;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6]), "+&r"(a.w[7]), "+&r"(a.w[8]), "+&r"(a.w[9]), "+&r"(a.w[10])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]), "r"(b.w[10]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<11>(mp<11>& d, const mp<11>& a, const mp<11>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %12, %23;\n\t"
        "subc.cc.u32 %1, %13, %24;\n\t"
        "subc.cc.u32 %2, %14, %25;\n\t"
        "subc.cc.u32 %3, %15, %26;\n\t"
        "subc.cc.u32 %4, %16, %27;\n\t"
        "subc.cc.u32 %5, %17, %28;\n\t"
        "subc.cc.u32 %6, %18, %29;\n\t"
        "subc.cc.u32 %7, %19, %30;\n\t"
        "subc.cc.u32 %8, %20, %31;\n\t"
        "subc.cc.u32 %9, %21, %32;\n\t"
        "subc.cc.u32 %10, %22, %33;\n\t"
        "subc.u32 %11, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(d.w[7]), "=&r"(d.w[8]), "=&r"(d.w[9]), "=&r"(d.w[10]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(a.w[7]), "r"(a.w[8]), "r"(a.w[9]), "r"(a.w[10]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]), "r"(b.w[10]));
    return brw != 0u;
}

template <>
__device__ __forceinline__ void mp_add<12>(mp<12>& a, const mp<12>& b) {
    asm("add.cc.u32 %0, %0, %12;\n\t"
        "addc.cc.u32 %1, %1, %13;\n\t"
        "addc.cc.u32 %2, %2, %14;\n\t"
        "addc.cc.u32 %3, %3, %15;\n\t"
        "addc.cc.u32 %4, %4, %16;\n\t"
        "addc.cc.u32 %5, %5, %17;\n\t"
        "addc.cc.u32 %6, %6, %18;\n\t"
        "addc.cc.u32 %7, %7, %19;\n\t"
        "addc.cc.u32 %8, %8, %20;\n\t"
        "addc.cc.u32 %9, %9, %21;\n\t"
        "addc.cc.u32 %10, %10, %22;\n\t"
        "addc.u32 %11, %11, %23;\n\t"
        : "+&r"(a.w[0]), "+&r"(a.w[1]), "+&r"(a.w[2]), "+&r"(a.w[3]), "+&r"(a.w[4]), "+&r"(a.w[5]), "+&r"(a.w[6]), "+&r"(a.w[7]), "+&r"(a.w[8]), "+&r"(a.w[9]), "+&r"(a.w[10]), "+&r"(a.w[11])
        : "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]), "r"(b.w[10]), "r"(b.w[11]));
}

template <>
__device__ __forceinline__ bool mp_sub_borrow<12>(mp<12>& d, const mp<12>& a, const mp<12>& b) {
    uint32_t brw;
    asm("sub.cc.u32 %0, %13, %25;\n\t"
        "subc.cc.u32 %1, %14, %26;\n\t"
        "subc.cc.u32 %2, %15, %27;\n\t"
        "subc.cc.u32 %3, %16, %28;\n\t"
        "subc.cc.u32 %4, %17, %29;\n\t"
        "subc.cc.u32 %5, %18, %30;\n\t"
        "subc.cc.u32 %6, %19, %31;\n\t"
        "subc.cc.u32 %7, %20, %32;\n\t"
        "subc.cc.u32 %8, %21, %33;\n\t"
        "subc.cc.u32 %9, %22, %34;\n\t"
        "subc.cc.u32 %10, %23, %35;\n\t"
        "subc.cc.u32 %11, %24, %36;\n\t"
        "subc.u32 %12, 0, 0;"
        : "=&r"(d.w[0]), "=&r"(d.w[1]), "=&r"(d.w[2]), "=&r"(d.w[3]), "=&r"(d.w[4]), "=&r"(d.w[5]), "=&r"(d.w[6]), "=&r"(d.w[7]), "=&r"(d.w[8]), "=&r"(d.w[9]), "=&r"(d.w[10]), "=&r"(d.w[11]), "=&r"(brw)
        : "r"(a.w[0]), "r"(a.w[1]), "r"(a.w[2]), "r"(a.w[3]), "r"(a.w[4]), "r"(a.w[5]), "r"(a.w[6]), "r"(a.w[7]), "r"(a.w[8]), "r"(a.w[9]), "r"(a.w[10]), "r"(a.w[11]), "r"(b.w[0]), "r"(b.w[1]), "r"(b.w[2]), "r"(b.w[3]), "r"(b.w[4]), "r"(b.w[5]), "r"(b.w[6]), "r"(b.w[7]), "r"(b.w[8]), "r"(b.w[9]), "r"(b.w[10]), "r"(b.w[11]));
    return brw != 0u;
}

// if (a >= b) { a -= b; return true; } else return false;
template <int W>
__device__ __forceinline__ bool mp_sub_if_ge(mp<W>& a, const mp<W>& b) {
    mp<W> d;
    const bool lt = mp_sub_borrow<W>(d, a, b);
    if (!lt) a = d;
    return !lt;
}

// a = 2 * a (the caller knows the result fits W limbs)
template <int W>
__device__ __forceinline__ void mp_dbl(mp<W>& a) {
#pragma unroll
    for (int i = W - 1; i >= 1; --i) a.w[i] = __funnelshift_l(a.w[i - 1], a.w[i], 1);
    a.w[0] <<= 1;
}

template <int W>
__device__ __forceinline__ bool mp_is_zero(const mp<W>& a) {
    uint32_t o = 0;
#pragma unroll
    for (int i = 0; i < W; ++i) o |= a.w[i];
    return o == 0u;
}

template <int W>
__device__ __forceinline__ void mp_zero(mp<W>& a) {
#pragma unroll
    for (int i = 0; i < W; ++i) a.w[i] = 0u;
}

// an entry of the count table: W consecutive words in shared or global memory
template <int W>
__device__ __forceinline__ mp<W> mp_load(const uint32_t* p) {
    mp<W> a;
#pragma unroll
    for (int i = 0; i < W; ++i) a.w[i] = p[i];
    return a;
}

}  // namespace pvq
