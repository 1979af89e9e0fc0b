// NVFP4 scalar steps shared by the quantizer kernels and the quantizing GEMM epilogue (device only).
// The sequence is the one that decides bit-exactness: v = a / (6 T) (IEEE division), sb = E4M3 of v
// (nearest even, saturating), d = float(sb) * T, rcp = 1 / d (0 when sb is 0), code = E2M1 of x * rcp.
#pragma once
#include <stdint.h>

namespace sol {
namespace qmath {

// max(|a|, |b|) per BF16 half (the sign bits of the result are garbage and masked off later)
__device__ __forceinline__ uint32_t absmax2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ uint32_t f32_to_e4m3_sat(float v) {
    uint16_t packed;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(packed) : "f"(0.0f), "f"(v));
    return packed & 0xFFu;
}

__device__ __forceinline__ float e4m3_to_f32(uint32_t code) {
    uint32_t e = (code >> 3) & 15u, m = code & 7u;
    if (e == 0) return __uint2float_rn(m) * 0x1p-9f;
    return __uint_as_float(((e + 120u) << 23) | (m << 20));
}

// Eight FP32 values -> eight E2M1 nibbles (element 0 in the lowest nibble).
__device__ __forceinline__ uint32_t pack_e2m1x8(float y0, float y1, float y2, float y3, float y4, float y5,
                                                float y6, float y7) {
    uint32_t out;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(out)
        : "f"(y0), "f"(y1), "f"(y2), "f"(y3), "f"(y4), "f"(y5), "f"(y6), "f"(y7));
    return out;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Eight packed BF16 values (four words) times rcp -> eight nibbles.
__device__ __forceinline__ uint32_t quantize8(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, float rcp) {
    return pack_e2m1x8(__fmul_rn(bf16_lo(w0), rcp), __fmul_rn(bf16_hi(w0), rcp), __fmul_rn(bf16_lo(w1), rcp),
                       __fmul_rn(bf16_hi(w1), rcp), __fmul_rn(bf16_lo(w2), rcp), __fmul_rn(bf16_hi(w2), rcp),
                       __fmul_rn(bf16_lo(w3), rcp), __fmul_rn(bf16_hi(w3), rcp));
}

// Two-lane FP32 arithmetic (one instruction for two IEEE operations, each rounded on its own: results
// are bit for bit those of the scalar forms).  A pair lives in a 64-bit register, low lane first.
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f32x2_of_bf16x2(uint32_t w) { return f32x2(bf16_lo(w), bf16_hi(w)); }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Eight packed BF16 values (four words) times rcp -> eight nibbles, the products taken two at a time.
__device__ __forceinline__ uint32_t quantize8_x2(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint64_t rcp2) {
    float y[8];
    f32x2_split(mul2(f32x2_of_bf16x2(w0), rcp2), y[0], y[1]);
    f32x2_split(mul2(f32x2_of_bf16x2(w1), rcp2), y[2], y[3]);
    f32x2_split(mul2(f32x2_of_bf16x2(w2), rcp2), y[4], y[5]);
    f32x2_split(mul2(f32x2_of_bf16x2(w3), rcp2), y[6], y[7]);
    return pack_e2m1x8(y[0], y[1], y[2], y[3], y[4], y[5], y[6], y[7]);
}

// Block scale byte and reciprocal from the block's max magnitude a, c = 6 T and T.
__device__ __forceinline__ uint32_t block_scale(float a, float c, float T, float &rcp) {
    const float sv = __fdiv_rn(a, c);
    const uint32_t sb = f32_to_e4m3_sat(sv);
    const float d = __fmul_rn(e4m3_to_f32(sb), T);
    rcp = sb ? __frcp_rn(d) : 0.0f;
    return sb;
}

}  // namespace qmath
}  // namespace sol
