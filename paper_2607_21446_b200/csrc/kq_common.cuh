// Shared device helpers of the KroQuant kernels: bf16 widening, the MXFP4 block
// encoder (E8M0 scale byte + E2M1 codes) and small PTX wrappers.
//
// Encoder, per 32-value block (paper Section 3.1 blockwise quantizer; Section 4.1
// "Data format": E2M1 elements with one E8M0 scale per 32 block, OCP Microscaling):
//   S    = max(biased_exponent(amax) - 2, 0)        (= floor(log2 amax) - 2 + 127, clamped)
//   v_c  = y_c * 2^(127 - S)                        (exact; |v_c| < 8)
//   code = hardware float -> E2M1 convert (round-to-nearest-even, saturating at 6)
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kq {

// One factor set as the kernels read it: g[k] = {G_k[0][0], G_k[0][1], G_k[1][0], G_k[1][1]}.
struct FactorSet { float4 g[5]; };


constexpr int kBlock = 32;  // channels per MX block

__device__ __forceinline__ float bf16lo_to_f32(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

// 8 bf16 (one 16-byte vector) -> 8 floats, channel order preserved.
__device__ __forceinline__ void widen8(const uint4& p, float (&x)[8]) {
    x[0] = bf16lo_to_f32(p.x); x[1] = bf16hi_to_f32(p.x);
    x[2] = bf16lo_to_f32(p.y); x[3] = bf16hi_to_f32(p.y);
    x[4] = bf16lo_to_f32(p.z); x[5] = bf16hi_to_f32(p.z);
    x[6] = bf16lo_to_f32(p.w); x[7] = bf16hi_to_f32(p.w);
}

// 8 fp16 (one 16-byte vector) -> 8 floats (exact), channel order preserved.
__device__ __forceinline__ void widen8_f16(const uint4& p, float (&x)[8]) {
    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
template <bool XF16>
__device__ __forceinline__ void widen8_any(const uint4& p, float (&x)[8]) {
    if (XF16) widen8_f16(p, x); else widen8(p, x);
}

// E8M0 byte from a block amax (amax >= 0, finite).
__device__ __forceinline__ uint32_t e8m0_from_amax(float amax) {
    int e = (int)((__float_as_uint(amax) >> 23) & 0xFFu) - 2;
    return (uint32_t)(e < 0 ? 0 : e);
}
// 2^(127 - S) as a float; S <= 252 keeps it a normal number.
__device__ __forceinline__ float inv_scale_from_e8m0(uint32_t S) { return __uint_as_float((254u - S) << 23); }
// 2^(S - 127); S == 0 is the subnormal 2^-127.
__device__ __forceinline__ float scale_from_e8m0(uint32_t S) {
    return __uint_as_float(S ? (S << 23) : 0x00400000u);
}

// Eight scaled values -> eight E2M1 codes packed into 32 bits: value i in nibble i
// (even channel in the low nibble of its byte).  The convert puts its FIRST source
// operand into the high nibble.
__device__ __forceinline__ uint32_t e2m1x8(float v0, float v1, float v2, float v3,
                                           float v4, float v5, float v6, float v7) {
    uint32_t out;
    asm("{\n\t"
        ".reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t"
        "}"
        : "=r"(out)
        : "f"(v0), "f"(v1), "f"(v2), "f"(v3), "f"(v4), "f"(v5), "f"(v6), "f"(v7));
    return out;
}

// two E2M1 codes (one byte, even element in the low nibble) -> two floats, by the hardware convert
__device__ __forceinline__ float2 e2m1x2_to_float2(uint32_t byte) {
    uint32_t h2;
    asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(h2) : "r"(byte));
    return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}
__device__ __forceinline__ float absmax8(const float (&y)[8]) {
    float m = fmaxf(fabsf(y[0]), fabsf(y[1]));
    m = fmaxf(m, fmaxf(fabsf(y[2]), fabsf(y[3])));
    m = fmaxf(m, fmaxf(fabsf(y[4]), fabsf(y[5])));
    m = fmaxf(m, fmaxf(fabsf(y[6]), fabsf(y[7])));
    return m;
}

// Position of the scale byte of (row t, block j) in the 128 x 4 tiled layout that block-scaled
// tensor-core GEMMs read (tiles of 512 bytes, row-tile-major; cb = ceil(blocks_per_row / 4)).
__device__ __forceinline__ int64_t tiled_scale_index(int64_t t, int j, int cb) {
    return ((t >> 7) * cb + (j >> 2)) * 512 + (t & 31) * 16 + ((t >> 5) & 3) * 4 + (j & 3);
}

// streaming (read-once / write-once) global accesses
__device__ __forceinline__ uint4 ld_stream_16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_16(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_stream_4(void* p, uint32_t v) {
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

}  // namespace kq
