// MXFP4 quantisation of one 32-element block held by one thread as 64 bytes of bf16 (four 16-byte
// words in memory order): block amax -> E8M0 byte (biased exponent - 2, floored at 0) -> 32
// round-to-nearest-even E2M1 codes, element 0 in the lowest nibble.  Shared by the activation quantiser
// (identity mode) and by the decode GEMM that quantises its activations itself, so that both produce the
// same bits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace prq {

// Eight floats -> four bytes of E2M1 codes (element 0 in the lowest nibble): round to nearest even,
// saturating; the sign of values that round to zero (and of negative zero) is kept.
__device__ __forceinline__ uint32_t cvt_e2m1x8(float f0, float f1, float f2, float f3, float f4, float f5, float f6,
                                               float f7) {
    uint32_t out;
    asm("{\n\t.reg .b8 t0, t1, t2, t3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n\t"
        "mov.b32 %0, {t0, t1, t2, t3};\n\t}"
        : "=r"(out)
        : "f"(f0), "f"(f1), "f"(f2), "f"(f3), "f"(f4), "f"(f5), "f"(f6), "f"(f7));
    return out;
}

__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) { return *reinterpret_cast<__nv_bfloat162*>(&w); }
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 h) { return *reinterpret_cast<uint32_t*>(&h); }

// q: the block's 32 bf16 values.  Returns the E8M0 byte; codes = the 16 bytes of packed E2M1 codes.
__device__ __forceinline__ uint32_t quant_block32(const uint4 (&q)[4], uint4& codes) {
    // block amax: packed bf16 |.| and max over the sixteen pairs, then the two halves
    __nv_bfloat162 am = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const __nv_bfloat162 a0 = __hmax2(__habs2(as_bf162(q[h].x)), __habs2(as_bf162(q[h].y)));
        const __nv_bfloat162 a1 = __hmax2(__habs2(as_bf162(q[h].z)), __habs2(as_bf162(q[h].w)));
        am = __hmax2(am, __hmax2(a0, a1));
    }
    const uint32_t mm = as_u32(am);
    const uint32_t m = max(mm & 0xffffu, mm >> 16);
    // E8M0 byte = biased exponent - 2 (floored at 0); 2^(127 - byte) as a packed bf16 pair.
    // Multiplying bf16 by a power of two is exact (results too small for bf16 round to code 0
    // in any case), so the scaling is done on pairs before widening to fp32.
    const int eb = static_cast<int>(m >> 7) - 2;
    const uint32_t byte = eb < 0 ? 0u : static_cast<uint32_t>(eb);
    const uint32_t inv1 = (254u - byte) << 7;
    const __nv_bfloat162 inv2 = as_bf162(inv1 | (inv1 << 16));
    uint32_t pk[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const uint32_t s0 = as_u32(__hmul2(as_bf162(q[h].x), inv2)), s1 = as_u32(__hmul2(as_bf162(q[h].y), inv2));
        const uint32_t s2 = as_u32(__hmul2(as_bf162(q[h].z), inv2)), s3 = as_u32(__hmul2(as_bf162(q[h].w), inv2));
        pk[h] = cvt_e2m1x8(__uint_as_float(s0 << 16), __uint_as_float(s0 & 0xffff0000u),
                           __uint_as_float(s1 << 16), __uint_as_float(s1 & 0xffff0000u),
                           __uint_as_float(s2 << 16), __uint_as_float(s2 & 0xffff0000u),
                           __uint_as_float(s3 << 16), __uint_as_float(s3 & 0xffff0000u));
    }
    codes = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    return byte;
}

}  // namespace prq
