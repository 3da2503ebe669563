// Second format, MXFP8 (E4M3 elements, one E8M0 scale byte per 32 elements): the activation quantiser and the host
// half of the weight preparation.  The paper's end-to-end setting runs the attention linears in this format
// (Experimental setup) as plain W8A8; the product itself is an instance of the kernel in prq_gemm.cu.
//
// Quantiser: one CTA owns 128 rows x 128 columns -- one 512-byte scale atom, which in this format is a whole reduction
// stage of the GEMM -- and a lane takes one 32-element block of a row, as in the MXFP4 quantiser's identity mode: four
// 16-byte loads, block amax, scale byte from the exponent field (biased exponent - 8: the largest E4M3 magnitude is
// 1.75 * 2^8), sixteen cvt.rn.satfinite.e4m3x2.f32, two 16-byte stores of codes.  With a scale vector the values are
// multiplied by inv_s[j] in fp32 first (Eq. (1), activation side, without a permutation: this format carries no tail).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>

#include "prq_internal.h"
#include "prq_kernels.h"
#include "prq_ptx.cuh"

namespace prq {
namespace {

__device__ __forceinline__ uint32_t cvt_e4m3x4(float f0, float f1, float f2, float f3) {
    uint32_t out;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(out)
        : "f"(f0), "f"(f1), "f"(f2), "f"(f3));
    return out;
}

__global__ void __launch_bounds__(256, 2)
quant_act_fp8_kernel(const uint16_t* __restrict__ x, int M, int ldx, int K, const float* __restrict__ inv_s,
                     uint8_t* __restrict__ codes, uint8_t* __restrict__ scales_row, uint8_t* __restrict__ scales_sf, int act_groups) {
    __shared__ __align__(16) uint8_t sf_atom[512];
    grid_launch_dependents();
    const int atom = blockIdx.x, group = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l4 = lane & 3, rw = lane >> 2;
    const int col = atom * 128 + l4 * 32;
    const bool col_ok = col < K;
    float sc[32];
    if (inv_s && col_ok) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 v = *reinterpret_cast<const float4*>(inv_s + col + 4 * i);
            sc[4 * i] = v.x; sc[4 * i + 1] = v.y; sc[4 * i + 2] = v.z; sc[4 * i + 3] = v.w;
        }
    }
    grid_dependency_wait();
    if (threadIdx.x < 128) reinterpret_cast<uint32_t*>(sf_atom)[threadIdx.x] = 0;
    __syncthreads();
    const int row0 = group * 128, n_rows = min(M, row0 + 128) - row0;
#pragma unroll 1
    for (int i = 0; i < 2; ++i) {
        const int r = i * 64 + warp * 8 + rw;                 // row inside the group
        if (!col_ok || r >= n_rows) continue;
        const uint16_t* xp = x + static_cast<size_t>(row0 + r) * ldx + col;
        uint4 q[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) q[h] = __ldg(reinterpret_cast<const uint4*>(xp + 8 * h));
        float v[32];
        const uint32_t* qw = reinterpret_cast<const uint32_t*>(q);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            v[2 * e] = __uint_as_float(qw[e] << 16);
            v[2 * e + 1] = __uint_as_float(qw[e] & 0xffff0000u);
        }
        if (inv_s) {
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] *= sc[e];
        }
        float am = 0.f;
#pragma unroll
        for (int e = 0; e < 32; ++e) am = fmaxf(am, fabsf(v[e]));
        const int eb = static_cast<int>(__float_as_uint(am) >> 23) - 8;
        const uint32_t byte = eb < 0 ? 0u : static_cast<uint32_t>(eb);
        const float inv = __uint_as_float((254u - byte) << 23);   // 2^(127 - byte), an exact multiply
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) pk[e] = cvt_e4m3x4(v[4 * e] * inv, v[4 * e + 1] * inv, v[4 * e + 2] * inv, v[4 * e + 3] * inv);
        uint4* cp = reinterpret_cast<uint4*>(codes + static_cast<size_t>(row0 + r) * K + col);
        cp[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        cp[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        sf_atom[(r & 31) * 16 + (r >> 5) * 4 + l4] = static_cast<uint8_t>(byte);
        if (scales_row) scales_row[static_cast<size_t>(row0 + r) * (K / kBlock) + atom * 4 + l4] = static_cast<uint8_t>(byte);
    }
    __syncthreads();
    // the atom's scale bytes, coalesced (rows past the end and blocks past K stay zero = 2^-127)
    if (threadIdx.x < 32)
        reinterpret_cast<uint4*>(scales_sf + (static_cast<size_t>(atom) * act_groups + group) * 512)[threadIdx.x] =
            reinterpret_cast<const uint4*>(sf_atom)[threadIdx.x];
}

// One value to E4M3 under the block scale 2^e: round to nearest, ties to the even mantissa, saturating at 448.
uint8_t e4m3_code(float v, int e) {
    uint32_t u;
    std::memcpy(&u, &v, 4);
    const uint8_t sign = static_cast<uint8_t>((u >> 24) & 0x80);
    const float a = std::ldexp(std::fabs(v), -e);             // exact (or underflows far below the smallest step)
    if (!(a < 464.f)) return sign | 0x7E;
    if (a < 0.015625f) {                                       // below 2^-6: multiples of 2^-9
        const int q = static_cast<int>(std::nearbyint(a * 512.f));
        return sign | static_cast<uint8_t>(q == 8 ? 0x08 : q);
    }
    uint32_t b;
    std::memcpy(&b, &a, 4);
    b += 0x7FFFFu + ((b >> 20) & 1u);                          // round the 23-bit mantissa to 3 bits, ties to even
    const int ex = static_cast<int>(b >> 23) - 127, man = static_cast<int>((b >> 20) & 7u);
    if (ex > 8 || (ex == 8 && man > 6)) return sign | 0x7E;
    return sign | static_cast<uint8_t>(((ex + 7) << 3) | man);
}

}  // namespace

cudaError_t launch_quant_act_fp8(const uint16_t* x, int M, int ldx, int K, const float* inv_s, uint8_t* codes,
                                 uint8_t* scales_row, uint8_t* scales_sf, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    const int groups = (M + kGroupRows - 1) / kGroupRows;
    cfg.gridDim = dim3((K + 127) / 128, groups);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, quant_act_fp8_kernel, x, M, ldx, K, inv_s, codes, scales_row, scales_sf, groups);
}

// Offline half of an MXFP8 layer for one alpha, on the host: s = max(amax, 1e-5)^alpha, W0 = fl32(W * s), quantise by rows.
prq_status prepare_layer_fp8(const uint16_t* W, int N, int K, const float* amax, float alpha, std::vector<float>& s,
                             std::vector<float>& inv_s, std::vector<uint8_t>& codes, std::vector<uint8_t>& scales) {
    prq_status st = channel_scales(amax, K, alpha, s, inv_s);
    if (st != PRQ_OK) return st;
    codes.assign(static_cast<size_t>(N) * K, 0);
    scales.assign(static_cast<size_t>(N) * K / kBlock, 0);
    for (int n = 0; n < N; ++n)
        for (int b = 0; b < K / kBlock; ++b) {
            float v[kBlock], am = 0.f;
            for (int i = 0; i < kBlock; ++i) {
                const int j = b * kBlock + i;
                const uint32_t u = static_cast<uint32_t>(W[static_cast<size_t>(n) * K + j]) << 16;
                float w;
                std::memcpy(&w, &u, 4);
                if (!std::isfinite(w)) return PRQ_ERR_NONFINITE;
                v[i] = w * s[j];                               // bf16 x fp32 -> fp32, one rounding
                am = std::fmax(am, std::fabs(v[i]));
            }
            if (!std::isfinite(am)) return PRQ_ERR_NONFINITE;
            uint32_t ab;
            std::memcpy(&ab, &am, 4);
            const int eb = static_cast<int>(ab >> 23) - 8;
            const int byte = am == 0.f ? 0 : (eb < 0 ? 0 : eb);
            scales[static_cast<size_t>(n) * (K / kBlock) + b] = static_cast<uint8_t>(byte);
            for (int i = 0; i < kBlock; ++i) codes[static_cast<size_t>(n) * K + b * kBlock + i] = e4m3_code(v[i], byte - 127);
        }
    return PRQ_OK;
}

}  // namespace prq
