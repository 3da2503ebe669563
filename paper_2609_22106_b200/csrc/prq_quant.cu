// Activation quantisation kernel ("the kernel quantizes the reordered activation to MXFP4 once",
// Kernel design paragraph; Eq. (1) activation side when the scale and permutation are applied online).
//
// One CTA owns a tile of 128 rows x 256 columns (one reduction stage of the GEMM): 8 warps x 16 rows,
// a warp covers the 256 columns of a row with one 16-byte load per lane (8 bf16).  A 32-element block
// is 4 adjacent lanes: amax by two shuffles, E8M0 byte from the exponent field, eight
// round-to-nearest-even E2M1 conversions per lane, one 4-byte packed store per lane (128 contiguous
// bytes per warp).  The scale bytes of the tile are collected in shared memory in the GEMM's
// 1024-byte (stage, 128-row group) order and written out coalesced; the bytes of tail blocks are
// also duplicated into the residual stages, which is all the "tail copy" this design needs.
//
// HBM-bound: 2 bytes read + 0.5 + 1/32 written per element.
#include <cuda_runtime.h>

#include "prq_internal.h"
#include "prq_kernels.h"

namespace prq {
namespace {

constexpr int kQuantThreads = 256;
constexpr int kRowsPerWarp = kGroupRows / (kQuantThreads / 32);  // 16

// Two floats -> one byte of E2M1 codes (lo in the low nibble), round to nearest even, saturating.
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi) {
    uint16_t out;
    asm("{\n\t.reg .b8 t;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t, %2, %1;\n\t"
        "cvt.u16.u8 %0, t;\n\t}"
        : "=h"(out)
        : "f"(lo), "f"(hi));
    return out;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <bool kScalePerm>
__global__ void __launch_bounds__(kQuantThreads)
quant_act_kernel(QuantParams p) {
    __shared__ __align__(16) uint8_t sf_tile[kSfGroupBytes];
    __shared__ int s_tile_start[kMaxExperts + 1];

    const int stage = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Which rows does this CTA own?  Dense: group g covers rows [128 g, 128 g + 128).  Grouped: the
    // scale groups are padded per expert, so walk the expert offsets to find ours.
    int row0, row_end, expert = 0;
    const int group = blockIdx.y;
    if (p.expert_offsets == nullptr) {
        row0 = group * kGroupRows;
        row_end = min(p.M, row0 + kGroupRows);
    } else {
        if (threadIdx.x == 0) {
            int acc = 0;
            for (int e = 0; e < p.n_experts; ++e) {
                s_tile_start[e] = acc;
                acc += (p.expert_offsets[e + 1] - p.expert_offsets[e] + kGroupRows - 1) / kGroupRows;
            }
            s_tile_start[p.n_experts] = acc;
        }
        __syncthreads();
        if (group >= s_tile_start[p.n_experts]) return;  // padding CTA of the launch grid
        int lo = 0, hi = p.n_experts - 1;
        while (lo < hi) {  // last expert whose first tile is <= group and that owns tiles
            int mid = (lo + hi + 1) >> 1;
            if (s_tile_start[mid] <= group) lo = mid; else hi = mid - 1;
        }
        expert = lo;
        row0 = p.expert_offsets[expert] + (group - s_tile_start[expert]) * kGroupRows;
        row_end = min(p.expert_offsets[expert + 1], row0 + kGroupRows);
    }

    for (int i = threadIdx.x; i < kSfGroupBytes / 4; i += kQuantThreads) reinterpret_cast<uint32_t*>(sf_tile)[i] = 0;
    __syncthreads();

    const int K = p.K, k_tail = p.k_tail;
    const int col0 = stage * kStageK + lane * 8;  // first of this lane's 8 columns
    const bool col_ok = col0 < K;                 // K % 32 == 0, so a lane is all in or all out
    const int blk_in_stage = lane >> 2;
    const int tail_blk0 = (K - k_tail) / kBlock;  // first tail block (global block index)
    const int gblk = stage * (kStageK / kBlock) + blk_in_stage;
    const StagePlan plan(K, k_tail);
    uint8_t* sf_base = p.scales_sf;
    const size_t sf_group_stride = kSfGroupBytes;
    const size_t sf_stage_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;

    float inv_s[8];
    int src[8];
    if (kScalePerm && col_ok) {
        const int32_t* perm = p.perm + static_cast<size_t>(expert) * K + col0;
        const float* isp = p.inv_s_perm + static_cast<size_t>(expert) * K + col0;
        const int4 p0 = *reinterpret_cast<const int4*>(perm), p1 = *reinterpret_cast<const int4*>(perm + 4);
        const float4 s0 = *reinterpret_cast<const float4*>(isp), s1 = *reinterpret_cast<const float4*>(isp + 4);
        src[0] = p0.x; src[1] = p0.y; src[2] = p0.z; src[3] = p0.w;
        src[4] = p1.x; src[5] = p1.y; src[6] = p1.z; src[7] = p1.w;
        inv_s[0] = s0.x; inv_s[1] = s0.y; inv_s[2] = s0.z; inv_s[3] = s0.w;
        inv_s[4] = s1.x; inv_s[5] = s1.y; inv_s[6] = s1.z; inv_s[7] = s1.w;
    }

#pragma unroll 4
    for (int i = 0; i < kRowsPerWarp; ++i) {
        const int r = warp + i * (kQuantThreads / 32);  // row inside the group
        const int row = row0 + r;
        if (row >= row_end) break;  // warp-uniform
        float v[8];
        if (col_ok) {
            const uint16_t* xrow = p.x + static_cast<size_t>(row) * p.ldx;
            if (kScalePerm) {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    v[e] = __uint_as_float(static_cast<uint32_t>(__ldg(xrow + src[e])) << 16) * inv_s[e];
            } else {
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(xrow + col0));
                v[0] = bf16_lo(q.x); v[1] = bf16_hi(q.x); v[2] = bf16_lo(q.y); v[3] = bf16_hi(q.y);
                v[4] = bf16_lo(q.z); v[5] = bf16_hi(q.z); v[6] = bf16_lo(q.w); v[7] = bf16_hi(q.w);
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = 0.f;
        }
        // block amax over the 4 lanes of a 32-element block (bit patterns of |v| order like the values)
        uint32_t am = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) am = max(am, __float_as_uint(v[e]) & 0x7fffffffu);
        am = max(am, __shfl_xor_sync(0xffffffffu, am, 1));
        am = max(am, __shfl_xor_sync(0xffffffffu, am, 2));
        // E8M0 byte = biased exponent - 2, floored at 0; multiply by 2^(127 - byte) (exact)
        const int eb = static_cast<int>(am >> 23) - 2;
        const uint32_t byte = eb < 0 ? 0u : static_cast<uint32_t>(eb);
        const float inv = __uint_as_float((254u - byte) << 23);
        uint32_t packed = 0;
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            uint32_t b = cvt_e2m1x2(v[e] * inv, v[e + 1] * inv);
            // keep the sign bit of inputs whose magnitude rounded to zero
            b |= ((__float_as_uint(v[e]) >> 28) & 0x8u) | ((__float_as_uint(v[e + 1]) >> 24) & 0x80u);
            packed |= b << (4 * e);
        }
        if (col_ok) {
            *reinterpret_cast<uint32_t*>(p.codes + static_cast<size_t>(row) * (K / 2) + col0 / 2) = packed;
            if ((lane & 3) == 0) {
                sf_tile[sf_offset_in_group(r, blk_in_stage)] = static_cast<uint8_t>(byte);
                if (p.scales_row) p.scales_row[static_cast<size_t>(row) * (K / kBlock) + gblk] = static_cast<uint8_t>(byte);
                if (gblk >= tail_blk0) {  // duplicate the tail block's scale into its residual stage
                    const int t = gblk - tail_blk0;
                    const int ts = plan.S1 + t / (kStageK / kBlock);
                    sf_base[ts * sf_stage_stride + group * sf_group_stride +
                            sf_offset_in_group(r, t % (kStageK / kBlock))] = static_cast<uint8_t>(byte);
                }
            }
        }
    }
    __syncthreads();
    // the tile's scale bytes, coalesced (rows past the end and blocks past K stay zero = 2^-127)
    if (threadIdx.x < kSfGroupBytes / 16) {
        reinterpret_cast<uint4*>(sf_base + stage * sf_stage_stride + group * sf_group_stride)[threadIdx.x] =
            reinterpret_cast<const uint4*>(sf_tile)[threadIdx.x];
    }
    // The CTA of the last main stage also zero-fills what nobody else writes in the residual stages:
    // blocks past k_tail, and every byte of rows past the end of the group.
    if (stage == plan.S1 - 1 && plan.S > plan.S1) {
        const int nb = kStageK / kBlock;
        for (int idx = threadIdx.x; idx < (plan.S - plan.S1) * kGroupRows * nb; idx += kQuantThreads) {
            const int ts = idx / (kGroupRows * nb);
            const int r = (idx / nb) % kGroupRows;
            const int b = idx % nb;
            const bool live = (row0 + r < row_end) && (ts * nb + b) < k_tail / kBlock;
            if (!live)
                sf_base[(plan.S1 + ts) * sf_stage_stride + group * sf_group_stride + sf_offset_in_group(r, b)] = 0;
        }
    }
}

}  // namespace

cudaError_t launch_quant_act(const QuantParams& p, bool scale_perm, int grid_groups, cudaStream_t stream) {
    const StagePlan plan(p.K, p.k_tail);
    dim3 grid(plan.S1, grid_groups);
    if (scale_perm) quant_act_kernel<true><<<grid, kQuantThreads, 0, stream>>>(p);
    else quant_act_kernel<false><<<grid, kQuantThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace prq
