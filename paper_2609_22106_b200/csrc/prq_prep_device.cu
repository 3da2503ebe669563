// Offline weight preparation (Algorithm 1 steps 3-7 and 11) with the heavy steps on the GPU.
//
// The result is bit-for-bit the one of the host path (prq_prep.cu): same scale rule, same rounding, same
// FP64 summation order.  What runs where:
//   host    s_j = max(amax_j, 1e-5)^alpha and 1 / s_j                        (K values, FP64)
//   kernel  err_j = sum_n (W0[n,j] - deq(Q(W0))[n,j])^2, W0 = fl32(W * s)    one warp per 32-channel block of
//           the ORIGINAL order, lane = channel, rows n ascending: the block maximum is a warp reduction and
//           every lane keeps its own FP64 sum in row order (each term is exact in FP64)
//   host    error-ranked top-k, permutation                                  (a sort of K numbers)
//   kernel  Wt = W0[:, perm], Q(Wt), R = Wt_tail - deq(Q(Wt))_tail, Q(R), packing: one thread per
//           (row, 32-channel block of the PERMUTED order), optionally with the block-scale search
//           (floor-rule exponent and its two neighbours, FP64 squared error in element order)
// W is read from device memory twice (51 MB at the paper's down-projection shape); codes and scale bytes
// come back to the host, which keeps the canonical copies and lays the scale bytes out for the GEMMs.
#include <cuda_runtime.h>

#include <cstdint>

#include "prq_internal.h"

namespace prq {
namespace {

__device__ __forceinline__ float bf16_to_float(uint16_t h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }

// E8M0 byte from the bit pattern of the block's largest magnitude: biased exponent - 2, floored at 0
__device__ __forceinline__ uint32_t scale_byte(uint32_t amax_bits) {
    const int e = static_cast<int>((amax_bits >> 23) & 0xff) - 2;
    return e < 0 ? 0u : static_cast<uint32_t>(e);
}

// E2M1 code of v under scale byte `byte`: |v| * 2^(127 - byte), then the seven thresholds with ties to the
// even code; the sign bit is kept (also on zero)
__device__ __forceinline__ uint32_t e2m1_code(float v, uint32_t byte) {
    const uint32_t bits = __float_as_uint(v);
    const float inv = __uint_as_float((254u - byte) << 23);
    const float a = __fmul_rn(__uint_as_float(bits & 0x7fffffffu), inv);
    uint32_t m;
    if (a <= 0.25f) m = 0;
    else if (a < 0.75f) m = 1;
    else if (a <= 1.25f) m = 2;
    else if (a < 1.75f) m = 3;
    else if (a <= 2.5f) m = 4;
    else if (a < 3.5f) m = 5;
    else if (a <= 5.0f) m = 6;
    else m = 7;
    return m | ((bits >> 28) & 8u);
}

// value[code & 7] * 2^(byte - 127): at most two significant bits times a power of two, exact in fp32
// (subnormal results included; the product overflows to infinity exactly where the FP64 route would)
__device__ __forceinline__ float e2m1_value(uint32_t code, uint32_t byte) {
    const uint32_t m = code & 7u;
    const float t = m == 0 ? 0.f : m == 1 ? 0.5f : m == 2 ? 1.f : m == 3 ? 1.5f : m == 4 ? 2.f : m == 5 ? 3.f : m == 6 ? 4.f : 6.f;
    const float p = __uint_as_float(byte == 0 ? 0x00400000u : byte << 23);   // 2^(byte - 127)
    const float x = __fmul_rn(t, p);
    return (code & 8u) ? -x : x;
}

// ---------------------------------------------------------------------------------------------- column errors
constexpr int kRowsInFlight = 16;   // rows whose loads are issued before the first of them is consumed

__global__ void __launch_bounds__(32) col_err_kernel(const uint16_t* __restrict__ W, const float* __restrict__ s, int N, int K,
                                                      double* __restrict__ err, int* __restrict__ nonfinite) {
    // one warp per CTA: a layer has only K / 32 of these warps (80 - 304 at the paper's shapes), each bound
    // by the latency of its own loads, so they are spread over as many SMs as there are
    const int lane = threadIdx.x;
    const int j = static_cast<int>(blockIdx.x) * kBlock + lane;
    const float sj = s[j];
    const uint16_t* p = W + j;
    double acc = 0.0;
    bool ok = true;
    for (int n0 = 0; n0 < N; n0 += kRowsInFlight) {
        // the warp reduction below orders memory operations, so the loads of a batch of rows are issued
        // explicitly before any of them is used (one DRAM latency per batch instead of one per row)
        uint16_t h[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) h[u] = n0 + u < N ? __ldg(p + static_cast<size_t>(n0 + u) * K) : uint16_t(0);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            if (n0 + u < N) {
                const float v = __fmul_rn(bf16_to_float(h[u]), sj);
                const uint32_t mag = __float_as_uint(v) & 0x7fffffffu;
                ok = ok && mag < 0x7f800000u;
                const uint32_t byte = scale_byte(__reduce_max_sync(0xffffffffu, mag));
                const double d = static_cast<double>(v) - static_cast<double>(e2m1_value(e2m1_code(v, byte), byte));
                acc = __dadd_rn(acc, __dmul_rn(d, d));
            }
        }
    }
    err[j] = acc;
    if (!ok) atomicExch(nonfinite, 1);
}

// ---------------------------------------------------------------------------------------------- quantise + pack
struct Block {
    uint32_t c[4];   // 32 codes, element i in nibble i % 8 of word i / 8 (the packed order: even column low)
};

__device__ __forceinline__ uint32_t quantize_block(const float (&v)[kBlock], Block& out) {
    uint32_t amax = 0;
#pragma unroll
    for (int i = 0; i < kBlock; ++i) amax = max(amax, __float_as_uint(v[i]) & 0x7fffffffu);
    const uint32_t byte = scale_byte(amax);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) word |= e2m1_code(v[w * 8 + i], byte) << (4 * i);
        out.c[w] = word;
    }
    return byte;
}

// squared error of the block under `byte`, FP64, element order; also returns the codes
__device__ __forceinline__ double block_error(const float (&v)[kBlock], uint32_t byte, Block& out) {
    double err = 0.0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t code = e2m1_code(v[w * 8 + i], byte);
            word |= code << (4 * i);
            const double d = static_cast<double>(v[w * 8 + i]) - static_cast<double>(e2m1_value(code, byte));
            err = __dadd_rn(err, __dmul_rn(d, d));
        }
        out.c[w] = word;
    }
    return err;
}

// floor-rule byte and its two neighbours; a neighbour wins only if strictly better, byte - 1 is looked at
// before byte + 1; an all-zero block keeps the floor rule
__device__ __forceinline__ uint32_t quantize_block_search(const float (&v)[kBlock], Block& out) {
    const uint32_t byte0 = quantize_block(v, out);
    bool zero = true;
#pragma unroll
    for (int i = 0; i < kBlock; ++i) zero = zero && v[i] == 0.f;
    if (zero) return byte0;
    Block tmp;
    double best_err = block_error(v, byte0, tmp);
    uint32_t best = byte0;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const int cand = static_cast<int>(byte0) + (c == 0 ? -1 : 1);
        if (cand < 0 || cand > 254) continue;
        const double err = block_error(v, static_cast<uint32_t>(cand), tmp);
        if (err < best_err) { best_err = err; best = static_cast<uint32_t>(cand); out = tmp; }
    }
    return best;
}

__global__ void __launch_bounds__(128) quant_perm_kernel(const uint16_t* __restrict__ W, const float* __restrict__ s,
                                                         const int32_t* __restrict__ perm, int N, int K, int k_tail, int search,
                                                         uint8_t* __restrict__ codes, uint8_t* __restrict__ scales) {
    const int nblk = K / kBlock;
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<long long>(N) * nblk) return;
    const int n = static_cast<int>(idx / nblk), b = static_cast<int>(idx - static_cast<long long>(n) * nblk);
    const size_t Ka = static_cast<size_t>(K) + k_tail;
    const uint16_t* wrow = W + static_cast<size_t>(n) * K;
    float v[kBlock];
#pragma unroll
    for (int i = 0; i < kBlock; ++i) {
        const int j = __ldg(perm + b * kBlock + i);
        v[i] = __fmul_rn(bf16_to_float(__ldg(wrow + j)), __ldg(s + j));
    }
    Block q;
    const uint32_t byte = search ? quantize_block_search(v, q) : quantize_block(v, q);
    uint8_t* crow = codes + static_cast<size_t>(n) * (Ka / 2);
    uint8_t* srow = scales + static_cast<size_t>(n) * (Ka / kBlock);
    srow[b] = static_cast<uint8_t>(byte);
    *reinterpret_cast<uint4*>(crow + b * 16) = make_uint4(q.c[0], q.c[1], q.c[2], q.c[3]);
    const int tail_blk0 = (K - k_tail) / kBlock;
    if (b >= tail_blk0) {
        // Eq. (2): residual of the tail block against its own quantisation (exact in fp32), quantised again
        float r[kBlock];
#pragma unroll
        for (int i = 0; i < kBlock; ++i)
            r[i] = __fsub_rn(v[i], e2m1_value((q.c[i >> 3] >> (4 * (i & 7))) & 0xfu, byte));
        Block qr;
        const uint32_t rbyte = search ? quantize_block_search(r, qr) : quantize_block(r, qr);
        const int rb = nblk + (b - tail_blk0);
        srow[rb] = static_cast<uint8_t>(rbyte);
        *reinterpret_cast<uint4*>(crow + rb * 16) = make_uint4(qr.c[0], qr.c[1], qr.c[2], qr.c[3]);
    }
}

struct DevBuf {
    void* p = nullptr;
    ~DevBuf() { if (p) cudaFree(p); }
    cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 1); }
    template <class T> T* as() { return static_cast<T*>(p); }
};

}  // namespace

prq_status prepare_layer_device(const uint16_t* W_dev, int N, int K, const float* amax, float alpha, int k_tail,
                                PrepResult& out, bool scale_search, cudaStream_t stream) {
    const size_t Ka = static_cast<size_t>(K) + k_tail;
    prq_status st = channel_scales(amax, K, alpha, out.s, out.inv_s);
    if (st != PRQ_OK) return st;
    out.col_err.assign(K, 0.0);
    out.codes.assign(static_cast<size_t>(N) * Ka / 2, 0);
    out.scales.assign(static_cast<size_t>(N) * Ka / kBlock, 0);

    DevBuf d_s, d_err, d_flag, d_perm, d_codes, d_scales;
    if (d_s.alloc(sizeof(float) * K) != cudaSuccess || d_err.alloc(sizeof(double) * K) != cudaSuccess ||
        d_flag.alloc(sizeof(int)) != cudaSuccess || d_perm.alloc(sizeof(int32_t) * K) != cudaSuccess ||
        d_codes.alloc(out.codes.size()) != cudaSuccess || d_scales.alloc(out.scales.size()) != cudaSuccess) {
        cudaGetLastError();
        return PRQ_ERR_OOM;
    }
    bool ok = cudaMemcpyAsync(d_s.p, out.s.data(), sizeof(float) * K, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemsetAsync(d_flag.p, 0, sizeof(int), stream) == cudaSuccess;
    if (!ok) return PRQ_ERR_CUDA;

    const int nblk = K / kBlock;
    col_err_kernel<<<nblk, 32, 0, stream>>>(W_dev, d_s.as<float>(), N, K, d_err.as<double>(), d_flag.as<int>());
    int nonfinite = 0;
    ok = cudaGetLastError() == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out.col_err.data(), d_err.p, sizeof(double) * K, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(&nonfinite, d_flag.p, sizeof(int), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) return PRQ_ERR_CUDA;
    if (nonfinite) return PRQ_ERR_NONFINITE;

    rank_and_permute(out.col_err, K, k_tail, out.perm);

    ok = cudaMemcpyAsync(d_perm.p, out.perm.data(), sizeof(int32_t) * K, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return PRQ_ERR_CUDA;
    const long long threads = static_cast<long long>(N) * nblk;
    quant_perm_kernel<<<static_cast<unsigned>((threads + 127) / 128), 128, 0, stream>>>(
        W_dev, d_s.as<float>(), d_perm.as<int32_t>(), N, K, k_tail, scale_search ? 1 : 0, d_codes.as<uint8_t>(), d_scales.as<uint8_t>());
    ok = cudaGetLastError() == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out.codes.data(), d_codes.p, out.codes.size(), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out.scales.data(), d_scales.p, out.scales.size(), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    return ok ? PRQ_OK : PRQ_ERR_CUDA;
}

}  // namespace prq
