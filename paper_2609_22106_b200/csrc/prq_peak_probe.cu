// Benchmark utility (no counterpart in the paper): what the block-scaled FP4 tensor pipe of this GPU
// sustains when nothing else is in the way.  One CTA per SM issues back-to-back
// tcgen05.mma.kind::mxf4.block_scale instructions (M = 128, N = 256, K = 64) on operands that sit in
// shared memory for the whole run -- no loads, no epilogue -- and the caller times the launch.  The
// number is the denominator "measured mxf4 peak" that the benchmark reports next to 4 x measured bf16.
// The operands are a fixed pseudo-random byte pattern (not zeros, which would draw less power and
// clock higher than real data) with unit block scales.
#include <cuda_runtime.h>

#include "prq.h"
#include "prq_ptx.cuh"

namespace prq {
namespace {

constexpr int kProbeN = 256;
constexpr int kATile = 128 * 128;          // 128 rows x 256 codes
constexpr int kBTile = kProbeN * 128;
constexpr int kSfBytes = 3 * 1024;         // scale atoms: 1 activation group + 2 weight groups
constexpr int kSmem = kATile + kBTile + kSfBytes + 1024;

__global__ void __launch_bounds__(64, 1) mxf4_peak_kernel(int n_mma, int* status) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t done;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_s;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&done), 1); abort_s = 0; fence_mbar_init(); }
    // codes: a hash of the byte index; scale bytes: 127 (2^0)
    for (int i = threadIdx.x; i < (kATile + kBTile) / 4; i += blockDim.x) {
        uint32_t h = static_cast<uint32_t>(i) * 2654435761u + 0x9e3779b9u * (blockIdx.x + 1);
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        reinterpret_cast<uint32_t*>(smem)[i] = h;
    }
    for (int i = threadIdx.x; i < kSfBytes / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem + kATile + kBTile)[i] = 0x7f7f7f7fu;
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_slot), 512); tmem_relinquish(); }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 1) {
        const bool leader = elect_one();
        const uint32_t sf_t = tmem_base + kProbeN;
        if (leader) {
            const uint32_t sfs = smem_base + kATile + kBTile;
            for (int c = 0; c < 6; ++c) tc_copy_sf_atom(sf_t + 4 * c, make_smem_desc(sfs + 512 * c, 16, 128, kSwizzleNone));
            const uint64_t pd = make_smem_desc(smem_base, 16, 1024, kSwizzle128B);
            const uint64_t qd = make_smem_desc(smem_base + kATile, 16, 1024, kSwizzle128B);
            const uint32_t idesc0 = make_idesc_mxf4(kProbeN, 0, 0), idesc2 = make_idesc_mxf4(kProbeN, 2, 2);
            for (int it = 0; it < n_mma; it += 4) {
                tc_mma_mxf4(tmem_base, pd, qd, idesc0, sf_t, sf_t + 8, it);
                tc_mma_mxf4(tmem_base, pd + 2, qd + 2, idesc2, sf_t, sf_t + 8, 1);
                tc_mma_mxf4(tmem_base, pd + 4, qd + 4, idesc0, sf_t + 4, sf_t + 16, 1);
                tc_mma_mxf4(tmem_base, pd + 6, qd + 6, idesc2, sf_t + 4, sf_t + 16, 1);
            }
            tc_commit(smem_u32(&done));
        }
        __syncwarp();
        mbar_wait(smem_u32(&done), 0, &abort_s);   // bounded
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    if (threadIdx.x == 0 && abort_s) atomicExch(status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

// One link of a chain of dependent launches with nothing in it: every CTA lets the next kernel of the stream be
// scheduled, waits for the previous one to finish, writes one word (so that the dependency is a real one) and
// leaves.  `grid` CTAs of `threads` threads in clusters of `cluster` -- the launch shape of the decode GEMM.
__global__ void handover_probe_kernel(int* sink) {
    grid_launch_dependents();
    grid_dependency_wait();
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicAdd(sink, 1);
}

}  // namespace

cudaError_t launch_handover_probe(int n, int grid, int threads, int cluster, int* sink, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    for (int i = 0; i < n; ++i) {
        cudaError_t e = cudaLaunchKernelEx(&cfg, handover_probe_kernel, sink);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_mxf4_peak_probe(int n_mma, int grid, int* status, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(mxf4_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    mxf4_peak_kernel<<<grid, 64, kSmem, stream>>>(n_mma, status);
    return cudaGetLastError();
}

}  // namespace prq
