// Prefill GEMM (M > 128): the block-scaled FP4 product of Eq. (3) with 128 x 224 output tiles and a
// stream-K schedule.
//
// Why stream-K.  The paper's down-projection at 2048 tokens is 16 x 12 = 192 tiles on 148 SMs:
// tile-per-CTA scheduling needs two waves and leaves the machine a third empty in the second.  Here the
// (tile, reduction-stage) space is cut into equal contiguous ranges, one per CTA (one CTA per SM).  A
// range covers the tail of one tile, whole tiles, and the head of another.  The CTA that holds a tile's
// first stage owns the tile; any other CTA working on it writes its fp32 partial accumulator to its
// workspace slot and raises the tile's flag.  Every CTA processes its leading (contributed) segment
// first and its trailing (owned) segment last, so an owner finds the contributions long finished and
// no CTA ever waits on work that is queued behind its own.
//
// Why 224 columns.  The instruction stream of the one issuing warp bounds the main loop, so the tile
// should be as wide as possible; two accumulators (so that the epilogue of one segment overlaps the
// main loop of the next) plus the scale columns must fit the 512 tensor-memory columns: 2 x 224 + 24.
// (A variant with a separate scale-copy warp and two scale sets was slower: the copy -> MMA -> release
// chain of a two-deep scale ring is longer than two stages.)
//
// Roles (6 warps):
//   warp 0    TMA producer: per 256-element reduction stage one tile load per operand and one flat bulk
//             copy per operand for the stage's scale bytes, all counted on the slot's "full" mbarrier;
//   warp 1    tcgen05 issuer: copies the stage's six 512-byte scale atoms shared -> tensor memory, issues
//             up to four K = 64 tcgen05.mma.kind::mxf4.block_scale steps, commits to the slot's "empty"
//             mbarrier.  The loop is specialised per ring slot so that every descriptor is a
//             loop-invariant register plus a constant;
//   warps 2-5 epilogue: tcgen05.ld of their 32-lane quarter, 32 columns at a time, into swizzled shared
//             staging, then one TMA store per warp and chunk (rows and columns outside M x N are clipped
//             by the tensor map).
//
// The activation tail is re-read, not copied: stages past the K main columns load the activation tile
// from column K - k and the weight tile from column K onwards (Kernel design paragraph).
// Every wait is bounded; on expiry the CTA raises an abort flag, all roles unwind, tensor memory is
// freed and PRQ_ERR_TIMEOUT is recorded in the device status word.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "prq_kernels.h"
#include "prq_ptx.cuh"

namespace prq {
namespace {

constexpr int kThreads = 192;
constexpr int BN = kPrefillTileN;
constexpr int kPTile = 128 * 128;                 // activation tile bytes (128 rows x 256 codes)
constexpr int kQTile = BN * 128;                  // weight tile bytes
constexpr int kSfp = kSfGroupBytes;               // 1 group of 128 rows
constexpr int kSfq = 2 * kSfGroupBytes;           // 2 groups (128 + 96 rows)
constexpr int kStageBytes = kPTile + kQTile + kSfp + kSfq;  // 48128
constexpr int kStages = 4;
constexpr int kStagingPerWarp = 2 * 4096;         // two 32-row x 128-byte chunks per epilogue warp
constexpr int kSmemBytes = kStages * kStageBytes + 4 * kStagingPerWarp + 1024;
constexpr int kTmemCols = 512;
constexpr int kSfCol = 2 * BN;                    // scale columns start behind the two accumulators
constexpr int kSfSetCols = 24;                    // 8 activation + 16 weight scale columns
constexpr int kChunkCols = 32;                    // accumulator columns per epilogue chunk
constexpr int kChunks = BN / kChunkCols;          // 7
static_assert(kStageBytes % 1024 == 0, "stage slots must keep 1024-byte alignment");
static_assert(kSmemBytes <= 232448 - 256, "shared memory budget");
static_assert(kSfCol + kSfSetCols <= kTmemCols, "tensor memory budget");

__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t src_smem, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(src_smem), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

struct Segment {
    int tile, s0, s1;   // reduction stages [s0, s1) of `tile`
};

// The contiguous range of (tile, stage) units of one CTA, walked segment by segment.
// All of this is 32-bit arithmetic (the host checks that W * G fits): 64-bit divisions cost hundreds of
// cycles each and sit on the critical path of every role's first instruction.
struct Range {
    uint32_t cur, end;
    int S;
    __device__ __forceinline__ bool next(Segment& g) {
        if (cur >= end) return false;
        g.tile = static_cast<int>(cur / static_cast<uint32_t>(S));
        g.s0 = static_cast<int>(cur - static_cast<uint32_t>(g.tile) * S);
        const uint32_t left = end - cur;
        g.s1 = left < static_cast<uint32_t>(S - g.s0) ? g.s0 + static_cast<int>(left) : S;
        cur += g.s1 - g.s0;
        return true;
    }
};

__device__ __forceinline__ uint32_t range_begin(uint32_t W, int g, int G) {
    return W * static_cast<uint32_t>(g) / static_cast<uint32_t>(G);
}

constexpr uint32_t kHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version 1, 128B swizzle
constexpr uint32_t kHiPlain = (128u >> 4) | (1u << 14);                // SBO 128, version 1, no swizzle
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; }

// One reduction stage of the issue loop with the ring slot Q known at compile time: every
// shared-memory descriptor is `lo_base` plus a constant.  Scale atoms first -- activation group
// (columns +0 / +4 for the two halves of the stage), weight groups 0 and 1 (columns +8, +12 / +16, +20)
// -- then up to four K = 64 MMAs, then the commit that frees the slot.  The copies and the MMAs are
// issued by one thread, so tensor memory sees them in order and one set of scale columns is enough.
// `rem` = reduction elements this stage still covers.
template <int Q>
__device__ __forceinline__ void issue_stage(uint32_t lo_base, uint32_t d_tmem, uint32_t sf_t, int rem,
                                            uint32_t accumulate, uint32_t empty_bar0) {
    constexpr uint32_t so = (Q * kStageBytes) >> 4;  // stage offset in 16-byte units
    constexpr uint32_t sfo = so + ((kPTile + kQTile) >> 4);
    constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
    constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
    const uint32_t plo = lo_base + so, qlo = lo_base + so + (kPTile >> 4), slo = lo_base + sfo;
    const uint32_t sfp_t = sf_t, sfq_t = sf_t + 8;
    tc_copy_sf_atom(sf_t, desc64(kHiPlain, slo));
    tc_copy_sf_atom(sf_t + 8, desc64(kHiPlain, slo + (kSfp >> 4)));
    tc_copy_sf_atom(sf_t + 12, desc64(kHiPlain, slo + ((kSfp + kSfGroupBytes) >> 4)));
    if (rem > 128) {
        tc_copy_sf_atom(sf_t + 4, desc64(kHiPlain, slo + (512 >> 4)));
        tc_copy_sf_atom(sf_t + 16, desc64(kHiPlain, slo + ((kSfp + 512) >> 4)));
        tc_copy_sf_atom(sf_t + 20, desc64(kHiPlain, slo + ((kSfp + kSfGroupBytes + 512) >> 4)));
    }
    tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo), desc64(kHiSw128, qlo), idesc0, sfp_t, sfq_t, accumulate);
    if (rem > 64) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 2), desc64(kHiSw128, qlo + 2), idesc2, sfp_t, sfq_t, 1);
    if (rem > 128) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 4), desc64(kHiSw128, qlo + 4), idesc0, sfp_t + 4, sfq_t + 8, 1);
    if (rem > 192) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 6), desc64(kHiSw128, qlo + 6), idesc2, sfp_t + 4, sfq_t + 8, 1);
    tc_commit(empty_bar0 + Q * 8);
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
               const __grid_constant__ CUtensorMap tm_y, const PrefillParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t staging_base = smem_base + kStages * kStageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const StagePlan plan(p.K, p.k_tail);
    const int S = plan.S, S1 = plan.S1;
    const int G = gridDim.x, g = blockIdx.x;
    const uint32_t W = static_cast<uint32_t>(p.m_tiles) * p.n_tiles * S;

    if (p.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[2048 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bar_acc_full[i]), 1);
            mbar_init(smem_u32(&bar_acc_empty[i]), 4);
        }
        abort_flag_s = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_act);
        tma_prefetch_desc(&tm_w);
        tma_prefetch_desc(&tm_y);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // set-up done: let the next kernel of the stream be scheduled (its launch latency then overlaps this
    // kernel), and wait until everything earlier kernels wrote (activation codes, workspace flags) or
    // still read (y) is settled
    grid_launch_dependents();
    grid_dependency_wait();
    const uint32_t tmem_base = tmem_slot;
    const int trace_cta0 = p.dbg >> 16;  // developer aid: first of the four traced CTAs
    long long* trace = (p.trace && static_cast<int>(blockIdx.x) >= trace_cta0 && static_cast<int>(blockIdx.x) < trace_cta0 + 4)
                           ? p.trace + (blockIdx.x - trace_cta0) * 512 : nullptr;
    if (trace && threadIdx.x == 0) trace[500] = clock64();
    const uint32_t lo_base = ((smem_base & 0x3FFFF) >> 4) | (1u << 16);

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
        Segment sg;
        int st = 0, it = 0;
        uint32_t ph = 0;
        bool ok = true;
        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            const uint8_t* sfp = p.act_sf + static_cast<size_t>(mi) * kSfGroupBytes;
            const uint8_t* sfq = p.w_sf + static_cast<size_t>(ni) * 2 * kSfGroupBytes;
            const size_t sfp_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;
            const size_t sfq_stride = static_cast<size_t>(p.w_groups) * kSfGroupBytes;
            for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                if (!mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1, abort_flag)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[it] = clock64();
                if (elect_one()) {
                    const uint32_t full = smem_u32(&bar_full[st]);
                    mbar_arrive_expect_tx(full, kStageBytes);
                    const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                    const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                    const uint32_t sb = smem_base + st * kStageBytes;
                    tma_load_2d(sb, &tm_act, xa, mi * 128, full);
                    tma_load_2d(sb + kPTile, &tm_w, xw, ni * BN, full);
                    bulk_load(sb + kPTile + kQTile, sfp + s * sfp_stride, kSfp, full);
                    bulk_load(sb + kPTile + kQTile + kSfp, sfq + s * sfq_stride, kSfq, full);
                }
                if (++st == kStages) { st = 0; ph ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            // let copies in flight land before shared memory is given up (bounded)
            for (int j = max(0, it - kStages); j < it; ++j) {
                const uint32_t bar = smem_u32(&bar_full[j % kStages]);
                const uint32_t php = (j / kStages) & 1;
                for (int tries = 0; tries < (1 << 16) && !mbar_try_wait(bar, php); ++tries) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
        Segment sg;
        const bool leader = elect_one();
        int it = 0, st = 0, seg_it = 0;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t sf_t = tmem_base + kSfCol;
        while (ok && r.next(sg)) {
            const int buf = seg_it & 1;
            if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), ((seg_it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + buf * BN;
            uint32_t accumulate = 0;
            for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                if (!mbar_wait(smem_u32(&bar_full[st]), ph, abort_flag)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[64 + it] = clock64();
                const int rem = s < S1 ? p.K - s * kStageK : p.k_tail - (s - S1) * kStageK;
                if (leader) {
                    const uint32_t eb = smem_u32(&bar_empty[0]);
                    switch (st) {
                        case 0: issue_stage<0>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                        case 1: issue_stage<1>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                        case 2: issue_stage<2>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                        default: issue_stage<3>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                    }
                }
                accumulate = 1;
                if (trace && lane == 0 && it < 64) trace[128 + it] = clock64();
                if (++st == kStages) { st = 0; ph ^= 1; }
            }
            if (!ok) break;
            if (leader) tc_commit(smem_u32(&bar_acc_full[buf]));
            ++seg_it;
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q4 = warp & 3;                 // tensor-memory lane quarter of this warp
        const int row_in_tile = q4 * 32 + lane;
        const uint32_t stage_smem = staging_base + (warp - 2) * kStagingPerWarp;
        Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
        Segment sg;
        int seg_it = 0, store_it = 0;
        bool ok = true;
        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            const int buf = seg_it & 1;
            const bool contributor = sg.s0 > 0;
            int n_contrib = 0;
            if (!contributor && sg.s1 < S) {
                // owner of a tile that other CTAs finish: they are the next CTAs in order
                const uint32_t last_unit = static_cast<uint32_t>(sg.tile + 1) * S - 1;
                int gl = g + 1;
                while (gl + 1 < G && range_begin(W, gl + 1, G) <= last_unit) ++gl;
                n_contrib = gl - g;
            }
            if (!mbar_wait(smem_u32(&bar_acc_full[buf]), (seg_it >> 1) & 1, abort_flag)) { ok = false; break; }
            if (trace && row_in_tile == 0 && seg_it < 8) trace[192 + 2 * seg_it] = clock64();
            tc_fence_after_sync();
            const uint32_t acc_t = tmem_base + buf * BN + (static_cast<uint32_t>(q4 * 32) << 16);
            if (contributor) {
                // partial accumulator -> this CTA's slot, stored column-major so that warps write full lines
                float* slot = p.partial + static_cast<size_t>(g) * (128 * BN) + row_in_tile;
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(acc_t + c * kChunkCols, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) __stcg(slot + (c * kChunkCols + i) * 128, __uint_as_float(v[i]));
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
                // publish: all four warps' stores, then one count on the tile's flag
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (row_in_tile == 0) atomicAdd(p.flags + sg.tile, 1);
            } else {
                if (n_contrib > 0) {
                    // wait (bounded) until every contribution to this tile has been published
                    if (lane == 0) {
                        volatile int* f = p.flags + sg.tile;
                        const long long t0 = clock64();
                        while (*f < n_contrib) {
                            if (*abort_flag) break;
                            if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; break; }
                        }
                    }
                    __syncwarp();
                    if (*abort_flag) { ok = false; break; }
                    __threadfence();
                    if (trace && row_in_tile == 0 && seg_it < 8) trace[208 + seg_it] = clock64();
                }
                const float* slot = p.partial + static_cast<size_t>(g + 1) * (128 * BN) + row_in_tile;
                const int y_row = mi * 128 + q4 * 32;
                // Contributions are fetched one chunk ahead (32 independent, coalesced loads in flight while
                // the current chunk is staged and stored); further contributors of the same tile are rare
                // (only when a tile is shared by more than two CTAs) and are read in place.
                float nx[32];
                if (n_contrib > 0) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) nx[i] = __ldcg(slot + i * 128);
                }
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(acc_t + c * kChunkCols, v);
                    tmem_ld_wait();
                    if (n_contrib > 0) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + nx[i]);
                        if (c + 1 < kChunks) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) nx[i] = __ldcg(slot + ((c + 1) * kChunkCols + i) * 128);
                        }
                        for (int cidx = 1; cidx < n_contrib; ++cidx) {
                            float t2[32];
                            const float* src = slot + static_cast<size_t>(cidx) * (128 * BN) + c * kChunkCols * 128;
#pragma unroll
                            for (int i = 0; i < 32; ++i) t2[i] = __ldcg(src + i * 128);
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + t2[i]);
                        }
                    }
                    const uint32_t sbuf = stage_smem + (store_it & 1) * 4096;
                    // the store issued two chunks ago has finished reading this buffer
                    if (lane == 0) bulk_wait_read<1>();
                    __syncwarp();
                    if (!p.y_bf16) {
                        // 128-byte staging rows, 16-byte unit index ^= row % 8
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            st_shared_v4(sbuf + lane * 128 + ((u ^ (lane & 7)) << 4), v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
                    } else {
                        // 64-byte staging rows (32 bf16), unit index ^= (row / 2) % 4
                        uint32_t h[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                            h[i] = *reinterpret_cast<uint32_t*>(&t2);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            st_shared_v4(sbuf + lane * 64 + ((u ^ ((lane >> 1) & 3)) << 4), h[4 * u], h[4 * u + 1], h[4 * u + 2], h[4 * u + 3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tm_y, sbuf, ni * BN + c * kChunkCols, y_row);
                        bulk_commit();
                    }
                    ++store_it;
                    if (c == kChunks - 1) {
                        // the accumulator has been read completely: hand it back before the stores drain
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
                    }
                }
                if (n_contrib > 0) {
                    // everyone has read the contributions: clear the flag for the next launch
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (row_in_tile == 0) p.flags[sg.tile] = 0;
                }
            }
            if (trace && row_in_tile == 0 && seg_it < 8) trace[193 + 2 * seg_it] = clock64();
            ++seg_it;
        }
        // shared staging must not be released while a store is still reading it
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
    }

    // ------------------------------------------------------------ teardown (normal and aborted)
    tc_fence_before_sync();
    __syncthreads();
    if (trace && threadIdx.x == 0) trace[501] = clock64();
    if (p.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[2049 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

}  // namespace

cudaError_t launch_prefill(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const CUtensorMap& tm_y,
                           const PrefillParams& p, int grid, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_kernel, tm_act, tm_w, tm_y, p);
}

}  // namespace prq
