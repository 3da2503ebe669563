// Prefill GEMM (M > 128) on CTA pairs: the block-scaled FP4 product of Eq. (3) with 256 x 224 output
// tiles computed by two CTAs of a cluster as one tcgen05 cta_group::2 unit, under a stream-K schedule.
//
// Why pairs.  With one CTA per 128 x 224 tile every SM pulls (128 + 224) operand rows per reduction
// stage from L2, and at the paper's down-projection shape the 148 SMs together ask for more than the
// L2 delivers: the loads, not the tensor cores, bound the main loop.  A pair shares the weight tile:
// each CTA loads its own 128 activation rows and only 112 of the 224 weight rows, the tensor cores read
// the other half from the peer's shared memory, and the bytes per SM and stage drop by 30 %.
//
// Why stream-K.  2048 tokens x 2560 features are 8 x 12 = 96 pair tiles on 74 pairs; tile-per-pair
// scheduling would leave a third of the machine idle in its second wave.  The (tile, reduction-stage)
// space is cut into equal contiguous ranges, one per pair.  A range covers the tail of one tile, whole
// tiles, and the head of another.  The pair that holds a tile's first stage owns it; any other pair
// working on it writes its fp32 partial accumulators to workspace slots (one per CTA) and raises the
// flags of the tile's two halves.  Every pair processes its leading (contributed) segment first and its
// trailing (owned) segment last, so an owner finds the contributions long finished and no pair ever
// waits on work that is queued behind its own.
//
// Roles (6 warps per CTA):
//   warp 0    TMA producer (both CTAs): per 256-element reduction stage its own activation tile, its
//             half of the weight tile, the scale bytes of its activation rows and of all 224 weight rows;
//             all four copies of both CTAs are counted on the LEADER's "full" mbarrier;
//   warp 1    leader CTA: tcgen05 issuer -- six scale-atom copies shared -> tensor memory (each CTA
//             copies from its own shared memory), up to four K = 64 MMAs, one commit that arrives on
//             the "empty" barrier of both CTAs.  In the other CTA this warp only allocates and frees
//             tensor memory;
//   warps 2-5 epilogue (both CTAs): tcgen05.ld of their 32-lane quarter of the CTA's 128 accumulator
//             rows, 32 columns at a time, into swizzled shared staging, then one TMA store per warp and
//             chunk (rows and columns outside M x N are clipped by the tensor map).
//
// The activation tail is re-read, not copied: stages past the K main columns load the activation tile
// from column K - k and the weight tile from column K onwards (Kernel design paragraph).
// Every wait is bounded; on expiry the CTA raises its abort flag and the peer's, all roles unwind, both
// CTAs meet at the closing cluster barrier, tensor memory is freed and PRQ_ERR_TIMEOUT is recorded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "prq_kernels.h"
#include "prq_ptx.cuh"

namespace prq {
namespace {

constexpr int kThreads = 192;
constexpr int BN = kPrefillTileN;                 // 224 weight rows per tile
constexpr int kHalfN = BN / 2;                    // weight rows each CTA of the pair loads
constexpr int kPTile = 128 * 128;                 // activation tile bytes (128 rows x 256 codes)
constexpr int kQTile = kHalfN * 128;              // half weight tile bytes
constexpr int kSfp = kSfGroupBytes;               // 1 group of 128 activation rows
constexpr int kSfq = 2 * kSfGroupBytes;           // 2 groups (128 + 96 weight rows)
constexpr int kStageBytes = kPTile + kQTile + kSfp + kSfq;  // 33792
constexpr int kStages = 5;
constexpr int kStagingPerWarp = 2 * 4096;         // two 32-row x 128-byte chunks per epilogue warp
constexpr int kSmemBytes = kStages * kStageBytes + 4 * kStagingPerWarp + 1024;
constexpr int kTmemCols = 512;
constexpr int kSfCol = 2 * BN;                    // scale columns start behind the two accumulators
constexpr int kSfSetCols = 24;                    // 8 activation + 16 weight scale columns
constexpr int kChunkCols = 32;                    // accumulator columns per epilogue chunk
constexpr int kChunks = BN / kChunkCols;          // 7
static_assert(kQTile % 1024 == 0 && kStageBytes % 1024 == 0, "operand tiles must keep 1024-byte alignment");
static_assert(kSmemBytes <= 232448 - 256, "shared memory budget");
static_assert(kSfCol + kSfSetCols <= kTmemCols, "tensor memory budget");

__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t src_smem, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(src_smem), "r"(x), "r"(y)
                 : "memory");
}
// y[tile] += staging tile, performed by the memory system (one fp32 add per element, so the sum of two
// contributions does not depend on their order).
__device__ __forceinline__ void tma_reduce_add_2d(const void* tmap, uint32_t src_smem, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(src_smem), "r"(x), "r"(y)
                 : "memory");
}
// All bulk stores of this thread are complete (written, not only read from shared memory).
__device__ __forceinline__ void bulk_wait_all_done() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

struct Segment {
    int tile, s0, s1;   // reduction stages [s0, s1) of `tile`
};

// The contiguous range of (tile, stage) units of one pair, walked segment by segment.
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
// -- then up to four K = 64 MMAs, then the commit that frees the slot in both CTAs.  The copies and
// the MMAs are issued by one thread, so tensor memory sees them in order and one set of scale columns
// is enough.  `rem` = reduction elements this stage still covers.
template <int Q>
__device__ __forceinline__ void issue_stage(uint32_t lo_base, uint32_t d_tmem, uint32_t sf_t, int rem,
                                            uint32_t accumulate, uint32_t empty_bar0) {
    constexpr uint32_t so = (Q * kStageBytes) >> 4;  // stage offset in 16-byte units
    constexpr uint32_t sfo = so + ((kPTile + kQTile) >> 4);
    // E2M1 x E2M1, E8M0 scales, both operands K-major, N = 224, M = 256 (two CTAs)
    constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | (1u << 23) | ((256u >> 4) << 24);
    constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
    const uint32_t plo = lo_base + so, qlo = lo_base + so + (kPTile >> 4), slo = lo_base + sfo;
    const uint32_t sfp_t = sf_t, sfq_t = sf_t + 8;
    tc_copy_sf_atom_pair(sf_t, desc64(kHiPlain, slo));
    tc_copy_sf_atom_pair(sf_t + 8, desc64(kHiPlain, slo + (kSfp >> 4)));
    tc_copy_sf_atom_pair(sf_t + 12, desc64(kHiPlain, slo + ((kSfp + kSfGroupBytes) >> 4)));
    if (rem > 128) {
        tc_copy_sf_atom_pair(sf_t + 4, desc64(kHiPlain, slo + (512 >> 4)));
        tc_copy_sf_atom_pair(sf_t + 16, desc64(kHiPlain, slo + ((kSfp + 512) >> 4)));
        tc_copy_sf_atom_pair(sf_t + 20, desc64(kHiPlain, slo + ((kSfp + kSfGroupBytes + 512) >> 4)));
    }
    tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo), desc64(kHiSw128, qlo), idesc0, sfp_t, sfq_t, accumulate);
    if (rem > 64) tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 2), desc64(kHiSw128, qlo + 2), idesc2, sfp_t, sfq_t, 1);
    if (rem > 128) tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 4), desc64(kHiSw128, qlo + 4), idesc0, sfp_t + 4, sfq_t + 8, 1);
    if (rem > 192) tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 6), desc64(kHiSw128, qlo + 6), idesc2, sfp_t + 4, sfq_t + 8, 1);
    tc_commit_pair(empty_bar0 + Q * 8, 3);
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfw,
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
    const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
    const StagePlan plan(p.K, p.k_tail);
    const int S = plan.S, S1 = plan.S1;
    const int G = gridDim.x >> 1, g = blockIdx.x >> 1;   // pairs
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
            mbar_init(smem_u32(&bar_acc_empty[i]), 8);   // four epilogue warps of each CTA
        }
        abort_flag_s = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_act);
        tma_prefetch_desc(&tm_w);
        tma_prefetch_desc(&tm_sfa);
        tma_prefetch_desc(&tm_sfw);
        tma_prefetch_desc(&tm_y);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish_pair();
    }
    // both CTAs' barriers and tensor memory must exist before either CTA signals the other
    tc_fence_before_sync();
    cluster_arrive();
    cluster_wait();
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
        // ------------------------------------------------------------ producer (both CTAs)
        Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
        Segment sg;
        int st = 0, it = 0;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t leader_full0 = cluster_map(smem_u32(&bar_full[0]), 0);
        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            // scale bytes: rows of 256 bytes, 4 per 128-row group
            const int sfa_row0 = (mi * 2 + static_cast<int>(rank)) * 4, sfa_stride = p.act_groups * 4;
            const int sfw_row0 = ni * 8, sfw_stride = p.w_groups * 4;
            for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                if (!mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1, abort_flag)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[it] = clock64();
                if (elect_one()) {
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&bar_full[st]), 2 * kStageBytes);
                    const uint32_t full = leader_full0 + st * 8;
                    const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                    const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                    const uint32_t sb = smem_base + st * kStageBytes;
                    tma_load_2d_pair(sb, &tm_act, xa, mi * 256 + static_cast<int>(rank) * 128, full);
                    tma_load_2d_pair(sb + kPTile, &tm_w, xw, ni * BN + static_cast<int>(rank) * kHalfN, full);
                    tma_load_2d_pair(sb + kPTile + kQTile, &tm_sfa, 0, sfa_row0 + s * sfa_stride, full);
                    tma_load_2d_pair(sb + kPTile + kQTile + kSfp, &tm_sfw, 0, sfw_row0 + s * sfw_stride, full);
                }
                if (++st == kStages) { st = 0; ph ^= 1; }
            }
        }
        // gave up: copies in flight still target this CTA's shared memory; their completion is counted on
        // the leader's barrier, which this CTA cannot poll, so give them time to land (they take a few
        // microseconds at most) before the CTA moves on to the teardown
        if (!ok) __nanosleep(50000);
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {
            Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
            Segment sg;
            const bool leader = elect_one();
            int it = 0, st = 0, seg_it = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t sf_t = tmem_base + kSfCol;
            // `ready`: the slot about to be consumed was already seen full by the probe issued one stage
            // earlier (before that stage's tcgen05 instructions, so that the probe's latency hides behind them)
            bool ready = false;
            while (ok && r.next(sg)) {
                const int buf = seg_it & 1;
                if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), ((seg_it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                uint32_t accumulate = 0;
                for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                    if (!ready && !mbar_wait(smem_u32(&bar_full[st]), ph, abort_flag)) { ok = false; break; }
                    if (trace && lane == 0 && it < 64) trace[64 + it] = clock64();
                    const int rem = s < S1 ? p.K - s * kStageK : p.k_tail - (s - S1) * kStageK;
                    const int nst = st + 1 == kStages ? 0 : st + 1;
                    const uint32_t nph = nst == 0 ? ph ^ 1 : ph;
                    ready = mbar_test_wait(smem_u32(&bar_full[nst]), nph);
                    if (leader) {
                        const uint32_t eb = smem_u32(&bar_empty[0]);
                        switch (st) {
                            case 0: issue_stage<0>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 1: issue_stage<1>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 2: issue_stage<2>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 3: issue_stage<3>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            default: issue_stage<4>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                        }
                    }
                    accumulate = 1;
                    if (trace && lane == 0 && it < 64) trace[128 + it] = clock64();
                    st = nst; ph = nph;
                }
                if (!ok) break;
                if (leader) tc_commit_pair(smem_u32(&bar_acc_full[buf]), 3);
                ++seg_it;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int q4 = warp & 3;                 // tensor-memory lane quarter of this warp
        const int row_in_tile = q4 * 32 + lane;  // row of this CTA's 128-row half
        const uint32_t stage_smem = staging_base + (warp - 2) * kStagingPerWarp;
        const uint32_t leader_acc_empty0 = cluster_map(smem_u32(&bar_acc_empty[0]), 0);
        Range r{range_begin(W, g, G), range_begin(W, g + 1, G), S};
        Segment sg;
        int seg_it = 0, store_it = 0;
        bool ok = true;
        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            const int buf = seg_it & 1;
            const bool contributor = sg.s0 > 0;
            int* flag = p.flags + 2 * sg.tile + rank;   // one flag per 128-row half of the tile
            int n_contrib = 0;
            if (!contributor && sg.s1 < S) {
                // owner of a tile that other pairs finish: they are the next pairs in order
                const uint32_t last_unit = static_cast<uint32_t>(sg.tile + 1) * S - 1;
                int gl = g + 1;
                while (gl + 1 < G && range_begin(W, gl + 1, G) <= last_unit) ++gl;
                n_contrib = gl - g;
            }
            // Direct fix-up (fp32 output, tile shared by exactly two pairs): the contributor stores its partial
            // tile straight into y and the owner adds its own on top with a TMA reduction; no workspace
            // round trip, and x + y is the same in either order.  Otherwise (bf16, or three and more pairs,
            // whose order of addition must stay fixed) the partials go through the workspace.
            const bool direct = !p.y_bf16 &&
                (contributor ? (sg.s1 == S && range_begin(W, g - 1, G) <= static_cast<uint32_t>(sg.tile) * S)
                             : n_contrib == 1);
            if (!mbar_wait(smem_u32(&bar_acc_full[buf]), (seg_it >> 1) & 1, abort_flag)) { ok = false; break; }
            if (trace && row_in_tile == 0 && seg_it < 8) trace[192 + 2 * seg_it] = clock64();
            tc_fence_after_sync();
            const uint32_t acc_t = tmem_base + buf * BN + (static_cast<uint32_t>(q4 * 32) << 16);
            if (contributor && !direct) {
                // partial accumulator -> this CTA's slot, stored column-major so that warps write full lines
                float* slot = p.partial + static_cast<size_t>(blockIdx.x) * (128 * BN) + row_in_tile;
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
                if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + buf * 8);
                // publish: all four warps' stores, then one count on the flag of this half
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (row_in_tile == 0) atomicAdd(flag, 1);
            } else {
                const bool add_ws = n_contrib > 0 && !direct;     // owner: add the partials parked in the workspace
                const bool reduce = n_contrib > 0 && direct;      // owner: add onto the contributor's values in y
                if (n_contrib > 0) {
                    // wait (bounded) until every contribution to this half has been published
                    if (lane == 0) {
                        volatile int* f = flag;
                        const long long t0 = clock64();
                        while (*f < n_contrib) {
                            if (*abort_flag) break;
                            if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; break; }
                        }
                    }
                    __syncwarp();
                    if (*abort_flag) { ok = false; break; }
                    __threadfence();
                    fence_proxy_async_all();
                    if (trace && row_in_tile == 0 && seg_it < 8) trace[208 + seg_it] = clock64();
                }
                // the contributors are the CTAs of the same rank in the following pairs
                const float* slot = p.partial + static_cast<size_t>(blockIdx.x + 2) * (128 * BN) + row_in_tile;
                const int y_row = mi * 256 + static_cast<int>(rank) * 128 + q4 * 32;
                // Contributions are fetched one chunk ahead (32 independent, coalesced loads in flight while
                // the current chunk is staged and stored); further contributors of the same tile are rare
                // (only when a tile is shared by more than two pairs) and are read in place.
                float nx[32];
                if (add_ws) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) nx[i] = __ldcg(slot + i * 128);
                }
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(acc_t + c * kChunkCols, v);
                    tmem_ld_wait();
                    if (add_ws) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + nx[i]);
                        if (c + 1 < kChunks) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) nx[i] = __ldcg(slot + ((c + 1) * kChunkCols + i) * 128);
                        }
                        for (int cidx = 1; cidx < n_contrib; ++cidx) {
                            float t2[32];
                            const float* src = slot + static_cast<size_t>(2 * cidx) * (128 * BN) + c * kChunkCols * 128;
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
                        if (reduce) tma_reduce_add_2d(&tm_y, sbuf, ni * BN + c * kChunkCols, y_row);
                        else tma_store_2d(&tm_y, sbuf, ni * BN + c * kChunkCols, y_row);
                        bulk_commit();
                    }
                    ++store_it;
                    if (c == kChunks - 1) {
                        // the accumulator has been read completely: hand it back before the stores drain
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + buf * 8);
                    }
                }
                if (contributor) {
                    // direct contribution: publish once all four warps' stores have been written
                    if (lane == 0) bulk_wait_all_done();
                    fence_proxy_async_all();
                    __threadfence();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (row_in_tile == 0) atomicAdd(flag, 1);
                } else if (n_contrib > 0) {
                    // everyone has seen (and, through the workspace, read) the contributions: clear the flag
                    // for the next launch
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (row_in_tile == 0) *flag = 0;
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
    // a CTA that gave up tells its peer, whose waits would otherwise run to their own limit
    if (abort_flag_s && lane == 0) st_cluster_u32(cluster_map(smem_u32(&abort_flag_s), rank ^ 1), 1);
    tc_fence_before_sync();
    cluster_arrive();
    cluster_wait();
    if (trace && threadIdx.x == 0) trace[501] = clock64();
    if (p.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[2049 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

}  // namespace

int prefill_pair_max_clusters() {
    static int cached = -1;
    if (cached >= 0) return cached;
    if (cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, prefill_pair_kernel, &cfg) != cudaSuccess) return 0;
    cached = n;
    return n;
}

cudaError_t launch_prefill_pair(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const CUtensorMap& tm_sfa,
                                const CUtensorMap& tm_sfw, const CUtensorMap& tm_y, const PrefillParams& p,
                                int pairs, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, prefill_pair_kernel, tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p);
}

}  // namespace prq
