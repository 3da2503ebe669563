// Prefill GEMM (M > 128) on CTA pairs: the block-scaled FP4 product of Eq. (3) with output tiles of 256 rows computed
// by two CTAs of a cluster as one tcgen05 cta_group::2 unit.  Three tile widths (template instances): 224 and 240
// columns under a stream-K schedule, and 288 columns for calls whose tiles all fit ONE wave of pairs at that width (see
// PCfg).  A fourth instance, 192 columns with a gated epilogue, serves prq_linear_gated.  The text below speaks of the
// 224-column tile; the 240-column one differs in the constants only (120 weight rows per CTA, a 16-column chunk closing
// the epilogue).
//
// Why pairs.  With one CTA per 128 x 224 tile every SM pulls (128 + 224) operand rows per reduction
// stage from L2, and at the paper's down-projection shape the 148 SMs together ask for more than the
// L2 delivers: the loads, not the tensor cores, bound the main loop.  A pair shares the weight tile:
// each CTA loads its own 128 activation rows and only 112 of the 224 weight rows, the tensor cores read
// the other half from the peer's shared memory, and the bytes per SM and stage drop by 30 %.
//
// Schedule (224 / 240 columns).  Every pair gets the same number of whole tiles, and the tiles left over are each cut
// along K into equal pieces for consecutive pairs, which the pairs work off FIRST.  A pair that computed a piece
// publishes its fp32 partial tile to a workspace slot and counts itself on the tile's "arrived" counters; once all
// pieces are there, every participant sums (in piece order: deterministic) a share of the tile's column chunks and
// stores them.  All of this fix-up traffic and waiting happens while the pairs' main loops are busy with their whole
// tiles; what is exposed at the end of every pair is one plain tile epilogue, whose chunks are each staged in a buffer
// of their own taken from the idle pipeline ring.  Stream-K is at its worst where the tiles exceed the pairs by little
// (the paper's down projection at 2048 tokens: 88 tiles on 74 pairs); such a call takes the 288-column instance instead:
// 72 tiles, one per pair, nothing published or fixed up.
//
// Roles (6 warps per CTA):
//   warp 0    TMA producer (both CTAs): per 256-element reduction stage its own activation tile, its
//             half of the weight tile, the scale bytes of its activation rows and of all weight rows of the tile;
//             all copies of both CTAs are counted on the LEADER's "full" mbarrier;
//   warp 1    leader CTA: tcgen05 issuer -- the stage's scale-atom copies shared -> tensor memory (each CTA
//             copies from its own shared memory), up to four K = 64 steps (one MMA each; two of 144 columns in the
//             288-column instance), one commit that arrives on the "empty" barrier of both CTAs.  In the other CTA
//             this warp only allocates and frees tensor memory;
//   warps 2-5 epilogue (both CTAs): tcgen05.ld of their 32-lane quarter of the CTA's 128 accumulator
//             rows, 32 columns at a time, into swizzled shared staging, then one TMA store per warp and
//             chunk (rows and columns outside M x N are clipped by the tensor map).  Gated instance: instead of
//             storing y, form silu(gate) * up per (gate, up) group of 32 + 32 columns, quantise it to MXFP4 and write
//             codes and scale bytes of the down projection's input (Eq. (1), middle line).
//
// The activation tail is re-read, not copied: stages past the K main columns load the activation tile
// from column K - k and the weight tile from column K onwards (Kernel design paragraph).
// Every wait is bounded (the limit is a launch parameter); on expiry the CTA raises its abort flag and the peer's, all
// roles unwind, both CTAs meet at the closing cluster barrier, tensor memory is freed and PRQ_ERR_TIMEOUT is recorded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "prq_kernels.h"
#include "prq_ptx.cuh"
#include "prq_quant_block.cuh"

namespace prq {
namespace {

constexpr int kThreads = 192;
constexpr int kPTile = 128 * 128;                 // activation tile bytes (128 rows x 256 codes)
constexpr int kSfp = kSfGroupBytes;               // 1 group of 128 activation rows
constexpr int kStages = 5;
constexpr int kStagingPerWarp = 2 * 4096;         // two 32-row x 128-byte chunks per epilogue warp
constexpr int kTmemCols = 512;
constexpr int kChunkCols = 32;                    // accumulator columns per epilogue chunk

// Everything that depends on the tile width BN (weight rows per tile): 224, 240 or 288.
//   224 / 240: two accumulators of BN columns and the scale columns must fit the 512 columns of tensor memory,
//   which 240 still does; the wider tile needs fewer operand bytes per multiply-add, its main loop runs within a
//   few percent of the tensor time, and it pads N = 2560 less (11 x 240 against 12 x 224).
//   288: ONE accumulator, for calls whose tiles all fit one wave of pairs at this width (the host decides): no
//   pair takes a second tile, so nothing needs a second accumulator, and no tile is split along K.  An MMA takes at
//   most 256 columns, so a reduction step is two instructions of 144 columns each (an MMA of 32 columns costs about as
//   much as one of 64: 256 + 32 measured 9 % slower than 144 + 144 predicts); each CTA loads 72 + 72 weight rows -- rows
//   [72 r, +72) and [144 + 72 r, +72) of the tile -- so that the accumulator's columns are the tile's weight rows in
//   order, and the scale bytes are tiled per 144-row half (two groups each).
template <int BN>
struct PCfg {
    static constexpr bool kWide = BN > 256;
    static constexpr int kHalfN = BN / 2;                    // weight rows each CTA of the pair loads
    static constexpr int kQTile = kHalfN * 128;              // half weight tile bytes
    static constexpr int kHalfGroups = kWide ? (BN / 2 + 127) / 128 : 0;                    // scale groups per 144-row half
    static constexpr int kSfqGroups = kWide ? 2 * kHalfGroups : (BN + 127) / 128;           // 128-row scale groups of a weight tile
    static constexpr int kSfq = kSfqGroups * kSfGroupBytes;
    static constexpr int kStageBytes = kPTile + kQTile + kSfp + kSfq;  // 33792 / 34816 / 39936
    // the alternating staging buffers serve epilogues that run under a main loop; the one-wave tile has only a last
    // epilogue, which stages in the idle ring
    static constexpr int kStagingBytes = kWide ? 0 : 4 * kStagingPerWarp;
    static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;
    static constexpr int kAccBufs = kWide ? 1 : 2;
    static constexpr int kSfCol = kAccBufs * BN;             // scale columns start behind the accumulator(s)
    static constexpr int kSfSetCols = 8 + 8 * kSfqGroups;    // 8 activation + 8 per weight group
    static constexpr int kChunks = (BN + kChunkCols - 1) / kChunkCols;   // 7, 7 and a 16-column one, or 9
    static constexpr int kLastCols = BN - (kChunks - 1) * kChunkCols;    // 32 or 16
    static constexpr int kSlotUnits = kChunks * 8 * 128;     // float4 per workspace slot (128 rows)
    static_assert(kQTile % 1024 == 0 && kStageBytes % 1024 == 0, "operand tiles must keep 1024-byte alignment");
    static_assert(kSmemBytes <= 232448 - 256, "shared memory budget");
    static_assert(kSfCol + kSfSetCols <= kTmemCols, "tensor memory budget");
    static_assert(kLastCols == 32 || kLastCols == 16, "epilogue chunks are 32 columns, the last one 32 or 16");
    static_assert(kWide || static_cast<size_t>(kSlotUnits) * 16 <= kPrefillSlotBytes, "workspace slot");
};

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
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

struct Segment {
    int tile, s0, s1;   // reduction stages [s0, s1) of `tile`
};

// The work of one pair, walked segment by segment: first its contiguous range of (tile, stage) units of
// the stream-K tiles, then its whole tiles (tile ids sk_tiles + wave * G + pair).
// All of this is 32-bit arithmetic (the host checks that W * G fits): 64-bit divisions cost hundreds of
// cycles each and sit on the critical path of every role's first instruction.
struct Range {
    uint32_t cur, end;
    int S;
    int next_whole, whole_left, G, total;
    __device__ __forceinline__ bool next(Segment& g) {
        if (cur < end) {
            g.tile = static_cast<int>(cur / static_cast<uint32_t>(S));
            g.s0 = static_cast<int>(cur - static_cast<uint32_t>(g.tile) * S);
            const uint32_t left = end - cur;
            g.s1 = left < static_cast<uint32_t>(S - g.s0) ? g.s0 + static_cast<int>(left) : S;
            cur += g.s1 - g.s0;
            return true;
        }
        if (whole_left > 0 && next_whole < total) {
            g.tile = next_whole;
            g.s0 = 0;
            g.s1 = S;
            next_whole += G;
            --whole_left;
            return true;
        }
        return false;
    }
};

__device__ __forceinline__ uint32_t range_begin(uint32_t W, int g, int G) {
    return W * static_cast<uint32_t>(g) / static_cast<uint32_t>(G);
}

// How the stream-K tiles are shared out.
//   aligned: tile t is cut into P(t) equal pieces for P(t) consecutive pairs (sk_base + 1 pairs for the
//            first sk_extra tiles, sk_base for the others), so that every pair has one piece at most and
//            publishes once;
//   ranges:  the (tile, stage) units are cut into G equal contiguous ranges; a range may hold the tail of
//            one tile and the head of the next (two pieces).  Used when the aligned split would be too
//            coarse to balance (fewer than two pairs per tile).
struct SkPlan {
    int aligned, base, extra, S, G;
    uint32_t W;
    // the pairs that work on `tile`: first pair and count
    __device__ __forceinline__ void participants(int tile, int g, int& first, int& P) const {
        if (aligned) {
            if (tile < extra) { first = tile * (base + 1); P = base + 1; }
            else { first = extra * (base + 1) + (tile - extra) * base; P = base; }
        } else {
            const uint32_t u0 = static_cast<uint32_t>(tile) * S, u1 = u0 + S - 1;
            int gf = g, gl = g;
            while (gf > 0 && range_begin(W, gf, G) > u0) --gf;
            while (gl + 1 < G && range_begin(W, gl + 1, G) <= u1) ++gl;
            first = gf; P = gl - gf + 1;
        }
    }
    // which of its two workspace slots pair `pair` uses for its piece of `tile`
    __device__ __forceinline__ int slot_index(int pair, int tile) const {
        return (!aligned && range_begin(W, pair, G) < static_cast<uint32_t>(tile) * S) ? 1 : 0;
    }
    // the stream-K units [b, e) of pair g
    __device__ __forceinline__ void range(int g, uint32_t& b, uint32_t& e) const {
        if (!aligned) { b = range_begin(W, g, G); e = range_begin(W, g + 1, G); return; }
        int tile, j, P;
        const int cut = extra * (base + 1);
        if (g < cut) { tile = g / (base + 1); j = g - tile * (base + 1); P = base + 1; }
        else { const int h = g - cut; tile = extra + h / base; j = h - (tile - extra) * base; P = base; }
        if (static_cast<uint32_t>(tile) * S >= W) { b = e = 0; return; }   // more pairs than pieces
        b = static_cast<uint32_t>(tile) * S + static_cast<uint32_t>(S * j) / P;
        e = static_cast<uint32_t>(tile) * S + static_cast<uint32_t>(S * (j + 1)) / P;
    }
};

constexpr uint32_t kHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version 1, 128B swizzle
constexpr uint32_t kHiPlain = (128u >> 4) | (1u << 14);                // SBO 128, version 1, no swizzle
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; }

// One reduction stage of the issue loop with the ring slot Q known at compile time: every
// shared-memory descriptor is `lo_base` plus a constant.  Scale atoms first -- activation group
// (columns +0 / +4 for the two halves of the stage), then the weight groups (G = 2 or 3 of them: columns
// +8 + 4 g for the first half of the stage, +8 + 4 G + 4 g for the second) -- then up to four K = 64 steps,
// then the commit that frees the slot in both CTAs.  A step is one MMA over all BN columns, or for the
// 288-column tile two (256 columns, then the 32 columns of the third weight group into accumulator
// columns 256 ..).  The copies and the MMAs are issued by one thread, so tensor memory sees them in order
// and one set of scale columns is enough.  `rem` = reduction elements this stage still covers.
template <int BN, int Q>
__device__ __forceinline__ void issue_stage(uint32_t lo_base, uint32_t d_tmem, uint32_t sf_t, int rem,
                                            uint32_t accumulate, uint32_t empty_bar0) {
    using C = PCfg<BN>;
    constexpr int kStageBytes = C::kStageBytes, kQTile = C::kQTile, G = C::kSfqGroups;
    constexpr uint32_t so = (Q * kStageBytes) >> 4;  // stage offset in 16-byte units
    constexpr uint32_t sfo = so + ((kPTile + kQTile) >> 4);
    // E2M1 x E2M1, E8M0 scales, both operands K-major, N = N1 (and N2), M = 256 (two CTAs)
    constexpr int N1 = C::kWide ? BN / 2 : BN, N2 = BN - N1;
    constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((N1 >> 3) << 17) | (1u << 23) | ((256u >> 4) << 24);
    constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
    constexpr uint32_t jdesc0 = (1u << 7) | (1u << 10) | (((N2 > 0 ? N2 : 16) >> 3) << 17) | (1u << 23) | ((256u >> 4) << 24);
    constexpr uint32_t jdesc2 = jdesc0 | (2u << 4) | (2u << 29);
    const uint32_t plo = lo_base + so, qlo = lo_base + so + (kPTile >> 4), slo = lo_base + sfo;
    const uint32_t sfp_t = sf_t, sfq_t = sf_t + 8;
    tc_copy_sf_atom_pair(sf_t, desc64(kHiPlain, slo));
#pragma unroll
    for (int g = 0; g < G; ++g)
        tc_copy_sf_atom_pair(sfq_t + 4 * g, desc64(kHiPlain, slo + ((kSfp + g * kSfGroupBytes) >> 4)));
    if (rem > 128) {
        tc_copy_sf_atom_pair(sf_t + 4, desc64(kHiPlain, slo + (512 >> 4)));
#pragma unroll
        for (int g = 0; g < G; ++g)
            tc_copy_sf_atom_pair(sfq_t + 4 * G + 4 * g, desc64(kHiPlain, slo + ((kSfp + g * kSfGroupBytes + 512) >> 4)));
    }
    // the second instruction of a step reads the CTA's weight rows from row N1 / 2 on and the scale columns of
    // the second half's groups
    constexpr uint32_t q2 = ((N1 / 2) * 128) >> 4, s2 = 4 * C::kHalfGroups;
    tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo), desc64(kHiSw128, qlo), idesc0, sfp_t, sfq_t, accumulate);
    if (N2 > 0) tc_mma_mxf4_pair(d_tmem + N1, desc64(kHiSw128, plo), desc64(kHiSw128, qlo + q2), jdesc0, sfp_t, sfq_t + s2, accumulate);
    if (rem > 64) {
        tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 2), desc64(kHiSw128, qlo + 2), idesc2, sfp_t, sfq_t, 1);
        if (N2 > 0) tc_mma_mxf4_pair(d_tmem + N1, desc64(kHiSw128, plo + 2), desc64(kHiSw128, qlo + q2 + 2), jdesc2, sfp_t, sfq_t + s2, 1);
    }
    if (rem > 128) {
        tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 4), desc64(kHiSw128, qlo + 4), idesc0, sfp_t + 4, sfq_t + 4 * G, 1);
        if (N2 > 0) tc_mma_mxf4_pair(d_tmem + N1, desc64(kHiSw128, plo + 4), desc64(kHiSw128, qlo + q2 + 4), jdesc0, sfp_t + 4, sfq_t + 4 * G + s2, 1);
    }
    if (rem > 192) {
        tc_mma_mxf4_pair(d_tmem, desc64(kHiSw128, plo + 6), desc64(kHiSw128, qlo + 6), idesc2, sfp_t + 4, sfq_t + 4 * G, 1);
        if (N2 > 0) tc_mma_mxf4_pair(d_tmem + N1, desc64(kHiSw128, plo + 6), desc64(kHiSw128, qlo + q2 + 6), jdesc2, sfp_t + 4, sfq_t + 4 * G + s2, 1);
    }
    tc_commit_pair(empty_bar0 + Q * 8, 3);
}

template <int BN, bool kGated = false>
__global__ void __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfw,
                    const __grid_constant__ CUtensorMap tm_y, const PrefillParams p) {
    using C = PCfg<BN>;
    constexpr int kHalfN = C::kHalfN, kQTile = C::kQTile, kStageBytes = C::kStageBytes, kSfCol = C::kSfCol;
    constexpr int kChunks = C::kChunks, kLastCols = C::kLastCols;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int fixup_gave_up_s;   // an epilogue warp's wait for a stream-K tile's pieces ended without them
    volatile int* abort_flag = &abort_flag_s;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t staging_base = smem_base + kStages * kStageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
    const StagePlan plan(p.K, p.k_tail);
    const int S = plan.S, S1 = plan.S1;
    const int G = gridDim.x >> 1, g = blockIdx.x >> 1;   // pairs
    const uint32_t W = static_cast<uint32_t>(p.sk_tiles) * S;   // stream-K units, shared out over all pairs
    const SkPlan plan_sk{p.sk_aligned, p.sk_base, p.sk_extra, S, G, W};
    uint32_t sk_b, sk_e;
    plan_sk.range(g, sk_b, sk_e);

    long long* const ptrace = kTraceBuild ? p.trace : nullptr;
    if (ptrace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        ptrace[2048 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bar_acc_full[i]), 1);
            mbar_init(smem_u32(&bar_acc_empty[i]), 8);   // four epilogue warps of each CTA
        }
        abort_flag_s = 0;
        fixup_gave_up_s = 0;
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
    // kernel).  Each role that touches global memory which earlier kernels wrote (activation codes,
    // workspace counters) or still read (y) passes grid_dependency_wait() first; the issuer touches none.
    if (ptrace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        ptrace[2048 + 400 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    grid_launch_dependents();
    const uint32_t tmem_base = tmem_slot;
    const int trace_cta0 = p.dbg >> 16;  // developer aid: first of the four traced CTAs
    long long* trace = (ptrace && static_cast<int>(blockIdx.x) >= trace_cta0 && static_cast<int>(blockIdx.x) < trace_cta0 + 4)
                           ? ptrace + (blockIdx.x - trace_cta0) * 512 : nullptr;
    if (trace && threadIdx.x == 0) trace[500] = clock64();
    const uint32_t lo_base = ((smem_base & 0x3FFFF) >> 4) | (1u << 16);

    if (warp == 0) {
        // ------------------------------------------------------------ producer (both CTAs)
        Range r{sk_b, sk_e, S, p.sk_tiles + g, p.whole_tiles, G, p.total_tiles};
        Segment sg;
        int st = 0, it = 0;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t leader_full0 = cluster_map(smem_u32(&bar_full[0]), 0);
        // The weights do not depend on earlier kernels of the stream: the weight tiles and weight scales of
        // the first ring pass are requested before the dependency wait, so that their latency overlaps the
        // tail of the previous kernel.
        // this CTA's half of the weight tile `ni` and the scale bytes of the whole tile, reduction stage s.
        // 224 / 240 columns: rows [rank * BN / 2, + BN / 2) of the tile.  288 columns: rows [72 rank, + 72) and
        // [144 + 72 rank, + 72), so that the two instructions of a step cover the tile's two halves in order.
        auto load_weights = [&](uint32_t sb, int ni, int s, uint32_t full) {
            const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
            if (C::kWide) {
                constexpr int q = BN / 4;   // 72 rows per box
                tma_load_2d_pair(sb + kPTile, &tm_w, xw, ni * BN + static_cast<int>(rank) * q, full);
                tma_load_2d_pair(sb + kPTile + q * 128, &tm_w, xw, ni * BN + BN / 2 + static_cast<int>(rank) * q, full);
            } else {
                tma_load_2d_pair(sb + kPTile, &tm_w, xw, ni * BN + static_cast<int>(rank) * kHalfN, full);
            }
            tma_load_2d_pair(sb + kPTile + kQTile + kSfp, &tm_sfw, 0, ni * 4 * C::kSfqGroups + s * p.w_groups * 4, full);
        };
        int pre = 0;
        {
            Range rr = r;
            while (pre < kStages && rr.next(sg)) {
                const int ni = sg.tile / p.m_tiles;
                for (int s = sg.s0; s < sg.s1 && pre < kStages; ++s, ++pre) {
                    if (elect_one()) load_weights(smem_base + pre * kStageBytes, ni, s, leader_full0 + pre * 8);
                }
            }
        }
        grid_dependency_wait();
        if (ptrace && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            ptrace[2048 + 401 + 2 * blockIdx.x] = static_cast<long long>(t);
        }
        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            // scale bytes: rows of 256 bytes, 4 per 128-row group
            const int sfa_row0 = (mi * 2 + static_cast<int>(rank)) * 4, sfa_stride = p.act_groups * 4;
            for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                if (!mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[it] = clock64();
                if (elect_one()) {
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&bar_full[st]), 2 * kStageBytes);
                    const uint32_t full = leader_full0 + st * 8;
                    const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                    const uint32_t sb = smem_base + st * kStageBytes;
                    tma_load_2d_pair(sb, &tm_act, xa, mi * 256 + static_cast<int>(rank) * 128, full);
                    tma_load_2d_pair(sb + kPTile + kQTile, &tm_sfa, 0, sfa_row0 + s * sfa_stride, full);
                    if (it >= pre) load_weights(sb, ni, s, full);
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
            Range r{sk_b, sk_e, S, p.sk_tiles + g, p.whole_tiles, G, p.total_tiles};
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
                // (the 288-column tile has one accumulator: the host gives such a call one tile per pair at most)
                const int buf = C::kAccBufs == 2 ? (seg_it & 1) : 0;
                if (trace && lane == 0 && seg_it < 8) trace[216 + 2 * seg_it] = clock64();
                if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), ((seg_it >> 1) & 1) ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                if (trace && lane == 0 && seg_it < 8) trace[217 + 2 * seg_it] = clock64();
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                uint32_t accumulate = 0;
                for (int s = sg.s0; s < sg.s1; ++s, ++it) {
                    if (!ready && !mbar_wait(smem_u32(&bar_full[st]), ph, abort_flag, p.wait_limit)) { ok = false; break; }
                    if (trace && lane == 0 && it < 64) trace[64 + it] = clock64();
                    const int rem = s < S1 ? p.K - s * kStageK : p.k_tail - (s - S1) * kStageK;
                    const int nst = st + 1 == kStages ? 0 : st + 1;
                    const uint32_t nph = nst == 0 ? ph ^ 1 : ph;
                    ready = mbar_test_wait(smem_u32(&bar_full[nst]), nph);
                    if (leader) {
                        const uint32_t eb = smem_u32(&bar_empty[0]);
                        switch (st) {
                            case 0: issue_stage<BN, 0>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 1: issue_stage<BN, 1>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 2: issue_stage<BN, 2>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            case 3: issue_stage<BN, 3>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
                            default: issue_stage<BN, 4>(lo_base, d_tmem, sf_t, rem, accumulate, eb); break;
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
        grid_dependency_wait();
        const int q4 = warp & 3;                 // tensor-memory lane quarter of this warp
        const int row_in_tile = q4 * 32 + lane;  // row of this CTA's 128-row half
        const uint32_t stage_smem = staging_base + (warp - 2) * kStagingPerWarp;
        const uint32_t leader_acc_empty0 = cluster_map(smem_u32(&bar_acc_empty[0]), 0);
        Range r{sk_b, sk_e, S, p.sk_tiles + g, p.whole_tiles, G, p.total_tiles};
        Segment sg;
        int seg_it = 0, store_it = 0;
        bool ok = true;

        // 32 accumulator columns of this warp's 32 rows -> y: swizzled shared staging, then one TMA store
        // (rows and columns outside M x N are clipped by the tensor map)
        // first column of a right edge narrower than 16 bytes, or -1 if N is a multiple of 16 bytes
        const int ragged_col = (p.N % (p.y_bf16 ? 8 : 4)) ? p.N - p.N % (p.y_bf16 ? 8 : 4) : -1;
        // `own_buf`: shared address of a staging buffer that belongs to this chunk alone (the CTA's last tile, see
        // below), or 0 for the warp's two alternating buffers
        auto store_chunk = [&](const uint32_t (&v)[32], int x, int y_row, int cols, uint32_t own_buf = 0) {
            // A tiled store clips at the tensor's edge in units of 16 bytes: where N is not a multiple of that,
            // it would fill the last column group up with zeros, i.e. write into the caller's bytes between
            // column N and the row stride.  That one chunk goes out with plain stores instead.
            if (ragged_col >= x && ragged_col < x + cols) {
                const int row = y_row + lane;
                if (row < p.M) {
                    if (p.y_bf16) {
                        __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<size_t>(row) * p.ldy + x;
                        for (int i = 0; i < cols && x + i < p.N; ++i) yp[i] = __float2bfloat16_rn(__uint_as_float(v[i]));
                    } else {
                        float* yp = reinterpret_cast<float*>(p.y) + static_cast<size_t>(row) * p.ldy + x;
                        for (int i = 0; i < cols && x + i < p.N; ++i) yp[i] = __uint_as_float(v[i]);
                    }
                }
                return;
            }
            // The 16-column chunk that closes a 240-column tile: 64 (32) contiguous bytes per row, written with
            // 16-byte stores (y and its row stride are 16-byte aligned -- the tensor map demands it -- and chunks
            // start at multiples of 16 columns).  Columns from N on are dropped 16 bytes at a time; a narrower
            // rest is the ragged chunk above.
            if (kLastCols == 16 && cols == 16) {
                const int row = y_row + lane;
                if (row < p.M) {
                    if (p.y_bf16) {
                        uint4* yp = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<size_t>(row) * p.ldy + x);
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            uint32_t h[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(v[8 * u + 2 * i]), __uint_as_float(v[8 * u + 2 * i + 1]));
                                h[i] = *reinterpret_cast<uint32_t*>(&t2);
                            }
                            if (x + 8 * u + 8 <= p.N) yp[u] = make_uint4(h[0], h[1], h[2], h[3]);
                        }
                    } else {
                        uint4* yp = reinterpret_cast<uint4*>(reinterpret_cast<float*>(p.y) + static_cast<size_t>(row) * p.ldy + x);
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (x + 4 * u + 4 <= p.N) yp[u] = make_uint4(v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
                    }
                }
                return;
            }
            const uint32_t sbuf = own_buf ? own_buf : stage_smem + (store_it & 1) * 4096;
            if (!own_buf) {
                // the store issued two chunks ago has finished reading this buffer
                if (lane == 0) bulk_wait_read<1>();
                __syncwarp();
            }
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
                tma_store_2d(&tm_y, sbuf, x, y_row);
                bulk_commit();
            }
            ++store_it;
        };

        // A stream-K tile is finished in two steps.  Publish: every pair that computed a piece of it writes
        // its fp32 partial tile to a workspace slot and counts itself on the "arrived" counter of its
        // 128-row half.  Fix up: once all P pieces have arrived, participant i sums, always in piece order,
        // the column chunks c = i, i + P, ... over all pieces and stores them to y; the last participant to
        // finish clears the counters for the next launch.  The fix-ups are deferred until all of the pair's
        // own pieces are published (a fix-up waits for other pairs; a publication must never wait), and
        // they run while the main loop works on the pair's whole tiles.
        struct Fixup { int tile, first_pair, P; };
        Fixup fix[2];
        int n_fix = 0;
        auto slot_of = [&](int pair, int tile) -> const float4* {
            const int k = plan_sk.slot_index(pair, tile);
            return reinterpret_cast<const float4*>(p.partial) +
                   static_cast<size_t>(2 * (2 * pair + static_cast<int>(rank)) + k) * C::kSlotUnits;
        };
        auto run_fixups = [&]() {
            for (int f = 0; f < n_fix && ok; ++f) {
                const Fixup fx = fix[f];
                int* arrived = p.flags + 2 * fx.tile + rank;
                int* finished = arrived + p.flag_stride;
                if (lane == 0) {
                    volatile int* a = arrived;
                    const long long t0 = clock64();
                    while (*a < fx.P) {
                        if (*abort_flag) { fixup_gave_up_s = 1; break; }
                        if (clock64() - t0 > p.wait_limit) { *abort_flag = 1; fixup_gave_up_s = 1; break; }
                    }
                }
                // The four warps decide together, on a word that is written only before this barrier: a warp
                // that saw the counter complete must not go on to the barrier at the end of the fix-up while
                // another one gave up a moment earlier and will never arrive there.
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (*reinterpret_cast<volatile int*>(&fixup_gave_up_s)) { ok = false; break; }
                __threadfence();
                const int mi = fx.tile % p.m_tiles, ni = fx.tile / p.m_tiles;
                const int y_row = mi * 256 + static_cast<int>(rank) * 128 + q4 * 32;
                for (int c = g - fx.first_pair; c < kChunks; c += fx.P) {
                    // unit (c, u) of row r sits at float4 index (c * 8 + u) * 128 + r of a slot
                    const size_t off = static_cast<size_t>(c) * 8 * 128 + row_in_tile;
                    const int cols = c == kChunks - 1 ? kLastCols : kChunkCols;
                    const int nu = cols >> 2;   // 16-byte units per row of this chunk
                    float4 a4[8], b4[8];
                    const float4* s0p = slot_of(fx.first_pair, fx.tile) + off;
#pragma unroll
                    for (int u = 0; u < 8; ++u) a4[u] = u < nu ? __ldcg(s0p + u * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int j = 1; j < fx.P; ++j) {
                        const float4* sp = slot_of(fx.first_pair + j, fx.tile) + off;
#pragma unroll
                        for (int u = 0; u < 8; ++u) b4[u] = u < nu ? __ldcg(sp + u * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            a4[u].x += b4[u].x; a4[u].y += b4[u].y; a4[u].z += b4[u].z; a4[u].w += b4[u].w;
                        }
                    }
                    uint32_t v[32];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        v[4 * u] = __float_as_uint(a4[u].x); v[4 * u + 1] = __float_as_uint(a4[u].y);
                        v[4 * u + 2] = __float_as_uint(a4[u].z); v[4 * u + 3] = __float_as_uint(a4[u].w);
                    }
                    store_chunk(v, ni * BN + c * kChunkCols, y_row, cols);
                }
                // all four warps have read what they need of this half
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (row_in_tile == 0) {
                    if (atomicAdd(finished, 1) == fx.P - 1) { *finished = 0; *arrived = 0; }
                }
                if (trace && row_in_tile == 0 && f < 2) trace[208 + f] = clock64();
            }
            n_fix = 0;
        };

        // accumulator columns [c * 32, c * 32 + cols) of this warp's rows -> v (waits for the data)
        auto load_chunk = [&](uint32_t acc_t, int c, uint32_t (&v)[32]) -> int {
            if (kLastCols == 16 && c == kChunks - 1) {
                uint32_t h[16];
                tmem_ld_32x16(acc_t + c * kChunkCols, h);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) { v[i] = h[i]; v[16 + i] = 0; }
                return 16;
            }
            tmem_ld_32x32(acc_t + c * kChunkCols, v);
            tmem_ld_wait();
            return kChunkCols;
        };

        while (ok && r.next(sg)) {
            const int mi = sg.tile % p.m_tiles, ni = sg.tile / p.m_tiles;
            const int buf = C::kAccBufs == 2 ? (seg_it & 1) : 0;
            const bool piece = sg.s1 - sg.s0 < S;
            // all of this pair's pieces are published: fix up now, overlapping the main loop of this whole tile
            if (!piece && n_fix > 0 && r.cur >= r.end) run_fixups();
            if (!ok) break;
            if (!mbar_wait(smem_u32(&bar_acc_full[buf]), (seg_it >> 1) & 1, abort_flag, p.wait_limit)) { ok = false; break; }
            if (trace && row_in_tile == 0 && seg_it < 8) trace[192 + 2 * seg_it] = clock64();
            tc_fence_after_sync();
            const uint32_t acc_t = tmem_base + buf * BN + (static_cast<uint32_t>(q4 * 32) << 16);
            if constexpr (kGated) {
                // Gated-producer epilogue (Eq. (1), middle line, with the activation function inside the producer):
                // the tile's columns are (gate, up) groups of 32 + 32 output features.  Per group a thread holds,
                // for its token row, 32 gate and 32 up sums: h = bf16(silu(gate) * up) is one 32-element block of
                // the down projection's input, quantised here exactly as the activation quantiser would (same
                // function), and written as 16 bytes of codes and one scale byte.  The product never exists in
                // global memory (unless the caller asks for it to check).
                static_assert(!kGated || BN % 64 == 0, "whole (gate, up) groups per tile");
                const int row = mi * 256 + static_cast<int>(rank) * 128 + row_in_tile;
                const int grp = row >> 7, rg = row & 127;
                const int C = p.out_C;
                const int tail_blk0 = (C - p.out_k_tail) / kBlock, S1o = C / kStageK;
#pragma unroll 1
                for (int j = 0; j < BN / 64; ++j) {
                    uint32_t vg[32], vu[32];
                    tmem_ld_32x32(acc_t + j * 64, vg);
                    tmem_ld_32x32(acc_t + j * 64 + 32, vu);
                    tmem_ld_wait();
                    if (j == BN / 64 - 1) {
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + buf * 8);
                    }
                    const int fb = (ni * BN) / 64 + j;            // 32-channel block of the down projection's input
                    if (fb * kBlock >= C || grp >= p.out_groups) continue;
                    uint4 q[4];
                    uint32_t* qw = reinterpret_cast<uint32_t*>(q);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float g0 = __uint_as_float(vg[2 * i]), g1 = __uint_as_float(vg[2 * i + 1]);
                        const float h0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(vu[2 * i]);
                        const float h1 = __fdividef(g1, 1.f + __expf(-g1)) * __uint_as_float(vu[2 * i + 1]);
                        const __nv_bfloat162 hh = __floats2bfloat162_rn(h0, h1);
                        qw[i] = *reinterpret_cast<const uint32_t*>(&hh);
                    }
                    const bool live = row < p.M;
                    if (!live) { q[0] = q[1] = q[2] = q[3] = make_uint4(0, 0, 0, 0); }
                    uint4 codes;
                    const uint32_t byte = live ? quant_block32(q, codes) : 0u;   // rows past M: scale bytes stay 2^-127
                    if (live) {
                        *reinterpret_cast<uint4*>(p.out_codes + static_cast<size_t>(row) * (C / 2) + fb * 16) = codes;
                        if (p.out_scales_row) p.out_scales_row[static_cast<size_t>(row) * (C / kBlock) + fb] = static_cast<uint8_t>(byte);
                        if (p.out_h) {
                            uint4* hp = reinterpret_cast<uint4*>(p.out_h + static_cast<size_t>(row) * C + fb * kBlock);
                            hp[0] = q[0]; hp[1] = q[1]; hp[2] = q[2]; hp[3] = q[3];
                        }
                    }
                    uint8_t* sfg = p.out_sf + static_cast<size_t>(grp) * kSfGroupBytes;
                    const size_t stage_stride = static_cast<size_t>(p.out_groups) * kSfGroupBytes;
                    sfg[(fb >> 3) * stage_stride + sf_offset_in_group(rg, fb & 7)] = static_cast<uint8_t>(byte);
                    if (fb >= tail_blk0) {   // the tail's scale bytes a second time, in the residual stages
                        const int t = fb - tail_blk0;
                        sfg[(S1o + (t >> 3)) * stage_stride + sf_offset_in_group(rg, t & 7)] = static_cast<uint8_t>(byte);
                    }
                }
            } else if (piece) {
                // publish this piece: partial accumulator -> workspace slot (one 512-byte line per warp store)
                const int k = plan_sk.slot_index(g, sg.tile);
                float4* slot = reinterpret_cast<float4*>(p.partial) +
                               static_cast<size_t>(2 * blockIdx.x + k) * C::kSlotUnits + row_in_tile;
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    const int nu = load_chunk(acc_t, c, v) >> 2;
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (u < nu)
                            __stcg(slot + (c * 8 + u) * 128,
                                   make_float4(__uint_as_float(v[4 * u]), __uint_as_float(v[4 * u + 1]),
                                               __uint_as_float(v[4 * u + 2]), __uint_as_float(v[4 * u + 3])));
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + buf * 8);
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (row_in_tile == 0) atomicAdd(p.flags + 2 * sg.tile + rank, 1);
                int first, P;
                plan_sk.participants(sg.tile, g, first, P);
                fix[n_fix++] = Fixup{sg.tile, first, P};
            } else if (r.cur >= r.end && r.whole_left == 0 && !(kTraceBuild && (p.dbg & 4))) {
                // The CTA's last tile.  Nothing overlaps this epilogue, and with two staging buffers per warp it
                // runs at the latency of the stores (a chunk waits for the store issued two chunks earlier).  The
                // pipeline ring is idle by now -- the accumulator is complete, so every load has landed and every
                // tensor-core read of both CTAs' shared memory is done -- and gives every chunk a staging buffer
                // of its own: the warp reads the accumulator and issues its stores without ever waiting for one.
                const int y_row = mi * 256 + static_cast<int>(rank) * 128 + q4 * 32;
                const uint32_t own0 = smem_base + static_cast<uint32_t>((warp - 2) * kChunks) * 4096u;
                static_assert(4 * kChunks * 4096 <= kStages * kStageBytes, "one staging buffer per warp and chunk fits the ring");
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    const int cols = load_chunk(acc_t, c, v);
                    store_chunk(v, ni * BN + c * kChunkCols, y_row, cols, own0 + c * 4096u);
                }
            } else {
                const int y_row = mi * 256 + static_cast<int>(rank) * 128 + q4 * 32;
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
                    uint32_t v[32];
                    const int cols = load_chunk(acc_t, c, v);
                    if (c == kChunks - 1) {
                        // the accumulator has been read completely: hand it back before the stores drain
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + buf * 8);
                    }
                    store_chunk(v, ni * BN + c * kChunkCols, y_row, cols);
                }
            }
            if (trace && row_in_tile == 0 && seg_it < 8) trace[193 + 2 * seg_it] = clock64();
            ++seg_it;
        }
        if (ok && n_fix > 0) run_fixups();   // no whole tiles: the fix-ups come last
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
    if (ptrace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        ptrace[2049 + 2 * blockIdx.x] = static_cast<long long>(t);
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

template <int BN, bool kGated = false>
int max_clusters_bn() {
    constexpr int kSmemBytes = PCfg<BN>::kSmemBytes;
    static int cached = -1;
    if (cached >= 0) return cached;
    if (cudaFuncSetAttribute(prefill_pair_kernel<BN, kGated>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return 0;
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
    if (cudaOccupancyMaxActiveClusters(&n, prefill_pair_kernel<BN, kGated>, &cfg) != cudaSuccess) return 0;
    cached = n;
    return n;
}

template <int BN, bool kGated = false>
cudaError_t launch_bn(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const CUtensorMap& tm_sfa,
                      const CUtensorMap& tm_sfw, const CUtensorMap& tm_y, const PrefillParams& p,
                      int pairs, cudaStream_t stream) {
    constexpr int kSmemBytes = PCfg<BN>::kSmemBytes;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(prefill_pair_kernel<BN, kGated>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
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
    return cudaLaunchKernelEx(&cfg, prefill_pair_kernel<BN, kGated>, tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p);
}

}  // namespace

int prefill_pair_max_clusters(int bn) {
    if (bn == kPrefillTileGated) return max_clusters_bn<kPrefillTileGated, true>();
    return bn == kPrefillTileOneWave ? max_clusters_bn<kPrefillTileOneWave>()
           : bn == kPrefillTileWide ? max_clusters_bn<kPrefillTileWide>() : max_clusters_bn<kPrefillTileN>();
}

cudaError_t launch_prefill_pair(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w,
                                const CUtensorMap& tm_sfa, const CUtensorMap& tm_sfw, const CUtensorMap& tm_y,
                                const PrefillParams& p, int pairs, cudaStream_t stream) {
    if (bn == kPrefillTileOneWave) {
        // one accumulator: no pair may be given a second tile or a piece of one
        if (p.whole_tiles + (p.sk_tiles > 0 ? 1 : 0) > 1 || (p.sk_tiles > 0 && p.sk_base != 1) || p.sk_extra != 0) return cudaErrorInvalidValue;
        return launch_bn<kPrefillTileOneWave>(tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p, pairs, stream);
    }
    if (bn == kPrefillTileGated) {
        // whole tiles only: a piece of a tile has no (gate, up) sums to put through the activation function
        if (p.sk_tiles != 0 || !p.out_codes || !p.out_sf) return cudaErrorInvalidValue;
        return launch_bn<kPrefillTileGated, true>(tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p, pairs, stream);
    }
    if (bn == kPrefillTileWide) return launch_bn<kPrefillTileWide>(tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p, pairs, stream);
    if (bn == kPrefillTileN) return launch_bn<kPrefillTileN>(tm_act, tm_w, tm_sfa, tm_sfw, tm_y, p, pairs, stream);
    return cudaErrorInvalidValue;
}

}  // namespace prq
