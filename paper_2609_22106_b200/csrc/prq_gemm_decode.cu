// Decode GEMM (M <= 128 tokens): the block-scaled FP4 product of Eq. (3) as a weight-streaming kernel.
//
// With few tokens the layer is bound by reading its 4-bit weights once.  The weight rows sit on the MMA
// M axis (128-row tiles), the tokens on the N axis (16, 32, 64 or 128 columns), and the reduction axis
// K + k is split over the CTAs of a thread-block cluster so that every SM streams a share of the
// weights.  Each CTA of a cluster accumulates its K-range in tensor memory and then pushes, through
// distributed shared memory, the partial sums of token t into a receive buffer of the CTA that owns
// token t (t mod cluster size); the owner adds up what it received and writes its tokens to y.  Up to 32
// tokens the pushes are asynchronous stores whose bytes are counted on an mbarrier of the owner, which
// therefore waits for exactly its own tokens; from 64 tokens on they are plain stores followed by one
// cluster barrier.  No global scratch, no atomics, and the summation order is fixed (peer 0, 1, ...), so
// the result is reproducible.  For up to 32 tokens two CTAs fit on an SM, so that the
// CTAs of the next kernel of the stream (the next layer's GEMM) are resident and streaming their weights
// while this one finishes.
//
// Roles per CTA (6 warps, 10 from 64 tokens on): warp 0 TMA producer, warp 1 tcgen05 issuer (scale copies + MMAs), warps 2-5 (2-9)
// epilogue and reduction.  The activation tail is re-read: stages past the K main columns load the
// token tile from column K - k and the weight tile from column K onwards (Kernel design paragraph).
// Every wait is bounded; the cluster barriers sit on the common path so that a CTA that gave up still
// arrives and its peers are released, and a CTA that gave up under the asynchronous exchange stays until its
// peers' deliveries into its receive buffer have landed.
// The kernel is latency-bound, not bandwidth-bound (with the weights resident in L2 it is only 0.5-1 us faster): what a
// launch costs is the chain token copies -> five stages of tcgen05 issue -> accumulator read -> exchange -> store behind
// its dependency, plus the hand-over to the next kernel.
//
// Fused variant (up to 16 tokens, activation already scaled and reordered by its producer): the kernel
// takes the bf16 activation itself.  The four epilogue warps first act as the activation quantiser of
// their CTA -- one 32-element block per thread and stage, codes written straight into the 128-byte-
// swizzled token tile of the pipeline slot, scale bytes into the slot's scale atom -- so that the
// separate quantiser launch, its round trip through global memory and one kernel-to-kernel hand-over
// leave the decode step (the Kernel design paragraph asks for one quantisation of the reordered activation
// per layer call; here it happens inside the product kernel).
// Every cluster quantises the K-range it reduces over, i.e. the bf16 activation is read once per 128-row
// weight tile; that extra L2 traffic grows with the token count and is why the variant stops at 16 tokens.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstring>

#include "prq_kernels.h"
#include "prq_ptx.cuh"
#include "prq_quant_block.cuh"

namespace prq {
namespace {

constexpr int kPTile = 128 * 128;   // weight tile bytes: 128 rows x 256 codes
constexpr int kSf = kSfGroupBytes;  // one 128-row scale group per operand and stage

constexpr uint32_t kHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kHiPlain = (128u >> 4) | (1u << 14);
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; }
constexpr int pow2_cols(int x) { int p = 32; while (p < x) p *= 2; return p; }

// kDense: the variant for layers with more 128-row weight tiles than the GPU has SMs (from 64 tokens on one
// CTA fills an SM, so tile 149 would wait for a second wave that leaves most SMs idle).  Such a layer is not
// K-split, so its CTAs need no receive buffer; with a 3-slot ring two of them share an SM and all tiles are
// resident at once (stacked gate / up projection, 152 tiles: 16.2 -> 12.1 us at 64 tokens, 20.0 -> 14.1 at 128).
template <int BN, bool kDense = false>
struct DCfg {
    static_assert(!kDense || BN >= 64, "up to 32 tokens two CTAs share an SM anyway");
    static constexpr int kQTile = BN * 128;
    static constexpr int kStageBytes = kPTile + kQTile + 2 * kSf;
    // ring depth: 5 / 4 stages leave room for two CTAs per SM at 16 / 32 tokens
    static constexpr int kStages = kDense ? 3 : BN == 16 ? 5 : BN == 32 ? 4 : BN == 64 ? 6 : 4;
    static constexpr int kCtasPerSm = (kDense || BN <= 32) ? 2 : 1;
    // epilogue warps: four (one per tensor-memory lane quarter); eight from 64 tokens on, where moving the
    // partial sums is most of the kernel -- two warps per quarter then take alternate 16-token chunks
    static constexpr int kEpiWarps = BN >= 64 ? 8 : 4;
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    // split-K exchange: up to 32 tokens asynchronous stores counted on the owner's mbarrier (the owner waits
    // only for its own tokens: 0.3 us less at M = 1 than a cluster barrier); from 64 tokens on plain stores and
    // one cluster barrier (the per-store barrier update costs more than it saves: 9.4 against 9.6 us at M = 128)
    static constexpr bool kAsyncExchange = BN <= 32;
    // receive buffer of the split-K exchange: [peer][token slot][128 rows] fp32, ceil(BN / splits) token
    // slots per peer, i.e. at most BN + 7 token rows of 512 bytes
    static constexpr int kRecvBytes = kDense ? 0 : (BN + 7) * 512;
    static constexpr int kSmemBytes = kStages * kStageBytes + kRecvBytes + 1024;
    static constexpr int kAccCols = BN < 32 ? 32 : BN;
    static constexpr int kSfCol = kAccCols;          // 8 weight-scale + 8 token-scale columns behind the accumulator
    static constexpr int kTmemCols = pow2_cols(kAccCols + 16);
    static_assert(kStageBytes % 1024 == 0, "stage slots must keep 1024-byte alignment");
    static_assert(BN * 128 * 4 <= kStages * kStageBytes, "the partial tile is parked in the pipeline buffers");
    static_assert(kCtasPerSm * (kSmemBytes + 256) <= 232448, "shared memory budget");
};

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of `local_addr` in the shared memory of CTA `peer` of this cluster.
__device__ __forceinline__ uint32_t peer_addr(uint32_t local_addr, uint32_t peer) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(peer));
    return ra;
}
// One reduction stage issued by the elected thread.  The ring slot is a run-time value on purpose: a
// CTA runs only a handful of stages, so one compact code path that stays in the instruction cache beats
// a specialised copy per slot, each of which would be fetched cold.
template <int BN>
__device__ __forceinline__ void issue_stage(uint32_t lo_base, uint32_t d_tmem, uint32_t sf_t, int slot, int rem,
                                            uint32_t accumulate, uint32_t empty_bar0) {
    using C = DCfg<BN>;
    constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
    constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
    const uint32_t plo = lo_base + slot * (C::kStageBytes >> 4), qlo = plo + (kPTile >> 4);
    const uint32_t slo = plo + ((kPTile + C::kQTile) >> 4);
    const uint32_t sfp_t = sf_t, sfq_t = sf_t + 8;
    tc_copy_sf_atom(sfp_t, desc64(kHiPlain, slo));
    tc_copy_sf_atom(sfq_t, desc64(kHiPlain, slo + (kSf >> 4)));
    if (rem > 128) {
        tc_copy_sf_atom(sfp_t + 4, desc64(kHiPlain, slo + (512 >> 4)));
        tc_copy_sf_atom(sfq_t + 4, desc64(kHiPlain, slo + ((kSf + 512) >> 4)));
    }
    tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo), desc64(kHiSw128, qlo), idesc0, sfp_t, sfq_t, accumulate);
    if (rem > 64) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 2), desc64(kHiSw128, qlo + 2), idesc2, sfp_t, sfq_t, 1);
    if (rem > 128) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 4), desc64(kHiSw128, qlo + 4), idesc0, sfp_t + 4, sfq_t + 4, 1);
    if (rem > 192) tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 6), desc64(kHiSw128, qlo + 6), idesc2, sfp_t + 4, sfq_t + 4, 1);
    tc_commit(empty_bar0 + slot * 8);
}

template <int BN, bool kFused, bool kBatch, bool kDense = false>
__global__ void __launch_bounds__(DCfg<BN, kDense>::kThreads, DCfg<BN, kDense>::kCtasPerSm)
decode_kernel(const __grid_constant__ DecodeMaps maps, const DecodeBatch b) {
    using C = DCfg<BN, kDense>;
    // which of the batched layers this cluster works for (one launch may run several layers over the same
    // tokens, each with its own weights, activation codes and output)
    const int tile_all = static_cast<int>(blockIdx.x) / b.splits;
    int lin = 0;   // (kBatch = false: a single layer, nothing to look up)
    if (kBatch)
        while (lin + 1 < b.n_lin && tile_all >= b.lay[lin].tile_end) ++lin;
    DecodeParams p;
    p.M = b.M; p.K = b.K; p.k_tail = b.k_tail; p.x = b.x; p.ldx = b.ldx; p.y_bf16 = b.y_bf16; p.splits = b.splits;
    p.status = b.status; p.trace = b.trace; p.dbg = b.dbg;
    {
        const DecodeLayer& l = b.lay[lin];
        p.N = l.N; p.w_groups = l.w_groups; p.act_sf = l.act_sf; p.w_sf = l.w_sf; p.y = l.y; p.ldy = l.ldy;
    }
    const CUtensorMap* const tm_act = &maps.act[lin];
    const CUtensorMap* const tm_w = &maps.w[lin];
    extern __shared__ uint8_t smem_raw[];
    constexpr int kStages = C::kStages;
    __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages], bar_acc_full;
    __shared__ __align__(8) uint64_t bar_recv;   // counts the bytes of partial sums that the peers deliver to this CTA
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const StagePlan plan(p.K, p.k_tail);
    const int S = plan.S, S1 = plan.S1;
    const int splits = p.splits;
    const int tile = tile_all - (lin ? b.lay[lin - 1].tile_end : 0);   // 128-row weight tile of this layer
    const int split = static_cast<int>(blockIdx.x) - tile_all * splits;   // = rank in the cluster
    const int s_begin = static_cast<int>(static_cast<long long>(S) * split / splits);
    const int s_end = static_cast<int>(static_cast<long long>(S) * (split + 1) / splits);
    const int n0 = tile * 128;

    long long* const ptrace = kTraceBuild ? p.trace : nullptr;
    const long long t_entry = kTraceBuild ? clock64() : 0;
    __shared__ int trace_slot_s;
    if (ptrace && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g));
        const int sl = static_cast<int>(atomicAdd(reinterpret_cast<unsigned long long*>(ptrace + 2040), 1ull)) & 63;
        trace_slot_s = sl;
        ptrace[2048 + sl * 4] = static_cast<long long>(g);
    }
    if (threadIdx.x == 0) {
        // a slot is full when its TMA bytes have landed and, fused, when the four quantiser warps are done
        for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&bar_full[i]), kFused ? 5 : 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        mbar_init(smem_u32(&bar_acc_full), 1);
        mbar_init(smem_u32(&bar_recv), 1);
        abort_flag_s = 0;
        fence_mbar_init();
        tma_prefetch_desc(tm_act);
        tma_prefetch_desc(tm_w);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // Split-K exchange, receiving side: this CTA owns tokens split, split + splits, ...; every CTA of the
    // cluster (itself included) delivers 512 bytes per owned token, counted on bar_recv.  The cluster
    // barrier only tells the peers that the barrier exists before they push: arrive here, wait just before
    // the pushes, so that it costs nothing.
    const int n_own = split < p.M ? (p.M - split + splits - 1) / splits : 0;
    if (C::kAsyncExchange && splits > 1) {
        if (threadIdx.x == 0) mbar_arrive_expect_tx(smem_u32(&bar_recv), static_cast<uint32_t>(n_own) * splits * 512u);
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    // set-up done: let the next kernel of the stream be scheduled (its launch latency then overlaps this
    // kernel).  The roles that touch what earlier kernels wrote (activation codes and scales) or may
    // still read (y) pass grid_dependency_wait() first; the weights depend on no kernel, so the producer
    // requests them before it waits and they stream in while the previous kernel (normally the
    // activation quantiser) is still running.
    const long long t_setup = kTraceBuild ? clock64() : 0;
    // Up to 32 tokens the next kernel may be scheduled from here on: two CTAs share an SM, and the next GEMM's set-up and
    // weight stream overlap this one.  From 64 tokens on a CTA fills its SM and what comes next in a decode step is the
    // small-CTA activation quantiser, whose blocks would squeeze in beside this kernel's CTAs and slow their chain for
    // nothing (they wait for this kernel's result anyway): there the trigger comes once the reduction has been issued
    // (quantise + GEMM step 9.1 -> 8.5 us at 64 tokens, 11.75 -> 11.67 at 128; GEMM-only loops unchanged).
    if (BN < 64) grid_launch_dependents();
    const uint32_t tmem_base = tmem_slot;
    long long* trace = (ptrace && blockIdx.x < 4) ? ptrace + blockIdx.x * 512 : nullptr;
    if (trace && threadIdx.x == 0) { trace[500] = clock64(); trace[502] = t_entry; trace[503] = t_setup; }
    const uint32_t lo_base = ((smem_base & 0x3FFFF) >> 4) | (1u << 16);

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const uint8_t* sfp = p.w_sf + static_cast<size_t>(tile) * kSfGroupBytes;
        const size_t sfp_stride = static_cast<size_t>(p.w_groups) * kSfGroupBytes;
        const size_t sfq_stride = kSfGroupBytes;  // one token group per stage
        int st = 0, it = 0;
        uint32_t ph = 0;
        bool ok = true;
        // first ring pass: weight tile and weight scales now, the token side after the dependency wait
        const int pre = min(kStages, s_end - s_begin);
        if (elect_one()) {
            for (int i = 0; i < pre; ++i) {
                const int s = s_begin + i;
                const uint32_t full = smem_u32(&bar_full[i]);
                mbar_arrive_expect_tx(full, kFused ? kPTile + kSf : C::kStageBytes);
                const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                const uint32_t sb = smem_base + i * C::kStageBytes;
                tma_load_2d(sb, tm_w, xw, n0, full);
                bulk_load(sb + kPTile + C::kQTile, sfp + s * sfp_stride, kSf, full);
            }
        }
        __syncwarp();
        if (!kFused) grid_dependency_wait();
        for (int s = s_begin; s < s_end; ++s, ++it) {
            if (it >= pre && !mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1, abort_flag)) { ok = false; break; }
            if (trace && lane == 0 && it < 64) trace[it] = clock64();
            if (elect_one()) {
                const uint32_t full = smem_u32(&bar_full[st]);
                const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                const uint32_t sb = smem_base + st * C::kStageBytes;
                if (it >= pre) {
                    mbar_arrive_expect_tx(full, kFused ? kPTile + kSf : C::kStageBytes);
                    tma_load_2d(sb, tm_w, xw, n0, full);
                    bulk_load(sb + kPTile + C::kQTile, sfp + s * sfp_stride, kSf, full);
                }
                if (!kFused) {
                    tma_load_2d(sb + kPTile, tm_act, xa, 0, full);
                    bulk_load(sb + kPTile + C::kQTile + kSf, p.act_sf + s * sfq_stride, kSf, full);
                }
            }
            if (++st == kStages) { st = 0; ph ^= 1; }
        }
        if (!ok && lane == 0) {
            for (int j = max(0, it - kStages); j < it; ++j) {
                const uint32_t bar = smem_u32(&bar_full[j % kStages]);
                const uint32_t php = (j / kStages) & 1;
                for (int tries = 0; tries < (1 << 16) && !mbar_try_wait(bar, php); ++tries) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ tcgen05 issuer
        const bool leader = elect_one();
        const uint32_t d_tmem = tmem_base;
        const uint32_t sf_t = tmem_base + C::kSfCol;
        const uint32_t eb = smem_u32(&bar_empty[0]);
        int st = 0, it = 0;
        uint32_t ph = 0, accumulate = 0;
        bool ok = true;
        bool ready = false;   // the next slot was already seen full by the probe issued one stage earlier
        for (int s = s_begin; s < s_end; ++s, ++it) {
            if (!ready && !mbar_wait(smem_u32(&bar_full[st]), ph, abort_flag)) { ok = false; break; }
            if (trace && lane == 0 && it < 64) trace[64 + it] = clock64();
            const int rem = s < S1 ? p.K - s * kStageK : p.k_tail - (s - S1) * kStageK;
            const int nst = st + 1 == kStages ? 0 : st + 1;
            const uint32_t nph = nst == 0 ? ph ^ 1 : ph;
            ready = mbar_test_wait(smem_u32(&bar_full[nst]), nph);
            if (leader) {
                issue_stage<BN>(lo_base, d_tmem, sf_t, st, rem, accumulate, eb);
            }
            accumulate = 1;
            if (trace && lane == 0 && it < 64) trace[128 + it] = clock64();
            st = nst; ph = nph;
        }
        if (ok && leader) tc_commit(smem_u32(&bar_acc_full));
        if (BN >= 64) grid_launch_dependents();
    } else {
        // ------------------------------------------------------------ epilogue, part 1: accumulator -> registers
        // -> (splits == 1) y, or this CTA's partial tile in shared memory, token-major: partial[t][row]
        const int q4 = warp & 3;
        const int chunk0 = (warp - 2) >> 2;          // which of the quarter's warps this is
        const int row = q4 * 32 + lane;              // weight row inside the tile
        const int n = n0 + row;
        const uint32_t acc_t = tmem_base + (static_cast<uint32_t>(q4 * 32) << 16);
        if constexpr (kFused) {
            static_assert(!kFused || C::kEpiWarps == 4, "the quantiser role is written for four warps");
            // ---- activation quantiser of this CTA: thread = (token, 32-column block) of a stage ----
            const int et = threadIdx.x - 64;
            const int tok0 = et >> 3, blk = et & 7;
            // token-scale atoms of all slots start as zeros (rows past M and the unused atom rows stay so)
            for (int i = 0; i < kStages; ++i)
                *reinterpret_cast<uint2*>(smem + i * C::kStageBytes + kPTile + C::kQTile + kSf + et * 8) = make_uint2(0, 0);
            asm volatile("bar.sync 1, 128;" ::: "memory");
            grid_dependency_wait();   // x is the previous kernel's output
            if (ptrace && blockIdx.x == 0 && threadIdx.x == 64) { unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)); ptrace[2048 + trace_slot_s * 4 + 1] = static_cast<long long>(g); }
            if (trace && et == 0) trace[200] = clock64();
            bool qok = true;
#pragma unroll 1
            for (int base = s_begin; base < s_end && qok; base += kStages) {
                const int n = min(kStages, s_end - base);
                // the loads of all stages of a ring pass are in flight together
                uint4 q[kStages][BN / 16][4];
#pragma unroll
                for (int i = 0; i < kStages; ++i) {
                    const int s = base + i;
                    const int col = (s < S1 ? s * kStageK : p.K - p.k_tail + (s - S1) * kStageK) + blk * kBlock;
#pragma unroll
                    for (int h = 0; h < BN / 16; ++h) {
                        const int tok = tok0 + 16 * h;
                        const bool live = i < n && tok < p.M && col < p.K;
                        const uint16_t* xp = p.x + static_cast<size_t>(tok) * p.ldx + col;
#pragma unroll
                        for (int w4 = 0; w4 < 4; ++w4)
                            q[i][h][w4] = live ? __ldg(reinterpret_cast<const uint4*>(xp + 8 * w4)) : make_uint4(0, 0, 0, 0);
                    }
                }
                const int pass = (base - s_begin) / kStages;
#pragma unroll
                for (int i = 0; i < kStages; ++i) {
                    if (i < n && qok) {
                        // a reused slot must have been drained by the tensor core
                        if (pass > 0 && !mbar_wait(smem_u32(&bar_empty[i]), (pass - 1) & 1, abort_flag)) { qok = false; break; }
                        uint8_t* slot = smem + i * C::kStageBytes;
#pragma unroll
                        for (int h = 0; h < BN / 16; ++h) {
                            const int tok = tok0 + 16 * h;
                            uint4 codes;
                            const uint32_t byte = quant_block32(q[i][h], codes);
                            // token tile: rows of 128 bytes, 16-byte piece c of row r at piece c ^ (r % 8)
                            *reinterpret_cast<uint4*>(slot + kPTile + tok * 128 + ((blk ^ (tok & 7)) << 4)) = codes;
                            if (tok < p.M)
                                slot[kPTile + C::kQTile + kSf + (blk >> 2) * 512 + tok * 16 + (blk & 3)] = static_cast<uint8_t>(byte);
                        }
                        fence_proxy_async_smem();   // the tensor core reads the slot through the async proxy
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_full[i]));
                        if (trace && et == 0 && pass == 0) trace[201 + i] = clock64();
                    }
                }
            }
        } else {
            grid_dependency_wait();   // y may still be read by an earlier kernel
            if (ptrace && blockIdx.x == 0 && threadIdx.x == 64) { unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)); ptrace[2048 + trace_slot_s * 4 + 1] = static_cast<long long>(g); }
        }
        if (mbar_wait(smem_u32(&bar_acc_full), 0, abort_flag)) {
            if (trace && row == 0) trace[192] = clock64();
            tc_fence_after_sync();
            float* partial = reinterpret_cast<float*>(smem);
#pragma unroll 1
            for (int c = chunk0; c < (BN + 15) / 16; c += C::kEpiWarps / 4) {
                uint32_t v[16];
                tmem_ld_32x16(acc_t + c * 16, v);
                tmem_ld_wait();
                if (c * 16 < p.M) {
                    if (splits == 1) {
                        if (n < p.N) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int tok = c * 16 + i;
                                if (tok < p.M) {
                                    if (p.y_bf16)
                                        reinterpret_cast<__nv_bfloat16*>(p.y)[static_cast<size_t>(tok) * p.ldy + n] =
                                            __float2bfloat16_rn(__uint_as_float(v[i]));
                                    else
                                        reinterpret_cast<float*>(p.y)[static_cast<size_t>(tok) * p.ldy + n] = __uint_as_float(v[i]);
                                }
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) partial[(c * 16 + i) * 128 + row] = __uint_as_float(v[i]);
                    }
                }
            }
            if (trace && row == 0) trace[193] = clock64();
        }
        tc_fence_before_sync();
    }

    if (splits > 1) {
        // ------------------------------------------------------------ split-K exchange
        // Token t belongs to CTA t mod splits; its slot there is t / splits.  Every CTA pushes its partial
        // sums (16-byte pieces of 4 weight rows, read back from the token-major tile parked above) into
        // the owners' receive buffers [peer][slot][row]; one cluster barrier later the owner has all of
        // them in its own shared memory.
        const uint32_t recv_base = smem_base + kStages * C::kStageBytes;
        const int slots = (p.M + splits - 1) / splits;        // token slots per peer in a receive buffer
        const int et = threadIdx.x - 64;                        // 0..127 for the epilogue warps
        const int j = et & 31, tq = et >> 5;
        if constexpr (C::kAsyncExchange)
            asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // every peer's bar_recv exists
        if (warp >= 2 && !abort_flag_s) {
            asm volatile("bar.sync 1, %0;" ::"n"(32 * C::kEpiWarps) : "memory");   // the parked tile is complete
            for (int tok = tq; tok < p.M; tok += C::kEpiWarps) {
                const int owner = tok % splits, slot = tok / splits;
                uint4 v;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_base + tok * 512 + j * 16));
                const uint32_t dst = peer_addr(recv_base + ((split * slots + slot) * 128 + 4 * j) * 4, owner);
                if constexpr (C::kAsyncExchange) {
                    const uint32_t rbar = peer_addr(smem_u32(&bar_recv), owner);
                    // asynchronous store into the owner's receive buffer; its bytes are counted on the owner's barrier
                    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                                 ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(rbar) : "memory");
                } else {
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};"
                                 ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                }
            }
            if (trace && et == 0) trace[195] = clock64();
            // the owner's wait: all partial sums of its tokens have arrived (nobody writes to this CTA after that)
            if (C::kAsyncExchange && n_own > 0) mbar_wait(smem_u32(&bar_recv), 0, abort_flag);
        }
        if constexpr (!C::kAsyncExchange) {
            // all threads of all CTAs: orders the pushes before the owners' reads, and nobody leaves before
            // everything addressed to its peers has been delivered
            __syncthreads();
            cluster_sync_all();
        }
        if (warp >= 2 && !abort_flag_s) {
            // this CTA's tokens: split, split + splits, ...; a thread owns 4 consecutive weight rows and
            // every fourth slot; the sum runs in peer order
            const int n = n0 + 4 * j;
            for (int slot = tq; split + slot * splits < p.M; slot += C::kEpiWarps) {
                const int tok = split + slot * splits;
                float4 v[8];
#pragma unroll
                for (int peer = 0; peer < 8; ++peer)
                    if (peer < splits)
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(v[peer].x), "=f"(v[peer].y), "=f"(v[peer].z), "=f"(v[peer].w)
                                     : "r"(recv_base + ((peer * slots + slot) * 128 + 4 * j) * 4));
                float4 sum = v[0];
#pragma unroll
                for (int peer = 1; peer < 8; ++peer)
                    if (peer < splits) { sum.x += v[peer].x; sum.y += v[peer].y; sum.z += v[peer].z; sum.w += v[peer].w; }
                if (n + 3 < p.N) {
                    if (p.y_bf16) {
                        __nv_bfloat162 lo = __floats2bfloat162_rn(sum.x, sum.y), hi = __floats2bfloat162_rn(sum.z, sum.w);
                        uint2 pk = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<size_t>(tok) * p.ldy + n) = pk;
                    } else {
                        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.y) + static_cast<size_t>(tok) * p.ldy + n) = sum;
                    }
                } else {
                    const float e[4] = {sum.x, sum.y, sum.z, sum.w};
                    for (int i = 0; i < 4 && n + i < p.N; ++i) {
                        if (p.y_bf16)
                            reinterpret_cast<__nv_bfloat16*>(p.y)[static_cast<size_t>(tok) * p.ldy + n + i] = __float2bfloat16_rn(e[i]);
                        else
                            reinterpret_cast<float*>(p.y)[static_cast<size_t>(tok) * p.ldy + n + i] = e[i];
                    }
                }
            }
            if (trace && et == 0) trace[194] = clock64();
        }
        // A CTA that gave up pushes nothing and sums nothing, but healthy peers still deliver their partial
        // sums into its receive buffer and count them on its barrier: it stays until they have (bounded), so
        // that no store of a peer reaches the shared memory of a CTA that has left.
        if (C::kAsyncExchange && abort_flag_s && n_own > 0 && threadIdx.x == 64)
            mbar_wait_after_abort(smem_u32(&bar_recv), 0);
    }

    // ------------------------------------------------------------ teardown (normal and aborted)
    tc_fence_before_sync();
    __syncthreads();
    if (trace && threadIdx.x == 0) trace[501] = clock64();
    if (ptrace && blockIdx.x == 0 && threadIdx.x == 64) { unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)); ptrace[2048 + trace_slot_s * 4 + 2] = static_cast<long long>(g); }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

template <int BN, bool kFused, bool kBatch, bool kDense = false>
cudaError_t launch_one(const DecodeMaps& maps, const DecodeBatch& b, cudaStream_t stream) {
    const DecodeBatch& p = b;
    const int n_tiles = b.lay[b.n_lin - 1].tile_end;
    using C = DCfg<BN, kDense>;
    if (kDense && p.splits != 1) return cudaErrorInvalidValue;   // the dense variant has no receive buffer
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(decode_kernel<BN, kFused, kBatch, kDense>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tiles * p.splits);
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, decode_kernel<BN, kFused, kBatch, kDense>, maps, b);
}

// more weight tiles than SMs, no K split, 64 tokens or more: the two-CTAs-per-SM variant
bool wants_dense(int bn, const DecodeBatch& b) {
    if (bn < 64 || b.splits != 1) return false;
    static int sm_count[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (sm_count[dev] == 0 && cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return b.lay[b.n_lin - 1].tile_end > sm_count[dev];
}

template <int BN>
int max_clusters(int splits) {
    using C = DCfg<BN>;
    cudaFuncSetAttribute(decode_kernel<BN, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(splits);
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, decode_kernel<BN, false, false>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

}  // namespace

cudaError_t launch_decode_batch(int bn, const DecodeMaps& maps, const DecodeBatch& b, cudaStream_t stream) {
    if (b.n_lin < 1 || b.n_lin > kMaxBatch) return cudaErrorInvalidValue;
    if (b.x != nullptr)   // fused activation quantiser: one layer, the 16-token tile only
        return (bn == 16 && b.n_lin == 1) ? launch_one<16, true, false>(maps, b, stream) : cudaErrorInvalidValue;
    const bool dense = wants_dense(bn, b);
    if (b.n_lin > 1) {
        switch (bn) {
            case 16: return launch_one<16, false, true>(maps, b, stream);
            case 32: return launch_one<32, false, true>(maps, b, stream);
            case 64: return dense ? launch_one<64, false, true, true>(maps, b, stream) : launch_one<64, false, true>(maps, b, stream);
            default: return dense ? launch_one<128, false, true, true>(maps, b, stream) : launch_one<128, false, true>(maps, b, stream);
        }
    }
    if (dense)
        return bn == 64 ? launch_one<64, false, false, true>(maps, b, stream) : launch_one<128, false, false, true>(maps, b, stream);
    switch (bn) {
        case 16: return launch_one<16, false, false>(maps, b, stream);
        case 32: return launch_one<32, false, false>(maps, b, stream);
        case 64: return launch_one<64, false, false>(maps, b, stream);
        default: return launch_one<128, false, false>(maps, b, stream);
    }
}

cudaError_t launch_decode(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w, const DecodeParams& p,
                          int n_tiles, cudaStream_t stream) {
    DecodeMaps maps;
    std::memset(&maps, 0, sizeof(maps));
    maps.act[0] = tm_act; maps.w[0] = tm_w;
    DecodeBatch b = {};
    b.x = p.x; b.status = p.status; b.trace = p.trace;
    b.M = p.M; b.K = p.K; b.k_tail = p.k_tail; b.ldx = p.ldx;
    b.y_bf16 = p.y_bf16; b.splits = p.splits; b.dbg = p.dbg;
    b.n_lin = 1;
    b.lay[0] = DecodeLayer{p.act_sf, p.w_sf, p.y, p.N, p.w_groups, p.ldy, n_tiles};
    return launch_decode_batch(bn, maps, b, stream);
}

int decode_max_active_clusters(int bn, int splits) {
    switch (bn) {
        case 16: return max_clusters<16>(splits);
        case 32: return max_clusters<32>(splits);
        case 64: return max_clusters<64>(splits);
        default: return max_clusters<128>(splits);
    }
}

}  // namespace prq
