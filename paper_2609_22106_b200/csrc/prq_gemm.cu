// Grouped (MoE) block-scaled FP4 GEMM over the augmented reduction K + k (Eq. (3)), per expert:
//     y[t, n] = sum_b 2^(ea[t,b] + ew[n,b] - 254) * sum_{i<32} a[t, 32 b + i] * w[n, 32 b + i]
// with a = E2M1 codes of [Q(x) | Q(x)_tail] and w = E2M1 codes of [Q(W D P) | Q(R)] of the expert that
// owns token row t (rows sorted by expert, boundaries in expert_offsets).
//
// sm_100a design.  One persistent CTA per SM, 12 warps:
//   warps 0, 2  producers: per 256-element reduction stage, one TMA tile load per operand (128-byte rows,
//           128B swizzle) and one flat bulk copy per operand for the stage's scale bytes, all landing
//           on the stage's "full" mbarrier;
//   warps 1, 3  MMA issuers: copy the stage's scale atoms shared -> tensor memory (tcgen05.cp), then issue
//           up to four K = 64 tcgen05.mma.kind::mxf4.block_scale steps into a tensor-memory accumulator
//           and commit to the stage's "empty" mbarrier; after the last stage commit "accumulator full";
//           (warps 0 + 1 and 2 + 3 are two pairs, each with its own ring of stage slots, scale columns and
//           accumulator, taking alternate units of the CTA)
//   warps 4-11 epilogue: tcgen05.ld of their 32-lane quarter, store to y, release the accumulator.
// A unit is 128 output features x one token tile of an expert: 128 tokens, or 64 when the experts hold few
// tokens each (the smaller tile buys a deeper ring).
// The augmented activation is never materialised: in the residual stages the activation tile is loaded
// again from column K - k while the weight tile continues at column K (the Kernel design paragraph's point
// that the tail is quantised once and used twice); only the tail's scale bytes were duplicated.
//
// Operand roles.  "P" is the operand on the MMA M axis: 128 output features of one expert.  "Q" is the
// operand on the MMA N axis: one token tile of that expert.  With the features on M, the lanes of a
// warp hold consecutive features of one token, stores are contiguous per token, and an expert with few
// tokens costs few stores.  (Dense layers have kernels of their own: prq_gemm_decode.cu for M <= 128,
// prq_gemm_prefill_pair.cu above.)
//
// Every wait is bounded; on expiry the CTA raises an abort flag, all roles unwind, tensor memory is
// freed and PRQ_ERR_TIMEOUT is recorded in the device status word.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "prq_kernels.h"
#include "prq_ptx.cuh"

namespace prq {
namespace {

constexpr int kRings = 2;       // independent (producer, issuer) warp pairs, taking alternate units
constexpr int kMainWarps = 2 * kRings;   // the epilogue warps follow
constexpr int kPTileBytes = 128 * 128;
constexpr int kRowCache = 256;   // experts whose row ranges are cached in shared memory

constexpr int cmin(int a, int b) { return a < b ? a : b; }
constexpr int pow2_at_least(int x) { int p = 32; while (p < x) p *= 2; return p; }

// high words of the shared-memory descriptors: stride between 8-row groups (1024 or 128 bytes, in 16-byte
// units), descriptor version bit, swizzle mode (2 = 128-byte)
constexpr uint32_t kHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kHiPlain = (128u >> 4) | (1u << 14);
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; }

// kFp8: the second format (MXFP8: one byte per element, E4M3).  A stage is still one 128-byte swizzled row per operand
// row, which then holds 128 elements = 4 blocks = ONE scale atom per 128-row group instead of two, and a K = 32 step
// per MMA (kind::mxf8f6f4) that takes one scale byte per row: the scale-id fields walk the four bytes of the word.
// BN: tokens per tile (MMA N), 128 or 64.  The 64-token instance is for launches whose experts hold a handful of
// tokens each (MoE decode): there the kernel is a stream of weight tiles, a CTA's throughput is the bytes its ring
// keeps in flight over the memory latency, and an 8 KB token tile instead of a 16 KB one buys two more ring slots.
// (The scale columns of a tile then start two tensor-memory columns into the group's atom.  A 32-token tile would
// start at odd columns, which the block-scaled MMA does not take: such an instance raised a misaligned-address
// error and was not pursued.)
template <bool kFp8, int BN>
struct Cfg {
    static_assert(BN == 128 || BN == 64, "token tile");
    static constexpr int kStageElems = kFp8 ? 128 : kStageK;
    static constexpr int kSfBytes = kFp8 ? 512 : kSfGroupBytes;    // scale bytes per (stage, 128-row group)
    // eight epilogue warps, two per tensor-memory lane quarter taking half of the tile's tokens each: with
    // K + k = 832 a tile is only 3.25 stages, and the epilogue is what the main loop waits for
    static constexpr int kEpiWarps = 8;
    static constexpr int kWarpTokens = BN / (kEpiWarps / 4);
    static constexpr int kStagingBytes = 1024;   // per epilogue warp
    static constexpr int kThreads = 32 * (kMainWarps + kEpiWarps);
    static constexpr int kQTileBytes = BN * 128;
    static constexpr int kSfpBytes = kSfBytes;
    static constexpr int kSfqBytes = kSfBytes;
    static constexpr int kStageBytes = kPTileBytes + kQTileBytes + kSfpBytes + kSfqBytes;
    // shared memory per CTA: 227 KB less the kernel's static arrays (barriers, per-expert tile and row tables), the
    // alignment slack and the epilogue's staging tiles
    static constexpr int kStaticBytes = 5632 + (BN == 128 ? 0 : 4 * (kMaxExperts + 1));
    static constexpr int kStages = cmin(8, (232448 - kStaticBytes - 1024 - kEpiWarps * kStagingBytes) / kStageBytes) & ~1;
    static constexpr int kRing = kStages / kRings;   // slots of each pair's ring
    // tensor memory columns: two accumulators, then scale words (2 atoms x 4 columns per operand)
    static constexpr int kAccStride = BN;
    static constexpr int kSfpCols = 8, kSfqCols = 8;   // per ring
    static constexpr int kAcc = 2;                     // one accumulator per ring
    static constexpr int kTmemCols = pow2_at_least(kAcc * kAccStride + kRings * (kSfpCols + kSfqCols));
    static constexpr int kSfpCol = kAcc * kAccStride;  // + ring * (kSfpCols + kSfqCols)
    static constexpr int kSfqCol = kSfpCol + kSfpCols;
    static_assert(kAcc == kRings, "every ring accumulates into its own buffer");
    static constexpr uint32_t kTxBytes = kStageBytes;
    static_assert(kRing >= 2, "tile too large for shared memory");
    static_assert(kTmemCols <= 512, "tile too large for tensor memory");
};

struct Unit {
    int p_row, q_row;            // first row of each operand tile in its code tensor
    const uint8_t* sfp;          // stage-0 scale tile of P; advance by sfp_stride per stage
    const uint8_t* sfq;
    size_t sfp_stride, sfq_stride;
    int row0, row_end;           // token rows covered / first row past the valid ones
    int n0;                      // first output feature
};

// Where a unit sits: expert, BN-row token tile (counted over all experts), feature tile.
struct GroupPos { int e, mt, ni; };

// The scale bytes of the activation come in 128-row groups, every expert's rows padded to whole groups
// (group_start[e] = groups before expert e); a BN-row tile is rows [lt * BN, lt * BN + BN) of its expert.
template <int BN>
__device__ __forceinline__ Unit make_unit(const GemmParams& p, const int* tile_start, const int* group_start,
                                           const int* row_start, int S, const GroupPos& g, int sf_bytes) {
    Unit t;
    const int e = g.e, lt = g.mt - tile_start[e], ni = g.ni;
    t.p_row = e * p.N + ni * 128;
    t.q_row = row_start[e] + lt * BN;
    t.sfp = p.w_sf + (static_cast<size_t>(e) * S * p.w_groups + ni) * sf_bytes;
    t.sfp_stride = static_cast<size_t>(p.w_groups) * sf_bytes;
    t.sfq = p.act_sf + static_cast<size_t>(group_start[e] + lt * BN / 128) * sf_bytes;
    t.sfq_stride = static_cast<size_t>(p.act_groups) * sf_bytes;
    t.row0 = t.q_row; t.row_end = min(row_start[e + 1], t.q_row + BN);
    t.n0 = ni * 128;
    return t;
}

// The units of one CTA, in order: a contiguous range of (feature tile, token tile) units, so that stepping to
// the next one is a couple of shared-memory reads (the next token tile, usually of the same expert) instead
// of a division and a search over the experts in every role's critical path; consecutive units of an expert
// also reuse its weight tile from L2.
template <int BN>
struct UnitIter {
    const GemmParams& p;
    const int* tile_start;
    const int* group_start;
    const int* row_start;
    int S, u, u_end, sf_bytes;
    GroupPos g;
    __device__ __forceinline__ UnitIter(const GemmParams& p_, const int* ts, const int* gs, const int* rs, int S_, int n_units,
                                        int sf_bytes_)
        : p(p_), tile_start(ts), group_start(gs), row_start(rs), S(S_), sf_bytes(sf_bytes_), g{0, 0, 0} {
        const int per = (n_units + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
        u = min(n_units, static_cast<int>(blockIdx.x) * per);
        u_end = min(n_units, u + per);
        if (u < u_end) {
            const int total_mt = tile_start[p.n_experts];
            g.mt = u % total_mt; g.ni = u / total_mt;
            int lo = 0, hi = p.n_experts - 1;
            while (lo < hi) {   // last expert whose first tile is <= mt
                const int mid = (lo + hi + 1) >> 1;
                if (tile_start[mid] <= g.mt) lo = mid; else hi = mid - 1;
            }
            g.e = lo;
        }
    }
    __device__ __forceinline__ bool valid() const { return u < u_end; }
    __device__ __forceinline__ Unit get() const { return make_unit<BN>(p, tile_start, group_start, row_start, S, g, sf_bytes); }
    // which BN-row part of its 128-row scale group the current tile is
    __device__ __forceinline__ int sub() const { return (g.mt - tile_start[g.e]) % (128 / BN); }
    __device__ __forceinline__ void next() {
        if (++u < u_end) {
            if (++g.mt == tile_start[p.n_experts]) { g.mt = 0; g.e = 0; ++g.ni; }
            while (tile_start[g.e + 1] <= g.mt) ++g.e;   // experts without rows have no tile: skipped here
        }
    }
};

template <bool kFp8, int BN>
__global__ void __launch_bounds__(Cfg<kFp8, BN>::kThreads, 1)
gemm_grouped_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
                    const GemmParams p) {
    using C = Cfg<kFp8, BN>;
    using Iter = UnitIter<BN>;
    extern __shared__ uint8_t smem_raw[];
    if (kTraceBuild && p.trace && threadIdx.x == 0 && blockIdx.x < 160) {
        unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g));
        p.trace[2048 + blockIdx.x * 4] = static_cast<long long>(g);
    }
    __shared__ __align__(8) uint64_t bar_full[C::kStages], bar_empty[C::kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int tile_start[kMaxExperts + 1];
    __shared__ int group_start_s[BN == 128 ? 1 : kMaxExperts + 1];
    __shared__ int row_cache[kRowCache + 1];
    volatile int* abort_flag = &abort_flag_s;
    const int* row_start = p.n_experts <= kRowCache ? row_cache : p.expert_offsets;
    const int* group_start = BN == 128 ? tile_start : group_start_s;   // with 128-row tiles the two coincide

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // reduction stages: the K main columns, then the k tail columns (MXFP4 only; the second format has no tail)
    const int S1 = (p.K + C::kStageElems - 1) / C::kStageElems;
    const int S = S1 + (kFp8 ? 0 : (p.k_tail + C::kStageElems - 1) / C::kStageElems);

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::kStages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_empty[i]), C::kEpiWarps); }
        abort_flag_s = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_act);
        tma_prefetch_desc(&tm_w);
    }
    // the expert row ranges are kept in shared memory (up to kRowCache experts): every role looks
    // them up once per tile, and a dependent global load there sits on the producer's critical path
    // (no offsets array: a dense layer, i.e. one expert that owns all M rows)
    if (p.n_experts <= kRowCache)
        for (int e = threadIdx.x; e <= p.n_experts; e += blockDim.x)
            row_cache[e] = p.expert_offsets ? p.expert_offsets[e] : (e == 0 ? 0 : p.M);
    __syncthreads();
    // first tile (and first 128-row scale group) of every expert
    if (warp == 2) warp_expert_starts(row_start, p.n_experts, BN, tile_start, BN == 128 ? nullptr : group_start_s);
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    // optional developer trace: SM clock stamps of the first iterations of each role (CTA 0..3 only)
    long long* const ptrace = kTraceBuild ? p.trace : nullptr;
    long long* trace = (ptrace && blockIdx.x < 4) ? ptrace + blockIdx.x * 512 : nullptr;
    if (trace && threadIdx.x == 0) trace[500] = clock64();
    // ... and every CTA's entry, start of work and end on the global timer (ns)
    auto gstamp = [&](int which) {
        if (ptrace && threadIdx.x == 0 && blockIdx.x < 160) {
            unsigned long long g; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g));
            ptrace[2048 + blockIdx.x * 4 + which] = static_cast<long long>(g);
        }
    };
    gstamp(1);
    const int n_units = tile_start[p.n_experts] * ((p.N + 127) / 128);

    // Warps 0..3 are two (producer, issuer) pairs.  Pair r takes the CTA's units r, r + 2, ... through its own ring
    // of kRing stage slots, its own scale columns and accumulator r: what a role spends per stage is mostly the
    // issue cost of its own asynchronous instructions (four copies, or nine tcgen05 instructions), and with few
    // tokens per expert that cost, not the memory system, paced a single pair.
    const int ring = warp >> 1;
    if (warp < kMainWarps && (warp & 1) == 0) {
        // ------------------------------------------------------------ producers
        // The whole warp walks the loop (a lone diverged lane runs this code several times slower);
        // one elected lane arms the barrier and issues the copies.
        int it = 0, st = 0;
        uint32_t ph = 0;
        bool ok = true;
        uint64_t* const full_bars = bar_full + ring * C::kRing;
        uint64_t* const empty_bars = bar_empty + ring * C::kRing;
        Iter ui(p, tile_start, group_start, row_start, S, n_units, C::kSfBytes);
        if (ring == 1) ui.next();
        for (; ui.valid() && ok; ui.next(), ui.next()) {
            const Unit t = ui.get();
            for (int s = 0; s < S; ++s, ++it) {
                if (!mbar_wait(smem_u32(&empty_bars[st]), ph ^ 1, abort_flag)) { ok = false; break; }
                if (trace && ring == 0 && lane == 0 && it < 64) trace[it] = clock64();
                if (elect_one()) {
                    const uint32_t full = smem_u32(&full_bars[st]);
                    mbar_arrive_expect_tx(full, C::kTxBytes);
                    // byte column of each operand in this stage
                    // (a stage is 128 bytes of either format's row; residual stages exist for MXFP4 only)
                    const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                    const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                    const uint32_t sb = smem_base + (ring * C::kRing + st) * C::kStageBytes;
                    tma_load_2d(sb, &tm_w, xw, t.p_row, full);
                    tma_load_2d(sb + kPTileBytes, &tm_act, xa, t.q_row, full);
                    bulk_load(sb + kPTileBytes + C::kQTileBytes, t.sfp + s * t.sfp_stride, C::kSfpBytes, full);
                    bulk_load(sb + kPTileBytes + C::kQTileBytes + C::kSfpBytes, t.sfq + s * t.sfq_stride,
                              C::kSfqBytes, full);
                }
                if (++st == C::kRing) { st = 0; ph ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            // let this ring's copies in flight land before shared memory is given up (bounded)
            for (int j = max(0, it - C::kRing); j < it; ++j) {
                const uint32_t bar = smem_u32(&full_bars[j % C::kRing]);
                const uint32_t ph = (j / C::kRing) & 1;
                for (int tries = 0; tries < (1 << 16) && !mbar_try_wait(bar, ph); ++tries) {}
            }
        }
    } else if (warp < kMainWarps) {
        // ------------------------------------------------------------ MMA issuers
        // The whole warp walks the loop and waits on the barriers; one elected lane issues the
        // tensor-core instructions (and therefore also the commits that track them).
        int it = 0, acc_it = 0, st = 0;   // acc_it counts this ring's units
        uint32_t ph = 0;
        bool ok = true;
        bool ready = false;   // the next slot was already seen full by the probe issued one stage earlier
        const bool leader = elect_one();
        uint64_t* const full_bars = bar_full + ring * C::kRing;
        uint64_t* const empty_bars = bar_empty + ring * C::kRing;
        const uint32_t sfp_t = tmem_base + C::kSfpCol + ring * (C::kSfpCols + C::kSfqCols);
        const uint32_t sfq_t = tmem_base + C::kSfqCol + ring * (C::kSfpCols + C::kSfqCols);
        const uint32_t lo_base = (((smem_base + ring * C::kRing * C::kStageBytes) & 0x3FFFF) >> 4) | (1u << 16);
        const int buf = ring;
        Iter ui(p, tile_start, group_start, row_start, S, n_units, C::kSfBytes);
        if (ring == 1) ui.next();
        for (; ui.valid() && ok; ui.next(), ui.next(), ++acc_it) {
            const uint32_t acc_ph = acc_it & 1;
            if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), acc_ph ^ 1, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + buf * C::kAccStride;
            // a scale atom holds the bytes of all 128 rows of the group: row r in lane r % 32 of column r / 32, so
            // a BN-row tile's scales start BN / 32 columns further per tile
            const uint32_t sfq_u = sfq_t + ui.sub() * (BN / 32);
            uint32_t accumulate = 0;
            for (int s = 0; s < S; ++s, ++it) {
                if (!ready && !mbar_wait(smem_u32(&full_bars[st]), ph, abort_flag)) { ok = false; break; }
                if (trace && ring == 0 && lane == 0 && it < 64) trace[64 + it] = clock64();
                const int rem = s < S1 ? p.K - s * C::kStageElems : p.k_tail - (s - S1) * C::kStageElems;
                const int ksteps = min(4, (rem + C::kStageElems / 4 - 1) / (C::kStageElems / 4));
                // probe the next slot now: the probe's latency hides behind this stage's tcgen05 instructions
                const int nst = st + 1 == C::kRing ? 0 : st + 1;
                const uint32_t nph = nst == 0 ? ph ^ 1 : ph;
                ready = mbar_test_wait(smem_u32(&full_bars[nst]), nph);
                if (leader) {
                    // Descriptors as (constant high word, 32-bit low word): the low word is the shared
                    // address in 16-byte units plus the leading-dimension field, so a stage's descriptors
                    // cost one add each instead of a 64-bit shift-and-or chain.
                    const uint32_t plo = lo_base + st * (C::kStageBytes >> 4);
                    const uint32_t qlo = plo + (kPTileBytes >> 4);
                    const uint32_t sfp_lo = qlo + (C::kQTileBytes >> 4), sfq_lo = sfp_lo + (C::kSfpBytes >> 4);
                    if constexpr (kFp8) {
                        // one atom per operand covers the stage's four blocks; step j takes byte j of the scale word
                        tc_copy_sf_atom(sfp_t, desc64(kHiPlain, sfp_lo));
                        tc_copy_sf_atom(sfq_t, desc64(kHiPlain, sfq_lo));
                        // E4M3 x E4M3 (format 0), E8M0 scales, both operands K-major, N = BN, M = 128
                        constexpr uint32_t idesc = ((BN >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (j < ksteps) {
                                tc_mma_mxf8(d_tmem, desc64(kHiSw128, plo + 2 * j), desc64(kHiSw128, qlo + 2 * j),
                                            idesc | (static_cast<uint32_t>(j) << 4) | (static_cast<uint32_t>(j) << 29), sfp_t, sfq_u, accumulate);
                                accumulate = 1;
                            }
                        }
                    } else {
#pragma unroll
                        for (int ka = 0; ka < 2; ++ka) {
                            if (ka * 2 < ksteps) {
                                tc_copy_sf_atom(sfp_t + ka * 4, desc64(kHiPlain, sfp_lo + ka * (512 >> 4)));
                                tc_copy_sf_atom(sfq_t + ka * 4, desc64(kHiPlain, sfq_lo + ka * (512 >> 4)));
                            }
                        }
                        constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
                        constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (j < ksteps) {
                                tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 2 * j), desc64(kHiSw128, qlo + 2 * j),
                                            (j & 1) ? idesc2 : idesc0, sfp_t + (j >> 1) * 4, sfq_u + (j >> 1) * 4, accumulate);
                                accumulate = 1;
                            }
                        }
                    }
                    tc_commit(smem_u32(&empty_bars[st]));
                }
                accumulate = 1;
                if (trace && ring == 0 && lane == 0 && it < 64) trace[128 + it] = clock64();
                st = nst; ph = nph;
            }
            if (!ok) break;
            if (leader) tc_commit(smem_u32(&bar_acc_full[buf]));
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------ epilogue (the warps after the two pairs)
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may read
        const int et = q * 32 + lane;           // 0..127: accumulator row
        int acc_it = 0;
        bool ok = true;
        for (Iter ui(p, tile_start, group_start, row_start, S, n_units, C::kSfBytes); ui.valid() && ok; ui.next(), ++acc_it) {
            const Unit t = ui.get();
            const int buf = acc_it % C::kAcc;
            const uint32_t acc_ph = (acc_it / C::kAcc) & 1;
            if (!mbar_wait(smem_u32(&bar_acc_full[buf]), acc_ph, abort_flag)) { ok = false; break; }
            if (trace && et == 0 && acc_it < 8) trace[192 + 2 * acc_it] = clock64();
            tc_fence_after_sync();
            const uint32_t acc_t = tmem_base + buf * C::kAccStride + (static_cast<uint32_t>(q * 32) << 16);
            // accumulator row = output feature n, column = token of this tile.  A warp takes 64 tokens of its
            // lane quarter (the two warps of a quarter take one half of a 128-token tile each): it reads all of
            // them into registers and hands the accumulator back to the issuer at once, so that the next tile
            // of this ring accumulates while the stores below run.  Sixteen tokens at a time, the warp then
            // parks its 32 features per token in a small shared tile (one contiguous row per token) and writes
            // the rows out in 16-byte pieces: 64 (bf16) or 128 (fp32) contiguous bytes per token and warp.  A
            // tile with few tokens costs few reads and few stores.
            const int n_tok = t.row_end - t.row0;
            const int nw = t.n0 + q * 32;                   // first feature of this warp
            const uint32_t stg = smem_base + C::kStages * C::kStageBytes + (warp - kMainWarps) * C::kStagingBytes;
            constexpr int kTW = C::kWarpTokens;
            const int tok0 = ((warp - kMainWarps) >> 2) * kTW;   // first token of this warp
            uint32_t r[kTW];
#pragma unroll
            for (int l = 0; l < kTW / 32; ++l)
                if (tok0 + l * 32 < n_tok) tmem_ld_32x32(acc_t + tok0 + l * 32, *reinterpret_cast<uint32_t (*)[32]>(&r[l * 32]));
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
            if (p.y_bf16) {
                // 16 tokens x 32 features x 2 bytes fill the warp's 1 KB staging tile
#pragma unroll
                for (int cc = 0; cc < kTW / 16; ++cc) {
                    const int c0 = tok0 + cc * 16;              // first token of the chunk
                    if (c0 >= n_tok) break;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const __nv_bfloat16 h = __float2bfloat16_rn(__uint_as_float(r[cc * 16 + i]));
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(stg + i * 64 + lane * 2), "h"(*reinterpret_cast<const uint16_t*>(&h)) : "memory");
                    }
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int tok = c0 + j * 8 + (lane >> 2), col = nw + (lane & 3) * 8;
                        uint4 v;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stg + j * 512 + lane * 16));
                        if (tok < n_tok && col < p.N) {
                            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<size_t>(t.row0 + tok) * p.ldy + col;
                            if (col + 8 <= p.N) *reinterpret_cast<uint4*>(yp) = v;
                            else {
                                const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
                                for (int i = 0; i < 8 && col + i < p.N; ++i) yp[i] = e[i];
                            }
                        }
                    }
                    __syncwarp();   // the tile is read before the next chunk overwrites it
                }
            } else {
                // 8 tokens x 32 features x 4 bytes
#pragma unroll
                for (int cc = 0; cc < kTW / 8; ++cc) {
                    const int c0 = tok0 + cc * 8;
                    if (c0 >= n_tok) break;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + i * 128 + lane * 4), "r"(r[cc * 8 + i]) : "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int tok = c0 + j * 4 + (lane >> 3), col = nw + (lane & 7) * 4;
                        uint4 v;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stg + j * 512 + lane * 16));
                        if (tok < n_tok && col < p.N) {
                            float* yp = reinterpret_cast<float*>(p.y) + static_cast<size_t>(t.row0 + tok) * p.ldy + col;
                            if (col + 4 <= p.N) *reinterpret_cast<uint4*>(yp) = v;
                            else {
                                const float* e = reinterpret_cast<const float*>(&v);
                                for (int i = 0; i < 4 && col + i < p.N; ++i) yp[i] = e[i];
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            if (trace && et == 0 && acc_it < 8) trace[193 + 2 * acc_it] = clock64();
        }
    }

    // ------------------------------------------------------------ teardown (normal and aborted)
    tc_fence_before_sync();
    __syncthreads();
    if (trace && threadIdx.x == 0) trace[501] = clock64();
    gstamp(2);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}


template <bool kFp8, int BN>
cudaError_t launch_grouped_impl(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                                cudaStream_t stream) {
    using C = Cfg<kFp8, BN>;
    constexpr int smem = C::kStages * C::kStageBytes + 1024 + C::kEpiWarps * C::kStagingBytes;  // + store staging
    static bool configured = false;  // the attribute is per function, setting it twice is harmless
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_grouped_kernel<kFp8, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    gemm_grouped_kernel<kFp8, BN><<<grid, C::kThreads, smem, stream>>>(tm_act, tm_w, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm_grouped(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                                cudaStream_t stream) {
    if (bn == 64) return launch_grouped_impl<false, 64>(tm_act, tm_w, p, grid, stream);
    if (bn != 128) return cudaErrorInvalidValue;
    return launch_grouped_impl<false, 128>(tm_act, tm_w, p, grid, stream);
}

cudaError_t launch_gemm_fp8(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                            cudaStream_t stream) {
    return launch_grouped_impl<true, 128>(tm_act, tm_w, p, grid, stream);
}

}  // namespace prq
