// Block-scaled FP4 GEMM over the augmented reduction K + k (Eq. (3)):
//     y[t, n] = sum_b 2^(ea[t,b] + ew[n,b] - 254) * sum_{i<32} a[t, 32 b + i] * w[n, 32 b + i]
// with a = E2M1 codes of [Q(x) | Q(x)_tail] and w = E2M1 codes of [Q(W D P) | Q(R)].
//
// sm_100a design.  One CTA per SM, 6 warps:
//   warp 0  producer: per 256-element reduction stage, one TMA tile load per operand (128-byte rows,
//           128B swizzle) and one flat bulk copy per operand for the stage's scale bytes, all landing
//           on the stage's "full" mbarrier;
//   warp 1  MMA issuer: copies the stage's scale atoms shared -> tensor memory (tcgen05.cp), then issues
//           up to four K = 64 tcgen05.mma.kind::mxf4.block_scale steps into a tensor-memory accumulator
//           and commits to the stage's "empty" mbarrier; after the last stage commits "accumulator full";
//   warps 2-5 epilogue: tcgen05.ld of their 32-lane quarter, store to y, release the accumulator.
// The augmented activation is never materialised: in the residual stages the activation tile is loaded
// again from column K - k while the weight tile continues at column K ("reuses the quantized
// representation of the tail", Kernel design paragraph); only the tail's scale bytes were duplicated.
//
// Operand roles.  "P" is the operand on the MMA M axis (always 128 rows), "Q" the operand on the MMA N
// axis (BN rows).  Dense and grouped kinds: P = activation tokens, Q = weight rows.  Swapped grouped kind
// (the default for stacked experts): P = 128 output features of one expert, Q = one 128-token group of
// that expert, so that an expert with few tokens costs few stores.  (M <= 128 and the large dense shapes
// have kernels of their own: prq_gemm_decode.cu, prq_gemm_prefill_pair.cu; this one serves the grouped
// product and, behind a developer switch, dense prefill with one CTA per tile.)
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

constexpr int kMainWarps = 2;   // producer + issuer; the epilogue warps follow
constexpr int kPTileBytes = 128 * 128;
constexpr int kKindPrefill = 0, kKindGrouped = 2, kKindGroupedSwap = 3;
constexpr int kRowCache = 256;   // experts whose row ranges are cached in shared memory

constexpr int cgcd(int a, int b) { return b == 0 ? a : cgcd(b, a % b); }
constexpr int cmin(int a, int b) { return a < b ? a : b; }
constexpr int cmax(int a, int b) { return a > b ? a : b; }
constexpr int pow2_at_least(int x) { int p = 32; while (p < x) p *= 2; return p; }

// high words of the shared-memory descriptors: stride between 8-row groups (1024 or 128 bytes, in 16-byte
// units), descriptor version bit, swizzle mode (2 = 128-byte)
constexpr uint32_t kHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kHiPlain = (128u >> 4) | (1u << 14);
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; }

template <int BN, int KIND>
struct Cfg {
    static constexpr bool kSwap = KIND == kKindGroupedSwap;
    // epilogue warps: four (one per tensor-memory lane quarter), or eight taking alternate column chunks
    // where the epilogue is what the main loop waits for (short reductions, many outputs)
    static constexpr int kEpiWarps = KIND == kKindGroupedSwap ? 8 : 4;
    static constexpr int kThreads = 32 * (kMainWarps + kEpiWarps);
    // 128-row scale groups of a Q tile; the weight scale buffer is laid out per BN-row tile, so a
    // tile's groups are contiguous and start at the tile's first row
    static constexpr int kNgq = (BN + 127) / 128;
    static constexpr int kQTileBytes = BN * 128;
    static constexpr int kSfpBytes = kSfGroupBytes;
    static constexpr int kSfqBytes = kNgq * kSfGroupBytes;
    static constexpr int kStageBytes = kPTileBytes + kQTileBytes + kSfpBytes + kSfqBytes;
    static constexpr int kStages = cmin(8, (232448 - 1024 - 16384 - 2048) / kStageBytes);
    // tensor memory columns: accumulators first, then scale words
    static constexpr int kAccStride = cmax(BN, 32);
    static constexpr int kSfpCols = 8;              // 2 atoms x 4 columns
    static constexpr int kSfqCols = 8 * kNgq;       // 2 atoms x 4 columns x groups
    static constexpr int kSfCols = kSfpCols + kSfqCols;
    static constexpr int kAcc = 2 * kAccStride + kSfCols <= 512 ? 2 : 1;
    static constexpr int kTmemCols = pow2_at_least(kAcc * kAccStride + kSfCols);
    static constexpr int kSfpCol = kAcc * kAccStride;
    static constexpr int kSfqCol = kSfpCol + kSfpCols;
    static constexpr uint32_t kTxBytes = kStageBytes;
    static_assert(kStages >= 2, "tile too large for shared memory");
    static_assert(kTmemCols <= 512, "tile too large for tensor memory");
    static_assert(BN % 16 == 0 && BN >= 16 && BN <= 256, "MMA N must be a multiple of 16 in [16, 256]");
};

struct Unit {
    int p_row, q_row;            // first row of each operand tile in its code tensor
    const uint8_t* sfp;          // stage-0 scale tile of P; advance by sfp_stride per stage
    const uint8_t* sfq;
    size_t sfp_stride, sfq_stride;
    int s_begin, s_end;          // reduction stages of this unit
    int row0, row_end;           // token rows covered / first row past the valid ones
    int n0;                      // first output feature
};

// Where a grouped unit sits: expert, 128-row token tile (counted over all experts), feature tile.
struct GroupPos { int e, mt, ni; };

template <int BN, int KIND>
__device__ __forceinline__ int unit_count(const GemmParams& p, const int* tile_start) {
    if (KIND == kKindPrefill) return ((p.M + 127) / 128) * ((p.N + BN - 1) / BN);
    if (KIND == kKindGroupedSwap) return tile_start[p.n_experts] * ((p.N + 127) / 128);
    return tile_start[p.n_experts] * ((p.N + BN - 1) / BN);
}

template <int BN, int KIND>
__device__ __forceinline__ Unit make_unit(const GemmParams& p, const int* tile_start, const int* row_start, int u, int S,
                                           const GroupPos& g) {
    Unit t;
    if (KIND == kKindPrefill) {
        const int m_tiles = (p.M + 127) / 128;
        const int mi = u % m_tiles, ni = u / m_tiles;
        t.p_row = mi * 128;
        t.q_row = ni * BN;
        t.sfp = p.act_sf + static_cast<size_t>(mi) * kSfGroupBytes;
        t.sfp_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;
        t.sfq = p.w_sf + static_cast<size_t>(ni) * Cfg<BN, KIND>::kNgq * kSfGroupBytes;
        t.sfq_stride = static_cast<size_t>(p.w_groups) * kSfGroupBytes;
        t.s_begin = 0; t.s_end = S;
        t.row0 = mi * 128; t.row_end = min(p.M, t.row0 + 128);
        t.n0 = ni * BN;
    } else if (KIND == kKindGroupedSwap) {
        // weights on the MMA M axis (128 output features), a 128-row group of one expert's tokens on N
        const int e = g.e, mt = g.mt, ni = g.ni;
        t.p_row = e * p.N + ni * 128;
        t.q_row = row_start[e] + (mt - tile_start[e]) * 128;
        t.sfp = p.w_sf + (static_cast<size_t>(e) * S * p.w_groups + ni) * kSfGroupBytes;
        t.sfp_stride = static_cast<size_t>(p.w_groups) * kSfGroupBytes;
        t.sfq = p.act_sf + static_cast<size_t>(mt) * kSfGroupBytes;
        t.sfq_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;
        t.s_begin = 0; t.s_end = S;
        t.row0 = t.q_row; t.row_end = min(row_start[e + 1], t.q_row + 128);
        t.n0 = ni * 128;
    } else {
        const int e = g.e, mt = g.mt, ni = g.ni;
        t.p_row = row_start[e] + (mt - tile_start[e]) * 128;
        t.q_row = e * p.N + ni * BN;
        t.sfp = p.act_sf + static_cast<size_t>(mt) * kSfGroupBytes;
        t.sfp_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;
        t.sfq = p.w_sf + (static_cast<size_t>(e) * S * p.w_groups + static_cast<size_t>(ni) * Cfg<BN, KIND>::kNgq) * kSfGroupBytes;
        t.sfq_stride = static_cast<size_t>(p.w_groups) * kSfGroupBytes;
        t.s_begin = 0; t.s_end = S;
        t.row0 = t.p_row; t.row_end = min(row_start[e + 1], t.p_row + 128);
        t.n0 = ni * BN;
    }
    return t;
}

// The units of one CTA, in order.  Dense kinds: u = blockIdx.x, + gridDim.x, ...  Grouped kinds: a
// contiguous range of units, so that stepping to the next one is a couple of shared-memory reads (the
// next token tile, usually of the same expert) instead of a division and a search over the experts in
// every role's critical path; consecutive units of an expert also reuse its weight tile from L2.
template <int BN, int KIND>
struct UnitIter {
    static constexpr bool kGroupedKind = KIND == kKindGrouped || KIND == kKindGroupedSwap;
    const GemmParams& p;
    const int* tile_start;
    const int* row_start;
    int S, u, u_end, step;
    GroupPos g;
    __device__ __forceinline__ UnitIter(const GemmParams& p_, const int* ts, const int* rs, int S_, int n_units)
        : p(p_), tile_start(ts), row_start(rs), S(S_), g{0, 0, 0} {
        if (kGroupedKind) {
            const int per = (n_units + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
            u = min(n_units, static_cast<int>(blockIdx.x) * per);
            u_end = min(n_units, u + per);
            step = 1;
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
        } else {
            u = blockIdx.x; u_end = n_units; step = gridDim.x;
        }
    }
    __device__ __forceinline__ bool valid() const { return u < u_end; }
    __device__ __forceinline__ Unit get() const { return make_unit<BN, KIND>(p, tile_start, row_start, u, S, g); }
    __device__ __forceinline__ void next() {
        u += step;
        if (kGroupedKind && u < u_end) {
            if (++g.mt == tile_start[p.n_experts]) { g.mt = 0; g.e = 0; ++g.ni; }
            while (tile_start[g.e + 1] <= g.mt) ++g.e;   // experts without rows have no tile: skipped here
        }
    }
};

template <int BN, int KIND>
__global__ void __launch_bounds__(Cfg<BN, KIND>::kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
            const GemmParams p) {
    using C = Cfg<BN, KIND>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[C::kStages], bar_empty[C::kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag_s;
    __shared__ int tile_start[(KIND == kKindGrouped || KIND == kKindGroupedSwap) ? kMaxExperts + 1 : 1];
    __shared__ int row_cache[(KIND == kKindGrouped || KIND == kKindGroupedSwap) ? kRowCache + 1 : 1];
    volatile int* abort_flag = &abort_flag_s;
    const int* row_start = ((KIND == kKindGrouped || KIND == kKindGroupedSwap) && p.n_experts <= kRowCache)
                               ? row_cache : p.expert_offsets;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const StagePlan plan(p.K, p.k_tail);
    const int S = plan.S, S1 = plan.S1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::kStages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_empty[i]), C::kEpiWarps); }
        abort_flag_s = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_act);
        tma_prefetch_desc(&tm_w);
    }
    if (KIND == kKindGrouped || KIND == kKindGroupedSwap) {
        // the expert row ranges are kept in shared memory (up to kRowCache experts): every role looks
        // them up once per tile, and a dependent global load there sits on the producer's critical path
        if (p.n_experts <= kRowCache)
            for (int e = threadIdx.x; e <= p.n_experts; e += blockDim.x) row_cache[e] = p.expert_offsets[e];
        __syncthreads();
        if (threadIdx.x == 64) {
            int acc = 0;
            for (int e = 0; e < p.n_experts; ++e) {
                tile_start[e] = acc;
                acc += (row_start[e + 1] - row_start[e] + 127) / 128;
            }
            tile_start[p.n_experts] = acc;
        }
    }
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
    const int n_units = unit_count<BN, KIND>(p, tile_start);

    const CUtensorMap* tm_p = C::kSwap ? &tm_w : &tm_act;
    const CUtensorMap* tm_q = C::kSwap ? &tm_act : &tm_w;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // The whole warp walks the loop (a lone diverged lane runs this code several times slower);
        // one elected lane arms the barrier and issues the copies.
        int it = 0, st = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (UnitIter<BN, KIND> ui(p, tile_start, row_start, S, n_units); ui.valid() && ok; ui.next()) {
            const Unit t = ui.get();
            for (int s = t.s_begin; s < t.s_end; ++s, ++it) {
                if (!mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1, abort_flag)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[it] = clock64();
                if (elect_one()) {
                    const uint32_t full = smem_u32(&bar_full[st]);
                    mbar_arrive_expect_tx(full, C::kTxBytes);
                    // byte column of each operand in this stage
                    const int xw = s < S1 ? s * 128 : p.K / 2 + (s - S1) * 128;
                    const int xa = s < S1 ? s * 128 : (p.K - p.k_tail) / 2 + (s - S1) * 128;
                    const uint32_t sb = smem_base + st * C::kStageBytes;
                    tma_load_2d(sb, tm_p, C::kSwap ? xw : xa, t.p_row, full);
                    tma_load_2d(sb + kPTileBytes, tm_q, C::kSwap ? xa : xw, t.q_row, full);
                    bulk_load(sb + kPTileBytes + C::kQTileBytes, t.sfp + s * t.sfp_stride, C::kSfpBytes, full);
                    bulk_load(sb + kPTileBytes + C::kQTileBytes + C::kSfpBytes, t.sfq + s * t.sfq_stride,
                              C::kSfqBytes, full);
                }
                if (++st == C::kStages) { st = 0; ph ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            // let this CTA's copies in flight land before shared memory is given up (bounded)
            for (int j = max(0, it - C::kStages); j < it; ++j) {
                const uint32_t bar = smem_u32(&bar_full[j % C::kStages]);
                const uint32_t ph = (j / C::kStages) & 1;
                for (int tries = 0; tries < (1 << 16) && !mbar_try_wait(bar, ph); ++tries) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop and waits on the barriers; one elected lane issues the
        // tensor-core instructions (and therefore also the commits that track them).
        int it = 0, acc_it = 0, st = 0;
        uint32_t ph = 0;
        bool ok = true;
        bool ready = false;   // the next slot was already seen full by the probe issued one stage earlier
        const bool leader = elect_one();
        const uint32_t sfp_t = tmem_base + C::kSfpCol;
        const uint32_t sfq_t = tmem_base + C::kSfqCol;
        const uint32_t lo_base = ((smem_base & 0x3FFFF) >> 4) | (1u << 16);
        for (UnitIter<BN, KIND> ui(p, tile_start, row_start, S, n_units); ui.valid() && ok; ui.next(), ++acc_it) {
            const Unit t = ui.get();
            const int buf = acc_it % C::kAcc;
            const uint32_t acc_ph = (acc_it / C::kAcc) & 1;
            if (!mbar_wait(smem_u32(&bar_acc_empty[buf]), acc_ph ^ 1, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + buf * C::kAccStride;
            uint32_t accumulate = 0;
            for (int s = t.s_begin; s < t.s_end; ++s, ++it) {
                if (!ready && !mbar_wait(smem_u32(&bar_full[st]), ph, abort_flag)) { ok = false; break; }
                if (trace && lane == 0 && it < 64) trace[64 + it] = clock64();
                const int rem = s < S1 ? p.K - s * kStageK : p.k_tail - (s - S1) * kStageK;
                const int ksteps = min(4, (rem + 63) / 64);
                // probe the next slot now: the probe's latency hides behind this stage's tcgen05 instructions
                const int nst = st + 1 == C::kStages ? 0 : st + 1;
                const uint32_t nph = nst == 0 ? ph ^ 1 : ph;
                ready = mbar_test_wait(smem_u32(&bar_full[nst]), nph);
                if (leader) {
                    // Descriptors as (constant high word, 32-bit low word): the low word is the shared
                    // address in 16-byte units plus the leading-dimension field, so a stage's descriptors
                    // cost one add each instead of a 64-bit shift-and-or chain.
                    const uint32_t plo = lo_base + st * (C::kStageBytes >> 4);
                    const uint32_t qlo = plo + (kPTileBytes >> 4);
                    const uint32_t sfp_lo = qlo + (C::kQTileBytes >> 4), sfq_lo = sfp_lo + (C::kSfpBytes >> 4);
#pragma unroll
                    for (int ka = 0; ka < 2; ++ka) {
                        if (ka * 2 < ksteps && !(kTraceBuild && (p.dbg & 1))) {
                            tc_copy_sf_atom(sfp_t + ka * 4, desc64(kHiPlain, sfp_lo + ka * (512 >> 4)));
#pragma unroll
                            for (int g = 0; g < C::kNgq; ++g)
                                tc_copy_sf_atom(sfq_t + ka * 4 * C::kNgq + g * 4,
                                                desc64(kHiPlain, sfq_lo + g * (kSfGroupBytes >> 4) + ka * (512 >> 4)));
                        }
                    }
                    constexpr uint32_t idesc0 = (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
                    constexpr uint32_t idesc2 = idesc0 | (2u << 4) | (2u << 29);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (j < ksteps && !(kTraceBuild && (p.dbg & 2))) {
                            tc_mma_mxf4(d_tmem, desc64(kHiSw128, plo + 2 * j), desc64(kHiSw128, qlo + 2 * j),
                                        (j & 1) ? idesc2 : idesc0, sfp_t + (j >> 1) * 4,
                                        sfq_t + (j >> 1) * 4 * C::kNgq, accumulate);
                            accumulate = 1;
                        }
                    }
                    tc_commit(smem_u32(&bar_empty[st]));
                }
                accumulate = 1;
                if (trace && lane == 0 && it < 64) trace[128 + it] = clock64();
                st = nst; ph = nph;
            }
            if (!ok) break;
            if (leader) tc_commit(smem_u32(&bar_acc_full[buf]));
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may read
        const int et = q * 32 + lane;           // 0..127: accumulator row
        int acc_it = 0;
        bool ok = true;
        for (UnitIter<BN, KIND> ui(p, tile_start, row_start, S, n_units); ui.valid() && ok; ui.next(), ++acc_it) {
            const Unit t = ui.get();
            const int buf = acc_it % C::kAcc;
            const uint32_t acc_ph = (acc_it / C::kAcc) & 1;
            if (!mbar_wait(smem_u32(&bar_acc_full[buf]), acc_ph, abort_flag)) { ok = false; break; }
            if (trace && et == 0 && acc_it < 8) trace[192 + 2 * acc_it] = clock64();
            tc_fence_after_sync();
            const uint32_t acc_t = tmem_base + buf * C::kAccStride + (static_cast<uint32_t>(q * 32) << 16);
            if (!C::kSwap) {
                const int row = t.row0 + et;
                const bool row_ok = row < t.row_end;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(acc_t + c * 32, r);
                    tmem_ld_wait();
                    const int col = t.n0 + c * 32;
                    if (row_ok && col < p.N) {
                        if (p.y_bf16) {
                            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<size_t>(row) * p.ldy + col;
                            if (col + 32 <= p.N) {
#pragma unroll
                                for (int i = 0; i < 32; i += 8) {
                                    uint4 v;
                                    __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                                    __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                                    __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
                                    __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
                                    v.x = *reinterpret_cast<uint32_t*>(&h0); v.y = *reinterpret_cast<uint32_t*>(&h1);
                                    v.z = *reinterpret_cast<uint32_t*>(&h2); v.w = *reinterpret_cast<uint32_t*>(&h3);
                                    *reinterpret_cast<uint4*>(yp + i) = v;
                                }
                            } else {
                                for (int i = 0; i < 32 && col + i < p.N; ++i) yp[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
                            }
                        } else {
                            float* yp = reinterpret_cast<float*>(p.y) + static_cast<size_t>(row) * p.ldy + col;
                            if (col + 32 <= p.N) {
#pragma unroll
                                for (int i = 0; i < 32; i += 4)
                                    *reinterpret_cast<uint4*>(yp + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
                            } else {
                                for (int i = 0; i < 32 && col + i < p.N; ++i) yp[i] = __uint_as_float(r[i]);
                            }
                        }
                    }
                }
            } else if (KIND == kKindGroupedSwap) {
                // accumulator row = output feature n, column = token of this expert's 128-row group.  Sixteen
                // tokens at a time, every warp parks its 32 features per token in a small shared tile (one
                // contiguous row per token) and writes the rows out in 16-byte pieces: 64 (bf16) or 128 (fp32)
                // contiguous bytes per token and warp.  A group with few tokens costs few stores.
                const int n_tok = t.row_end - t.row0;
                const int nw = t.n0 + q * 32;                   // first feature of this warp
                const uint32_t stg = smem_base + C::kStages * C::kStageBytes + (warp - kMainWarps) * 2048;
                constexpr int kPerQuarter = C::kEpiWarps / 4;   // warps sharing a lane quarter take alternate chunks
#pragma unroll 1
                for (int c = (warp - kMainWarps) >> 2; c * 16 < n_tok; c += kPerQuarter) {
                    uint32_t r[16];
                    tmem_ld_32x16(acc_t + c * 16, r);
                    tmem_ld_wait();
                    if (p.y_bf16) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const __nv_bfloat16 h = __float2bfloat16_rn(__uint_as_float(r[i]));
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(stg + i * 64 + lane * 2), "h"(*reinterpret_cast<const uint16_t*>(&h)) : "memory");
                        }
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const int tok = c * 16 + j * 8 + (lane >> 2), col = nw + (lane & 3) * 8;
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
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + i * 128 + lane * 4), "r"(r[i]) : "memory");
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int tok = c * 16 + j * 4 + (lane >> 3), col = nw + (lane & 7) * 4;
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
                    }
                    __syncwarp();   // the tile is read before the next chunk overwrites it
                }
            }
            // hand the accumulator back to the MMA issuer
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
            if (trace && et == 0 && acc_it < 8) trace[193 + 2 * acc_it] = clock64();
        }
    }

    // ------------------------------------------------------------ teardown (normal and aborted)
    tc_fence_before_sync();
    __syncthreads();
    if (trace && threadIdx.x == 0) trace[501] = clock64();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, static_cast<int>(PRQ_ERR_TIMEOUT));
}

template <int BN, int KIND>
cudaError_t launch_one(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                       cudaStream_t stream) {
    using C = Cfg<BN, KIND>;
    constexpr int smem = C::kStages * C::kStageBytes + 1024 + (KIND == kKindGroupedSwap ? C::kEpiWarps * 2048 : 0);  // + store staging
    static bool configured = false;  // per template instance; the attribute is per function, setting it twice is harmless
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<BN, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    gemm_kernel<BN, KIND><<<grid, C::kThreads, smem, stream>>>(tm_act, tm_w, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm(GemmKind kind, int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w,
                        const GemmParams& p, int grid, cudaStream_t stream, bool* unsupported) {
    *unsupported = false;
#define PRQ_CASE(KINDV, BNV) \
    if (bn == BNV) return launch_one<BNV, KINDV>(tm_act, tm_w, p, grid, stream);
    if (kind == GemmKind::kPrefill) {
        PRQ_CASE(kKindPrefill, 128)
        PRQ_CASE(kKindPrefill, 160)
        PRQ_CASE(kKindPrefill, 192)
        PRQ_CASE(kKindPrefill, 256)
    } else if (kind == GemmKind::kGrouped) {
        PRQ_CASE(kKindGrouped, 128)
        PRQ_CASE(kKindGrouped, 256)
    } else if (kind == GemmKind::kGroupedSwap) {
        PRQ_CASE(kKindGroupedSwap, 128)
    }
#undef PRQ_CASE
    *unsupported = true;
    return cudaSuccess;
}

}  // namespace prq
