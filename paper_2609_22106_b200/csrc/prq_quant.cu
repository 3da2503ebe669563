// Activation quantisation kernel: the one MXFP4 quantisation of the reordered activation per layer call
// (Kernel design paragraph; Eq. (1) activation side when the scale and permutation are applied online).
//
// One CTA owns 128 rows x 128 columns: exactly one 512-byte scale atom of the GEMM's layout.  In
// identity mode a lane takes one whole 32-element block (a row of the tile is 4 lanes, a warp covers
// eight rows per step, two steps), with all eight 16-byte loads of a lane issued first, so that about
// 100 KB per SM are in flight -- the kernel is HBM-bound (2 bytes read + 0.5 + 1/32 written per element),
// latency is hidden by loads in flight rather than by occupancy, and the instruction count per element
// is what decides how close it gets (8 elements per lane: 11.3 us, 16: 10.3 us, 32: 9.8 us at 2048 x
// 9728).  Block amax by packed 16-bit maxima without any shuffle, E8M0 byte from the exponent field, 32
// round-to-nearest-even E2M1 conversions per lane, one 16-byte packed store per lane.  (Scale +
// permute mode keeps 8 elements per lane and 4 lanes per block.)  The atom's scale bytes are collected in shared memory and
// written out as one coalesced 512-byte piece; the bytes of tail blocks are also duplicated into the
// residual stages, which is all the "tail copy" this design needs (the GEMM re-reads the tail codes).
//
// The scale + permute mode has two structures.  From 512 rows on (and while two slices of rows fit shared memory)
// quant_act_rows_kernel runs: persistent CTAs that bring whole rows into shared memory by bulk copies and gather
// from there (see that kernel).  Smaller batches keep the column-atom CTAs of quant_act_kernel, whose rows can be
// cut into parts so that a few rows still fill the GPU.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdlib>

#include "prq_internal.h"
#include "prq_kernels.h"
#include "prq_ptx.cuh"
#include "prq_quant_block.cuh"

namespace prq {
namespace {

constexpr int kQuantThreads = 256;
constexpr int kAtomK = 128;    // columns per CTA (4 blocks = one scale atom)
constexpr int kSteps = kGroupRows / (2 * (kQuantThreads / 32));  // 8 steps of 16 rows
constexpr int kPermBatch = 4;   // scale + permute mode: steps whose loads are in flight together

// Scale byte from the block's largest magnitude given as fp32 bits: biased exponent - 2, floored at 0.
__device__ __forceinline__ uint32_t scale_byte(uint32_t amax_f32_bits) {
    const int eb = static_cast<int>(amax_f32_bits >> 23) - 2;
    return eb < 0 ? 0u : static_cast<uint32_t>(eb);
}

// Eight values (as fp32) -> 4 bytes of codes under the block scale 2^(byte - 127).
__device__ __forceinline__ uint32_t encode8(const float (&v)[8], uint32_t byte) {
    const float inv = __uint_as_float((254u - byte) << 23);  // 2^(127 - byte), exact multiply
    return cvt_e2m1x8(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv, v[4] * inv, v[5] * inv, v[6] * inv, v[7] * inv);
}

template <bool kScalePerm, bool kBatch>
__global__ void __launch_bounds__(kQuantThreads, kScalePerm ? 3 : 4)
quant_act_kernel(const QuantBatch b) {
    __shared__ __align__(16) uint8_t sf_atom[512];
    __shared__ int s_tile_start[kMaxExperts + 1];

    // Launched with programmatic stream serialisation: this CTA may be running while the previous kernel
    // of the stream still is.  Nothing that an earlier kernel may write or still read is touched before the
    // wait (x may be that kernel's output, and it may still be reading the buffers written here); the
    // layer's own permutation and reciprocal scales are constants of the prepared weights, and a dense
    // launch requests them first so that their latency overlaps the wait.
    grid_launch_dependents();

    // which of the batched layers this CTA works for (one launch may quantise the same activation for
    // several layers, each with its own scale, permutation and outputs)
    // (kBatch = false: a single layer, nothing to look up -- the division alone costs the small-batch
    // launches 0.2 us)
    const int lin = kBatch ? static_cast<int>(blockIdx.y) / b.groups_per_lin : 0;
    QuantParams p;
    p.x = b.x; p.M = b.M; p.ldx = b.ldx; p.K = b.K; p.n_experts = b.n_experts; p.act_groups = b.act_groups;
    p.expert_offsets = b.expert_offsets;
    {
        const QuantLayer& l = b.lay[lin];
        p.k_tail = l.k_tail; p.perm = l.perm; p.inv_s_perm = l.inv_s_perm;
        p.codes = l.codes; p.scales_row = l.scales_row; p.scales_sf = l.scales_sf;
    }
    // Which (128-column atom, 128-row group, share of the group's rows) this CTA takes.  In scale + permute mode the
    // atoms of the tail are some twenty times slower than the others: their source columns are scattered over the
    // whole row, every 2-byte read is a 32-byte sector of its own, and the CTA runs at the rate at which its SM's L1
    // takes sectors (about 20 us for 128 rows against 1 us for a head atom, whose window is nearly contiguous).  A
    // launch could not end before its slowest CTA, which the next kernel of the stream then waited for (8 - 11 us
    // per call at 4096 tokens).  So the tail atoms are cut into `tail_split` shares of the rows each and come first
    // in the grid, the head atoms after them.
    // (counted over the whole layer: the tail units of ALL row groups precede every head atom.)
    int group = static_cast<int>(blockIdx.y) - lin * b.groups_per_lin;
    int atom = blockIdx.x, tail_share = 0, tail_split = 1;
    if (kScalePerm && b.n_tail > 0) {
        const int units = b.n_tail * b.tail_split, n_head = b.n_atoms - b.n_tail;
        const int id = group * static_cast<int>(gridDim.x) + atom, first = units * b.groups_per_lin;
        if (id < first) {
            group = id / units;
            const int u = id - group * units;
            tail_split = b.tail_split; tail_share = u % tail_split; atom = n_head + u / tail_split;
        } else {
            const int r = id - first;
            group = r / n_head; atom = r - group * n_head;
        }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = lane >> 4, hl = lane & 15;   // which of the warp's two rows, lane inside the row
    float inv_s[8];
    int src[8];
    auto load_layer_constants = [&](int expert_) {
        const int c0 = atom * kAtomK + hl * 8;
        if (c0 < p.K) {
            const int32_t* perm = p.perm + static_cast<size_t>(expert_) * p.K + c0;
            const float* isp = p.inv_s_perm + static_cast<size_t>(expert_) * p.K + c0;
            const int4 p0 = *reinterpret_cast<const int4*>(perm), p1 = *reinterpret_cast<const int4*>(perm + 4);
            const float4 s0 = *reinterpret_cast<const float4*>(isp), s1 = *reinterpret_cast<const float4*>(isp + 4);
            src[0] = p0.x; src[1] = p0.y; src[2] = p0.z; src[3] = p0.w;
            src[4] = p1.x; src[5] = p1.y; src[6] = p1.z; src[7] = p1.w;
            inv_s[0] = s0.x; inv_s[1] = s0.y; inv_s[2] = s0.z; inv_s[3] = s0.w;
            inv_s[4] = s1.x; inv_s[5] = s1.y; inv_s[6] = s1.z; inv_s[7] = s1.w;
        }
    };
    const bool dense = p.expert_offsets == nullptr;
    if (kScalePerm && dense) load_layer_constants(0);
    grid_dependency_wait();

    // Which rows does this CTA own?  Dense: group g covers rows [128 g, 128 g + 128).  Grouped: the
    // scale groups are padded per expert, so walk the expert offsets to find ours.
    int row0, row_end, expert = 0;
    if (p.expert_offsets == nullptr) {
        row0 = group * kGroupRows;
        row_end = min(p.M, row0 + kGroupRows);
    } else {
        if (threadIdx.x < 32) warp_expert_starts(p.expert_offsets, p.n_experts, kGroupRows, s_tile_start, nullptr);
        __syncthreads();
        if (group >= s_tile_start[p.n_experts]) return;  // padding CTA of the launch grid
        int lo = 0, hi = p.n_experts - 1;
        while (lo < hi) {  // last expert whose first tile is <= group
            int mid = (lo + hi + 1) >> 1;
            if (s_tile_start[mid] <= group) lo = mid; else hi = mid - 1;
        }
        expert = lo;
        row0 = p.expert_offsets[expert] + (group - s_tile_start[expert]) * kGroupRows;
        row_end = min(p.expert_offsets[expert + 1], row0 + kGroupRows);
    }

    if (threadIdx.x < 128) reinterpret_cast<uint32_t*>(sf_atom)[threadIdx.x] = 0;
    __syncthreads();

    const int K = p.K, k_tail = p.k_tail;
    const int col0 = atom * kAtomK + hl * 8;      // first of this lane's 8 columns
    const bool col_ok = col0 < K;                 // K % 32 == 0, so a lane is all in or all out
    const int blk_in_atom = hl >> 2;
    const int gblk = atom * (kAtomK / kBlock) + blk_in_atom;
    const int tail_blk0 = (K - k_tail) / kBlock;  // first tail block (global block index)
    const StagePlan plan(K, k_tail);
    const int stage = atom >> 1;
    uint8_t* sf_base = p.scales_sf;
    const size_t sf_stage_stride = static_cast<size_t>(p.act_groups) * kSfGroupBytes;
    uint8_t* sf_group = sf_base + static_cast<size_t>(group) * kSfGroupBytes;
    const int n_rows = row_end - row0;            // 1..128
    // With few groups the rows of a group are split over gridDim.z CTAs (1, 2, 4 or 8 parts of whole
    // 16-row steps) so that a small batch still fills the GPU; only the scale + permute mode is split.
    const int n_parts = kScalePerm ? static_cast<int>(gridDim.z) * tail_split : 1;
    const int part = kScalePerm ? static_cast<int>(blockIdx.z) * tail_split + tail_share : 0;
    const int part_steps = kSteps / n_parts;

    if (kScalePerm && !dense) load_layer_constants(expert);   // grouped: the expert is known only now

    // row of step i: 16 rows per step, 2 per warp
    auto row_of = [&](int i) { return i * 16 + warp * 2 + half; };

    if (!kScalePerm) {
        // ---- identity.  Here a lane takes one whole 32-element block (64 contiguous bytes, four 16-byte
        // loads): no shuffle at all, a row of the tile is 4 lanes, a warp covers 8 rows and the tile is
        // done in 2 steps of 64 rows.  All eight loads are issued first, then the arithmetic runs on
        // packed bf16 pairs. ----
        const int l4 = lane & 3, rw = lane >> 2;
        const int c8 = warp * 8 + rw;                        // row inside a 64-row step
        const int colb = atom * kAtomK + l4 * 32;            // first of this lane's 32 columns
        const bool okb = colb < K;                           // K % 32 == 0: a lane is all in or all out
        const int gb = atom * (kAtomK / kBlock) + l4;        // this lane's block
        const uint16_t* xp = p.x + static_cast<size_t>(row0 + c8) * p.ldx + colb;
        const size_t x_step = static_cast<size_t>(64) * p.ldx;
        uint4 q[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                q[i][h] = make_uint4(0, 0, 0, 0);
                if (okb && i * 64 + c8 < n_rows) q[i][h] = __ldg(reinterpret_cast<const uint4*>(xp + i * x_step + 8 * h));
            }
        }
        uint8_t* cp = p.codes + static_cast<size_t>(row0 + c8) * (K / 2) + colb / 2;
        const size_t c_step = static_cast<size_t>(64) * (K / 2);
        uint8_t* rp = p.scales_row ? p.scales_row + static_cast<size_t>(row0 + c8) * (K / kBlock) + gb : nullptr;
        const size_t r_step = static_cast<size_t>(64) * (K / kBlock);
        const bool tail_lane = okb && gb >= tail_blk0;
        uint8_t* tp = nullptr;                                // this lane's duplicate slot in the residual stages
        if (tail_lane) {
            const int t = gb - tail_blk0;
            tp = sf_group + (plan.S1 + t / 8) * sf_stage_stride + ((t % 8) >> 2) * 512 + ((t % 8) & 3);
        }
        // row r = 64 i + c8 of the group: atom offset (r % 32) * 16 + (r / 32) * 4 + block
        const int in_atom0 = (c8 & 31) * 16 + (c8 >> 5) * 4;
        uint8_t* ap = sf_atom + in_atom0 + l4;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            uint4 packed;
            const uint32_t byte = quant_block32(q[i], packed);
            const bool row_ok = i * 64 + c8 < n_rows;
            if (okb && row_ok) {
                *reinterpret_cast<uint4*>(cp + i * c_step) = packed;
                ap[i * 8] = static_cast<uint8_t>(byte);
                if (rp) rp[i * r_step] = static_cast<uint8_t>(byte);
                if (tail_lane) tp[in_atom0 + i * 8] = static_cast<uint8_t>(byte);
            }
        }
    } else {
        // ---- scale + permute: gathered 2-byte loads (the head of the permutation is nearly the identity,
        // so they coalesce), multiply by the stored reciprocal scale in fp32.  The loads of four steps
        // (32 per lane) are issued before any arithmetic. ----
        // Everything that does not depend on the row is computed once: per-lane pointers that advance by
        // a fixed stride per 16-row step, the lane's slot in the residual stages, and -- for lanes past K --
        // zero sources and factors so that the arithmetic below needs no per-element select.
        const int w2h = warp * 2 + half;                       // row inside a 16-row step
        const size_t x_step = static_cast<size_t>(16) * p.ldx;
        const size_t c_step = static_cast<size_t>(16) * (K / 2);
        const size_t r_step = static_cast<size_t>(16) * (K / kBlock);
        const bool sf_lane = col_ok && (hl & 3) == 0;          // the lane that writes the block's scale byte
        const bool tail_lane = sf_lane && gblk >= tail_blk0;
        uint8_t* tp = nullptr;
        if (tail_lane) {
            const int t = gblk - tail_blk0;
            tp = sf_group + (plan.S1 + t / 8) * sf_stage_stride + ((t % 8) >> 2) * 512 + ((t % 8) & 3);
        }
        if (!col_ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e) { src[e] = 0; inv_s[e] = 0.f; }
        }
#pragma unroll 1
        for (int i0 = part * part_steps; i0 < (part + 1) * part_steps; i0 += kPermBatch) {
            if (i0 * 16 >= n_rows) break;   // nothing but padding rows from here on (their scale bytes are zero already)
            const int rb = i0 * 16 + w2h;   // this lane's row in the batch's first step
            const uint16_t* xb = p.x + static_cast<size_t>(row0 + rb) * p.ldx;
            uint8_t* cp = p.codes + static_cast<size_t>(row0 + rb) * (K / 2) + col0 / 2;
            uint8_t* rp = p.scales_row ? p.scales_row + static_cast<size_t>(row0 + rb) * (K / kBlock) + gblk : nullptr;
            uint32_t raw[kPermBatch][8];
#pragma unroll
            for (int ii = 0; ii < kPermBatch; ++ii) {
                if (ii >= part_steps) break;
                const bool ld_ok = col_ok && rb + 16 * ii < n_rows;
                const uint16_t* xrow = xb + ii * x_step;
#pragma unroll
                for (int e = 0; e < 8; ++e) raw[ii][e] = ld_ok ? static_cast<uint32_t>(__ldg(xrow + src[e])) : 0u;
            }
#pragma unroll
            for (int ii = 0; ii < kPermBatch; ++ii) {
                if (ii >= part_steps) break;
                const int r = rb + 16 * ii;
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(raw[ii][e] << 16) * inv_s[e];
                const float a01 = fmaxf(fabsf(v[0]), fabsf(v[1])), a23 = fmaxf(fabsf(v[2]), fabsf(v[3]));
                const float a45 = fmaxf(fabsf(v[4]), fabsf(v[5])), a67 = fmaxf(fabsf(v[6]), fabsf(v[7]));
                uint32_t am = __float_as_uint(fmaxf(fmaxf(a01, a23), fmaxf(a45, a67)));
                am = max(am, __shfl_xor_sync(0xffffffffu, am, 1));
                am = max(am, __shfl_xor_sync(0xffffffffu, am, 2));
                const uint32_t byte = scale_byte(am);
                const uint32_t packed = encode8(v, byte);
                if (col_ok && r < n_rows) {
                    *reinterpret_cast<uint32_t*>(cp + ii * c_step) = packed;
                    if (sf_lane) {
                        const int in_atom = (r & 31) * 16 + (r >> 5) * 4;
                        sf_atom[in_atom + blk_in_atom] = static_cast<uint8_t>(byte);
                        if (rp) rp[ii * r_step] = static_cast<uint8_t>(byte);
                        if (tail_lane) tp[in_atom] = static_cast<uint8_t>(byte);
                    }
                }
            }
        }
    }
    __syncthreads();
    // the atom's scale bytes, coalesced (rows past the end and blocks past K stay zero = 2^-127)
    if (n_parts == 1) {
        if (threadIdx.x < 32) {
            reinterpret_cast<uint4*>(sf_group + stage * sf_stage_stride + (atom & 1) * 512)[threadIdx.x] =
                reinterpret_cast<const uint4*>(sf_atom)[threadIdx.x];
        }
    } else if (threadIdx.x < kGroupRows / n_parts) {
        // this part's rows only: the four scale bytes of row r sit at (r % 32) * 16 + (r / 32) * 4
        const int r = part * (kGroupRows / n_parts) + threadIdx.x;
        const int off = (r & 31) * 16 + (r >> 5) * 4;
        *reinterpret_cast<uint32_t*>(sf_group + stage * sf_stage_stride + (atom & 1) * 512 + off) =
            *reinterpret_cast<const uint32_t*>(sf_atom + off);
    }
    if (part != 0) return;
    const int n_atoms = b.n_atoms;
    // An odd atom count leaves the second half of the last main stage without an owner: zero it.
    if (atom == n_atoms - 1 && (n_atoms & 1) && threadIdx.x >= 32 && threadIdx.x < 64)
        reinterpret_cast<uint4*>(sf_group + stage * sf_stage_stride + 512)[threadIdx.x - 32] = make_uint4(0, 0, 0, 0);
    // The CTA of the last atom also zero-fills what nobody else writes in the residual stages:
    // blocks past k_tail, and every byte of rows past the end of the group.
    if (atom == n_atoms - 1 && plan.S > plan.S1) {
        const int nb = kStageK / kBlock;
        for (int idx = threadIdx.x; idx < (plan.S - plan.S1) * kGroupRows * nb; idx += kQuantThreads) {
            const int ts = idx / (kGroupRows * nb);
            const int r = (idx / nb) % kGroupRows;
            const int b = idx % nb;
            const bool live = (r < n_rows) && (ts * nb + b) < k_tail / kBlock;
            if (!live) sf_group[(plan.S1 + ts) * sf_stage_stride + sf_offset_in_group(r, b)] = 0;
        }
    }
}


// ---------------------------------------------------------------------------------------------------------
// Scale + permute mode, second structure: whole rows through shared memory.  A persistent CTA takes consecutive
// slices of kRowsR rows; the rows of the next slices arrive by bulk copies (one per row, no instruction per element)
// while the current slice is quantised, and every gather of the permutation is a shared-memory read.  The lanes of
// a warp are 8 different rows reading the SAME source column, for the 4 blocks of one 128-column atom side by side:
// the staged rows are 16 bytes further apart than a multiple of 128 bytes, so the 8 rows fall into 8 different
// groups of four banks and a gather costs about one pass however scattered the permutation is -- against one
// 32-byte sector per 2-byte read when the tail of the permutation is gathered from global memory.  The column's
// source offset and reciprocal scale are the same for all rows of a warp: they are kept as one 16-byte record per
// column pair in shared memory (built once per layer and expert) instead of living in registers per lane.  A lane
// takes one row of one block: 32 values held in registers (no shuffle for the amax), 16 bytes of codes, one scale
// byte; the four bytes of (row, atom) meet by two shuffles and leave as the one word the GEMM's layout has for them.
// The tail's bytes are also collected in shared memory and written once more where the residual stages read them;
// rows and blocks that do not exist get zero bytes; row-major scales are written if asked for.  Several layers that
// read the same activation are quantised from the one copy of the rows.
// Threads per CTA: 256 where two CTAs share an SM, 512 where the rows of a wide layer leave room for one only.
constexpr int kRowsR = 8;                        // rows per slice
constexpr int kRowsMaxBufs = 8;                  // slices of rows in shared memory at most (at least 2)
static_assert(32 / kRowsR == 4, "a warp is 8 rows x the 4 blocks of an atom");
constexpr int kRowsSlices = kGroupRows / kRowsR; // slices per 128-row group

template <int kRowsThreads>
__global__ void __launch_bounds__(kRowsThreads, 512 / kRowsThreads)
quant_act_rows_kernel(const QuantBatch b, int n_slices, int n_buf) {
    extern __shared__ __align__(16) uint8_t rows_smem_raw[];
    // 256-byte aligned in the shared address space (the records are addressed with XORs)
    uint8_t* const rows_smem = rows_smem_raw + ((256u - (smem_u32(rows_smem_raw) & 255u)) & 255u);
    __shared__ int s_tile_start[kMaxExperts + 1];
    __shared__ int s_row_start[kMaxExperts + 1];
    __shared__ __align__(8) uint64_t bar_rows[kRowsMaxBufs];
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;
    grid_launch_dependents();
    const int K = b.K, nblk = K / kBlock;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t row_bytes = K * 2 + 16;       // staged row: 16 bytes past a multiple of 128
    const uint32_t buf_bytes = kRowsR * row_bytes;
    // per pair of destination columns: {byte offsets of the two source columns in a staged row, their two
    // reciprocal scales}; the records come first so that a block's sixteen are 256 aligned bytes
    uint4* rec = reinterpret_cast<uint4*>(rows_smem);
    const uint32_t rec_base = smem_u32(rows_smem);
    uint8_t* const rows_buf = rows_smem + (K / 2) * 16;
    uint8_t* sfb = rows_buf + n_buf * buf_bytes;     // 2 x [kRowsR][K / 32]: the tail blocks' scale bytes, per slice parity
    int rec_lin = -1, rec_expert = -1;           // which layer's constants the records hold
    if (threadIdx.x == 0) {
        for (int i = 0; i < kRowsMaxBufs; ++i) mbar_init(smem_u32(&bar_rows[i]), 1);
        abort_flag_s = 0;
        fence_mbar_init();
    }

    // The layer's (expert's) permutation and reciprocal scales as one 16-byte record per column pair, so that a
    // lane fetches them with one shared-memory read (the same for all rows of a warp).  The loads of four records
    // are in flight together: the build is in front of the first slice.
    auto build_records = [&](int lin, int expert) {
        const int2* perm2 = reinterpret_cast<const int2*>(b.lay[lin].perm + static_cast<size_t>(expert) * K);
        const float2* inv2 = reinterpret_cast<const float2*>(b.lay[lin].inv_s_perm + static_cast<size_t>(expert) * K);
#pragma unroll 1
        for (int c0 = threadIdx.x; c0 < K / 2; c0 += 4 * kRowsThreads) {
            int2 p2[4];
            float2 s2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int c2 = c0 + i * kRowsThreads;
                if (c2 < K / 2) { p2[i] = __ldg(perm2 + c2); s2[i] = __ldg(inv2 + c2); }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int c2 = c0 + i * kRowsThreads;
                if (c2 < K / 2)
                    rec[c2] = make_uint4(static_cast<uint32_t>(p2[i].x) * 2, static_cast<uint32_t>(p2[i].y) * 2,
                                         __float_as_uint(s2[i].x), __float_as_uint(s2[i].y));
            }
        }
        rec_lin = lin; rec_expert = expert;
    };
    const bool dense = b.expert_offsets == nullptr;
    // a dense layer's constants belong to the prepared weights, not to an earlier kernel of the stream: fetch them
    // while that kernel may still be running
    if (dense) build_records(0, 0);
    grid_dependency_wait();
    if (!dense) {
        // the experts' row ranges, once per CTA: every slice looks its expert up, and a dependent global load
        // there would sit in front of each of them
        for (int e = threadIdx.x; e <= b.n_experts; e += kRowsThreads) s_row_start[e] = b.expert_offsets[e];
        __syncthreads();
        if (threadIdx.x < 32) warp_expert_starts(s_row_start, b.n_experts, kGroupRows, s_tile_start, nullptr);
    }
    __syncthreads();
    const int n_groups = dense ? b.groups_per_lin : s_tile_start[b.n_experts];

    // where a slice sits: its group, its first row (in x) and how many of its rows exist
    struct Slice { int group, expert, r_first, row0, n_rows; };
    auto slice_at = [&](int sl) {
        Slice t;
        t.group = sl / kRowsSlices; t.r_first = (sl % kRowsSlices) * kRowsR; t.expert = 0;
        int g_row0, g_end;
        if (dense) {
            g_row0 = t.group * kGroupRows; g_end = min(b.M, g_row0 + kGroupRows);
        } else if (t.group >= n_groups) {   // padding of the launch grid
            g_row0 = 0; g_end = 0;
        } else {
            int lo = 0, hi = b.n_experts - 1;
            while (lo < hi) {  // last expert whose first group is <= group
                const int mid = (lo + hi + 1) >> 1;
                if (s_tile_start[mid] <= t.group) lo = mid; else hi = mid - 1;
            }
            t.expert = lo;
            g_row0 = s_row_start[lo] + (t.group - s_tile_start[lo]) * kGroupRows;
            g_end = min(s_row_start[lo + 1], g_row0 + kGroupRows);
        }
        t.row0 = g_row0 + t.r_first;
        t.n_rows = max(0, min(kRowsR, g_end - t.row0));
        return t;
    };
    auto request = [&](const Slice& t, int buf) {   // one thread
        if (t.n_rows == 0) return;
        const uint32_t bar = smem_u32(&bar_rows[buf]);
        mbar_arrive_expect_tx(bar, t.n_rows * K * 2);
        for (int r = 0; r < t.n_rows; ++r)
            bulk_load(smem_u32(rows_buf + buf * buf_bytes + r * row_bytes), b.x + static_cast<size_t>(t.row0 + r) * b.ldx, K * 2, bar);
    };

    const int rl = lane % kRowsR, side = lane / kRowsR;
    const uint32_t byte_sel = side == 0 ? 0x3210u : side == 1 ? 0x2301u : side == 2 ? 0x1032u : 0x0123u;
    const size_t sf_stage_stride = static_cast<size_t>(b.act_groups) * kSfGroupBytes;
    uint32_t phases = 0;                         // bit i: parity of buffer i's next completion
    // a CTA's slices are consecutive: with stacked experts its records then change a few times, not per slice.  The
    // rows of the next n_buf - 1 slices are on their way while a slice is quantised: a narrow layer's slice is
    // quantised in a fraction of the time its rows take to arrive.
    const int per_cta = (n_slices + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    int sl = min(n_slices, static_cast<int>(blockIdx.x) * per_cta);
    const int sl_end = min(n_slices, sl + per_cta);
    if (threadIdx.x == 0)
        for (int d = 0; d < n_buf - 1 && sl + d < sl_end; ++d) request(slice_at(sl + d), d);
    for (int it = 0; sl < sl_end; ++it, ++sl) {
        const int buf = it % n_buf;
        // the buffer of the slice before this one: its readers passed the barrier of their slice
        if (threadIdx.x == 0 && sl + n_buf - 1 < sl_end) request(slice_at(sl + n_buf - 1), (it + n_buf - 1) % n_buf);
        const Slice cur = slice_at(sl);
        if (!dense && cur.group >= n_groups) continue;
        if (cur.n_rows > 0) {
            if (!mbar_wait(smem_u32(&bar_rows[buf]), (phases >> buf) & 1u, abort_flag)) break;
            phases ^= 1u << buf;
        }
        const bool row_ok = rl < cur.n_rows;
        const uint32_t xrow_a = smem_u32(rows_buf + buf * buf_bytes + rl * row_bytes);
        const size_t row = static_cast<size_t>(cur.row0 + rl);
        const int g = cur.r_first + rl;                        // row inside its 128-row group
        const int sf_row_off = (g & 31) * 16 + (g >> 5) * 4;
        uint8_t* tailb = sfb + (it & 1) * (kRowsR * nblk);     // [kRowsR][tail blocks] of this slice
        for (int lin = 0; lin < b.n_lin; ++lin) {
            const QuantLayer& l = b.lay[lin];
            if (rec_lin != lin || rec_expert != cur.expert) {
                if (rec_lin >= 0) __syncthreads();             // the old records are still being read
                build_records(lin, cur.expert);
                __syncthreads();
            }
            const StagePlan plan(K, l.k_tail);
            const int tail_blk0 = (K - l.k_tail) / kBlock, n_tail_blk = l.k_tail / kBlock;
            uint8_t* sf_group = l.scales_sf + static_cast<size_t>(cur.group) * kSfGroupBytes;
            uint8_t* crow = l.codes + row * (K / 2);
            // A warp takes whole 128-column atoms, its four sides one block each: the four scale bytes of
            // (row, atom) meet by two shuffles and go out as the one word the GEMM's layout has for them.  Rows
            // and blocks that do not exist contribute zero bytes (an odd atom count leaves half a stage of them).
#pragma unroll 1
            for (int a = warp; a < 2 * plan.S1; a += kRowsThreads / 32) {
                const int blk = a * 4 + side;
                const int j0 = blk * kBlock;
                uint32_t byte = 0;
                if (row_ok && blk < nblk) {
                    // At step t a lane visits the block's column pair t ^ side: where the permutation is (nearly)
                    // the identity, the four blocks side by side would otherwise read the same banks.  (A block's
                    // records are 256 aligned bytes, so the exchange is one XOR on the address.)
                    const uint32_t rec_blk = rec_base + (blk * 256 ^ (side << 4));
                    float v[32];
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        uint4 rc;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(rc.x), "=r"(rc.y), "=r"(rc.z), "=r"(rc.w) : "r"(rec_blk ^ (t << 4)));
                        uint16_t x0, x1;
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(x0) : "r"(xrow_a + rc.x));
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(x1) : "r"(xrow_a + rc.y));
                        v[2 * t] = __uint_as_float(static_cast<uint32_t>(x0) << 16) * __uint_as_float(rc.z);
                        v[2 * t + 1] = __uint_as_float(static_cast<uint32_t>(x1) << 16) * __uint_as_float(rc.w);
                    }
                    float am;
                    {
                        float m[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            m[i] = fmaxf(fmaxf(fabsf(v[4 * i]), fabsf(v[4 * i + 1])), fmaxf(fabsf(v[4 * i + 2]), fabsf(v[4 * i + 3])));
                        am = fmaxf(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])), fmaxf(fmaxf(m[4], m[5]), fmaxf(m[6], m[7])));
                    }
                    byte = scale_byte(__float_as_uint(am));
                    const float inv = __uint_as_float((254u - byte) << 23);  // 2^(127 - byte), exact multiply
                    uint32_t pk[4];
#pragma unroll
                    for (int h = 0; h < 4; ++h)
                        pk[h] = cvt_e2m1x8(v[8 * h] * inv, v[8 * h + 1] * inv, v[8 * h + 2] * inv, v[8 * h + 3] * inv,
                                           v[8 * h + 4] * inv, v[8 * h + 5] * inv, v[8 * h + 6] * inv, v[8 * h + 7] * inv);
                    // byte t of pk holds pair t ^ side: exchange the bytes inside every word accordingly
                    *reinterpret_cast<uint4*>(crow + j0 / 2) =
                        make_uint4(__byte_perm(pk[0], 0, byte_sel), __byte_perm(pk[1], 0, byte_sel),
                                   __byte_perm(pk[2], 0, byte_sel), __byte_perm(pk[3], 0, byte_sel));
                    if (l.scales_row) l.scales_row[row * nblk + blk] = static_cast<uint8_t>(byte);
                    if (blk >= tail_blk0) tailb[rl * nblk + blk - tail_blk0] = static_cast<uint8_t>(byte);
                }
                uint32_t w = byte << (8 * side);
                w |= __shfl_xor_sync(0xffffffffu, w, 8);
                w |= __shfl_xor_sync(0xffffffffu, w, 16);
                if (side == 0)
                    *reinterpret_cast<uint32_t*>(sf_group + (a >> 1) * sf_stage_stride + (a & 1) * 512 + sf_row_off) = w;
            }
            // every warp is through with this slice's rows (their buffer may be refilled from now on) and the tail's
            // bytes are in shared memory
            __syncthreads();
            if (n_tail_blk > 0) {
                // the tail's bytes once more, where the residual stages read them (zeros past the tail and the rows)
                for (int idx = threadIdx.x; idx < kRowsR * (plan.S - plan.S1) * 2; idx += kRowsThreads) {
                    const int r = idx % kRowsR, sa = idx / kRowsR, ts = sa >> 1, ah = sa & 1;
                    const int t0 = ts * 8 + ah * 4;
                    uint32_t w = 0;
                    if (r < cur.n_rows) {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (t0 + i < n_tail_blk) w |= static_cast<uint32_t>(tailb[r * nblk + t0 + i]) << (8 * i);
                    }
                    const int gr = cur.r_first + r;
                    *reinterpret_cast<uint32_t*>(sf_group + (plan.S1 + ts) * sf_stage_stride + ah * 512 + (gr & 31) * 16 + (gr >> 5) * 4) = w;
                }
            }
        }
    }
    if (abort_flag_s) {
        // copies may still be on their way into this CTA's shared memory: give them one more bounded wait
        for (int i = 0; i < n_buf; ++i) mbar_wait_after_abort(smem_u32(&bar_rows[i]), (phases >> i) & 1u);
        if (threadIdx.x == 0 && b.status) atomicExch(b.status, static_cast<int>(PRQ_ERR_TIMEOUT));
    }
}

template <int kRowsThreads>
cudaError_t launch_rows_impl(const QuantBatch& b, size_t smem, int n_buf, int sm_count, cudaStream_t stream) {
    static size_t configured = 0;   // the attribute is per function; raise it when a larger K comes
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(quant_act_rows_kernel<kRowsThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    const int n_slices = b.groups_per_lin * kRowsSlices;
    const int per_sm = 512 / kRowsThreads;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_slices < per_sm * sm_count ? n_slices : per_sm * sm_count);
    cfg.blockDim = dim3(kRowsThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, quant_act_rows_kernel<kRowsThreads>, b, n_slices, n_buf);
}

}  // namespace

cudaError_t launch_quant_act_batch(const QuantBatch& b, bool scale_perm, cudaStream_t stream) {
    const QuantBatch& p = b;
    const int grid_groups = b.groups_per_lin * b.n_lin;
    cudaLaunchConfig_t cfg = {};
    const int n_atoms = (p.K + kAtomK - 1) / kAtomK;
    int parts = 1;
    if (scale_perm) {
        // split the rows of a group (a CTA has a fixed cost of about a microsecond, so no further than needed)
        static int sm_count[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        if (sm_count[dev] == 0) {
            int n = 0;
            cudaError_t e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return e;
            sm_count[dev] = n;
        }
        const long long tiles = static_cast<long long>(n_atoms) * grid_groups;
        while (parts < 4 && tiles * parts < 8LL * sm_count[dev]) parts *= 2;   // 3 CTAs per SM: keep the last wave short
        if (parts == 4 && tiles * parts < 4LL * sm_count[dev]) parts = 8;
        if (const char* ev = dev_knobs_enabled() ? getenv("PRQ_QUANT_PARTS") : nullptr) { const int v = atoi(ev); if (v == 1 || v == 2 || v == 4 || v == 8) parts = v; }
        // Whole rows through shared memory when there are rows enough to fill the GPU that way, a slice's rows fit
        // twice, and the rows can be fetched by bulk copies (16-byte aligned).
        // (dense layers: with stacked experts of K = 768 the row structure measured 25-40 % slower than the column atoms
        // at 128 experts -- 26.7 against 19.0 us at 1024 tokens, 78.7 against 63.5 at 8192 -- also with the experts' row
        // ranges cached in shared memory and seven slices in flight: narrow rows leave two of the eight warps without
        // an atom, and a slice of 8 rows is little work per barrier)
        int rows = b.M >= 512 && b.expert_offsets == nullptr ? 1 : 0;
        if (const char* ev = dev_knobs_enabled() ? getenv("PRQ_QUANT_ROWS") : nullptr) rows = atoi(ev);
        const size_t buf_bytes = static_cast<size_t>(kRowsR) * (p.K * 2 + 16);
        const size_t fixed = static_cast<size_t>(p.K) * 8 + 2 * static_cast<size_t>(kRowsR) * (p.K / 32) + 256;   // + alignment slack
        if (rows && 2 * buf_bytes + fixed <= 200 * 1024 && (reinterpret_cast<uintptr_t>(b.x) & 15) == 0 && b.ldx % 8 == 0) {
            QuantBatch br = b;
            br.n_atoms = n_atoms; br.n_tail = 0; br.tail_split = 1;
            // Two CTAs per SM where two slices of rows fit twice (8.7 KB of static shared memory and 1 KB reserved per
            // CTA beside the dynamic part); then as many slices in flight as the CTA's share of the SM holds.
            const size_t half_sm = 227 * 1024 / 2 - 10 * 1024;
            const bool two = 2 * buf_bytes + fixed <= half_sm;
            const size_t budget = two ? half_sm : 200 * 1024;
            int n_buf = static_cast<int>((budget - fixed) / buf_bytes);
            n_buf = n_buf > kRowsMaxBufs ? kRowsMaxBufs : n_buf;
            const size_t smem = n_buf * buf_bytes + fixed;
            return two ? launch_rows_impl<256>(br, smem, n_buf, sm_count[dev], stream)
                       : launch_rows_impl<512>(br, smem, n_buf, sm_count[dev], stream);
        }
    }
    // the tail atoms of the scale + permute mode in shares of 16 rows (128 / 8), see the kernel
    QuantBatch bb = b;
    bb.n_atoms = n_atoms;
    bb.n_tail = 0; bb.tail_split = 1;
    // (dense launches only: a grouped launch has a CTA per expert group and column atom already, each with the fixed
    // cost of finding its expert -- eight times as many tail CTAs made the 128-expert quantiser 35-50 % slower, and its
    // launches are long enough for a 20 us CTA not to be their end)
    if (scale_perm && b.expert_offsets == nullptr) {
        int k_max = 0;
        for (int i = 0; i < b.n_lin; ++i) k_max = b.lay[i].k_tail > k_max ? b.lay[i].k_tail : k_max;
        bb.n_tail = (k_max + kAtomK - 1) / kAtomK < n_atoms ? (k_max + kAtomK - 1) / kAtomK : n_atoms;
        bb.tail_split = 8 / parts;
    }
    cfg.gridDim = dim3(n_atoms - bb.n_tail + bb.n_tail * bb.tail_split, grid_groups, parts);
    cfg.blockDim = dim3(kQuantThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (b.n_lin > 1)
        return scale_perm ? cudaLaunchKernelEx(&cfg, quant_act_kernel<true, true>, bb)
                          : cudaLaunchKernelEx(&cfg, quant_act_kernel<false, true>, bb);
    return scale_perm ? cudaLaunchKernelEx(&cfg, quant_act_kernel<true, false>, bb)
                      : cudaLaunchKernelEx(&cfg, quant_act_kernel<false, false>, bb);
}

cudaError_t launch_quant_act(const QuantParams& p, bool scale_perm, int grid_groups, cudaStream_t stream) {
    QuantBatch b = {};
    b.x = p.x; b.expert_offsets = p.expert_offsets; b.M = p.M; b.ldx = p.ldx; b.K = p.K;
    b.n_experts = p.n_experts; b.act_groups = p.act_groups;
    b.n_lin = 1;
    b.groups_per_lin = grid_groups;
    b.lay[0] = QuantLayer{p.perm, p.inv_s_perm, p.codes, p.scales_row, p.scales_sf, p.k_tail};
    b.status = p.status;
    return launch_quant_act_batch(b, scale_perm, stream);
}

}  // namespace prq
