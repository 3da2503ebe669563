// Launch interfaces of the device kernels (used by the C-ABI entry points).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "prq_internal.h"

namespace prq {

// Developer trace (clock stamps written to a caller-supplied buffer) is compiled in only with -DPRQ_TRACE=1:
// even a never-taken branch per stage shows in the latency-bound decode kernel (0.05-0.15 us).
#ifndef PRQ_TRACE
#define PRQ_TRACE 0
#endif
constexpr bool kTraceBuild = PRQ_TRACE != 0;

// Default limit of every wait inside a kernel, in SM clock cycles (about two seconds).  A wait that runs out
// makes its CTA unwind and record PRQ_ERR_TIMEOUT; it never spins without bound.
constexpr long long kDefaultWaitLimitCycles = 4000000000ll;

struct QuantParams {
    const uint16_t* x;       // M x K bf16, row stride ldx
    int M, ldx, K, k_tail;
    int n_experts;
    int act_groups;          // 128-row scale groups per stage in scales_sf
    const int32_t* expert_offsets;  // nullptr when dense
    const int32_t* perm;     // E x K (scale+perm mode)
    const float* inv_s_perm; // E x K
    uint8_t* codes;          // M x K/2
    uint8_t* scales_row;     // M x K/32 or nullptr
    uint8_t* scales_sf;      // S x act_groups x 1024
    int* status;             // device status word (a bounded wait that ran out is recorded there)
};

cudaError_t launch_quant_act(const QuantParams& p, bool scale_perm, int grid_groups, cudaStream_t stream);

// Several dense layers that read the same activation (q / k / v, gate / up), quantised by one launch: the
// fields that differ per layer; everything else comes from `base`.
constexpr int kMaxBatch = 4;
struct QuantLayer {                      // what differs per batched layer
    const int32_t* perm;
    const float* inv_s_perm;
    uint8_t* codes;
    uint8_t* scales_row;
    uint8_t* scales_sf;
    int k_tail;
};
// The common fields come first and layer 0 right behind them, so that a launch for a single layer reads
// one 128-byte line of kernel parameters.
struct QuantBatch {
    const uint16_t* x;
    const int32_t* expert_offsets;
    int M, ldx, K;
    int n_experts;
    int act_groups;
    int n_lin;                           // 1 .. kMaxBatch
    int groups_per_lin;                  // blockIdx.y = layer * groups_per_lin + group
    int n_atoms, n_tail, tail_split;     // set by the launcher: 128-column atoms, how many of them are tail atoms
                                         // (scale + permute mode), and into how many row shares each of those is cut
    QuantLayer lay[kMaxBatch];
    int* status;                         // device status word
};
cudaError_t launch_quant_act_batch(const QuantBatch& b, bool scale_perm, cudaStream_t stream);

struct GemmParams {
    int M;                   // activation rows (all experts)
    int N, K, k_tail;
    int n_experts;
    int act_groups;          // 128-row groups per stage in act_sf
    int w_groups;            // 128-row groups per stage per expert in w_sf
    const uint8_t* act_sf;
    const uint8_t* w_sf;
    const int32_t* expert_offsets;  // grouped only
    void* y;
    int ldy;
    int y_bf16;
    int* status;             // device status word
    long long* trace;        // developer trace buffer (nullptr in normal use)
    int dbg;                 // developer switches for timing experiments (0 in normal use)
};

// Grouped (MoE) kernel: 128 output features of one expert on the MMA M axis, `bn` (128 or 64) tokens of that expert
// on the N axis; `grid` persistent CTAs.  `tm_w` has 128-row boxes, `tm_act` bn-row boxes.
cudaError_t launch_gemm_grouped(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                                cudaStream_t stream);


// The same kernel for the second format (MXFP8), dense layers of any M: `p.expert_offsets` null, `p.n_experts` 1;
// scale bytes in 512-byte groups per (128-element stage, 128-row group); code maps over K-byte rows.
cudaError_t launch_gemm_fp8(const CUtensorMap& tm_act, const CUtensorMap& tm_w, const GemmParams& p, int grid,
                            cudaStream_t stream);

// Activation quantiser of the second format: x (M x K bf16, row stride ldx), optionally times inv_s[j] (null: identity),
// to E4M3 codes (M x K bytes), row-major scale bytes (or null) and tile-ordered scale bytes
// [stage = 128 columns][128-row group][512].
cudaError_t launch_quant_act_fp8(const uint16_t* x, int M, int ldx, int K, const float* inv_s, uint8_t* codes,
                                 uint8_t* scales_row, uint8_t* scales_sf, cudaStream_t stream);

// Decode kernel (M <= 128): cluster split-K with a distributed-shared-memory reduction.
struct DecodeParams {
    int M, N, K, k_tail;
    int w_groups;               // 128-row scale groups per stage in w_sf
    const uint8_t* act_sf;      // one group per stage
    const uint8_t* w_sf;
    const uint16_t* x;          // fused variant: bf16 activation M x K (leading dimension ldx), else null
    int ldx;
    void* y;
    int ldy, y_bf16;
    int splits;                 // = cluster size, 1..8
    int* status;
    long long* trace;
    int dbg;
};
// Several dense layers over the same tokens (q / k / v, gate / up) in one launch.
struct DecodeLayer {                 // what differs per batched layer
    const uint8_t* act_sf;
    const uint8_t* w_sf;
    void* y;
    int N, w_groups, ldy;
    int tile_end;                    // 128-row weight tiles of layers 0 .. this one together
};
// The common fields come first and layer 0 right behind them, so that a launch for a single layer reads
// one 128-byte line of kernel parameters.
struct DecodeBatch {
    const uint16_t* x;               // fused variant (one layer): bf16 activation, else null
    int* status;
    long long* trace;
    int M, K, k_tail, ldx;
    int y_bf16, splits, dbg;
    int n_lin;                       // 1 .. kMaxBatch
    DecodeLayer lay[kMaxBatch];
};
struct DecodeMaps {
    CUtensorMap act[kMaxBatch];
    CUtensorMap w[kMaxBatch];
};
// `bn` in {16, 32, 64, 128} is the token tile; the grid is (all tiles) * splits CTAs in clusters of `splits`.
cudaError_t launch_decode_batch(int bn, const DecodeMaps& maps, const DecodeBatch& b, cudaStream_t stream);
// `bn` in {16, 32, 64, 128} is the token tile; the grid is n_tiles * splits CTAs in clusters of `splits`.
cudaError_t launch_decode(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w, const DecodeParams& p,
                          int n_tiles, cudaStream_t stream);
// How many clusters of `splits` CTAs of the decode kernel can be resident at once on the current device.
int decode_max_active_clusters(int bn, int splits);

// Prefill kernel (M > 128): 256 x 224 or 256 x 240 output tiles, each computed by two CTAs of a cluster.
constexpr int kPrefillTileN = 224;
constexpr int kPrefillTileWide = 240;
constexpr int kPrefillTileOneWave = 288;   // one accumulator: only for calls whose tiles fit one wave of pairs at this width
constexpr int kPrefillTileGated = 192;     // gated-producer epilogue: three (gate, up) groups of 32 + 32 columns per tile
constexpr size_t kPrefillSlotBytes = 128 * 256 * sizeof(float);   // workspace per partial tile of one CTA
struct PrefillParams {
    int M, N, K, k_tail;
    int m_tiles, n_tiles;       // 256-row x 224- (240-) column tiles
    int sk_tiles, whole_tiles;  // tiles 0 .. sk_tiles-1 are split stream-K over all pairs, then pair g
                                // computes the whole tiles sk_tiles + wave * pairs + g, wave < whole_tiles
    int sk_aligned, sk_base, sk_extra;  // how the stream-K tiles are cut (see SkPlan in the kernel)
    int act_groups, w_groups;   // 128-row scale groups per stage in act_sf / w_sf
    const uint8_t* act_sf;
    const uint8_t* w_sf;
    float* partial;             // two fp32 slots (128 rows x tile width, rounded up to 32 columns) per CTA
    int* flags;                 // "arrived" counter per 128-row half of a tile (index 2 * tile + half) ...
    int flag_stride;            // ... and, this many ints further, its "finished" counter; all zero between launches
    void* y;                    // output matrix and its row stride in elements: used only for the column group at
    int ldy;                    // the right edge that is narrower than 16 bytes (the tiled stores cover the rest)
    int y_bf16;
    int* status;
    long long* trace;
    int dbg;
    long long wait_limit;       // SM clock cycles after which a wait inside the kernel gives up (PRQ_ERR_TIMEOUT)
    int total_tiles;            // m_tiles * n_tiles: whole-tile waves stop here (the last wave may be short)
    // Gated-producer epilogue (kPrefillTileGated only): the layer is a gate and an up projection interleaved in
    // groups of 32 output features; instead of y the kernel writes Q(silu(gate) * up), the MXFP4 activation of the
    // down projection that follows (C input channels, tail k_tail), straight into that layer's buffers.
    uint8_t* out_codes;         // M x C/2
    uint8_t* out_sf;            // scale bytes in the GEMM's tile order, tail bytes duplicated
    uint8_t* out_scales_row;    // M x C/32, or null
    uint16_t* out_h;            // M x C bf16 (the product before quantisation), or null: for checks
    int out_C, out_k_tail, out_groups;
};
// `bn` = tile width (kPrefillTileN, kPrefillTileWide, kPrefillTileOneWave, or kPrefillTileGated for the gated-producer
// epilogue).  `tm_w` has boxes of bn / 2 rows (288: bn / 4 = 72 rows, loaded twice per CTA and stage); `tm_sfa` / `tm_sfw`
// view the scale bytes as rows of 256 bytes with boxes of 4 / 8 (288: 16) rows (one / two / four 128-row groups);
// `tm_y` has 32 x 32 boxes (any valid map for the gated instance, which stores nothing through it).
cudaError_t launch_prefill_pair(int bn, const CUtensorMap& tm_act, const CUtensorMap& tm_w,
                                const CUtensorMap& tm_sfa, const CUtensorMap& tm_sfw, const CUtensorMap& tm_y,
                                const PrefillParams& p, int pairs, cudaStream_t stream);
// How many pairs of the pair kernel can be resident at once on the current device.
int prefill_pair_max_clusters(int bn);

// Benchmark utility: `grid` CTAs each issuing n_mma block-scaled FP4 MMAs (128 x 256 x 64) from shared memory.
cudaError_t launch_mxf4_peak_probe(int n_mma, int grid, int* status, cudaStream_t stream);

// Benchmark utility: `n` empty kernels in a row, each launched like the decode GEMM (programmatic dependent
// launch, `grid` CTAs of `threads` threads in clusters of `cluster`) and each waiting for the one before it.
cudaError_t launch_handover_probe(int n, int grid, int threads, int cluster, int* sink, cudaStream_t stream);

}  // namespace prq
