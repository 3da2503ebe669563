// Internal declarations shared by the translation units of libprq.
#pragma once
#include <cstdlib>
#include <cstddef>
#include <cstdint>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "prq.h"

namespace prq {

// Developer switches (PRQ_DECODE_SPLITS, PRQ_GROUPED_BN, PRQ_TRACE_PTR, ...) are looked at only when the
// process was started with PRQ_DEV=1; that one variable is read once, so that a normal call makes no
// getenv at all.
inline bool dev_knobs_enabled() {
    static const bool on = [] { const char* v = std::getenv("PRQ_DEV"); return v && v[0] == '1'; }();
    return on;
}


constexpr int kBlock = 32;        // MXFP4 block length
constexpr int kStageK = 256;      // reduction elements per pipeline stage (one 128-byte swizzled row)
constexpr int kGroupRows = 128;   // rows per scale-factor group
constexpr int kSfGroupBytes = 1024;  // one (stage, 128-row group) of scale bytes: 2 atoms of 512 bytes
constexpr int kMaxExperts = 1024;

// Reduction stages of a layer: S1 cover the K main columns, S - S1 the k_tail residual columns.
struct StagePlan {
    int K, k_tail, S1, S;
    __host__ __device__ StagePlan() : K(0), k_tail(0), S1(0), S(0) {}
    __host__ __device__ StagePlan(int K_, int k_) : K(K_), k_tail(k_) {
        S1 = (K_ + kStageK - 1) / kStageK;
        S = S1 + (k_ + kStageK - 1) / kStageK;
    }
};

// Byte offset of the scale of (row r of a 128-row group, block b of a stage) inside the group's
// 1024-byte tile: two 512-byte atoms (4 blocks each); inside an atom 16 bytes per (r % 32) holding
// 4 bytes per (r / 32), one per block.  This is the order the tensor-memory scale copy consumes.
__host__ __device__ inline int sf_offset_in_group(int r, int blk_in_stage) {
    return (blk_in_stage >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (blk_in_stage & 3);
}

struct PrepResult {
    std::vector<float> s, inv_s;
    std::vector<double> col_err;
    std::vector<int32_t> perm;
    std::vector<uint8_t> codes;   // N x (K + k)/2
    std::vector<uint8_t> scales;  // N x (K + k)/32
};

// Algorithm 1 steps 3-7 and 11 for one layer and one alpha, on the host.
// Returns PRQ_ERR_NONFINITE if W or amax hold a NaN or an infinity.
// scale_search: every weight block (main part and residual) takes the best of the floor-rule scale and its
// two neighbours (the "E8M0-W" variant of the ablation study); ranking and permutation are unaffected.
prq_status prepare_layer(const uint16_t* W, int N, int K, const float* amax, float alpha, int k_tail,
                         PrepResult& out, bool scale_search = false);
// The pieces of it that stay on the host when the rest runs on the GPU:
// s_j = max(amax_j, 1e-5)^alpha and its reciprocal (FP64, stored fp32; PRQ_ERR_NONFINITE on a bad amax) ...
prq_status channel_scales(const float* amax, int K, float alpha, std::vector<float>& s, std::vector<float>& inv_s);
// ... and the error-ranked top-k with its permutation [unselected ascending | selected ascending]
// (ties: the lower channel index ranks first).
void rank_and_permute(const std::vector<double>& col_err, int K, int k_tail, std::vector<int32_t>& perm);
// Eq. (1), middle line: rows of the producer weights permuted (and, for the up projection, scaled by 1 / s and
// rounded once to bf16); with duplicate_tail the last k_tail rows are repeated.  Host buffers.
prq_status fold_producer(const int32_t* perm, const float* inv_s, int C, int k_tail, const uint16_t* W_up,
                         const uint16_t* W_gate, int H, bool duplicate_tail, uint16_t* out_up, uint16_t* out_gate);
// Offline half of a layer in the second format (MXFP8) for one alpha, on the host: scales as above, W0 = fl32(W * s),
// E4M3 codes (N x K bytes) and E8M0 scale bytes (N x K/32) by rows.  No permutation, no tail.
prq_status prepare_layer_fp8(const uint16_t* W, int N, int K, const float* amax, float alpha, std::vector<float>& s,
                             std::vector<float>& inv_s, std::vector<uint8_t>& codes, std::vector<uint8_t>& scales);
// Gate and up projection rows interleaved in groups of 32 (rows 64 b .. 64 b + 31 = gate rows 32 b .., rows 64 b + 32 ..
// 64 b + 63 = up rows 32 b ..): the layout prq_linear_gated expects.  Host buffers, C % 32 == 0.
void stack_gate_up(const uint16_t* W_gate, const uint16_t* W_up, int C, int H, uint16_t* out);
// The same result computed on the current device from a DEVICE copy of W (column errors, permuted
// quantisation, residual and packing as kernels; scales and ranking on the host in between).  Allocates its
// temporaries, runs on `stream` and synchronises it.
prq_status prepare_layer_device(const uint16_t* W_dev, int N, int K, const float* amax, float alpha, int k_tail,
                                PrepResult& out, bool scale_search, cudaStream_t stream);

}  // namespace prq

struct prq_weights {
    int n_experts = 0, N = 0, K = 0, k_tail = 0;
    float alpha = 0.f;
    prq::StagePlan plan;
    int w_groups = 0;  // ceil(N / 128) scale groups per expert (layout for 128- and 256-row weight tiles)
    int device = -1;
    // canonical host copies (all experts concatenated)
    std::vector<uint8_t> h_codes, h_scales;
    std::vector<int32_t> h_perm;
    std::vector<float> h_s, h_inv_s;
    std::vector<double> h_col_err;
    // device copies
    uint8_t* d_codes = nullptr;      // E x N x (K + k)/2
    uint8_t* d_sf = nullptr;         // E x S x w_groups x 1024 (+ padding)
    // Dense layers also keep the scale bytes grouped per 224-, 240- and 288-row weight tile of the prefill kernel
    // (two or three 128-row groups per tile, the last partly empty) so that those tile widths need no re-alignment.
    // A handle prepared as a gated producer (prq_prep_opts::gated_producer) keeps the 192-row tiling instead, the
    // one prq_linear_gated runs.
    uint8_t* d_sf_alt[4] = {nullptr, nullptr, nullptr, nullptr};
    int w_groups_alt[4] = {0, 0, 0, 0};
    bool gated = false;
    // Second format (prq_prep_opts::format = PRQ_FMT_MXFP8): d_codes holds N x K bytes of E4M3 codes, d_sf the scale
    // bytes as [128-element stage][128-row group][512]; k_tail is 0, perm the identity; none of the MXFP4 tilings exist.
    int format = 0;
    CUtensorMap tm_w_fp8;
    float* d_inv_s = nullptr;        // K: the activation side's factors (original = permuted order)
    // tensor maps of the weight side, encoded once (dense layers; a handle is immutable afterwards):
    // codes with 128-row boxes (decode kernel), codes with half-tile boxes and the scale bytes of the
    // 224-row [0], 240-row [1], 288-row [2] and 192-row [3] tilings (CTA-pair prefill kernel)
    CUtensorMap tm_w_decode, tm_w_pair[4], tm_sfw_pair[4];
    bool maps_ready = false;
    int32_t* d_perm = nullptr;       // E x K
    float* d_inv_s_perm = nullptr;   // E x K : inv_s[perm[j]] in the new channel order
    size_t d_codes_bytes = 0, d_sf_bytes = 0;
};
