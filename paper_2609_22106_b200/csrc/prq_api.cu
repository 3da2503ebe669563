// C-ABI entry points of libprq: argument checks, the weight handle, tensor-map construction,
// kernel selection.  See include/prq.h for the contract of every call.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "prq_internal.h"
#include "prq_kernels.h"

namespace prq {
namespace {

__device__ int g_device_status = 0;
__device__ int g_probe_sink = 0;   // the hand-over probe's kernels count themselves here; nothing reads it

std::atomic<unsigned long long> g_launches{0};

struct DeviceInfo {
    bool ok = false;
    int num_sms = 0;
    int* status_ptr = nullptr;
    int max_clusters[4][9] = {};  // decode kernel: [token-tile index][cluster size], 0 = not queried yet
    int max_pairs = 0;            // prefill pair kernel: co-resident CTA pairs, 0 = not queried yet
    int max_pairs_gated = 0;      // the same for its gated-producer instance
};
std::mutex g_dev_mutex;
DeviceInfo g_dev[64];

// Per-device facts, looked up once: sm_100 check, SM count, address of the status word.
prq_status device_info(int dev, DeviceInfo** out) {
    if (dev < 0 || dev >= 64) return PRQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceInfo& d = g_dev[dev];
    if (!d.ok) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return PRQ_ERR_CUDA;
        if (prop.major != 10) return PRQ_ERR_UNSUPPORTED_ARCH;
        d.num_sms = prop.multiProcessorCount;
        // the address of a __device__ variable belongs to the device that is current during the look-up
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess) return PRQ_ERR_CUDA;
        if (cur != dev && cudaSetDevice(dev) != cudaSuccess) return PRQ_ERR_CUDA;
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_device_status);
        if (cur != dev) cudaSetDevice(cur);
        if (e != cudaSuccess) return PRQ_ERR_CUDA;
        d.status_ptr = static_cast<int*>(p);
        d.ok = true;
    }
    *out = &d;
    return PRQ_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Packed E2M1 codes are plain bytes: a row-major (rows x row_bytes) byte matrix, boxes of 128 bytes
// (256 codes, one swizzle row) x box_rows rows, 128-byte swizzle, zero fill outside the matrix.
prq_status make_code_map(CUtensorMap* map, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PRQ_ERR_CUDA;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PRQ_OK : PRQ_ERR_CUDA;
}

// Scale bytes in the tensor-core layout are a flat array of 1024-byte groups; seen as rows of 256 bytes,
// a box of 4 rows is one group.  No swizzle: the bytes land in shared memory in array order.
prq_status make_sf_map(CUtensorMap* map, const void* base, uint64_t total_bytes, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PRQ_ERR_CUDA;
    cuuint64_t dims[2] = {256, total_bytes / 256};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {256, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PRQ_OK : PRQ_ERR_CUDA;
}

// Output matrix for the epilogue's TMA stores: boxes of 32 columns x 32 rows (128-byte rows with the
// 128-byte swizzle for fp32, 64-byte rows with the 64-byte swizzle for bf16).
prq_status make_out_map(CUtensorMap* map, void* y, int M, int N, int ldy, bool bf16) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PRQ_ERR_CUDA;
    const uint64_t es = bf16 ? 2 : 4;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldy) * es};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, y, dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PRQ_OK : PRQ_ERR_CUDA;
}

constexpr int kNumAlt = 4;
// weight tile widths of the prefill kernel, each with its own scale layout; the last one only in gated-producer handles,
// which in turn have none of the others
// (the one-wave tile is tiled per 144-row half: its two MMAs per step take 144 columns each)
constexpr int kAltTileRows[kNumAlt] = {kPrefillTileN, kPrefillTileWide, kPrefillTileOneWave / 2, kPrefillTileGated};
constexpr int kAltGated = 3;
bool alt_wanted(bool gated, int a) { return gated ? a == kAltGated : a != kAltGated; }

// Weight-side tensor maps of a dense handle, encoded once at creation (cloning re-encodes: other addresses).
prq_status build_weight_maps(prq_weights* w) {
    w->maps_ready = false;
    if (w->n_experts != 1) return PRQ_OK;
    const uint64_t Ka = static_cast<uint64_t>(w->K) + w->k_tail;
    prq_status st = make_code_map(&w->tm_w_decode, w->d_codes, Ka / 2, w->N, 128);
    for (int v = 0; v < kNumAlt; ++v) {   // 224-, 240- and 288-row tilings, or the 192-row one
        if (!alt_wanted(w->gated, v)) continue;
        const int rows = kAltTileRows[v], gpt = (rows + kGroupRows - 1) / kGroupRows;
        const bool one_wave = v == 2;   // a 288-row tile = two 144-row halves: boxes of 72 weight rows, four scale groups
        // each CTA of a pair loads half a tile (the 288-row tile: a quarter, twice)
        if (st == PRQ_OK) st = make_code_map(&w->tm_w_pair[v], w->d_codes, Ka / 2, w->N, rows / 2);
        if (st == PRQ_OK && w->d_sf_alt[v])
            st = make_sf_map(&w->tm_sfw_pair[v], w->d_sf_alt[v],
                             static_cast<uint64_t>(w->plan.S) * w->w_groups_alt[v] * kSfGroupBytes, 4 * gpt * (one_wave ? 2 : 1));
    }
    if (st == PRQ_OK) w->maps_ready = true;
    return st;
}

int env_int(const char* name, int dflt) {
    if (!dev_knobs_enabled()) return dflt;
    const char* v = std::getenv(name);
    return v && *v ? std::atoi(v) : dflt;
}

// Developer aid: PRQ_TRACE_PTR holds the address of a device buffer (4 x 512 int64) that the GEMM
// fills with clock stamps.  Unset in normal use.
long long* trace_ptr() {
    if (!dev_knobs_enabled()) return nullptr;
    const char* v = std::getenv("PRQ_TRACE_PTR");
    return v && *v ? reinterpret_cast<long long*>(std::strtoull(v, nullptr, 0)) : nullptr;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Online calls launch on the current device with pointers and tensor maps of the handle's device.
bool handle_device_is_current(const prq_weights* w) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == w->device;
}

int dense_groups(int M) { return (M + kGroupRows - 1) / kGroupRows; }
// Scale groups of a grouped buffer: every expert's rows are padded to whole 128-row groups, which costs at most
// one group per expert; a single expert needs exactly the dense count, so that the two layouts coincide.
int grouped_groups(int M, int n_groups) { return n_groups == 1 ? dense_groups(M) : (M + kGroupRows - 1) / kGroupRows + n_groups; }

int decode_bn(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128; }

// Cluster size (= number of K-splits) of the decode kernel: the one that puts the most SMs to work in
// the first wave, given how many clusters of each size the device can hold at once.
int decode_splits_for(int n_tiles, int S, int M, DeviceInfo* di) {
    const int bn = decode_bn(M);
    const int bi = bn == 16 ? 0 : bn == 32 ? 1 : bn == 64 ? 2 : 3;
    const int forced = env_int("PRQ_DECODE_SPLITS", 0);
    const int limit = std::min(8, S);
    if (forced > 0) return std::min(forced, limit);
    if (bn <= 32) {
        // Up to 32 tokens two CTAs share an SM, and a few clusters more than fit at once cost less than
        // a longer reduction per CTA does (measured at 20 tiles: 8 splits beat 6 at every token count):
        // the largest cluster that oversubscribes the SMs by at most a fifth.
        int best = 1;
        for (int s = 1; s <= limit; ++s)
            if (static_cast<long long>(n_tiles) * s * 5 <= static_cast<long long>(di->num_sms) * 6) best = s;
        return best;
    }
    int best = 1, best_ctas = 0;
    for (int s = 1; s <= limit; ++s) {
        int mc;
        {
            std::lock_guard<std::mutex> lock(g_dev_mutex);
            if (di->max_clusters[bi][s] == 0) di->max_clusters[bi][s] = std::max(1, decode_max_active_clusters(bn, s));
            mc = di->max_clusters[bi][s];
        }
        const int ctas = std::min(n_tiles, mc) * s;
        const bool one_wave = mc >= n_tiles;
        // prefer configurations that fit in one wave; among them the most CTAs
        const int score = ctas + (one_wave ? 100000 : 0);
        if (score > best_ctas) { best_ctas = score; best = s; }
    }
    return best;
}

int decode_splits(const prq_weights* w, int M, DeviceInfo* di) {
    return decode_splits_for((w->N + 127) / 128, w->plan.S, M, di);
}


// How the pair kernel shares out the tiles of one call: every pair gets `whole` whole tiles; the `sk`
// tiles left over are each cut into equal pieces for `base` (the first `extra` tiles: base + 1)
// consecutive pairs.
struct PairSchedule {
    int bn, pairs;
    long long tiles, whole, sk;
    int base, extra;
    long long stages_per_pair;   // reduction stages of the busiest pair
};

PairSchedule pair_schedule(int bn, int M, int N, int S, int max_pairs) {
    PairSchedule ps = {};
    ps.bn = bn;
    ps.tiles = static_cast<long long>((M + 255) / 256) * ((N + bn - 1) / bn);
    ps.pairs = static_cast<int>(std::min<long long>(ps.tiles * S, max_pairs));
    if (ps.pairs < 1) return ps;
    ps.whole = ps.tiles / ps.pairs;
    ps.sk = ps.tiles - ps.whole * ps.pairs;
    if (env_int("PRQ_PURE_SK", 0)) { ps.whole = 0; ps.sk = ps.tiles; }
    // Pieces have at least `min_piece` stages: a piece costs a whole partial tile of traffic whatever its
    // length, so short reductions are cut into few pieces or not at all (the left-over tiles then go whole
    // to as many pairs) and the pairs left over sit that phase out.  (Cutting the unit space into equal
    // contiguous ranges, two pieces per pair, balances better on paper and measured worse: 47.7 vs 45.5 us
    // on the 4096-token down projection, 28.3 vs 20.0 us with 1024 tokens; PRQ_SK_RANGES=1 still selects it.)
    const long long min_piece = std::max(1, env_int("PRQ_SK_MIN_PIECE", 9));
    const long long cap = std::max<long long>(1, std::min<long long>(8, S / min_piece));
    ps.base = 1;
    if (ps.sk > 0) {
        ps.base = static_cast<int>(std::max<long long>(1, std::min<long long>(ps.pairs / ps.sk, cap)));
        ps.extra = ps.base >= 2 && ps.base == ps.pairs / ps.sk && ps.base < cap ? static_cast<int>(ps.pairs % ps.sk) : 0;
    }
    ps.stages_per_pair = ps.whole * S + (ps.sk > 0 ? (S + ps.base - 1) / ps.base : 0);
    return ps;
}

// Tile width of the pair kernel: the main loop is bound by the operand bytes an SM takes in per stage
// (33792 with 224-column tiles, 34816 with 240-column ones), so the width whose busiest pair takes in
// fewer bytes wins; 224 on a tie.  With the paper's down projection that is 240 from 2048 tokens on
// (11 instead of 12 column tiles) and 224 below (the tile counts do not fill the pairs either way).
// Third width, 288 columns with a single accumulator: only where every tile of the call fits ONE wave of pairs at
// that width while the narrower tilings would leave tiles over (so that they need a second wave or stream-K
// pieces).  Every pair then runs one tile's reduction and one epilogue, nothing is published or fixed up.  The
// paper's down projection at 2048 tokens is such a call: 8 x 9 = 72 tiles on 74 pairs instead of 88 tiles of which
// 14 are cut into four pieces.
PairSchedule choose_pair_schedule(int M, int N, int S, int max_pairs) {
    const PairSchedule narrow = pair_schedule(kPrefillTileN, M, N, S, max_pairs);
    const PairSchedule wide = pair_schedule(kPrefillTileWide, M, N, S, max_pairs);
    const PairSchedule one = pair_schedule(kPrefillTileOneWave, M, N, S, max_pairs);
    const bool one_ok = one.tiles <= max_pairs && one.whole == 0 && one.base == 1 && one.extra == 0;
    const int forced = env_int("PRQ_PAIR_BN", 0);
    if (forced == kPrefillTileN) return narrow;
    if (forced == kPrefillTileWide) return wide;
    if (forced == kPrefillTileOneWave && one_ok) return one;
    const PairSchedule best = wide.stages_per_pair * 34816 < narrow.stages_per_pair * 33792 ? wide : narrow;
    if (one_ok && forced == 0 && best.stages_per_pair > S) return one;
    return best;
}

// Two counters ("arrived", "finished") per 128-row half of a 256 x 224 pair tile: first all the "arrived"
// counters, then all the "finished" ones.
size_t prefill_flag_count(const prq_weights* w, int M) {
    return 2 * static_cast<size_t>((M + 255) / 256) * ((w->N + kPrefillTileN - 1) / kPrefillTileN);
}
size_t prefill_flag_bytes(const prq_weights* w, int M) {
    return (2 * prefill_flag_count(w, M) * sizeof(int) + 255) & ~static_cast<size_t>(255);
}

}  // namespace
}  // namespace prq

using namespace prq;

extern "C" {

const char* prq_status_string(prq_status s) {
    switch (s) {
        case PRQ_OK: return "ok";
        case PRQ_ERR_INVALID_ARG: return "invalid argument";
        case PRQ_ERR_ALIGNMENT: return "misaligned pointer or stride";
        case PRQ_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case PRQ_ERR_CUDA: return "CUDA runtime error";
        case PRQ_ERR_OOM: return "out of memory";
        case PRQ_ERR_TIMEOUT: return "a device-side wait expired";
        case PRQ_ERR_NONFINITE: return "non-finite input";
        case PRQ_ERR_WORKSPACE: return "workspace too small";
        case PRQ_ERR_STATIC_SCRATCH: return "problem exceeds the library's built-in scratch (too many output tiles or SMs)";
    }
    return "unknown status";
}

unsigned long long prq_kernel_launch_count(void) { return g_launches.load(); }

prq_status prq_mxf4_peak_probe(int n_mma, int* n_ctas, prq_stream_t stream) {
    if (n_mma < 4 || n_mma > (1 << 24) || n_mma % 4) return PRQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PRQ_ERR_CUDA;
    DeviceInfo* di;
    prq_status st = device_info(dev, &di);
    if (st != PRQ_OK) return st;
    if (n_ctas) *n_ctas = di->num_sms;
    cudaError_t e = launch_mxf4_peak_probe(n_mma, di->num_sms, di->status_ptr, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_handover_probe(int n, int grid, int threads, int cluster, prq_stream_t stream) {
    if (n < 1 || n > 4096 || grid < 1 || threads < 32 || threads > 1024 || cluster < 1 || cluster > 8 || grid % cluster)
        return PRQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PRQ_ERR_CUDA;
    DeviceInfo* di;
    prq_status st = device_info(dev, &di);
    if (st != PRQ_OK) return st;
    void* sink = nullptr;
    if (cudaGetSymbolAddress(&sink, g_probe_sink) != cudaSuccess) return PRQ_ERR_CUDA;
    cudaError_t e = launch_handover_probe(n, grid, threads, cluster, static_cast<int*>(sink), static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(n);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_last_device_status(prq_stream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PRQ_ERR_CUDA;
    DeviceInfo* di;
    prq_status st = device_info(dev, &di);
    if (st != PRQ_OK) return st;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PRQ_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, di->status_ptr, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PRQ_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        cudaMemcpy(di->status_ptr, &zero, sizeof(int), cudaMemcpyHostToDevice);
    }
    return static_cast<prq_status>(v);
}

void prq_weights_free(prq_weights* w) {
    if (!w) return;
    int cur = 0;
    cudaGetDevice(&cur);
    if (w->device >= 0 && w->device != cur) cudaSetDevice(w->device);
    cudaFree(w->d_codes);
    cudaFree(w->d_sf);
    cudaFree(w->d_perm);
    cudaFree(w->d_inv_s_perm);
    cudaFree(w->d_inv_s);
    for (uint8_t* p : w->d_sf_alt) cudaFree(p);
    if (w->device >= 0 && w->device != cur) cudaSetDevice(cur);
    delete w;
}

prq_status prq_prepare_weights(const uint16_t* W, int n_experts, int N, int K, const float* act_amax, float alpha,
                               int k_tail, prq_weights** out) {
    return prq_prepare_weights_opts(W, n_experts, N, K, act_amax, alpha, k_tail, nullptr, out);
}

static prq_status create_handle(const uint16_t* W, bool w_on_device, prq_stream_t stream, int n_experts, int N, int K,
                                const float* act_amax, float alpha, int k_tail, const prq_prep_opts* opts, prq_weights** out);

prq_status prq_prepare_weights_opts(const uint16_t* W, int n_experts, int N, int K, const float* act_amax, float alpha,
                                    int k_tail, const prq_prep_opts* opts, prq_weights** out) {
    return create_handle(W, false, nullptr, n_experts, N, K, act_amax, alpha, k_tail, opts, out);
}

prq_status prq_prepare_weights_stacked(const uint16_t* const* Ws, const int* Ns, int n, int K, const float* act_amax, float alpha,
                                       int k_tail, const prq_prep_opts* opts, prq_weights** out) {
    if (!Ws || !Ns || n < 1 || K < kBlock) return PRQ_ERR_INVALID_ARG;
    long long N = 0;
    for (int i = 0; i < n; ++i) {
        if (!Ws[i] || Ns[i] < 1) return PRQ_ERR_INVALID_ARG;
        N += Ns[i];
    }
    if (N > 0x7fffffffll) return PRQ_ERR_INVALID_ARG;
    try {
        std::vector<uint16_t> W(static_cast<size_t>(N) * K);
        size_t row = 0;
        for (int i = 0; i < n; ++i) {
            std::memcpy(&W[row * K], Ws[i], sizeof(uint16_t) * static_cast<size_t>(Ns[i]) * K);
            row += Ns[i];
        }
        return create_handle(W.data(), false, nullptr, 1, static_cast<int>(N), K, act_amax, alpha, k_tail, opts, out);
    } catch (const std::bad_alloc&) {
        return PRQ_ERR_OOM;
    }
}

prq_status prq_prepare_weights_device(const uint16_t* W_device, int n_experts, int N, int K, const float* act_amax,
                                      float alpha, int k_tail, const prq_prep_opts* opts, prq_stream_t stream,
                                      prq_weights** out) {
    return create_handle(W_device, true, stream, n_experts, N, K, act_amax, alpha, k_tail, opts, out);
}

// Options as this version of the library understands them; a caller built against an earlier header passes a shorter
// struct, whose missing fields read as zero.
struct PrepOptions { bool scale_search = false, gated = false; int format = PRQ_FMT_MXFP4; bool valid = true; };
static PrepOptions read_opts(const prq_prep_opts* opts) {
    PrepOptions o;
    if (!opts) return o;
    if (opts->struct_size < 16) { o.valid = false; return o; }
    o.scale_search = opts->weight_scale_search != 0;
    if (opts->struct_size >= offsetof(prq_prep_opts, gated_producer) + sizeof(int)) o.gated = opts->gated_producer != 0;
    if (opts->struct_size >= offsetof(prq_prep_opts, format) + sizeof(int)) o.format = opts->format;
    if (o.format != PRQ_FMT_MXFP4 && o.format != PRQ_FMT_MXFP8) o.valid = false;
    return o;
}

static prq_status create_handle_fp8(const uint16_t* W, int N, int K, const float* act_amax, float alpha, int dev, prq_weights** out);

static prq_status create_handle(const uint16_t* W, bool w_on_device, prq_stream_t stream, int n_experts, int N, int K,
                                const float* act_amax, float alpha, int k_tail, const prq_prep_opts* opts, prq_weights** out) {
    const PrepOptions po = read_opts(opts);
    if (!po.valid) return PRQ_ERR_INVALID_ARG;
    const bool scale_search = po.scale_search;
    const bool gated = po.gated;
    if (po.format == PRQ_FMT_MXFP8) {
        // plain W8A8: no tail, no expert stack, no search; the preparation runs on the host
        if (k_tail != 0 || n_experts != 1 || scale_search || gated || w_on_device) return PRQ_ERR_INVALID_ARG;
        if (!W || !act_amax || !out || N < 1 || K < kBlock || K % kBlock || !std::isfinite(alpha)) return PRQ_ERR_INVALID_ARG;
        int dev8 = 0;
        if (cudaGetDevice(&dev8) != cudaSuccess) return PRQ_ERR_CUDA;
        DeviceInfo* di8;
        prq_status st8 = device_info(dev8, &di8);
        if (st8 != PRQ_OK) return st8;
        return create_handle_fp8(W, N, K, act_amax, alpha, dev8, out);
    }
    if (!W || !act_amax || !out) return PRQ_ERR_INVALID_ARG;
    if (n_experts < 1 || n_experts > kMaxExperts || N < 1 || K < kBlock) return PRQ_ERR_INVALID_ARG;
    if (gated && (n_experts != 1 || N % 64)) return PRQ_ERR_INVALID_ARG;   // whole (gate, up) groups of 32 + 32 rows
    if (K % kBlock || k_tail % kBlock || k_tail < 0 || k_tail > K) return PRQ_ERR_INVALID_ARG;
    if (!std::isfinite(alpha)) return PRQ_ERR_INVALID_ARG;
    if (static_cast<long long>(n_experts) * N > 0x7fffffffll) return PRQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PRQ_ERR_CUDA;
    DeviceInfo* di;
    prq_status st = device_info(dev, &di);
    if (st != PRQ_OK) return st;

    prq_weights* w = new (std::nothrow) prq_weights;
    if (!w) return PRQ_ERR_OOM;
    w->n_experts = n_experts; w->N = N; w->K = K; w->k_tail = k_tail; w->alpha = alpha;
    w->plan = StagePlan(K, k_tail);
    w->w_groups = (N + kGroupRows - 1) / kGroupRows;
    w->device = dev;
    w->gated = gated;
    const size_t Ka = static_cast<size_t>(K) + k_tail;
    const size_t E = n_experts;
    try {
        w->h_codes.resize(E * N * Ka / 2);
        w->h_scales.resize(E * N * Ka / kBlock);
        w->h_perm.resize(E * K);
        w->h_s.resize(E * K);
        w->h_inv_s.resize(E * K);
        w->h_col_err.resize(E * K);
        const int S = w->plan.S, S1 = w->plan.S1, nb = kStageK / kBlock;
        // scale bytes in stage order, padded by a few groups so that a tile's bulk copy never runs off the end
        w->d_sf_bytes = (E * S * w->w_groups + 4) * kSfGroupBytes;
        std::vector<uint8_t> sf(w->d_sf_bytes, 0);
        std::vector<float> inv_s_perm(E * K);
        std::vector<uint8_t> sf_alt[kNumAlt];
        for (int a = 0; a < kNumAlt && E == 1; ++a) {
            if (!alt_wanted(gated, a)) continue;
            w->w_groups_alt[a] = ((N + kAltTileRows[a] - 1) / kAltTileRows[a]) * ((kAltTileRows[a] + kGroupRows - 1) / kGroupRows);
            sf_alt[a].assign((static_cast<size_t>(S) * w->w_groups_alt[a] + 4) * kSfGroupBytes, 0);
        }
        PrepResult r;
        for (size_t e = 0; e < E; ++e) {
            st = w_on_device ? prepare_layer_device(W + e * N * K, N, K, act_amax + e * K, alpha, k_tail, r, scale_search,
                                                     static_cast<cudaStream_t>(stream))
                             : prepare_layer(W + e * N * K, N, K, act_amax + e * K, alpha, k_tail, r, scale_search);
            if (st != PRQ_OK) { delete w; return st; }
            std::memcpy(&w->h_codes[e * N * Ka / 2], r.codes.data(), r.codes.size());
            std::memcpy(&w->h_scales[e * N * Ka / kBlock], r.scales.data(), r.scales.size());
            std::memcpy(&w->h_perm[e * K], r.perm.data(), sizeof(int32_t) * K);
            std::memcpy(&w->h_s[e * K], r.s.data(), sizeof(float) * K);
            std::memcpy(&w->h_inv_s[e * K], r.inv_s.data(), sizeof(float) * K);
            std::memcpy(&w->h_col_err[e * K], r.col_err.data(), sizeof(double) * K);
            for (int j = 0; j < K; ++j) inv_s_perm[e * K + j] = r.inv_s[r.perm[j]];
            const int nblk_main = K / kBlock, nblk = static_cast<int>(Ka / kBlock);
            for (int n = 0; n < N; ++n) {
                const uint8_t* srow = &r.scales[static_cast<size_t>(n) * nblk];
                const int g = n / kGroupRows, rr = n % kGroupRows;
                for (int b = 0; b < nblk; ++b) {
                    const int stage = b < nblk_main ? b / nb : S1 + (b - nblk_main) / nb;
                    const int bis = b < nblk_main ? b % nb : (b - nblk_main) % nb;
                    sf[((e * S + stage) * w->w_groups + g) * kSfGroupBytes + sf_offset_in_group(rr, bis)] = srow[b];
                    for (int a = 0; a < kNumAlt && E == 1; ++a) {
                        if (!alt_wanted(gated, a)) continue;
                        const int tile_rows = kAltTileRows[a], gpt = (tile_rows + kGroupRows - 1) / kGroupRows;
                        const int ga = (n / tile_rows) * gpt + (n % tile_rows) / kGroupRows;
                        sf_alt[a][(static_cast<size_t>(stage) * w->w_groups_alt[a] + ga) * kSfGroupBytes +
                                  sf_offset_in_group((n % tile_rows) % kGroupRows, bis)] = srow[b];
                    }
                }
            }
        }
        w->d_codes_bytes = w->h_codes.size() + 256;
        if (cudaMalloc(&w->d_codes, w->d_codes_bytes) != cudaSuccess || cudaMalloc(&w->d_sf, w->d_sf_bytes) != cudaSuccess ||
            cudaMalloc(&w->d_perm, sizeof(int32_t) * E * K) != cudaSuccess ||
            cudaMalloc(&w->d_inv_s_perm, sizeof(float) * E * K) != cudaSuccess) {
            cudaGetLastError();
            prq_weights_free(w);
            return PRQ_ERR_OOM;
        }
        bool ok = cudaMemcpy(w->d_codes, w->h_codes.data(), w->h_codes.size(), cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(w->d_sf, sf.data(), sf.size(), cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(w->d_perm, w->h_perm.data(), sizeof(int32_t) * E * K, cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(w->d_inv_s_perm, inv_s_perm.data(), sizeof(float) * E * K, cudaMemcpyHostToDevice) == cudaSuccess;
        for (int a = 0; a < kNumAlt && E == 1 && ok; ++a) {
            if (!alt_wanted(gated, a)) continue;
            if (cudaMalloc(&w->d_sf_alt[a], sf_alt[a].size()) != cudaSuccess) {
                cudaGetLastError();
                prq_weights_free(w);
                return PRQ_ERR_OOM;
            }
            ok = cudaMemcpy(w->d_sf_alt[a], sf_alt[a].data(), sf_alt[a].size(), cudaMemcpyHostToDevice) == cudaSuccess;
        }
        if (!ok) { prq_weights_free(w); return PRQ_ERR_CUDA; }
        if (build_weight_maps(w) != PRQ_OK) { prq_weights_free(w); return PRQ_ERR_CUDA; }
    } catch (const std::bad_alloc&) {
        prq_weights_free(w);
        return PRQ_ERR_OOM;
    }
    *out = w;
    return PRQ_OK;
}

// Second format: host preparation, scale bytes in [128-element stage][128-row group][512], one upload.
static prq_status create_handle_fp8(const uint16_t* W, int N, int K, const float* act_amax, float alpha, int dev, prq_weights** out) {
    prq_weights* w = new (std::nothrow) prq_weights;
    if (!w) return PRQ_ERR_OOM;
    w->n_experts = 1; w->N = N; w->K = K; w->k_tail = 0; w->alpha = alpha;
    w->plan = StagePlan(K, 0);
    w->w_groups = (N + kGroupRows - 1) / kGroupRows;
    w->device = dev;
    w->format = PRQ_FMT_MXFP8;
    try {
        prq_status st = prepare_layer_fp8(W, N, K, act_amax, alpha, w->h_s, w->h_inv_s, w->h_codes, w->h_scales);
        if (st != PRQ_OK) { delete w; return st; }
        w->h_perm.resize(K);
        for (int j = 0; j < K; ++j) w->h_perm[j] = j;
        w->h_col_err.assign(K, 0.0);
        const int S8 = (K + 127) / 128, nblk = K / kBlock;
        w->d_sf_bytes = (static_cast<size_t>(S8) * w->w_groups + 4) * 512;
        std::vector<uint8_t> sf(w->d_sf_bytes, 0);
        for (int n = 0; n < N; ++n)
            for (int b = 0; b < nblk; ++b)
                sf[(static_cast<size_t>(b / 4) * w->w_groups + n / kGroupRows) * 512 + sf_offset_in_group(n % kGroupRows, b % 4)] =
                    w->h_scales[static_cast<size_t>(n) * nblk + b];
        w->d_codes_bytes = w->h_codes.size() + 256;
        if (cudaMalloc(&w->d_codes, w->d_codes_bytes) != cudaSuccess || cudaMalloc(&w->d_sf, w->d_sf_bytes) != cudaSuccess ||
            cudaMalloc(&w->d_inv_s, sizeof(float) * K) != cudaSuccess) {
            cudaGetLastError();
            prq_weights_free(w);
            return PRQ_ERR_OOM;
        }
        bool ok = cudaMemcpy(w->d_codes, w->h_codes.data(), w->h_codes.size(), cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(w->d_sf, sf.data(), sf.size(), cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(w->d_inv_s, w->h_inv_s.data(), sizeof(float) * K, cudaMemcpyHostToDevice) == cudaSuccess;
        if (!ok || make_code_map(&w->tm_w_fp8, w->d_codes, static_cast<uint64_t>(K), N, 128) != PRQ_OK) {
            prq_weights_free(w);
            return PRQ_ERR_CUDA;
        }
        w->maps_ready = true;
    } catch (const std::bad_alloc&) {
        prq_weights_free(w);
        return PRQ_ERR_OOM;
    }
    *out = w;
    return PRQ_OK;
}

prq_status prq_weights_format(const prq_weights* w, int* format) {
    if (!w || !format) return PRQ_ERR_INVALID_ARG;
    *format = w->format;
    return PRQ_OK;
}

size_t prq_act_bytes_for(const prq_weights* w, int M, prq_buf which) {
    if (!w || M < 0 || w->n_experts != 1) return 0;
    if (w->format == PRQ_FMT_MXFP4) return prq_act_bytes(M, w->K, w->k_tail, 1, which);
    switch (which) {
        case PRQ_BUF_CODES: return static_cast<size_t>(M) * w->K;
        case PRQ_BUF_SCALES_ROW: return static_cast<size_t>(M) * w->K / kBlock;
        case PRQ_BUF_SCALES_SF: return static_cast<size_t>((w->K + 127) / 128) * std::max(dense_groups(M), 1) * 512;
    }
    return 0;
}

prq_status prq_prepare_weights_search(const uint16_t* W, int N, int K, const uint16_t* Zcal, int T, const float* alphas,
                                      int n_alphas, int k_tail, prq_weights** out, float* alpha_star, double* nrmse) {
    if (!W || !Zcal || !alphas || !out || !alpha_star || T < 1 || n_alphas < 1) return PRQ_ERR_INVALID_ARG;
    if (N < 1 || K < kBlock || K % kBlock || k_tail % kBlock || k_tail < 0 || k_tail > K) return PRQ_ERR_INVALID_ARG;
    auto bf = [](uint16_t h) { uint32_t u = static_cast<uint32_t>(h) << 16; float f; std::memcpy(&f, &u, 4); return f; };
    // step 1: per-channel maxima of the calibration activations
    std::vector<float> amax(K, 0.f);
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < K; ++j) amax[j] = std::max(amax[j], std::fabs(bf(Zcal[static_cast<size_t>(t) * K + j])));
    // the target Z W^T in double, rows split over host threads
    std::vector<double> yref(static_cast<size_t>(T) * N);
    {
        std::vector<double> Wd(static_cast<size_t>(N) * K);
        for (size_t i = 0; i < Wd.size(); ++i) Wd[i] = bf(W[i]);
        unsigned nt = std::max(1u, std::min(std::thread::hardware_concurrency(), 64u));
        std::vector<std::thread> th;
        for (unsigned ti = 0; ti < nt; ++ti)
            th.emplace_back([&, ti] {
                std::vector<double> z(K);
                for (int t = ti; t < T; t += nt) {
                    for (int j = 0; j < K; ++j) z[j] = bf(Zcal[static_cast<size_t>(t) * K + j]);
                    for (int n = 0; n < N; ++n) {
                        const double* wr = &Wd[static_cast<size_t>(n) * K];
                        double acc = 0.0;
                        for (int j = 0; j < K; ++j) acc += z[j] * wr[j];
                        yref[static_cast<size_t>(t) * N + n] = acc;
                    }
                }
            });
        for (auto& x : th) x.join();
    }
    double ref_norm2 = 0.0;
    for (double v : yref) ref_norm2 += v * v;

    const size_t x_bytes = static_cast<size_t>(T) * K * 2;
    const size_t c_bytes = prq_act_bytes(T, K, k_tail, 1, PRQ_BUF_CODES);
    const size_t sf_bytes = prq_act_bytes(T, K, k_tail, 1, PRQ_BUF_SCALES_SF);
    const size_t y_bytes = static_cast<size_t>(T) * N * 4;
    void *dx = nullptr, *dc = nullptr, *dsf = nullptr, *dy = nullptr, *dws = nullptr;
    size_t ws_bytes = 0;
    std::vector<float> y(static_cast<size_t>(T) * N);
    prq_weights* best = nullptr;
    double best_err = 0.0;
    prq_status st = PRQ_OK;
    // the per-alpha pipeline runs on the device from one upload of W (bit-identical to the host path)
    uint16_t* dW = nullptr;
    const size_t w_bytes = sizeof(uint16_t) * static_cast<size_t>(N) * K;
    if (cudaMalloc(&dW, w_bytes) != cudaSuccess) { cudaGetLastError(); return PRQ_ERR_OOM; }
    if (cudaMemcpy(dW, W, w_bytes, cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(dW); return PRQ_ERR_CUDA; }
    for (int a = 0; a < n_alphas && st == PRQ_OK; ++a) {
        prq_weights* w = nullptr;
        st = prq_prepare_weights_device(dW, 1, N, K, amax.data(), alphas[a], k_tail, nullptr, nullptr, &w);
        if (st != PRQ_OK) break;
        if (!dx) {
            ws_bytes = prq_linear_workspace_bytes(w, T);
            bool ok = cudaMalloc(&dx, x_bytes) == cudaSuccess && cudaMalloc(&dc, c_bytes) == cudaSuccess &&
                      cudaMalloc(&dsf, sf_bytes) == cudaSuccess && cudaMalloc(&dy, y_bytes) == cudaSuccess &&
                      cudaMalloc(&dws, ws_bytes) == cudaSuccess;
            ok = ok && cudaMemset(dws, 0, ws_bytes) == cudaSuccess;
            ok = ok && cudaMemcpy(dx, Zcal, x_bytes, cudaMemcpyHostToDevice) == cudaSuccess;
            if (!ok) { cudaGetLastError(); prq_weights_free(w); st = PRQ_ERR_OOM; break; }
        }
        st = prq_quantize_act(w, PRQ_ACT_SCALE_PERM, dx, T, K, nullptr, dc, nullptr, dsf, nullptr);
        if (st == PRQ_OK) st = prq_linear(w, dc, dsf, T, dy, N, PRQ_F32, dws, ws_bytes, nullptr);
        if (st == PRQ_OK) st = prq_last_device_status(nullptr);
        if (st == PRQ_OK && cudaMemcpy(y.data(), dy, y_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) st = PRQ_ERR_CUDA;
        if (st != PRQ_OK) { prq_weights_free(w); break; }
        double d2 = 0.0;
        for (size_t i = 0; i < y.size(); ++i) { const double d = static_cast<double>(y[i]) - yref[i]; d2 += d * d; }
        const double err = std::sqrt(d2 / ref_norm2);
        if (nrmse) nrmse[a] = err;
        if (!best || err < best_err) {
            prq_weights_free(best);
            best = w; best_err = err; *alpha_star = alphas[a];
        } else {
            prq_weights_free(w);
        }
    }
    cudaFree(dx); cudaFree(dc); cudaFree(dsf); cudaFree(dy); cudaFree(dws); cudaFree(dW);
    if (st != PRQ_OK) { prq_weights_free(best); return st; }
    *out = best;
    return PRQ_OK;
}

prq_status prq_prepare_weights_host(const uint16_t* W, int N, int K, const float* act_amax, float alpha, int k_tail,
                                    uint8_t* codes, uint8_t* scales, int32_t* perm, float* s_out, float* inv_s_out,
                                    double* col_err) {
    return prq_prepare_weights_host_opts(W, N, K, act_amax, alpha, k_tail, nullptr, codes, scales, perm, s_out,
                                         inv_s_out, col_err);
}

prq_status prq_prepare_weights_host_opts(const uint16_t* W, int N, int K, const float* act_amax, float alpha,
                                         int k_tail, const prq_prep_opts* opts, uint8_t* codes, uint8_t* scales,
                                         int32_t* perm, float* s_out, float* inv_s_out, double* col_err) {
    const PrepOptions po = read_opts(opts);
    if (!po.valid) return PRQ_ERR_INVALID_ARG;
    const bool scale_search = po.scale_search;
    if (!W || !act_amax || !codes || !scales || !perm) return PRQ_ERR_INVALID_ARG;
    if (po.format == PRQ_FMT_MXFP8) {
        // second format: codes N x K bytes, scales N x K/32, identity permutation, no ranking
        if (N < 1 || K < kBlock || K % kBlock || k_tail != 0 || scale_search || !std::isfinite(alpha)) return PRQ_ERR_INVALID_ARG;
        try {
            std::vector<float> s8, inv8;
            std::vector<uint8_t> c8, sc8;
            prq_status st8 = prepare_layer_fp8(W, N, K, act_amax, alpha, s8, inv8, c8, sc8);
            if (st8 != PRQ_OK) return st8;
            std::memcpy(codes, c8.data(), c8.size());
            std::memcpy(scales, sc8.data(), sc8.size());
            for (int j = 0; j < K; ++j) perm[j] = j;
            if (s_out) std::memcpy(s_out, s8.data(), sizeof(float) * K);
            if (inv_s_out) std::memcpy(inv_s_out, inv8.data(), sizeof(float) * K);
            if (col_err) std::fill(col_err, col_err + K, 0.0);
        } catch (const std::bad_alloc&) {
            return PRQ_ERR_OOM;
        }
        return PRQ_OK;
    }
    if (N < 1 || K < kBlock || K % kBlock || k_tail % kBlock || k_tail < 0 || k_tail > K) return PRQ_ERR_INVALID_ARG;
    if (!std::isfinite(alpha)) return PRQ_ERR_INVALID_ARG;
    PrepResult r;
    try {
        prq_status st = prepare_layer(W, N, K, act_amax, alpha, k_tail, r, scale_search);
        if (st != PRQ_OK) return st;
    } catch (const std::bad_alloc&) {
        return PRQ_ERR_OOM;
    }
    std::memcpy(codes, r.codes.data(), r.codes.size());
    std::memcpy(scales, r.scales.data(), r.scales.size());
    std::memcpy(perm, r.perm.data(), sizeof(int32_t) * K);
    if (s_out) std::memcpy(s_out, r.s.data(), sizeof(float) * K);
    if (inv_s_out) std::memcpy(inv_s_out, r.inv_s.data(), sizeof(float) * K);
    if (col_err) std::memcpy(col_err, r.col_err.data(), sizeof(double) * K);
    return PRQ_OK;
}

prq_status prq_weights_clone(const prq_weights* w, prq_weights** out) {
    if (!w || !out || w->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
    prq_weights* c = new (std::nothrow) prq_weights;
    if (!c) return PRQ_ERR_OOM;
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != w->device) cudaSetDevice(w->device);
    prq_status st = PRQ_OK;
    try {
        c->n_experts = w->n_experts; c->N = w->N; c->K = w->K; c->k_tail = w->k_tail; c->alpha = w->alpha;
        c->plan = w->plan; c->w_groups = w->w_groups; c->device = w->device; c->gated = w->gated;
        c->h_codes = w->h_codes; c->h_scales = w->h_scales; c->h_perm = w->h_perm;
        c->h_s = w->h_s; c->h_inv_s = w->h_inv_s; c->h_col_err = w->h_col_err;
        c->d_codes_bytes = w->d_codes_bytes; c->d_sf_bytes = w->d_sf_bytes;
        const size_t EK = static_cast<size_t>(w->n_experts) * w->K;
        auto dup = [&](void* dst_pp, const void* src, size_t bytes) {
            void** pp = static_cast<void**>(dst_pp);
            if (st != PRQ_OK || !src) return;
            if (cudaMalloc(pp, bytes) != cudaSuccess) { cudaGetLastError(); st = PRQ_ERR_OOM; return; }
            if (cudaMemcpy(*pp, src, bytes, cudaMemcpyDeviceToDevice) != cudaSuccess) st = PRQ_ERR_CUDA;
        };
        dup(&c->d_codes, w->d_codes, w->d_codes_bytes);
        dup(&c->d_sf, w->d_sf, w->d_sf_bytes);
        dup(&c->d_perm, w->d_perm, sizeof(int32_t) * EK);
        dup(&c->d_inv_s_perm, w->d_inv_s_perm, sizeof(float) * EK);
        for (int a = 0; a < kNumAlt; ++a) {
            c->w_groups_alt[a] = w->w_groups_alt[a];
            if (w->d_sf_alt[a])
                dup(&c->d_sf_alt[a], w->d_sf_alt[a], (static_cast<size_t>(w->plan.S) * w->w_groups_alt[a] + 4) * kSfGroupBytes);
        }
    } catch (const std::bad_alloc&) {
        st = PRQ_ERR_OOM;
    }
    if (st == PRQ_OK) st = build_weight_maps(c);
    if (cur != w->device) cudaSetDevice(cur);
    if (st != PRQ_OK) { prq_weights_free(c); return st; }
    *out = c;
    return PRQ_OK;
}

prq_status prq_weights_offline_copy(const prq_weights* w, prq_weights** out) {
    if (!w || !out) return PRQ_ERR_INVALID_ARG;
    // [Q(W D P) | Q(R)] read as a plain matrix of K + k reduction columns has the stage order of this layer's
    // layout only if the residual stages start on a stage boundary
    if (w->k_tail > 0 && w->K % kStageK != 0) return PRQ_ERR_INVALID_ARG;
    prq_weights* c = nullptr;
    prq_status st = prq_weights_clone(w, &c);
    if (st != PRQ_OK) return st;
    const int Kw = w->K + w->k_tail;
    const size_t E = static_cast<size_t>(w->n_experts);
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != c->device) cudaSetDevice(c->device);
    try {
        c->K = Kw; c->k_tail = 0; c->plan = StagePlan(Kw, 0);
        // the activation arrives permuted, scaled and with its tail columns doubled: nothing is left to apply
        c->h_perm.resize(E * Kw);
        for (size_t e = 0; e < E; ++e)
            for (int j = 0; j < Kw; ++j) c->h_perm[e * Kw + j] = j;
        c->h_s.assign(E * Kw, 1.f);
        c->h_inv_s.assign(E * Kw, 1.f);
        c->h_col_err.assign(E * Kw, 0.0);
        cudaFree(c->d_perm); c->d_perm = nullptr;
        cudaFree(c->d_inv_s_perm); c->d_inv_s_perm = nullptr;
        bool ok = cudaMalloc(&c->d_perm, sizeof(int32_t) * E * Kw) == cudaSuccess &&
                  cudaMalloc(&c->d_inv_s_perm, sizeof(float) * E * Kw) == cudaSuccess;
        if (!ok) { cudaGetLastError(); st = PRQ_ERR_OOM; }
        ok = ok && cudaMemcpy(c->d_perm, c->h_perm.data(), sizeof(int32_t) * E * Kw, cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(c->d_inv_s_perm, c->h_inv_s.data(), sizeof(float) * E * Kw, cudaMemcpyHostToDevice) == cudaSuccess;
        if (!ok && st == PRQ_OK) st = PRQ_ERR_CUDA;
    } catch (const std::bad_alloc&) {
        st = PRQ_ERR_OOM;
    }
    if (st == PRQ_OK) st = build_weight_maps(c);
    if (cur != c->device) cudaSetDevice(cur);
    if (st != PRQ_OK) { prq_weights_free(c); return st; }
    *out = c;
    return PRQ_OK;
}

prq_status prq_fold_producer(const int32_t* perm, const float* inv_s, int C, int k_tail, const uint16_t* W_up,
                             const uint16_t* W_gate, int H, int duplicate_tail, uint16_t* out_up, uint16_t* out_gate) {
    if (!perm || !inv_s || !W_up || !out_up || C < 1 || H < 1 || k_tail < 0 || k_tail > C) return PRQ_ERR_INVALID_ARG;
    if ((W_gate == nullptr) != (out_gate == nullptr)) return PRQ_ERR_INVALID_ARG;
    return fold_producer(perm, inv_s, C, k_tail, W_up, W_gate, H, duplicate_tail != 0, out_up, out_gate);
}

prq_status prq_weights_info(const prq_weights* w, int* n_experts, int* N, int* K, int* k_tail, float* alpha) {
    if (!w) return PRQ_ERR_INVALID_ARG;
    if (n_experts) *n_experts = w->n_experts;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (k_tail) *k_tail = w->k_tail;
    if (alpha) *alpha = w->alpha;
    return PRQ_OK;
}

prq_status prq_weights_get(const prq_weights* w, int expert, prq_field which, void* dst, size_t dst_bytes) {
    if (!w || !dst || expert < 0 || expert >= w->n_experts) return PRQ_ERR_INVALID_ARG;
    const size_t Ka = static_cast<size_t>(w->K) + w->k_tail, N = w->N, K = w->K, e = expert;
    const void* src = nullptr;
    size_t bytes = 0;
    switch (which) {
        case PRQ_FIELD_CODES: bytes = w->format == PRQ_FMT_MXFP8 ? N * K : N * Ka / 2; src = &w->h_codes[e * bytes]; break;
        case PRQ_FIELD_SCALES: bytes = N * Ka / kBlock; src = &w->h_scales[e * bytes]; break;
        case PRQ_FIELD_PERM: bytes = K * sizeof(int32_t); src = &w->h_perm[e * K]; break;
        case PRQ_FIELD_TOPK: bytes = w->k_tail * sizeof(int32_t); src = w->h_perm.data() + e * K + (K - w->k_tail); break;
        case PRQ_FIELD_S: bytes = K * sizeof(float); src = &w->h_s[e * K]; break;
        case PRQ_FIELD_INV_S: bytes = K * sizeof(float); src = &w->h_inv_s[e * K]; break;
        case PRQ_FIELD_COL_ERR: bytes = K * sizeof(double); src = &w->h_col_err[e * K]; break;
        default: return PRQ_ERR_INVALID_ARG;
    }
    if (dst_bytes != bytes) return PRQ_ERR_INVALID_ARG;
    if (bytes) std::memcpy(dst, src, bytes);
    return PRQ_OK;
}

size_t prq_act_bytes(int M, int K, int k_tail, int n_groups, prq_buf which) {
    if (M < 0 || K < kBlock || K % kBlock || k_tail % kBlock || k_tail < 0 || k_tail > K || n_groups < 1) return 0;
    const StagePlan plan(K, k_tail);
    switch (which) {
        case PRQ_BUF_CODES: return static_cast<size_t>(M) * K / 2;
        case PRQ_BUF_SCALES_ROW: return static_cast<size_t>(M) * K / kBlock;
        case PRQ_BUF_SCALES_SF: {
            const int groups = n_groups == 1 ? dense_groups(M) : grouped_groups(M, n_groups);
            return static_cast<size_t>(plan.S) * std::max(groups, 1) * kSfGroupBytes;
        }
    }
    return 0;
}

prq_status prq_quantize_act(const prq_weights* w, prq_act_mode mode, const void* x, int M, int ldx,
                            const int32_t* expert_offsets, void* codes, void* scales_row, void* scales_sf,
                            prq_stream_t stream) {
    if (!w || M < 0) return PRQ_ERR_INVALID_ARG;
    if (mode != PRQ_ACT_IDENTITY && mode != PRQ_ACT_SCALE_PERM) return PRQ_ERR_INVALID_ARG;
    if (M == 0) return PRQ_OK;
    if (!x || !codes || !scales_sf || ldx < w->K) return PRQ_ERR_INVALID_ARG;
    if (w->format == PRQ_FMT_MXFP8) {
        if (expert_offsets) return PRQ_ERR_INVALID_ARG;
        if (!aligned16(x) || !aligned16(codes) || !aligned16(scales_sf) || ldx % 8) return PRQ_ERR_ALIGNMENT;
        if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
        cudaError_t e8 = launch_quant_act_fp8(static_cast<const uint16_t*>(x), M, ldx, w->K, mode == PRQ_ACT_SCALE_PERM ? w->d_inv_s : nullptr,
                                              static_cast<uint8_t*>(codes), static_cast<uint8_t*>(scales_row),
                                              static_cast<uint8_t*>(scales_sf), static_cast<cudaStream_t>(stream));
        g_launches.fetch_add(1);
        return e8 == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
    }
    // stacked experts need their row boundaries; a single layer may be given a two-entry offsets array too
    // (the grouped layout with one group), as prq_linear_grouped accepts it
    if (w->n_experts > 1 && expert_offsets == nullptr) return PRQ_ERR_INVALID_ARG;
    if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(codes) || !aligned16(scales_sf) || ldx % 8) return PRQ_ERR_ALIGNMENT;
    QuantParams p;
    p.x = static_cast<const uint16_t*>(x);
    p.M = M; p.ldx = ldx; p.K = w->K; p.k_tail = w->k_tail;
    p.n_experts = w->n_experts;
    p.expert_offsets = expert_offsets;
    p.act_groups = expert_offsets ? grouped_groups(M, w->n_experts) : dense_groups(M);
    p.perm = w->d_perm;
    p.inv_s_perm = w->d_inv_s_perm;
    p.codes = static_cast<uint8_t*>(codes);
    p.scales_row = static_cast<uint8_t*>(scales_row);
    p.scales_sf = static_cast<uint8_t*>(scales_sf);
    DeviceInfo* di;
    prq_status st = device_info(w->device, &di);
    if (st != PRQ_OK) return st;
    p.status = di->status_ptr;
    cudaError_t e = launch_quant_act(p, mode == PRQ_ACT_SCALE_PERM, p.act_groups, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_quantize_act_multi(int n, const prq_weights* const* ws, prq_act_mode mode, const void* x, int M, int ldx,
                                  void* const* codes, void* const* scales_sf, prq_stream_t stream) {
    if (n < 1 || n > PRQ_MULTI_MAX || !ws || !codes || !scales_sf || M < 0) return PRQ_ERR_INVALID_ARG;
    if (mode != PRQ_ACT_IDENTITY && mode != PRQ_ACT_SCALE_PERM) return PRQ_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i) {
        if (!ws[i] || ws[i]->n_experts != 1 || ws[i]->K != ws[0]->K || ws[i]->device != ws[0]->device) return PRQ_ERR_INVALID_ARG;
        if (ws[i]->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
        if (M > 0 && (!codes[i] || !scales_sf[i])) return PRQ_ERR_INVALID_ARG;
    }
    if (M == 0) return PRQ_OK;
    if (!x || ldx < ws[0]->K) return PRQ_ERR_INVALID_ARG;
    if (!handle_device_is_current(ws[0])) return PRQ_ERR_INVALID_ARG;
    if (!aligned16(x) || ldx % 8) return PRQ_ERR_ALIGNMENT;
    for (int i = 0; i < n; ++i)
        if (!aligned16(codes[i]) || !aligned16(scales_sf[i])) return PRQ_ERR_ALIGNMENT;
    QuantBatch b = {};
    b.x = static_cast<const uint16_t*>(x);
    b.M = M; b.ldx = ldx; b.K = ws[0]->K;
    b.n_experts = 1;
    b.act_groups = dense_groups(M);
    b.n_lin = n;
    b.groups_per_lin = b.act_groups;
    for (int i = 0; i < n; ++i)
        b.lay[i] = QuantLayer{ws[i]->d_perm, ws[i]->d_inv_s_perm, static_cast<uint8_t*>(codes[i]), nullptr,
                              static_cast<uint8_t*>(scales_sf[i]), ws[i]->k_tail};
    DeviceInfo* di;
    prq_status st = device_info(ws[0]->device, &di);
    if (st != PRQ_OK) return st;
    b.status = di->status_ptr;
    cudaError_t e = launch_quant_act_batch(b, mode == PRQ_ACT_SCALE_PERM, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

size_t prq_linear_workspace_bytes(const prq_weights* w, int M) {
    if (!w || M < 0) return 0;
    if (M > 128 && w->format == PRQ_FMT_MXFP4) {
        // stream-K prefill: one flag per 128 x 256 tile, one fp32 partial tile per CTA (at most one CTA per SM)
        DeviceInfo* di;
        if (device_info(w->device, &di) != PRQ_OK) return 0;
        return prefill_flag_bytes(w, M) + 2 * static_cast<size_t>(di->num_sms) * kPrefillSlotBytes;
    }
    return 0;  // decode: the split-K partial sums meet in distributed shared memory
}

static prq_status check_linear_common(const prq_weights* w, const void* codes, const void* scales_sf, void* y, int ldy,
                                      prq_dtype y_dtype) {
    if (!w || !codes || !scales_sf || !y) return PRQ_ERR_INVALID_ARG;
    if (y_dtype != PRQ_F32 && y_dtype != PRQ_BF16) return PRQ_ERR_INVALID_ARG;
    if (ldy < w->N) return PRQ_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(scales_sf) || !aligned16(y)) return PRQ_ERR_ALIGNMENT;
    if (ldy % (y_dtype == PRQ_F32 ? 4 : 8)) return PRQ_ERR_ALIGNMENT;
    return PRQ_OK;
}

prq_status prq_linear(const prq_weights* w, const void* codes, const void* scales_sf, int M, void* y, int ldy,
                      prq_dtype y_dtype, void* workspace, size_t workspace_bytes, prq_stream_t stream) {
    if (w && M == 0) return PRQ_OK;
    prq_status st = check_linear_common(w, codes, scales_sf, y, ldy, y_dtype);
    if (st != PRQ_OK) return st;
    if (M < 0 || w->n_experts != 1 || !w->maps_ready) return PRQ_ERR_INVALID_ARG;
    if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
    DeviceInfo* di;
    st = device_info(w->device, &di);
    if (st != PRQ_OK) return st;

    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.N = w->N; p.K = w->K; p.k_tail = w->k_tail;
    p.n_experts = 1;
    p.act_groups = dense_groups(M);
    if (w->format == PRQ_FMT_MXFP8) {
        // second format: the tile-per-CTA kernel (128 output features x 128 tokens) over the layer as one expert
        p.w_groups = w->w_groups;
        p.act_sf = static_cast<const uint8_t*>(scales_sf);
        p.w_sf = w->d_sf;
        p.y = y; p.ldy = ldy; p.y_bf16 = y_dtype == PRQ_BF16;
        p.status = di->status_ptr;
        CUtensorMap tm_act8;
        st = make_code_map(&tm_act8, codes, static_cast<uint64_t>(w->K), M, 128);
        if (st != PRQ_OK) return st;
        cudaError_t e8 = launch_gemm_fp8(tm_act8, w->tm_w_fp8, p, di->num_sms, static_cast<cudaStream_t>(stream));
        g_launches.fetch_add(1);
        return e8 == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
    }
    p.w_groups = w->w_groups;
    p.act_sf = static_cast<const uint8_t*>(scales_sf);
    p.w_sf = w->d_sf;
    p.y = y; p.ldy = ldy; p.y_bf16 = y_dtype == PRQ_BF16;
    p.status = di->status_ptr;
    p.trace = trace_ptr();
    p.dbg = env_int("PRQ_DBG", 0);

    CUtensorMap tm_act;
    if (M <= 128) {
        // weight-streaming kernel: weights on the MMA M axis, K split over a thread-block cluster
        DecodeParams q;
        std::memset(&q, 0, sizeof(q));
        q.M = M; q.N = w->N; q.K = w->K; q.k_tail = w->k_tail;
        q.w_groups = w->w_groups;
        q.act_sf = p.act_sf; q.w_sf = w->d_sf;
        q.y = y; q.ldy = ldy; q.y_bf16 = p.y_bf16;
        q.status = p.status; q.trace = p.trace; q.dbg = p.dbg;
        q.splits = decode_splits(w, M, di);
        const int bn = decode_bn(M);
        st = make_code_map(&tm_act, codes, w->K / 2, M, bn);
        if (st != PRQ_OK) return st;
        cudaError_t e = launch_decode(bn, tm_act, w->tm_w_decode, q, (w->N + 127) / 128, static_cast<cudaStream_t>(stream));
        g_launches.fetch_add(1);
        return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
    } else {
        // stream-K kernel on CTA pairs with 256 x 224 or 256 x 240 tiles (scale bytes grouped per weight tile)
        if (w->gated) return PRQ_ERR_INVALID_ARG;   // a gated-producer handle has the tiling of prq_linear_gated only
        PrefillParams q;
        std::memset(&q, 0, sizeof(q));
        if (di->max_pairs == 0)
            di->max_pairs = std::min(std::min(std::min(prefill_pair_max_clusters(kPrefillTileN), prefill_pair_max_clusters(kPrefillTileWide)),
                                              prefill_pair_max_clusters(kPrefillTileOneWave)), di->num_sms / 2);
        const PairSchedule ps = choose_pair_schedule(M, w->N, w->plan.S, std::min(di->max_pairs, env_int("PRQ_GRID", 1 << 20)));
        const int pair_bn = ps.bn, variant = pair_bn == kPrefillTileOneWave ? 2 : pair_bn == kPrefillTileWide ? 1 : 0, pairs = ps.pairs;
        if (pairs < 1) return PRQ_ERR_CUDA;
        q.M = M; q.N = w->N; q.K = w->K; q.k_tail = w->k_tail;
        q.m_tiles = (M + 255) / 256; q.n_tiles = (w->N + pair_bn - 1) / pair_bn;
        q.act_groups = p.act_groups; q.w_groups = w->w_groups_alt[variant];
        q.act_sf = p.act_sf; q.w_sf = w->d_sf_alt[variant];
        q.y = y; q.ldy = ldy;
        q.y_bf16 = p.y_bf16; q.status = p.status; q.trace = p.trace; q.dbg = p.dbg;
        // developer switch: a short limit lets a test watch a wait run out (cycles; default about two seconds)
        const int short_limit = env_int("PRQ_WAIT_LIMIT_CYCLES", 0);
        q.wait_limit = short_limit > 0 ? short_limit : kDefaultWaitLimitCycles;
        const size_t flag_bytes = prefill_flag_bytes(w, M);
        const long long tiles = ps.tiles, whole = ps.whole, sk = ps.sk;
        if (sk > 0 && !env_int("PRQ_SK_RANGES", 0)) {
            q.sk_aligned = 1;
            q.sk_base = ps.base;
            q.sk_extra = ps.extra;
        }
        q.sk_tiles = static_cast<int>(sk); q.whole_tiles = static_cast<int>(whole);
        q.total_tiles = static_cast<int>(tiles);
        if (sk * w->plan.S * pairs >= (1ll << 32) || tiles >= (1ll << 30)) return PRQ_ERR_INVALID_ARG;  // 32-bit range arithmetic
        if (!workspace || workspace_bytes < flag_bytes + static_cast<size_t>(4 * pairs) * kPrefillSlotBytes) return PRQ_ERR_WORKSPACE;
        q.flag_stride = static_cast<int>(prefill_flag_count(w, M));
        if (!aligned16(workspace)) return PRQ_ERR_ALIGNMENT;
        q.flags = static_cast<int*>(workspace);
        q.partial = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + flag_bytes);
        CUtensorMap tm_y, tm_sfa;
        const uint64_t Sg = static_cast<uint64_t>(w->plan.S);
        st = make_code_map(&tm_act, codes, w->K / 2, M, 128);
        if (st == PRQ_OK) st = make_sf_map(&tm_sfa, p.act_sf, Sg * p.act_groups * kSfGroupBytes, 4);
        if (st == PRQ_OK) st = make_out_map(&tm_y, y, M, w->N, ldy, y_dtype == PRQ_BF16);
        if (st != PRQ_OK) return st;
        cudaError_t e = launch_prefill_pair(pair_bn, tm_act, w->tm_w_pair[variant], tm_sfa, w->tm_sfw_pair[variant], tm_y, q,
                                            pairs, static_cast<cudaStream_t>(stream));
        g_launches.fetch_add(1);
        return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
    }
}

prq_status prq_linear_multi(int n, const prq_weights* const* ws, const void* const* codes, const void* const* scales_sf,
                            int M, void* const* y, const int* ldy, prq_dtype y_dtype, prq_stream_t stream) {
    if (n < 1 || n > PRQ_MULTI_MAX || !ws || !codes || !scales_sf || !y || !ldy) return PRQ_ERR_INVALID_ARG;
    if (M < 0 || M > 128) return PRQ_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i) {
        if (!ws[i]) return PRQ_ERR_INVALID_ARG;
        if (M == 0) continue;
        prq_status st = check_linear_common(ws[i], codes[i], scales_sf[i], y[i], ldy[i], y_dtype);
        if (st != PRQ_OK) return st;
        if (ws[i]->n_experts != 1 || !ws[i]->maps_ready || ws[i]->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
        // one stage plan and one cluster size for the whole launch
        if (ws[i]->K != ws[0]->K || ws[i]->k_tail != ws[0]->k_tail || ws[i]->device != ws[0]->device) return PRQ_ERR_INVALID_ARG;
    }
    if (M == 0) return PRQ_OK;
    if (!handle_device_is_current(ws[0])) return PRQ_ERR_INVALID_ARG;
    DeviceInfo* di;
    prq_status st = device_info(ws[0]->device, &di);
    if (st != PRQ_OK) return st;
    const int bn = decode_bn(M);
    DecodeMaps maps;
    std::memset(&maps, 0, sizeof(maps));
    DecodeBatch b = {};
    b.status = di->status_ptr; b.trace = trace_ptr(); b.dbg = env_int("PRQ_DBG", 0);
    b.M = M; b.K = ws[0]->K; b.k_tail = ws[0]->k_tail;
    b.y_bf16 = y_dtype == PRQ_BF16;
    b.n_lin = n;
    int tiles = 0;
    for (int i = 0; i < n; ++i) {
        tiles += (ws[i]->N + 127) / 128;
        st = make_code_map(&maps.act[i], codes[i], ws[i]->K / 2, M, bn);
        if (st != PRQ_OK) return st;
        maps.w[i] = ws[i]->tm_w_decode;
        b.lay[i] = DecodeLayer{static_cast<const uint8_t*>(scales_sf[i]), ws[i]->d_sf, y[i], ws[i]->N, ws[i]->w_groups,
                               ldy[i], tiles};
    }
    b.splits = decode_splits_for(tiles, ws[0]->plan.S, M, di);
    cudaError_t e = launch_decode_batch(bn, maps, b, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_stack_gate_up(const uint16_t* W_gate, const uint16_t* W_up, int C, int H, uint16_t* out) {
    if (!W_gate || !W_up || !out || C < kBlock || C % kBlock || H < 1) return PRQ_ERR_INVALID_ARG;
    stack_gate_up(W_gate, W_up, C, H, out);
    return PRQ_OK;
}

prq_status prq_linear_gated(const prq_weights* w, const void* codes, const void* scales_sf, int M, const prq_weights* wd,
                            void* out_codes, void* out_scales_row, void* out_scales_sf, void* h_check, prq_stream_t stream) {
    if (!w || !wd || M < 0) return PRQ_ERR_INVALID_ARG;
    if (!w->gated || !w->maps_ready || w->n_experts != 1 || wd->n_experts != 1 || w->device != wd->device) return PRQ_ERR_INVALID_ARG;
    if (w->format != PRQ_FMT_MXFP4 || wd->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
    const int C = wd->K, kd = wd->k_tail;
    if (w->N != 2 * C || C % kStageK || kd % kStageK) return PRQ_ERR_INVALID_ARG;
    if (M == 0) return PRQ_OK;
    if (!codes || !scales_sf || !out_codes || !out_scales_sf) return PRQ_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(scales_sf) || !aligned16(out_codes) || !aligned16(out_scales_sf) || !aligned16(h_check))
        return PRQ_ERR_ALIGNMENT;
    if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
    DeviceInfo* di;
    prq_status st = device_info(w->device, &di);
    if (st != PRQ_OK) return st;
    if (di->max_pairs_gated == 0)
        di->max_pairs_gated = std::max(1, std::min(prefill_pair_max_clusters(kPrefillTileGated), di->num_sms / 2));

    PrefillParams q;
    std::memset(&q, 0, sizeof(q));
    q.M = M; q.N = w->N; q.K = w->K; q.k_tail = w->k_tail;
    q.m_tiles = (M + 255) / 256; q.n_tiles = (w->N + kPrefillTileGated - 1) / kPrefillTileGated;
    const long long tiles = static_cast<long long>(q.m_tiles) * q.n_tiles;
    if (tiles >= (1ll << 30)) return PRQ_ERR_INVALID_ARG;
    // whole tiles only, wave after wave (a piece of a tile has no gate and up sums to put through the activation)
    const int pairs = static_cast<int>(std::min<long long>(tiles, di->max_pairs_gated));
    q.sk_tiles = 0; q.whole_tiles = static_cast<int>((tiles + pairs - 1) / pairs); q.total_tiles = static_cast<int>(tiles);
    q.act_groups = dense_groups(M); q.w_groups = w->w_groups_alt[kAltGated];
    q.act_sf = static_cast<const uint8_t*>(scales_sf); q.w_sf = w->d_sf_alt[kAltGated];
    q.status = di->status_ptr; q.trace = trace_ptr(); q.dbg = env_int("PRQ_DBG", 0);
    q.wait_limit = kDefaultWaitLimitCycles;
    q.out_codes = static_cast<uint8_t*>(out_codes);
    q.out_sf = static_cast<uint8_t*>(out_scales_sf);
    q.out_scales_row = static_cast<uint8_t*>(out_scales_row);
    q.out_h = static_cast<uint16_t*>(h_check);
    q.out_C = C; q.out_k_tail = kd; q.out_groups = dense_groups(M);
    CUtensorMap tm_act, tm_sfa;
    st = make_code_map(&tm_act, codes, w->K / 2, M, 128);
    if (st == PRQ_OK) st = make_sf_map(&tm_sfa, q.act_sf, static_cast<uint64_t>(w->plan.S) * q.act_groups * kSfGroupBytes, 4);
    if (st != PRQ_OK) return st;
    // (the kernel stores nothing through an output map in this mode: the activation map fills the parameter)
    cudaError_t e = launch_prefill_pair(kPrefillTileGated, tm_act, w->tm_w_pair[kAltGated], tm_sfa, w->tm_sfw_pair[kAltGated],
                                        tm_act, q, pairs, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_linear_fused(const prq_weights* w, prq_act_mode mode, const void* x, int M, int ldx, void* y, int ldy,
                            prq_dtype y_dtype, prq_stream_t stream) {
    if (!w || M < 0 || M > PRQ_FUSED_MAX_M || mode != PRQ_ACT_IDENTITY || w->n_experts != 1 || !w->maps_ready ||
        w->format != PRQ_FMT_MXFP4)
        return PRQ_ERR_INVALID_ARG;
    if (M == 0) return PRQ_OK;
    if (!x || !y || ldx < w->K || ldy < w->N) return PRQ_ERR_INVALID_ARG;
    if (y_dtype != PRQ_F32 && y_dtype != PRQ_BF16) return PRQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || ldx % 8 || ldy % (y_dtype == PRQ_F32 ? 4 : 8)) return PRQ_ERR_ALIGNMENT;
    if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
    DeviceInfo* di;
    prq_status st = device_info(w->device, &di);
    if (st != PRQ_OK) return st;
    DecodeParams q;
    std::memset(&q, 0, sizeof(q));
    q.M = M; q.N = w->N; q.K = w->K; q.k_tail = w->k_tail;
    q.w_groups = w->w_groups;
    q.w_sf = w->d_sf;
    q.x = static_cast<const uint16_t*>(x); q.ldx = ldx;
    q.y = y; q.ldy = ldy; q.y_bf16 = y_dtype == PRQ_BF16;
    q.status = di->status_ptr; q.trace = trace_ptr(); q.dbg = env_int("PRQ_DBG", 0);
    q.splits = decode_splits(w, M, di);
    // the kernel takes no activation tensor map in this mode; the weight map fills the parameter
    cudaError_t e = launch_decode(decode_bn(M), w->tm_w_decode, w->tm_w_decode, q, (w->N + 127) / 128, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

prq_status prq_linear_grouped(const prq_weights* w, const void* codes, const void* scales_sf,
                              const int32_t* expert_offsets, int M_total, void* y, int ldy, prq_dtype y_dtype,
                              prq_stream_t stream) {
    if (w && M_total == 0) return PRQ_OK;
    prq_status st = check_linear_common(w, codes, scales_sf, y, ldy, y_dtype);
    if (st != PRQ_OK) return st;
    if (M_total < 0 || !expert_offsets || w->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
    if (!handle_device_is_current(w)) return PRQ_ERR_INVALID_ARG;
    DeviceInfo* di;
    st = device_info(w->device, &di);
    if (st != PRQ_OK) return st;
    const size_t Ka = static_cast<size_t>(w->K) + w->k_tail;

    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.M = M_total; p.N = w->N; p.K = w->K; p.k_tail = w->k_tail;
    p.n_experts = w->n_experts;
    p.act_groups = grouped_groups(M_total, w->n_experts);
    p.w_groups = w->w_groups;
    p.act_sf = static_cast<const uint8_t*>(scales_sf);
    p.w_sf = w->d_sf;
    p.expert_offsets = expert_offsets;
    p.y = y; p.ldy = ldy; p.y_bf16 = y_dtype == PRQ_BF16;
    p.status = di->status_ptr;
    p.trace = trace_ptr();
    // output features on the MMA M axis, one 128-token group of an expert on the N axis (contiguous stores per
    // token, cheap for experts with few tokens)
    // token tile: 64 rows when the experts hold a handful of tokens each (the smaller tile leaves room for a deeper
    // ring of weight tiles in flight), 128 otherwise (every extra token tile of an expert re-reads its weight tiles)
    int bn = static_cast<long long>(M_total) <= 64LL * w->n_experts ? 64 : 128;
    bn = env_int("PRQ_GROUPED_BN", bn);   // developer switch
    if (bn == 0) bn = 128;
    if (bn != 64 && bn != 128) return PRQ_ERR_INVALID_ARG;
    CUtensorMap tm_act, tm_w;
    st = make_code_map(&tm_act, codes, w->K / 2, M_total, bn);
    if (st == PRQ_OK) st = make_code_map(&tm_w, w->d_codes, Ka / 2, static_cast<uint64_t>(w->n_experts) * w->N, 128);
    if (st != PRQ_OK) return st;
    cudaError_t e = launch_gemm_grouped(bn, tm_act, tm_w, p, di->num_sms, static_cast<cudaStream_t>(stream));
    g_launches.fetch_add(1);
    return e == cudaSuccess ? PRQ_OK : PRQ_ERR_CUDA;
}

// Device scratch layout of prq_forward_host: [workspace | x | codes | scales_sf | y], each 256-byte aligned.
namespace {
size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }
struct HostFwdLayout {
    size_t ws, x, codes, sf, y, total;
};
HostFwdLayout host_fwd_layout(const prq_weights* w, int M) {
    HostFwdLayout l;
    l.ws = 0;
    l.x = align256(prq_linear_workspace_bytes(w, M));
    l.codes = l.x + align256(static_cast<size_t>(M) * w->K * 2);
    l.sf = l.codes + align256(prq_act_bytes(M, w->K, w->k_tail, 1, PRQ_BUF_CODES));
    l.y = l.sf + align256(prq_act_bytes(M, w->K, w->k_tail, 1, PRQ_BUF_SCALES_SF));
    l.total = l.y + align256(static_cast<size_t>(M) * w->N * 4);
    return l;
}
}  // namespace

size_t prq_forward_host_scratch_bytes(const prq_weights* w, int M) {
    if (!w || M < 0 || w->n_experts != 1 || w->format != PRQ_FMT_MXFP4) return 0;
    return host_fwd_layout(w, M).total;
}

prq_status prq_forward_host(const prq_weights* w, prq_act_mode mode, const uint16_t* x_host, int M, void* y_host,
                            prq_dtype y_dtype, void* dev_scratch, size_t scratch_bytes, prq_stream_t stream) {
    if (!w || w->n_experts != 1 || M < 0 || w->format != PRQ_FMT_MXFP4) return PRQ_ERR_INVALID_ARG;
    if (M == 0) return PRQ_OK;
    if (!x_host || !y_host || !dev_scratch) return PRQ_ERR_INVALID_ARG;
    if (y_dtype != PRQ_F32 && y_dtype != PRQ_BF16) return PRQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_scratch) & 255) return PRQ_ERR_ALIGNMENT;
    const HostFwdLayout l = host_fwd_layout(w, M);
    if (scratch_bytes < l.total) return PRQ_ERR_WORKSPACE;
    uint8_t* base = static_cast<uint8_t*>(dev_scratch);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t x_bytes = static_cast<size_t>(M) * w->K * 2;
    if (cudaMemcpyAsync(base + l.x, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return PRQ_ERR_CUDA;
    prq_status st = prq_quantize_act(w, mode, base + l.x, M, w->K, nullptr, base + l.codes, nullptr, base + l.sf, stream);
    if (st != PRQ_OK) return st;
    st = prq_linear(w, base + l.codes, base + l.sf, M, base + l.y, w->N, y_dtype, base + l.ws, l.x, stream);
    if (st != PRQ_OK) return st;
    const size_t y_bytes = static_cast<size_t>(M) * w->N * (y_dtype == PRQ_F32 ? 4 : 2);
    if (cudaMemcpyAsync(y_host, base + l.y, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return PRQ_ERR_CUDA;
    return PRQ_OK;
}

}  // extern "C"

// ---- prq_linear_static_scratch: the GEMM for callers that cannot hand over (or allocate) a workspace ----
namespace prq {
namespace {

// Built-in scratch of the stream-K prefill kernel: two counters per 128-row half of an output tile, then
// two fp32 partial tiles per CTA.  It is part of the library image, so every GPU that loads the library
// carries it until the process exits: 64 KB of counters + 2 x 160 x 128 KB of partial tiles = 42,008,576 bytes.
constexpr int kStaticMaxFlags = 8192;   // tile halves
constexpr int kStaticMaxCtas = 160;
constexpr size_t kStaticFlagBytes = 2 * static_cast<size_t>(kStaticMaxFlags) * sizeof(int);
constexpr size_t kStaticScratchBytes = kStaticFlagBytes + 2 * static_cast<size_t>(kStaticMaxCtas) * kPrefillSlotBytes;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticScratchDev {
    bool ready = false;
    void* ptr = nullptr;
};
StaticScratchDev g_static_dev[64];

// Device address of the array on device `dev` (which must be current).  In host code the array's name
// is only a handle for the runtime, not an address a kernel could use, so the address is looked up
// once per device and cached.
prq_status static_scratch_address(int dev, void** out) {
    if (dev < 0 || dev >= 64) return PRQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    StaticScratchDev& d = g_static_dev[dev];
    if (!d.ready) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return PRQ_ERR_CUDA;
        }
        d.ptr = p;
        d.ready = true;
    }
    *out = d.ptr;
    return PRQ_OK;
}

}  // namespace
}  // namespace prq

extern "C" prq_status prq_linear_static_scratch(const prq_weights* w, const void* codes, const void* scales_sf, int M,
                                                void* y, int ldy, prq_dtype y_dtype, prq_stream_t stream) {
    if (!w || M < 0) return PRQ_ERR_INVALID_ARG;
    if (M <= 128) return prq_linear(w, codes, scales_sf, M, y, ldy, y_dtype, nullptr, 0, stream);  // needs no scratch
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return PRQ_ERR_CUDA;
    if (dev != w->device) return PRQ_ERR_INVALID_ARG;  // the handle's device must be current
    DeviceInfo* di;
    prq_status st = device_info(dev, &di);
    if (st != PRQ_OK) return st;
    if (prefill_flag_count(w, M) > static_cast<size_t>(kStaticMaxFlags) || di->num_sms > kStaticMaxCtas) return PRQ_ERR_STATIC_SCRATCH;
    void* scratch = nullptr;
    st = static_scratch_address(dev, &scratch);
    if (st != PRQ_OK) return st;
    // The array still holds whatever the previous call left there.  The partial tiles are always written
    // before they are read; the tile flags must start at zero.
    if (cudaMemsetAsync(scratch, 0, prefill_flag_bytes(w, M), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return PRQ_ERR_CUDA;
    return prq_linear(w, codes, scales_sf, M, y, ldy, y_dtype, scratch, kStaticScratchBytes, stream);
}
