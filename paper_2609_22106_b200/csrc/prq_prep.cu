// Offline weight preparation (Algorithm 1 steps 3-7 and 11) on the host, multi-threaded.
//
// For one layer and one alpha:
//   s_j   = max(amax_j, 1e-5)^alpha                     "Offline scaling": D = diag(s)
//   W0    = fl32(W * s)                                  scaled weight W D
//   err_j = sum_n (W0[n,j] - deq(Q(W0))[n,j])^2          column-wise MXFP4 error, blocks of 32 input
//                                                        channels in the original order, FP64, n ascending
//   top-k by (err descending, index ascending); perm = [unselected ascending | selected ascending]
//   Wt    = W0[:, perm]; codes/scales of Q(Wt); R = Wt_tail - deq(Q(Wt))_tail (Eq. (2)); Q(R)
//   export [Q(Wt) | Q(R)]                                right factor of Eq. (3)
//
// The MXFP4 quantiser here works on the fp32 bit pattern (exponent field arithmetic), like the
// device kernel does, so that host prep and device quantisation follow one definition:
// block scale 2^(floor(log2 amax) - 2) stored as E8M0, E2M1 elements rounded to nearest with
// ties to the even code, saturation at 6, sign kept on zero.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <thread>

#include "prq_internal.h"

namespace prq {
namespace {

inline float bf16_bits_to_float(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}
inline uint32_t float_bits(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    return u;
}
inline float bits_float(uint32_t u) {
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

const float kE2M1[8] = {0.f, 0.5f, 1.f, 1.5f, 2.f, 3.f, 4.f, 6.f};

// E8M0 byte of a block from the largest magnitude's bit pattern: biased exponent minus 2,
// floored at 0 (zero and tiny amax land on byte 0).
inline uint8_t scale_byte_from_amax_bits(uint32_t amax_bits) {
    int e = static_cast<int>((amax_bits >> 23) & 0xff) - 2;
    return static_cast<uint8_t>(e < 0 ? 0 : e);
}

// Code of one value given the block's scale byte: |v| * 2^(127 - byte) is exact, then the
// seven decision thresholds of E2M1 with ties to the even code.
inline uint8_t e2m1_code(float v, uint8_t byte) {
    const uint32_t bits = float_bits(v);
    const float inv = bits_float(static_cast<uint32_t>(254 - byte) << 23);
    const float a = bits_float(bits & 0x7fffffffu) * inv;
    uint8_t m;
    if (a <= 0.25f) m = 0;
    else if (a < 0.75f) m = 1;
    else if (a <= 1.25f) m = 2;
    else if (a < 1.75f) m = 3;
    else if (a <= 2.5f) m = 4;
    else if (a < 3.5f) m = 5;
    else if (a <= 5.0f) m = 6;
    else m = 7;
    return static_cast<uint8_t>(m | ((bits >> 28) & 8u));
}

inline float e2m1_value(uint8_t code, uint8_t byte) {
    // value[code & 7] * 2^(byte - 127), computed in double and exact in fp32 for every byte
    // the quantiser produces together with a representable input
    const double x = std::ldexp(static_cast<double>(kE2M1[code & 7]), static_cast<int>(byte) - 127);
    return static_cast<float>((code & 8) ? -x : x);
}

// Quantise one block of 32 floats; codes one per element (unpacked).
inline uint8_t quantize_block(const float* v, uint8_t* codes) {
    uint32_t amax_bits = 0;
    for (int i = 0; i < kBlock; ++i) amax_bits = std::max(amax_bits, float_bits(v[i]) & 0x7fffffffu);
    const uint8_t byte = scale_byte_from_amax_bits(amax_bits);
    for (int i = 0; i < kBlock; ++i) codes[i] = e2m1_code(v[i], byte);
    return byte;
}

// The same with the weight-side block-scale search (the "E8M0-W" variant of the ablation study): the
// block is quantised with the floor-rule byte and with its two neighbours; a neighbour wins only with a
// strictly smaller sum of squared errors (FP64, element order; byte - 1 is looked at before byte + 1).
inline double block_error(const float* v, uint8_t byte, uint8_t* codes) {
    double err = 0.0;
    for (int i = 0; i < kBlock; ++i) {
        codes[i] = e2m1_code(v[i], byte);
        const double d = static_cast<double>(v[i]) - static_cast<double>(e2m1_value(codes[i], byte));
        err += d * d;
    }
    return err;
}
inline uint8_t quantize_block_search(const float* v, uint8_t* codes) {
    uint8_t tmp[kBlock];
    const uint8_t byte0 = quantize_block(v, codes);
    bool zero = true;
    for (int i = 0; i < kBlock; ++i) zero = zero && v[i] == 0.f;
    if (zero) return byte0;
    double best_err = block_error(v, byte0, tmp);
    uint8_t best = byte0;
    const int cand[2] = {static_cast<int>(byte0) - 1, static_cast<int>(byte0) + 1};
    for (int c = 0; c < 2; ++c) {
        if (cand[c] < 0 || cand[c] > 254) continue;
        const double err = block_error(v, static_cast<uint8_t>(cand[c]), tmp);
        if (err < best_err) { best_err = err; best = static_cast<uint8_t>(cand[c]); std::memcpy(codes, tmp, kBlock); }
    }
    return best;
}

template <class F>
void parallel_for(long n, F&& body) {
    unsigned hw = std::thread::hardware_concurrency();
    long nt = std::max(1u, std::min(hw ? hw : 1u, 64u));
    nt = std::min<long>(nt, std::max<long>(1, n));
    if (nt <= 1) {
        body(0, n);
        return;
    }
    std::vector<std::thread> th;
    for (long t = 0; t < nt; ++t) {
        long lo = n * t / nt, hi = n * (t + 1) / nt;
        th.emplace_back([=, &body] { body(lo, hi); });
    }
    for (auto& x : th) x.join();
}

double scale_power(double a, float alpha) {
    if (alpha == 0.f) return 1.0;
    if (alpha == 1.f) return a;
    if (alpha == 0.5f) return std::sqrt(a);
    if (alpha == 0.25f) return std::sqrt(std::sqrt(a));
    if (alpha == 0.75f) return std::sqrt(a) * std::sqrt(std::sqrt(a));
    return std::pow(a, static_cast<double>(alpha));
}

}  // namespace

// bf16 of the exact product of a bf16 weight and an fp32 scale, rounded once.  The product has up to 32
// significant bits: it is first brought to fp32 with round-to-odd (truncate toward zero, then set the last bit if
// anything was lost), after which the usual round-to-nearest-even to 8 bits cannot double-round.
static uint16_t scaled_bf16(uint16_t w, float s) {
    const double p = static_cast<double>(bf16_bits_to_float(w)) * static_cast<double>(s);   // exact
    float f = static_cast<float>(p);
    if (static_cast<double>(f) != p && std::isfinite(f)) {
        if (std::fabs(static_cast<double>(f)) > std::fabs(p)) f = std::nextafterf(f, 0.f);   // now truncated
        f = bits_float(float_bits(f) | 1u);                                                 // sticky bit
    }
    const uint32_t u = float_bits(f);
    if ((u & 0x7f800000u) == 0x7f800000u) return static_cast<uint16_t>(u >> 16);            // infinity stays
    return static_cast<uint16_t>((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}

prq_status fold_producer(const int32_t* perm, const float* inv_s, int C, int k_tail, const uint16_t* W_up,
                         const uint16_t* W_gate, int H, bool duplicate_tail, uint16_t* out_up, uint16_t* out_gate) {
    const long rows = static_cast<long>(C) + (duplicate_tail ? k_tail : 0);
    for (int j = 0; j < C; ++j)
        if (perm[j] < 0 || perm[j] >= C || !std::isfinite(inv_s[j])) return PRQ_ERR_INVALID_ARG;
    parallel_for(rows, [&](long lo, long hi) {
        for (long jp = lo; jp < hi; ++jp) {
            const long pos = jp < C ? jp : C - k_tail + (jp - C);   // position in the permuted order
            const long j = perm[pos];
            const float s = inv_s[j];
            const uint16_t* src = W_up + j * H;
            uint16_t* dst = out_up + jp * H;
            for (int h = 0; h < H; ++h) dst[h] = scaled_bf16(src[h], s);
            if (W_gate && out_gate) std::memcpy(out_gate + jp * H, W_gate + j * H, sizeof(uint16_t) * H);
        }
    });
    return PRQ_OK;
}

prq_status channel_scales(const float* amax, int K, float alpha, std::vector<float>& s, std::vector<float>& inv_s) {
    s.resize(K);
    inv_s.resize(K);
    for (int j = 0; j < K; ++j) {
        if (!std::isfinite(amax[j])) return PRQ_ERR_NONFINITE;
        double a = std::max(static_cast<double>(amax[j]), 1e-5);
        s[j] = static_cast<float>(scale_power(a, alpha));
        inv_s[j] = static_cast<float>(1.0 / static_cast<double>(s[j]));
    }
    return PRQ_OK;
}

void rank_and_permute(const std::vector<double>& col_err, int K, int k_tail, std::vector<int32_t>& perm) {
    perm.resize(K);
    std::vector<int32_t> order(K);
    for (int j = 0; j < K; ++j) order[j] = j;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return col_err[a] > col_err[b]; });
    std::vector<uint8_t> sel(K, 0);
    for (int i = 0; i < k_tail; ++i) sel[order[i]] = 1;
    int head = 0, tail = K - k_tail;
    for (int j = 0; j < K; ++j) {
        if (sel[j]) perm[tail++] = j;
        else perm[head++] = j;
    }
}

prq_status prepare_layer(const uint16_t* W, int N, int K, const float* amax, float alpha, int k_tail,
                         PrepResult& out, bool scale_search) {
    const long Ka = static_cast<long>(K) + k_tail;
    const int nblk = K / kBlock;
    out.col_err.assign(K, 0.0);
    out.codes.assign(static_cast<size_t>(N) * Ka / 2, 0);
    out.scales.assign(static_cast<size_t>(N) * Ka / kBlock, 0);
    if (channel_scales(amax, K, alpha, out.s, out.inv_s) != PRQ_OK) return PRQ_ERR_NONFINITE;

    // scaled weight, fp32 (one rounding of the exact product)
    std::vector<float> W0(static_cast<size_t>(N) * K);
    std::atomic<bool> finite{true};
    parallel_for(N, [&](long lo, long hi) {
        bool ok = true;
        for (long n = lo; n < hi; ++n)
            for (int j = 0; j < K; ++j) {
                float w = bf16_bits_to_float(W[n * K + j]);
                float v = w * out.s[j];
                ok = ok && std::isfinite(v);
                W0[n * K + j] = v;
            }
        if (!ok) finite.store(false);
    });
    if (!finite.load()) return PRQ_ERR_NONFINITE;

    // column errors: each thread owns a range of 32-channel blocks and walks the rows in order
    parallel_for(nblk, [&](long lo, long hi) {
        uint8_t codes[kBlock];
        for (long n = 0; n < N; ++n)
            for (long b = lo; b < hi; ++b) {
                const float* v = &W0[n * K + b * kBlock];
                uint8_t byte = quantize_block(v, codes);
                for (int i = 0; i < kBlock; ++i) {
                    double d = static_cast<double>(v[i]) - static_cast<double>(e2m1_value(codes[i], byte));
                    out.col_err[b * kBlock + i] += d * d;
                }
            }
    });

    // error-ranked top-k and the permutation
    rank_and_permute(out.col_err, K, k_tail, out.perm);

    // permuted quantisation, residual and its quantisation, packed export
    const int tail_blk0 = (K - k_tail) / kBlock;
    parallel_for(N, [&](long lo, long hi) {
        float v[kBlock], r[kBlock];
        uint8_t codes[kBlock];
        for (long n = lo; n < hi; ++n) {
            uint8_t* crow = &out.codes[n * (Ka / 2)];
            uint8_t* srow = &out.scales[n * (Ka / kBlock)];
            for (int b = 0; b < nblk; ++b) {
                for (int i = 0; i < kBlock; ++i) v[i] = W0[n * K + out.perm[b * kBlock + i]];
                uint8_t byte = scale_search ? quantize_block_search(v, codes) : quantize_block(v, codes);
                srow[b] = byte;
                for (int i = 0; i < kBlock; i += 2)
                    crow[(b * kBlock + i) / 2] = static_cast<uint8_t>(codes[i] | (codes[i + 1] << 4));
                if (b >= tail_blk0) {
                    for (int i = 0; i < kBlock; ++i) r[i] = v[i] - e2m1_value(codes[i], byte);  // exact
                    uint8_t rbyte = scale_search ? quantize_block_search(r, codes) : quantize_block(r, codes);
                    const int rb = nblk + (b - tail_blk0);
                    srow[rb] = rbyte;
                    for (int i = 0; i < kBlock; i += 2)
                        crow[(rb * kBlock + i) / 2] = static_cast<uint8_t>(codes[i] | (codes[i + 1] << 4));
                }
            }
        }
    });
    return PRQ_OK;
}

void stack_gate_up(const uint16_t* W_gate, const uint16_t* W_up, int C, int H, uint16_t* out) {
    const size_t row = static_cast<size_t>(H) * sizeof(uint16_t);
    for (int b = 0; b < C / kBlock; ++b) {
        std::memcpy(out + static_cast<size_t>(2 * b) * kBlock * H, W_gate + static_cast<size_t>(b) * kBlock * H, row * kBlock);
        std::memcpy(out + static_cast<size_t>(2 * b + 1) * kBlock * H, W_up + static_cast<size_t>(b) * kBlock * H, row * kBlock);
    }
}

}  // namespace prq
