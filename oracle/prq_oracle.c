/*
 * PRQuant oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, scalar CPU statement of what the compensated W4A4 MXFP4 linear
 * layer computes.  It exists so that the CUDA library can be checked against
 * something written directly from the paper; it shares no code, header, table
 * or helper with the CUDA library and must never be called from it.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * Every function names the passage of the paper it follows.  Floating point is
 * FP64 unless the step is defined on fp32 values (the quantiser input, the
 * scaled weight), in which case the fp32 value is produced by rounding an exact
 * FP64 result once.
 *
 * Readings taken where the paper is silent (the MXFP4 details come from the OCP
 * microscaling format the paper cites in its Introduction):
 *   - block = 32 consecutive input channels of one row; shared scale 2^e with
 *     e = clamp(floor(log2(amax)) - 2, -127, 127), stored as the byte e + 127;
 *     an all-zero block stores byte 0;
 *   - elements are E2M1 (values 0, .5, 1, 1.5, 2, 3, 4, 6 and a sign bit),
 *     rounded to nearest with ties to the even code, magnitudes above 6
 *     saturate to 6, the sign bit of the input is kept even when the magnitude
 *     rounds to zero;
 *   - packed storage: byte i of a row = code[2i] | code[2i+1] << 4;
 *   - "column-wise quantization error" of channel j = sum over output rows of
 *     the squared difference between the scaled weight and its MXFP4 image,
 *     accumulated in FP64 in ascending row order;
 *   - top-k ties break toward the lower channel index; the permutation lists the
 *     unselected channels in ascending order, then the selected ones ascending;
 *   - s_j = max(amax_j, 1e-5)^alpha;
 *   - weight-side block-scale search (the "E8M0-W" variant of the ablation study, for which the
 *     paper gives only the name "local block-scale search"): for every block of Q(W D P) and of
 *     Q(R) the candidates are the floor-rule exponent e0 and its neighbours e0 - 1 and e0 + 1
 *     (bytes kept in [0, 254]); the block is quantised with each, the squared error is summed in
 *     FP64 in element order, and a neighbour replaces e0 only if its error is strictly smaller
 *     (e0 - 1 is looked at before e0 + 1).  The column-error ranking of step 4 keeps the floor
 *     rule, so the permutation does not depend on the option; R is the residual of the searched
 *     quantisation.  An all-zero block keeps byte 0.
 *
 * Pins (see tests/test_oracle_*.py): hand-worked encodings, a brute-force
 * nearest-value quantiser in exact rational arithmetic, the worked prep example,
 * k = 0 reducing to plain MXFP4, Eq. (1) invariance, exact residual identity,
 * brute-force top-k, Eq. (3) = main + correction.  The normalised error and the alpha
 * selection of the Python front end (first minimum over the grid) are pinned by a hand-worked
 * error norm and a hand-decided three-candidate search (tests/test_oracle_alpha.py).  The gated activation
 * silu(g) * u of the producer is pinned by closed-form values and identities (tests/test_oracle_gated.py); the
 * second format (MXFP8) by hand-worked encodings and a brute-force nearest-value search over the whole code
 * table (tests/test_oracle_mxfp8.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_BLOCK 32

/* E2M1 magnitudes by 3-bit index (OCP MX element format cited in the Introduction). */
static const double orc_e2m1_value[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

static float orc_bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static int orc_signbit_f32(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    return (int)(u >> 31);
}

/* Shared block scale (E8M0 byte) of one block of 32 fp32 values.
 * floor(log2(amax)) - 2 puts amax/2^e in [4, 8), i.e. just inside the E2M1
 * range up to its saturation band. */
static uint8_t orc_block_scale_byte(const float *v) {
    double amax = 0.0;
    for (int i = 0; i < ORC_BLOCK; ++i) {
        double a = fabs((double)v[i]);
        if (a > amax) amax = a;
    }
    if (amax == 0.0) return 0;
    int ex;
    (void)frexp(amax, &ex); /* amax = m * 2^ex with m in [0.5, 1)  =>  floor(log2) = ex - 1 */
    int e = (ex - 1) - 2;
    if (e < -127) e = -127;
    if (e > 127) e = 127;
    return (uint8_t)(e + 127);
}

/* One element: a = |v| / 2^e is exact in FP64; round to the nearest E2M1
 * magnitude, ties to the even code, saturating at 6. */
static uint8_t orc_e2m1_code(float v, int e) {
    double a = ldexp(fabs((double)v), -e);
    uint8_t mag;
    if (a <= 0.25) mag = 0;
    else if (a < 0.75) mag = 1;
    else if (a <= 1.25) mag = 2;
    else if (a < 1.75) mag = 3;
    else if (a <= 2.5) mag = 4;
    else if (a < 3.5) mag = 5;
    else if (a <= 5.0) mag = 6;
    else mag = 7;
    return (uint8_t)(mag | (orc_signbit_f32(v) << 3));
}

/* The MXFP4 quantiser Q of Eq. (2), storage half: rows x cols fp32 -> packed
 * codes (rows x cols/2 bytes) and scale bytes (rows x cols/32). */
int orc_quantize_rows(const float *v, long rows, long cols, uint8_t *codes, uint8_t *scales) {
    if (cols % ORC_BLOCK) return 1;
    for (long r = 0; r < rows; ++r) {
        for (long b = 0; b < cols / ORC_BLOCK; ++b) {
            const float *blk = v + r * cols + b * ORC_BLOCK;
            uint8_t byte = orc_block_scale_byte(blk);
            scales[r * (cols / ORC_BLOCK) + b] = byte;
            int e = (int)byte - 127;
            for (int i = 0; i < ORC_BLOCK; i += 2) {
                uint8_t lo = orc_e2m1_code(blk[i], e);
                uint8_t hi = orc_e2m1_code(blk[i + 1], e);
                codes[(r * cols + b * ORC_BLOCK + i) / 2] = (uint8_t)(lo | (hi << 4));
            }
        }
    }
    return 0;
}

/* Squared error of one block quantised with the scale 2^e, FP64, element order. */
static double orc_block_error(const float *blk, int e) {
    double err = 0.0;
    for (int i = 0; i < ORC_BLOCK; ++i) {
        uint8_t c = orc_e2m1_code(blk[i], e);
        double x = ldexp(orc_e2m1_value[c & 7], e);
        double d = (double)blk[i] - ((c & 8) ? -x : x);
        err += d * d;
    }
    return err;
}

/* Q with the weight-side block-scale search ("E8M0-W", Ablation study): like orc_quantize_rows,
 * but every block takes the best of the floor-rule exponent and its two neighbours. */
int orc_quantize_rows_search(const float *v, long rows, long cols, uint8_t *codes, uint8_t *scales) {
    if (cols % ORC_BLOCK) return 1;
    for (long r = 0; r < rows; ++r) {
        for (long b = 0; b < cols / ORC_BLOCK; ++b) {
            const float *blk = v + r * cols + b * ORC_BLOCK;
            int byte0 = (int)orc_block_scale_byte(blk), best = byte0;
            int zero = 1;
            for (int i = 0; i < ORC_BLOCK; ++i) zero = zero && blk[i] == 0.0f;
            if (!zero) {
                double best_err = orc_block_error(blk, byte0 - 127);
                const int cand[2] = {byte0 - 1, byte0 + 1};
                for (int c = 0; c < 2; ++c) {
                    if (cand[c] < 0 || cand[c] > 254) continue;
                    double err = orc_block_error(blk, cand[c] - 127);
                    if (err < best_err) { best_err = err; best = cand[c]; }
                }
            }
            scales[r * (cols / ORC_BLOCK) + b] = (uint8_t)best;
            int e = best - 127;
            for (int i = 0; i < ORC_BLOCK; i += 2) {
                uint8_t lo = orc_e2m1_code(blk[i], e);
                uint8_t hi = orc_e2m1_code(blk[i + 1], e);
                codes[(r * cols + b * ORC_BLOCK + i) / 2] = (uint8_t)(lo | (hi << 4));
            }
        }
    }
    return 0;
}

static double orc_dequant_one(const uint8_t *codes, const uint8_t *scales, long cols, long r, long j) {
    uint8_t byte = codes[(r * cols + j) / 2];
    uint8_t c = (j & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 0xF);
    double mag = orc_e2m1_value[c & 7];
    int e = (int)scales[r * (cols / ORC_BLOCK) + j / ORC_BLOCK] - 127;
    double x = ldexp(mag, e);
    return (c & 8) ? -x : x;
}

/* The dequantise half of Q: sign * value[code & 7] * 2^(byte - 127), in FP64 (exact). */
int orc_dequantize_rows(const uint8_t *codes, const uint8_t *scales, long rows, long cols, double *out) {
    if (cols % ORC_BLOCK) return 1;
    for (long r = 0; r < rows; ++r)
        for (long j = 0; j < cols; ++j) out[r * cols + j] = orc_dequant_one(codes, scales, cols, r, j);
    return 0;
}

/* Algorithm 1 step 1: per-channel maxima of |Z_cal| (exact, any precision). */
int orc_channel_amax(const uint16_t *z_bf16, long T, long K, float *amax) {
    for (long j = 0; j < K; ++j) amax[j] = 0.0f;
    for (long t = 0; t < T; ++t)
        for (long j = 0; j < K; ++j) {
            float a = fabsf(orc_bf16_to_f32(z_bf16[t * K + j]));
            if (a > amax[j]) amax[j] = a;
        }
    return 0;
}

/* Method, "Offline scaling": s_j = (max_t |Z_tj|)^alpha, stored in fp32, and the
 * reciprocal the activation side multiplies by.  The grid values 0, .25, .5, .75, 1
 * use only correctly rounded operations so that any implementation agrees. */
int orc_scales_from_amax(const float *amax, long K, double alpha, float *s, float *inv_s) {
    for (long j = 0; j < K; ++j) {
        double a = (double)amax[j];
        if (a < 1e-5) a = 1e-5;
        double p;
        if (alpha == 0.0) p = 1.0;
        else if (alpha == 1.0) p = a;
        else if (alpha == 0.5) p = sqrt(a);
        else if (alpha == 0.25) p = sqrt(sqrt(a));
        else if (alpha == 0.75) p = sqrt(a) * sqrt(sqrt(a));
        else p = pow(a, alpha);
        s[j] = (float)p;
        inv_s[j] = (float)(1.0 / (double)s[j]);
    }
    return 0;
}

typedef struct {
    double err;
    int32_t idx;
} orc_rank_t;

static int orc_rank_cmp(const void *pa, const void *pb) {
    const orc_rank_t *a = (const orc_rank_t *)pa, *b = (const orc_rank_t *)pb;
    if (a->err > b->err) return -1;
    if (a->err < b->err) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/* Algorithm 1 steps 3-7 and 11 for one alpha:
 *   W0 = fl32(W * s)                                  (step 3, scaled weight W D)
 *   err_j = sum_n (W0[n,j] - deq(Q(W0))[n,j])^2       (step 4, original channel order)
 *   top-k by err, perm = [unselected asc | selected asc]   (steps 4-5)
 *   Wt = W0[:, perm]                                  (step 6, Eq. (1) W D P)
 *   Qw = Q(Wt);  R = Wt_tail - deq(Qw)_tail           (step 7, Eq. (2))
 *   export [Qw | Q(R)]                                (step 11, right factor of Eq. (3))
 * Outputs: s, inv_s (K), col_err (K), perm (K, new -> old), wcodes N x (K+k)/2,
 * wscales N x (K+k)/32, R (N x k fp32, may be NULL). */
int orc_prepare_ex(const uint16_t *W_bf16, long N, long K, const float *amax, double alpha, long k,
                   int scale_search, float *s, float *inv_s, double *col_err, int32_t *perm,
                   uint8_t *wcodes, uint8_t *wscales, float *R_out) {
    if (K % ORC_BLOCK || k % ORC_BLOCK || k < 0 || k > K) return 1;
    long Ka = K + k;
    orc_scales_from_amax(amax, K, alpha, s, inv_s);

    float *W0 = (float *)malloc(sizeof(float) * N * K);
    uint8_t *c0 = (uint8_t *)malloc((size_t)N * K / 2);
    uint8_t *s0 = (uint8_t *)malloc((size_t)N * K / ORC_BLOCK);
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K; ++j)
            W0[n * K + j] = (float)((double)orc_bf16_to_f32(W_bf16[n * K + j]) * (double)s[j]);

    orc_quantize_rows(W0, N, K, c0, s0);
    for (long j = 0; j < K; ++j) col_err[j] = 0.0;
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K; ++j) {
            double d = (double)W0[n * K + j] - orc_dequant_one(c0, s0, K, n, j);
            col_err[j] += d * d;
        }

    orc_rank_t *rank = (orc_rank_t *)malloc(sizeof(orc_rank_t) * K);
    for (long j = 0; j < K; ++j) {
        rank[j].err = col_err[j];
        rank[j].idx = (int32_t)j;
    }
    qsort(rank, (size_t)K, sizeof(orc_rank_t), orc_rank_cmp);
    uint8_t *selected = (uint8_t *)calloc((size_t)K, 1);
    for (long i = 0; i < k; ++i) selected[rank[i].idx] = 1;
    long head = 0, tail = K - k;
    for (long j = 0; j < K; ++j) {
        if (selected[j]) perm[tail++] = (int32_t)j;
        else perm[head++] = (int32_t)j;
    }

    float *Wt = (float *)malloc(sizeof(float) * N * K);
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K; ++j) Wt[n * K + j] = W0[n * K + perm[j]];
    uint8_t *c1 = (uint8_t *)malloc((size_t)N * K / 2);
    uint8_t *s1 = (uint8_t *)malloc((size_t)N * K / ORC_BLOCK);
    if (scale_search) orc_quantize_rows_search(Wt, N, K, c1, s1);
    else orc_quantize_rows(Wt, N, K, c1, s1);

    float *R = (float *)malloc(sizeof(float) * (size_t)(N * (k ? k : 1)));
    for (long n = 0; n < N; ++n)
        for (long i = 0; i < k; ++i) {
            long j = K - k + i;
            /* the difference is exactly representable in fp32 (both terms are
             * multiples of the weight's last bit and the result is no larger) */
            R[n * k + i] = (float)((double)Wt[n * K + j] - orc_dequant_one(c1, s1, K, n, j));
        }
    uint8_t *cr = (uint8_t *)malloc((size_t)(N * (k ? k : ORC_BLOCK)) / 2);
    uint8_t *sr = (uint8_t *)malloc((size_t)(N * (k ? k : ORC_BLOCK)) / ORC_BLOCK);
    if (k) {
        if (scale_search) orc_quantize_rows_search(R, N, k, cr, sr);
        else orc_quantize_rows(R, N, k, cr, sr);
    }

    for (long n = 0; n < N; ++n) {
        memcpy(wcodes + n * (Ka / 2), c1 + n * (K / 2), (size_t)K / 2);
        memcpy(wscales + n * (Ka / ORC_BLOCK), s1 + n * (K / ORC_BLOCK), (size_t)K / ORC_BLOCK);
        if (k) {
            memcpy(wcodes + n * (Ka / 2) + K / 2, cr + n * (k / 2), (size_t)k / 2);
            memcpy(wscales + n * (Ka / ORC_BLOCK) + K / ORC_BLOCK, sr + n * (k / ORC_BLOCK), (size_t)k / ORC_BLOCK);
        }
    }
    if (R_out && k) memcpy(R_out, R, sizeof(float) * N * k);

    free(W0); free(c0); free(s0); free(rank); free(selected); free(Wt); free(c1); free(s1); free(R); free(cr); free(sr);
    return 0;
}

int orc_prepare(const uint16_t *W_bf16, long N, long K, const float *amax, double alpha, long k,
                float *s, float *inv_s, double *col_err, int32_t *perm,
                uint8_t *wcodes, uint8_t *wscales, float *R_out) {
    return orc_prepare_ex(W_bf16, N, K, amax, alpha, k, 0, s, inv_s, col_err, perm, wcodes, wscales, R_out);
}

/* Eq. (1), activation side: Zt = Z D^-1 P, i.e. xt[t,j'] = fl32(x[t,perm[j']] * inv_s[perm[j']]);
 * identity when perm and inv_s are NULL (folded into the producer layers).  Then Q by rows
 * (the one quantisation of the reordered activation of the Kernel design paragraph). */
int orc_quantize_act(const uint16_t *x_bf16, long M, long K, const int32_t *perm, const float *inv_s,
                     uint8_t *codes, uint8_t *scales) {
    if (K % ORC_BLOCK) return 1;
    float *row = (float *)malloc(sizeof(float) * K);
    for (long t = 0; t < M; ++t) {
        for (long j = 0; j < K; ++j) {
            long src = perm ? perm[j] : j;
            double v = (double)orc_bf16_to_f32(x_bf16[t * K + src]);
            if (inv_s) v = v * (double)inv_s[src];
            row[j] = (float)v;
        }
        orc_quantize_rows(row, 1, K, codes + t * (K / 2), scales + t * (K / ORC_BLOCK));
    }
    free(row);
    return 0;
}

/* "Online copy": the augmented activation [Q(Zt) | Q(Zt)[:, K-k:K]] -- the copied
 * blocks keep their own codes and scales (Kernel design paragraph). */
int orc_augment_act(const uint8_t *codes, const uint8_t *scales, long M, long K, long k,
                    uint8_t *codes_aug, uint8_t *scales_aug) {
    if (K % ORC_BLOCK || k % ORC_BLOCK || k > K) return 1;
    long Ka = K + k;
    for (long t = 0; t < M; ++t) {
        memcpy(codes_aug + t * (Ka / 2), codes + t * (K / 2), (size_t)K / 2);
        memcpy(codes_aug + t * (Ka / 2) + K / 2, codes + t * (K / 2) + (K - k) / 2, (size_t)k / 2);
        memcpy(scales_aug + t * (Ka / ORC_BLOCK), scales + t * (K / ORC_BLOCK), (size_t)K / ORC_BLOCK);
        memcpy(scales_aug + t * (Ka / ORC_BLOCK) + K / ORC_BLOCK,
               scales + t * (K / ORC_BLOCK) + (K - k) / ORC_BLOCK, (size_t)k / ORC_BLOCK);
    }
    return 0;
}

/* Eq. (3): y[t,n] = sum_{j < Ka} deq(A)[t,j] * deq(W)[n,j], FP64, ascending j.
 * Rows of y are independent; they are split across threads and nothing else is
 * reordered. */
int orc_matmul(const uint8_t *acodes, const uint8_t *ascales, long M,
               const uint8_t *wcodes, const uint8_t *wscales, long N, long Ka, double *y) {
    if (Ka % ORC_BLOCK) return 1;
    double *A = (double *)malloc(sizeof(double) * (size_t)(M * Ka));
    double *W = (double *)malloc(sizeof(double) * (size_t)(N * Ka));
    orc_dequantize_rows(acodes, ascales, M, Ka, A);
    orc_dequantize_rows(wcodes, wscales, N, Ka, W);
    long t;
#pragma omp parallel for schedule(static)
    for (t = 0; t < M; ++t)
        for (long n = 0; n < N; ++n) {
            double acc = 0.0;
            const double *a = A + t * Ka, *w = W + n * Ka;
            for (long j = 0; j < Ka; ++j) acc += a[j] * w[j];
            y[t * N + n] = acc;
        }
    free(A);
    free(W);
    return 0;
}

/* Unquantised reference Y = Z W^T in FP64 from the bf16 inputs (the target of the
 * normalised reconstruction error after Eq. (3)). */
int orc_matmul_bf16(const uint16_t *x_bf16, long M, const uint16_t *W_bf16, long N, long K, double *y) {
    long t;
#pragma omp parallel for schedule(static)
    for (t = 0; t < M; ++t)
        for (long n = 0; n < N; ++n) {
            double acc = 0.0;
            for (long j = 0; j < K; ++j)
                acc += (double)orc_bf16_to_f32(x_bf16[t * K + j]) * (double)orc_bf16_to_f32(W_bf16[n * K + j]);
            y[t * N + n] = acc;
        }
    return 0;
}

/* A finite double rounded once to bf16 (8 significant bits, fp32's exponent range, subnormals kept), ties to the
 * even significand; returns the bf16 bit pattern. */
static uint16_t orc_double_to_bf16(double v) {
    double a = fabs(v), r;
    float f;
    uint32_t u;
    if (a == 0.0) {
        r = 0.0;
    } else if (a < ldexp(1.0, -126)) {
        r = ldexp(nearbyint(ldexp(a, 133)), -133);          /* subnormal range: fixed quantum 2^-133 */
    } else {
        int e;
        double m = frexp(a, &e);                            /* a = m 2^e, m in [0.5, 1) */
        r = ldexp(nearbyint(ldexp(m, 8)), e - 8);           /* 8 significant bits; nearbyint = ties to even */
    }
    f = (float)(v < 0.0 || (v == 0.0 && signbit(v)) ? -r : r);   /* exact, or +-infinity past the top of the range */
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

/* Eq. (1), middle line, and the "offline copy" of the Activation tail construction paragraph: the producer
 * weights that make the gated FFN emit Z D^-1 P directly.  Row j' of the folded up projection is row perm[j'] of
 * W_up times inv_s[perm[j']] (the exact product rounded once to bf16), row j' of the folded gate projection is
 * row perm[j'] of W_gate; with dup != 0 rows C .. C+k-1 of both repeat rows C-k .. C-1, so that the FFN emits
 * [Z~, Z~_tail].  W_up, W_gate: C x H bf16 (C = input channels of the down projection); outputs (C or C+k) x H.
 * W_gate / out_gate may be NULL. */
int orc_fold_producer(const uint16_t *W_up, const uint16_t *W_gate, long C, long H, const int32_t *perm,
                      const float *inv_s, long k, int dup, uint16_t *out_up, uint16_t *out_gate) {
    long rows = C + (dup ? k : 0), jp, h;
    if (k < 0 || k > C) return 1;
    for (jp = 0; jp < rows; ++jp) {
        long src_new = jp < C ? jp : C - k + (jp - C);      /* position in the permuted order */
        long j = perm[src_new];                             /* original channel */
        for (h = 0; h < H; ++h) {
            out_up[jp * H + h] = orc_double_to_bf16((double)orc_bf16_to_f32(W_up[j * H + h]) * (double)inv_s[j]);
            if (W_gate && out_gate) out_gate[jp * H + h] = W_gate[j * H + h];
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------------------
 * Second format: MXFP8 (OCP MX, E4M3 elements), the format the paper's end-to-end setting runs the attention
 * linears in (Experimental setup); plain W8A8 -- Eq. (2)'s compensation is defined for MXFP4 and is not applied.
 * The paper gives only the format's name; the reading mirrors the MXFP4 one:
 *   - blocks of 32 along the reduction axis, E8M0 scale 2^e with e = clamp(floor(log2 amax) - 8, -127, 127)
 *     (8 = exponent of the largest E4M3 magnitude 448 = 1.75 * 2^8), byte e + 127; all-zero block: byte 0;
 *   - elements: E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; subnormals below 2^-6 in steps of
 *     2^-9; no infinities; the all-ones pattern is NaN and never produced), round to nearest, ties to the even
 *     mantissa, magnitudes above 448 saturate to 448 (so amax / 2^e in (448, 512) saturates, as (6, 8) does in
 *     MXFP4); the sign of values that round to zero is kept. */
static double orc_e4m3_value(uint8_t code) {
    int ex = (code >> 3) & 15, man = code & 7;
    double mag = ex == 0 ? ldexp((double)man, -9) : ldexp(1.0 + man / 8.0, ex - 7);
    return (code & 0x80) ? -mag : mag;
}

static uint8_t orc_fp8_block_scale_byte(const float *v) {
    double amax = 0.0;
    for (int i = 0; i < ORC_BLOCK; ++i) {
        double a = fabs((double)v[i]);
        if (a > amax) amax = a;
    }
    if (amax == 0.0) return 0;
    int ex;
    (void)frexp(amax, &ex);
    int e = (ex - 1) - 8;
    if (e < -127) e = -127;
    if (e > 127) e = 127;
    return (uint8_t)(e + 127);
}

static uint8_t orc_e4m3_code(float v, int e) {
    double a = ldexp(fabs((double)v), -e);   /* exact */
    uint8_t sign = (uint8_t)(orc_signbit_f32(v) << 7);
    if (a >= 464.0) return (uint8_t)(sign | 0x7E);          /* past the midpoint to the next step: saturate at 448 */
    if (a < ldexp(1.0, -6)) {                                /* subnormal range: multiples of 2^-9 */
        int q = (int)nearbyint(ldexp(a, 9));                 /* ties to even */
        return (uint8_t)(sign | (q == 8 ? 0x08 : q));
    }
    int ex;
    double m = frexp(a, &ex);                                /* a = m 2^ex, m in [0.5, 1) */
    int q = (int)nearbyint(ldexp(m, 4));                     /* 4 significant bits: 8 .. 16 */
    int eu = ex - 1;
    if (q == 16) { q = 8; eu += 1; }
    if (eu > 8 || (eu == 8 && q > 14)) return (uint8_t)(sign | 0x7E);
    return (uint8_t)(sign | ((eu + 7) << 3) | (q - 8));
}

/* Q of the second format, storage half: rows x cols fp32 -> codes (rows x cols bytes), scale bytes (rows x cols/32). */
int orc_fp8_quantize_rows(const float *v, long rows, long cols, uint8_t *codes, uint8_t *scales) {
    if (cols % ORC_BLOCK) return 1;
    for (long r = 0; r < rows; ++r)
        for (long b = 0; b < cols / ORC_BLOCK; ++b) {
            const float *blk = v + r * cols + b * ORC_BLOCK;
            uint8_t byte = orc_fp8_block_scale_byte(blk);
            scales[r * (cols / ORC_BLOCK) + b] = byte;
            for (int i = 0; i < ORC_BLOCK; ++i) codes[r * cols + b * ORC_BLOCK + i] = orc_e4m3_code(blk[i], (int)byte - 127);
        }
    return 0;
}

int orc_fp8_dequantize_rows(const uint8_t *codes, const uint8_t *scales, long rows, long cols, double *out) {
    if (cols % ORC_BLOCK) return 1;
    for (long r = 0; r < rows; ++r)
        for (long j = 0; j < cols; ++j)
            out[r * cols + j] = ldexp(orc_e4m3_value(codes[r * cols + j]), (int)scales[r * (cols / ORC_BLOCK) + j / ORC_BLOCK] - 127);
    return 0;
}

/* Offline half for one alpha: s as in the MXFP4 path, W0 = fl32(W * s), Q by rows.  No permutation, no tail. */
int orc_fp8_prepare(const uint16_t *W_bf16, long N, long K, const float *amax, double alpha, float *s, float *inv_s,
                    uint8_t *wcodes, uint8_t *wscales) {
    if (K % ORC_BLOCK) return 1;
    orc_scales_from_amax(amax, K, alpha, s, inv_s);
    float *W0 = (float *)malloc(sizeof(float) * N * K);
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K; ++j)
            W0[n * K + j] = (float)((double)orc_bf16_to_f32(W_bf16[n * K + j]) * (double)s[j]);
    orc_fp8_quantize_rows(W0, N, K, wcodes, wscales);
    free(W0);
    return 0;
}

/* Online half, activation side: xt[t,j] = fl32(x[t,j] * inv_s[j]) (inv_s may be NULL: identity), then Q by rows. */
int orc_fp8_quantize_act(const uint16_t *x_bf16, long M, long K, const float *inv_s, uint8_t *codes, uint8_t *scales) {
    if (K % ORC_BLOCK) return 1;
    float *row = (float *)malloc(sizeof(float) * K);
    for (long t = 0; t < M; ++t) {
        for (long j = 0; j < K; ++j) {
            double v = (double)orc_bf16_to_f32(x_bf16[t * K + j]);
            if (inv_s) v = v * (double)inv_s[j];
            row[j] = (float)v;
        }
        orc_fp8_quantize_rows(row, 1, K, codes + t * K, scales + t * (K / ORC_BLOCK));
    }
    free(row);
    return 0;
}

/* y[t,n] = sum_j deq(A)[t,j] deq(W)[n,j] in FP64, ascending j. */
int orc_fp8_matmul(const uint8_t *acodes, const uint8_t *ascales, const uint8_t *wcodes, const uint8_t *wscales,
                   long M, long N, long K, double *y) {
    if (K % ORC_BLOCK) return 1;
    double *a = (double *)malloc(sizeof(double) * M * K);
    double *w = (double *)malloc(sizeof(double) * N * K);
    orc_fp8_dequantize_rows(acodes, ascales, M, K, a);
    orc_fp8_dequantize_rows(wcodes, wscales, N, K, w);
    long t;
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (t = 0; t < M; ++t)
        for (long n = 0; n < N; ++n) {
            double acc = 0.0;
            for (long j = 0; j < K; ++j) acc += a[t * K + j] * w[n * K + j];
            y[t * N + n] = acc;
        }
    free(a); free(w);
    return 0;
}

/* Gated FFN activation of the producer (the function f of Eq. (1), middle line, for a SiLU-gated FFN):
 * h[i] = bf16( silu(g[i]) * u[i] ) with silu(g) = g / (1 + exp(-g)), evaluated in FP64 and rounded once.
 * g, u: n doubles (the gate and up projections' sums); h: n bf16 bit patterns. */
void orc_silu_mul_bf16(const double *g, const double *u, long n, uint16_t *h) {
    long i;
    for (i = 0; i < n; ++i) {
        double s = g[i] / (1.0 + exp(-g[i]));
        h[i] = orc_double_to_bf16(s * u[i]);
    }
}

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
