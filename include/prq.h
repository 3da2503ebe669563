/*
 * prq.h -- C ABI of libprq: the PRQuant compensated W4A4 MXFP4 linear layer on
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the inference hot path of the paper's Method section:
 * offline, a weight W (N x K) is scaled per input channel, its k hardest channels
 * are permuted into a contiguous tail and the tail's quantisation residual is
 * appended, giving one MXFP4 matrix over K + k columns (Algorithm 1, Eq. (2));
 * online, the activation is quantised to MXFP4 once and a single block-scaled FP4
 * GEMM over K + k, which re-reads the activation tail against the residual
 * columns, produces y (Eq. (3), "Kernel design for efficient inference").
 *
 * Conventions
 *   - Every function returns a prq_status; nothing throws across the boundary and
 *     outputs are left untouched when an argument check fails.
 *   - "host" / "device" is stated for every pointer.  Device buffers are owned by
 *     the caller (for example torch tensors); online calls never allocate, never
 *     synchronise the device and run on the given CUDA stream.
 *   - bf16 values are raw 16-bit patterns.  MXFP4 storage: 32-element blocks along
 *     the reduction axis, one E8M0 scale byte per block (value 2^(byte-127)),
 *     E2M1 elements packed two per byte with the even column in the low nibble.
 *   - K % 32 == 0, k_tail % 32 == 0 and 0 <= k_tail <= K are required: the tail starts and
 *     ends on 32-element block boundaries, which is the condition of the Kernel design
 *     paragraph under which copying the quantised tail equals quantising the widened row.
 *   - A prq_weights handle is immutable after creation and may be used from several
 *     streams at once.  It belongs to the device that was current when it was made, and
 *     every online call must be made with that device current (else INVALID_ARG).
 *   - A kernel that gives up on a bounded wait records PRQ_ERR_TIMEOUT in a device
 *     status word that prq_last_device_status() reads; it never traps or spins forever.
 */
#ifndef PRQ_H_
#define PRQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PRQ_OK = 0,
    PRQ_ERR_INVALID_ARG = 1,
    PRQ_ERR_ALIGNMENT = 2,
    PRQ_ERR_UNSUPPORTED_ARCH = 3,
    PRQ_ERR_CUDA = 4,
    PRQ_ERR_OOM = 5,
    PRQ_ERR_TIMEOUT = 6,
    PRQ_ERR_NONFINITE = 7,
    PRQ_ERR_WORKSPACE = 8,
    PRQ_ERR_STATIC_SCRATCH = 9
} prq_status;

typedef struct prq_weights prq_weights; /* opaque: prepared weights of one layer (or of E stacked experts) */
typedef void *prq_stream_t;             /* a cudaStream_t; NULL is the default stream */

typedef enum { PRQ_F32 = 0, PRQ_BF16 = 1 } prq_dtype;

/* Which activation transform prq_quantize_act applies before quantising. */
typedef enum {
    PRQ_ACT_IDENTITY = 0,  /* x is already Z D^-1 P (folded into the producer layers, Eq. (1)) */
    PRQ_ACT_SCALE_PERM = 1 /* apply x[t, perm[j]] * inv_s[perm[j]] online */
} prq_act_mode;

/* Host-side views that prq_weights_get copies out (for parity checks and export). */
typedef enum {
    PRQ_FIELD_CODES = 0,   /* uint8  N x (K+k)/2   packed E2M1 codes of [Q(W D P) | Q(R)]            */
    PRQ_FIELD_SCALES = 1,  /* uint8  N x (K+k)/32  E8M0 bytes, row-major                             */
    PRQ_FIELD_PERM = 2,    /* int32  K             new position -> original channel                   */
    PRQ_FIELD_TOPK = 3,    /* int32  k             selected channels, ascending (= perm[K-k..K))      */
    PRQ_FIELD_S = 4,       /* float  K             s_j = max(amax_j, 1e-5)^alpha, original order      */
    PRQ_FIELD_INV_S = 5,   /* float  K             fl32(1 / s_j)                                      */
    PRQ_FIELD_COL_ERR = 6  /* double K             column-wise quantisation error used for the ranking */
} prq_field;

typedef enum {
    PRQ_BUF_CODES = 0,      /* M x K/2 bytes                                                    */
    PRQ_BUF_SCALES_ROW = 1, /* M x K/32 bytes, row-major (optional output, parity view)         */
    PRQ_BUF_SCALES_SF = 2   /* scale bytes in the GEMM's tile order, tail scales duplicated     */
} prq_buf;

/* ---- offline (Algorithm 1) ------------------------------------------------------------- */

/* Algorithm 1 steps 3-7 and 11 for one given alpha: scale W by s = amax^alpha, rank the input
 * channels by the MXFP4 quantisation error of the scaled weight, move the k_tail worst to a
 * contiguous tail, quantise, compute the tail residual R (Eq. (2)), quantise it and store
 * [Q(W D P) | Q(R)] on the current device in the GEMM's layout.
 *   W         host, n_experts x N x K bf16, row-major (ld = K)
 *   act_amax  host, n_experts x K float: max_t |Z_cal[t, j]| per input channel (step 1)
 *   out       receives the handle; release it with prq_weights_free
 * Runs on the host (multi-threaded) and uploads once.  Errors: INVALID_ARG (NULL, sizes,
 * alignment of K / k_tail), NONFINITE (W, amax), UNSUPPORTED_ARCH (no sm_100 device), CUDA, OOM. */
prq_status prq_prepare_weights(const uint16_t *W, int n_experts, int N, int K, const float *act_amax,
                               float alpha, int k_tail, prq_weights **out);

/* Options of the offline pipeline.  Set struct_size = sizeof(prq_prep_opts); NULL means all defaults.
 *   weight_scale_search  0 (default): every weight block takes the floor-rule scale.
 *                        1: the "E8M0-W" variant of the paper's ablation study (local block-scale search):
 *                           every block of Q(W D P) and of Q(R) takes, of the floor-rule exponent and its
 *                           two neighbours, the one with the smallest squared quantisation error (a
 *                           neighbour only if strictly better).  Channel ranking, permutation and scales s
 *                           are not affected; R is the residual of the searched quantisation.  The GEMM is
 *                           untouched.
 *   gated_producer       0 (default): an ordinary layer.
 *                        1: the layer is the stacked gate / up projection of a gated FFN in the row order of
 *                           prq_stack_gate_up, to be run by prq_linear_gated.  The prepared weights are the same;
 *                           the handle keeps the scale-byte tiling of that call's kernel instead of those of
 *                           prq_linear, which therefore refuses it for more than 128 tokens.
 *   format               PRQ_FMT_MXFP4 (default): the paper's format for the FFN / expert layers.
 *                        PRQ_FMT_MXFP8: E4M3 elements with the same 32-element E8M0 block scales, the format the
 *                           paper's end-to-end setting runs the attention linears in (Experimental setup), as plain
 *                           W8A8: k_tail must be 0 (Eq. (2)'s compensation is defined for MXFP4), alpha still scales.
 *                           Served by prq_quantize_act and prq_linear (dense layers, any M); buffer sizes come from
 *                           prq_act_bytes_for.  The other online calls return INVALID_ARG for such a handle.
 * A caller compiled against an earlier header may pass its smaller struct: fields beyond struct_size read as 0. */
typedef enum { PRQ_FMT_MXFP4 = 0, PRQ_FMT_MXFP8 = 1 } prq_format;
typedef struct prq_prep_opts {
    size_t struct_size;
    int weight_scale_search;
    int gated_producer;
    int format;
} prq_prep_opts;

/* prq_prepare_weights with options (opts may be NULL).  Errors as prq_prepare_weights, plus INVALID_ARG for a
 * struct_size smaller than the first version of the struct (16 bytes). */
prq_status prq_prepare_weights_opts(const uint16_t *W, int n_experts, int N, int K, const float *act_amax,
                                    float alpha, int k_tail, const prq_prep_opts *opts, prq_weights **out);

/* Several layers that read the SAME activation (q / k / v, gate / up), prepared as ONE PRQuant layer: their weights are
 * stacked along the output axis and go through Algorithm 1 together -- the scale s depends on the shared input only,
 * and one permutation and one tail are chosen from the stacked matrix's column errors -- so that one activation
 * quantisation and one product serve the whole group.  (The paper applies the method per linear; this is the same method
 * applied to the fused projection.)  The handle is an ordinary one with N = sum of N_i: layer i's outputs are columns
 * [sum_{j<i} N_j, + N_i) of prq_linear's y.
 *   Ws        host array of n host pointers, layer i: N_i x K bf16 row-major
 *   Ns        host array of n row counts        act_amax  host, K floats        opts  may be NULL
 * Errors as prq_prepare_weights_opts; INVALID_ARG for n < 1 or a NULL entry. */
prq_status prq_prepare_weights_stacked(const uint16_t *const *Ws, const int *Ns, int n, int K, const float *act_amax,
                                       float alpha, int k_tail, const prq_prep_opts *opts, prq_weights **out);

/* prq_prepare_weights_opts for weights that already sit in DEVICE memory (Algorithm 1 steps 3-7 and 11 with
 * the heavy steps as kernels on the current device; the K channel scales and the ranking of the K column
 * errors stay on the host).  The handle is bit-for-bit the one prq_prepare_weights_opts builds from a host
 * copy of the same W.
 *   W_device  device, n_experts x N x K bf16 row-major (read only; not kept)
 *   act_amax  HOST, n_experts x K fp32          opts  may be NULL
 *   stream    the kernels and copies run there; the call synchronises it before it returns
 * Allocates temporaries on the device (codes, scale bytes and a few arrays of K elements) and frees them.
 * Errors as prq_prepare_weights; a NaN or an infinity in W * s gives NONFINITE. */
prq_status prq_prepare_weights_device(const uint16_t *W_device, int n_experts, int N, int K, const float *act_amax,
                                      float alpha, int k_tail, const prq_prep_opts *opts, prq_stream_t stream,
                                      prq_weights **out);

/* The same per-alpha pipeline as prq_prepare_weights, host buffers in and out, no device involved
 * (offline tooling, export, checks on machines without a GPU).  One layer.
 *   codes   host out, N x (K+k)/2    scales  host out, N x (K+k)/32    perm  host out, K int32
 *   s, inv_s (K floats) and col_err (K doubles) are optional (NULL to skip). */
prq_status prq_prepare_weights_host(const uint16_t *W, int N, int K, const float *act_amax, float alpha,
                                    int k_tail, uint8_t *codes, uint8_t *scales, int32_t *perm, float *s,
                                    float *inv_s, double *col_err);

/* prq_prepare_weights_host with options (opts may be NULL).  With format = PRQ_FMT_MXFP8: k_tail must be 0, codes is
 * N x K bytes, perm comes back as the identity and col_err as zeros. */
prq_status prq_prepare_weights_host_opts(const uint16_t *W, int N, int K, const float *act_amax, float alpha,
                                         int k_tail, const prq_prep_opts *opts, uint8_t *codes, uint8_t *scales,
                                         int32_t *perm, float *s, float *inv_s, double *col_err);

/* Algorithm 1 steps 1-10: derive amax from the calibration rows, run the per-alpha pipeline for
 * every candidate, evaluate Eq. (3) on the calibration rows with the GPU kernels and keep the
 * alpha with the smallest normalised error ||Yhat - Z W^T||_F / ||Z W^T||_F (first minimum).
 *   Zcal       host, T x K bf16 (one layer; n_experts must be 1)
 *   alphas     host, n_alphas candidates
 *   alpha_star receives the chosen alpha; nrmse (host, n_alphas doubles, nullable) every error */
prq_status prq_prepare_weights_search(const uint16_t *W, int N, int K, const uint16_t *Zcal, int T,
                                      const float *alphas, int n_alphas, int k_tail, prq_weights **out,
                                      float *alpha_star, double *nrmse);

void prq_weights_free(prq_weights *w);

/* A second, independent device copy of a handle's prepared weights (same device): serving several
 * streams from separate memory, or benchmarks that rotate over more weight bytes than the L2 holds.
 * Not part of the paper's method.  Free it with prq_weights_free. */
prq_status prq_weights_clone(const prq_weights *w, prq_weights **out);

/* The "offline copy" form of a prepared layer (Activation tail construction paragraph: the producer layers emit the k tail
 * channels a second time, so that the activation already has K + k columns and nothing is re-read).
 * Returns an independent handle (its own device copy, free it with prq_weights_free) that presents the same
 * bytes [Q(W D P) | Q(R)] as a plain MXFP4 layer with K' = K + k input channels and no tail:
 *   prq_quantize_act(view, PRQ_ACT_IDENTITY, x_wide, ...)   x_wide: M x (K + k), columns [K, K + k) a copy of
 *                                                           columns [K - k, K) of the permuted, scaled activation
 *   prq_linear / prq_linear_fused / prq_linear_grouped(view, ...)
 * give bit for bit what the original handle gives on the first K columns (block alignment makes quantising
 * the widened row equal to widening the quantised row).  Scaling and permutation are the producer's job in
 * this form: the view's perm is the identity on K + k channels and its scales are 1.
 * INVALID_ARG if k > 0 and K is not a multiple of 256 (the residual columns would not start on a stage of the
 * scale-byte layout; all of the paper's shapes satisfy it). */
prq_status prq_weights_offline_copy(const prq_weights *w, prq_weights **out);

/* Eq. (1), middle line: fold a down projection's inverse scaling and permutation into the layers that produce
 * its input, so that the gated FFN emits Z D^-1 P directly and prq_quantize_act runs in PRQ_ACT_IDENTITY mode:
 *   out_up  [j', :] = bf16( W_up[perm[j'], :] * inv_s[perm[j']] )     (exact product, rounded once, ties to even)
 *   out_gate[j', :] =       W_gate[perm[j'], :]
 * for j' in [0, C); with duplicate_tail != 0 rows C .. C + k_tail - 1 of both outputs repeat rows C - k_tail ..
 * C - 1 (the "offline copy" of the Activation tail construction paragraph; pair it with
 * prq_weights_offline_copy).  All pointers are HOST memory:
 *   perm, inv_s   C entries each, as prq_weights_get returns them (PRQ_FIELD_PERM, PRQ_FIELD_INV_S)
 *   W_up, W_gate  C x H bf16 row-major (C = input channels of the down projection = output features of the
 *                 producers, H = their input features); W_gate and out_gate may both be NULL
 *   out_up, out_gate   (C or C + k_tail) x H bf16, caller-owned
 * INVALID_ARG for a perm entry outside [0, C), a non-finite inv_s, k_tail outside [0, C]. */
prq_status prq_fold_producer(const int32_t *perm, const float *inv_s, int C, int k_tail, const uint16_t *W_up,
                             const uint16_t *W_gate, int H, int duplicate_tail, uint16_t *out_up,
                             uint16_t *out_gate);

/* Rows of a gate and an up projection interleaved in groups of 32, the row order prq_linear_gated expects:
 *   out[64 b + i] = W_gate[32 b + i],  out[64 b + 32 + i] = W_up[32 b + i]     (b < C / 32, i < 32)
 * so that 64 consecutive output features of the stacked layer are the gate and the up sums of ONE 32-channel block
 * of the down projection's input.  All pointers are HOST memory: W_gate, W_up C x H bf16 row-major (normally the
 * outputs of prq_fold_producer, so that the product arrives scaled and in the down projection's channel order),
 * out 2 C x H.  INVALID_ARG unless C % 32 == 0. */
prq_status prq_stack_gate_up(const uint16_t *W_gate, const uint16_t *W_up, int C, int H, uint16_t *out);

/* Shape of a handle.  Any output pointer may be NULL. */
prq_status prq_weights_info(const prq_weights *w, int *n_experts, int *N, int *K, int *k_tail, float *alpha);

/* Format of a handle (a prq_format).  INVALID_ARG for NULL. */
prq_status prq_weights_format(const prq_weights *w, int *format);

/* Copy one canonical host-side view of expert `expert` into dst (host, dst_bytes must match).  For an MXFP8 handle
 * PRQ_FIELD_CODES is N x K bytes of E4M3 codes. */
prq_status prq_weights_get(const prq_weights *w, int expert, prq_field which, void *dst, size_t dst_bytes);

/* ---- online ------------------------------------------------------------------------------ */

/* Size in bytes of an activation-side buffer for M rows.  For grouped calls pass the total row
 * count and n_groups = number of experts (each group's scale tiles are padded to 128 rows);
 * dense calls pass n_groups = 1.  Returns 0 for invalid arguments. */
size_t prq_act_bytes(int M, int K, int k_tail, int n_groups, prq_buf which);

/* The same sizes for the layer behind a handle, whatever its format (MXFP8: one byte per code, scale bytes in
 * 512-byte groups per 128-element stage).  Dense layers; returns 0 for invalid arguments. */
size_t prq_act_bytes_for(const prq_weights *w, int M, prq_buf which);

/* The single MXFP4 quantisation of the reordered activation that the Kernel design paragraph calls for.
 * One launch: optional scale + permute (Eq. (1), activation side), per-32 amax, E8M0 scale,
 * E2M1 round-to-nearest-even codes.  The quantised tail is not copied: only its k_tail/32 scale
 * bytes per row are duplicated into the tile-ordered scale buffer, the GEMM re-reads the codes.
 *   w               handle (gives K, k_tail, perm, inv_s); required
 *   mode            PRQ_ACT_IDENTITY or PRQ_ACT_SCALE_PERM
 *   x               device, M x K bf16, row stride ldx elements (ldx >= K, ldx % 8 == 0, 16-byte aligned)
 *   expert_offsets  device, n_experts + 1 int32 row boundaries when w stacks experts (rows sorted by
 *                   expert; expert e uses its own perm / inv_s); NULL for a dense layer
 *   codes           device out, PRQ_BUF_CODES bytes (16-byte aligned)
 *   scales_row      device out or NULL, PRQ_BUF_SCALES_ROW bytes
 *   scales_sf       device out, PRQ_BUF_SCALES_SF bytes (16-byte aligned)
 * A single layer (n_experts == 1) may also be given a two-entry expert_offsets {0, M}: the buffers then have
 * the grouped layout with one group, which prq_linear_grouped consumes.
 * Precondition: x is finite.  The kernel does not look for NaN or infinities (a scan would cost a second pass
 * over a memory-bound kernel); a block that holds one gets a meaningless scale byte and the product is
 * undefined for that row.  The offline calls do check W and amax (NONFINITE).
 * Errors: INVALID_ARG / ALIGNMENT before anything is enqueued.  In scale + permute mode a dense layer of 512 rows or
 * more is fetched by bulk copies whose waits are bounded like every device wait of this library: if one ran out the
 * kernel returns early and PRQ_ERR_TIMEOUT is recorded in the device status word (prq_last_device_status); the output
 * buffers are then incomplete.
 * M == 0 is a no-op. */
prq_status prq_quantize_act(const prq_weights *w, prq_act_mode mode, const void *x, int M, int ldx,
                            const int32_t *expert_offsets, void *codes, void *scales_row, void *scales_sf,
                            prq_stream_t stream);

/* Scratch prq_linear needs for M rows: 0 for M <= 128 (the split-K partial sums of the decode kernel meet
 * in distributed shared memory); for larger M the stream-K prefill kernel needs two counters per 128-row
 * half of an output tile and two fp32 partial tiles per SM (about 34 MB on a B200).  Calls on different
 * streams that may overlap need separate workspaces. */
size_t prq_linear_workspace_bytes(const prq_weights *w, int M);

/* Eq. (3): y = [Q(x) | Q(x)_tail] [Q(W D P) | Q(R)]^T, one block-scaled FP4 GEMM over K + k with fp32
 * accumulation.  Reads activation columns [0, K) and then [K - k, K) again; no M x (K + k) buffer exists.
 *   codes, scales_sf  device, as written by prq_quantize_act for the same w and M
 *   y                 device out, M x N, row stride ldy elements, dtype y_dtype (fp32 for parity)
 *                     (only columns [0, N) of a row are written: y may be a column slice of a wider matrix)
 *   workspace         device, at least prq_linear_workspace_bytes(w, M) bytes, 16-byte aligned (may be NULL
 *                     when that is 0); zero-filled by the caller before its first use, the kernel leaves
 *                     its flags zeroed again -- except after a wait inside the kernel ran out
 *                     (prq_last_device_status returned PRQ_ERR_TIMEOUT): zero-fill it again then
 * M <= 128 takes the weight-streaming cluster split-K kernel, larger M the stream-K prefill kernel.
 * Errors: INVALID_ARG, ALIGNMENT (y, ldy, workspace), WORKSPACE (too small), CUDA (launch failed). */
prq_status prq_linear(const prq_weights *w, const void *codes, const void *scales_sf, int M, void *y, int ldy,
                      prq_dtype y_dtype, void *workspace, size_t workspace_bytes, prq_stream_t stream);

/* prq_linear for callers that can neither allocate device memory nor hand over a workspace.  (The paper
 * has no counterpart to this call; it exists for deployment.)  Think of an inference server whose memory
 * pool already owns the whole GPU, so that a later cudaMalloc would fail, or of a plugin that runs inside
 * a host application which forbids allocation calls on its threads.  The product is the same as
 * prq_linear's; the stream-K scratch (tile flags and fp32 partial tiles) lives in an array that is part
 * of the library image instead of in caller memory.
 *   - Arguments as for prq_linear, minus the workspace.  The handle's device must be the current device.
 *   - Limits: at most 8192 output half-tiles, counted as 2 * ceil(M/256) * ceil(N/224) (an upper bound: the
 *     kernel may pick 240-column tiles, of which there are no more), and at most 160 SMs; beyond
 *     that the call returns PRQ_ERR_STATIC_SCRATCH and launches nothing.  M <= 128 needs no scratch and is
 *     passed on.
 *   - Cost: the array is 42,008,576 bytes (64 KB of counters + 2 x 160 partial tiles of 128 KB) on every
 *     GPU that loads the library, until the process exits.
 *   - The call itself performs no allocation (no cudaMalloc / cudaFree, no allocating library routine); it
 *     enqueues one small memset of the flags and the kernel.  The first call on a device also looks up the
 *     array's device address; make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents (the flags are cleared on
 *     every call, the partial tiles are written before they are read).  Two calls that can overlap on the
 *     GPU -- different streams, or one stream per thread -- race on it: serialise them, or give the
 *     overlapping callers prq_linear with workspaces of their own. */
prq_status prq_linear_static_scratch(const prq_weights *w, const void *codes, const void *scales_sf, int M, void *y,
                                     int ldy, prq_dtype y_dtype, prq_stream_t stream);

/* Eq. (1), middle line, with the producer's activation function inside the producer's GEMM: the gate and up
 * projections of a gated FFN as one layer whose output never exists in bf16.  One launch computes
 *   g, u = the two halves of prq_linear(w_gu, codes, scales_sf)      (fp32 sums, never stored)
 *   h    = bf16( silu(g) * u ),  silu(g) = g / (1 + exp(-g)) in fp32
 *   Q(h) = the MXFP4 quantisation prq_quantize_act(w_down, PRQ_ACT_IDENTITY, h) would give
 * and writes Q(h) -- codes, tile-ordered scale bytes with the tail's bytes duplicated, optionally row-major scale
 * bytes -- ready for prq_linear(w_down, ...).  With the down projection's 1 / s and permutation folded into the
 * producers (prq_fold_producer, then prq_stack_gate_up) this is the whole activation side of Eq. (1): the separate
 * quantiser launch and the bf16 round trip of h (2 x M x C bytes written, M x C read back) are gone.
 *   w_gu              handle of the stacked layer (2 C output features), prepared with gated_producer = 1
 *   codes, scales_sf  device, the quantised hidden state as prq_quantize_act wrote it for w_gu and M
 *   w_down            handle of the down projection (gives C = its input channels and its tail k); needs
 *                     C % 256 == 0 and k % 256 == 0 (whole reduction stages; the paper's shapes have both)
 *   out_codes         device out, prq_act_bytes(M, C, k, 1, PRQ_BUF_CODES) bytes, 16-byte aligned
 *   out_scales_row    device out or NULL, PRQ_BUF_SCALES_ROW bytes
 *   out_scales_sf     device out, PRQ_BUF_SCALES_SF bytes, 16-byte aligned
 *   h_check           device out or NULL: M x C bf16, the product before quantisation (for checks; costs the traffic
 *                     the call exists to avoid)
 * The exponential is the GPU's fast one: h is within one bf16 unit in the last place of the exactly evaluated
 * product, and Q(h) is bit-for-bit the quantisation of the h this call forms.  Every token count takes the same
 * kernel (256-token tiles); a decode-shaped instance is not built.  Needs no workspace.
 * Errors: INVALID_ARG (shapes, a handle not prepared as gated producer, devices), ALIGNMENT, CUDA. */
prq_status prq_linear_gated(const prq_weights *w_gu, const void *codes, const void *scales_sf, int M,
                            const prq_weights *w_down, void *out_codes, void *out_scales_row, void *out_scales_sf,
                            void *h_check, prq_stream_t stream);

/* Decode step in one launch (Kernel design paragraph: the kernel quantises the reordered activation once
 * and multiplies): y = prq_linear(prq_quantize_act(x)) for up to PRQ_FUSED_MAX_M tokens, with the
 * activation quantised inside the GEMM kernel -- no code or scale buffer exists.  The result is bit-for-bit
 * the one of the two calls.
 *   mode   PRQ_ACT_IDENTITY only (the scale and the permutation were folded into x's producer, Eq. (1));
 *          PRQ_ACT_SCALE_PERM returns INVALID_ARG -- use the two calls
 *   x      device, M x K bf16, row stride ldx elements (multiple of 8), 16-byte aligned
 *   M      1 .. PRQ_FUSED_MAX_M (0 is a no-op); larger M returns INVALID_ARG
 *   y      device out, M x N, row stride ldy elements, dtype y_dtype
 * Dense layers only.  Needs no workspace.  Errors: INVALID_ARG, ALIGNMENT, CUDA. */
#define PRQ_FUSED_MAX_M 16
prq_status prq_linear_fused(const prq_weights *w, prq_act_mode mode, const void *x, int M, int ldx, void *y,
                            int ldy, prq_dtype y_dtype, prq_stream_t stream);

/* Several dense layers that read the same activation (q / k / v, gate / up), each with its own prepared
 * weights, served by one launch each of the quantiser and of the GEMM instead of n.  (Not in the paper: it
 * only saves launches; every layer's result is bit-for-bit the one of its own prq_quantize_act /
 * prq_linear calls.)  At decode batch sizes a launch costs as much as the work in it.
 *   n          1 .. PRQ_MULTI_MAX layers, all dense, on one device, with the same K
 *   ws         host array of n handles
 * prq_quantize_act_multi: x device, M x K bf16 (row stride ldx); codes[i], scales_sf[i] device out, sized by
 *   prq_act_bytes for layer i (k_tail may differ between the layers).  No row-major scales.
 * prq_linear_multi: M <= 128 only (the weight-streaming kernel); the layers must also share k_tail.
 *   codes[i], scales_sf[i] as written by the quantiser for layer i; y[i] device out, M x N_i, row stride ldy[i].
 * The pointer arrays are host arrays, read before the call returns.  Errors as for the single-layer calls. */
#define PRQ_MULTI_MAX 4
prq_status prq_quantize_act_multi(int n, const prq_weights *const *ws, prq_act_mode mode, const void *x, int M,
                                  int ldx, void *const *codes, void *const *scales_sf, prq_stream_t stream);
prq_status prq_linear_multi(int n, const prq_weights *const *ws, const void *const *codes,
                            const void *const *scales_sf, int M, void *const *y, const int *ldy,
                            prq_dtype y_dtype, prq_stream_t stream);

/* The same product for stacked experts (MoE): rows [expert_offsets[e], expert_offsets[e+1]) of the
 * activation use expert e's weights.  expert_offsets: device, n_experts + 1 int32, non-decreasing,
 * last = M_total. */
prq_status prq_linear_grouped(const prq_weights *w, const void *codes, const void *scales_sf,
                              const int32_t *expert_offsets, int M_total, void *y, int ldy, prq_dtype y_dtype,
                              prq_stream_t stream);

/* Whole online path from HOST buffers: copies x (host, M x K bf16, pinned for speed) to the device,
 * quantises, multiplies and copies y (M x N, y_dtype) back to y_host, all on `stream`, using
 * caller-provided device scratch of at least prq_forward_host_scratch_bytes(w, M) bytes (zero-filled
 * before its first use).  Returns after enqueueing; synchronise the stream before reading y_host. */
size_t prq_forward_host_scratch_bytes(const prq_weights *w, int M);
prq_status prq_forward_host(const prq_weights *w, prq_act_mode mode, const uint16_t *x_host, int M,
                            void *y_host, prq_dtype y_dtype, void *dev_scratch, size_t scratch_bytes,
                            prq_stream_t stream);

/* ---- diagnostics ----------------------------------------------------------------------- */

const char *prq_status_string(prq_status s);

/* Synchronises `stream`, then reads and clears the status word of the CURRENT device, which a kernel sets
 * when a bounded wait expired (PRQ_ERR_TIMEOUT).  PRQ_OK when nothing went wrong.  After PRQ_ERR_TIMEOUT the
 * outputs of the calls since the last check are undefined and a prq_linear workspace must be zero-filled
 * again; the context stays usable. */
prq_status prq_last_device_status(prq_stream_t stream);

/* Number of kernels this library has launched in this process (for benchmark bookkeeping). */
unsigned long long prq_kernel_launch_count(void);

/* Benchmark utility (the paper has no counterpart): launches, on `stream`, one CTA per SM that issues
 * n_mma back-to-back block-scaled FP4 tensor-core instructions (M = 128, N = 256, K = 64, i.e.
 * 2 * 128 * 256 * 64 flop each) on operands resident in shared memory -- no loads, no epilogue.  The
 * caller times the launch; SMs * n_mma * 4,194,304 flop / time is the FP4 tensor rate this GPU sustains
 * at the clocks it holds under that load.  n_mma: multiple of 4, 4 .. 2^24.  *n_ctas (nullable) receives
 * the number of CTAs launched.  Errors: INVALID_ARG, CUDA. */
prq_status prq_mxf4_peak_probe(int n_mma, int *n_ctas, prq_stream_t stream);

/* Benchmark utility (the paper has no counterpart): enqueues, on `stream`, n empty kernels, each launched the way
 * the decode GEMM is (programmatic dependent launch; `grid` CTAs of `threads` threads in clusters of `cluster`
 * CTAs) and each waiting for the one before it.  The caller times the chain; time / n is what one dependent
 * launch costs on this GPU before any work is done -- the floor under every latency-bound call of this library.
 * n: 1 .. 4096; grid a multiple of cluster; cluster 1 .. 8.  Errors: INVALID_ARG, CUDA. */
prq_status prq_handover_probe(int n, int grid, int threads, int cluster, prq_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* PRQ_H_ */
