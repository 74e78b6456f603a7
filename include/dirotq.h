/*
 * libdirotq -- rotation-aware W4A4 linear layer (DiRotQ) for NVIDIA B200 (sm_100a).
 *
 * The layer computes, for activations X [M,K] and a weight W [K,N] (paper Sec. 4.1: Y = XW),
 *
 *     Y ~= [ X U_h , Q4(X U_l R) ] [ U_h^T W ; Q4((U_l R)^T W) ]          (paper Eq. 5)
 *
 * where V = [U_h, U_l R] is the calibrated orthogonal rotation (Sec. 4.2; here the argument
 * `Q`, column j = basis vector j, the first r columns = U_h), Q4 is the symmetric 4-bit
 * quantizer of Eq. 1 with z = 0, s = max|.|/7, applied per group of `group` consecutive
 * low-precision coefficients (Sec. 5.1: group size 64, 16-bit scales), per token for the
 * activations and per output column for the weights.  The first r rotated coefficients and the
 * first r rows of the folded weight stay bf16.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the name says `host`.
 *     The library allocates no device memory.  `stream` is a cudaStream_t passed as void*.
 *   - Calls enqueue work on `stream` and return without synchronising, unless stated.
 *   - Argument errors are reported before anything is launched.  A CUDA launch error is
 *     returned as DIROTQ_ERR_CUDA.  Device-side waits are bounded; when one expires the kernel
 *     records a code in the workspace status word (see dirotq_workspace_status) and returns.
 *   - A workspace must be zero-filled once before its first use: its first word is a sticky
 *     device status (0 = no wait ever expired).
 *   - Supported shapes: K % 64 == 0, N % 16 == 0, r a multiple of 16 with r < K and r <= 4096 (the paper keeps
 *     about a tenth of the coefficients in 16 bits: r = 112..128 for K = 1152, 304..320 for K = 3072),
 *     group in {64, 128} with K % group == 0, M >= 1.  Pointers must be 16-byte aligned.
 *   - Groups are counted from the first low-precision coefficient; the last one may be ragged.
 *     Rounding is to nearest, ties to even; scales are bf16 values; a group whose absolute
 *     maximum is zero has scale 0 and codes 0.
 */
#ifndef DIROTQ_H_
#define DIROTQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DIROTQ_API __attribute__((visibility("default")))
#else
#define DIROTQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dirotq_layer dirotq_layer_t; /* opaque host-side handle of a prepared layer */
typedef void* dirotq_stream_t;              /* a cudaStream_t */

typedef enum {
    DIROTQ_OK = 0,
    DIROTQ_ERR_INVALID_ARG = 1,
    DIROTQ_ERR_UNSUPPORTED_SHAPE = 2,
    DIROTQ_ERR_BUFFER_TOO_SMALL = 3,
    DIROTQ_ERR_ARCH = 4,           /* device is not sm_100 */
    DIROTQ_ERR_CUDA = 5,           /* a CUDA runtime / driver call failed */
    DIROTQ_ERR_DEVICE_TIMEOUT = 6  /* a bounded device-side wait expired */
} dirotq_status_t;

enum { DIROTQ_DTYPE_F32 = 0, DIROTQ_DTYPE_BF16 = 1, DIROTQ_DTYPE_F64 = 2 };
enum { DIROTQ_LAYOUT_KN = 0 /* W[k*N + n] */, DIROTQ_LAYOUT_NK = 1 /* W[n*K + k] */ };

/* Human-readable name of a status code (static string, never NULL). */
DIROTQ_API const char* dirotq_status_string(dirotq_status_t s);

/* Library version (major*10000 + minor*100 + patch). */
DIROTQ_API int dirotq_version(void);

/* Last CUDA error text recorded by this thread's most recent failing call ("" if none). */
DIROTQ_API const char* dirotq_last_error(void);

/* ---- sizes (host only, no CUDA call) ------------------------------------------------------ */

/* Bytes of the device blob that holds a prepared layer: the bf16 rotation (K*K*2), the packed
 * INT4 weight codes ((K-r rounded up to a group) * N / 2), their scales, the bf16 rank-r slice
 * and the bias. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes(int K, int N, int r, int group, size_t* bytes);

/* Bytes of the scratch buffer dirotq_prepare_layer needs (the fp64 folded weight, K*N*8). */
DIROTQ_API dirotq_status_t dirotq_prepare_scratch_bytes(int K, int N, size_t* bytes);

/* Bytes of the workspace one dirotq_linear call on M tokens needs (activation codes, scales,
 * the bf16 rank-r coefficients, a status word). */
DIROTQ_API dirotq_status_t dirotq_workspace_bytes(const dirotq_layer_t* layer, int M, size_t* bytes);

/* ---- offline: Eq. 5, right factor -------------------------------------------------------- */

/* Folds W~ = Q^T W in fp64 with the unrounded Q, keeps rows < r as bf16, quantizes rows >= r
 * to INT4 per (group, output column) with round-to-nearest and packs them, rounds Q to bf16
 * for the online rotation, converts the bias.
 *   W      device, [K,N] in `w_layout`, dtype `w_dtype` (F32 or BF16)
 *   Q      device, [K,K] row-major (Q[k*K + j] = component k of basis vector j), F64 or F32
 *   bias   device bf16 [N], or NULL
 *   blob   device, dirotq_layer_bytes() bytes, 1024-byte aligned; must outlive the handle
 *   scratch device, dirotq_prepare_scratch_bytes() bytes; free to reuse once `stream` has
 *          passed this call
 * On success *layer_out receives a host handle (free it with dirotq_layer_destroy). */
DIROTQ_API dirotq_status_t dirotq_prepare_layer(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                     const void* bias, int K, int N, int r, int group, void* blob,
                                     size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                     dirotq_stream_t stream, dirotq_layer_t** layer_out);

/* Frees the host handle (not the blob). */
DIROTQ_API dirotq_status_t dirotq_layer_destroy(dirotq_layer_t* layer);

/* Shape of a prepared layer.  Any output pointer may be NULL.  K_lp = n_g*group is the padded
 * width of the activation-code rows in the workspace. */
DIROTQ_API dirotq_status_t dirotq_layer_info(const dirotq_layer_t* layer, int* K, int* N, int* r, int* group, int* n_g,
                                  int* K_lp);

/* ---- online: Eq. 5, the whole right-hand side --------------------------------------------- */

/* y[M,N] (bf16, row-major) = DiRotQ-linear(x[M,K] bf16 row-major).  Two kernels are enqueued:
 * rotate+split+quantize (x Q_b on the bf16 tensor cores, Eq. 1 in the epilogue), then the
 * INT4 x INT4 group GEMM on the 8-bit tensor-core path (exact integer group sums) with the
 * per-group rescale, the bf16 rank-r branch and the bias.  Concurrent calls on one layer need distinct workspaces. */
DIROTQ_API dirotq_status_t dirotq_linear(const void* x, int M, const dirotq_layer_t* layer, void* y, void* workspace,
                              size_t workspace_bytes, dirotq_stream_t stream);

/* Same computation with HOST input and output (pinned memory, or the copies do not overlap):
 * copies x into x_dev, runs dirotq_linear, copies y_dev into y_host; x_dev [M,K] and y_dev [M,N]
 * are device staging buffers of the caller.  For M >= 2048 the call is cut into up to 8 row chunks
 * (token rows are independent) whose two copies run on two copy streams the library creates once
 * per device, overlapping each other and the kernels on `stream`; everything is ordered after the
 * work already on `stream`, and later work on `stream` (or a synchronisation of it) is ordered
 * after the last copy into y_host.  Not for use during stream capture. */
DIROTQ_API dirotq_status_t dirotq_linear_host(const void* x_host, int M, const dirotq_layer_t* layer, void* y_host,
                                   void* x_dev, void* y_dev, void* workspace, size_t workspace_bytes,
                                   dirotq_stream_t stream);

/* Reads the workspace status word.  SYNCHRONISES `stream`.  *device_code is 0 when every wait
 * completed; otherwise the role that gave up.  Returns DIROTQ_ERR_DEVICE_TIMEOUT in that case. */
DIROTQ_API dirotq_status_t dirotq_workspace_status(const void* workspace, dirotq_stream_t stream, int* device_code);

/* Diagnostics: the W4A4 kernel sums, per role, the SM cycles spent blocked on each kind of barrier
 * into 64-bit counters kept next to the status word.  Copies them out (SYNCHRONISES `stream`):
 * out[0] TMA producer waiting for a free stage, [1] MMA issuer waiting for operands (TMA + unpack),
 * [2] MMA issuer waiting for a free accumulator tile, [3] unpack warp waiting for TMA data,
 * [4] first epilogue warp waiting for a finished accumulator tile, [5] same warp waiting for
 * scales, [6] that warp's total cycles, [7] the MMA role's total cycles; all summed over CTAs
 * and over the calls since the workspace was last zeroed.  No counterpart in the paper. */
DIROTQ_API dirotq_status_t dirotq_workspace_wait_counters(const void* workspace, dirotq_stream_t stream,
                                                          unsigned long long out[8]);

/* ---- exports for parity checks ------------------------------------------------------------- */

/* Runs only the first kernel (rotation, split, Eq. 1) and leaves its results in `workspace`.
 * xrot_f32, if not NULL, receives the fp32 rotated activations [M,K] in the column order of Q. */
DIROTQ_API dirotq_status_t dirotq_rotate_quantize(const void* x, int M, const dirotq_layer_t* layer, void* workspace,
                                       size_t workspace_bytes, float* xrot_f32, dirotq_stream_t stream);

/* Runs only the second kernel (INT4 group GEMM, rescale, rank-r branch, bias) on a workspace
 * that dirotq_rotate_quantize filled for the same layer geometry and M.  Together the two calls
 * equal dirotq_linear; several layers that share one input and one rotation (the paper shares
 * nothing but allows it: the rotation depends only on the input's calibration statistics,
 * Sec. 4.2) can reuse a single rotate/quantize pass. */
DIROTQ_API dirotq_status_t dirotq_w4a4_gemm(int M, const dirotq_layer_t* layer, const void* workspace,
                                            size_t workspace_bytes, void* y, dirotq_stream_t stream);

/* Copies the first kernel's results out of the workspace into plain layouts:
 * xh bf16 [M,r]; codes int8 [M,K-r], one code per byte; scales bf16 [M,n_g]. */
DIROTQ_API dirotq_status_t dirotq_workspace_export(const dirotq_layer_t* layer, int M, const void* workspace, void* xh_bf16,
                                        int8_t* codes, void* scales_bf16, dirotq_stream_t stream);

/* Integer GEMM alone on caller-supplied activation codes (int8, one per byte, [M,K_lp] with
 * zero codes in columns >= K-r): partials[g][m][n] = sum over group g of q_x q_w, int32.
 * The codes are first converted into the workspace (its activation codes and scales are
 * overwritten), then the production kernel runs with unit scales and stores the group sums. */
DIROTQ_API dirotq_status_t dirotq_int_gemm_debug(const int8_t* act_codes, int M, const dirotq_layer_t* layer,
                                      int32_t* partials, void* workspace, size_t workspace_bytes,
                                      dirotq_stream_t stream);

/* Tuning knob of the second kernels (all four formats): output columns per tile.
 * 0 (default): chosen per call from M, N and the number of SMs (INT4: 256 columns unless 128-column tiles fill the
 * SMs so much better that they win although a narrow tile costs about 0.73 of a wide one, and 64 columns when even
 * 128-column tiles would keep under half of the SMs busy, i.e. for calls with few token rows; NVFP4 likewise with 0.6
 * and no 64-column plan);
 * 128 or 256: forced; 64: the grouped INT4 kernel's plan for few token rows, forced, one CTA per tile; 66: the same
 * tiles with the K-groups of a tile cut over a cluster of up to four CTAs (partial tiles added in one of them through
 * distributed shared memory) wherever every tile's cluster is resident at once and every CTA keeps two k-blocks; never
 * chosen automatically, because its outputs differ from the other plans' in fp32 summation order (a bf16 step on a few
 * values), and with 0 a token's output bits do not depend on how many tokens a call has; 192: the grouped INT4 kernel's plan
 * with three epilogue warpgroups (64 columns per thread), never chosen automatically: on the FLUX shapes it measured
 * between the other two; 512: the NVFP4 kernel in pairs of CTAs (clusters of two, tcgen05.mma.cta_group::2, 256 token
 * rows x 256 columns per pair, each CTA loading its own rows and one half of the weight tile), forced; 0 takes it
 * where its schedule is the shortest (a pair does two wide tiles' work in about 0.9 of a wide tile's time: every FLUX
 * shape at M = 4608).  A value that names a plan of
 * one kernel leaves the other formats' kernels choosing for themselves.  Process-wide; results do not depend on it (each
 * output element is accumulated in the same order).  Other values: DIROTQ_ERR_INVALID_ARG. */
DIROTQ_API dirotq_status_t dirotq_set_gemm_tile(int columns);

/* Tuning knob of the first kernel (rotation): tile plan.  0 (default): chosen per call from M, K and the number of
 * SMs; 1: 128 tokens x 128 rotated columns; 2: 128 x 256; 3: 256 x 256 (two MMAs share one tile of the rotation: a
 * third fewer operand bytes per flop, no overlap of the epilogue; pays where a layer has many tiles per SM, e.g.
 * K = 12288 at M = 4608); 4: 256 x 256 per PAIR of CTAs (clusters of two: tcgen05.mma.cta_group::2, each CTA loads its
 * own 128 rows of x and half of the rotation tile; the epilogue stays overlapped); 5: 128 x 64 (groups of 64 only, else
 * plan 1 is taken; for calls with few token rows, chosen when plan 1 would keep under half of the SMs busy).
 * Process-wide; results do not depend on it.  Other values: DIROTQ_ERR_INVALID_ARG. */
DIROTQ_API dirotq_status_t dirotq_set_rotation_tile(int plan);

/* Projection form, first step (x~_h = x U_hb): with few token-row tiles (M / 128 at most half the number of SMs) and K >= 2048 the
 * reduction over K is cut into up to 8 ranges that run as tiles of their own; their fp32 sums are parked in the
 * workspace's code region (not yet in use at that point) and a small kernel adds them in range order and rounds to
 * bf16.  On (default) or off, process-wide.  x~_h may differ in the last bf16 digit between the two settings (another
 * summation order); each setting is deterministic. */
DIROTQ_API dirotq_status_t dirotq_set_first_step_split(int enabled);

/* The second kernel of a layer is launched as a programmatic dependent launch: it may be scheduled onto SMs that
 * the first kernel's thread blocks have left and runs its set-up there, then waits (griddepcontrol.wait) for the
 * whole first kernel before it reads anything.  Results are unaffected; the launch gap between the two kernels
 * shrinks, which matters for small layers.  enabled == 0 switches this off process-wide (plain stream order),
 * anything else on (default).  Works in stream capture. */
DIROTQ_API dirotq_status_t dirotq_set_dependent_launch(int enabled);

/* Unpacks a prepared layer: wcodes int8 [K-r,N]; wscales bf16 [n_g,N]; wh bf16 [r,N];
 * q_bf16 [K,K] in the layout of the Q argument.  Any pointer may be NULL. */
DIROTQ_API dirotq_status_t dirotq_layer_export(const dirotq_layer_t* layer, int8_t* wcodes, void* wscales_bf16,
                                    void* wh_bf16, void* q_bf16, dirotq_stream_t stream);

/* ---- residual weights rounded by the caller (paper Sec. 4.1 and App. F.1: the residual weight is rounded with
 * GPTQ, which minimises the activation-weighted output error instead of rounding each value to nearest) ----
 *
 * As dirotq_prepare_layer (asym == 0) or dirotq_prepare_layer_asym (asym != 0), except that the INT4 codes and
 * scales of the folded rows r..K-1 are the caller's: wcodes int8 [K-r,N] (row j = rotated column r+j; values
 * outside -7..7 are clamped) and wscales bf16 [n_g,N], both DEVICE, row-major, read during the call only.
 * W and Q are still needed: the rows below r of Q^T W are kept in bf16 and Q is rounded for the online GEMM.
 * Any offline rounding (GPTQ on a calibration Hessian, a search over clipping ratios, ...) can be deployed
 * this way; the online path is the same. */
DIROTQ_API dirotq_status_t dirotq_prepare_layer_codes(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                      const void* bias, const int8_t* wcodes, const void* wscales_bf16,
                                                      int asym, int K, int N, int r, int group, void* blob,
                                                      size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                      dirotq_stream_t stream, dirotq_layer_t** layer_out);

/* ---- residual weights rounded with GPTQ inside the library (paper Sec. 4.1: the residual weight is rounded so as
 * to minimise ||X W - X W^||^2 on calibration tokens rather than value by value; App. "Quantization details":
 * damping 0.01, block size 128) ----
 *
 * As dirotq_prepare_layer (asym == 0) or dirotq_prepare_layer_asym (asym != 0), except that the folded rows
 * r..K-1 are rounded by the GPTQ algorithm: the Hessian is X~_l^T X~_l of the calibration tokens calib_x (bf16
 * [calib_tokens, K], DEVICE, row-major) rotated by the layer's own bf16 rotation; damp * mean(diag) is added to
 * its diagonal (the paper uses damp = 0.01); rows are rounded in order, each row's rounding error is spread over
 * the rows not yet rounded (weights from the upper Cholesky factor of the inverse Hessian), the rows behind the
 * current block of `block` rows (a multiple of `group`, at most 128; the paper uses 128) are corrected once per
 * block; a group's scale bf16(max|w|/7) is taken from its rows as they stand when the group starts.  Everything
 * runs on the device in fp64, offline; the factorisation is an unblocked one whose cost grows with (K-r)^3, which
 * is seconds at K = 3072.  scratch: DEVICE, dirotq_prepare_scratch_bytes_gptq bytes, free again when the call's
 * work on `stream` has completed.  The online path and every export are those of the round-to-nearest layer. */
DIROTQ_API dirotq_status_t dirotq_prepare_scratch_bytes_gptq(int K, int N, int r, int calib_tokens, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_gptq(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                     const void* bias, const void* calib_x, int calib_tokens, double damp,
                                                     int block, int asym, int K, int N, int r, int group, void* blob,
                                                     size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                     dirotq_stream_t stream, dirotq_layer_t** layer_out);

/* ---- layers that share one rotation (paper Sec. 4.2: the rotation belongs to a layer's INPUT, so linears that read
 * the same activations, e.g. the q, k and v projections of a block, are rotated by the same Q) ----
 *
 * A sibling layer is prepared like dirotq_prepare_layer (asym == 0) or dirotq_prepare_layer_asym (asym != 0) with the
 * SAME Q, r and group as the layer that owns the rotation, but its blob holds no copy of Q (K*K*2 bytes less).  It is
 * used through dirotq_w4a4_gemm on a workspace filled by dirotq_rotate_quantize of the owning layer; dirotq_linear,
 * dirotq_linear_host, dirotq_linear_noalloc, dirotq_rotate_quantize and the q_bf16 output of dirotq_layer_export
 * refuse it with DIROTQ_ERR_INVALID_ARG.  Q is still an argument: the weights are folded with it. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_sibling(int K, int N, int r, int group, int asym, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_sibling(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                        const void* bias, int asym, int K, int N, int r, int group,
                                                        void* blob, size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                        dirotq_stream_t stream, dirotq_layer_t** layer_out);

/* ---- projection form: a cheaper first stage (NOT the paper's Eq. 5; the formulation its remarks on the cost of the
 * online rotation point towards: paper Sec. 4.2 keeps only the leading r directions in 16 bits, App. E notes that the
 * rotation's cost and memory grow with the layer width) ----
 *
 *     x~_h = bf16(x U_hb)                       U_hb = bf16(U_h), U_h [K,r] the leading principal directions
 *     x~_l = (x H+- - x~_h V) / sqrt(group)     H+- block-diagonal, one Hadamard block of entries +-1 per quantization
 *                                               group (H = H+- / sqrt(group) is orthonormal); V = bf16(U_hb^T H+-) [r,K]
 *     y    = bf16( x~_h ((V H+-^T / group) W) + Q4(x~_l) Q4(H^T W) + bias )   Q4 as in dirotq_prepare_layer, over all K columns
 *
 * x H+- = sqrt(group) x~_l + x~_h V holds by construction and H+- H+-^T = group I, so the layer is x W exactly when
 * nothing is quantized, for any U_h; with V unrounded, x~_l is the block-Hadamard transform of the rounded projection's
 * residual x - x~_h U_hb^T.  Both terms of x~_l are matrix products (they run on the tensor core).
 * 4 M K r + 2 M K group flops instead of 2 M K^2 in the first stage, and no K x K matrix in the layer.  Uh: DEVICE, row-major [K,r],
 * uh_dtype DIROTQ_DTYPE_F64 or _F32; scratch: dirotq_prepare_scratch_bytes_ph bytes.  Such a layer is accepted by
 * dirotq_workspace_bytes, dirotq_linear, dirotq_linear_host, dirotq_rotate_quantize (xrot_f32 must be NULL),
 * dirotq_w4a4_gemm, dirotq_workspace_export (codes [M,K]), dirotq_int_gemm_debug, dirotq_layer_export (wcodes [K,N],
 * q_bf16 must be NULL), dirotq_layer_info (K_lp = K, n_g = K / group) and dirotq_layer_destroy. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_ph(int K, int N, int r, int group, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_scratch_bytes_ph(int K, int N, int r, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_ph(const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                                   const void* bias, int K, int N, int r, int group, void* blob,
                                                   size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                   dirotq_stream_t stream, dirotq_layer_t** layer_out);
/* The projection form with NVFP4 operands (as dirotq_prepare_layer_nvfp4, with Uh in place of Q; Hadamard blocks of 64,
 * E2M1 blocks of 16).  Accepted by the same calls as an NVFP4 layer; q_bf16 of dirotq_layer_export_nvfp4 and xrot_f32 of
 * dirotq_rotate_quantize must be NULL; scratch: dirotq_prepare_scratch_bytes_ph bytes. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_nvfp4_ph(int K, int N, int r, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_nvfp4_ph(const void* W, int w_dtype, int w_layout, const void* Uh,
                                                         int uh_dtype, const void* bias, int K, int N, int r,
                                                         int act_scale_log2, void* blob, size_t blob_bytes, void* scratch,
                                                         size_t scratch_bytes, dirotq_stream_t stream,
                                                         dirotq_layer_t** layer_out);
/* uh_bf16 [K,r]: the rounded projection the layer applies (U_hb); v_bf16 [r,K]: V = bf16(U_hb^T H+-).  DEVICE outputs,
 * row-major; projection-form layers only (DIROTQ_ERR_INVALID_ARG otherwise). */
DIROTQ_API dirotq_status_t dirotq_layer_export_uh(const dirotq_layer_t* layer, void* uh_bf16, dirotq_stream_t stream);
DIROTQ_API dirotq_status_t dirotq_layer_export_v(const dirotq_layer_t* layer, void* v_bf16, dirotq_stream_t stream);

/* ---- asymmetric activation codes (paper Sec. 3, Eq. 1 with z = min X; Sec. 5.1: the 4-bit INT setting
 * quantizes the activations asymmetrically) ---- */

/* Same layer, but every group of G low-precision coefficients of a token is quantized to unsigned
 * codes u in 0..15 with a bf16 scale s = (max - min) / 15 and a bf16 zero-point z = min, x^ = s u + z
 * (weights stay symmetric).  The additional z term of the product, sum_g z[m,g] s_w[g,n] sum_{j in g}
 * q_w[j,n], is precomputed on the weight side by prepare and evaluated on the bf16 tensor-core
 * branch together with the rank-r product.  dirotq_workspace_bytes, dirotq_linear, dirotq_linear_host,
 * dirotq_linear_noalloc, dirotq_rotate_quantize, dirotq_w4a4_gemm, dirotq_layer_export,
 * dirotq_int_gemm_debug (codes 0..15), dirotq_layer_info and dirotq_layer_destroy accept such a layer;
 * dirotq_workspace_export does not (use dirotq_workspace_export_asym).  Arguments as for
 * dirotq_layer_bytes / dirotq_prepare_layer. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_asym(int K, int N, int r, int group, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_asym(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                     const void* bias, int K, int N, int r, int group, void* blob,
                                                     size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                     dirotq_stream_t stream, dirotq_layer_t** layer_out);
/* Parity exports: xh bf16 [M,r]; codes u8 [M,K-r] (0..15); scales, zeros bf16 [M,n_g]; zero_term fp32 [n_g,N]
 * = s_w[g,n] * sum_{j in g} q_w[j,n] (exact).  Any pointer of the first call may be NULL. */
DIROTQ_API dirotq_status_t dirotq_workspace_export_asym(const dirotq_layer_t* layer, int M, const void* workspace,
                                                        void* xh_bf16, uint8_t* codes, void* scales_bf16, void* zeros_bf16,
                                                        dirotq_stream_t stream);
DIROTQ_API dirotq_status_t dirotq_layer_export_zero_term(const dirotq_layer_t* layer, float* zero_term,
                                                         dirotq_stream_t stream);

/* ---- W4A8 (paper Sec. 5.1 and the "INT W4A8" rows of Table 1: for 8-bit settings the activations get
 * one dynamic scale per token and the weights one static scale per output channel) ---- */

/* Same layer with 8-bit activations and per-channel 4-bit weights, both symmetric (Eq. 1, z = 0): every
 * token's K - r low-precision coefficients share one bf16 scale s_x[m] = max|x~| / 127 and are rounded to
 * int8 codes in [-127, 127]; every output column of the folded weight has one bf16 scale
 * s_w[n] = max|W~_l[:,n]| / 7 and int4 codes.  y = s_x s_w (q_x . q_w) + x~_h W~_h + bias, the integer
 * product accumulated exactly in int32 over the whole of K (tcgen05.mma kind::i8).  A token's scale needs
 * its whole rotated row, so the first stage is two kernels here (rotation writing fp32 coefficients and row
 * maxima into the workspace, then the quantizer); the workspace is correspondingly larger
 * (dirotq_workspace_bytes).  dirotq_linear, dirotq_linear_host, dirotq_linear_noalloc,
 * dirotq_rotate_quantize, dirotq_w4a4_gemm (the second kernel, whatever the format), dirotq_layer_export
 * (wscales then [1,N]), dirotq_int_gemm_debug (partials then [M,N], codes int8 [M,K_lp] read in place,
 * K_lp = K - r rounded up to 128) and dirotq_layer_destroy accept such a layer. */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_w4a8(int K, int N, int r, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_w4a8(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                     const void* bias, int K, int N, int r, void* blob, size_t blob_bytes,
                                                     void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                                     dirotq_layer_t** layer_out);
/* Parity export: xh bf16 [M,r]; codes int8 [M,K-r]; scales bf16 [M].  Any pointer may be NULL. */
DIROTQ_API dirotq_status_t dirotq_workspace_export_w4a8(const dirotq_layer_t* layer, int M, const void* workspace,
                                                        void* xh_bf16, int8_t* codes, void* scales_bf16,
                                                        dirotq_stream_t stream);

/* ---- NVFP4 variant (paper Sec. 5.1: the 4-bit float setting is NVFP4, blocks of 16 with an FP8 scale) ---- */

/* Same layer with the 4-bit float format instead of INT4: elements are E2M1 (1 sign, 2 exponent,
 * 1 mantissa bit: q_max = 6, Sec. 3), every block of 16 consecutive low-precision coefficients
 * shares an FP8 E4M3 scale, and each tensor has one power-of-two scale 2^e (the second level of
 * the NVFP4 format; the paper does not say how it is chosen):
 *     Q(X) = e2m1_rne(X / s) * s,   s = e4m3_rne(max|X| / 6 / 2^e) * 2^e.
 * The weights' exponent is derived inside prepare from the folded weight (largest block scale
 * <= 256); the activations' exponent `act_scale_log2` is a calibration constant supplied by the
 * caller (ceil(log2(max|x~_l| / 1536)) over the calibration batch).  Blocks are counted from the
 * first low-precision coefficient.  The block scales are applied inside the tensor core
 * (tcgen05.mma kind::mxf4nvf4), so the second kernel has no per-group pass.
 * dirotq_workspace_bytes, dirotq_linear, dirotq_linear_host, dirotq_linear_noalloc,
 * dirotq_rotate_quantize, dirotq_w4a4_gemm, dirotq_workspace_status and dirotq_layer_destroy accept
 * such a layer; the INT4 exports and dirotq_int_gemm_debug do not.  Shapes as for INT4 (group ignored). */
DIROTQ_API dirotq_status_t dirotq_layer_bytes_nvfp4(int K, int N, int r, size_t* bytes);
DIROTQ_API dirotq_status_t dirotq_prepare_layer_nvfp4(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                                      const void* bias, int K, int N, int r, int act_scale_log2, void* blob,
                                                      size_t blob_bytes, void* scratch, size_t scratch_bytes,
                                                      dirotq_stream_t stream, dirotq_layer_t** layer_out);

/* Parity exports of the NVFP4 variant.  codes: one E2M1 code per byte (bit 3 = sign, bits 2..0 index
 * into {0, .5, 1, 1.5, 2, 3, 4, 6}); scales: E4M3 bytes.  Activations: xh bf16 [M,r], codes [M,K-r],
 * scales [M,ceil((K-r)/16)].  Weights: wcodes [K-r,N], wscales [ceil((K-r)/16),N], wh bf16 [r,N]
 * (true values, the internal power-of-two pre-scale undone), q_bf16 [K,K], *weight_scale_log2
 * (DEVICE int) = exponent of the weights' per-tensor scale.  Any pointer may be NULL. */
DIROTQ_API dirotq_status_t dirotq_workspace_export_nvfp4(const dirotq_layer_t* layer, int M, const void* workspace,
                                                         void* xh_bf16, uint8_t* codes, uint8_t* scales_e4m3,
                                                         dirotq_stream_t stream);
DIROTQ_API dirotq_status_t dirotq_layer_export_nvfp4(const dirotq_layer_t* layer, uint8_t* wcodes, uint8_t* wscales_e4m3,
                                                     void* wh_bf16, void* q_bf16, int* weight_scale_log2,
                                                     dirotq_stream_t stream);

/* ---- for callers that cannot allocate (no counterpart in the paper) ------------------------- */

/* dirotq_linear without a workspace argument.  Meant for callers that are not allowed to call
 * cudaMalloc where they run -- a plug-in inside a runtime that owns all device memory, code on a
 * stream being captured, a fixed-memory real-time loop.  The workspace is a 16 MiB array built
 * into the library's device image (resident on every GPU that loads the library, until exit);
 * the call allocates nothing and calls no allocating routine.
 *   - A call whose workspace (dirotq_workspace_bytes) exceeds 16 MiB returns
 *     DIROTQ_ERR_BUFFER_TOO_SMALL and prints the two sizes on stderr; roughly M*K <= 16 Mi.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array: calls that may overlap on the GPU (different streams) race.
 *     Calls on one stream are safe.  The status word is cleared at the start of every call.
 *   - device_status: optional DEVICE int32 that receives the status word of this call (0 = every
 *     wait completed), copied on `stream`; NULL to skip.
 * Same arguments, layouts and results as dirotq_linear otherwise. */
DIROTQ_API dirotq_status_t dirotq_linear_noalloc(const void* x, int M, const dirotq_layer_t* layer, void* y,
                                                 int* device_status, dirotq_stream_t stream);

/* ---- measurement aid (no counterpart in the paper) ------------------------------------------ */

/* Issue-rate probe of the tensor pipe: every SM issues 4*iters back-to-back 128x256 tcgen05.mma
 * instructions on operands resident in shared memory (kind 0: int8 -> int32, K = 32 per
 * instruction; kind 1: bf16 -> fp32, K = 16; kind 2: E4M3 -> fp32, K = 32, the instruction the
 * W4A4 kernel computes its exact integer group sums with), twice (warm-up + timed).  SYNCHRONISES.
 * status_word: device int32, zero-filled (receives a code if the bounded completion wait
 * expires).  *tera_ops_per_s receives 2*M*N*K*instructions / time. */
DIROTQ_API dirotq_status_t dirotq_mma_rate_probe(int kind, int iters, void* status_word, float* tera_ops_per_s,
                                                 dirotq_stream_t stream);

/* ---- calibration of the NVFP4 activations' power-of-two scale (paper Sec. 5.1 / App. E: FP8 block scales need a
 * second-level scale; here 2^e with e = ceil(log2(max|X| / (6 * 256))), an argument of the NVFP4 layers' preparation) ----
 *
 * Both calls find the largest low-precision coefficient of a batch of calibration tokens on the device, SYNCHRONISE
 * `stream` and return e in *act_scale_log2 (HOST).  device_word: 4 bytes of DEVICE scratch; scratch: DEVICE, at least
 * 16 + 4 r K bytes, 16-byte aligned (DIROTQ_ERR_BUFFER_TOO_SMALL otherwise).
 * dirotq_act_scale_log2_from_rotated: from fp32 rotated activations [M,K] in the column order of Q (what
 * dirotq_rotate_quantize exports; the first r columns are the 16-bit ones and are skipped).
 * dirotq_act_scale_log2_ph: projection form, from the tokens x (bf16 [M,K]) and U_h ([K,r] row-major, f64 or f32)
 * alone: x~_h = bf16(x U_hb), V = bf16(U_hb^T H+-) with Hadamard blocks of 64, largest |(x H+- - x~_h V) / 8| (fp32
 * arithmetic).  K + r <= 51200. */
DIROTQ_API dirotq_status_t dirotq_act_scale_log2_from_rotated(const float* xrot_f32, int M, int K, int r, void* device_word,
                                                              int* act_scale_log2, dirotq_stream_t stream);
DIROTQ_API dirotq_status_t dirotq_act_scale_log2_ph(const void* x, int M, const void* Uh, int uh_dtype, int K, int r,
                                                    void* scratch, size_t scratch_bytes, int* act_scale_log2,
                                                    dirotq_stream_t stream);

/* ---- failure-path check (no counterpart in the paper) ---------------------------------------- */

/* Every wait on a barrier inside the library's kernels is bounded: when its time runs out the
 * waiting role records a code in the workspace's status word and the kernel returns, so that a
 * logic error shows up as DIROTQ_ERR_DEVICE_TIMEOUT from dirotq_workspace_status and not as a hung
 * GPU.  This entry point runs that give-up path on purpose and harmlessly: one warp of one small
 * kernel waits, with the same wait routine, on a barrier in its own shared memory that nothing
 * arrives on, gives up after limit_us microseconds (1..100000), writes code 5 to the status word
 * at the start of `workspace` (a device buffer of at least 256 bytes whose first word is zero) and
 * exits normally.  It touches no other memory, no TMA and no tensor memory.  Enqueues on `stream`,
 * does not synchronise.  Zero the status word (256 bytes) before reusing the workspace. */
DIROTQ_API dirotq_status_t dirotq_wait_selftest(void* workspace, unsigned int limit_us, dirotq_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* DIROTQ_H_ */
