/*
 * dgq.h - C ABI of the B200 (sm_100a) hot path of DGQ, distribution-aware group
 * quantization for text-to-image diffusion models.
 *
 * Equations of the paper are unnumbered; they are numbered here in order of
 * appearance: Eq. 1 linear quantizer, Eq. 2 log quantizer (Sec. 3.1); Eq. 3
 * softmax attention score (Sec. 3.2); Eq. 4 range-variability metric D_d,
 * Eq. 5 d* = argmax D_d, Eq. 6 per-group scale and zero-point, Eq. 7
 * per-timestep parameter sets, Eq. 8 log-quantized cross-attention codes,
 * Eq. 9 split product A_hat V_hat (Sec. 3.3).
 *
 * Conventions
 *  - "dev" pointers are CUDA device memory owned by the caller; "host" pointers
 *    are ordinary host memory owned by the caller.  The library never frees or
 *    keeps a caller's pointer beyond the call.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *  - Every function returns a dgq_status.  Nothing throws, aborts or prints.
 *    There is no CPU fallback: unsupported shapes or alignments are errors.
 *  - dgq_quantize_act, dgq_linear and dgq_cross_attn_logq only enqueue work on
 *    `stream`; they allocate nothing and do not synchronise.  The calibration
 *    and weight-preparation calls allocate library-owned objects and
 *    synchronise with the host.
 *  - The kernels these three calls enqueue are launched so that the next kernel
 *    on the stream may be scheduled while the current one finishes; each waits
 *    for everything enqueued before it on the stream before it reads or writes
 *    memory, so stream order is kept as with ordinary launches, also inside a
 *    captured CUDA graph.  Setting DGQ_PDL=0 in the environment before the
 *    first call falls back to ordinary launches.
 *  - Device-side waits are bounded.  A kernel that gives up on a wait records
 *    DGQ_ERR_TIMEOUT in a device status word read by dgq_device_status().
 */
#ifndef DGQ_H_
#define DGQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int dgq_status;
enum {
  DGQ_OK = 0,
  DGQ_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, unknown enum, timestep out of range */
  DGQ_ERR_ALIGNMENT = 2,     /* pointer not 16-byte aligned or leading dimension not a multiple of 8 elements */
  DGQ_ERR_UNSUPPORTED = 3,   /* valid request outside what the kernels implement (stated per call) */
  DGQ_ERR_WORKSPACE = 4,     /* workspace missing or too small */
  DGQ_ERR_CUDA = 5,          /* a CUDA runtime / driver call failed */
  DGQ_ERR_TIMEOUT = 6,       /* a bounded device-side wait gave up (see dgq_device_status) */
  DGQ_ERR_NOT_CALIBRATED = 7 /* the table row of the requested timestep was never filled */
};

/* dim_select / dgq_groups_info dim */
enum { DGQ_DIM_AUTO = 0, DGQ_DIM_CHANNEL = 1, DGQ_DIM_PIXEL = 2, DGQ_DIM_BOTH = 3 };
/* outlier_mode */
enum { DGQ_OUTLIER_KMEANS = 0, DGQ_OUTLIER_EXPLICIT = 1 };
/* quantizer parameter source */
enum { DGQ_MODE_STATIC = 0, DGQ_MODE_DYNAMIC_TOKEN = 1 };
/* code layout written by dgq_quantize_act and read by dgq_linear */
enum { DGQ_CODES_U8 = 0, DGQ_CODES_S8_CENTRED = 1 };
/* scope of the maximum in Eq. 8 */
enum { DGQ_SCALE_PER_PROMPT = 0, DGQ_SCALE_PER_PROMPT_HEAD = 1, DGQ_SCALE_PER_CALL = 2 };

#define DGQ_MAX_GROUPS 32    /* groups along either dimension */
#define DGQ_K_ATOM 32        /* every channel group is padded to a multiple of this many codes */

/* Library-owned, opaque.  Created by the call that returns them, freed by *_destroy. */
typedef struct dgq_groups dgq_groups; /* grouping of one layer + per-timestep (s, 1/s, Z) tables */
typedef struct dgq_weight dgq_weight; /* low-bit weight of one layer in the kernel's layout */

typedef struct {
  int act_bits;        /* b of Eq. 1 / Eq. 6: 2..8 */
  int n_groups;        /* K of the K-means grouping, 1..DGQ_MAX_GROUPS-1 */
  int dim_select;      /* DGQ_DIM_AUTO (Eq. 5) or a forced dimension; DGQ_DIM_BOTH groups both */
  int outlier_mode;    /* DGQ_OUTLIER_KMEANS (the paper) or DGQ_OUTLIER_EXPLICIT (one extra group) */
  float outlier_tau;   /* EXPLICIT: a vector is an outlier if its range width > tau * median width */
  int n_timesteps;     /* T of Eq. 7: number of table rows */
  int rows_per_sample; /* P: pixels (tokens) per sample; row i is pixel position i mod P */
} dgq_calib_config;

typedef struct { int n, h, w, c; } dgq_conv_desc; /* NHWC input of a 3x3, stride 1, zero-pad 1 conv */

/* ---------------------------------------------------------------- calibration (Sec. 3.3, Eq. 4-7)
 * X_cal: dev fp16 [n_rows, C] row-major with leading dimension `ld` elements;
 * n_rows a multiple of rows_per_sample.
 * *inout == NULL: computes per-channel and per-pixel extrema (Eq. 4), picks d*
 *   (Eq. 5) unless forced, groups the vectors along it by K-means on their
 *   (min, max) range, fixes the grouping and the padded code layout for the
 *   layer, fills table row `timestep` from the cells' ranges (Eq. 6) and returns
 *   a new object in *inout.
 * *inout != NULL: keeps the grouping and (re)fills table row `timestep` (Eq. 7).
 * Synchronous with the host (the grouping runs on the host).
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED (C > 8192), CUDA. */
dgq_status dgq_calibrate_groups(const dgq_calib_config* cfg, const void* X_cal, int64_t n_rows, int C,
                                int64_t ld, int timestep, dgq_groups** inout, void* stream);

/* Builds the same object from host arrays (for tables calibrated elsewhere).
 * col_group[C] in [0,G), row_group[P] in [0,R); scale[T*R*G] (fp32, > 0) and
 * zp[T*R*G]; every row counts as filled.  1/s is recomputed in fp32. */
dgq_status dgq_groups_from_host(int C, int P, int act_bits, int G, int R, int T, const int32_t* col_group,
                                const int32_t* row_group, const float* scale, const int32_t* zp,
                                dgq_groups** out);
dgq_status dgq_groups_destroy(dgq_groups* g);
/* Any out pointer may be NULL.  K_pad = length of one padded code row. */
dgq_status dgq_groups_info(const dgq_groups* g, int* C, int* P, int* K_pad, int* G, int* R, int* T,
                           int* dim, int* act_bits, double* D_channel, double* D_pixel);
/* Copies to host arrays (any may be NULL): perm[K_pad] = channel stored at each
 * padded position, -1 for padding; col_group[C]; group_off[G+1] = first padded
 * position of each group; row_group[P]; scale, zp [T*R*G]. */
dgq_status dgq_groups_export(const dgq_groups* g, int32_t* perm, int32_t* col_group, int32_t* group_off,
                             int32_t* row_group, float* scale, int32_t* zp);

/* ---------------------------------------------------------------- activation quantizer (Eq. 1 with Eq. 6)
 * X: dev fp16 [M, C], leading dimension `ld` (for a conv input: NHWC flattened
 * to [n*h*w, C]).  Xq: dev bytes [M, K_pad], channels permuted group-contiguous,
 * each group padded to a multiple of DGQ_K_ATOM.
 *   q = clamp(rint(x * inv_s) + Z, 0, 2^b - 1) in fp32, with (inv_s, Z) of the
 *   cell (pixel group of row i mod P, channel group of the column).
 * DGQ_MODE_STATIC: parameters from table row `timestep`.
 * DGQ_MODE_DYNAMIC_TOKEN: Eq. 6 applied to each token's members of each channel
 *   group; the parameters are written to dyn_scale, dyn_zp (dev [M, G]) for
 *   dgq_linear.  Inputs must be finite.
 * DGQ_CODES_U8 stores q (padding = Z); DGQ_CODES_S8_CENTRED stores q - Z as a
 *   signed byte (padding = 0) and needs L - 127 <= Z <= 128 for every cell,
 *   else UNSUPPORTED (static mode only).
 * Errors: INVALID_ARG, ALIGNMENT, NOT_CALIBRATED, UNSUPPORTED, CUDA. */
dgq_status dgq_quantize_act(const dgq_groups* g, int timestep, int mode, int layout, const void* X, int64_t M,
                            int64_t ld, void* Xq, float* dyn_scale, int32_t* dyn_zp, void* stream);

/* ---------------------------------------------------------------- weights (offline)
 * Per-out-channel symmetric round-to-nearest codes (stands in for the paper's
 * BRECQ / AdaRound weights, Sec. 4.1), permuted and padded to the layer's code
 * layout, int4 packed two per byte, with the per-group column sums the
 * de-quantizer needs.  W: dev fp16 [N, K] (K = C), or [N, 3, 3, C] when conv is
 * non-NULL.  w_bits 8 or 4.  Synchronous with the host. */
dgq_status dgq_weight_prepare(const dgq_groups* g, const void* W, int N, int K, int w_bits,
                              const dgq_conv_desc* conv, dgq_weight** out, void* stream);
/* The same from codes quantized elsewhere: wq host int8 [N, K] (or [N,3,3,C]),
 * sw host fp32 [N]. */
dgq_status dgq_weight_from_codes(const dgq_groups* g, const int8_t* wq, const float* sw, int N, int K,
                                 int w_bits, const dgq_conv_desc* conv, dgq_weight** out);
dgq_status dgq_weight_destroy(dgq_weight* w);
/* Host copies of the codes in original channel order (int8 [N, K]) and scales. */
dgq_status dgq_weight_export(const dgq_weight* w, int8_t* wq, float* sw);

/* ---------------------------------------------------------------- group-quantized layer
 * Y[t, o] = bias[o] + sw[o] * sum_g s[t, g] * ( acc_g[t, o] - Z[t, g] * wsum_g[o] ),
 * acc_g the int32 product of the codes of channel group g with the weight codes
 * (Eq. 1's de-quantizer applied per group; the tensor-core accumulator is
 * switched at every group boundary).  Xq as written by dgq_quantize_act in
 * `layout`.  STATIC: (s, Z) of table row `timestep`, cell of (row mod P, g).
 * DYNAMIC_TOKEN: dyn_scale, dyn_zp dev [M, G].  bias dev fp16 [N] or NULL.
 * Y dev fp16 [M, N] with leading dimension ldy.  conv != NULL: 3x3 stride-1
 * zero-padded convolution of the NHWC code tensor as an implicit GEMM; needs
 * the S8_CENTRED layout, STATIC mode and channel-only grouping (R = 1).
 * workspace: dev, 256-byte aligned, at least dgq_linear_workspace_bytes(); only
 * 4-bit weights need one (a kernel in front of the GEMM expands them to bytes
 * there, once per call instead of once per row tile; the bytes stay in L2).
 * Contents undefined on entry and exit; calls that may overlap on the GPU need
 * separate workspaces unless they use the same weight.  NULL / 0 for 8-bit
 * weights.  NULL with 4-bit weights is allowed: the GEMM then expands the
 * weights itself, stage by stage and once per row tile (slower); a non-NULL
 * workspace that is too small is an error.
 * Errors: INVALID_ARG, ALIGNMENT, NOT_CALIBRATED, WORKSPACE, UNSUPPORTED (K_pad *
 * 255 * 127 would overflow int32; more column blocks of 64-128 outputs than the
 * GPU has SMs; conv shape outside the supported tiling), CUDA. */
dgq_status dgq_linear(const dgq_groups* g, const dgq_weight* w, int timestep, int mode, int layout,
                      const void* Xq, const float* dyn_scale, const int32_t* dyn_zp, const void* bias,
                      void* Y, int64_t M, int64_t ldy, const dgq_conv_desc* conv, void* workspace,
                      size_t workspace_bytes, void* stream);
/* Bytes of workspace dgq_linear needs for this weight and M rows (0 for 8-bit weights). */
dgq_status dgq_linear_workspace_bytes(const dgq_groups* g, const dgq_weight* w, int64_t M, size_t* bytes);

/* ---------------------------------------------------------------- cross-attention (Eq. 3, 8, 9)
 * Q dev fp16 [B, nq, H, d]; K, V dev fp16 [B, nk, H, d]; O dev fp16 [B, nq, H, d].
 * A = softmax(Q K^T / sqrt(d)) in fp32; s = max of A over the columns j >= 1
 * within `scale_gran`; codes = clamp(rint(-log2(A / s)), 0, 2^bits - 1) for
 * j >= 1; O = A[:, 0] V[0] + s * sum_{j>=1} 2^-code V[j].  Column 0 (<start>)
 * stays in fp32.  fixed_scale (dev, [B], [B*H] or [1] by granularity) replaces
 * the dynamic maximum when non-NULL.  scale_out (same shape) and codes_out
 * (dev u8 [B, H, nq, nk-1]) are optional outputs.
 * workspace: dev, at least dgq_cross_attn_workspace_bytes(); contents undefined
 * on entry.  d a multiple of 8, d <= 160, 2 <= nk <= 128.
 * One kernel: with a dynamic scale its thread blocks exchange their maxima
 * through the workspace and meet at a grid barrier, so it is launched
 * cooperatively (and, inside a stream capture, becomes a cooperative kernel
 * node); grids larger than one resident wave run as two ordinary kernels.
 * Errors: INVALID_ARG (nk < 2), ALIGNMENT, UNSUPPORTED, WORKSPACE, CUDA. */
dgq_status dgq_cross_attn_logq(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                               int d, int score_bits, int scale_gran, const float* fixed_scale, void* O,
                               float* scale_out, uint8_t* codes_out, void* workspace,
                               size_t workspace_bytes, void* stream);

/* The same attention with a quantized value operand V_hat (Eq. 9 writes the product as A_hat V_hat
 * without naming V's quantizer).  Reading taken here: Eq. 1 with the range of Eq. 6 over one
 * head's [nk, d] slab of one prompt at `v_bits` (2..8) bits, code decided in fp32,
 * V_hat = s (q - Z); rows j >= 1 enter the product as fp16, row 0 (<start>) in fp32.  Everything
 * else, workspace included, as for dgq_cross_attn_logq.  Errors: as there, INVALID_ARG also for
 * v_bits outside 2..8. */
dgq_status dgq_cross_attn_logq_qv(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                                  int d, int score_bits, int scale_gran, const float* fixed_scale, int v_bits,
                                  void* O, float* scale_out, uint8_t* codes_out, void* workspace,
                                  size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- self-attention (Eq. 2, Eq. 3; Sec. 3.3
 * applies the log quantizer "to both self and cross-attentions")
 * Q dev fp16 [B, nq, H, d]; K, V dev fp16 [B, nk, H, d]; O dev fp16 [B, nq, H, d]; any nk >= 1.
 * A = softmax(Q K^T / sqrt(d)) in fp32; codes = clamp(rint(-log2(A / s)), 0, 2^bits - 1) over ALL keys
 * (there is no <start> column here); O = s * sum_j 2^-code_j V[j].  s is the largest score of each query
 * row, or fixed_scale[b] (dev [B]) when non-NULL; the paper states the dynamic scale for cross-attention
 * only, the row maximum is this library's reading.  codes_out (dev u8 [B, H, nq, nk]) is optional.
 * No workspace: the keys are walked twice by the same thread block.  d in {40, 64, 80, 128, 160}.
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, CUDA. */
dgq_status dgq_self_attn_logq(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk, int d,
                              int score_bits, const float* fixed_scale, void* O, uint8_t* codes_out, void* stream);
dgq_status dgq_cross_attn_workspace_bytes(int B, int H, int nq, int nk, int d, size_t* bytes);

/* ---------------------------------------------------------------- cross-attention without a caller workspace
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 * Same computation, arguments and results as dgq_cross_attn_logq, for callers that
 * have no way to obtain device memory for the workspace: code running inside a
 * region where allocation is forbidden (a plugin or runtime callback that is only
 * handed its input and output buffers, a real-time loop that must not call the
 * allocator, a host that has already committed all device memory).  The scratch
 * space lives in a fixed array inside the library image instead:
 *   - DGQ_NOALLOC_SCRATCH_BYTES of device memory are held by every GPU that loads
 *     the library, from load until the process exits, whether or not this call is
 *     ever used;
 *   - the problem must satisfy B * H * nq <= DGQ_NOALLOC_MAX_ROWS and
 *     B * H <= DGQ_NOALLOC_MAX_HEADS, else DGQ_ERR_WORKSPACE is returned and
 *     nothing is launched;
 *   - the first call on each device looks up the device address of the array
 *     (with that device current) and remembers it; make that first call before
 *     starting any stream capture.  Later calls only enqueue work on `stream`;
 *   - the call itself performs no allocation and frees nothing;
 *   - all calls on a device share the one array.  It still holds the previous
 *     call's statistics on entry; nothing in it has to start clean, because the
 *     first kernel writes every entry that the second one reads.  Two calls whose
 *     kernels can overlap on the GPU (different streams without an ordering
 *     between them) race on it:
 *     serialise them, or use dgq_cross_attn_logq with separate workspaces.
 * Errors: those of dgq_cross_attn_logq, checked first and in the same order; then
 * DGQ_ERR_WORKSPACE for a problem beyond the limits above; DGQ_ERR_UNSUPPORTED when
 * the current device's ordinal is 64 or more (the library remembers one address per
 * device ordinal below that). */
#define DGQ_NOALLOC_MAX_ROWS (1 << 18)
#define DGQ_NOALLOC_MAX_HEADS 256
#define DGQ_NOALLOC_SCRATCH_BYTES (4 * (DGQ_NOALLOC_MAX_ROWS / 128 + DGQ_NOALLOC_MAX_HEADS) + 8 * DGQ_NOALLOC_MAX_ROWS)
dgq_status dgq_cross_attn_logq_noalloc(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                                       int d, int score_bits, int scale_gran, const float* fixed_scale, void* O,
                                       float* scale_out, uint8_t* codes_out, void* stream);

/* ---------------------------------------------------------------- status
 * Synchronises the current device and returns the device status word of the
 * current device in *status (DGQ_OK, or the first error a kernel recorded),
 * then clears it. */
dgq_status dgq_device_status(int* status);
/* Diagnostic: enqueues a one-warp kernel whose only wait, on a barrier nobody arrives at, gives up
 * after max_polls (1..65536) polls of at most a microsecond each, so that the time-out path of the
 * bounded waits (status word, dgq_device_status, a usable device afterwards) can be exercised
 * without making a wait of a working kernel run out.  Errors: INVALID_ARG, CUDA. */
dgq_status dgq_selftest_wait_timeout(uint32_t max_polls, void* stream);
const char* dgq_status_string(dgq_status s);
/* Number of kernels the library has launched in this process (all devices). */
uint64_t dgq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DGQ_H_ */
