/*
 * sparq.h -- C ABI of the B200 (sm_100a) SPARQ library.
 *
 * SPARQ (arXiv 2105.11010, "Post-Training Sparsity-Aware Quantization") trims
 * already-quantized unsigned 8-bit activations to an n-bit window that starts at the
 * leading one (bSPARQ, Section 3.1) and lets a lone non-zero activation of an adjacent
 * pair keep the 2n-bit budget of the pair (vSPARQ, Section 3.2, Eq. 2).  The trimmed
 * value is still an 8-bit integer (window << shift), so the dot product of Eq. 1 is an
 * ordinary u8 x s8 -> s32 contraction over the transformed activations.
 *
 * Conventions common to all entry points
 *   - Unless a parameter says HOST, every data pointer is a DEVICE pointer that the
 *     caller owns; the library neither frees nor keeps it after the enqueued work ends.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  A call
 *     validates its arguments on the host, enqueues its kernels on `stream` and returns
 *     without synchronizing.
 *   - Return value: SPARQ_OK (0) or a negative sparq_status.  On error nothing has been
 *     enqueued and sparq_last_error() describes the reason (the entry points that enqueue
 *     more than one kernel -- the host-buffer forms, sparq_gemm_s8_static,
 *     sparq_gemm_s8_sparse24 -- may have enqueued their earlier kernels when a later launch
 *     fails; their outputs are then undefined).  No entry point throws, aborts or traps the
 *     device.
 *   - Consecutive fused launches on one stream overlap at their edges (programmatic
 *     dependent launch): a launch may set itself up, and fetch its WEIGHTS, while its
 *     predecessor is finishing -- never its activations, scale, bias or residual.  The
 *     library keeps, per device and stream, the output ranges of the last fused launch and
 *     fetches weights early only when they are clear of them, so a layer whose weights the
 *     previous layer has just written still sees the finished values; kernels of other
 *     libraries never release their successor early.  Nothing for the caller to do.
 *   - The library is thread-compatible: concurrent calls are allowed, the error string
 *     is per host thread.
 */
#ifndef SPARQ_H_
#define SPARQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SPARQ_API __attribute__((visibility("default")))
#else
#define SPARQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPARQ_OK = 0,
    SPARQ_ERR_INVALID_ARG = -1, /* null pointer, negative size, bad mode / width / placement set */
    SPARQ_ERR_UNSUPPORTED = -2, /* a shape or alignment the library has no kernel for */
    SPARQ_ERR_CUDA = -3,        /* a CUDA runtime / driver call failed (text in sparq_last_error) */
    SPARQ_ERR_TIMEOUT = -4      /* a bounded device-side wait expired (reported by sparq_check) */
} sparq_status;

enum { SPARQ_MODE_NONE = 0, SPARQ_MODE_BSPARQ = 1, SPARQ_MODE_VSPARQ = 2 };
enum { SPARQ_ROUND_TRUNCATE = 0, SPARQ_ROUND_NEAREST = 1 };

/* Named placement sets: bit s set <=> the window may occupy bits [s+n-1 : s], i.e. be
 * shifted left by s.  Section 3.1 (5opt/3opt/2opt, n = 4); Section 5.1 (6opt n = 3,
 * 7opt n = 2). */
#define SPARQ_SET_5OPT 0x1Fu
#define SPARQ_SET_3OPT 0x15u
#define SPARQ_SET_2OPT 0x11u
#define SPARQ_SET_6OPT 0x3Fu
#define SPARQ_SET_7OPT 0x7Fu

/* The activation transform.
 *   mode            NONE: activations are used as they are (plain A8W8).
 *                   BSPARQ: every activation is trimmed on its own (Section 3.1; the
 *                   "-vS" columns of Tables 2, 4 and 5).
 *                   VSPARQ: activations are taken in pairs (2j, 2j+1) along the reduction
 *                   axis; if one is zero the other keeps a 2n-bit window (all 8 bits when
 *                   n = 4), otherwise both are trimmed by bSPARQ (Eq. 2).
 *   window_bits     n = 2, 3 or 4.
 *   placement_mask  allowed shifts; must contain 0 and 8-n, have no bit above 8-n and no
 *                   gap between consecutive shifts wider than n.
 *   rounding        TRUNCATE drops the bits below the window ("Trim"); NEAREST adds half a
 *                   window LSB first ("+R"; ties go up; the top of the 8-bit range
 *                   saturates to the all-ones window at the highest placement).
 * With mode NONE the other three fields are ignored. */
typedef struct {
    int32_t mode;
    int32_t window_bits;
    uint32_t placement_mask;
    int32_t rounding;
} sparq_params;

/* What happens to the int32 accumulators (not in the paper beyond its quantization
 * scheme, Section 5: per-layer activation scale times per-kernel weight scale).  For
 * output column j, in fp32 and in this order, one IEEE operation each:
 *     t = (float)acc;  y = fma(t, scale[j], bias ? bias[j] : 0);
 *     if (residual) y = fma((float)residual[m][j], residual_scale, y);
 *     if (relu) y = y > 0 ? y : 0;
 *     f32_out = y;     u8_out = clamp(rint(y * inv_out_scale), 0, 255)   (NaN -> 0)
 * Each output pointer may be NULL (that output is not produced); at least one must be
 * non-NULL.  Outputs are M x N row-major with leading dimension N (= NHWC for the
 * convolution).  scale may be NULL only if f32_out and u8_out are both NULL. */
typedef struct {
    const float *scale;   /* [N] device */
    const float *bias;    /* [N] device, or NULL */
    int32_t relu;         /* 0 / 1 */
    float inv_out_scale;  /* multiplier onto the next layer's u8 grid */
    int32_t *acc_out;     /* raw accumulators, or NULL */
    float *f32_out;       /* dequantized fp32, or NULL */
    uint8_t *u8_out;      /* requantized activations for the next layer, or NULL */
    /* Producer-side SPARQ.  The transform depends on the activations only (Section 3, first
     * paragraph), so the layer that PRODUCES them can apply it once, and the consumer then
     * runs with mode NONE at plain A8W8 speed.  If next_transform is non-NULL and its mode is
     * not NONE, u8_out holds T(requantized row) with pairs (2j, 2j+1) along the N axis (the
     * channels of an NHWC output, i.e. the next layer's reduction axis); acc_out and f32_out
     * are unaffected.  Needs N to be a multiple of 4 (else SPARQ_ERR_UNSUPPORTED). */
    const sparq_params *next_transform;   /* HOST pointer, or NULL */
    /* Residual input: the u8 identity tensor of a residual block (M x N row-major like the
     * outputs, on its own scale), added before the ReLU so that the last convolution of a
     * bottleneck writes the block's output in one pass.  Not in the paper, whose transform
     * acts on whatever activations a layer receives.  NULL = no residual.  Must be 16-byte
     * aligned (else SPARQ_ERR_UNSUPPORTED), needs scale (a dequantized output), and may be
     * the same buffer as u8_out only if every row is read before it is written, which this
     * library does not promise: pass distinct buffers. */
    const uint8_t *residual;              /* [M x N] device, or NULL */
    float residual_scale;
} sparq_epilogue;

/* Standalone transform (Sections 3.1-3.2): out[r][k] = T(in[r][:])[k] for `rows` rows of
 * `row_len` bytes, rows stored back to back.  Pairs are (2j, 2j+1) inside a row and never
 * cross rows; an odd row_len pairs the last element with an implicit zero.  `out` may be
 * the same buffer as `in` (in place) but must not partially overlap it.  Any alignment is
 * accepted; 16-byte aligned buffers with an even row_len take the fast vector path.
 * rows == 0 or row_len == 0 is a no-op. */
SPARQ_API int sparq_quantize(const uint8_t *in, uint8_t *out, size_t rows, size_t row_len,
                   const sparq_params *p, void *stream);

/* Fused dot products (Eq. 1 with Eq. 2 applied on the fly):
 *     acc[m][j] = sum_k T(A)[m][k] * B[j][k]        u8 x s8 -> s32
 * A is M x K with leading dimension lda (K contiguous); vSPARQ pairs are (2j, 2j+1) along
 * K.  B is N x K with leading dimension ldb (K contiguous: one row per output column,
 * which is the layout of convolution weights [cout][r][s][cin]).  The result goes through
 * the epilogue `e`.
 * Requirements (else SPARQ_ERR_UNSUPPORTED): A and B 16-byte aligned, lda and ldb
 * multiples of 16, K a multiple of 16 and at most 65536; M, N >= 1 (M == 0 or N == 0 is a
 * no-op that returns SPARQ_OK). */
SPARQ_API int sparq_gemm_s8(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                  int64_t M, int64_t N, int64_t K,
                  const sparq_params *p, const sparq_epilogue *e, void *stream);

/* Fused convolution (Section 4: the convolution mapped onto the same dot product, here
 * without materializing im2col).  x is NHWC u8 [n][h][w][c]; wgt is s8 [cout][r][s][c];
 * dilation 1.  The reduction runs over (r, s, c) with c fastest, so vSPARQ pairs are
 * adjacent input channels of one pixel, and taps outside the image contribute zero.
 * Output pixel (img, ho, wo) is row (img*Ho + ho)*Wo + wo of the M x cout outputs, with
 * Ho = (h + 2*pad_h - r)/stride_h + 1 and Wo likewise.
 * Requirements (else SPARQ_ERR_UNSUPPORTED): x and wgt 16-byte aligned, c a multiple of
 * 16 (a count that is not a multiple of 64 is read in 64-channel blocks whose tail is zero
 * fill: correct, at the speed of the next multiple of 64), r, s in 1..7, strides in 1..8,
 * pads < filter size, r*s*c <= 65536. */
SPARQ_API int sparq_conv2d_nhwc_s8(const uint8_t *x, int n, int h, int w, int c,
                         const int8_t *wgt, int cout, int r, int s,
                         int stride_h, int stride_w, int pad_h, int pad_w,
                         const sparq_params *p, const sparq_epilogue *e, void *stream);

/* ---- Host-buffer forms -----------------------------------------------------------------
 * The same operations for callers whose activations live in HOST memory (pinned memory
 * gives asynchronous copies; pageable memory works but is slower).  The library copies
 * the input into a device staging buffer that it owns (grown on demand, kept for later
 * calls, freed by sparq_shutdown), runs the device entry point on `stream`, copies the
 * requested outputs back and SYNCHRONIZES `stream` before returning.  Calls that share a
 * device share the staging buffers, so do not issue two host-buffer calls concurrently on
 * one device.  Parameters (weights, scale, bias) stay DEVICE pointers: they are resident
 * model data, not per-step inputs. */

/* in_host / out_host: HOST pointers, rows * row_len bytes each (may be the same). */
SPARQ_API int sparq_quantize_host(const uint8_t *in_host, uint8_t *out_host, size_t rows, size_t row_len,
                        const sparq_params *p, void *stream);

/* A_host: HOST, M x K with leading dimension lda.  B: DEVICE.  In `e`, scale and bias are
 * DEVICE pointers and acc_out / f32_out / u8_out / residual are HOST pointers (M x N each). */
SPARQ_API int sparq_gemm_s8_host(const uint8_t *A_host, int64_t lda, const int8_t *B, int64_t ldb,
                       int64_t M, int64_t N, int64_t K,
                       const sparq_params *p, const sparq_epilogue *e, void *stream);

/* x_host: HOST NHWC tensor.  wgt: DEVICE.  In `e`, scale and bias are DEVICE pointers and
 * the output pointers are HOST pointers (n*Ho*Wo x cout each). */
SPARQ_API int sparq_conv2d_nhwc_s8_host(const uint8_t *x_host, int n, int h, int w, int c,
                              const int8_t *wgt, int cout, int r, int s,
                              int stride_h, int stride_w, int pad_h, int pad_w,
                              const sparq_params *p, const sparq_epilogue *e, void *stream);

/* ---- For callers that cannot allocate device memory ---------------------------------------
 * (The paper has no counterpart: this is a deployment variant of sparq_gemm_s8.)
 *
 * Some hosts of this library must not call cudaMalloc once they are running: a serving
 * process whose framework has already claimed all free device memory for its own pool
 * (a later cudaMalloc fails or fragments the pool), or a control loop that cannot take
 * the device-wide synchronization an allocation implies.  The other entry points
 * allocate lazily (the status word, staging buffers); this one allocates nothing, on the
 * host's behalf or through any library: no cudaMalloc, no cudaFree, no torch allocator.
 *
 * It computes exactly what sparq_gemm_s8 computes, as two kernels: the standalone
 * transform writes T(A) into scratch, then the plain u8 x s8 GEMM with the same epilogue
 * reads it.  The scratch (and the status word of the bounded waits) lives in a fixed
 * array inside the library image, SPARQ_STATIC_SCRATCH_BYTES long, which every GPU that
 * loads the library holds until the process exits.
 *
 *   - Limit: M * K <= SPARQ_STATIC_SCRATCH_BYTES and lda == K; anything larger returns
 *     SPARQ_ERR_UNSUPPORTED with the limit in sparq_last_error().  Other requirements as
 *     for sparq_gemm_s8.
 *   - The first call on a device looks up the array's device address (set-up, once per
 *     device, with that device current).  Like the first use of any kernel of a library,
 *     it also makes the CUDA runtime load the library's device code, and the driver
 *     reserves the array's SPARQ_STATIC_SCRATCH_BYTES then: memory taken by the driver for
 *     the code image, not an allocation this entry point makes, but it does come out of
 *     the device's free memory at that moment.  So make one call at start-up, before the
 *     host's own pool claims the device, and outside any stream capture; every later call
 *     leaves the free device memory exactly as it found it.
 *   - The call is synchronous: it returns after `stream` has drained, so the outputs are
 *     complete and a device-side timeout is reported by this call (SPARQ_ERR_TIMEOUT),
 *     not by sparq_check.
 *   - All calls share the one array, which keeps the previous call's contents.  Calls that
 *     overlap on the GPU (other host threads, other streams, other processes' contexts do
 *     not count) race on it: issue them one at a time per device. */
#define SPARQ_STATIC_SCRATCH_BYTES (8u << 20)
SPARQ_API int sparq_gemm_s8_static(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                         int64_t M, int64_t N, int64_t K,
                         const sparq_params *p, const sparq_epilogue *e, void *stream);

/* ---- Packed stream ------------------------------------------------------------------------
 * The encoded form that the multiplier of Eq. 4 consumes, as a storage / bandwidth format
 * for activations between layers (the paper names the metadata as the method's footprint
 * cost and leaves grouping it open, Sections 5.1 and 6).  Defined for mode BSPARQ or VSPARQ
 * (else SPARQ_ERR_INVALID_ARG); row_len must be a multiple of 16 and all pointers 16-byte
 * aligned (else SPARQ_ERR_UNSUPPORTED).  The description below is for window_bits = 4; the
 * 3- and 2-bit forms follow it.
 *
 * A pair (2j, 2j+1) of a row becomes
 *   one data byte  (in1 << 4) | in2: the two 4-bit windows of bSPARQ(a), bSPARQ(b) when the
 *                  pair is multiplied as two windows, or the lone non-zero activation whole
 *                  (its two nibbles, Eq. 3) when vSPARQ finds its partner zero;
 *   one state      id(shift1) * ns + id(shift2) for two windows, where ns is the number of
 *                  placements in the set and id(s) the rank of shift s in it (the ShiftCtrl
 *                  fields); ns*ns when the second slot is zero; ns*ns + 1 when the first is
 *                  (the MuxCtrl states; VSPARQ only).  The placement of a window is the
 *                  lowest allowed one that holds the trimmed / rounded value.
 * States take cb = sparq_packed_ctrl_bits(p) bits: 5 / 4 / 3 for 5opt / 3opt / 2opt with
 * VSPARQ, i.e. 6.5 / 6 / 5.5 bits per activation instead of 8.
 *   data plane: rows * row_len / 2 bytes, pairs in order.
 *   ctrl plane: rows * row_len / 16 * cb bytes: per 16 activations the 8 states, pair j at
 *               bits [j*cb, (j+1)*cb) of a little-endian integer of cb bytes.
 * For window_bits n = 3 or 2 (Section 5.1) the fields are n bits wide: per 16 activations the
 * data plane holds 2n bytes, pair j's field (in1 << n) | in2 at bits [j*2n, (j+1)*2n) of a
 * little-endian integer (rows * row_len / 16 * 2n bytes in all; n = 4 is the byte-per-pair
 * form above).  A lone non-zero value owns the pair's 2n-bit window at a shift s_l in
 * 0..8-2n and travels as that window's two n-bit halves; its states are ns*ns + s_l (second
 * slot zero) and ns*ns + (9 - 2n) + s_l (first slot zero).  6opt and 7opt with VSPARQ take
 * cb = 6: 6 and 5 bits per activation.
 * sparq_unpack returns T(x) exactly (what sparq_quantize writes), so a consumer may run
 * with mode NONE on the unpacked tensor.  rows == 0 or row_len == 0 is a no-op. */

/* Control bits per pair (2..6), or a negative sparq_status. */
SPARQ_API int sparq_packed_ctrl_bits(const sparq_params *p);

/* in: rows x row_len activations.  data, ctrl: the two planes (sizes above), caller-owned. */
SPARQ_API int sparq_pack(const uint8_t *in, size_t rows, size_t row_len, const sparq_params *p,
               uint8_t *data, uint8_t *ctrl, void *stream);

/* out: rows x row_len bytes = T(x).  p must be the parameters the stream was packed with
 * (the rounding field is ignored). */
SPARQ_API int sparq_unpack(const uint8_t *data, const uint8_t *ctrl, size_t rows, size_t row_len,
                 const sparq_params *p, uint8_t *out, void *stream);

/* ---- Uniform min-max quantization (Section 5) ----------------------------------------------
 * Section 5: the paper's models are quantized uniformly from min-max statistics, unsigned
 * symmetric per layer for activations and signed symmetric per kernel for weights, with the
 * statistics gathered over a few calibration batches.  These three calls are that front
 * end on the device; the data set and the calibration run are the caller's.
 * x is fp32 (SPARQ_DTYPE_F32) or bf16 (SPARQ_DTYPE_BF16, widened exactly), 16-byte aligned,
 * any length.  fp32 arithmetic, one IEEE operation per step, as written below. */
#define SPARQ_DTYPE_F32 0
#define SPARQ_DTYPE_BF16 1

/* *max_inout = max(*max_inout, max_i |x[i]|), NaNs skipped: a running maximum on the DEVICE
 * (4-byte aligned), so calibration batches fold into it with no host round trip.  The
 * caller sets it to 0 before the first batch.  n == 0 is a no-op. */
SPARQ_API int sparq_absmax(const void *x, int dtype, size_t n, float *max_inout, void *stream);

/* out[i] = clamp(rint(x[i] * inv), 0, 255) with inv = 255 / *max_dev (0 if *max_dev is 0);
 * rint is to nearest even; negatives and NaN give 0.  max_dev is a DEVICE pointer (the
 * statistic sparq_absmax gathered); the layer's activation scale is *max_dev / 255.
 * out: n bytes, 16-byte aligned. */
SPARQ_API int sparq_quantize_act_u8(const void *x, int dtype, size_t n, const float *max_dev, uint8_t *out,
                          void *stream);

/* Weights [cout][k] fp32 (k = r*s*c for a convolution): for kernel j with a_j = max |w[j][:]|,
 * out[j][i] = clamp(rint(w[j][i] * (127 / a_j)), -127, 127) (all zero if a_j is 0; NaN -> 0)
 * and scale_out[j] = a_j / 127.  The GEMM epilogue's scale[j] is then the activation scale
 * times scale_out[j]. */
SPARQ_API int sparq_quantize_weight_s8(const float *w, int64_t cout, int64_t k, int8_t *out, float *scale_out,
                             void *stream);

/* ---- 2:4 sparse weights (Sections 4 and 5.3) ---------------------------------------------
 * Weights pruned 2:4 arrive compressed as a sparse tensor core stores them: per output
 * channel j and per group of four consecutive reduction indices, the two kept values
 * vals[j][2g], vals[j][2g+1] and their coordinates pos[j][2g] < pos[j][2g+1] in 0..3.  The
 * coordinates select two of the group's four activations, and vSPARQ then pairs THOSE two
 * (Section 5.3), so the transform depends on the output channel:
 *     acc[m][j] = sum_g T2(A[m][4g+p0], A[m][4g+p1]) . (v0, v1)
 * The library computes this exactly as a dense contraction over expanded operands: the
 * activations of a group become the six pairs a pattern could select, transformed
 * ((0,1) (0,2) (0,3) (1,2) (1,3) (2,3): 12 bytes per 4), and a weight row holds its two
 * values in its own pattern's two columns.  With mode NONE or BSPARQ the transform is per
 * element and the expansion is the dense form of the weights (K' = K); with VSPARQ
 * K' = 3K.  The expanded tensors are ordinary operands of sparq_gemm_s8 /
 * sparq_conv2d_nhwc_s8 with mode NONE (for a convolution expand along the channel axis:
 * rows = pixels, K = c; weights [cout][r][s][c] -> [cout][r][s][c']). */

/* K' for these parameters, or a negative sparq_status (K must be a multiple of 4). */
SPARQ_API int64_t sparq_sparse24_expanded_k(int64_t K, const sparq_params *p);

/* vals [N][K/2] s8, pos [N][K/2] u8 -> w_exp [N][K'] s8 (4-byte aligned).  A group whose
 * coordinates are not strictly increasing in 0..3 is expanded as zeros and recorded:
 * the next sparq_check returns SPARQ_ERR_INVALID_ARG. */
SPARQ_API int sparq_sparse24_expand_weights(const int8_t *vals, const uint8_t *pos, int64_t N, int64_t K,
                                  const sparq_params *p, int8_t *w_exp, void *stream);

/* A [rows][K] u8 -> a_exp [rows][K'] u8: the transformed candidate pairs (VSPARQ), or T(A)
 * itself (NONE, BSPARQ).  K a multiple of 16, both pointers 16-byte aligned. */
SPARQ_API int sparq_sparse24_expand_activations(const uint8_t *A, size_t rows, size_t K, const sparq_params *p,
                                      uint8_t *a_exp, void *stream);

/* The product above followed by the epilogue `e`.  w_exp: expanded weights for the same
 * parameters.  workspace: M * K' bytes, 16-byte aligned, caller-owned (VSPARQ only; may be
 * NULL otherwise).  Other requirements as for sparq_gemm_s8. */
SPARQ_API int sparq_gemm_s8_sparse24(const uint8_t *A, const int8_t *w_exp, int64_t M, int64_t N, int64_t K,
                           const sparq_params *p, const sparq_epilogue *e, uint8_t *workspace, void *stream);

/* Synchronizes `stream` and reports what the device-side code recorded since the last
 * check: SPARQ_OK, SPARQ_ERR_TIMEOUT if a bounded wait inside a kernel gave up (its
 * outputs are then undefined), SPARQ_ERR_INVALID_ARG if sparq_sparse24_expand_weights met
 * bad coordinates, or SPARQ_ERR_CUDA if the stream is in error. */
SPARQ_API int sparq_check(void *stream);

/* Diagnostic: launches a one-CTA kernel that waits, with a limit of `limit_cycles` SM clock
 * cycles (1e3 .. 1e8), on a barrier that nothing ever completes, using the wait, abort-flag
 * and tensor-memory code of the fused kernels (whose own limit is about a second and whose
 * barriers always complete, so their give-up path cannot be reached on demand).  The kernel
 * always returns normally; afterwards sparq_check(stream) reports SPARQ_ERR_TIMEOUT once and
 * SPARQ_OK from then on, and every other entry point keeps working.  With use_static_word
 * the bit is recorded in sparq_gemm_s8_static's own status word instead, which the next
 * call of that entry point reports and clears.  report: 4 words on the DEVICE -- the first
 * wait gave up (1), a second wait with a 1000x longer limit left through the CTA's abort
 * flag (1), the cycles that second wait spent, the kernel reached its end (1).  The paper has
 * no counterpart. */
SPARQ_API int sparq_selftest_wait_timeout(int64_t limit_cycles, int use_static_word, uint32_t *report, void *stream);

/* Diagnostic: the tensor core's own rate, the ceiling the fused kernels are measured against.
 * One CTA per SM issues iters x 4 tcgen05.mma kind::i8 instructions of 128 x bn x 32
 * (u8 x s8 -> s32; bn = 64, 128 or 256; iters <= 1e6) on operands resident in shared memory,
 * with no global-memory traffic, transform or epilogue, and writes the SM-clock cycles from
 * its first issue to the retirement of its last MMA to cycles_out[cta] (DEVICE, one int64 per
 * SM).  MACs per launch = SMs * iters * 4 * 128 * bn * 32.  Returns the number of CTAs
 * launched (> 0) or a negative sparq_status.  The paper has no counterpart. */
SPARQ_API int sparq_selftest_mma_rate(int bn, int iters, int64_t *cycles_out, void *stream);

/* Text of the calling thread's most recent error ("" if none).  The pointer stays valid
 * until the thread's next failing call. */
SPARQ_API const char *sparq_last_error(void);

/* Releases what the library itself holds on the current device (the status word, the
 * host-buffer forms' staging buffers) and forgets the cached tensor-map encodings.  Safe to call more than once; later calls re-create what they need. */
SPARQ_API int sparq_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* SPARQ_H_ */
