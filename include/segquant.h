/*
 * segquant.h -- C ABI of the B200 (sm_100a) SegLinear + DualScale W8A8 linear layer.
 *
 * The layer computes  Y = X W^T + b  with 8-bit codes:
 *   SegLinear (Sec. 4.2.2): the K axis (input-segmented mode, fed by a concat / stack /
 *   reshape) and the N axis (output-segmented mode, consumed by a chunk / split) are
 *   partitioned into segments and every segment is quantized with its own scale.
 *   DualScale (Sec. 4.3.2): a polarity-asymmetric activation is split into
 *   X_+ = max(X,0) and X_- = min(X,0), each quantized with its own scale s_+ / s_-,
 *   both multiplied with the same quantized weight and recombined as
 *   s_+ s_w (X^_+ W^) + s_- s_w (X^_- W^).
 *
 * Conventions for every entry point
 *   - Matrices are row-major with an explicit leading dimension in ELEMENTS.
 *     X [M,K] activations, W [N,K] weights (nn.Linear order), Y [M,N].
 *   - "dev" pointers are CUDA device pointers of the current device, "host" pointers are
 *     ordinary host memory that is only read during the call.
 *   - The caller owns every buffer.  The library allocates no device memory and keeps no
 *     state between calls other than a cached driver entry point, per-device kernel attributes (both
 *     guarded for concurrent callers) and the test-only overrides of segquant_set_tuning.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronizing, except segquant_last_device_status.
 *   - Every entry point returns an sq_status.  Anything checkable on the host is rejected
 *     before any launch; nothing aborts or throws.  There is no CPU fallback.
 *   - SQ_OK from a launching call means the work was enqueued.  A bounded wait inside a kernel that
 *     expires is reported only through segquant_last_device_status; Y is undefined unless that call
 *     returns SQ_OK as well.
 */
#ifndef SEGQUANT_H_
#define SEGQUANT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SQ_OK = 0,
    SQ_ERR_NULL = 1,        /* a required pointer is NULL */
    SQ_ERR_SHAPE = 2,       /* M/N/K/ld out of range (<= 0, ld < extent, K too large for int32 sums) */
    SQ_ERR_SEGTABLE = 3,    /* segment bounds not ascending / not starting at 0 / not ending at K or N */
    SQ_ERR_ALIGN = 4,       /* pointer, leading dimension or segment bound violates an alignment rule */
    SQ_ERR_UNSUPPORTED = 5, /* unknown code / dtype, or more segments than the kernels support */
    SQ_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed (launch, tensor-map encode, ...) */
    SQ_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (read back by segquant_last_device_status) */
    SQ_ERR_WORKSPACE = 8    /* workspace NULL or smaller than segquant_workspace_bytes() */
} sq_status;

typedef enum { SQ_CODE_INT8 = 0, SQ_CODE_E4M3 = 1 } sq_code;   /* 8-bit code type */
typedef enum { SQ_F32 = 0, SQ_BF16 = 1 } sq_dtype;             /* real-valued element type */
typedef enum { SQ_ACT_NONE = 0, SQ_ACT_SILU = 1, SQ_ACT_GELU = 2, SQ_ACT_GEGLU = 3 } sq_act;   /* activation in front of the quantizer */

/* flags */
#define SQ_FLAG_QMIN_SYM 1u  /* int8 DualScale: clamp the negative path to -127 instead of -128 */

/* limits */
#define SQ_MAX_P 64   /* K-segments per layer */
#define SQ_MAX_Q 64   /* N-segments per layer */

/* Segment table (the output of the paper's graph pattern detection, App. B Alg. 1):
 * K-partition kb[0..P] with kb[0]=0, kb[P]=K and N-partition nb[0..Q] with nb[0]=0, nb[Q]=N,
 * both strictly ascending, in HOST memory (copied during the call). */
typedef struct {
    int32_t P;
    const int32_t *kb;
    int32_t Q;
    const int32_t *nb;
} sq_segtable;

/* Bytes of device scratch every call below accepts as `workspace` (a small constant; it holds
 * device status words and reduction partials).  The buffer must be 256-byte aligned and zero-filled
 * once by the caller after allocating it.  Two calls that may run concurrently need two workspaces. */
size_t segquant_workspace_bytes(void);

/* Optional larger workspace for the GEMM entry points (and the plan): with at least this many bytes -- zero-filled
 * once, like the small one -- a layer with ONE K-segment whose output tiles would leave a good part of the GPU idle
 * (fewer tiles than SM pairs, or a small last wave) is computed with SPLIT tiles: the K loop of every tile is cut so
 * that all SM pairs get the same number of K-blocks, the CTAs that worked on part of a tile leave their raw
 * accumulators in this workspace, and the last of them to finish adds them up (exact int32 sums for int8 codes;
 * fp32 sums in the order of the K ranges for e4m3, within the tolerance of the fp32 epilogue) and runs the usual
 * epilogue (Sec. 4.2.2 / 4.3.2 products unchanged: the accumulators are the same sums).  Nothing waits inside the
 * kernel.  The size depends on the device (its SM count; about 38 MB on a 148-SM GPU) and weakly on M and N
 * (dual != 0 for the DualScale entry point).  Returns 0 if the device cannot be queried.  The counters in it are
 * left at zero by every completed launch; after SQ_ERR_TIMEOUT zero-fill the workspace again.  Layers that do not
 * qualify, and smaller workspaces, run exactly as before. */
size_t segquant_split_workspace_bytes(int64_t M, int64_t N, int dual);

/* Step "calibration" -- Sec. 4.3.2 scale formula (s_- = |min x| / |q_min|, s_+ = max x / q_max),
 * strict min/max (App. B, Dual Scale Sensitivity Analysis), one scalar per segment (App. B,
 * per-tensor 8-bit scheme; Sec. 4.2.2 "independently within each segment").
 *   is_weight = 0: X is a calibration batch [rows,K] (dev, dtype dt, leading dimension ld).
 *       dual != 0: s_pos[p] = max(max x,0)/q_max and s_neg[p] = max(-min x,0)/|q_min| per K-segment p.
 *       dual == 0: s_pos[p] = max|x|/q_max; s_neg is ignored (may be NULL).
 *   is_weight = 1: X is the weight matrix [rows=N,K]; s_pos[p*Q+q] = max|W block(p,q)|/q_max.
 *   q_max = 127 (int8) or 448 (e4m3); |q_min| = 128 (int8; 127 with SQ_FLAG_QMIN_SYM) or 448.
 *   A segment whose extremum is 0 gets scale 1.  Inputs must be finite.  rows < 2^37, K <= 16 776 960.
 *   s_pos / s_neg: dev float arrays written by the call.  Alignment: X 16 bytes, ld*sizeof(dt)
 *   a multiple of 16 bytes. */
sq_status segquant_calib_scales(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                const sq_segtable *seg, sq_code code, int is_weight, int dual,
                                uint32_t flags, float *s_pos, float *s_neg,
                                void *workspace, size_t ws_bytes, void *stream);

/* Calibration for callers that cannot allocate device memory.  (The paper has no counterpart; this is
 * a property of the library, not of the method.)  Some users of this library run where cudaMalloc is
 * off limits: inside a host process whose device memory is entirely owned by another component's pool,
 * in a plugin that is handed its tensors and nothing else, or under a policy that forbids allocation
 * after start-up.  segquant_calib_scales needs a caller-provided workspace for its reduction partials;
 * this variant computes exactly the same scales with the partials kept in a fixed 8 KiB array inside
 * the library's device image, and takes no workspace.  It calls no allocating routine.
 *   Arguments, results and alignment rules are those of segquant_calib_scales, minus the workspace.
 *   Limit: at most SQ_STATIC_CALIB_MAX_BLOCKS scale values per call (P for activations, P*Q for
 *   weights); more is refused with SQ_ERR_UNSUPPORTED before any launch.
 *   The first call on a device looks up the array's device address (once per device, with that device
 *   current); make that first call outside any stream capture.
 *   Every call on one GPU shares the array: each call resets the entries it uses before reducing into
 *   them, so calls in stream order are independent, but two calls that overlap on the GPU (different
 *   streams or threads without ordering between them) race and may both return wrong scales.
 *   Every GPU that loads the library carries the 8 KiB array until the process exits. */
#define SQ_STATIC_CALIB_MAX_BLOCKS 1024
sq_status segquant_calib_scales_static(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                       const sq_segtable *seg, sq_code code, int is_weight, int dual,
                                       uint32_t flags, float *s_pos, float *s_neg, void *stream);

/* Step "activation quantization" -- Sec. 4.3.2 Q_dual with the polarity split X_+ / X_-, plus the
 * clip of the Sec. 3 uniform quantizer; x/s is one IEEE fp32 division, rounding is half-to-even.
 *   s_neg != NULL (dual): x >= 0 -> c_pos = clip(round(x/s_pos[p]), 0, q_max), c_neg = 0;
 *                         x <  0 -> c_neg = clip(round(x/s_neg[p]), q_min, 0), c_pos = 0.
 *   s_neg == NULL (single scale): c_pos = clip(round(x/s_pos[p]), -q_max, q_max); c_neg unused.
 *   e4m3 codes: "round" is the round-to-nearest-even cast to e4m3 (finite, max 448, subnormals
 *   kept), saturating; a result of -0 is stored as +0.
 *   X [M,K] dev (dtype dt, ld elements); c_pos, c_neg [M,K] dev, 1 byte per code, leading dimension
 *   ldc bytes.  Alignment: X, c_pos, c_neg 16 bytes; ld*sizeof(dt) and ldc multiples of 16 bytes.
 *   Inputs must be finite: every finite x, however large, gets the clipped code of the definition; the codes of
 *   infinities and NaNs are unspecified (an int8 DualScale +inf sets both of its codes). */
sq_status segquant_quantize_act(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                const sq_segtable *seg, const float *s_pos, const float *s_neg,
                                sq_code code, uint32_t flags, void *c_pos, void *c_neg, int64_t ldc,
                                void *stream);

/* The act-to-linear segment fused into the quantizer -- Sec. 4.3.2 ("the computation path from an activation
 * function to its subsequent linear operator"), App. B (DualScale is applied behind SiLU and GELU), Sec. 4.2.2 last
 * paragraph with App. B "Extra Hyperparameter Settings" (SmoothQuant's migration with one strength per segment: a
 * per-channel multiplier in front of the quantizer, the reciprocal smoothing factor, made offline).
 *   H [M,K] dev is the PRE-activation; per element a = act(h) (SQ_ACT_SILU: h / (1 + exp(-h)); SQ_ACT_GELU:
 *   (h / 2) erfc(-h / sqrt 2); SQ_ACT_NONE: a = h), rounded once to dtype dt (the dtype the unfused graph would
 *   have stored it in), then x = a * mult[k] as one fp32 multiply (mult dev [K] fp32, or NULL), then the codes
 *   of segquant_quantize_act for x.  The activation never goes through device memory.
 *   Accuracy of the activation: evaluated in fp32 with relative error <= (|h| + 8) 2^-23 (SiLU) and
 *   (3 h^2 + 48) 2^-24 (GELU); where the exact value lies that close to a rounding boundary of dt the stored
 *   value, and with it the code, may be that of the neighbouring dt value.  With SQ_ACT_NONE the codes are exact.
 *   SQ_ACT_GEGLU (gated GELU; App. B names it without a form): H is [M, 2K] with ld >= 2K, value half in columns
 *   [0, K), gate half in [K, 2K), a[k] = H[k] * GELU(H[K + k]) with relative error <= (3 g^2 + 49) 2^-24, g the
 *   gate; K, mult, the segment table and the codes refer to the K outputs.  The gate half must start on a 16-byte
 *   boundary: K a multiple of 8 (bf16) or 4 (fp32), else SQ_ERR_ALIGN.
 *   Everything else as for segquant_quantize_act. */
sq_status segquant_quantize_act_fused(const void *H, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                      const sq_segtable *seg, const float *s_pos, const float *s_neg,
                                      sq_code code, uint32_t flags, sq_act act, const float *mult,
                                      void *c_pos, void *c_neg, int64_t ldc, void *stream);

/* Comparison scheme: zero-point (asymmetric) quantization, App. A -- X^ = round(X / s_X) + z_X with an integer
 * zero-point, recovered by s_X s_W (X^ W^ - z_X rowsum(W^)) for symmetric weight codes (the paper's rowsum runs
 * over the input dimension).  int8 codes only.
 *   segquant_calib_zero_point: per K-segment p, from strict min/max over the calibration batch with the range
 *     widened to contain 0:  s_x[p] = (hi - lo) / 255,  z_x[p] = -128 - round(lo / s_x[p])  (lo maps to -128);
 *     a zero range gives s = 1, z = 0.  s_x dev float [P], z_x dev int32 [P].
 *   segquant_quantize_act_zero_point: codes[m][k] = clip(round(x / s_x[p]) + z_x[p], -128, 127), one IEEE fp32
 *     division, round half to even.  codes [M,K] dev, ldc bytes.
 *   segquant_fold_zero_point (offline): the correction term does not depend on the token, so it is folded into
 *     the bias:  bias_folded[n] = bias[n] - sum_p s_x[p] s_w[p*Q+q(n)] z_x[p] * (sum over K-segment p of Wq[n][k]),
 *     evaluated in fp32 (exact integer sums; per K-segment one product of the two scales and one FMA, ascending p).
 *     bias may be NULL (zero).  The layer then runs as segquant_seglinear_gemm(codes, ..., s_x, s_w, bias_folded).
 *   Alignment and limits as for the corresponding symmetric calls. */
sq_status segquant_calib_zero_point(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                    const sq_segtable *seg, float *s_x, int32_t *z_x,
                                    void *workspace, size_t ws_bytes, void *stream);
sq_status segquant_quantize_act_zero_point(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                           const sq_segtable *seg, const float *s_x, const int32_t *z_x,
                                           void *codes, int64_t ldc, void *stream);
sq_status segquant_fold_zero_point(const void *Wq, int64_t ldw, int64_t N, int64_t K, const sq_segtable *seg,
                                   const float *s_x, const int32_t *z_x, const float *s_w, const float *bias,
                                   float *bias_folded, void *stream);

/* Step "weight quantization" (offline) -- Sec. 4.2.2: every block W(p,q) is quantized separately,
 * W^ = clip(round(W / s_w[p*Q+q]), -q_max, q_max) (App. A symmetric case).
 *   W [N,K] dev (dtype dt, ld elements); s_w dev [P*Q]; Wq [N,K] dev codes, leading dimension ldq bytes. */
sq_status segquant_quantize_weight(const void *W, sq_dtype dt, int64_t N, int64_t K, int64_t ld,
                                   const sq_segtable *seg, const float *s_w, sq_code code,
                                   uint32_t flags, void *Wq, int64_t ldq, void *stream);

/* Steps "low-bit GEMM" + "dequantizing epilogue", single activation scale per K-segment --
 * Sec. 4.2.2 (output-segmented: Y^ = [X^ W^_1, ..., X^ W^_N]; input-segmented: Y^ = sum_i X^_i W^_i)
 * with the App. A symmetric recovery Y = s_X s_W Y^ applied per segment pair:
 *   y[m][n] = sum_p s_x[p] * s_w[p*Q+q(n)] * acc[p][m][n] + bias[n],
 *   acc[p][m][n] = sum_{k in K-segment p} Xq[m][k] * Wq[n][k]   (int32 for int8 codes, exact;
 *   fp32 tensor-core accumulation for e4m3 codes).
 *   Xq [M,K], Wq [N,K] dev codes (ldx, ldw in bytes); s_x dev [P]; s_w dev [P*Q]; bias dev [N] fp32 or
 *   NULL; Y [M,N] dev of y_dtype (bf16 round-to-nearest-even, or fp32), ldy in elements.
 *   acc_dump: NULL, or a dev buffer [P][M][N] (int32 for int8, fp32 for e4m3) that receives the raw
 *   accumulators (used by parity tests).
 *   Alignment: Xq, Wq, Y 16 bytes; ldx, ldw multiples of 16; ldy*sizeof(y_dtype) a multiple of 16;
 *   N a multiple of 8; interior K-segment bounds multiples of 32, K a multiple of 16.
 *   Limits: P <= SQ_MAX_P, Q <= SQ_MAX_Q, P * Q <= 2048 (1024 for the dual entry point), K <= 131072
 *   (int8: |acc| stays below 2^31).
 *   The epilogue multiplies c = s_x*s_w in fp32 and accumulates with fp32 FMAs in ascending p. */
sq_status segquant_seglinear_gemm(const void *Xq, int64_t ldx, const void *Wq, int64_t ldw,
                                  int64_t M, int64_t N, int64_t K, const sq_segtable *seg, sq_code code,
                                  const float *s_x, const float *s_w, const float *bias,
                                  void *Y, sq_dtype y_dtype, int64_t ldy, void *acc_dump,
                                  void *workspace, size_t ws_bytes, void *stream);

/* The same two steps for a DualScale layer -- Sec. 4.3.2 last display, combined with segments:
 *   y[m][n] = sum_p ( s_pos[p]*s_w[p*Q+q(n)]*acc_pos[p][m][n] + s_neg[p]*s_w[p*Q+q(n)]*acc_neg[p][m][n] ) + bias[n]
 *   where acc_pos / acc_neg are the contractions of Xq_pos / Xq_neg with the SAME weight tile.
 *   acc_dump (optional): [P][2][M][N], polarity 0 = positive path.
 *   Layers with several K-segments pass them through tensor memory one after the other and keep fp32
 *   running sums in registers, so P is only bounded by SQ_MAX_P. */
sq_status segquant_dualscale_gemm(const void *Xq_pos, const void *Xq_neg, int64_t ldx,
                                  const void *Wq, int64_t ldw, int64_t M, int64_t N, int64_t K,
                                  const sq_segtable *seg, sq_code code,
                                  const float *s_pos, const float *s_neg, const float *s_w,
                                  const float *bias, void *Y, sq_dtype y_dtype, int64_t ldy,
                                  void *acc_dump, void *workspace, size_t ws_bytes, void *stream);

/* Bytes of device scratch segquant_layer_forward needs for the code matrices of an [M,K] input. */
size_t segquant_layer_scratch_bytes(int64_t M, int64_t K, int dual);

/* The whole per-call path of one layer -- quantize (Sec. 4.3.2 Q_dual) -> GEMM -> epilogue -- as
 * one call: X [M,K] of dtype dt in -> Y [M,N] out.  s_neg == NULL selects the single-scale layer.
 *   x_on_host / y_on_host != 0: X / Y are HOST buffers (pinned memory recommended); the call copies
 *   X to `x_stage` (dev, M*ld*sizeof(dt) bytes) before and Y from `y_stage` (dev, M*ldy*sizeof(y_dtype)
 *   bytes) after the kernels, on `stream`.  With device X / Y the stage pointers are ignored.
 *   scratch: dev, segquant_layer_scratch_bytes(M,K,dual) bytes, 256-byte aligned (code matrices). */
sq_status segquant_layer_forward(const void *X, int x_on_host, void *x_stage, sq_dtype dt,
                                 int64_t M, int64_t K, int64_t ld,
                                 const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg, sq_code code,
                                 const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                                 uint32_t flags, void *Y, int y_on_host, void *y_stage, sq_dtype y_dtype, int64_t ldy,
                                 void *scratch, size_t scratch_bytes,
                                 void *workspace, size_t ws_bytes, void *stream);

/* segquant_layer_forward for host X and Y with the copies overlapped with the kernels: the rows are cut
 * into `chunks` pieces of whole 256-row tiles; piece i is copied in on `stream_in`, quantized and
 * multiplied on `stream`, copied out on `stream_out`, so that piece i+1 arrives and piece i-1 leaves while
 * piece i is computed.  Results are identical to segquant_layer_forward.  The three streams must differ;
 * `stream` completes when the last output copy has, so synchronizing `stream` is enough.  X and Y should
 * be pinned host memory (otherwise the copies do not overlap); x_stage / y_stage / scratch / workspace as
 * for segquant_layer_forward.  The call creates and releases a few CUDA events; it allocates no device
 * memory.  1 <= chunks <= 64. */
sq_status segquant_layer_forward_pipelined(const void *X, void *x_stage, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                           const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg,
                                           sq_code code, const float *s_pos, const float *s_neg, const float *s_w,
                                           const float *bias, uint32_t flags, void *Y, void *y_stage,
                                           sq_dtype y_dtype, int64_t ldy, void *scratch, size_t scratch_bytes,
                                           void *workspace, size_t ws_bytes, int chunks, void *stream,
                                           void *stream_in, void *stream_out);

/* 4-bit weights with per-channel scales, 8-bit activations with dynamic per-token scales -- App. B "Extra
 * Hyperparameter Settings" ("In 4-bit settings, weights are quantized per-channel, and activations are quantized
 * dynamically per-token"), Table 1 rows "4/8 (int)"; combined with input segmentation (Sec. 4.2.2 item 2) and
 * DualScale (Sec. 4.3.2) every row gets one scale per K-segment (and polarity) from its own extrema.
 *   segquant_quantize_per_row: for every row r of X [rows,K] and K-segment p
 *       s_neg == NULL: s_pos[r*P+p] = max|x| / q_max,  codes clip(round(x / s), -q_max, q_max) into c_pos;
 *       s_neg != NULL: s_pos[r*P+p] = max(max x, 0) / 127, s_neg[r*P+p] = max(-min x, 0) / 128 and the DualScale codes
 *                      of segquant_quantize_act into c_pos / c_neg (bits = 8 only);
 *     bits = 8: q_max = 127 (tokens of an activation matrix); bits = 4: q_max = 7 (output channels of a weight
 *     matrix; symmetric 4-bit codes in [-7, 7], one int8 per code, to be packed by segquant_pack_w4).
 *     An extremum of 0 gives scale 1.  s_pos / s_neg: dev float [rows*P], written.  K <= 16384 (a row is held in
 *     one thread block's registers); more is refused with SQ_ERR_UNSUPPORTED.  Alignment as segquant_quantize_act.
 *   segquant_pack_w4 / segquant_unpack_w4: int8 codes in [-8, 7] <-> two 4-bit two's-complement codes per byte,
 *     code 2j in the low nibble of byte j.  Wq8 [N,K] (ld8 bytes, 16-byte aligned), Wq4 [N,K/2] (ld4 bytes, 8-byte
 *     aligned, a multiple of 8); K a multiple of 16.  The GEMM reads 8-bit operands, so a layer keeps its weights
 *     packed (half the bytes) and unpacks them into an int8 scratch matrix in front of the GEMM.
 *   segquant_w4a8_gemm: y[m][n] = sum_p ( s_pos[m*P+p] s_w[n*P+p] acc_pos[p][m][n]
 *                                        + s_neg[m*P+p] s_w[n*P+p] acc_neg[p][m][n] ) + bias[n]
 *     with the accumulators of segquant_dualscale_gemm (Xq_neg == NULL: single path, s_neg ignored).  s_pos / s_neg
 *     dev [M*P], s_w dev [N*P] as written by segquant_quantize_per_row; the segment table must have Q = 1.  Per
 *     term one fp32 product of the two scales and one FMA, ascending p.  Other arguments, alignment and limits
 *     as segquant_dualscale_gemm. */
sq_status segquant_quantize_per_row(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                    const sq_segtable *seg, int bits, uint32_t flags, float *s_pos, float *s_neg,
                                    void *c_pos, void *c_neg, int64_t ldc, void *stream);
sq_status segquant_pack_w4(const void *Wq8, int64_t ld8, int64_t N, int64_t K, void *Wq4, int64_t ld4, void *stream);
sq_status segquant_unpack_w4(const void *Wq4, int64_t ld4, int64_t N, int64_t K, void *Wq8, int64_t ld8, void *stream);
sq_status segquant_w4a8_gemm(const void *Xq_pos, const void *Xq_neg, int64_t ldx, const void *Wq8, int64_t ldw,
                             int64_t M, int64_t N, int64_t K, const sq_segtable *seg,
                             const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                             void *Y, sq_dtype y_dtype, int64_t ldy, void *acc_dump,
                             void *workspace, size_t ws_bytes, void *stream);

/* A layer call prepared once and replayed.  segquant_plan_layer does everything segquant_layer_forward does on
 * the host for device X and Y -- argument checks, tile plan, kernel choice, tensor-map encoding, attribute set-up --
 * and stores the result in caller-owned memory instead of launching; segquant_plan_run then issues the layer's
 * two kernels (quantize, GEMM + epilogue) on `stream` with no further checks, queries or encoding, for callers
 * that run the same layer on the same buffers again and again (its host cost is two kernel launches).
 *   The plan is plain data: it may be copied or freed at will and owns nothing.  It refers to the buffers by
 *   address: X, Wq, the scale tables, bias, Y, scratch and workspace must stay where they were (their CONTENTS
 *   may change between runs); after any pointer, shape or pitch change build a new plan.  A plan belongs to the
 *   device that was current when it was built and to this process; segquant_plan_run on a zeroed or failed
 *   plan, or with another device current, returns SQ_ERR_UNSUPPORTED.  Arguments as for segquant_layer_forward
 *   with device X and Y. */
#define SQ_PLAN_BYTES 4096
typedef struct { uint64_t opaque[SQ_PLAN_BYTES / 8]; } sq_plan;
sq_status segquant_plan_layer(sq_plan *plan, const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                              const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg, sq_code code,
                              const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                              uint32_t flags, void *Y, sq_dtype y_dtype, int64_t ldy,
                              void *scratch, size_t scratch_bytes, void *workspace, size_t ws_bytes);
sq_status segquant_plan_run(const sq_plan *plan, void *stream);

/* Synchronizes `stream`, reads the device status word of `workspace` and clears it.  Returns SQ_OK,
 * SQ_ERR_TIMEOUT (a bounded wait inside a kernel expired; *detail, if not NULL, receives a code that
 * names the wait) or SQ_ERR_CUDA. */
sq_status segquant_last_device_status(void *workspace, void *stream, uint32_t *detail);

/* Tile plan of the GEMM kernel: tile_n in {0 (automatic), 32, 64, 128, 256}; stages 0 (automatic) or
 * 2..8 (shared-memory ring depth); cta_group 0 (automatic: CTA pairs on 256-row tiles when M > 128),
 * 1 (one CTA per 128-row tile) or 2; segment_mode for layers with several K-segments: 0 (automatic:
 * segments pass through tensor memory one after the other, running sums in registers), 1 (all
 * accumulators of a tile resident in tensor memory; at most 16 of them), 2 (sequential) or 4
 * (automatic, but single-scale layers keep 256 x 256 tiles instead of 256 x 512 ones) or 5 (256 x 512
 * tiles for single-scale layers even where the automatic choice expects no gain from them), 6 (split
 * tiles wherever the layer and the workspace allow them) or 7 (never split tiles).
 * Process-wide (atomic words read when a launch or a plan is prepared); meant for benchmarking sweeps and
 * tests only: production callers leave everything automatic.  Values the layer cannot use are replaced by the
 * automatic choice. */
sq_status segquant_set_tuning(int tile_n, int stages, int cta_group, int segment_mode);

/* The fused activation of segquant_quantize_act_fused has two implementations with identical results: one that
 * evaluates SiLU / GELU per element, and, for bf16 inputs, one that looks the stored activation up in a table of
 * all 65536 bf16 values which every thread block builds in shared memory first (about 9 us per launch, then one
 * load per element).  fused_table_mode: 0 automatic (the table from 8 Mi elements up for GELU, 16 Mi for SiLU), 1 the table wherever it
 * applies, 2 never.  Process-wide and for tests and sweeps, like segquant_set_tuning. */
sq_status segquant_set_quantize_tuning(int fused_table_mode);

/* Text of the CUDA error behind the most recent SQ_ERR_CUDA of a GEMM launch ("no error" if none). */
const char *segquant_last_cuda_error(void);

/* Number of kernels the library has launched in this process (all entry points). */
uint64_t segquant_launch_count(void);

const char *segquant_status_string(sq_status s);

#ifdef __cplusplus
}
#endif
#endif /* SEGQUANT_H_ */
