/*
 * twn.h -- C ABI of the Ternary Weight Networks hot path for NVIDIA B200 (sm_100a).
 *
 * Threshold ternarization of fp32 master weights with 2-bit packing, and the
 * ternary-weight contractions (inner product, convolution forward, backward
 * for data, straight-through weight gradient) that consume the packed codes.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The caller owns every buffer.  Unless a function says otherwise it
 *     allocates nothing, frees nothing and keeps no pointer after it returns.
 *   - Work is enqueued on `stream` (a cudaStream_t) and the call returns after
 *     the launch; results are ready when the stream reaches that point.
 *   - Return value: TWN_OK or a negative twn_status.  Errors that the host can
 *     see (bad sizes, misalignment, NULL) are returned before anything is
 *     launched.  Errors only the device can see (non-finite weights, invalid
 *     codes, a bounded wait that ran out) are written to `status` of the
 *     twn_stats_t / status word the call was given and read back with
 *     twn_read_status() after the caller synchronises.
 *   - Results are deterministic: same inputs, same bits.
 *   - bf16 tensors are passed as `const void*` / `void*`; conv tensors are
 *     NHWC; filters are [Cout][kh][kw][Cin] with Cin fastest.
 *   - There is no CPU path.  On a device that is not sm_100 every compute
 *     call returns TWN_ERR_UNSUPPORTED_ARCH.
 */
#ifndef TWN_H_
#define TWN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *twn_stream_t; /* == cudaStream_t */

typedef enum {
    TWN_OK = 0,
    TWN_ERR_INVALID_ARG = -1,
    TWN_ERR_MISALIGNED = -2,
    TWN_ERR_WORKSPACE = -3,
    TWN_ERR_NONFINITE = -4,   /* device: a master weight is NaN or +-Inf           */
    TWN_ERR_TIMEOUT = -5,     /* device: a bounded wait inside a kernel ran out    */
    TWN_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed               */
    TWN_ERR_UNSUPPORTED_ARCH = -7,
    TWN_ERR_BAD_CODE = -8,    /* device: an int8 code outside {-1,0,+1}            */
    TWN_ERR_TOO_LARGE = -9    /* a size beyond what a fixed-capacity entry point takes */
} twn_status;

enum { TWN_F32 = 0, TWN_BF16 = 1 };

/* Result of one ternarization; lives in device memory so that the contraction
 * kernels read alpha without a host round trip.  64 bytes. */
typedef struct {
    double delta;        /* threshold: delta_factor * (1/n) * sum |W_i|  (Sec. 2.3)     */
    double alpha;        /* scale: mean of |W_i| over |W_i| > delta, 0 if none (Eq. 5)  */
    double sum_abs;      /* sum |W_i|                                                  */
    double sum_abs_kept; /* sum of |W_i| over |W_i| > delta                            */
    uint64_t n_neg, n_zero, n_pos; /* code counts, padding excluded                    */
    int32_t status;      /* twn_status written by the device                           */
    int32_t reserved;
} twn_stats_t;

/* Convolution geometry.  Output extent Ho = (H + 2*pad_h - kh)/stride_h + 1. */
typedef struct {
    int64_t B, H, W, Cin, Cout;
    int32_t kh, kw, stride_h, stride_w, pad_h, pad_w;
} twn_conv_desc_t;

/* What follows the contraction, per output element with channel n:
 *   y = acc * alpha;  y = y * scale[n] + shift[n];  y += residual;  y = max(y, 0)
 * each step only if its field is set.  (Eq. 2 puts alpha on the input; a scalar
 * commutes with the sum, so it is applied once per output here.)
 * With residual_op = TWN_RESIDUAL_GATE the tensor given as `residual` is not added but gates
 * the result: y is kept where residual > 0 and is 0 elsewhere.  This is the backward pass of
 * a ReLU fused into the backward-for-data pass of the layer above it: with `residual` = the
 * lower layer's output and `scale` = its folded batch-norm scale, twn_conv2d_bwd_data writes
 * the lower layer's dZ directly (Algorithm 1, TernaryBackward, followed by the chain rule
 * through y = relu(z * scale + shift)). */
enum { TWN_RESIDUAL_ADD = 0, TWN_RESIDUAL_GATE = 1 };
typedef struct {
    const float *scale;    /* fp32 [N] or NULL (folded batch-norm scale)            */
    const float *shift;    /* fp32 [N] or NULL                                      */
    const void *residual;  /* same shape and leading dimension as Y, or NULL        */
    int32_t residual_dtype;/* TWN_F32 | TWN_BF16                                    */
    int32_t relu;          /* 0 | 1                                                 */
    int32_t out_dtype;     /* TWN_F32 | TWN_BF16 (round to nearest even)            */
    int32_t residual_op;   /* TWN_RESIDUAL_ADD (0) | TWN_RESIDUAL_GATE              */
} twn_epilogue_t;

/* ---- library ---------------------------------------------------------- */

/* Text for a twn_status.  Host; static storage. */
const char *twn_strerror(int status);

/* Copies the device status word at `dev_status` (e.g. &stats->status) to
 * *host_out with a blocking copy on `stream`.  Returns TWN_OK or TWN_ERR_CUDA. */
int twn_read_status(const int32_t *dev_status, int32_t *host_out, twn_stream_t stream);

/* ---- ternarization (Sec. 2.3: Eq. 3, Eq. 5, threshold rule; Algorithm 1) -- */

/* Bytes of scratch twn_ternarize needs (independent of the tensor size). */
size_t twn_ternarize_workspace_bytes(void);

/*
 * Per-layer threshold ternarization fused with 2-bit packing.
 *   delta  = delta_factor * (1/n) * sum_i |W_i|,  n = rows*cols (zeros count)
 *   code_i = +1 if W_i > delta, -1 if W_i < -delta, 0 if |W_i| <= delta   (Eq. 3)
 *   alpha  = mean of |W_i| over { i : |W_i| > delta }                      (Eq. 5)
 * The paper's rule of thumb is delta_factor = 0.75; any value >= 0 is accepted.
 *
 * W        fp32 [rows, cols], contiguous, 16-byte aligned.  rows = filters
 *          (output channels), cols = fan-in.
 * stats    one twn_stats_t, 8-byte aligned; written completely.
 * packed   uint32 [rows][ld_codes/16].  A field is two bits: 00 = 0, 01 = +1,
 *          11 = -1 (10 is never written).  Code j of a row lives in word j/16;
 *          inside the word the even elements fill the low half-word and the odd
 *          elements the high half-word, each from its top bits down: element
 *          e = j%16 is at bit position 14 - 2*(e/2) + 16*(e%2).  (The paper fixes
 *          no encoding; with this one a left shift by 2*(e/2) and one mask turn
 *          the fields of elements e, e+1 into the sign and top exponent bit of a
 *          pair of bf16 tensor-core operands, +-2 or 0.)
 *          ld_codes is a multiple of 64 (rows start 16-byte aligned),
 *          ld_codes >= cols; the padding is written as 00.  16-byte aligned.
 * codes_i8 optional int8 [rows, cols] copy of the codes (16-byte aligned), or NULL.
 * workspace/workspace_bytes  scratch of at least twn_ternarize_workspace_bytes(),
 *          256-byte aligned; contents need not be preserved or initialised.
 *          Two calls that overlap on the device must not share it.
 * The sums are fp64 with a fixed reduction order.  The comparison is done in
 * fp32 against delta rounded toward -inf, which decides exactly as the fp64
 * comparison does.  n = 0 gives delta = alpha = 0.
 * Device status: TWN_ERR_NONFINITE if any W_i is NaN/Inf (other outputs
 * are then unspecified).
 */
int twn_ternarize(const float *W, int64_t rows, int64_t cols, double delta_factor,
                  twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                  int8_t *codes_i8, void *workspace, size_t workspace_bytes,
                  twn_stream_t stream);

/*
 * The first loop of Algorithm 1 for a whole network: ternarizes up to 32 tensors (layers) with one
 * launch per sweep instead of one per tensor.  Every tensor gets its own per-layer threshold,
 * codes and scale exactly as from a twn_ternarize call of its own (same reduction order, same bits).
 *   items     HOST array of `count` descriptors; the fields have the meaning and the alignment
 *             rules of the twn_ternarize arguments of the same name (device pointers inside).
 *             Read during the call only.
 *   workspace device scratch of at least twn_ternarize_batch_workspace_bytes(count), 256-byte
 *             aligned; contents need not be preserved or initialised.
 * Errors: TWN_ERR_INVALID_ARG for count > 32 or a bad descriptor (nothing is launched).
 */
typedef struct {
    const float *W;
    int64_t rows, cols;
    twn_stats_t *stats;
    uint32_t *packed;
    int64_t ld_codes;
    int8_t *codes_i8;     /* optional */
} twn_ternarize_item_t;
size_t twn_ternarize_batch_workspace_bytes(int count);
int twn_ternarize_batch(const twn_ternarize_item_t *items, int count, double delta_factor,
                        void *workspace, size_t workspace_bytes, twn_stream_t stream);

/*
 * twn_ternarize for callers that may not allocate.  (The paper has no counterpart;
 * this is a packaging variant of the call above, same arithmetic, same results.)
 *
 * Some hosts of this library cannot obtain device memory for the scratch buffer
 * twn_ternarize asks for: code that runs inside another framework's memory plan
 * and is handed exactly its input and output tensors, plugins loaded by a serving
 * process whose allocator is frozen once the model is up, and callers on a path
 * where cudaMalloc's implicit device synchronisation is not acceptable.  For them
 * the scratch lives inside the library: a static device array of
 * TWN_TERNARIZE_STATIC_SCRATCH_BYTES that every GPU which loads the library holds
 * until the process exits.  This call allocates and frees nothing, on the host or
 * on the device, and calls no routine that does.
 *
 * Arguments and results are those of twn_ternarize without workspace/workspace_bytes.
 * Limits and rules:
 *   - rows*cols may not exceed TWN_TERNARIZE_STATIC_MAX_WEIGHTS; a larger tensor is
 *     refused with TWN_ERR_TOO_LARGE before anything is launched.
 *   - The first call on each device looks up the array's device address (once per
 *     device, with that device current).  Make that first call outside any stream
 *     capture.
 *   - All calls share the one array.  It keeps whatever the previous call left; the
 *     words that must start at zero are cleared on `stream` at the start of every
 *     call.  Two calls whose kernels can overlap on the GPU (different streams,
 *     no dependency between them) race on it and give wrong results: order them.
 */
#define TWN_TERNARIZE_STATIC_SCRATCH_BYTES 65792u
#define TWN_TERNARIZE_STATIC_MAX_WEIGHTS 2147483648LL /* 2^31 weights = 8 GiB of fp32 */
int twn_ternarize_static(const float *W, int64_t rows, int64_t cols, double delta_factor,
                         twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                         int8_t *codes_i8, twn_stream_t stream);

/*
 * Parameter update of Algorithm 1 (UpdateParameters; the paper trains with SGD with momentum and
 * an L2 weight decay, Sec. 3) on the fp32 master weights, in place:
 *     g = dW + weight_decay * W;   V = momentum * V + g;   W = W - lr * V
 * Every operation is a separately rounded fp32 operation in exactly this order (no fused
 * multiply-add): the result is defined to the bit.  dW is the straight-through gradient of
 * twn_conv2d_bwd_weight (or any fp32 gradient of the same shape), V the momentum buffer.
 * The next iteration begins by ternarizing the updated weights; its threshold needs
 * sum |W|, which this call accumulates while the updated weights are still in registers:
 *   stats_next (optional) receives sum_abs, delta = delta_factor * sum_abs / n and status
 *              (TWN_ERR_NONFINITE if an updated weight is NaN/Inf) of the updated tensor,
 * so that twn_ternarize_codes can write the codes and the scale without the first sweep.
 * W, dW, V: fp32 [n], 16-byte aligned.  workspace as for twn_ternarize.  Deterministic.
 */
int twn_sgd_update(float *W, const float *dW, float *V, int64_t n, float lr, float momentum,
                   float weight_decay, double delta_factor, twn_stats_t *stats_next,
                   void *workspace, size_t workspace_bytes, twn_stream_t stream);

/*
 * Second sweep of twn_ternarize alone: codes by Eq. 3 against the threshold already in
 * stats->delta (written by twn_sgd_update or by an earlier twn_ternarize of the same weights),
 * 2-bit packing, alpha by Eq. 5 and the counts.  Arguments as for twn_ternarize; stats->delta,
 * sum_abs and status are read and kept, the other fields are written.
 */
int twn_ternarize_codes(const float *W, int64_t rows, int64_t cols, twn_stats_t *stats,
                        uint32_t *packed, int64_t ld_codes, int8_t *codes_i8,
                        void *workspace, size_t workspace_bytes, twn_stream_t stream);

/* twn_sgd_update and twn_ternarize_codes for up to 32 tensors (the layers of a network) in one
 * launch each; every tensor gets the bits of a call of its own.  items: HOST arrays, read during
 * the call only; fields as the arguments of the single-tensor calls.  workspace: at least
 * twn_ternarize_batch_workspace_bytes(count), 256-byte aligned. */
typedef struct {
    float *W;
    const float *dW;
    float *V;
    int64_t n;
    twn_stats_t *stats_next;   /* optional */
} twn_sgd_item_t;
int twn_sgd_update_batch(const twn_sgd_item_t *items, int count, float lr, float momentum,
                         float weight_decay, double delta_factor, void *workspace,
                         size_t workspace_bytes, twn_stream_t stream);
int twn_ternarize_codes_batch(const twn_ternarize_item_t *items, int count, void *workspace,
                              size_t workspace_bytes, twn_stream_t stream);

/*
 * Per-filter threshold ternarization fused with 2-bit packing: Algorithm 1 as printed,
 * whose first loop runs over the filters of a layer.  Row r of W is one filter and gets
 *   delta_r = delta_factor * (1/cols) * sum_i |W_r,i|          (Sec. 2.3, n = cols)
 *   codes by Eq. 3 against delta_r
 *   alpha_r = mean of |W_r,i| over { i : |W_r,i| > delta_r }   (Eq. 5)
 * W        fp32 [rows, cols], contiguous, 4-byte aligned (a 16-byte aligned matrix with
 *          cols % 4 == 0 takes the fast path: filters of up to 16384 weights cross HBM once).
 * stats    twn_stats_t [rows], 8-byte aligned; entry r is written completely (status
 *          TWN_ERR_NONFINITE when filter r holds a NaN/Inf; the other filters are unaffected).
 * packed   uint32 [rows][ld_codes/16], layout and padding as for twn_ternarize; 16-byte aligned.
 * codes_i8 optional int8 [rows, cols] copy of the codes, or NULL.
 * Needs no scratch memory.  Deterministic; the comparison is done as in twn_ternarize.
 * The contraction kernels take one alpha per call, so for per-filter scales pass stats = NULL
 * to them and fold the alphas into the epilogue's per-channel scale with twn_rows_scale
 * (forward), or into the scale of twn_act_bwd (backward: the gradient with respect to the
 * ternary weights' output carries alpha_r on the reduction index of the backward-for-data pass).
 */
int twn_ternarize_rows(const float *W, int64_t rows, int64_t cols, double delta_factor,
                       twn_stats_t *stats, uint32_t *packed, int64_t ld_codes,
                       int8_t *codes_i8, twn_stream_t stream);

/* scale_out[r] = alpha_r * scale_in[r] (scale_in NULL: 1), r < rows, fp32: the per-filter scales
 * of Algorithm 1 as the per-channel scale of twn_epilogue_t.  The most severe status of the
 * `rows` entries is merged into *dev_status (optional). */
int twn_rows_scale(const twn_stats_t *stats, int64_t rows, const float *scale_in, float *scale_out,
                   int32_t *dev_status, twn_stream_t stream);

/* ---- 2-bit storage (Sec. 2.1, model compression) ------------------------- */

/*
 * Packs int8 codes in {-1,0,+1} ([rows, cols], contiguous) into the layout
 * described at twn_ternarize.  `counts` (optional) receives n_neg/n_zero/n_pos
 * and a status; its other fields are zeroed.  A code outside {-1,0,+1} sets
 * TWN_ERR_BAD_CODE there (and packs as 0).
 */
int twn_pack(const int8_t *codes, int64_t rows, int64_t cols, uint32_t *packed,
             int64_t ld_codes, twn_stats_t *counts, twn_stream_t stream);

/* Inverse of twn_pack: int8 [rows, cols] from packed rows.  The unused field
 * 10 unpacks as 0 and sets TWN_ERR_BAD_CODE in *dev_status (optional). */
int twn_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes,
               int8_t *codes, int32_t *dev_status, twn_stream_t stream);

/*
 * Re-lays the packed filters of a convolution for the backward-for-data pass:
 * from [Cout][kh][kw][Cin] (rows of ld_fwd codes) to [Cin][kh][kw][Cout]
 * (rows of ld_bwd codes, same tap order, no spatial flip; padding 00).
 * For an inner-product layer use kh = kw = 1: a plain transpose.
 */
int twn_transpose_codes(const uint32_t *packed_fwd, int64_t ld_fwd, const twn_conv_desc_t *desc,
                        uint32_t *packed_bwd, int64_t ld_bwd, twn_stream_t stream);

/* twn_transpose_codes for up to 32 filter banks in one launch (all layers of a training step).
 * items: HOST array, read during the call only; fields as the arguments of twn_transpose_codes. */
typedef struct {
    const uint32_t *packed_fwd;
    int64_t ld_fwd;
    twn_conv_desc_t desc;
    uint32_t *packed_bwd;
    int64_t ld_bwd;
} twn_transpose_item_t;
int twn_transpose_codes_batch(const twn_transpose_item_t *items, int count, twn_stream_t stream);

/* ---- ternary-weight contractions (Eq. 2; Algorithm 1, TernaryForward/Backward) ---- */

/*
 * Inner product (fully-connected layer):  Y[M,N] = epi( alpha * X[M,K] * T^T ).
 *   X         bf16 [M, ldx], row-major, 16-byte aligned, ldx >= K, ldx % 8 == 0.
 *   T_packed  N rows of K codes (row n = output unit n, the [out, in] order of the
 *             master weights) in the layout of twn_ternarize, row pitch ld_codes.
 *   stats     the twn_stats_t of the ternarization; only alpha is read, on the
 *             device.  NULL means alpha = 1.
 *   epi       optional epilogue (NULL: none, fp32 output).
 *   Y         [M, ldy] fp32 or bf16 (epi->out_dtype), ldy >= N, 4-byte aligned.
 *   dev_status optional device int32 that receives TWN_ERR_TIMEOUT if a bounded
 *             wait inside the kernel runs out (the kernel then exits early and the
 *             output is unspecified).  Must be zero (TWN_OK) before the call.
 * Products are exact (the codes are exactly -1/0/+1 in bf16); accumulation is fp32
 * on the tensor cores; alpha and the epilogue are applied in fp32.
 */
int twn_gemm(const void *X, int64_t ldx, const uint32_t *T_packed, int64_t ld_codes,
             const twn_stats_t *stats, int64_t M, int64_t N, int64_t K,
             const twn_epilogue_t *epi, void *Y, int64_t ldy, int32_t *dev_status,
             twn_stream_t stream);

/*
 * Convolution forward (cross-correlation, zero padding):
 *   Y[b,ho,wo,o] = epi( alpha * sum_{r,s,c} X[b, ho*stride_h - pad_h + r, wo*stride_w - pad_w + s, c]
 *                                           * T[o,r,s,c] )
 *   X      bf16 NHWC [B,H,W,Cin], contiguous, 16-byte aligned.
 *   T_fwd  Cout rows of kh*kw*Cin codes ([Cout][kh][kw][Cin]), row pitch ld_codes.
 *   Y      NHWC [B,Ho,Wo,Cout], contiguous, fp32 or bf16.
 * Requires Cin % 16 == 0 (Cin % 8 == 0 for a 1x1 filter) and kh*kw <= 64; other
 * layers go through twn_im2col + twn_gemm.  Other arguments as in twn_gemm.
 */
int twn_conv2d_fwd(const twn_conv_desc_t *desc, const void *X, const uint32_t *T_fwd, int64_t ld_codes,
                   const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                   int32_t *dev_status, twn_stream_t stream);

/*
 * twn_conv2d_fwd that also returns the batch statistics of its output, for the batch normalisation
 * that follows every ternary convolution while the network is trained (Sec. 2.4; the block of Fig. 1):
 *   bn_sum[o]   = sum over (b, ho, wo) of z[b,ho,wo,o]
 *   bn_sumsq[o] = sum over (b, ho, wo) of z[b,ho,wo,o]^2
 * with z = alpha * acc * scale[o] + shift[o], the value before the residual and the ReLU of the
 * epilogue (with scale = shift = NULL: the plain convolution output).  The sums are taken of the
 * fp32 values in the kernel's epilogue, not of a rounded copy: per thread in fp32 over at most a
 * tile's pixels, across tiles in fp64 and in a fixed order (deterministic).
 *   bn_sum, bn_sumsq  fp64 [Cout], overwritten; 8-byte aligned.
 *   workspace         at least twn_conv2d_fwd_bn_workspace_bytes(desc) bytes, 16-byte aligned: per-tile
 *                     partial sums.
 * Everything else as in twn_conv2d_fwd.  twn_bn_finalize turns the sums over n = B*Ho*Wo values into the
 * mean, the biased variance and the affine of the normalisation:
 *   scale[o] = gamma[o] / sqrt(var[o] + eps),  shift[o] = beta[o] - mean[o] * scale[o]
 * (gamma / beta NULL: 1 / 0; scale, shift fp32 [C]; mean, var fp64 [C]; any output may be NULL).
 */
size_t twn_conv2d_fwd_bn_workspace_bytes(const twn_conv_desc_t *desc);
int twn_conv2d_fwd_bn(const twn_conv_desc_t *desc, const void *X, const uint32_t *T_fwd, int64_t ld_codes,
                      const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y, double *bn_sum,
                      double *bn_sumsq, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                      twn_stream_t stream);
int twn_bn_finalize(const double *sum, const double *sumsq, int64_t n, int64_t C, const float *gamma,
                    const float *beta, double eps, float *scale, float *shift, double *mean, double *var,
                    twn_stream_t stream);

/*
 * Convolution backward for data (Algorithm 1: ordinary back-propagation with
 * T = alpha * W~ in place of W), the adjoint of twn_conv2d_fwd:
 *   dX[b,h,w,c] = epi( alpha * sum over (r,s,o) with ho*stride_h - pad_h + r == h,
 *                      wo*stride_w - pad_w + s == w  of  dZ[b,ho,wo,o] * T[o,r,s,c] )
 *   dZ     bf16 NHWC [B,Ho,Wo,Cout], contiguous.
 *   T_bwd  the output of twn_transpose_codes: Cin rows of kh*kw*Cout codes.
 *   dX     NHWC [B,H,W,Cin], fp32 or bf16; every element is written.
 *   epi    scale/shift are indexed by the input channel c; `residual` (shape of dX)
 *          lets a second gradient branch be added in the same pass.
 * Requires Cout % 16 == 0 (Cout % 8 == 0 for a 1x1 filter).  A strided layer runs as
 * stride_h*stride_w launches, one per residue class of (h, w) modulo the stride.
 */
int twn_conv2d_bwd_data(const twn_conv_desc_t *desc, const void *dZ, const uint32_t *T_bwd, int64_t ld_codes,
                        const twn_stats_t *stats, const twn_epilogue_t *epi, void *dX,
                        int32_t *dev_status, twn_stream_t stream);

/*
 * Straight-through weight gradient (Algorithm 1, UpdateParameters; Fig. 1 caption): the
 * gradient with respect to T = alpha*W~, applied to the fp32 master weights unchanged.  No
 * alpha factor and no mask enter:
 *   dW[o,r,s,c] = sum_{b,ho,wo} dZ[b,ho,wo,o] * X[b, ho*stride_h - pad_h + r, wo*stride_w - pad_w + s, c]
 *   X   bf16 NHWC [B,H,W,Cin];  dZ  bf16 NHWC [B,Ho,Wo,Cout];  both contiguous, 16-byte aligned.
 *   dW  fp32 [Cout][kh][kw][Cin], overwritten.
 *   workspace  at least twn_conv2d_bwd_weight_workspace_bytes(desc) bytes, 16-byte aligned:
 *              per-split partial sums, added in a fixed order (deterministic).
 * Requires Cin % 8 == 0 and Cout % 8 == 0 (layers with fewer channels: run it on the
 * twn_im2col matrix as a 1x1 convolution).  bf16 products, fp32 accumulation.
 * dev_status as in twn_gemm.
 */
size_t twn_conv2d_bwd_weight_workspace_bytes(const twn_conv_desc_t *desc);
int twn_conv2d_bwd_weight(const twn_conv_desc_t *desc, const void *X, const void *dZ, float *dW,
                          void *workspace, size_t workspace_bytes, int32_t *dev_status,
                          twn_stream_t stream);

/* ---- binary precision weights (Sec. 3: the BPWN baseline of the experiments) -------- */

/*
 * The paper compares ternary weights with binary precision weights, which "use the sign function to
 * binarize the weights" and, like the ternary ones, carry one scale per layer.  The same contraction
 * kernels run on them from a 1-bit packing:
 *   B_i   = +1 if W_i >= 0, -1 if W_i < 0   (a two-valued code has no zero: W_i = 0 and -0.0 give +1)
 *   alpha = (1/n) * sum_i |W_i|               (the scale that minimises ||W - alpha B||^2 for B = sign W)
 * One sweep over the weights (no threshold is needed): 4 bytes read, 1/32 byte written per weight.
 *   W       fp32 [rows, cols], contiguous, 4-byte aligned.
 *   stats   one twn_stats_t: alpha, sum_abs (= sum_abs_kept), n_pos, n_neg, status are written;
 *           delta = 0 and n_zero = 0.  TWN_ERR_NONFINITE as for twn_ternarize.
 *   packed  uint32 [rows][ld_codes/32].  A bit is 1 for -1 and 0 for +1.  Code j of a row lives in
 *           word j/32; inside the word the even elements fill the low half-word and the odd elements
 *           the high half-word, each from its top bit down: element e = j%32 is bit 15 - e/2 + 16*(e%2)
 *           (a left shift by e/2 and one mask turn elements e, e+1 into the sign bits of a bf16 pair).
 *           ld_codes is a multiple of 128 (rows start 16-byte aligned), ld_codes >= cols; padding bits
 *           are 0.  16-byte aligned.
 *   workspace  at least twn_binarize_workspace_bytes(), 256-byte aligned, as for twn_ternarize.
 * Deterministic (fixed-order fp64 sum).
 */
size_t twn_binarize_workspace_bytes(void);
int twn_binarize(const float *W, int64_t rows, int64_t cols, twn_stats_t *stats, uint32_t *packed,
                 int64_t ld_codes, void *workspace, size_t workspace_bytes, twn_stream_t stream);

/* int8 codes (+1 / -1) from 1-bit packed rows; [Cout][kh][kw][Cin] -> [Cin][kh][kw][Cout] re-layout of
 * 1-bit codes for the backward-for-data pass (as twn_unpack and twn_transpose_codes for ternary codes). */
int twn_unpack_b1(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes, int8_t *codes,
                  twn_stream_t stream);
int twn_transpose_codes_b1(const uint32_t *packed_fwd, int64_t ld_fwd, const twn_conv_desc_t *desc,
                           uint32_t *packed_bwd, int64_t ld_bwd, twn_stream_t stream);

/* twn_gemm, twn_conv2d_fwd and twn_conv2d_bwd_data on 1-bit binary codes: Y = epi(alpha * X (*) B), the
 * forward block of Eq. 2 and the backward pass of Algorithm 1 with B = sign(W) in place of the ternary
 * W~.  Arguments as for the ternary calls, except that the packed rows are in the 1-bit layout above
 * (row pitch a multiple of 128 codes) and that a filter with more than one tap needs channel runs of
 * 32 codes (Cin % 32 == 0 forward, Cout % 32 == 0 backward) instead of 16. */
int twn_gemm_b1(const void *X, int64_t ldx, const uint32_t *B_packed, int64_t ld_codes,
                const twn_stats_t *stats, int64_t M, int64_t N, int64_t K,
                const twn_epilogue_t *epi, void *Y, int64_t ldy, int32_t *dev_status,
                twn_stream_t stream);
int twn_conv2d_fwd_b1(const twn_conv_desc_t *desc, const void *X, const uint32_t *B_fwd, int64_t ld_codes,
                      const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                      int32_t *dev_status, twn_stream_t stream);
int twn_conv2d_bwd_data_b1(const twn_conv_desc_t *desc, const void *dZ, const uint32_t *B_bwd, int64_t ld_codes,
                           const twn_stats_t *stats, const twn_epilogue_t *epi, void *dX,
                           int32_t *dev_status, twn_stream_t stream);

/* ---- layer glue (Sec. 2.4: conv, affine, ReLU, pooling; standard back-propagation) ---- */

/*
 * Patch matrix for layers whose channel count is too small for twn_conv2d_fwd (Cin = 1, 3):
 *   Xcol[m, (r*kw + s)*Cin + c] = X[b, ho*stride_h - pad_h + r, wo*stride_w - pad_w + s, c]
 * with m = (b*Ho + ho)*Wo + wo, zero outside the image and in columns K..ldk-1.
 * Xcol is bf16 [B*Ho*Wo, ldk], ldk >= kh*kw*Cin, ldk % 8 == 0, 16-byte aligned.  The
 * convolution is then twn_gemm(Xcol, ldk, T_fwd, ...) with K = kh*kw*Cin.
 */
int twn_im2col(const twn_conv_desc_t *desc, const void *X, void *Xcol, int64_t ldk, twn_stream_t stream);

/*
 * Folded form of a stride-2 layer with very few input channels (Sec. 3.1: the first layer of
 * ResNet-18 is a 7x7 stride-2 convolution on 3 channels).  The paper has no counterpart; it
 * replaces the patch matrix by a tensor barely larger than the input.  Requirements (else
 * TWN_ERR_INVALID_ARG): stride_h = stride_w = 2, kh <= 8, kw <= 8, 4*Cin <= 16.
 *   Xf[b, i, j, (dy*2 + dx)*Cin + c] = X[b, 2i + dy - pad_h, 2j + dx - pad_w, c]   (0 outside the
 *   image; channels 4*Cin..15 are 0), bf16 [B, Hf, Wf, 16], Hf = Ho + ceil(kh/2) - 1, Wf = Wo + 3.
 * The layer is then the stride-1 sum over folded rows r' < ceil(kh/2) of the 64 consecutive
 * elements Xf[b, ho + r', wo .. wo+3, 0..15] against folded codes
 *   Tf[o][r'*64 + s'*16 + (dy*2 + dx)*Cin + c] = T[o][2r' + dy][2s' + dx][c]   (0 where no tap),
 * uint32 [Cout][ldf/16] in the packed format of twn_ternarize, ldf = 64*ceil(kh/2).
 * twn_fold_dims writes Hf, Wf, ldf (any may be NULL); twn_fold_input and twn_fold_codes build Xf
 * (16-byte aligned, overwritten completely) and Tf from X and the packed codes of twn_ternarize
 * (alpha and the statistics are unchanged).  twn_conv2d_fwd_folded equals twn_im2col + twn_gemm on
 * the same layer; twn_conv2d_bwd_weight_folded equals the weight gradient of that layer,
 * dW fp32 [Cout][kh][kw][Cin] overwritten; workspace as in twn_conv2d_bwd_weight (Cout % 8 == 0).
 */
int twn_fold_dims(const twn_conv_desc_t *desc, int64_t *Hf, int64_t *Wf, int64_t *ldf);
int twn_fold_input(const twn_conv_desc_t *desc, const void *X, void *Xf, twn_stream_t stream);
int twn_fold_codes(const twn_conv_desc_t *desc, const uint32_t *packed, int64_t ld_codes,
                   uint32_t *packed_folded, int64_t ld_folded, twn_stream_t stream);
int twn_conv2d_fwd_folded(const twn_conv_desc_t *desc, const void *Xf, const uint32_t *Tf, int64_t ld_folded,
                          const twn_stats_t *stats, const twn_epilogue_t *epi, void *Y,
                          int32_t *dev_status, twn_stream_t stream);
size_t twn_conv2d_bwd_weight_folded_workspace_bytes(const twn_conv_desc_t *desc);
int twn_conv2d_bwd_weight_folded(const twn_conv_desc_t *desc, const void *Xf, const void *dZ, float *dW,
                                 void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                 twn_stream_t stream);

/* Max pooling, window k x k (k <= 15), padding with -inf.  X, Y bf16 NHWC; `argmax` (optional,
 * one byte per output element) records the window position r*k+s of the first maximum in
 * scan order, for the backward pass. */
int twn_maxpool2d_fwd(const void *X, int64_t B, int64_t H, int64_t W, int64_t C, int k, int stride,
                      int pad, void *Y, uint8_t *argmax, twn_stream_t stream);
/* dX[b,h,w,c] = sum of dY over the windows whose recorded maximum is (h,w).  Deterministic. */
int twn_maxpool2d_bwd(const void *dY, const uint8_t *argmax, int64_t B, int64_t H, int64_t W, int64_t C,
                      int k, int stride, int pad, void *dX, twn_stream_t stream);

/* Backward through a max-pool that directly follows a layer y = relu(z * scale[c] + shift[c]),
 * fused with the backward through that ReLU and scale:
 *   dZ[b,h,w,c] = scale[c] * sum of dY over the windows whose recorded maximum is (h,w) and whose
 *                 pooled value is positive
 * (the pooled value is the layer's output at the window's arg-max, so "pooled > 0" is the ReLU gate
 * there; everywhere else the gradient is 0 anyway).  pooled: the bf16 output of twn_maxpool2d_fwd,
 * same shape as dY.  scale fp32 [C] or NULL (1).  Equals twn_maxpool2d_bwd followed by twn_act_bwd
 * up to one rounding to bf16 instead of two.  Deterministic. */
int twn_maxpool2d_bwd_act(const void *dY, const uint8_t *argmax, const void *pooled, const float *scale,
                          int64_t B, int64_t H, int64_t W, int64_t C, int k, int stride, int pad,
                          void *dZ, twn_stream_t stream);

/* Global average pooling: X bf16 [B, HW, C] -> Y bf16 [B, C]; backward dX = dY / HW. */
int twn_avgpool_fwd(const void *X, int64_t B, int64_t HW, int64_t C, void *Y, twn_stream_t stream);
int twn_avgpool_bwd(const void *dY, int64_t B, int64_t HW, int64_t C, void *dX, twn_stream_t stream);

/*
 * Backward through the epilogue y = relu(z*scale[c] + shift[c] (+ residual)):
 *   dPre = dY * [Y > 0]   (Y = the block's bf16 output; Y NULL: no ReLU, dPre = dY)
 *   dZ   = dPre * scale[c]  (scale NULL: 1)
 * n elements with channel c = index % C.  dZ and dPre are bf16; either may be NULL.
 * dPre is what flows into a residual branch, dZ into the convolution's backward passes.
 */
int twn_act_bwd(const void *dY, const void *Y, const float *scale, int64_t n, int64_t C, void *dZ,
                void *dPre, twn_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* TWN_H_ */
