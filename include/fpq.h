/*
 * fpq - low-bit floating-point quantized conv / linear layers for sm_100a.
 *
 * C ABI of the inference hot path of "Low-Bitwidth Floating Point Quantization
 * for Efficient High-Quality Diffusion Models": the layer that every U-Net
 * convolution and linear becomes once its weights are mapped to FP8 or FP4 and
 * its input activations to FP8 (Sec. VI-A: weights and activations of conv and
 * linear layers are quantized, everything else stays FP32).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.
 *   - The caller owns every buffer.  The library allocates no device memory in
 *     these calls and keeps no state except one sticky device status word
 *     (fpq_read_status) and host-side tables of things worked out once (launch
 *     plans per device, how each weight format is run).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls only enqueue work; they do not synchronise unless stated.
 *   - Calls may come from several host threads (each with its own stream and
 *     buffers); the library takes turns inside where it keeps per-device tables.
 *     fpq_set_path_policy and fpq_linear_static are the exceptions stated at their
 *     declarations.
 *   - The first layer call on a device (fpq_linear, fpq_conv2d and their forms) sets kernel
 *     attributes and asks the driver how many thread-block clusters fit: make it outside any
 *     stream capture.  Later calls only enqueue kernels and can be captured.
 *   - Errors are return codes (negative).  Whatever the host can check (null or
 *     misaligned pointers, impossible formats, shapes, workspace size, an activation
 *     scale that is not a positive finite number) is rejected before anything is launched.
 *
 * Number format (Sec. IV-B, format equation): a code has 1 sign bit, exp_bits
 * exponent bits p and man_bits mantissa bits d, value
 *     (-1)^s 2^(p - exp_bias) (1 + d / 2^man_bits)            for p > 0
 *     (-1)^s d 2^(1 - exp_bias - man_bits)                    for p = 0
 * bit (e+m) = sign, bits [m, e+m) = p, bits [0, m) = d.  1 + e + m <= 8; formats
 * of up to 4 bits are stored two per byte (even index in the low nibble).
 * exp_bias is limited to 2^exp_bits - man_bits - 104 <= exp_bias <= 126 - man_bits
 * (every grid value and the rounding constants of its binades are normal FP32
 * numbers); anything else is FPQ_ERR_FORMAT.
 * `scale` is the real value of one unit of the code domain: real = scale *
 * value(code).  It plays the role of the paper's real-valued exponent bias:
 * b_paper = exp_bias - log2(scale).
 */
#ifndef FPQ_H
#define FPQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t fpq_status;

enum {
    FPQ_OK = 0,
    FPQ_ERR_NULL = -1,        /* a required pointer is NULL */
    FPQ_ERR_FORMAT = -2,      /* impossible (exp_bits, man_bits, exp_bias, sat_mode) */
    FPQ_ERR_SHAPE = -3,       /* negative / overflowing / inconsistent sizes */
    FPQ_ERR_ALIGN = -4,       /* pointer not aligned as documented */
    FPQ_ERR_UNSUPPORTED = -5, /* operand formats the contraction has no path for */
    FPQ_ERR_WORKSPACE = -6,   /* workspace missing or too small */
    FPQ_ERR_CUDA = -7,        /* a CUDA runtime / driver call failed */
    FPQ_ERR_TIMEOUT = -8,     /* a bounded device-side wait expired (device status) */
    FPQ_ERR_NAN_INPUT = -9,   /* a NaN was quantized (to code 0) (device status) */
    FPQ_ERR_TOO_LARGE = -10,  /* problem exceeds a fixed built-in capacity */
    FPQ_ERR_SCALE = -11       /* an activation scale is zero, negative, infinite or NaN */
};

enum { FPQ_SAT_PAPER = 0, FPQ_SAT_NATIVE = 1 };

/*
 * sat_mode selects the clipping value c (Sec. IV-B, c = (2 - 2^-m) 2^(2^e - b - 1)):
 *   FPQ_SAT_PAPER   every exponent field is finite, c as printed;
 *   FPQ_SAT_NATIVE  c is lowered to the largest finite value of the OCP FP8 type
 *                   with the same (e, m): E4M3 -> 1.75 * 2^(15-b) (448 at b = 7),
 *                   E5M2 -> 1.75 * 2^(30-b); the reserved codes are never
 *                   produced.  Other (e, m) are unaffected.
 */
typedef struct {
    int32_t exp_bits, man_bits, exp_bias, sat_mode;
} fpq_format;

enum { FPQ_LINEAR = 0, FPQ_CONV2D = 1 };

/* What a weight tensor belongs to.  Linear: [N][K] (C = K, R = S = 1).
 * Conv: [N][C][R][S], K = C*R*S. */
typedef struct {
    int32_t kind;
    int32_t N, C, R, S;
} fpq_layer_desc;

/* scale = maxabs / c(fmt), one FP32 division.  Host function. */
float fpq_scale_from_max(float maxabs, fpq_format fmt);

/* Clipping value c of a format (host function; 0 if the format is invalid). */
float fpq_format_max(fpq_format fmt);

/*
 * Weight encode (offline, once per layer).  For each weight: t = w * (1.0f /
 * scale[n]) in FP32, clip to +-c, then
 *   rounding_bits == NULL : round to nearest on the element's own step, ties to
 *                           even (Sec. IV-B, rounding equation and step equation);
 *   rounding_bits != NULL : floor(t / s) + h on the signed value, h the weight's
 *                           bit, then clamp (Sec. V-B, learned rounding with the
 *                           decision hardened to 0 / 1 as at inference).
 * w            [N][K] row-major FP32 (conv weights pass K = C*R*S in [C][R][S] order)
 * scale        [N] FP32, one per output channel (per-tensor = N equal entries)
 * rounding_bits 1 bit per weight, LSB first along K, each row padded to a byte:
 *              [N][ceil(K/8)]
 * codes (out)  [N][K] bytes, or [N][ceil(K/2)] for formats of <= 4 bits
 * Zero results are always code 0.  NaN -> code 0 and FPQ_ERR_NAN_INPUT in the
 * device status word.  +-Inf -> +-c.
 */
fpq_status fpq_quantize_weight(const float* w, int64_t N, int64_t K, const float* scale,
                               fpq_format fmt, const uint8_t* rounding_bits, uint8_t* codes,
                               void* stream);

/*
 * Activation quantize, standalone form (Sec. IV-B; one static per-tensor scale,
 * Sec. VI-A).  x: n FP32 values; codes (out): n bytes (ceil(n/2) for <= 4 bits).
 * Round to nearest, ties to even.
 */
fpq_status fpq_quantize_act(const float* x, int64_t n, float scale, fpq_format fmt, uint8_t* codes,
                            void* stream);

/*
 * Contraction-ready copy of encoded weights.  `codes` is the output of
 * fpq_quantize_weight for the layer `d`; `prepared` must hold
 * fpq_prepared_size(fmt, d) bytes and be 128-byte aligned.  The layout is
 * internal: rows of C padded with zero codes to a multiple of 128, taps
 * outermost within a row ([N][R*S][C_pad]).  May be saved and reloaded as bytes.
 * E4M3 (bias 7, FPQ_SAT_NATIVE), E5M2 (bias 15, FPQ_SAT_NATIVE) and E2M1 (bias 1) codes are
 * kept as they are (E2M1 two per byte).  Any other format whose every value is also a finite E4M3 value - E1M2 with bias 1,
 * E2M1 with bias 2, small formats such as E3M2 bias 3 or E2M3 bias 1 - is re-encoded here,
 * exactly, into one E4M3 byte per weight.  A format whose every value is the sum of two finite
 * E4M3 values (the largest E4M3 magnitude not above it, and the rest: E3M4 bias 4, E2M5 bias 2,
 * E4M3 bias 7 with all exponent fields finite, where 480 = 448 + 32; and, after a factor 2^k that
 * the layer's dequantization takes back exactly, formats such as the paper's default E4M3 with
 * bias 8) is prepared as those two terms, two bytes per weight ([N][R*S][2 C_pad]); fpq_linear /
 * fpq_conv2d then contract over twice the reduction length on the tensor cores - exact products,
 * FP32 sums, as for one term.  The paper's E5M2 (bias 16, all exponent fields finite) is prepared
 * the same way as two terms of the tensor cores' own E5M2.  Every other format (beyond two such
 * terms, e.g. 6 exponent bits) is copied unchanged and takes the FP32 grid-value route of the layer calls.
 */
size_t fpq_prepared_size(fpq_format fmt, const fpq_layer_desc* d);
fpq_status fpq_prepare_weight(const uint8_t* codes, fpq_format fmt, const fpq_layer_desc* d,
                              void* prepared, void* stream);

/*
 * Quantized linear layer (Sec. V-B, Y = W A, and Sec. VI-A):
 *   y[i][n] = (x_scale * w_scale[n]) * sum_k value(q(x[i][k])) * value(wq[n][k]) + bias[n]
 * x FP32 [M][K] row-major, y FP32 [M][N] row-major, both 16-byte aligned; bias
 * [N] or NULL.  The activations are quantized with (fx, x_scale) exactly as
 * fpq_quantize_act does; products are exact and accumulated in FP32 on the
 * tensor cores (layers of at most 8 rows with K a multiple of 4 run on the CUDA
 * cores instead: the same exact products, another order of the FP32 additions;
 * the workspace is then left untouched).  Supported operand pairs: fx = E4M3 bias 7 FPQ_SAT_NATIVE or
 * fx = E5M2 bias 15 FPQ_SAT_NATIVE (the two 8-bit types the tensor cores read; Sec. V-A searches the
 * activation encodings too) with
 * fw = E4M3 bias 7 FPQ_SAT_NATIVE, fw = E5M2 bias 15 FPQ_SAT_NATIVE, fw = E2M1 bias 1, or any fw that fpq_prepare_weight
 * re-encodes exactly into one or two terms of those types (see there) run on the tensor cores.  An activation
 * format fx whose every value is one value or the sum of two values of such a type (the same classification:
 * E3M4 bias 4, E2M5 bias 2, E4M3 with all exponent fields finite, the small formats inside E4M3) with a weight
 * format that is read directly or re-encoded into one term runs there too: the activations are quantized with the
 * general arithmetic, written as [first terms | second terms], and contracted over twice the reduction length
 * against the weights repeated (a copy in the workspace, which must then be 256-byte aligned).  Every other valid
 * pair (any fx, any fw) works on FP32 grid values: activations quantized to their grid values in FP32, weights
 * decoded to FP32, one FP32 contraction (on the tensor cores as exact TF32 products when K is a multiple of 4,
 * else FP32 multiply-adds on the CUDA cores) - the same arithmetic model (exact products, FP32 sums) at roughly a
 * third of the speed; the workspace is then FP32 scratch (fpq_linear_workspace_size says how much) and must be
 * 256-byte aligned.
 * This holds for fpq_linear and fpq_conv2d and their host-buffer forms (and for fpq_linear_static as far as
 * its fixed scratch reaches: FPQ_ERR_WORKSPACE beyond); the staged (quantize_input / contract) and two-tensor
 * forms take only the pairs the tensor cores read directly or after the one-term re-encode, and return
 * FPQ_ERR_UNSUPPORTED otherwise.
 * workspace: fpq_linear_workspace_size bytes, 128-byte aligned; contents are
 * scratch.
 */
size_t fpq_linear_workspace_size(int64_t M, int64_t N, int64_t K, fpq_format fx, fpq_format fw);
fpq_status fpq_linear(const float* x, const void* w_prepared, const float* w_scale, float x_scale,
                      fpq_format fx, fpq_format fw, const float* bias, float* y, int64_t M,
                      int64_t N, int64_t K, void* workspace, size_t ws_bytes, void* stream);

/*
 * Quantized 2-D convolution (cross-correlation, zero padding, square stride):
 * x FP32 NCHW [B][C][H][W], y FP32 NCHW [B][C_out][H_out][W_out],
 * H_out = (H + 2 pad - R) / stride + 1.  Same arithmetic as fpq_linear with
 * k running over (c, r, s); padding contributes code 0.
 */
size_t fpq_conv2d_workspace_size(int B, int C, int H, int W, int C_out, int R, int S, int pad,
                                 int stride, fpq_format fx, fpq_format fw);
fpq_status fpq_conv2d(const float* x, const void* w_prepared, const float* w_scale, float x_scale,
                      fpq_format fx, fpq_format fw, const float* bias, float* y, int B, int C, int H,
                      int W, int C_out, int R, int S, int pad, int stride, void* workspace,
                      size_t ws_bytes, void* stream);

/*
 * The two stages of fpq_linear / fpq_conv2d as separate calls (the layer call
 * is exactly stage 1 followed by stage 2 on the same stream):
 *   stage 1, *_quantize_input: activation quantize (Sec. IV-B rounding equation,
 *            static per-tensor scale) written to `workspace` in the operand
 *            layout of the contraction (linear: [M][K rounded up to 16] codes;
 *            conv: channels-last codes with the zero padding frame materialised,
 *            [B][H + 2 pad][W + 2 pad][C rounded up to 16]);
 *   stage 2, *_contract: the low-bit contraction on those codes and the
 *            dequantize + bias epilogue (Sec. V-B, Y = W A; Sec. VI-A).
 * Arguments, alignment rules and errors are those of the layer calls.
 */
fpq_status fpq_linear_quantize_input(const float* x, float x_scale, fpq_format fx, fpq_format fw,
                                     int64_t M, int64_t N, int64_t K, void* workspace,
                                     size_t ws_bytes, void* stream);
fpq_status fpq_linear_contract(const void* workspace, size_t ws_bytes, const void* w_prepared,
                               const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                               const float* bias, float* y, int64_t M, int64_t N, int64_t K,
                               void* stream);
fpq_status fpq_conv2d_quantize_input(const float* x, float x_scale, fpq_format fx, fpq_format fw,
                                     int B, int C, int H, int W, int C_out, int R, int S, int pad,
                                     int stride, void* workspace, size_t ws_bytes, void* stream);
fpq_status fpq_conv2d_contract(const void* workspace, size_t ws_bytes, const void* w_prepared,
                               const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                               const float* bias, float* y, int B, int C, int H, int W, int C_out,
                               int R, int S, int pad, int stride, void* stream);

/*
 * Host-buffer forms of the two layers: x_host / y_host are host pointers
 * (pinned memory for asynchronous copies), x_dev / y_dev are device staging
 * buffers of the same sizes owned by the caller.  The call copies x in, runs the
 * layer, copies y out and returns when y_host is complete.  Large batches are
 * pipelined in up to 8 slices (rows / images) so that the copy-in of one slice,
 * the layer on the previous one and the copy-out of the one before overlap; the
 * result is the same bit for bit.  For this the library keeps two streams and a
 * few events per device, created at the first host-form call (the one exception
 * to "allocates nothing"); host-form calls on one device must not run concurrently.
 * A linear layer is sliced only if K and N are multiples of 4 (slices of x and y
 * must keep fpq_linear's 16-byte alignment).
 */
fpq_status fpq_linear_host(const float* x_host, float* x_dev, const void* w_prepared,
                           const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                           const float* bias, float* y_dev, float* y_host, int64_t M, int64_t N,
                           int64_t K, void* workspace, size_t ws_bytes, void* stream);
fpq_status fpq_conv2d_host(const float* x_host, float* x_dev, const void* w_prepared,
                           const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                           const float* bias, float* y_dev, float* y_host, int B, int C, int H,
                           int W, int C_out, int R, int S, int pad, int stride, void* workspace,
                           size_t ws_bytes, void* stream);

/*
 * fpq_linear without a workspace argument.  (The paper has no counterpart: this
 * entry point exists for integration reasons only.)
 *
 * Who it is for: code that runs where device memory cannot be requested - a
 * plug-in called on someone else's stream that must not trigger the implicit
 * device-wide synchronisation of cudaMalloc / cudaFree, a latency-critical
 * serving loop whose memory was handed out once at start-up, or a host that
 * gives the library no allocator at all.  Such a caller still owns x, y and the
 * weights, but has nowhere to put the intermediate activation codes that
 * fpq_linear writes to its `workspace`.
 *
 * Here those codes go to a fixed array inside the library image, of
 * FPQ_STATIC_SCRATCH_BYTES bytes, which every GPU that loads the library keeps
 * resident until the process ends.  The call makes no cudaMalloc, cudaFree or
 * other allocating call.  Results are identical to fpq_linear's.
 *
 *   - Limit: M * (K rounded up to 16) <= FPQ_STATIC_SCRATCH_BYTES, otherwise
 *     FPQ_ERR_TOO_LARGE and nothing is launched.  All other arguments, alignment
 *     rules and errors are fpq_linear's.
 *   - The first call on each device looks up the array's device address (with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps whatever the last call
 *     left in it; each call overwrites every byte it later reads, so stale
 *     contents are harmless, but two calls that overlap on the GPU (different
 *     streams, or host threads launching concurrently) race on it.  Serialise
 *     them on one stream.
 */
#define FPQ_STATIC_SCRATCH_BYTES (8u << 20)
fpq_status fpq_linear_static(const float* x, const void* w_prepared, const float* w_scale,
                             float x_scale, fpq_format fx, fpq_format fw, const float* bias,
                             float* y, int64_t M, int64_t N, int64_t K, void* stream);

/*
 * Convolution whose input is the channel concatenation of two tensors that are quantized
 * separately, each with its own scale (Sec. VI-A: the skip connection and the previous layer's
 * output of a decoder block have different value distributions and are quantized apart before
 * they are concatenated):
 *   y[b][n][oy][ox] = w_scale[n] * ( x1_scale * sum over the C1 channels of x1
 *                                  + x2_scale * sum over the C2 channels of x2 ) + bias[n]
 * with the sums as in fpq_conv2d.  x1 is NCHW [B][C1][H][W], x2 is [B][C2][H][W]; the
 * concatenated FP32 tensor is never formed.  The weights are [C_out][C1 + C2][R][S] codes from
 * fpq_quantize_weight (x1's channels first), passed through fpq_prepare_weight_split (buffer of
 * fpq_prepared_size_split bytes, 128-byte aligned): that copy starts x2's channels at a multiple
 * of 128 so that no 128-wide chunk of the reduction mixes the two scales.
 * workspace: fpq_conv2d_split_workspace_size bytes, 128-byte aligned, scratch.
 * Formats, alignment, errors and stream behaviour as fpq_conv2d (three kernels).
 */
size_t fpq_prepared_size_split(fpq_format fmt, int32_t N, int32_t C1, int32_t C2, int32_t R, int32_t S);
fpq_status fpq_prepare_weight_split(const uint8_t* codes, fpq_format fmt, int32_t N, int32_t C1, int32_t C2,
                                    int32_t R, int32_t S, void* prepared, void* stream);
size_t fpq_conv2d_split_workspace_size(int B, int C1, int C2, int H, int W, int C_out, int R, int S, int pad,
                                       int stride, fpq_format fx, fpq_format fw);
fpq_status fpq_conv2d_split(const float* x1, int C1, float x1_scale, const float* x2, int C2, float x2_scale,
                            const void* w_prepared, const float* w_scale, fpq_format fx, fpq_format fw,
                            const float* bias, float* y, int B, int H, int W, int C_out, int R, int S, int pad,
                            int stride, void* workspace, size_t ws_bytes, void* stream);

/*
 * Zero census of a quantized tensor (the sparsity measurement of the paper's evaluation, Sec.
 * "Sparsity": the fraction of weights that are zero after quantization).  Counts the values of
 * `codes` whose code is 0; the quantizers never produce a negative zero, so this is every zero.
 *   codes   n codes as written by fpq_quantize_weight / fpq_quantize_act: one per byte, or for
 *           formats of at most 4 bits two per byte, even index in the low nibble (a high nibble
 *           of padding after an odd n is not counted)
 *   count   DEVICE out, one uint64 (8-byte aligned), overwritten
 * One memset and one kernel on `stream`.  Errors: FPQ_ERR_FORMAT, FPQ_ERR_SHAPE (n < 0),
 * FPQ_ERR_NULL, FPQ_ERR_ALIGN, FPQ_ERR_CUDA.
 */
fpq_status fpq_zero_census(const uint8_t* codes, int64_t n, fpq_format fmt, uint64_t* count, void* stream);

/*
 * Encoding and bias search of one tensor (Sec. V-A, Algorithm 1; offline, once per weight or
 * activation tensor).  For every encoding candidate enc_host[i] (exponent and mantissa bits; the
 * integer exp_bias only fixes the unit, sat_mode must be FPQ_SAT_PAPER) and every clipping value
 * clip[j] > 0 the tensor is quantized, round to nearest even, with the format whose largest value
 * is clip[j] - that is with scale = clip[j] / fpq_format_max(enc_host[i]) (FP32 division), which
 * is the real-valued bias b = exp_bias - log2(scale) of the clipping equation (Sec. IV-B) - and
 *   mse[i * n_clip + j] = (1/n) sum_k (x[k] - scale * q(x[k] / scale))^2.
 * best[0], best[1] receive the encoding and clipping index that Algorithm 1 selects: candidates
 * are visited encoding by encoding, clipping values in the inner loop, and one replaces the best
 * so far only if its error is strictly smaller (the best so far starts at +infinity).
 *
 *   x          n FP32 values (n >= 0); a NaN makes every mse NaN and sets FPQ_ERR_NAN_INPUT in
 *              the status word
 *   enc_host   HOST array of n_enc formats, 1 <= n_enc <= 8
 *   clip       DEVICE array of n_clip positive finite FP32 values, 1 <= n_clip <= 256,
 *              n_enc * n_clip <= 1024 (the paper uses 4 x 111 for FP8 and 2 x 111 for FP4)
 *   mse        DEVICE out, n_enc * n_clip doubles
 *   best       DEVICE out, 2 int32
 *   workspace  fpq_search_workspace_size(n_enc, n_clip) bytes, 8-byte aligned; contents need
 *              not be kept between calls
 * Three kernels on `stream`, no allocation, no host synchronisation.  Errors: FPQ_ERR_NULL,
 * FPQ_ERR_SHAPE (counts out of range, n < 0), FPQ_ERR_FORMAT, FPQ_ERR_UNSUPPORTED (sat_mode),
 * FPQ_ERR_ALIGN, FPQ_ERR_WORKSPACE, FPQ_ERR_CUDA.
 */
size_t fpq_search_workspace_size(int32_t n_enc, int32_t n_clip);
fpq_status fpq_search_format(const float* x, int64_t n, const fpq_format* enc_host, int32_t n_enc, const float* clip,
                             int32_t n_clip, double* mse, int32_t* best, void* workspace, size_t ws_bytes,
                             void* stream);

/*
 * The clipping candidates of Sec. V-A: count evenly spaced values up to the largest magnitude
 * of the data, clip_host[j] = maxabs * (j + 1) / count rounded once to FP32 (zero is left out:
 * no format has a largest value of 0).  HOST output.  FPQ_ERR_SHAPE unless 1 <= count <= 256
 * and maxabs is positive and finite.
 */
fpq_status fpq_search_clip_candidates(float maxabs, int32_t count, float* clip_host);

/*
 * Rounding learning (Sec. V-B): one evaluation of the objective and of its gradient for the weights
 * of a bias-free linear layer (the paper's own example; a convolution is the same call on its
 * unfolded input rows).  With sigma(t) = 1 / (1 + exp(-t)), gamma = scale[n] and, per weight,
 * a = clamp(w * (1.0f / gamma); -c, c), s = the grid step of a's binade (Sec. IV-B step equation):
 *     Wq(alpha)  = gamma * clamp(s * (floor(a / s) + sigma(alpha)); -c, c)      learned-rounding equation
 *     mse        = mean over [M][N] of (A Wq^T - A W^T)^2                        layer-output error
 *     lambda     = 1 - (2 |sigma(alpha) - 0.5|)^20                               regulariser, per weight
 *     objective  = mse + reg * sum of lambda over all weights
 *     grad       = d objective / d alpha  (floor has zero derivative; a clamp passes the derivative
 *                  inside [-c, c] and blocks it outside)
 * The paper prints "+ lambda(alpha)" without saying how the per-weight terms combine or how they
 * are weighted: they are summed and the caller gives the weight `reg`.  The activations are used as
 * given (FP32, the same on both sides of the difference, as in the paper's equations).
 * Everything is computed at FP32 accuracy, the precision the method is stated in.  The two
 * contractions (A (Wq - W)^T, which is A Wq^T - A W^T by linearity, and its transpose product with A)
 * run on the tensor cores when K is a multiple of 4 and `a` is 16-byte aligned: every FP32 product as
 * the sum of three TF32 products of exact operand splits, the reduction added up in FP32 (errors of a
 * few 1e-6 of the sum of absolute terms); otherwise they are FP32 multiply-adds on the CUDA cores.
 * The sums of squares and of lambda are accumulated in double.
 *   w       [N][K] FP32 weights, scale [N] (as fpq_quantize_weight)
 *   fmt     weight format (any valid format; the paper learns rounding for FP4 only)
 *   alpha   [N][K] FP32, read; overwritten by alpha - lr * grad when lr != 0 (plain gradient descent)
 *   a       [M][K] FP32 calibration activations, row-major
 *   reg,lr  finite
 *   grad    out, [N][K] FP32
 *   loss    out, 2 doubles (8-byte aligned): {mse, sum of lambda}
 *   workspace  fpq_round_learn_workspace_size(M, N, K) bytes, 256-byte aligned, contents not kept
 * One memset and four to seven kernels on `stream`; no allocation, no host synchronisation.  A NaN weight
 * contributes nothing and sets FPQ_ERR_NAN_INPUT in the device status.  Limits: 1 <= M < 2^31 - 128,
 * 1 <= N, K <= 65535 * 128, N * K < 2^40.  Errors: FPQ_ERR_FORMAT, FPQ_ERR_SHAPE, FPQ_ERR_NULL,
 * FPQ_ERR_ALIGN, FPQ_ERR_WORKSPACE, FPQ_ERR_CUDA.  The workspace size is 0 for shapes out of range.
 */
size_t fpq_round_learn_workspace_size(int64_t M, int64_t N, int64_t K);
fpq_status fpq_round_learn_step(const float* w, const float* scale, fpq_format fmt, float* alpha, const float* a,
                                int64_t M, int64_t N, int64_t K, float reg, float lr, float* grad, double* loss,
                                void* workspace, size_t ws_bytes, void* stream);

/*
 * Rounding learning for a convolution (Sec. V-B: the method also applies to convolutional layers): writes
 * the convolution's input rows out, so that fpq_round_learn_step on `rows` and the weights flattened to
 * [C_out][C*R*S] (the layout fpq_quantize_weight takes) is the step for the convolution.
 *   x     FP32 NCHW [B][C][H][W]
 *   rows  out, FP32 [B*H_out*W_out][C*R*S]: row (b, oy, ox), column (c, r, s) =
 *         x[b][c][oy*stride - pad + r][ox*stride - pad + s], 0 in the padding;
 *         H_out = (H + 2 pad - R) / stride + 1, likewise W_out
 * One kernel on `stream`.  Errors: FPQ_ERR_SHAPE (sizes out of range, window larger than the padded
 * input, R or S above 64), FPQ_ERR_NULL, FPQ_ERR_ALIGN, FPQ_ERR_CUDA.
 */
fpq_status fpq_round_learn_unfold(const float* x, int32_t B, int32_t C, int32_t H, int32_t W, int32_t R, int32_t S,
                                  int32_t pad, int32_t stride, float* rows, void* stream);

/*
 * The inference rule of Sec. V-B: sigma(alpha) < 0.5 rounds down, sigma(alpha) >= 0.5 rounds up, i.e.
 * decision bit = (alpha >= 0).  Writes the bits in the layout fpq_quantize_weight reads (1 bit per
 * weight, LSB first along K, every row padded to a whole byte; padding bits are 0).
 *   alpha [N][K] FP32; rounding_bits out, N * ceil(K / 8) bytes.  One kernel on `stream`.
 * Errors: FPQ_ERR_SHAPE, FPQ_ERR_NULL, FPQ_ERR_ALIGN, FPQ_ERR_CUDA.
 */
fpq_status fpq_round_learn_harden(const float* alpha, int64_t N, int64_t K, uint8_t* rounding_bits, void* stream);

/*
 * Which route fpq_linear / fpq_conv2d take (process-wide setting, not thread-safe against
 * concurrent layer calls).  Every route multiplies the same codes exactly and adds in FP32, so the
 * results agree within the layer tolerance; routes that run the same MMAs in the same order agree
 * bit for bit.
 *   FPQ_PATH_FUSED        one kernel: the activation quantize (Sec. IV-B rounding equation) runs
 *                         inside the contraction's operand staging, the codes never reach global
 *                         memory (the layer of Sec. VI-A as one pass: FP32 in -> quantize -> low-bit
 *                         MAC -> FP32 out).  Stride-1 convolutions whose whole weight tensor fits in
 *                         the shared memory of a pair of SMs run on CTA pairs (tcgen05 cta_group::2);
 *                         linear layers and the other stride-1 convolutions use the general fused
 *                         form; other geometries fall back to two kernels.
 *   FPQ_PATH_TWO_KERNELS  always *_quantize_input followed by *_contract.
 *   FPQ_PATH_TWO_KERNELS_NARROW  the same, and the contraction never takes its CTA-pair form (M = 256
 *                         MMAs for long reductions with many tiles): for measurements and tests.
 *   FPQ_PATH_AUTO         the library's choice per shape (default): the CTA-pair kernel where it
 *                         applies and measured faster, else two kernels.
 */
enum { FPQ_PATH_AUTO = 0, FPQ_PATH_FUSED = 1, FPQ_PATH_TWO_KERNELS = 2, FPQ_PATH_TWO_KERNELS_NARROW = 3 };
fpq_status fpq_set_path_policy(int32_t policy);
int32_t fpq_get_path_policy(void);

/*
 * Which kernels fpq_conv2d would run for this shape under the current policy, for logs and
 * benchmarks (pointer alignment is assumed to be as documented; nothing is launched):
 *   FPQ_ROUTE_TWO_KERNELS  activation-quantize kernel, then the contraction kernel;
 *   FPQ_ROUTE_FUSED        the general one-kernel form;
 *   FPQ_ROUTE_PAIR_FUSED   the one-kernel form on CTA pairs with resident weights;
 *   FPQ_ROUTE_OTHER        operand formats that are not read as they are: weights or activations as one or two
 *                          terms of a tensor-core type, or the FP32 grid-value route;
 *   negative               the error fpq_conv2d would return for these arguments.
 */
enum { FPQ_ROUTE_TWO_KERNELS = 0, FPQ_ROUTE_FUSED = 1, FPQ_ROUTE_PAIR_FUSED = 2, FPQ_ROUTE_OTHER = 3 };
int32_t fpq_conv2d_route(int B, int C, int H, int W, int C_out, int R, int S, int pad, int stride,
                         fpq_format fx, fpq_format fw);

/*
 * Diagnostic (the paper has no counterpart): launches one warp that waits on a barrier nobody ever
 * arrives on, with the same bounded wait every role of the layer kernels uses, limited to
 * limit_cycles SM clock cycles (1 .. 1e9).  The wait runs out, the warp records FPQ_ERR_TIMEOUT in the
 * device status word and the kernel returns: the context stays usable, which is what a caller's
 * failure handling relies on.  Returns FPQ_OK when the kernel was enqueued (the time-out shows in
 * fpq_read_status), FPQ_ERR_SHAPE for a limit out of range, FPQ_ERR_CUDA.
 */
fpq_status fpq_selftest_bounded_wait(int64_t limit_cycles, void* stream);

/* Waits for `stream`, then returns and clears the sticky device status word:
 * FPQ_OK, FPQ_ERR_TIMEOUT, FPQ_ERR_NAN_INPUT, or FPQ_ERR_CUDA.  The word keeps one bit per kind of
 * event; when both have happened FPQ_ERR_TIMEOUT (an incomplete output) is the one reported. */
fpq_status fpq_read_status(void* stream);

const char* fpq_status_string(fpq_status s);

#ifdef __cplusplus
}
#endif
#endif /* FPQ_H */
