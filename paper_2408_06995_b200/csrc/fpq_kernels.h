// Internal launch interface between the translation units of the fpq library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fpq_common.cuh"

namespace fpq {

cudaError_t launch_quantize_act(const float* x, int64_t n, float scale, const QFormat& f, uint8_t* codes,
                                cudaStream_t st);
cudaError_t launch_quantize_weight(const float* w, int64_t N, int64_t K, const float* scale, const QFormat& f,
                                   const uint8_t* rbits, uint8_t* codes, cudaStream_t st);
// (e5m2 != 0: the codes are OCP E5M2 instead of E4M3, the tensor cores' other 8-bit activation type)
cudaError_t launch_quantize_rows_e4m3(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, uint8_t* codes,
                                      cudaStream_t st, int e5m2 = 0);
cudaError_t launch_quantize_nchw_to_nhwc_e4m3(const float* x, int B, int C, int H, int W, int pad, int Cp, int row,
                                              int c_off, float scale, uint8_t* codes, cudaStream_t st, int e5m2 = 0);
cudaError_t launch_zero_census(const uint8_t* codes, int64_t n, int four_bit, unsigned long long* count, cudaStream_t st);
// Code-to-code table of an exact re-encode (weight format -> E4M3), passed to the kernel by value.
struct CodeTable {
    uint8_t t[256];
};
// table != NULL: every code is looked up and the prepared copy holds one byte per weight.  table2 != NULL as
// well: Cp counts two halves per row, the first filled through table, the second through table2.
cudaError_t launch_prepare_weight(const uint8_t* codes, int N, int C, int RS, int Cp, int four_bit, int C1, int C1p,
                                  const CodeTable* table, const CodeTable* table2, uint8_t* prepared, cudaStream_t st);
// Activations of a format that is one term or the sum of two terms of a tensor-core type: general quantizer, then
// the tables (t2 == NULL: one term).  Rows / pixels hold [first terms | second terms], Kp (Cp) positions each.
cudaError_t launch_quantize_rows_terms(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, const QFormat& f,
                                       const CodeTable& t1, const CodeTable* t2, uint8_t* codes, cudaStream_t st);
cudaError_t launch_quantize_nchw_to_nhwc_terms(const float* x, int B, int C, int H, int W, int pad, int Cp, float scale,
                                               const QFormat& f, const CodeTable& t1, const CodeTable* t2, uint8_t* codes,
                                               cudaStream_t st);
// every row of src [rows][row_bytes] (row_bytes a multiple of 16) twice side by side in dst [rows][2 * row_bytes]
cudaError_t launch_repeat_rows(const void* src, int64_t rows, int64_t row_bytes, void* dst, cudaStream_t st);
cudaError_t launch_quantize_rows_e4m3_twice(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, uint8_t* codes,
                                            cudaStream_t st, int e5m2 = 0);

// One warp waits, with the kernels' own bounded wait, on a barrier nobody arrives on: after `limit` cycles it
// records FPQ_ERR_TIMEOUT in the status word and returns (nothing hangs, nothing faults).
cudaError_t launch_bounded_wait_selftest(long long limit, int* status, cudaStream_t st);

// Geometry of one contraction launch (linear: taps = 1, rows of Ca codes).
struct GemmProblem {
    int conv;            // 0 linear, 1 conv
    int after_stage1;    // launched right behind this library's own activation-quantize kernel
    int w4;              // weights are E2M1
    int w_e5m2;          // weights are E5M2 (bias 15, native saturation): the tensor cores' second 8-bit type
    int a_e5m2;          // activation codes are E5M2 (bias 15, native saturation) instead of E4M3
    int64_t M;           // linear rows
    int N;               // outputs / out channels
    int Cp;              // padded reduction length per tap in the weight copy (multiple of 128)
    int Ca;              // padded channels (row length) of the activation codes (multiple of 16)
    int B, H, W, Ho, Wo; // conv geometry
    int R, S, pad, stride;
    const uint8_t* a_codes;   // [M][Ca] or framed [B][Hp][Wp][Ca]; unused by the fused form
    const float* x;           // fused form: FP32 activations ([M][C] or NCHW); NULL = read a_codes
    int C;                    // fused form: channels / reduction length of x
    const void* w_prepared;   // [N][R*S][Cp]
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
    // input made of two concatenated tensors with their own scales: the first c_seg 128-wide chunks
    // of the reduction belong to the first tensor (x_scale), the rest to the second (x_scale2); 0 = one tensor
    int c_seg;
    float x_scale2;
};

// Returns FPQ_OK or an error; enqueues one kernel.
fpq_status launch_gemm(const GemmProblem& p, cudaStream_t st);

// Stride-1 convolution from FP32 NCHW activations (p.x) in one kernel on CTA pairs, weights resident in
// shared memory.  FPQ_ERR_UNSUPPORTED when the shape is outside its range (nothing was enqueued).
fpq_status launch_pair_conv(const GemmProblem& p, cudaStream_t st);
bool pair_conv_applies(const GemmProblem& p);     // p.x only has to be non-NULL and 16-byte aligned
bool pair_conv_preferred(const GemmProblem& p);   // ... and it measured faster than the two-kernel route on shapes like this

// The contraction of a stride-1 convolution (activation codes already in the workspace) on CTA pairs with
// M = 256 MMAs.  FPQ_ERR_UNSUPPORTED when the shape is outside its range (nothing was enqueued).
fpq_status launch_pair_gemm(const GemmProblem& p, cudaStream_t st);
bool pair_gemm_preferred(const GemmProblem& p);   // in range, and faster than the general contraction on shapes like this

// Linear layer with at most 8 rows on the CUDA cores (one pass over the weights).
bool small_m_linear_applies(int64_t M, int64_t K);
fpq_status launch_small_m_linear(const float* x, int M, int K, const void* w_prepared, int w4, int N, const float* w_scale,
                                 float x_scale, const float* bias, float* y, cudaStream_t st);

// Encoding / bias search: limits, scratch size, and the launch (three kernels).
int search_max_enc();
int search_max_clip();
int search_max_cand();
size_t search_workspace_bytes(int n_enc, int n_clip);
fpq_status launch_search(const float* x, int64_t n, const fpq_format* enc, int n_enc, const float* clip, int n_clip,
                         double* mse, int32_t* best, void* workspace, cudaStream_t st);

// Rounding learning (Sec. V-B): scratch size, one objective + gradient evaluation (a memset and four kernels),
// and the hardening of alpha into decision bits.
size_t round_learn_workspace_bytes(int64_t M, int64_t N, int64_t K);
fpq_status launch_round_learn(const float* w, const float* scale, const QFormat& f, float* alpha, const float* a,
                              int64_t M, int64_t N, int64_t K, float reg, float lr, float* grad, double* loss,
                              void* workspace, cudaStream_t st);
fpq_status launch_unfold(const float* x, int B, int C, int H, int W, int R, int S, int pad, int stride, int Ho, int Wo,
                         float* rows, cudaStream_t st);
fpq_status launch_sgemm_nt(const float* P, int64_t ldp, const float* Q, int64_t ldq, float* C, int64_t ldc, int64_t I,
                           int64_t J, int64_t R, cudaStream_t st);
fpq_status launch_round_harden(const float* alpha, int64_t N, int64_t K, uint8_t* bits, cudaStream_t st);

// C = P Q^T in FP32 on the tensor cores (three TF32 products per term): P [I][ldp], Q [J][ldq], reduction of
// length R contiguous in both, cut into slices of kb_per_split 32-wide blocks.  epi 0: slice z is written to
// C + z * split_stride, row-major [I][ldc]; epi 1 (one slice): C[j][i] (leading dimension ldc) and *sq_sum +=
// the sum of the squared outputs.  passes = 1: the operands hold TF32 numbers (at most 11 significant bits) and one
// product per term is exact.  epi 2 (one slice): C is the layer's output, sum * (x_scale * w_scale[j]) + bias[j], row-major
// [I][ldc] (howo = 0) or NCHW with i = image * howo + pixel.  FPQ_ERR_UNSUPPORTED (nothing enqueued) unless tf32x3_applies.
bool tf32x3_applies(const float* P, int64_t ldp, const float* Q, int64_t ldq, int64_t I, int64_t J, int64_t R);
fpq_status launch_tf32x3(const float* P, int64_t ldp, const float* Q, int64_t ldq, int64_t I, int64_t J, int64_t R,
                         int kb_per_split, int epi, float* C, int64_t ldc, int64_t split_stride, double* sq_sum,
                         cudaStream_t st, int passes = 3, const float* w_scale = nullptr, float x_scale = 1.0f,
                         const float* bias = nullptr, int howo = 0);
// XT[k][m] = X[m][k] for X [M][K] with leading dimension ldx, XT with leading dimension ldt
cudaError_t launch_transpose(const float* X, int64_t ldx, int64_t M, int64_t K, float* XT, int64_t ldt, cudaStream_t st);

// Layer on the CUDA cores for operand formats the tensor-core contraction has no type for (any valid pair):
// activations quantized to their grid values in FP32, weight codes decoded to FP32, FP32 multiply-add
// contraction (exact products, FP32 sums, as on the tensor cores), dequantize + bias.
struct GeneralLayer {
    int conv;                 // 0 linear ([M][K] rows), 1 convolution (NCHW)
    int64_t M, N, K;          // K = C * R * S for a convolution
    int B, C, H, W, R, S, pad, stride, Ho, Wo;
    QFormat fx, fw;           // fw: the format of the codes in the prepared copy
    int Cp;                   // padded channels of the prepared copy ([N][R*S][Cp])
    int w_two_term;           // the prepared copy holds two E4M3 terms per weight ([N][R*S][2 Cp])
    float w_mul;              // power of two the sum of the two terms is multiplied by (1 unless w_two_term)
    const float* x;
    const void* w_prepared;
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
};
size_t general_layer_workspace_bytes(const GeneralLayer& g);
fpq_status launch_general_layer(const GeneralLayer& g, void* workspace, cudaStream_t st);

}  // namespace fpq
