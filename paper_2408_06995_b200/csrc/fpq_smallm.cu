// Quantized linear layer with a handful of rows (the time-embedding projections of a
// U-Net: M = batch): y = (x_scale * w_scale[n]) * sum_k value(q(x[i][k])) * value(wq[n][k]) + bias[n]
// (Sec. V-B, Y = W A; Sec. VI-A).  With M <= 8 the tensor-core path spends its time on launch
// and pipeline set-up, while the whole layer is one pass over the weights: a warp per
// output column reads that column's codes once, decodes them on the CUDA cores and keeps one FP32
// sum per row (the few activation rows come from the caches, quantized again by every warp).  Every product of an E4M3 value and an E4M3 / E2M1 value is exact in FP32, so
// this path differs from the tensor-core path only in the order of the FP32 additions.
#include <cuda_fp16.h>

#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

constexpr int SMALLM_THREADS = 128;
constexpr int SMALLM_MAX_ROWS = 8;

// two E4M3 codes (low byte first) -> their values
__device__ __forceinline__ float2 e4m3x2_values(uint16_t codes)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(codes));
    return __half22float2(*reinterpret_cast<__half2*>(&h2));
}

// one E2M1 code (bias 1): 0, 0.5, 1, 1.5, 2, 3, 4, 6 with a sign bit, built as FP32 bits
__device__ __forceinline__ float e2m1_value(uint32_t code)
{
    const uint32_t mag = code & 7u;
    const uint32_t normal = ((126u + (mag >> 1)) << 23) | ((mag & 1u) << 22);     // (1 + d/2) 2^(p-1)
    const uint32_t sub = (mag & 1u) ? 0x3f000000u : 0u;                            // d * 0.5
    return __uint_as_float((mag >= 2u ? normal : sub) | ((code & 8u) << 28));
}

// MR = rows held per thread (M rounded up to 1, 2, 4 or 8).  A warp owns an output column; per step a
// lane takes 4 bytes of that column's codes (4 or 8 reduction elements) and the matching 16 or 32
// bytes of every activation row, quantizes the activations to E4M3 values on the fly (Sec. IV-B; hardware
// convert there and back) and adds the products.  Weights and activations of several steps are
// requested before the first is used: the layer is one round trip to memory, not a chain of them.
template <bool W4, int MR>
__global__ void __launch_bounds__(SMALLM_THREADS) small_m_linear_kernel(const float* __restrict__ x, int M, int K, int Kp,
                                                                        const uint8_t* __restrict__ w, int N,
                                                                        const float* __restrict__ w_scale, float x_scale,
                                                                        float rinv, const float* __restrict__ bias,
                                                                        float* __restrict__ y, int* status)
{
    constexpr int PER = W4 ? 8 : 4;                   // reduction elements per lane and step
    constexpr int STEP = 32 * PER;
    constexpr int U = (MR * PER >= 32) ? 2 : (MR * PER >= 16 ? 4 : 8);     // steps in flight
    bool nan = false;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_bytes = W4 ? Kp / 2 : Kp;
    for (int n = blockIdx.x * (SMALLM_THREADS / 32) + warp; n < N; n += gridDim.x * (SMALLM_THREADS / 32)) {
        float acc[MR];
#pragma unroll
        for (int m = 0; m < MR; ++m)
            acc[m] = 0.f;
        const uint8_t* wr = w + (int64_t)n * row_bytes;
        for (int kb = 0; kb < K; kb += U * STEP) {
            uint32_t cw[U];
            float4 xv[U][MR][PER / 4];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int k0 = kb + u * STEP + lane * PER;
                const bool in = k0 < K;               // K is a multiple of 4: a group of four never straddles the end
                cw[u] = in ? __ldg(reinterpret_cast<const uint32_t*>(wr + (W4 ? k0 / 2 : k0))) : 0u;
#pragma unroll
                for (int m = 0; m < MR; ++m)
#pragma unroll
                    for (int e = 0; e < PER / 4; ++e)
                        xv[u][m][e] = (in && m < M && k0 + 4 * e < K)
                                          ? __ldg(reinterpret_cast<const float4*>(x + (int64_t)m * K + k0) + e)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float wv[PER];
                if (W4) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        wv[e] = e2m1_value(cw[u] >> (4 * e));               // even index in the low nibble
                } else {
                    const float2 a = e4m3x2_values((uint16_t)(cw[u] & 0xffffu)), b = e4m3x2_values((uint16_t)(cw[u] >> 16));
                    wv[0] = a.x; wv[1] = a.y; wv[2] = b.x; wv[3] = b.y;
                }
#pragma unroll
                for (int m = 0; m < MR; ++m) {
#pragma unroll
                    for (int e = 0; e < PER / 4; ++e) {
                        const float4 t = xv[u][m][e];
                        const uint32_t c4 = e4m3x4_from_scaled(__fmul_rn(t.x, rinv), __fmul_rn(t.y, rinv),
                                                               __fmul_rn(t.z, rinv), __fmul_rn(t.w, rinv), nan);
                        const float2 lo = e4m3x2_values((uint16_t)(c4 & 0xffffu)), hi = e4m3x2_values((uint16_t)(c4 >> 16));
                        acc[m] = fmaf(lo.x, wv[4 * e], acc[m]);
                        acc[m] = fmaf(lo.y, wv[4 * e + 1], acc[m]);
                        acc[m] = fmaf(hi.x, wv[4 * e + 2], acc[m]);
                        acc[m] = fmaf(hi.y, wv[4 * e + 3], acc[m]);
                    }
                }
            }
        }
        const float sv = x_scale * __ldg(w_scale + n), bv = bias ? __ldg(bias + n) : 0.f;
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            float a = acc[m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0 && m < M)
                y[(int64_t)m * N + n] = fmaf(a, sv, bv);
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

bool small_m_linear_applies(int64_t M, int64_t K)
{
    // (rows are read as 16-byte pieces: K a multiple of 4)
    return M >= 1 && M <= SMALLM_MAX_ROWS && K % 4 == 0 && K <= (1 << 20);
}

template <bool W4, int MR>
static void launch_small(int blocks, const float* x, int M, int K, int Kp, const uint8_t* w, int N, const float* w_scale,
                         float x_scale, const float* bias, float* y, cudaStream_t st)
{
    small_m_linear_kernel<W4, MR><<<blocks, SMALLM_THREADS, 0, st>>>(x, M, K, Kp, w, N, w_scale, x_scale, 1.0f / x_scale,
                                                                     bias, y, status_word());
}

fpq_status launch_small_m_linear(const float* x, int M, int K, const void* w_prepared, int w4, int N, const float* w_scale,
                                 float x_scale, const float* bias, float* y, cudaStream_t st)
{
    const int Kp = (int)round_up(K, 128);
    int blocks = (N + SMALLM_THREADS / 32 - 1) / (SMALLM_THREADS / 32);
    if (blocks > 148 * 16)
        blocks = 148 * 16;
    const uint8_t* w = (const uint8_t*)w_prepared;
    const int mr = M <= 1 ? 1 : (M <= 2 ? 2 : (M <= 4 ? 4 : 8));
#define FPQ_SMALL(W4, MR) launch_small<W4, MR>(blocks, x, M, K, Kp, w, N, w_scale, x_scale, bias, y, st)
    if (w4) {
        if (mr == 1) FPQ_SMALL(true, 1); else if (mr == 2) FPQ_SMALL(true, 2); else if (mr == 4) FPQ_SMALL(true, 4); else FPQ_SMALL(true, 8);
    } else {
        if (mr == 1) FPQ_SMALL(false, 1); else if (mr == 2) FPQ_SMALL(false, 2); else if (mr == 4) FPQ_SMALL(false, 4); else FPQ_SMALL(false, 8);
    }
#undef FPQ_SMALL
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq
