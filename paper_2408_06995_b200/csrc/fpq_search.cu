// Encoding and bias search of one tensor (Sec. V-A, Algorithm 1): the mean squared
// error of quantizing the tensor with every (encoding, clipping value) candidate, all
// candidates in one pass over the data, then the selection rule of Algorithm 1.
//
// The work is arithmetic, not memory: each FP32 element read once (4 bytes) is
// quantized and compared a few hundred times.  A thread keeps 16 elements in registers
// and walks the candidate list; per candidate and element the quantize-dequantize-error
// chain is nine instructions (see search_mse_kernel).
#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

constexpr int SEARCH_THREADS = 256;
constexpr int SEARCH_PER_THREAD = 16;
constexpr int SEARCH_MAX_ENC = 8;
constexpr int SEARCH_MAX_CLIP = 256;
constexpr int SEARCH_MAX_CAND = 1024;
constexpr int SEARCH_MAX_BLOCKS = 1184;

struct SearchEnc {
    uint32_t cmax_bits;      // FP32 bit pattern of the format's own clipping value
    uint32_t ebmin_bits;     // exponent field (in place, << 23) of the smallest normal value
    uint32_t cbase;          // added to an exponent field: the rounding constant 1.5 * 2^(23 - m) of that binade
    float cmax;
};

struct SearchArgs {
    SearchEnc enc[SEARCH_MAX_ENC];
    int n_enc, n_clip;
    int64_t n;
    const float* x;
    const float* clip;
    double* partial;         // [gridDim.x][n_enc * n_clip]
    int* status;
};

// Per candidate (i, j): scale = clip[j] / c(F_i) and 1 / scale, both FP32 divisions.
// Per element: t = |x| / scale, clipped at c; the step s of t's binade (the smallest normal
// binade for everything below it); C = 1.5 * 2^23 * s, so that (t + C) - C is t rounded to a
// multiple of s, ties to the even multiple (the hardware's FP32 rounding does the work);
// error = |x| - scale * q with one rounding (FMA).  The quantizer is odd, so signs drop out.
__global__ void __launch_bounds__(SEARCH_THREADS) search_mse_kernel(const SearchArgs a)
{
    extern __shared__ double s_dyn[];
    const int ncand = a.n_enc * a.n_clip;
    double* wsum = s_dyn;                                                   // [8 warps][ncand]
    float* s_rinv = reinterpret_cast<float*>(wsum + (SEARCH_THREADS / 32) * ncand);   // [ncand]
    float* s_scale = s_rinv + ncand;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int c = threadIdx.x; c < ncand; c += SEARCH_THREADS) {
        const int i = c / a.n_clip, j = c - i * a.n_clip;
        const float scale = __fdiv_rn(__ldg(a.clip + j), a.enc[i].cmax);
        s_scale[c] = scale;
        s_rinv[c] = __fdiv_rn(1.0f, scale);
    }
    for (int c = threadIdx.x; c < (SEARCH_THREADS / 32) * ncand; c += SEARCH_THREADS)
        wsum[c] = 0.0;
    __syncthreads();

    bool nan = false;
    const int64_t chunk = (int64_t)SEARCH_THREADS * SEARCH_PER_THREAD;
    const int64_t nchunks = (a.n + chunk - 1) / chunk;
    for (int64_t ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        float ax[SEARCH_PER_THREAD];
        const int64_t base = ch * chunk;
        if (base + chunk <= a.n && ((uintptr_t)a.x % 16) == 0) {
#pragma unroll
            for (int v = 0; v < SEARCH_PER_THREAD / 4; ++v) {
                const float4 f = __ldg(reinterpret_cast<const float4*>(a.x + base) + v * SEARCH_THREADS + threadIdx.x);
                ax[4 * v] = fabsf(f.x);
                ax[4 * v + 1] = fabsf(f.y);
                ax[4 * v + 2] = fabsf(f.z);
                ax[4 * v + 3] = fabsf(f.w);
            }
        } else {
#pragma unroll
            for (int v = 0; v < SEARCH_PER_THREAD; ++v) {
                const int64_t k = base + (int64_t)v * SEARCH_THREADS + threadIdx.x;
                ax[v] = k < a.n ? fabsf(__ldg(a.x + k)) : 0.f;      // a zero adds no error to any candidate
            }
        }
#pragma unroll
        for (int v = 0; v < SEARCH_PER_THREAD; ++v)
            nan |= __float_as_uint(ax[v]) > 0x7f800000u;

        int c = 0;
        for (int i = 0; i < a.n_enc; ++i) {
            const uint32_t cmax_bits = a.enc[i].cmax_bits, ebmin = a.enc[i].ebmin_bits, cbase = a.enc[i].cbase;
            for (int j = 0; j < a.n_clip; ++j, ++c) {
                const float rinv = s_rinv[c], nscale = -s_scale[c];
                float acc = 0.f;
#pragma unroll
                for (int v = 0; v < SEARCH_PER_THREAD; ++v) {
                    const uint32_t tb = min(__float_as_uint(__fmul_rn(ax[v], rinv)), cmax_bits);
                    const float big = __uint_as_float(max(tb & 0x7f800000u, ebmin) + cbase);
                    const float q = __fsub_rn(__fadd_rn(__uint_as_float(tb), big), big);
                    const float err = __fmaf_rn(nscale, q, ax[v]);
                    acc = __fmaf_rn(err, err, acc);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
                    acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (lane == 0)
                    wsum[warp * ncand + c] += (double)acc;
            }
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < ncand; c += SEARCH_THREADS) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < SEARCH_THREADS / 32; ++w)
            s += wsum[w * ncand + c];
        a.partial[(int64_t)blockIdx.x * ncand + c] = s;
    }
    if (nan)
        flag_status(a.status, FPQ_ERR_NAN_INPUT);
}

// Block partial sums -> mse.  A block of 32 x 32 threads owns 32 candidates: thread (slice, ci) adds
// the blocks slice, slice + 32, ... of candidate c0 + ci (coalesced along ci), then the 32 slices are
// added in order: the same order whatever the timing.
__global__ void __launch_bounds__(1024) search_reduce_kernel(const double* __restrict__ partial, int blocks, int ncand,
                                                             int64_t n, double* __restrict__ mse)
{
    __shared__ double s_part[32][33];
    const int ci = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + ci;
    double s = 0.0;
    if (c < ncand)
        for (int b = slice; b < blocks; b += 32)
            s += partial[(int64_t)b * ncand + c];
    s_part[slice][ci] = s;
    __syncthreads();
    if (slice == 0 && c < ncand) {
        double t = 0.0;
#pragma unroll
        for (int k = 0; k < 32; ++k)
            t += s_part[k][ci];
        mse[c] = n > 0 ? t / (double)n : 0.0;
    }
}

// Selection rule of Algorithm 1 (Sec. V-A): the candidate with the smallest error; among equal errors the one
// that comes first in encoding-major, candidate-minor order (the flat index).  The listing's start value for
// the best error is read as +infinity; a NaN error never wins.  One warp: every lane takes the flat indices
// lane, lane + 32, ..., then a shuffle tree reduces the (error, index) pairs with the smaller index breaking ties.
__global__ void __launch_bounds__(32) search_select_kernel(const double* __restrict__ mse, int n_enc, int n_clip,
                                                           int32_t* __restrict__ best)
{
    const int ncand = n_enc * n_clip, lane = threadIdx.x;
    double err = INFINITY;
    int arg = 0x7fffffff;                        // "nothing yet": loses every tie
    for (int c = lane; c < ncand; c += 32) {
        const double e = mse[c];
        if (e < err) {                           // false for NaN; indices grow, so the first of equal errors stays
            err = e;
            arg = c;
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        const double oe = __shfl_xor_sync(0xffffffffu, err, d);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, d);
        if (oe < err || (oe == err && oa < arg)) {
            err = oe;
            arg = oa;
        }
    }
    if (lane == 0) {
        const bool none = arg == 0x7fffffff;
        best[0] = none ? -1 : arg / n_clip;
        best[1] = none ? -1 : arg % n_clip;
    }
}

size_t search_workspace_bytes(int n_enc, int n_clip)
{
    return (size_t)SEARCH_MAX_BLOCKS * (size_t)n_enc * (size_t)n_clip * sizeof(double);
}

fpq_status launch_search(const float* x, int64_t n, const fpq_format* enc, int n_enc, const float* clip, int n_clip,
                         double* mse, int32_t* best, void* workspace, cudaStream_t st)
{
    SearchArgs a{};
    for (int i = 0; i < n_enc; ++i) {
        QFormat q;
        if (!resolve_format(enc[i], &q))
            return FPQ_ERR_FORMAT;
        a.enc[i].cmax_bits = q.cmax_bits;
        a.enc[i].ebmin_bits = (uint32_t)(128 - q.B) << 23;
        a.enc[i].cbase = ((uint32_t)(23 - q.m) << 23) | 0x400000u;
        a.enc[i].cmax = format_cmax(enc[i]);
    }
    a.n_enc = n_enc;
    a.n_clip = n_clip;
    a.n = n;
    a.x = x;
    a.clip = clip;
    a.partial = (double*)workspace;
    a.status = status_word();
    if (!a.status)
        return FPQ_ERR_CUDA;
    const int ncand = n_enc * n_clip;
    const int64_t chunk = (int64_t)SEARCH_THREADS * SEARCH_PER_THREAD;
    int64_t blocks = (n + chunk - 1) / chunk;
    if (blocks > SEARCH_MAX_BLOCKS)
        blocks = SEARCH_MAX_BLOCKS;
    if (blocks < 1)
        blocks = 1;
    const size_t smem = (size_t)(SEARCH_THREADS / 32) * ncand * sizeof(double) + (size_t)ncand * 2 * sizeof(float);
    static std::mutex attr_mutex;
    std::lock_guard<std::mutex> lock(attr_mutex);
    static bool smem_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return FPQ_ERR_CUDA;
    if (!smem_set[dev]) {
        const size_t most = (size_t)(SEARCH_THREADS / 32) * SEARCH_MAX_CAND * sizeof(double) +
                            (size_t)SEARCH_MAX_CAND * 2 * sizeof(float);
        if (cudaFuncSetAttribute(search_mse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most) != cudaSuccess)
            return FPQ_ERR_CUDA;
        smem_set[dev] = true;
    }
    search_mse_kernel<<<(unsigned)blocks, SEARCH_THREADS, smem, st>>>(a);
    if (cudaGetLastError() != cudaSuccess)
        return FPQ_ERR_CUDA;
    search_reduce_kernel<<<(ncand + 31) / 32, 1024, 0, st>>>((const double*)workspace, (int)blocks, ncand, n, mse);
    search_select_kernel<<<1, 32, 0, st>>>(mse, n_enc, n_clip, best);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

int search_max_enc() { return SEARCH_MAX_ENC; }
int search_max_clip() { return SEARCH_MAX_CLIP; }
int search_max_cand() { return SEARCH_MAX_CAND; }

}  // namespace fpq
