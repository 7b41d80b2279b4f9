// Low-bit contraction on the 5th-generation tensor cores: TMA-fed tcgen05.mma
// (kind::f8f6f4, E4M3 activations x E4M3 or E2M1 weights, FP32 accumulate in
// tensor memory) with the dequantize + bias epilogue.  The same kernel serves the
// linear layer (2-D operand) and the implicit-GEMM convolution (4-D activation
// tensor walked tap by tap; zero padding is the TMA out-of-bounds fill, code 0).
//
// One CTA computes a 128 x BN output tile.  Warp 0 issues TMA loads, warp 1
// owns tensor memory and issues the MMAs, warps 2-5 run the epilogue.
#include <cuda.h>

#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

constexpr int BM = 128;        // output rows per CTA (TMEM lanes)
constexpr int BK = 128;        // reduction elements per pipeline stage (one 128-byte swizzled row)
constexpr int UMMA_K = 32;     // reduction elements per MMA instruction
constexpr int NUM_THREADS = 192;

struct GemmArgs {
    int conv;
    int64_t M;                 // linear rows
    int N;
    int cchunks;               // 128-wide chunks of the reduction per tap
    int taps, S, pad, stride;
    int Wt, Ht, Bt;            // conv tile: Wt * Ht * Bt = 128 output pixels
    int tiles_x, tiles_y;
    int Ho, Wo, B;
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
    int* status;
    uint32_t idesc;
    uint32_t b_stage_tx;       // bytes one weight-tile load reports to its barrier
};

template <int BN, int STAGES>
struct SmemLayout {
    static constexpr int A_BYTES = BM * BK;            // 16 KiB
    static constexpr int B_BYTES = BN * BK;            // footprint (4-bit codes sit in 16-byte containers)
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int BAR_OFF = STAGES * STAGE_BYTES;
    static constexpr int SCALE_OFF = BAR_OFF + 256;
    static constexpr int TOTAL = SCALE_OFF + 2 * BN * 4;
    static constexpr int DYN_BYTES = TOTAL + 1024;     // slack for 1024-byte alignment
};

template <int BN, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS) fpq_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                               const __grid_constant__ CUtensorMap tmB,
                                                               const GemmArgs g)
{
    using L = SmemLayout<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + L::BAR_OFF;             // STAGES x 8 bytes
    const uint32_t bar_empty = bar_full + 8 * STAGES;             // STAGES x 8 bytes
    const uint32_t bar_acc = bar_empty + 8 * STAGES;              // accumulator ready
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * (2 * STAGES + 1));
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_scale = reinterpret_cast<float*>(smem + L::SCALE_OFF);
    float* s_bias = s_scale + BN;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n0 = blockIdx.y * BN;
    const int num_iters = g.taps * g.cchunks;

    // tile origin
    int64_t m0 = 0;
    int x0 = 0, y0 = 0, b0 = 0;
    if (g.conv) {
        int t = blockIdx.x;
        x0 = (t % g.tiles_x) * g.Wt;
        t /= g.tiles_x;
        y0 = (t % g.tiles_y) * g.Ht;
        b0 = (t / g.tiles_y) * g.Bt;
    } else {
        m0 = (int64_t)blockIdx.x * BM;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < num_iters; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                if (!mbar_wait(bar_empty + 8 * s, ph ^ 1) || *abort_flag) {
                    *abort_flag = 1;
                    atomicMin(g.status, FPQ_ERR_TIMEOUT);
                    break;
                }
                const int tap = it / g.cchunks, cc = it - tap * g.cchunks;
                const uint32_t a_dst = smem_base + s * L::STAGE_BYTES;
                const uint32_t b_dst = a_dst + L::A_BYTES;
                mbar_expect_tx(bar_full + 8 * s, L::A_BYTES + g.b_stage_tx);
                if (g.conv) {
                    const int r = tap / g.S, sx = tap - r * g.S;
                    tma_load_4d(a_dst, &tmA, bar_full + 8 * s, cc * BK, x0 * g.stride - g.pad + sx,
                                y0 * g.stride - g.pad + r, b0);
                } else {
                    tma_load_4d(a_dst, &tmA, bar_full + 8 * s, cc * BK, (int)m0, 0, 0);
                }
                tma_load_3d(b_dst, &tmB, bar_full + 8 * s, cc * BK, tap, n0);
                issued = it + 1;
            }
            if (*abort_flag) {
                // let the copies still in flight land before the CTA's shared memory is released
                for (int it = max(0, issued - STAGES); it < issued; ++it)
                    (void)mbar_wait(bar_full + 8 * (it % STAGES), (it / STAGES) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            for (int it = 0; it < num_iters; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                if (!mbar_wait(bar_full + 8 * s, ph) || *abort_flag) {
                    *abort_flag = 1;
                    atomicMin(g.status, FPQ_ERR_TIMEOUT);
                    break;
                }
                tc_fence_after();
                const uint32_t a_addr = smem_base + s * L::STAGE_BYTES;
                const uint64_t adesc = smem_desc_k_sw128(a_addr);
                const uint64_t bdesc = smem_desc_k_sw128(a_addr + L::A_BYTES);
#pragma unroll
                for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                    // 32 reduction elements = 32 bytes inside the swizzled row: +2 in 16-byte units
                    mma_f8f6f4(tmem_acc, adesc + 2 * kk, bdesc + 2 * kk, g.idesc, (it | kk) != 0);
                }
                mma_commit(bar_empty + 8 * s);     // stage reusable once these MMAs have read it
            }
            mma_commit(bar_acc);                   // accumulator complete
        }
    } else {
        // ---------------- epilogue: 4 warps, one TMEM lane quarter each ----------------
        const int et = threadIdx.x - 64;           // 0..127
        for (int i = et; i < BN; i += 128) {
            const int n = n0 + i;
            s_scale[i] = (n < g.N) ? g.x_scale * __ldg(g.w_scale + n) : 0.f;
            s_bias[i] = (g.bias && n < g.N) ? __ldg(g.bias + n) : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int quarter = warp & 3;              // TMEM lanes this warp may read
        const int row = quarter * 32 + lane;       // row of the tile held by this thread
        bool ok = mbar_wait(bar_acc, 0);
        if (!ok) {
            *abort_flag = 1;
            atomicMin(g.status, FPQ_ERR_TIMEOUT);
        }
        ok = ok && !*abort_flag;
        tc_fence_after();
        if (ok) {
            bool row_valid;
            float* yrow;
            int64_t nstride;
            if (g.conv) {
                const int xl = row % g.Wt, yl = (row / g.Wt) % g.Ht, bl = row / (g.Wt * g.Ht);
                const int ox = x0 + xl, oy = y0 + yl, b = b0 + bl;
                row_valid = ox < g.Wo && oy < g.Ho && b < g.B;
                nstride = (int64_t)g.Ho * g.Wo;
                yrow = g.y + ((int64_t)b * g.N * g.Ho + oy) * g.Wo + ox;   // + n * Ho * Wo
            } else {
                const int64_t m = m0 + row;
                row_valid = m < g.M;
                nstride = 1;
                yrow = g.y + m * g.N;
            }
            const bool vec_ok = !g.conv && (g.N % 4 == 0);
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                if (!row_valid)
                    continue;
                const int nb = n0 + c * 32;
                if (vec_ok && nb + 32 <= g.N) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 v;
                        v.x = fmaf(__uint_as_float(r[j + 0]), s_scale[c * 32 + j + 0], s_bias[c * 32 + j + 0]);
                        v.y = fmaf(__uint_as_float(r[j + 1]), s_scale[c * 32 + j + 1], s_bias[c * 32 + j + 1]);
                        v.z = fmaf(__uint_as_float(r[j + 2]), s_scale[c * 32 + j + 2], s_bias[c * 32 + j + 2]);
                        v.w = fmaf(__uint_as_float(r[j + 3]), s_scale[c * 32 + j + 3], s_bias[c * 32 + j + 3]);
                        *reinterpret_cast<float4*>(yrow + nb + j) = v;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (nb + j < g.N)
                            yrow[(int64_t)(nb + j) * nstride] =
                                fmaf(__uint_as_float(r[j]), s_scale[c * 32 + j], s_bias[c * 32 + j]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, BN);
    }
}

// ---- host side --------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

static int pow2_at_least(int v)
{
    int p = 1;
    while (p < v)
        p <<= 1;
    return p;
}

template <int BN, int STAGES>
static fpq_status launch_variant(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& g, dim3 grid,
                                 cudaStream_t st)
{
    using L = SmemLayout<BN, STAGES>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(fpq_gemm_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 L::DYN_BYTES) != cudaSuccess)
            return FPQ_ERR_CUDA;
        configured = true;
    }
    fpq_gemm_kernel<BN, STAGES><<<grid, NUM_THREADS, L::DYN_BYTES, st>>>(tmA, tmB, g);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

fpq_status launch_gemm(const GemmProblem& p, cudaStream_t st)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc)
        return FPQ_ERR_CUDA;

    GemmArgs g{};
    g.conv = p.conv;
    g.M = p.M;
    g.N = p.N;
    g.cchunks = p.Cp / BK;
    g.taps = p.R * p.S;
    g.S = p.S;
    g.pad = p.pad;
    g.stride = p.stride;
    g.Ho = p.Ho;
    g.Wo = p.Wo;
    g.B = p.B;
    g.w_scale = p.w_scale;
    g.x_scale = p.x_scale;
    g.bias = p.bias;
    g.y = p.y;
    g.status = status_word();

    const int BN = (p.N <= 64) ? 64 : 128;
    g.idesc = idesc_f8f6f4(0u, p.w4 ? 5u : 0u, (uint32_t)BN);
    g.b_stage_tx = (uint32_t)(BN * BK) / (p.w4 ? 2 : 1);

    // activation codes
    CUtensorMap tmA, tmB;
    cuuint64_t dimsA[4], stridesA[3];
    cuuint32_t boxA[4], estrA[4];
    int64_t mtiles;
    if (p.conv) {
        if (p.stride < 1 || p.stride > 8)
            return FPQ_ERR_UNSUPPORTED;
        int wcap = 256 / p.stride;
        if (wcap > 128)
            wcap = 128;
        g.Wt = pow2_at_least(p.Wo);
        if (g.Wt > wcap)
            g.Wt = wcap;
        g.Ht = pow2_at_least(p.Ho);
        if (g.Ht > BM / g.Wt)
            g.Ht = BM / g.Wt;
        g.Bt = BM / (g.Wt * g.Ht);
        g.tiles_x = (p.Wo + g.Wt - 1) / g.Wt;
        g.tiles_y = (p.Ho + g.Ht - 1) / g.Ht;
        int tiles_b = (p.B + g.Bt - 1) / g.Bt;
        mtiles = (int64_t)g.tiles_x * g.tiles_y * tiles_b;
        dimsA[0] = (cuuint64_t)p.Ca; dimsA[1] = (cuuint64_t)p.W; dimsA[2] = (cuuint64_t)p.H; dimsA[3] = (cuuint64_t)p.B;
        stridesA[0] = (cuuint64_t)p.Ca;
        stridesA[1] = (cuuint64_t)p.Ca * p.W;
        stridesA[2] = (cuuint64_t)p.Ca * p.W * p.H;
        boxA[0] = BK; boxA[1] = (cuuint32_t)(g.Wt * p.stride); boxA[2] = (cuuint32_t)(g.Ht * p.stride); boxA[3] = (cuuint32_t)g.Bt;
        estrA[0] = 1; estrA[1] = (cuuint32_t)p.stride; estrA[2] = (cuuint32_t)p.stride; estrA[3] = 1;
    } else {
        mtiles = (p.M + BM - 1) / BM;
        dimsA[0] = (cuuint64_t)p.Ca; dimsA[1] = (cuuint64_t)p.M; dimsA[2] = 1; dimsA[3] = 1;
        stridesA[0] = (cuuint64_t)p.Ca;
        stridesA[1] = (cuuint64_t)p.Ca * p.M;
        stridesA[2] = (cuuint64_t)p.Ca * p.M;
        boxA[0] = BK; boxA[1] = BM; boxA[2] = 1; boxA[3] = 1;
        estrA[0] = estrA[1] = estrA[2] = estrA[3] = 1;
    }
    if (mtiles <= 0 || mtiles > 0x7fffffff)
        return FPQ_ERR_SHAPE;
    if (enc(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void*)p.a_codes, dimsA, stridesA, boxA, estrA,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return FPQ_ERR_CUDA;

    // prepared weights [N][taps][Cp]
    cuuint64_t dimsB[3] = {(cuuint64_t)p.Cp, (cuuint64_t)g.taps, (cuuint64_t)p.N};
    cuuint64_t rowB = p.w4 ? (cuuint64_t)p.Cp / 2 : (cuuint64_t)p.Cp;
    cuuint64_t stridesB[2] = {rowB, rowB * g.taps};
    cuuint32_t boxB[3] = {BK, 1, (cuuint32_t)BN};
    cuuint32_t estrB[3] = {1, 1, 1};
    if (enc(&tmB, p.w4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
            (void*)p.w_prepared, dimsB, stridesB, boxB, estrB, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return FPQ_ERR_CUDA;

    dim3 grid((unsigned)mtiles, (unsigned)((p.N + BN - 1) / BN), 1);
    if (BN == 64)
        return launch_variant<64, 4>(tmA, tmB, g, grid, st);
    return launch_variant<128, 3>(tmA, tmB, g, grid, st);
}

}  // namespace fpq
