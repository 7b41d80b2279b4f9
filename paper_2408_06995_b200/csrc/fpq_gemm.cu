// Low-bit contraction on the 5th-generation tensor cores: TMA-fed tcgen05.mma
// (kind::f8f6f4, E4M3 activations x E4M3 or E2M1 weights, FP32 accumulate in
// tensor memory) with the dequantize + bias epilogue.  One persistent kernel serves
// the linear layer and the implicit-GEMM convolution.
//
// A CTA (one per SM) walks 128 x BN output tiles.  Warp 0 issues TMA loads into two
// shared-memory rings (activations, weights), warp 1 owns tensor memory and issues
// the MMAs into one of two accumulators, warps 2-5 drain the other accumulator
// (scale, bias, FP32 stores), so a tile's epilogue overlaps the next tile's main loop.
//
// Activation operand, three addressing modes:
//   ROWS  linear: 128 rows of [M][Ca] codes per 128-wide reduction chunk;
//   FLAT  stride-1 convolution on the zero-framed channels-last codes
//         [B][Hp][Wp][Ca] seen as one list of pixels: output position q reads input
//         positions q + r*Wp + s, so one load of 128 + (R-1)*Wp + (S-1) pixel rows
//         serves all R*S taps through matrix descriptors whose start address is moved
//         by whole 128-byte rows (the 128-byte swizzle is a function of the shared-memory
//         address itself, so TMA-written data and a shifted descriptor stay consistent;
//         the descriptor's base-offset field stays 0);
//   TAPS  any stride: one 4-D box (channels, x, y, image) per tap.
#include <cuda.h>

#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

constexpr int BM = 128;        // output rows per tile (TMEM lanes)
constexpr int BK = 128;        // reduction elements per chunk (one 128-byte swizzled row)
constexpr int UMMA_K = 32;     // reduction elements per MMA instruction
constexpr int NUM_THREADS = 192;
constexpr int SMEM_BUDGET = 220 * 1024;

enum { MODE_ROWS = 0, MODE_FLAT = 1, MODE_TAPS = 2 };

struct GemmArgs {
    int mode;
    int64_t M;                 // ROWS: rows; FLAT: framed pixels B*Hp*Wp
    int N;
    int cchunks;               // 128-wide chunks of the reduction per tap
    int taps, S, stride;
    int Wp, HpWp;              // framed geometry
    int Wt, Ht, Bt;            // TAPS: tile of Wt * Ht * Bt = 128 output pixels
    int tiles_x, tiles_y;
    int Ho, Wo, B;
    int m_tiles, n_tiles;
    int a_boxes, a_box_rows;   // activation stage = a_boxes TMA boxes of a_box_rows pixel rows
    int a_stage_bytes, b_stage_bytes;
    int a_stages, b_stages;
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
    int* status;
    uint32_t idesc;
    uint32_t a_stage_tx, b_stage_tx;   // bytes one stage's loads report to its barrier
};

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1) fpq_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                  const __grid_constant__ CUtensorMap tmB,
                                                                  const GemmArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    // layout: [A ring][B ring][barriers + flags][scale | bias]
    const uint32_t a_ring = smem_base;
    const uint32_t b_ring = a_ring + g.a_stages * g.a_stage_bytes;
    const uint32_t ctl_off = g.a_stages * g.a_stage_bytes + g.b_stages * g.b_stage_bytes;
    const uint32_t bars = smem_base + ctl_off;
    // barrier slots (8 bytes each): a_full[8] a_empty[8] b_full[8] b_empty[8] acc_full[2] acc_empty[2]
    const uint32_t a_full = bars, a_empty = bars + 64, b_full = bars + 128, b_empty = bars + 192;
    const uint32_t acc_full = bars + 256, acc_empty = bars + 272;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + ctl_off + 288);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_scale = reinterpret_cast<float*>(smem + ctl_off + 320);   // [2][BN]
    float* s_bias = s_scale + 2 * BN;                                   // [2][BN]

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = g.m_tiles * g.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(a_full + 8 * s, 1);
            mbar_init(a_empty + 8 * s, 1);
            mbar_init(b_full + 8 * s, 1);
            mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, 4);      // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t ia = 0, ib = 0;              // loads issued so far into each ring
            bool dead = false;
            for (int t = blockIdx.x; t < total_tiles && !dead; t += gridDim.x) {
                const int mt = t / g.n_tiles, nt = t - mt * g.n_tiles;
                const int n0 = nt * BN;
                int x0 = 0, y0 = 0, b0 = 0;
                if (g.mode == MODE_TAPS) {
                    int r = mt;
                    x0 = (r % g.tiles_x) * g.Wt;
                    r /= g.tiles_x;
                    y0 = (r % g.tiles_y) * g.Ht;
                    b0 = (r / g.tiles_y) * g.Bt;
                }
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    for (int tap = 0; tap < g.taps; ++tap) {
                        if (g.mode == MODE_TAPS || tap == 0) {
                            const uint32_t s = ia % g.a_stages, ph = (ia / g.a_stages) & 1;
                            if (!mbar_wait(a_empty + 8 * s, ph ^ 1) || *abort_flag) { dead = true; break; }
                            const uint32_t dst = a_ring + s * g.a_stage_bytes;
                            mbar_expect_tx(a_full + 8 * s, g.a_stage_tx);
                            if (g.mode == MODE_TAPS) {
                                const int r = tap / g.S, sx = tap - r * g.S;
                                tma_load_4d(dst, &tmA, a_full + 8 * s, cc * BK, x0 * g.stride + sx, y0 * g.stride + r, b0);
                            } else {
                                for (int bx = 0; bx < g.a_boxes; ++bx)
                                    tma_load_4d(dst + bx * g.a_box_rows * 128, &tmA, a_full + 8 * s, cc * BK,
                                                mt * BM + bx * g.a_box_rows, 0, 0);
                            }
                            ++ia;
                        }
                        const uint32_t s = ib % g.b_stages, ph = (ib / g.b_stages) & 1;
                        if (!mbar_wait(b_empty + 8 * s, ph ^ 1) || *abort_flag) { dead = true; break; }
                        mbar_expect_tx(b_full + 8 * s, g.b_stage_tx);
                        tma_load_3d(b_ring + s * g.b_stage_bytes, &tmB, b_full + 8 * s, cc * BK, tap, n0);
                        ++ib;
                    }
                }
            }
            if (dead) {
                *abort_flag = 1;
                atomicMin(g.status, FPQ_ERR_TIMEOUT);
                // let the copies still in flight land before the CTA's shared memory is released
                for (uint32_t i = (ia > (uint32_t)g.a_stages ? ia - g.a_stages : 0); i < ia; ++i)
                    (void)mbar_wait(a_full + 8 * (i % g.a_stages), (i / g.a_stages) & 1);
                for (uint32_t i = (ib > (uint32_t)g.b_stages ? ib - g.b_stages : 0); i < ib; ++i)
                    (void)mbar_wait(b_full + 8 * (i % g.b_stages), (i / g.b_stages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t ia = 0, ib = 0, it = 0;
            bool dead = false;
            for (int t = blockIdx.x; t < total_tiles && !dead; t += gridDim.x, ++it) {
                const uint32_t buf = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1) || *abort_flag) { dead = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                uint32_t first = 1;
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    uint32_t a_addr = 0;
                    for (int tap = 0; tap < g.taps; ++tap) {
                        if (g.mode == MODE_TAPS || tap == 0) {
                            const uint32_t s = ia % g.a_stages, ph = (ia / g.a_stages) & 1;
                            if (!mbar_wait(a_full + 8 * s, ph) || *abort_flag) { dead = true; break; }
                            a_addr = a_ring + s * g.a_stage_bytes;
                        }
                        const uint32_t sb = ib % g.b_stages, phb = (ib / g.b_stages) & 1;
                        if (!mbar_wait(b_full + 8 * sb, phb) || *abort_flag) { dead = true; break; }
                        tc_fence_after();
                        uint32_t a_tap = a_addr;
                        if (g.mode == MODE_FLAT) {
                            const int r = tap / g.S, sx = tap - r * g.S;
                            a_tap += (uint32_t)(r * g.Wp + sx) * 128u;
                        }
                        const uint64_t adesc = smem_desc_k_sw128(a_tap);
                        const uint64_t bdesc = smem_desc_k_sw128(b_ring + sb * g.b_stage_bytes);
#pragma unroll
                        for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                            // 32 reduction elements = 32 bytes inside the swizzled row: +2 in 16-byte units
                            mma_f8f6f4(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, g.idesc, first ? 0u : 1u);
                            first = 0;
                        }
                        mma_commit(b_empty + 8 * sb);
                        ++ib;
                        if (g.mode == MODE_TAPS || tap == g.taps - 1) {
                            mma_commit(a_empty + 8 * (ia % g.a_stages));
                            ++ia;
                        }
                    }
                }
                mma_commit(acc_full + 8 * buf);
            }
            if (dead) {
                *abort_flag = 1;
                atomicMin(g.status, FPQ_ERR_TIMEOUT);
            }
        }
    } else {
        // ---------------- epilogue: 4 warps, one TMEM lane quarter each ----------------
        const int et = threadIdx.x - 64;           // 0..127
        const int quarter = warp & 3;              // TMEM lanes this warp may read
        const int row = quarter * 32 + lane;       // row of the tile held by this thread
        uint32_t it = 0;
        bool dead = false;
        for (int t = blockIdx.x; t < total_tiles && !dead; t += gridDim.x, ++it) {
            const int mt = t / g.n_tiles, nt = t - mt * g.n_tiles;
            const int n0 = nt * BN;
            const uint32_t buf = it & 1, aph = (it >> 1) & 1;
            float* sc = s_scale + buf * BN;
            float* bi = s_bias + buf * BN;
            for (int i = et; i < BN; i += 128) {
                const int n = n0 + i;
                sc[i] = (n < g.N) ? g.x_scale * __ldg(g.w_scale + n) : 0.f;
                bi[i] = (g.bias && n < g.N) ? __ldg(g.bias + n) : 0.f;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");

            // where this thread's row goes
            bool row_valid;
            float* yrow;
            int64_t nstride;
            if (g.mode == MODE_ROWS) {
                const int64_t m = (int64_t)mt * BM + row;
                row_valid = m < g.M;
                nstride = 1;
                yrow = g.y + m * g.N;
            } else {
                int ox, oy, b;
                if (g.mode == MODE_FLAT) {
                    const int64_t q = (int64_t)mt * BM + row;
                    b = (int)(q / g.HpWp);
                    const int rem = (int)(q - (int64_t)b * g.HpWp);
                    oy = rem / g.Wp;
                    ox = rem - oy * g.Wp;
                } else {
                    int r = mt;
                    const int x0 = (r % g.tiles_x) * g.Wt;
                    r /= g.tiles_x;
                    const int y0 = (r % g.tiles_y) * g.Ht;
                    const int b0 = (r / g.tiles_y) * g.Bt;
                    ox = x0 + row % g.Wt;
                    oy = y0 + (row / g.Wt) % g.Ht;
                    b = b0 + row / (g.Wt * g.Ht);
                }
                row_valid = ox < g.Wo && oy < g.Ho && b < g.B;
                nstride = (int64_t)g.Ho * g.Wo;
                yrow = g.y + ((int64_t)b * g.N * g.Ho + oy) * g.Wo + ox;   // + n * Ho * Wo
            }

            bool ok = mbar_wait(acc_full + 8 * buf, aph);
            if (!ok || *abort_flag) { dead = true; }
            tc_fence_after();
            if (!dead) {
                const bool vec_ok = (g.mode == MODE_ROWS) && (g.N % 4 == 0);
                const uint32_t t_addr = tmem_base + buf * BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    if (n0 + c * 32 >= g.N)
                        break;                                  // whole chunk past the last column
                    uint32_t r[32];
                    tmem_ld32(t_addr + c * 32, r);
                    tmem_ld_wait();
                    if (!row_valid)
                        continue;
                    const int nb = n0 + c * 32;
                    if (vec_ok && nb + 32 <= g.N) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 v;
                            v.x = fmaf(__uint_as_float(r[j + 0]), sc[c * 32 + j + 0], bi[c * 32 + j + 0]);
                            v.y = fmaf(__uint_as_float(r[j + 1]), sc[c * 32 + j + 1], bi[c * 32 + j + 1]);
                            v.z = fmaf(__uint_as_float(r[j + 2]), sc[c * 32 + j + 2], bi[c * 32 + j + 2]);
                            v.w = fmaf(__uint_as_float(r[j + 3]), sc[c * 32 + j + 3], bi[c * 32 + j + 3]);
                            *reinterpret_cast<float4*>(yrow + nb + j) = v;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (nb + j < g.N)
                                yrow[(int64_t)(nb + j) * nstride] =
                                    fmaf(__uint_as_float(r[j]), sc[c * 32 + j], bi[c * 32 + j]);
                        }
                    }
                }
            }
            // hand the accumulator back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0)
                mbar_arrive(acc_empty + 8 * buf);
        }
        if (dead) {
            *abort_flag = 1;
            atomicMin(g.status, FPQ_ERR_TIMEOUT);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
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

static int sm_count()
{
    static int n[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return 148;
    if (!n[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
            v = 148;
        n[dev] = v;
    }
    return n[dev];
}

template <int BN>
static fpq_status launch_variant(const CUtensorMap& tmA, const CUtensorMap& tmB, GemmArgs& g, cudaStream_t st)
{
    g.b_stage_bytes = BN * BK;
    // split the shared-memory budget between the two rings
    const int ctl = 320 + 4 * BN * 4 + 1024;
    int a_stages = (g.mode == MODE_TAPS) ? 4 : 2;
    int b_stages = (SMEM_BUDGET - ctl - a_stages * g.a_stage_bytes) / g.b_stage_bytes;
    if (g.mode != MODE_TAPS && b_stages > 6 && SMEM_BUDGET - ctl - 3 * g.a_stage_bytes >= 4 * g.b_stage_bytes) {
        a_stages = 3;
        b_stages = (SMEM_BUDGET - ctl - a_stages * g.a_stage_bytes) / g.b_stage_bytes;
    }
    if (b_stages > 8)
        b_stages = 8;
    if (b_stages < 2)
        return FPQ_ERR_UNSUPPORTED;
    g.a_stages = a_stages;
    g.b_stages = b_stages;
    const int dyn = a_stages * g.a_stage_bytes + b_stages * g.b_stage_bytes + ctl;
    if (cudaFuncSetAttribute(fpq_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET) !=
        cudaSuccess)
        return FPQ_ERR_CUDA;
    const int64_t tiles = (int64_t)g.m_tiles * g.n_tiles;
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    fpq_gemm_kernel<BN><<<grid, NUM_THREADS, dyn, st>>>(tmA, tmB, g);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

fpq_status launch_gemm(const GemmProblem& p, cudaStream_t st)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc)
        return FPQ_ERR_CUDA;

    GemmArgs g{};
    g.N = p.N;
    g.cchunks = p.Cp / BK;
    g.taps = p.R * p.S;
    g.S = p.S;
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
    g.n_tiles = (p.N + BN - 1) / BN;
    g.idesc = idesc_f8f6f4(0u, p.w4 ? 5u : 0u, (uint32_t)BN);
    g.b_stage_tx = (uint32_t)(BN * BK) / (p.w4 ? 2 : 1);

    CUtensorMap tmA, tmB;
    cuuint64_t dimsA[4], stridesA[3];
    cuuint32_t boxA[4], estrA[4] = {1, 1, 1, 1};
    const int Hp = p.H + 2 * p.pad, Wp = p.W + 2 * p.pad;
    int64_t mtiles;
    if (!p.conv) {
        g.mode = MODE_ROWS;
        g.M = p.M;
        mtiles = (p.M + BM - 1) / BM;
        g.a_boxes = 1;
        g.a_box_rows = BM;
        dimsA[0] = (cuuint64_t)p.Ca; dimsA[1] = (cuuint64_t)p.M; dimsA[2] = 1; dimsA[3] = 1;
        stridesA[0] = (cuuint64_t)p.Ca; stridesA[1] = stridesA[2] = (cuuint64_t)p.Ca * p.M;
        boxA[0] = BK; boxA[1] = BM; boxA[2] = 1; boxA[3] = 1;
    } else {
        const int64_t framed = (int64_t)p.B * Hp * Wp;
        const int halo_rows = BM + (p.R - 1) * Wp + (p.S - 1);
        // FLAT wastes the frame positions; take it when that costs little more than TAPS' exact tiles
        const int64_t flat_tiles = (framed + BM - 1) / BM;
        const int64_t exact_tiles = ((int64_t)p.B * p.Ho * p.Wo + BM - 1) / BM;
        const bool flat_ok = p.stride == 1 && halo_rows <= 2 * 256 - 16 && flat_tiles * 4 <= exact_tiles * 5 + 4;
        if (flat_ok) {
            g.mode = MODE_FLAT;
            g.M = framed;
            g.Wp = Wp;
            g.HpWp = Hp * Wp;
            mtiles = flat_tiles;
            g.a_boxes = halo_rows > 256 ? 2 : 1;
            g.a_box_rows = (int)round_up((halo_rows + g.a_boxes - 1) / g.a_boxes, 8);
            dimsA[0] = (cuuint64_t)p.Ca; dimsA[1] = (cuuint64_t)framed; dimsA[2] = 1; dimsA[3] = 1;
            stridesA[0] = (cuuint64_t)p.Ca; stridesA[1] = stridesA[2] = (cuuint64_t)p.Ca * framed;
            boxA[0] = BK; boxA[1] = (cuuint32_t)g.a_box_rows; boxA[2] = 1; boxA[3] = 1;
        } else {
            if (p.stride < 1 || p.stride > 8)
                return FPQ_ERR_UNSUPPORTED;
            g.mode = MODE_TAPS;
            int wcap = 256 / p.stride;
            if (wcap > BM)
                wcap = BM;
            g.Wt = pow2_at_least(p.Wo);
            if (g.Wt > wcap)
                g.Wt = wcap;
            g.Ht = pow2_at_least(p.Ho);
            if (g.Ht > BM / g.Wt)
                g.Ht = BM / g.Wt;
            g.Bt = BM / (g.Wt * g.Ht);
            g.tiles_x = (p.Wo + g.Wt - 1) / g.Wt;
            g.tiles_y = (p.Ho + g.Ht - 1) / g.Ht;
            const int tiles_b = (p.B + g.Bt - 1) / g.Bt;
            mtiles = (int64_t)g.tiles_x * g.tiles_y * tiles_b;
            g.a_boxes = 1;
            g.a_box_rows = BM;
            dimsA[0] = (cuuint64_t)p.Ca; dimsA[1] = (cuuint64_t)Wp; dimsA[2] = (cuuint64_t)Hp; dimsA[3] = (cuuint64_t)p.B;
            stridesA[0] = (cuuint64_t)p.Ca;
            stridesA[1] = (cuuint64_t)p.Ca * Wp;
            stridesA[2] = (cuuint64_t)p.Ca * Wp * Hp;
            boxA[0] = BK; boxA[1] = (cuuint32_t)(g.Wt * p.stride); boxA[2] = (cuuint32_t)(g.Ht * p.stride);
            boxA[3] = (cuuint32_t)g.Bt;
            estrA[1] = estrA[2] = (cuuint32_t)p.stride;
        }
    }
    if (mtiles <= 0 || mtiles * g.n_tiles > 0x7fffffff)
        return FPQ_ERR_SHAPE;
    g.m_tiles = (int)mtiles;
    g.a_stage_bytes = g.a_boxes * g.a_box_rows * 128;
    g.a_stage_tx = (uint32_t)g.a_stage_bytes;
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

    if (BN == 64)
        return launch_variant<64>(tmA, tmB, g, st);
    return launch_variant<128>(tmA, tmB, g, st);
}

}  // namespace fpq
