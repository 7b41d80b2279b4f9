// FP32 contractions of the rounding-learning step (Sec. V-B: the reconstruction error D = A (Wq - W)^T and
// its gradient D^T A) on the tensor cores: C[i][j] = sum_r P[i][r] Q[j][r] with both operands row-major and
// the reduction index contiguous.
//
// The tensor cores multiply TF32 numbers (FP32 with 10 mantissa bits; an FP32 operand is read as its TF32
// head, the low 13 mantissa bits are ignored) and add in FP32.  Every operand x is used as hi + lo, hi that
// head and lo = x - hi (exact in FP32, itself read as its 11 leading bits), and three products are
// accumulated, lo * hi + hi * lo + hi * hi: what is left out (lo * lo and the bits of lo below its 11th) is
// below 2^-19 of |p| |q| per term.
//
// Per CTA one 128 x 256 output tile and one slice of the reduction.  Warp 0: TMA producer (FP32 tiles of P
// and Q, 128 / 256 rows x 32 floats, 128-byte swizzled; these are the hi operands as they are).  Warps 2-9:
// write lo of each landed tile beside it (the same element-wise map whatever the swizzle); they are also
// the epilogue.  Warp 1: tensor-memory owner and MMA issuer (kind::tf32, N = 256, 12 MMAs of K = 8 per
// 32-wide block: at N = 128 the operand reads of the MMAs alone would take all of the shared-memory bandwidth).
// The tensor core adds each MMA's result into the accumulator with truncation, a bias of about 2^-26 of the
// running sum per MMA, so a long reduction is accumulated in chunks of 8 blocks (96 MMAs) into two
// accumulators used in turn, and the split warps add the finished chunks up in registers (FP32, round to
// nearest).  Every wait is bounded; nothing here uses TMA multicast.
#include <cuda.h>

#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"
#include "fpq_tensormap.h"

namespace fpq {

namespace {

constexpr int TM = 128, TN = 256, TK = 32;           // TK floats = one 128-byte row
constexpr int T_P_BYTES = TM * 128, T_Q_BYTES = TN * 128;
constexpr int T_RAW_BYTES = T_P_BYTES + T_Q_BYTES;
constexpr int T_STAGE_BYTES = 2 * T_RAW_BYTES;       // P | Q as loaded (read by the tensor core as their TF32 heads) | P lo | Q lo
constexpr int T_STAGES = 2;
constexpr int T_XF_W0 = 2, T_NUM_XF = 8;
constexpr int T_THREADS = 32 * (T_XF_W0 + T_NUM_XF);
constexpr int T_SCALE_BYTES = T_NUM_XF * 2 * (TN / 2) * 4;      // per epilogue warp: scales and biases of its columns (epi 2)
constexpr int T_SMEM = T_STAGES * T_STAGE_BYTES + 1024 + 256 + T_SCALE_BYTES;
constexpr int T_CHUNK = 8;                           // 32-wide blocks accumulated in tensor memory before they are added up

struct Tf32Args {
    int I, J;                  // rows of P (output rows), rows of Q (output columns)
    int kblocks;               // 32-wide blocks of the reduction
    int kb_per_split;          // blocks per slice (blockIdx.y)
    int tiles_j;
    int epi;                   // 0: C[z][i][j] = the slice's sum, row-major;  1: C[j][i] (transposed) and the sum of squares
    int passes;                // 3: full FP32 products;  1: the operands are TF32 numbers already (hi * hi is all there is)
    // epi 2: the layer's output y = sum * (x_scale * w_scale[j]) + bias[j], row-major [I][J] (howo = 0) or NCHW with
    // i = image * howo + pixel
    const float* w_scale;
    const float* bias;
    float x_scale;
    int howo;
    float* C;
    int64_t ldc, split_stride;
    double* sq_sum;
    int* status;
    uint32_t idesc;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

// D (+)= A * B on TF32 operands; acc == 0 overwrites D
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                         uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.u32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc)
        : "memory");
}

// what an FP32 number loses when the tensor core reads it as TF32 (the low 13 mantissa bits are ignored): exact
__device__ __forceinline__ float tail_tf32(float x)
{
    return x - __uint_as_float(__float_as_uint(x) & 0xffffe000u);
}

__device__ __forceinline__ float4 tail4(const float4 v)
{
    return make_float4(tail_tf32(v.x), tail_tf32(v.y), tail_tf32(v.z), tail_tf32(v.w));
}

__global__ void __launch_bounds__(T_THREADS, 1) tf32x3_gemm_kernel(const __grid_constant__ CUtensorMap tmP,
                                                                   const __grid_constant__ CUtensorMap tmQ,
                                                                   const Tf32Args g)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bars = smem_base + T_STAGES * T_STAGE_BYTES;
    const uint32_t full = bars, ready = bars + 32, empty = bars + 64, acc_full = bars + 96, acc_empty = bars + 112;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + T_STAGES * T_STAGE_BYTES + 128);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int ti = (int)blockIdx.x / g.tiles_j, tj = (int)blockIdx.x - ti * g.tiles_j;
    const int z = blockIdx.y;
    const int kb_lo = z * g.kb_per_split;
    const int kb_hi = min(g.kblocks, kb_lo + g.kb_per_split);

    if (threadIdx.x == 0) {
        for (int s = 0; s < T_STAGES; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(ready + 8 * s, T_NUM_XF);
            mbar_init(empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full + 8 * b, 1);
            mbar_init(acc_empty + 8 * b, T_NUM_XF);
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmP);
        tma_prefetch_desc(&tmQ);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), 2 * TN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            uint32_t s = 0, ph = 0;
            for (int kb = kb_lo; kb < kb_hi; ++kb) {
                if (!mbar_wait(empty + 8 * s, ph ^ 1)) { flag_status(g.status, FPQ_ERR_TIMEOUT); break; }
                mbar_expect_tx(full + 8 * s, (uint32_t)T_RAW_BYTES);
                const uint32_t st = smem_base + s * T_STAGE_BYTES;
                tma_load_2d(st, &tmP, full + 8 * s, kb * TK, ti * TM);
                tma_load_2d(st + T_P_BYTES, &tmQ, full + 8 * s, kb * TK, tj * TN);
                if (++s == T_STAGES) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            uint32_t s = 0, ph = 0, acc = 0;
            bool dead = false;
            int in_chunk = 0, chunk = 0;
            for (int kb = kb_lo; kb < kb_hi; ++kb) {
                const uint32_t buf = chunk & 1;
                if (in_chunk == 0) {
                    // a fresh accumulator: the split warps must have added up what it held two chunks ago
                    if (chunk >= 2 && !mbar_wait(acc_empty + 8 * buf, ((chunk >> 1) - 1) & 1)) { dead = true; break; }
                    tc_fence_after();
                    acc = 0;
                }
                if (!mbar_wait(ready + 8 * s, ph)) { dead = true; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + buf * TN;
                const uint32_t st = smem_base + s * T_STAGE_BYTES;
                // (the tensor core reads an FP32 operand as its TF32 head: the tiles as loaded are the hi parts)
                const uint32_t p_hi = smem_desc_lo(st), q_hi = smem_desc_lo(st + T_P_BYTES);
                const uint32_t p_lo = smem_desc_lo(st + T_RAW_BYTES), q_lo = smem_desc_lo(st + T_RAW_BYTES + T_P_BYTES);
#pragma unroll
                for (uint32_t kk = 0; kk < 4; ++kk) {
                    // 8 floats = 32 bytes per MMA: two 16-byte units further along the row
                    if (g.passes == 3) {
                        mma_tf32(d, p_lo + 2 * kk, q_hi + 2 * kk, SMEM_DESC_HI_K_SW128, g.idesc, acc);
                        mma_tf32(d, p_hi + 2 * kk, q_lo + 2 * kk, SMEM_DESC_HI_K_SW128, g.idesc, 1u);
                        acc = 1u;
                    }
                    mma_tf32(d, p_hi + 2 * kk, q_hi + 2 * kk, SMEM_DESC_HI_K_SW128, g.idesc, acc);
                    acc = 1u;
                }
                mma_commit(empty + 8 * s);          // the stage is free once these MMAs have read it
                if (++s == T_STAGES) { s = 0; ph ^= 1; }
                if (++in_chunk == T_CHUNK || kb + 1 == kb_hi) {
                    mma_commit(acc_full + 8 * buf);
                    in_chunk = 0;
                    ++chunk;
                }
            }
            if (dead)
                flag_status(g.status, FPQ_ERR_TIMEOUT);
        }
    } else {
        // ---------------- split warps, then epilogue ----------------
        const int tid = threadIdx.x - 32 * T_XF_W0;
        // as epilogue, warp w owns tensor-memory lane quarter w % 4 and half of the columns
        constexpr int HALF = TN / 2;
        const int quarter = warp & 3, half = (warp - T_XF_W0) >> 2;
        const int i = ti * TM + quarter * 32 + lane;
        float sum[HALF];
#pragma unroll
        for (int v = 0; v < HALF; ++v)
            sum[v] = 0.f;
        const int nchunks = (kb_hi - kb_lo + T_CHUNK - 1) / T_CHUNK;
        int drained = 0;
        bool dead = false;
        // adds chunk c (complete in its accumulator) to the sums and hands the accumulator back
        auto drain = [&](int c) {
            const uint32_t buf = c & 1;
            if (!mbar_wait(acc_full + 8 * buf, (c >> 1) & 1)) { dead = true; return; }
            tc_fence_after();
#pragma unroll
            for (int h = 0; h < HALF / 32; ++h) {
                uint32_t r[32];
                tmem_ld32(tmem_base + buf * TN + (uint32_t)(half * HALF + h * 32) + ((uint32_t)(quarter * 32) << 16), r);
                tmem_ld_wait();
#pragma unroll
                for (int v = 0; v < 32; ++v)
                    sum[h * 32 + v] += __uint_as_float(r[v]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0)
                mbar_arrive(acc_empty + 8 * buf);
        };
        // epi 2: the warp's own copy of x_scale * w_scale | bias of its columns, fetched before the main loop
        float* w_sc = reinterpret_cast<float*>(smem + T_STAGES * T_STAGE_BYTES + 256) + (warp - T_XF_W0) * 2 * HALF;
        if (g.epi == 2) {
#pragma unroll
            for (int q = 0; q < 2 * HALF / 32; ++q) {
                const int e = q * 32 + lane;                       // [0, HALF): scale, [HALF, 2 HALF): bias
                const int col = tj * TN + half * HALF + (e < HALF ? e : e - HALF);
                float v = 0.f;
                if (col < g.J)
                    v = e < HALF ? g.x_scale * __ldg(g.w_scale + col) : (g.bias ? __ldg(g.bias + col) : 0.f);
                w_sc[e] = v;
            }
            __syncwarp();
        }
        uint32_t s = 0, ph = 0;
        for (int kb = kb_lo; kb < kb_hi && !dead; ++kb) {
            if (!mbar_wait(full + 8 * s, ph)) { dead = true; break; }
            float4* raw = reinterpret_cast<float4*>(smem + s * T_STAGE_BYTES);
            float4* low = raw + T_RAW_BYTES / 16;
            if (g.passes == 3) {
#pragma unroll
                for (int q = 0; q < T_RAW_BYTES / 16 / (32 * T_NUM_XF); ++q) {
                    const int e = q * (32 * T_NUM_XF) + tid;
                    low[e] = tail4(raw[e]);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0)
                mbar_arrive(ready + 8 * s);
            if (++s == T_STAGES) { s = 0; ph ^= 1; }
            // half a chunk later the previous chunk's MMAs are long done: add it up now, off the critical path
            const int done = kb - kb_lo + 1;
            if (done % T_CHUNK == T_CHUNK / 2 && done / T_CHUNK > drained)
                drain(drained++);
        }
        while (!dead && drained < nchunks)
            drain(drained++);
        float sq = 0.f;
        if (!dead && kb_hi > kb_lo) {
#pragma unroll
            for (int c = 0; c < HALF / 32; ++c) {
                const int j0 = tj * TN + half * HALF + c * 32;
                if (j0 >= g.J)
                    break;
                const float* r = sum + c * 32;
                if (g.epi == 0) {
                    if (i < g.I) {
                        float* dst = g.C + (int64_t)z * g.split_stride + (int64_t)i * g.ldc + j0;
                        if ((g.ldc & 3) == 0 && j0 + 32 <= g.J) {
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                reinterpret_cast<float4*>(dst)[v] = make_float4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                        } else {
#pragma unroll
                            for (int v = 0; v < 32; ++v)
                                if (j0 + v < g.J)
                                    dst[v] = r[v];
                        }
                    }
                } else if (g.epi == 2) {
                    if (i < g.I) {
                        float o[32];
#pragma unroll
                        for (int v = 0; v < 32; ++v)
                            o[v] = fmaf(r[v], w_sc[c * 32 + v], w_sc[HALF + c * 32 + v]);
                        if (g.howo == 0) {
                            float* dst = g.C + (int64_t)i * g.ldc + j0;
                            if ((g.ldc & 3) == 0 && j0 + 32 <= g.J) {
#pragma unroll
                                for (int v = 0; v < 8; ++v)
                                    reinterpret_cast<float4*>(dst)[v] = make_float4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                            } else {
#pragma unroll
                                for (int v = 0; v < 32; ++v)
                                    if (j0 + v < g.J)
                                        dst[v] = o[v];
                            }
                        } else {
                            // NCHW: for one channel the 32 lanes write 32 consecutive pixels (of one image, mostly)
                            const int b = i / g.howo, pix = i - b * g.howo;
#pragma unroll
                            for (int v = 0; v < 32; ++v)
                                if (j0 + v < g.J)
                                    g.C[((int64_t)b * g.J + j0 + v) * g.howo + pix] = o[v];
                        }
                    }
                } else {
                    // transposed: for one column the 32 lanes write 32 consecutive floats
#pragma unroll
                    for (int v = 0; v < 32; ++v) {
                        if (j0 + v < g.J && i < g.I) {
                            const float d = r[v];
                            g.C[(int64_t)(j0 + v) * g.ldc + i] = d;
                            sq = fmaf(d, d, sq);
                        }
                    }
                }
            }
        }
        if (g.epi == 1) {
            double t = (double)sq;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0 && t != 0.0)
                atomicAdd(g.sq_sum, t);
        }
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * TN);
    }
}

// XT[k][m] = X[m][k]: X [M][K] with leading dimension ldx, XT [K][ldt] (ldt >= M).  32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) transpose_kernel(const float* __restrict__ X, int64_t ldx, int64_t M, int64_t K,
                                                        float* __restrict__ XT, int64_t ldt)
{
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t m0 = (int64_t)blockIdx.y * 32, k0 = (int64_t)blockIdx.x * 32;
#pragma unroll
    for (int r = ty; r < 32; r += 8)
        tile[r][tx] = (m0 + r < M && k0 + tx < K) ? X[(m0 + r) * ldx + k0 + tx] : 0.f;
    __syncthreads();
#pragma unroll
    for (int r = ty; r < 32; r += 8)
        if (k0 + r < K && m0 + tx < M)
            XT[(k0 + r) * ldt + m0 + tx] = tile[tx][r];
}

// rows x R floats, row-major with leading dimension ld: boxes of box_rows rows x 32 floats, zeros outside
bool encode_rows(EncodeTiledFn enc, CUtensorMap* tm, const float* base, int64_t rows, int64_t R, int64_t ld, int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)R, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {TK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tf32x3_applies(const float* P, int64_t ldp, const float* Q, int64_t ldq, int64_t I, int64_t J, int64_t R)
{
    return I >= 1 && J >= 1 && R >= 1 && I < (1 << 30) && J < (1 << 30) && R < (1ll << 35) && ldp % 4 == 0 && ldq % 4 == 0 &&
           (uintptr_t)P % 16 == 0 && (uintptr_t)Q % 16 == 0;
}

// C = P Q^T over slices of the reduction.  epi 0: slice z goes to C + z * split_stride, row-major with leading
// dimension ldc; epi 1 (splits must be 1): C[j][i] with leading dimension ldc, and *sq_sum += sum of squares.
fpq_status launch_tf32x3(const float* P, int64_t ldp, const float* Q, int64_t ldq, int64_t I, int64_t J, int64_t R,
                         int kb_per_split, int epi, float* C, int64_t ldc, int64_t split_stride, double* sq_sum,
                         cudaStream_t st, int passes, const float* w_scale, float x_scale, const float* bias, int howo)
{
    static std::mutex mu;
    static EncodeTiledFn enc = nullptr;
    static bool attr_set[64] = {};
    if (!tf32x3_applies(P, ldp, Q, ldq, I, J, R) || kb_per_split < 1 || (passes != 1 && passes != 3))
        return FPQ_ERR_UNSUPPORTED;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!enc) {
            enc = tensor_map_encoder();
            if (!enc)
                return FPQ_ERR_CUDA;
        }
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
            return FPQ_ERR_CUDA;
        if (!attr_set[dev]) {
            if (cudaFuncSetAttribute(tf32x3_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, T_SMEM) != cudaSuccess)
                return FPQ_ERR_CUDA;
            attr_set[dev] = true;
        }
    }
    CUtensorMap tmP, tmQ;
    if (!encode_rows(enc, &tmP, P, I, R, ldp, TM) || !encode_rows(enc, &tmQ, Q, J, R, ldq, TN))
        return FPQ_ERR_CUDA;
    Tf32Args g{};
    g.I = (int)I;
    g.J = (int)J;
    g.kblocks = (int)((R + TK - 1) / TK);
    g.kb_per_split = kb_per_split;
    g.tiles_j = (int)((J + TN - 1) / TN);
    g.epi = epi;
    g.passes = passes;
    g.w_scale = w_scale;
    g.x_scale = x_scale;
    g.bias = bias;
    g.howo = howo;
    g.C = C;
    g.ldc = ldc;
    g.split_stride = split_stride;
    g.sq_sum = sq_sum;
    g.status = status_word();
    if (!g.status)
        return FPQ_ERR_CUDA;
    // kind::tf32: FP32 accumulator, TF32 (format 2) on both sides, K-major, N = 256, M = 128
    g.idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
    const int splits = (g.kblocks + kb_per_split - 1) / kb_per_split;
    if ((epi == 1 || epi == 2) && splits != 1)
        return FPQ_ERR_UNSUPPORTED;
    const int64_t tiles = ((I + TM - 1) / TM) * (int64_t)g.tiles_j;
    if (tiles > 0x7fffffff || splits > 65535)
        return FPQ_ERR_SHAPE;
    dim3 grid((unsigned)tiles, (unsigned)splits);
    tf32x3_gemm_kernel<<<grid, T_THREADS, T_SMEM, st>>>(tmP, tmQ, g);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

cudaError_t launch_transpose(const float* X, int64_t ldx, int64_t M, int64_t K, float* XT, int64_t ldt, cudaStream_t st)
{
    dim3 grid((unsigned)((K + 31) / 32), (unsigned)((M + 31) / 32));
    transpose_kernel<<<grid, 256, 0, st>>>(X, ldx, M, K, XT, ldt);
    return cudaGetLastError();
}

}  // namespace fpq
