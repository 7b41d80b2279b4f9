// Rounding learning (Sec. V-B): one evaluation of the objective
//     mean((A Wq(alpha)^T - A W^T)^2) + reg * sum_i lambda(alpha_i)
// and of its gradient with respect to alpha, for a bias-free linear layer with FP32 calibration
// activations A [M][K].  The paper runs this step in FP32, so the two contractions here are FP32
// FMA contractions on the CUDA cores (register-tiled, 128 x 128 x 16 tiles), not reduced-precision
// tensor-core products.
//
//   soft_weight_kernel      E = Wq(alpha) - W and dWq/dalpha per weight; sum of lambda
//   sgemm128<true>          D = A E^T            (= Yq - Y by linearity), sum of D^2; with few output tiles the
//                           reduction is cut into slices that reduce_d_kernel adds
//   sgemm128<false>         partial sums of D^T A over slices of the M rows
//   grad_finalize_kernel    slices added in a fixed order, chain rule, optional descent update
//   harden_kernel           the inference rule: decision bit = (sigma(alpha) >= 0.5)
//   unfold_kernel           a convolution's input rows, so that the same step serves convolution weights
#include <math.h>

#include "fpq_kernels.h"

namespace fpq {

namespace {

constexpr int TILE = 128;      // output tile edge
constexpr int BK = 16;         // reduction elements per shared-memory stage
constexpr int LDS = TILE + 4;  // padded row length of a stage (floats)

// sigma(alpha), sigma (1 - sigma) and u = 2 |sigma - 0.5| = tanh(|alpha| / 2), each from expressions without
// cancellation (1 - sigma and sigma - 0.5 formed by subtraction lose most of their bits once sigma saturates,
// and the regulariser raises u to the 19th power).
struct SoftTerms {
    float sig, sp, u;
};
__device__ __forceinline__ SoftTerms soft_terms(float al)
{
    float t = expf(-fabsf(al));
    float inv = 1.0f / (1.0f + t);
    SoftTerms o;
    o.sig = al >= 0.f ? inv : t * inv;
    o.sp = t * inv * inv;
    o.u = tanhf(0.5f * fabsf(al));
    return o;
}

// Two FP32 values in one 64-bit register, and the packed multiply-add on such pairs (each half an IEEE fused
// multiply-add, round to nearest): half the issue slots of two scalar instructions.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(unsigned long long& d, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Adds one value per thread over the block and then into *dst (one atomic per block).
__device__ __forceinline__ void block_atomic_add(double v, double* dst)
{
    __shared__ double warp_part[32];
    v = warp_sum(v);
    int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0)
        warp_part[wid] = v;
    __syncthreads();
    if (wid == 0) {
        int nw = (blockDim.x + 31) >> 5;
        double s = lane < nw ? warp_part[lane] : 0.0;
        s = warp_sum(s);
        if (lane == 0)
            atomicAdd(dst, s);
    }
}

// Learned-rounding equation of Sec. V-B with the sigmoid kept soft.  One thread per weight.
__global__ void __launch_bounds__(256) soft_weight_kernel(const float* __restrict__ w, const float* __restrict__ scale,
                                                          QFormat f, const float* __restrict__ alpha,
                                                          float* __restrict__ E, float* __restrict__ DQ,
                                                          double* __restrict__ reg_sum, int64_t N, int64_t K,
                                                          int* __restrict__ status)
{
    int64_t total = N * K;
    float lam_acc = 0.f;
    const float c = __uint_as_float(f.cmax_bits);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / K;
        float g = __ldg(scale + n);
        float r = __fdiv_rn(1.0f, g);
        float wv = __ldg(w + i);
        float t = __fmul_rn(wv, r);
        float al = __ldg(alpha + i);
        SoftTerms st = soft_terms(al);
        float sig = st.sig, u = st.u;
        float u2 = u * u, u4 = u2 * u2, u8 = u4 * u4, u16 = u8 * u8;
        lam_acc += 1.0f - u16 * u4;
        if (t != t) {
            E[i] = 0.f;
            DQ[i] = 0.f;
            flag_status(status, FPQ_ERR_NAN_INPUT);
            continue;
        }
        float a = fminf(fmaxf(t, -c), c);
        int Eb = (int)((__float_as_uint(a) >> 23) & 0xffu);
        int e_eff = max(Eb - 127, 1 - f.B);                               // binade whose step applies
        float s = __uint_as_float((uint32_t)(e_eff - f.m + 127) << 23);     // step, a power of two
        float s_inv = __uint_as_float((uint32_t)(f.m - e_eff + 127) << 23);
        float fl = floorf(a * s_inv);                                       // exact: power-of-two scaling
        float pre = s * (fl + sig);
        float q = fminf(fmaxf(pre, -c), c);
        E[i] = fmaf(g, q, -wv);
        DQ[i] = (pre >= -c && pre <= c) ? g * s * st.sp : 0.f;
    }
    block_atomic_add((double)lam_acc, reg_sum);
}

// C[i][j] = sum_r P(i, r) Q(j, r) over r in [z * r_per_split, min(R, (z + 1) * r_per_split)), z = blockIdx.z,
// written to C + z * I * ldc.  RED_CONTIG: P(i, r) = P[i * ldp + r] (reduction index contiguous); otherwise
// P(i, r) = P[r * ldp + i] (output index contiguous); the same for Q.  256 threads, 8 x 8 outputs per thread,
// next stage fetched into registers while the current one is multiplied.  sq_sum (optional) receives the sum
// of the squared outputs.
template <bool RED_CONTIG>
__global__ void __launch_bounds__(256, 2) sgemm128(const float* __restrict__ P, int64_t ldp, const float* __restrict__ Q,
                                                   int64_t ldq, float* __restrict__ C, int64_t ldc, int I, int J,
                                                   int64_t R, int64_t r_per_split, double* __restrict__ sq_sum)
{
    __shared__ __align__(16) float Ps[2][BK][LDS];
    __shared__ __align__(16) float Qs[2][BK][LDS];

    const int t = threadIdx.x;
    const int i0 = blockIdx.x * TILE, j0 = blockIdx.y * TILE;
    const int64_t r_begin = (int64_t)blockIdx.z * r_per_split;
    const int64_t r_end = min(R, r_begin + r_per_split);
    C += (int64_t)blockIdx.z * I * ldc;
    const bool vec_p = (ldp % 4 == 0) && (((uintptr_t)P) % 16 == 0);
    const bool vec_q = (ldq % 4 == 0) && (((uintptr_t)Q) % 16 == 0);

    float4 pf[2], qf[2];

    // fetch one stage (16 reduction elements x 128 outputs of each operand) into registers
    auto fetch = [&](const float* __restrict__ X, int64_t ld, int x0, int X_extent, bool vec, int64_t r0, float4* out) {
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (RED_CONTIG) {
                int row = (t >> 2) + 64 * pass;
                int64_t r = r0 + (t & 3) * 4;
                int xi = x0 + row;
                if (xi < X_extent) {
                    const float* src = X + (int64_t)xi * ld + r;
                    if (vec && r + 3 < r_end) {
                        v = __ldg(reinterpret_cast<const float4*>(src));
                    } else {
                        if (r + 0 < r_end) v.x = __ldg(src + 0);
                        if (r + 1 < r_end) v.y = __ldg(src + 1);
                        if (r + 2 < r_end) v.z = __ldg(src + 2);
                        if (r + 3 < r_end) v.w = __ldg(src + 3);
                    }
                }
            } else {
                int64_t r = r0 + (t >> 5) + 8 * pass;
                int xi = x0 + (t & 31) * 4;
                if (r < r_end) {
                    const float* src = X + r * ld + xi;
                    if (vec && xi + 3 < X_extent) {
                        v = __ldg(reinterpret_cast<const float4*>(src));
                    } else {
                        if (xi + 0 < X_extent) v.x = __ldg(src + 0);
                        if (xi + 1 < X_extent) v.y = __ldg(src + 1);
                        if (xi + 2 < X_extent) v.z = __ldg(src + 2);
                        if (xi + 3 < X_extent) v.w = __ldg(src + 3);
                    }
                }
            }
            out[pass] = v;
        }
    };
    // registers -> shared memory, reduction index outermost
    auto stash = [&](float (*S)[LDS], const float4* in) {
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
            if (RED_CONTIG) {
                int row = (t >> 2) + 64 * pass;
                int r4 = (t & 3) * 4;
                S[r4 + 0][row] = in[pass].x;
                S[r4 + 1][row] = in[pass].y;
                S[r4 + 2][row] = in[pass].z;
                S[r4 + 3][row] = in[pass].w;
            } else {
                int r = (t >> 5) + 8 * pass;
                *reinterpret_cast<float4*>(&S[r][(t & 31) * 4]) = in[pass];
            }
        }
    };

    unsigned long long acc2[8][4];   // acc2[a][b] = outputs (a, 2 b) and (a, 2 b + 1) of the thread's 8 x 8
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
            acc2[a][b] = 0ull;

    const int ty = t >> 4, tx = t & 15;
    int buf = 0;
    if (r_begin < r_end) {
        fetch(P, ldp, i0, I, vec_p, r_begin, pf);
        fetch(Q, ldq, j0, J, vec_q, r_begin, qf);
        stash(Ps[0], pf);
        stash(Qs[0], qf);
    }
    __syncthreads();
    for (int64_t r0 = r_begin; r0 < r_end; r0 += BK) {
        const bool more = r0 + BK < r_end;
        if (more) {
            fetch(P, ldp, i0, I, vec_p, r0 + BK, pf);
            fetch(Q, ldq, j0, J, vec_q, r0 + BK, qf);
        }
#pragma unroll
        for (int r = 0; r < BK; ++r) {
            float4 p0 = *reinterpret_cast<const float4*>(&Ps[buf][r][ty * 4]);
            float4 p1 = *reinterpret_cast<const float4*>(&Ps[buf][r][64 + ty * 4]);
            float4 q0 = *reinterpret_cast<const float4*>(&Qs[buf][r][tx * 4]);
            float4 q1 = *reinterpret_cast<const float4*>(&Qs[buf][r][64 + tx * 4]);
            float pv[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
            unsigned long long qq[4] = {pack2(q0.x, q0.y), pack2(q0.z, q0.w), pack2(q1.x, q1.y), pack2(q1.z, q1.w)};
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                unsigned long long pp = pack2(pv[a], pv[a]);
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    fma2(acc2[a][b], pp, qq[b]);
            }
        }
        if (more) {
            stash(Ps[buf ^ 1], pf);
            stash(Qs[buf ^ 1], qf);
        }
        __syncthreads();
        buf ^= 1;
    }

    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
            unpack2(acc2[a][b], acc[a][2 * b], acc[a][2 * b + 1]);

    float sq = 0.f;
    const bool vec_c = (ldc % 4 == 0) && (((uintptr_t)C) % 16 == 0);
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        int i = i0 + (a < 4 ? ty * 4 + a : 64 + ty * 4 + (a - 4));
        if (i >= I)
            continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int j = j0 + h * 64 + tx * 4;
            float* dst = C + (int64_t)i * ldc + j;
            const float* v = &acc[a][h * 4];
            if (vec_c && j + 3 < J) {
                *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                sq += v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
            } else {
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (j + b < J) {
                        dst[b] = v[b];
                        sq += v[b] * v[b];
                    }
            }
        }
    }
    if (sq_sum)
        block_atomic_add((double)sq, sq_sum);
}

// grad = (2 / (M N)) (sum of the slices of D^T A) * dWq/dalpha + reg * dlambda/dalpha; alpha -= lr * grad when
// lr != 0.  Thread 0 of block 0 turns the sum of squares into the mean.
__global__ void __launch_bounds__(256) grad_finalize_kernel(const float* __restrict__ GP, int splits,
                                                            const float* __restrict__ DQ, float* __restrict__ alpha,
                                                            float* __restrict__ grad, double* __restrict__ loss,
                                                            int64_t total, float coef, double inv_mn, float reg, float lr)
{
    if (blockIdx.x == 0 && threadIdx.x == 0)
        loss[0] *= inv_mn;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        float g = 0.f;
        for (int z = 0; z < splits; ++z)
            g += GP[(int64_t)z * total + i];
        float al = alpha[i];
        SoftTerms st = soft_terms(al);
        float u = st.u;
        float u2 = u * u, u4 = u2 * u2, u8 = u4 * u4, u16 = u8 * u8;
        float u19 = u16 * u2 * u;
        float dlam = -40.0f * u19 * (al > 0.f ? 1.f : (al < 0.f ? -1.f : 0.f)) * st.sp;
        float gr = fmaf(coef * g, DQ[i], reg * dlam);
        grad[i] = gr;
        if (lr != 0.f)
            alpha[i] = al - lr * gr;
    }
}

// D = sum over the reduction slices of the first contraction (fixed order), and the sum of its squares.
__global__ void __launch_bounds__(256) reduce_d_kernel(const float* __restrict__ DP, int splits, float* __restrict__ D,
                                                       int64_t total, int64_t N, int64_t N4, double* __restrict__ sq_sum)
{
    float sq = 0.f;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        if (i % N4 >= N)
            continue;                                   // padding columns are never written or read
        float v = 0.f;
        for (int z = 0; z < splits; ++z)
            v += DP[(int64_t)z * total + i];
        D[i] = v;
        sq += v * v;
    }
    block_atomic_add((double)sq, sq_sum);
}

// One thread per output byte: bit k of a row = (alpha >= 0), i.e. sigma(alpha) >= 0.5 rounds up.
__global__ void __launch_bounds__(256) harden_kernel(const float* __restrict__ alpha, int64_t N, int64_t K,
                                                     int64_t row_bytes, uint8_t* __restrict__ bits)
{
    int64_t total = N * row_bytes;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / row_bytes, b = i - n * row_bytes;
        uint32_t v = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int64_t k = b * 8 + j;
            if (k < K && alpha[n * K + k] >= 0.f)
                v |= 1u << j;
        }
        bits[i] = (uint8_t)v;
    }
}

// Input rows of a convolution written out: row (b, oy, ox), column (c, r, s) in the weight's own [C][R][S]
// order, zero where the tap falls into the padding.  One thread per output element (writes coalesced).
__global__ void __launch_bounds__(256) unfold_kernel(const float* __restrict__ x, int C, int H, int W, int R, int S,
                                                     int pad, int stride, int Ho, int Wo, int64_t total,
                                                     float* __restrict__ rows)
{
    const int64_t K = (int64_t)C * R * S;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t m = i / K;
        int k = (int)(i - m * K);
        int s = k % S, r = (k / S) % R, c = k / (S * R);
        int ox = (int)(m % Wo), oy = (int)((m / Wo) % Ho);
        int64_t b = m / ((int64_t)Wo * Ho);
        int iy = oy * stride - pad + r, ix = ox * stride - pad + s;
        float v = 0.f;
        if (iy >= 0 && iy < H && ix >= 0 && ix < W)
            v = __ldg(x + ((b * C + c) * H + iy) * W + ix);
        rows[i] = v;
    }
}

int grid_for(int64_t total)
{
    int64_t blocks = (total + 255) / 256;
    return (int)(blocks < 1 ? 1 : (blocks > 148 * 16 ? 148 * 16 : blocks));
}

struct Plan {
    int64_t N4;
    int splits1;            // slices of K in the first contraction (1 = written straight to D)
    int64_t k_per_split;
    int splits;             // slices of M in the second contraction
    int64_t r_per_split;
    size_t off_E, off_DQ, off_D, off_DP, off_GP, bytes;
    // tensor-core route (K a multiple of 4): A^T and D^T with rows of Mp floats, slices of 32-wide blocks of M
    int64_t Mp;
    int kb_per_split_tc, splits_tc;
    int kb_per_split1_tc, splits1_tc;       // first contraction: sliced too when it has few output tiles
    size_t off_AT, off_DT;
};

// As many slices of a reduction of length R as still fit into one wave of two resident blocks per SM (one more
// would add a second, nearly empty wave), each at least 128 long.
void slice(int64_t tiles, int64_t R, int* splits, int64_t* per)
{
    int64_t want = (2 * 148) / tiles;
    int64_t cap = (R + 127) / 128;
    int64_t s = want < cap ? want : cap;
    s = s < 1 ? 1 : (s > 64 ? 64 : s);
    *per = round_up((R + s - 1) / s, BK);
    *splits = (int)((R + *per - 1) / *per);
}

Plan make_plan(int64_t M, int64_t N, int64_t K)
{
    Plan p;
    p.N4 = round_up(N, 4);
    slice(((N + TILE - 1) / TILE) * ((K + TILE - 1) / TILE), M, &p.splits, &p.r_per_split);
    int64_t tiles1 = ((M + TILE - 1) / TILE) * ((N + TILE - 1) / TILE);
    p.splits1 = 1;
    p.k_per_split = K;
    if (tiles1 < 148)
        slice(tiles1, K, &p.splits1, &p.k_per_split);
    size_t o = 0;
    p.off_E = o;
    o += (size_t)round_up(N * K * 4, 256);
    p.off_DQ = o;
    o += (size_t)round_up(N * K * 4, 256);
    p.off_D = o;
    o += (size_t)round_up(M * p.N4 * 4, 256);
    {
        const int64_t tiles1 = ((M + 127) / 128) * ((N + 255) / 256);       // 128 x 256 output tiles
        const int64_t kblocks = (K + 31) / 32;
        p.kb_per_split1_tc = (int)kblocks;
        p.splits1_tc = 1;
        if (tiles1 * 2 <= 148 && kblocks >= 16) {
            int64_t per = (kblocks + 148 / tiles1 - 1) / (148 / tiles1);
            per = per < 8 ? 8 : per;
            p.kb_per_split1_tc = (int)per;
            p.splits1_tc = (int)((kblocks + per - 1) / per);
        }
    }
    p.off_DP = o;
    {
        const int slices = p.splits1 > p.splits1_tc ? p.splits1 : p.splits1_tc;
        if (slices > 1)
            o += (size_t)round_up((int64_t)slices * M * p.N4 * 4, 256);
    }
    // second contraction on the tensor cores: one CTA per SM, so about 148 / tiles slices of at least 4 blocks
    p.Mp = round_up(M, 4);
    {
        const int64_t tiles2 = ((N + 127) / 128) * ((K + 255) / 256);       // 128 x 256 output tiles
        const int64_t kblocks = (M + 31) / 32;
        int64_t want = 148 / tiles2;
        want = want < 1 ? 1 : (want > 64 ? 64 : want);
        int64_t per = (kblocks + want - 1) / want;
        per = per < 4 ? 4 : per;
        p.kb_per_split_tc = (int)per;
        p.splits_tc = (int)((kblocks + per - 1) / per);
    }
    p.off_GP = o;
    o += (size_t)round_up((int64_t)(p.splits > p.splits_tc ? p.splits : p.splits_tc) * N * K * 4, 256);
    p.off_AT = o;
    o += (size_t)round_up(K * p.Mp * 4, 256);
    p.off_DT = o;
    o += (size_t)round_up(N * p.Mp * 4, 256);
    p.bytes = o;
    return p;
}

}  // namespace

size_t round_learn_workspace_bytes(int64_t M, int64_t N, int64_t K) { return make_plan(M, N, K).bytes; }

fpq_status launch_round_learn(const float* w, const float* scale, const QFormat& f, float* alpha, const float* a,
                              int64_t M, int64_t N, int64_t K, float reg, float lr, float* grad, double* loss,
                              void* workspace, cudaStream_t st)
{
    Plan p = make_plan(M, N, K);
    char* ws = (char*)workspace;
    float* E = (float*)(ws + p.off_E);
    float* DQ = (float*)(ws + p.off_DQ);
    float* D = (float*)(ws + p.off_D);
    float* DP = (float*)(ws + p.off_DP);
    float* GP = (float*)(ws + p.off_GP);
    int* status = status_word();
    if (!status)
        return FPQ_ERR_CUDA;
    if (cudaMemsetAsync(loss, 0, 2 * sizeof(double), st) != cudaSuccess)
        return FPQ_ERR_CUDA;
    soft_weight_kernel<<<grid_for(N * K), 256, 0, st>>>(w, scale, f, alpha, E, DQ, loss + 1, N, K, status);
    double inv_mn = 1.0 / ((double)M * (double)N);
    if (tf32x3_applies(a, K, E, K, M, N, K) && M <= (1 << 21) && N <= (1 << 21) && K <= (1 << 21)) {
        // Both contractions on the tensor cores (three TF32 products per FP32 product): D^T = (A E^T)^T is written
        // transposed by the first one's epilogue and A^T by a transpose kernel, so that the second one, D^T A,
        // again reduces over the contiguous index of both operands.
        float* AT = (float*)(ws + p.off_AT);
        float* DT = (float*)(ws + p.off_DT);
        if (launch_transpose(a, K, M, K, AT, p.Mp, st) != cudaSuccess)
            return FPQ_ERR_CUDA;
        fpq_status s1;
        if (p.splits1_tc == 1) {
            s1 = launch_tf32x3(a, K, E, K, M, N, K, p.kb_per_split1_tc, 1, DT, p.Mp, 0, loss, st);
        } else {
            // few output tiles and a long reduction: slices of it, added up in a fixed order, then transposed
            s1 = launch_tf32x3(a, K, E, K, M, N, K, p.kb_per_split1_tc, 0, DP, p.N4, M * p.N4, nullptr, st);
            if (s1 == FPQ_OK) {
                reduce_d_kernel<<<grid_for(M * p.N4), 256, 0, st>>>(DP, p.splits1_tc, D, M * p.N4, N, p.N4, loss);
                if (launch_transpose(D, p.N4, M, N, DT, p.Mp, st) != cudaSuccess)
                    return FPQ_ERR_CUDA;
            }
        }
        if (s1 != FPQ_OK)
            return s1;
        s1 = launch_tf32x3(DT, p.Mp, AT, p.Mp, N, K, M, p.kb_per_split_tc, 0, GP, K, N * K, nullptr, st);
        if (s1 != FPQ_OK)
            return s1;
        grad_finalize_kernel<<<grid_for(N * K), 256, 0, st>>>(GP, p.splits_tc, DQ, alpha, grad, loss, N * K,
                                                              (float)(2.0 * inv_mn), inv_mn, reg, lr);
        return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
    }
    dim3 g1((unsigned)((M + TILE - 1) / TILE), (unsigned)((N + TILE - 1) / TILE), (unsigned)p.splits1);
    if (p.splits1 == 1) {
        sgemm128<true><<<g1, 256, 0, st>>>(a, K, E, K, D, p.N4, (int)M, (int)N, K, K, loss);
    } else {
        sgemm128<true><<<g1, 256, 0, st>>>(a, K, E, K, DP, p.N4, (int)M, (int)N, K, p.k_per_split, nullptr);
        reduce_d_kernel<<<grid_for(M * p.N4), 256, 0, st>>>(DP, p.splits1, D, M * p.N4, N, p.N4, loss);
    }
    dim3 g2((unsigned)((N + TILE - 1) / TILE), (unsigned)((K + TILE - 1) / TILE), (unsigned)p.splits);
    sgemm128<false><<<g2, 256, 0, st>>>(D, p.N4, a, K, GP, K, (int)N, (int)K, M, p.r_per_split, nullptr);
    grad_finalize_kernel<<<grid_for(N * K), 256, 0, st>>>(GP, p.splits, DQ, alpha, grad, loss, N * K,
                                                          (float)(2.0 * inv_mn), inv_mn, reg, lr);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

fpq_status launch_round_harden(const float* alpha, int64_t N, int64_t K, uint8_t* bits, cudaStream_t st)
{
    int64_t row_bytes = (K + 7) / 8;
    if (N * row_bytes == 0)
        return FPQ_OK;
    harden_kernel<<<grid_for(N * row_bytes), 256, 0, st>>>(alpha, N, K, row_bytes, bits);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

// C[i][j] = sum_r P[i][r] Q[j][r] (both operands with the reduction index contiguous), FP32 multiply-adds.
fpq_status launch_sgemm_nt(const float* P, int64_t ldp, const float* Q, int64_t ldq, float* C, int64_t ldc, int64_t I,
                           int64_t J, int64_t R, cudaStream_t st)
{
    if (I == 0 || J == 0)
        return FPQ_OK;
    dim3 g((unsigned)((I + TILE - 1) / TILE), (unsigned)((J + TILE - 1) / TILE), 1);
    sgemm128<true><<<g, 256, 0, st>>>(P, ldp, Q, ldq, C, ldc, (int)I, (int)J, R, R, nullptr);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

fpq_status launch_unfold(const float* x, int B, int C, int H, int W, int R, int S, int pad, int stride, int Ho, int Wo,
                         float* rows, cudaStream_t st)
{
    int64_t total = (int64_t)B * Ho * Wo * C * R * S;
    if (total == 0)
        return FPQ_OK;
    unfold_kernel<<<grid_for(total), 256, 0, st>>>(x, C, H, W, R, S, pad, stride, Ho, Wo, total, rows);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq
