// Low-bit contraction on the 5th-generation tensor cores: TMA-fed tcgen05.mma
// (kind::f8f6f4, E4M3 activations x E4M3 or E2M1 weights, FP32 accumulate in
// tensor memory) with the dequantize + bias epilogue.  One persistent kernel serves
// the linear layer and the implicit-GEMM convolution.
//
// A CTA (one per SM) walks 128 x BN output tiles.  Warp 0 issues TMA loads into two
// shared-memory rings (activations, weights), warp 1 owns tensor memory and issues
// the MMAs into one of two accumulators, warps 2-9 drain the other accumulator
// (scale, bias, FP32 stores), so a tile's epilogue overlaps the next tile's main loop.
//
// The reduction of a tile is a list of blocks, block j = (128-wide chunk cc, tap), each
// 4 MMAs of K = 32.  Activation operand, three addressing modes:
//   ROWS  linear: 128 rows of [M][Ca] codes per chunk;
//   FLAT  stride-1 convolution on the zero-framed channels-last codes
//         [B][Hp][Wp][Ca] seen as one list of pixels: output position q reads input
//         positions q + r*Wp + s, so one load of 128 + (R-1)*Wp + (S-1) pixel rows per
//         chunk serves all R*S taps through matrix descriptors whose start address is
//         moved by whole 128-byte rows;
//   TAPS  any stride: one 4-D box (channels, x, y, image) per block.
// A ring stage carries the data of several blocks (one barrier handshake per stage);
// weights whose whole reduction fits in shared memory stay resident across row tiles, or a
// row tile's activation panel stays resident across its column tiles.
//
// Layers with few tiles and a long reduction run as thread-block clusters: the CTAs of a
// cluster reduce disjoint chunk ranges of one tile and add their partial sums through
// distributed shared memory.  A layer whose input is two concatenated tensors with their own
// scales keeps one accumulator per tensor (or gives each tensor its own CTAs of the cluster).
#include <cuda.h>

#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"
#include "fpq_tensormap.h"

namespace fpq {

constexpr int BM = 128;        // output rows per tile (TMEM lanes)
constexpr int BK = 128;        // reduction elements per block (one 128-byte swizzled row)
// Warp roles.  Plain form: producer, MMA issuer, 8 epilogue warps (two per TMEM lane quarter,
// each half of the columns).  Fused form: producer, MMA issuer, 4 epilogue warps and 16
// transform warps that quantize FP32 activations into the A ring - the conversion is bound by
// instruction issue, so it gets most of the SM's warps.
constexpr int NUM_XFORM_WARPS = 16;
__host__ __device__ constexpr int epi_warps(bool fused) { return fused ? 4 : 8; }
__host__ __device__ constexpr int num_threads(bool fused)
{
    return 64 + 32 * epi_warps(fused) + (fused ? 32 * NUM_XFORM_WARPS + 32 : 0);   // + one L2-prefetch warp
}
constexpr int SMEM_BUDGET = 227 * 1024;   // the most dynamic shared memory a CTA can have on sm_100

// MODE_FLAT2 is FLAT with two row tiles per unit; it has its own instantiation because the kernels are
// sensitive to code size (the extra path cost the plain FLAT kernel 7 us when it was a run-time branch)
enum { MODE_ROWS = 0, MODE_FLAT = 1, MODE_TAPS = 2, MODE_FLAT2 = 3 };

struct GemmArgs {
    int mode;
    int64_t M;                 // ROWS: rows; FLAT: framed pixels B*Hp*Wp
    int N;
    int cchunks;               // 128-wide chunks of the reduction per tap
    int taps, S, stride;
    int nblk;                  // blocks per tile = cchunks * taps
    int Wp, HpWp;              // framed geometry
    FastDiv div_HpWp, div_Wp, div_tiles, div_Wt, div_Ht, div_tx, div_ty;
    int Wt, Ht, Bt;            // TAPS: tile of Wt * Ht * Bt = 128 output pixels
    int tiles_x, tiles_y;
    int Ho, Wo, B;
    int m_tiles, n_tiles;
    int m_fastest;             // tile order: consecutive tiles share the column tile
    // activation ring: a stage holds the data of a_span consecutive blocks
    int a_boxes, a_box_rows;   // one chunk load = a_boxes TMA boxes of a_box_rows pixel rows
    int a_chunk_bytes, a_span, a_stage_bytes, a_stages;
    // weight ring: a stage holds b_span consecutive blocks; resident = the whole reduction,
    // reloaded only when the column tile changes
    int b_span, b_stage_bytes, b_stages, b_resident;
    // one weight load covers b_box_t taps x b_box_c chunks of the column tile (a TMA load costs its SM about 400
    // cycles whatever its size): b_box_t > 1 inside a chunk's taps, b_box_c > 1 over chunks of a tap-less layer
    int b_box_t, b_box_c;
    int a_box_c;               // row-major activations: one load covers the a_box_c chunks of a stage (1 = one per chunk)
    int y_tma;                 // row-major output leaves through TMA stores
    int vec_scale;             // w_scale / bias are 16-byte aligned
    int stage_scales;          // x_scale * w_scale[n] and bias[n] of all N columns sit in shared memory
    int contiguous;            // tile order: 1 = every CTA walks a contiguous range, 0 = CTAs interleave
    int a_resident;            // a row tile's whole activation panel stays in the ring while the CTA walks its column tiles
    int ksplit;                // > 1: the CTAs of a cluster of this size share one output tile, each reducing a range of chunks
    // input of two concatenated tensors: chunks [0, seg_chunk) carry x_scale and are shared out over the
    // cluster's first seg_ranks CTAs, the others carry x_scale2 and go to the remaining CTAs; 0 = one tensor
    int seg_chunk, seg_ranks;
    float x_scale2;
    int seg_acc;               // two tensors without a cluster: each has its own accumulator, the epilogue joins them
    int pair;                  // a tile unit is two consecutive row tiles (256 rows) that share every weight stage;
                               // m_tiles then counts pairs
    uint32_t a_chunk_tx, b_block_tx;   // bytes one load reports to its barrier
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
    int* status;
    uint32_t idesc;
    int wait_prior_grid;       // launched with programmatic stream serialization behind the quantize kernel
    // fused form: the FP32 activations themselves (NCHW for FLAT, [M][K] for ROWS)
    const float* x;
    float rinv;                // 1.0f / x_scale
    int C, H, W, pad;          // channels (ROWS: K), image size, zero padding
};

// Fused activation-quantize prologue, NCHW source: one 128-channel chunk of the rows
// [q0, q0 + rows) of the framed pixel list, written as E4M3 codes in the K-major,
// 128-byte-swizzled layout the MMA reads.  Warp tw owns channels [16 (tw % 8), +16) of every other 32-row batch; its
// lanes walk the pixel rows, so global loads are coalesced along x and each thread ends
// with one 16-byte store per row (8 consecutive rows hit 8 different 16-byte columns: no
// bank conflicts).  Frame positions and channels past C are code 0.  The loads of the next
// row are issued before the current one is converted.
struct NchwRows {
    const GemmArgs& g;
    uint32_t q0;
    int rows, cg, HW;
    // source address of channel cg at pixel row i, or nullptr for a frame / out-of-range row
    __device__ __forceinline__ const float* src(int i) const
    {
        const uint32_t f = q0 + (uint32_t)i;
        if (i >= rows || (int64_t)f >= g.M || cg >= g.C)
            return nullptr;
        const uint32_t b = fdiv(f, g.div_HpWp);
        const uint32_t rem = f - b * (uint32_t)g.HpWp;
        const uint32_t yp = fdiv(rem, g.div_Wp);
        const int y = (int)yp - g.pad, x = (int)(rem - yp * (uint32_t)g.Wp) - g.pad;
        if ((unsigned)y >= (unsigned)g.H || (unsigned)x >= (unsigned)g.W)
            return nullptr;
        return g.x + ((int64_t)(b * (uint32_t)g.C + (uint32_t)cg) * g.H + y) * g.W + x;
    }
    __device__ __forceinline__ void load(float (&a)[16], const float* p) const
    {
        if (cg + 16 <= g.C) {
#pragma unroll
            for (int q = 0; q < 16; ++q)
                a[q] = __ldcg(p + (int64_t)q * HW);
        } else {
#pragma unroll
            for (int q = 0; q < 16; ++q)
                a[q] = (cg + q < g.C) ? __ldcg(p + (int64_t)q * HW) : 0.f;
        }
    }
};

// Sixteen codes for the MMA operand.  Unlike codes that are stored, a minus zero may stay:
// as an operand it only ever contributes a signed zero to the sum.  NaN still becomes code 0.
__device__ __forceinline__ uint32_t e4m3x4_operand(float t0, float t1, float t2, float t3, bool& nan)
{
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(t1), "f"(t0));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(t3), "f"(t2));
    const uint32_t v = (uint32_t)lo | ((uint32_t)hi << 16);
    const uint32_t nan_bytes = ((v & 0x7f7f7f7fu) + 0x01010101u) & 0x80808080u;
    if (nan_bytes) {
        nan = true;
        return v & ~((nan_bytes >> 7) * 0xffu);
    }
    return v;
}

__device__ __forceinline__ uint4 e4m3x16(const float (&a)[16], float r, bool& nan)
{
    uint4 v;
    v.x = e4m3x4_operand(__fmul_rn(a[0], r), __fmul_rn(a[1], r), __fmul_rn(a[2], r), __fmul_rn(a[3], r), nan);
    v.y = e4m3x4_operand(__fmul_rn(a[4], r), __fmul_rn(a[5], r), __fmul_rn(a[6], r), __fmul_rn(a[7], r), nan);
    v.z = e4m3x4_operand(__fmul_rn(a[8], r), __fmul_rn(a[9], r), __fmul_rn(a[10], r), __fmul_rn(a[11], r), nan);
    v.w = e4m3x4_operand(__fmul_rn(a[12], r), __fmul_rn(a[13], r), __fmul_rn(a[14], r), __fmul_rn(a[15], r), nan);
    return v;
}

__device__ __forceinline__ void fill_chunk_nchw(const GemmArgs& g, uint8_t* dst, uint32_t q0, int rows, int c_base,
                                                int tw, int lane, bool& nan)
{
    const int cgrp = tw & 7;
    const NchwRows R{g, q0, rows, c_base + cgrp * 16, g.H * g.W};
    const uint4 zero = make_uint4(0, 0, 0, 0);
    float a[16], b[16];
    int i = lane + 32 * (tw >> 3);
    const float* pa = R.src(i);
    if (pa)
        R.load(a, pa);
    while (i < rows) {
        const int i2 = i + 64;
        const float* pb = R.src(i2);
        if (pb)
            R.load(b, pb);
        *reinterpret_cast<uint4*>(dst + i * 128 + ((cgrp ^ (i & 7)) << 4)) = pa ? e4m3x16(a, g.rinv, nan) : zero;
        i = i2 + 64;
        pa = R.src(i);
        if (pa)
            R.load(a, pa);
        if (i2 < rows)
            *reinterpret_cast<uint4*>(dst + i2 * 128 + ((cgrp ^ (i2 & 7)) << 4)) = pb ? e4m3x16(b, g.rinv, nan) : zero;
    }
}

// The same for a row-major [M][K] source: 8 consecutive threads read the 128 reduction
// elements of one row (512 contiguous bytes), a warp covers 4 rows per pass.
__device__ __forceinline__ void fill_chunk_rows(const GemmArgs& g, uint8_t* dst, int64_t m0, int k_base, int tid,
                                                bool& nan)
{
    const bool vec = (g.C % 4) == 0;
#pragma unroll 2
    for (int it = 0; it < (BM * 8) / (32 * NUM_XFORM_WARPS); ++it) {
        const int idx = it * (32 * NUM_XFORM_WARPS) + tid;
        const int i = idx >> 3, j = idx & 7;
        const int64_t m = m0 + i;
        const int k = k_base + 16 * j;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m < g.M && k < g.C) {
            const float* p = g.x + m * g.C + k;
            float a[16];
            if (vec && k + 16 <= g.C) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 t = __ldcg(reinterpret_cast<const float4*>(p) + q);
                    a[4 * q] = t.x; a[4 * q + 1] = t.y; a[4 * q + 2] = t.z; a[4 * q + 3] = t.w;
                }
            } else {
#pragma unroll
                for (int q = 0; q < 16; ++q)
                    a[q] = (k + q < g.C) ? __ldcg(p + q) : 0.f;
            }
            v = e4m3x16(a, g.rinv, nan);
        }
        *reinterpret_cast<uint4*>(dst + i * 128 + ((j ^ (i & 7)) << 4)) = v;
    }
}

// FUSED = false: the activation operand is read as codes (TMA, written by a quantize kernel).
// FUSED = true : 16 more warps read the FP32 activations and quantize them straight into the
//                activation ring, so the codes never exist in global memory.
template <int BN, bool FUSED, int MODE>
__global__ void __launch_bounds__(num_threads(FUSED), 1) fpq_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                  const __grid_constant__ CUtensorMap tmB,
                                                                  const __grid_constant__ CUtensorMap tmY,
                                                                  const GemmArgs g)
{
    constexpr int NUM_EPI_WARPS = epi_warps(FUSED);
    constexpr uint32_t B_BLOCK_BYTES = BN * BK;          // smem footprint (4-bit codes sit in 16-byte containers)
    constexpr uint32_t BSTEP = B_BLOCK_BYTES / 16;       // the same in descriptor units
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    // layout: [A ring][B ring][epilogue staging for TMA stores, 2 x 4 KiB per warp][barriers + flags]
    //         [x_scale * w_scale | bias, all N columns, when they fit]
    const uint32_t a_ring = smem_base;
    const uint32_t b_ring = a_ring + g.a_stages * g.a_stage_bytes;
    const uint32_t ctl_off = g.a_stages * g.a_stage_bytes + g.b_stages * g.b_stage_bytes;
    const uint32_t bars = smem_base + ctl_off + (g.y_tma ? NUM_EPI_WARPS * 8192 : 0);
    // barrier slots (8 bytes each): a_full[8] a_empty[8] b_full[8] b_empty[8] acc_full[2] acc_empty[2]
    const uint32_t a_full = bars, a_empty = bars + 64, b_full = bars + 128, b_empty = bars + 192;
    const uint32_t acc_full = bars + 256, acc_empty = bars + 272;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (bars - smem_base) + 288);
    const int n_pad = (g.N + 31) & ~31;
    float* s_scale = reinterpret_cast<float*>(smem + (bars - smem_base) + 512);   // [n_pad], if staged
    float* s_bias = s_scale + n_pad;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = g.m_tiles * g.n_tiles;
    // every CTA walks a contiguous range of the tile list, so consecutive tiles share the row tile
    // (or, in column-tile-major order, the column tile) and its resident operand
    // (a resident operand that several tiles share); otherwise the CTAs interleave, so that at any time the whole GPU works on one
    // compact region of the activations and of the output
    // Split reduction (few tiles, long reduction): a cluster of ksplit CTAs owns one tile, CTA k of the
    // cluster reduces the chunks [c_lo, c_hi) into its own accumulator; the partial sums meet in shared
    // memory after the role loops below.
    // two row tiles per unit: only the plain form of the stride-1 convolution uses it
    constexpr bool pair = MODE == MODE_FLAT2;
    constexpr bool FLATM = MODE == MODE_FLAT || MODE == MODE_FLAT2;
    const int tile_rows = pair ? 2 * BM : BM;
    const int ksplit = g.ksplit;
    const uint32_t krank = ksplit > 1 ? cluster_rank() : 0u;
    int c_lo = 0, c_hi = g.cchunks;
    if (ksplit > 1 && !g.seg_chunk) {
        c_lo = (int)krank * g.cchunks / ksplit;
        c_hi = ((int)krank + 1) * g.cchunks / ksplit;
    } else if (ksplit > 1) {
        // a CTA's range never crosses from one input tensor into the other: their scales differ
        const int first = (int)krank < g.seg_ranks;
        const int k = first ? (int)krank : (int)krank - g.seg_ranks;
        const int ranks = first ? g.seg_ranks : ksplit - g.seg_ranks;
        const int base = first ? 0 : g.seg_chunk, len = first ? g.seg_chunk : g.cchunks - g.seg_chunk;
        c_lo = base + k * len / ranks;
        c_hi = base + (k + 1) * len / ranks;
    }
    const int nblk = (c_hi - c_lo) * g.taps;
    const int t_lo = ksplit > 1 ? (int)blockIdx.x / ksplit
                                : g.contiguous ? (int)((int64_t)blockIdx.x * total_tiles / gridDim.x) : (int)blockIdx.x;
    const int t_hi = ksplit > 1 ? t_lo + 1
                                : g.contiguous ? (int)((int64_t)(blockIdx.x + 1) * total_tiles / gridDim.x) : total_tiles;
    const int t_step = (ksplit > 1 || g.contiguous) ? 1 : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(a_full + 8 * s, FUSED ? NUM_XFORM_WARPS : 1);
            mbar_init(a_empty + 8 * s, 1);
            mbar_init(b_full + 8 * s, 1);
            mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, NUM_EPI_WARPS);      // one arrival per epilogue warp
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        if (g.y_tma)
            tma_prefetch_desc(&tmY);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), (g.seg_acc || pair) ? 4 * BN : 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // tile index -> (row tile, column tile)
    auto decode_tile = [&](int t, int& mt, int& nt) {
        const int q = (int)fdiv((uint32_t)t, g.div_tiles);
        if (g.m_fastest) { nt = q; mt = t - q * g.m_tiles; }
        else             { mt = q; nt = t - q * g.n_tiles; }
    };

    // row `row` of row tile mt -> its address in y (column 0), the column stride, and whether it exists
    auto row_target = [&](int mt, int row, bool& row_valid, float*& yrow, int64_t& nstride) {
        if (MODE == MODE_ROWS) {
            const int64_t m = (int64_t)mt * BM + row;
            row_valid = m < g.M;
            nstride = 1;
            yrow = g.y + m * g.N;
        } else {
            int ox, oy, b;
            if (FLATM) {
                const uint32_t q = (uint32_t)mt * BM + row;
                b = (int)fdiv(q, g.div_HpWp);
                const uint32_t rem = q - (uint32_t)b * g.HpWp;
                oy = (int)fdiv(rem, g.div_Wp);
                ox = (int)rem - oy * g.Wp;
            } else {
                const uint32_t r1 = fdiv((uint32_t)mt, g.div_tx);
                const int x0 = (mt - (int)r1 * g.tiles_x) * g.Wt;
                const uint32_t r2 = fdiv(r1, g.div_ty);
                const int y0 = ((int)r1 - (int)r2 * g.tiles_y) * g.Ht;
                const int b0 = (int)r2 * g.Bt;
                const uint32_t q1 = fdiv((uint32_t)row, g.div_Wt);
                ox = x0 + (row - (int)q1 * g.Wt);
                const uint32_t q2 = fdiv(q1, g.div_Ht);
                oy = y0 + ((int)q1 - (int)q2 * g.Ht);
                b = b0 + (int)q2;
            }
            row_valid = ox < g.Wo && oy < g.Ho && b < g.B;
            nstride = (int64_t)g.Ho * g.Wo;
            yrow = g.y + ((int64_t)b * g.N * g.Ho + oy) * g.Wo + ox;   // + n * Ho * Wo
        }
    };

    // Every wait below is bounded; a role whose wait expires records FPQ_ERR_TIMEOUT and
    // leaves its loop, the other roles then run into their own limits and follow.
    if (warp == 0) {
        // ---------------- TMA producer (one thread; its loops never divide) ----------------
        if (elect_one()) {
            uint32_t sa = 0, pa = 0, sb = 0, pb = 0;   // stage and phase of the next load per ring
            uint32_t na = 0, nb = 0;                   // stages issued (for the abort path)
            int resident_nt = -1, resident_mt = -1;
            bool dead = false;
            bool prior_done = !g.wait_prior_grid;
            // `count` consecutive weight blocks (chunk c2, tap t2 onward; taps fastest) of column tile n0, one load per box
            const int b_box = g.b_box_t * g.b_box_c;
            auto load_weights = [&](uint32_t dst, uint32_t bar, int n0, int c2, int t2, int count) {
                for (int l = 0; l < count; l += b_box, dst += b_box * B_BLOCK_BYTES) {
                    tma_load_4d(dst, &tmB, bar, 0, n0, t2, c2);
                    t2 += g.b_box_t;
                    if (t2 >= g.taps) { t2 = 0; c2 += g.b_box_c; }
                }
            };
            for (int t = t_lo; t < t_hi && !dead; t += t_step) {
                int mt, nt;
                decode_tile(t, mt, nt);
                const int n0 = nt * BN;
                int x0 = 0, y0 = 0, b0 = 0;
                if (MODE == MODE_TAPS) {
                    const uint32_t r1 = fdiv((uint32_t)mt, g.div_tx);
                    x0 = (mt - (int)r1 * g.tiles_x) * g.Wt * g.stride;
                    const uint32_t r2 = fdiv(r1, g.div_ty);
                    y0 = ((int)r1 - (int)r2 * g.tiles_y) * g.Ht * g.stride;
                    b0 = (int)r2 * g.Bt;
                }
                const bool load_b = !(g.b_resident && resident_nt == nt);
                resident_nt = nt;
                const bool load_a = !(g.a_resident && resident_mt == mt);
                resident_mt = mt;
                int cc = c_lo, tap = 0, r = 0, sx = 0; // block j = (cc, tap), tap = (r, sx)
                int ja = 0, jb = 0;                    // position inside the current A / B stage
                bool early_b = false;
                for (int j = 0; j < nblk; ++j) {
                    if (jb == 0 && load_b && !prior_done && g.b_resident) {
                        // the weights do not depend on the kernel in front: fetch them before waiting for it
                        if (!mbar_wait(b_empty + 8 * sb, pb ^ 1)) { dead = true; break; }
                        mbar_expect_tx(b_full + 8 * sb, (uint32_t)g.nblk * g.b_block_tx);
                        load_weights(b_ring + sb * g.b_stage_bytes, b_full + 8 * sb, n0, 0, 0, g.nblk);
                        ++nb;
                        if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                        early_b = true;
                    }
                    if (!prior_done) {
                        // the activation codes are written by the preceding grid
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        prior_done = true;
                    }
                    if (ja == 0 && !FUSED && load_a) {
                        // activation stage: the data of the next a_span blocks
                        if (!mbar_wait(a_empty + 8 * sa, pa ^ 1)) { dead = true; break; }
                        const int nblocks = min(g.a_span, nblk - j);
                        const int nloads = (MODE == MODE_TAPS) ? nblocks : nblocks / g.taps;
                        const bool a_wide = MODE == MODE_ROWS && g.a_box_c > 1;
                        mbar_expect_tx(a_full + 8 * sa, (uint32_t)(a_wide ? g.a_box_c : nloads) * g.a_chunk_tx);
                        uint32_t dst = a_ring + sa * g.a_stage_bytes;
                        if (a_wide) {
                            // all chunks of the stage in one box (chunks past the last one read as zeros)
                            tma_load_4d(dst, &tmA, a_full + 8 * sa, 0, mt * tile_rows, cc, 0);
                        } else if (MODE == MODE_TAPS) {
                            int c2 = cc, t2 = tap, r2 = r, s2 = sx;
                            for (int l = 0; l < nloads; ++l, dst += g.a_chunk_bytes) {
                                tma_load_4d(dst, &tmA, a_full + 8 * sa, c2 * BK, x0 + s2, y0 + r2, b0);
                                if (++s2 == g.S) { s2 = 0; ++r2; }
                                if (++t2 == g.taps) { t2 = 0; r2 = 0; s2 = 0; ++c2; }
                            }
                        } else {
                            for (int l = 0; l < nloads; ++l, dst += g.a_chunk_bytes)
                                for (int bx = 0; bx < g.a_boxes; ++bx)
                                    tma_load_4d(dst + bx * g.a_box_rows * 128, &tmA, a_full + 8 * sa, (cc + l) * BK,
                                                mt * tile_rows + bx * g.a_box_rows, 0, 0);
                        }
                        ++na;
                        if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                    }
                    if (jb == 0 && load_b && !early_b) {
                        if (!mbar_wait(b_empty + 8 * sb, pb ^ 1)) { dead = true; break; }
                        // (a box that reaches past the last chunk is filled with zeros there and reports its full size)
                        const int nblocks = (min(g.b_span, nblk - j) + b_box - 1) / b_box * b_box;
                        mbar_expect_tx(b_full + 8 * sb, (uint32_t)nblocks * g.b_block_tx);
                        load_weights(b_ring + sb * g.b_stage_bytes, b_full + 8 * sb, n0, cc, tap, nblocks);
                        ++nb;
                        if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                    }
                    if (++ja == g.a_span) ja = 0;
                    if (++jb == g.b_span) jb = 0;
                    if (++sx == g.S) { sx = 0; ++r; }
                    if (++tap == g.taps) { tap = 0; r = 0; sx = 0; ++cc; }
                }
            }
            if (dead) {
                flag_status(g.status, FPQ_ERR_TIMEOUT);
                // let the copies still in flight land before the CTA's shared memory is released
                for (uint32_t i = (na > (uint32_t)g.a_stages ? na - g.a_stages : 0); i < na; ++i)
                    (void)mbar_wait(a_full + 8 * (i % g.a_stages), (i / g.a_stages) & 1);
                for (uint32_t i = (nb > (uint32_t)g.b_stages ? nb - g.b_stages : 0); i < nb; ++i)
                    (void)mbar_wait(b_full + 8 * (i % g.b_stages), (i / g.b_stages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one thread) ----------------
        // The tensor pipe retires one 128 x BN x 32 MMA every BN/2 cycles and its queue is
        // shallow, so this thread has only a few hundred cycles per block of 4: operand
        // positions are kept as descriptor low words (16-byte units) and the two common
        // loop shapes (3x3 taps over one loaded chunk; one block per chunk) are
        // straight-line code.
        if (elect_one()) {
            // (the limits of this role's waits start counting once the kernel in front has finished: its run time
            // is not this kernel's)
            if (g.wait_prior_grid)
                asm volatile("griddepcontrol.wait;" ::: "memory");
            uint32_t sa = 0, pa = 0, sb = 0, pb = 0, it = 0;
            uint32_t sa0 = 0, pa0 = 0;                 // ring position of the resident activation panel
            int resident_nt = -1, resident_mt = -1;
            bool dead = false;
            const uint32_t a_chunk_step = (uint32_t)g.a_chunk_bytes >> 4;
            const uint32_t b_res = smem_desc_lo(b_ring);           // resident weights start here
            const uint32_t HI = SMEM_DESC_HI_K_SW128;
            for (int t = t_lo; t < t_hi && !dead; t += t_step, ++it) {
                int mt, nt;
                decode_tile(t, mt, nt);
                const bool new_b = !(g.b_resident && resident_nt == nt);
                if (g.b_resident && new_b && resident_nt >= 0) {
                    // the resident weights are done with once everything issued so far has run
                    mma_commit(b_empty + 8 * sb);
                    if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                }
                resident_nt = nt;
                // resident activation panel: a tile of the same row tile re-reads the stages already
                // filled (no wait), and the stages are handed back only when the row tile changes
                const bool reuse_a = g.a_resident && resident_mt == mt;
                resident_mt = mt;
                if (reuse_a) { sa = sa0; pa = pa0; } else { sa0 = sa; pa0 = pa; }
                bool keep_a = false;
                if (g.a_resident && t + t_step < t_hi) {
                    int mt2, nt2;
                    decode_tile(t + t_step, mt2, nt2);
                    keep_a = mt2 == mt;
                }
                const uint32_t buf = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1)) { dead = true; break; }
                if (g.b_resident && new_b)
                    if (!mbar_wait(b_full + 8 * sb, pb)) { dead = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                // chunks from seg_from on (the second input tensor) add up in the accumulator 2 * BN columns further
                const int seg_from = (!FUSED && g.seg_acc) ? g.seg_chunk : 0x7fffffff;

                if (pair) {
                    // 3 x 3 taps over a 256-row chunk, weights streamed one tap per stage: every
                    // weight block feeds the MMAs of both row tiles (accumulators d0, d1), which halves
                    // the weight bytes that have to reach shared memory per MMA
                    const uint32_t Wp8 = (uint32_t)g.Wp * 8u;
                    const uint32_t d0 = tmem_base + buf * 2 * BN, d1 = d0 + BN;
                    for (int cc = c_lo; cc < c_hi && !dead; ++cc) {
                        if (!mbar_wait(a_full + 8 * sa, pa)) { dead = true; break; }
                        tc_fence_after();
                        const uint32_t ac = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                        uint32_t bst = 0;
#pragma unroll
                        for (int tap = 0; tap < 9; ++tap) {
                            if (!mbar_wait(b_full + 8 * sb, pb)) { dead = true; break; }
                            tc_fence_after();
                            bst = smem_desc_lo(b_ring + sb * g.b_stage_bytes);
                            const uint32_t al = ac + (tap / 3) * Wp8 + (tap % 3) * 8u;
                            const uint32_t al1 = al + BM * 8u;           // 128 rows of 128 bytes further down
                            const uint32_t bl = bst;
                            if (tap == 0 && cc == c_lo) {
                                mma_f8f6f4<false>(d0, al, bl, HI, g.idesc);
                                mma_f8f6f4<false>(d1, al1, bl, HI, g.idesc);
                            } else {
                                mma_f8f6f4<true>(d0, al, bl, HI, g.idesc);
                                mma_f8f6f4<true>(d1, al1, bl, HI, g.idesc);
                            }
                            mma_f8f6f4<true>(d0, al + 2, bl + 2, HI, g.idesc);
                            mma_f8f6f4<true>(d1, al1 + 2, bl + 2, HI, g.idesc);
                            mma_f8f6f4<true>(d0, al + 4, bl + 4, HI, g.idesc);
                            mma_f8f6f4<true>(d1, al1 + 4, bl + 4, HI, g.idesc);
                            mma_f8f6f4<true>(d0, al + 6, bl + 6, HI, g.idesc);
                            mma_f8f6f4<true>(d1, al1 + 6, bl + 6, HI, g.idesc);
                            mma_commit(b_empty + 8 * sb);
                            if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                        }
                        mma_commit(a_empty + 8 * sa);
                        if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                    }
                } else if (FLATM && g.taps == 9 && g.S == 3) {
                    const uint32_t Wp8 = (uint32_t)g.Wp * 8u;
                    const int chunks_per_stage = g.a_span / 9;
                    for (int cc = c_lo; cc < c_hi && !dead;) {
                        if (!reuse_a)
                            if (!mbar_wait(a_full + 8 * sa, pa)) { dead = true; break; }
                        tc_fence_after();
                        const uint32_t abase = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                        const int nch = min(chunks_per_stage, c_hi - cc);
                        for (int c = 0; c < nch && !dead; ++c, ++cc) {
                            const uint32_t ac = abase + c * a_chunk_step;
                            const uint32_t bres = b_res + (uint32_t)cc * 9u * BSTEP;
                            const uint32_t d = cc >= seg_from ? d_tmem + 2 * BN : d_tmem;
                            const bool fresh = cc == c_lo || cc == seg_from;
                            uint32_t bst = 0;
#pragma unroll
                            for (int tap = 0; tap < 9; ++tap) {
                                if (!g.b_resident && tap % 3 == 0) {
                                    if (!mbar_wait(b_full + 8 * sb, pb)) { dead = true; break; }
                                    tc_fence_after();
                                    bst = smem_desc_lo(b_ring + sb * g.b_stage_bytes);
                                }
                                // tap (r, s) reads the chunk r * Wp + s pixel rows (128 B each) further down
                                const uint32_t al = ac + (tap / 3) * Wp8 + (tap % 3) * 8u;
                                const uint32_t bl = g.b_resident ? bres + tap * BSTEP : bst + (tap % 3) * BSTEP;
                                // 32 reduction elements = 32 bytes inside the swizzled row: +2 units
                                if (tap == 0 && fresh)
                                    mma_f8f6f4<false>(d, al, bl, HI, g.idesc);
                                else
                                    mma_f8f6f4<true>(d, al, bl, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 2, bl + 2, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 4, bl + 4, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 6, bl + 6, HI, g.idesc);
                                if (!g.b_resident && tap % 3 == 2) {
                                    mma_commit(b_empty + 8 * sb);
                                    if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                                }
                            }
                        }
                        if (!keep_a)
                            mma_commit(a_empty + 8 * sa);
                        if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                    }
                } else if (g.taps == 1 && MODE != MODE_TAPS && g.a_span <= 4 &&
                           (g.b_resident || g.b_span == g.a_span)) {
                    // one block per 128-wide chunk; a stage carries up to 4 chunks of both operands
                    for (int cc = c_lo; cc < c_hi && !dead;) {
                        if (!reuse_a)
                            if (!mbar_wait(a_full + 8 * sa, pa)) { dead = true; break; }
                        uint32_t bbase = b_res + (uint32_t)cc * BSTEP;
                        if (!g.b_resident) {
                            if (!mbar_wait(b_full + 8 * sb, pb)) { dead = true; break; }
                            bbase = smem_desc_lo(b_ring + sb * g.b_stage_bytes);
                        }
                        tc_fence_after();
                        const uint32_t abase = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                        const int n = min(g.a_span, c_hi - cc);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if (c < n) {
                                const uint32_t al = abase + c * (BM * BK / 16), bl = bbase + c * BSTEP;
                                const uint32_t d = cc + c >= seg_from ? d_tmem + 2 * BN : d_tmem;
                                if (cc + c == c_lo || cc + c == seg_from)
                                    mma_f8f6f4<false>(d, al, bl, HI, g.idesc);
                                else
                                    mma_f8f6f4<true>(d, al, bl, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 2, bl + 2, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 4, bl + 4, HI, g.idesc);
                                mma_f8f6f4<true>(d, al + 6, bl + 6, HI, g.idesc);
                            }
                        }
                        if (!g.b_resident) {
                            mma_commit(b_empty + 8 * sb);
                            if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                        }
                        if (!keep_a)
                            mma_commit(a_empty + 8 * sa);
                        if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                        cc += n;
                    }
                } else {
                    // general shape: block by block
                    uint32_t a_lo = 0, b_lo = b_res;       // operands of the current block
                    uint32_t a_chunk_lo = 0;               // FLAT/ROWS: current chunk in its stage
                    uint32_t row_off8 = 0;                 // FLAT: (r * Wp + s) * 8 of the current tap
                    const uint32_t row_wrap8 = (uint32_t)(g.Wp - g.S) * 8u;
                    const bool flat = FLATM, taps_mode = MODE == MODE_TAPS;
                    int tap = 0, sx = 0, ja = 0, jb = 0;
                    int ccg = c_lo;                        // chunk of the current block
                    for (int j = 0; j < nblk; ++j) {
                        if (ja == 0) {
                            if (!reuse_a)
                                if (!mbar_wait(a_full + 8 * sa, pa)) { dead = true; break; }
                            a_chunk_lo = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                            a_lo = a_chunk_lo;
                            tc_fence_after();
                        }
                        if (jb == 0 && !g.b_resident) {
                            if (!mbar_wait(b_full + 8 * sb, pb)) { dead = true; break; }
                            tc_fence_after();
                            b_lo = smem_desc_lo(b_ring + sb * g.b_stage_bytes);
                        }
                        const uint32_t al = flat ? a_chunk_lo + row_off8 : a_lo;
                        const uint32_t d = ccg >= seg_from ? d_tmem + 2 * BN : d_tmem;
                        if (j == 0 || (tap == 0 && ccg == seg_from))
                            mma_f8f6f4<false>(d, al, b_lo, HI, g.idesc);
                        else
                            mma_f8f6f4<true>(d, al, b_lo, HI, g.idesc);
                        mma_f8f6f4<true>(d, al + 2, b_lo + 2, HI, g.idesc);
                        mma_f8f6f4<true>(d, al + 4, b_lo + 4, HI, g.idesc);
                        mma_f8f6f4<true>(d, al + 6, b_lo + 6, HI, g.idesc);
                        const bool last = (j == nblk - 1);
                        b_lo += BSTEP;
                        if (++jb == g.b_span || last) {
                            jb = 0;
                            if (!g.b_resident) {
                                mma_commit(b_empty + 8 * sb);
                                if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                            }
                        }
                        // next block's activation operand
                        row_off8 += 8;
                        if (++sx == g.S) { sx = 0; row_off8 += row_wrap8; }
                        if (taps_mode) a_lo += a_chunk_step;
                        if (++tap == g.taps) {
                            tap = 0; sx = 0; row_off8 = 0;
                            ++ccg;
                            a_chunk_lo += a_chunk_step;
                            if (!taps_mode) a_lo = a_chunk_lo;
                        }
                        if (++ja == g.a_span || last) {
                            ja = 0;
                            if (!keep_a)
                                mma_commit(a_empty + 8 * sa);
                            if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                        }
                    }
                }
                if (dead)
                    break;
                mma_commit(acc_full + 8 * buf);
            }
            if (dead)
                flag_status(g.status, FPQ_ERR_TIMEOUT);
        }
    } else if (warp < 2 + NUM_EPI_WARPS) {
        // ---------------- epilogue: warp w reads TMEM lane quarter w % 4 and the column
        // slice (w - 2) / 4 of the accumulator: y = acc * (x_scale * w_scale[n]) + bias[n] ----------------
        constexpr int HALF = BN / (NUM_EPI_WARPS / 4);   // columns per warp
        constexpr int CHUNKS = HALF / 32;                // 32-column TMEM loads per warp
        constexpr int G = FUSED ? 1 : CHUNKS;            // chunks held in registers at a time
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;       // row of the tile held by this thread
        if (g.stage_scales) {
            // only these warps use the scales: they fetch them while the first loads and MMAs run
            for (int i = threadIdx.x - 64; i < n_pad; i += 32 * NUM_EPI_WARPS) {
                s_scale[i] = (i < g.N) ? g.x_scale * __ldg(g.w_scale + i) : 0.f;
                s_bias[i] = (g.bias && i < g.N) ? __ldg(g.bias + i) : 0.f;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * NUM_EPI_WARPS) : "memory");
        }
        // row-major output: the warp's 32 x 32 block goes through a 128-byte-swizzled staging
        // buffer and leaves as one TMA store (whole 128-byte lines; rows past M and columns
        // past N are clipped by the tensor map)
        uint8_t* stage0 = smem + ctl_off + (warp - 2) * 8192;     // two 4 KiB buffers, used in turn
        // (as in the MMA role: bounded waits start counting after the kernel in front)
        if (g.wait_prior_grid)
            asm volatile("griddepcontrol.wait;" ::: "memory");
        uint32_t nstore = 0;
        uint32_t it = 0;
        bool dead = false;
        for (int t = t_lo; t < t_hi && !dead; t += t_step, ++it) {
            int mt, nt;
            decode_tile(t, mt, nt);
            const int n0 = nt * BN;
            const uint32_t buf = it & 1, aph = (it >> 1) & 1;

            // where this thread's row goes
            bool row_valid;
            float* yrow;
            int64_t nstride;
            row_target(pair ? 2 * mt : mt, row, row_valid, yrow, nstride);
            const int ncol0 = n0 + half * HALF;    // first output column of this warp

            // With more output columns than the shared-memory table holds, the warp fetches the scales and biases
            // of its own columns of this tile now, while the tile's MMAs still run (fetched after the accumulator was
            // complete they cost 0.7 us per 32 columns): [HALF] x_scale * w_scale, then [HALF] bias, in the warp's
            // own slice of shared memory (nobody else reads it: no barrier).
            float* w_sc = s_scale + (warp - 2) * 2 * HALF;
            if (!g.stage_scales && ksplit == 1) {
                __syncwarp();
#pragma unroll
                for (int q = 0; q < 2 * HALF / 32; ++q) {
                    const int i = q * 32 + lane;                   // [0, HALF): scale, [HALF, 2 HALF): bias
                    const int col = ncol0 + (i < HALF ? i : i - HALF);
                    float v = 0.f;
                    if (col < g.N)
                        v = i < HALF ? g.x_scale * __ldg(g.w_scale + col) : (g.bias ? __ldg(g.bias + col) : 0.f);
                    w_sc[i] = v;
                }
                __syncwarp();
            }

            if (!mbar_wait(acc_full + 8 * buf, aph)) { dead = true; }
            tc_fence_after();
            if (ksplit > 1) {
                // partial sums of this CTA's chunk range: column-major [BN][128] at the start of the
                // rings, which are idle once the accumulator is complete; the cluster adds them up below
                float* red = reinterpret_cast<float*>(smem);
                if (!dead && ncol0 < g.N) {
                    const uint32_t t_addr = tmem_base + buf * BN + half * HALF + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
                    for (int c = 0; c < CHUNKS; ++c) {
                        if (ncol0 + c * 32 >= g.N)
                            break;
                        uint32_t r[32];
                        tmem_ld32(t_addr + c * 32, r);
                        tmem_ld_wait();
                        float* dst = red + (half * HALF + c * 32) * BM + row;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            dst[j * BM] = __uint_as_float(r[j]);
                    }
                }
            } else if (!dead && ncol0 < g.N) {
                // (two accumulators when the unit is a pair of row tiles)
                for (int h = 0; h < (pair ? 2 : 1); ++h) {
                    if (h)
                        row_target(2 * mt + 1, row, row_valid, yrow, nstride);
                    const uint32_t t_addr = tmem_base + (pair ? buf * 2 + h : buf) * BN + half * HALF +
                                            ((uint32_t)(quarter * 32) << 16);
#pragma unroll
                    for (int c0 = 0; c0 < CHUNKS; c0 += G) {
                        if (ncol0 + c0 * 32 >= g.N)
                            break;
                        uint32_t r[G][32];
#pragma unroll
                        for (int c = 0; c < G; ++c)
                            tmem_ld32(t_addr + (c0 + c) * 32, r[c]);
                        tmem_ld_wait();
#pragma unroll
                        for (int cl = 0; cl < G; ++cl) {
                            const int nb = ncol0 + (c0 + cl) * 32;
                            if (nb >= g.N)
                                break;
                            const bool full = nb + 32 <= g.N;
                            // dequantize + bias in place
                            {
                                // (from the table of all columns, or from the warp's copy for this tile)
                                const float4* s4 = reinterpret_cast<const float4*>(g.stage_scales ? s_scale + nb : w_sc + (nb - ncol0));
                                const float4* b4 = reinterpret_cast<const float4*>(g.stage_scales ? s_bias + nb : w_sc + HALF + (nb - ncol0));
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    const float4 sv = s4[j], bv = b4[j];
                                    r[cl][4 * j + 0] = __float_as_uint(fmaf(__uint_as_float(r[cl][4 * j + 0]), sv.x, bv.x));
                                    r[cl][4 * j + 1] = __float_as_uint(fmaf(__uint_as_float(r[cl][4 * j + 1]), sv.y, bv.y));
                                    r[cl][4 * j + 2] = __float_as_uint(fmaf(__uint_as_float(r[cl][4 * j + 2]), sv.z, bv.z));
                                    r[cl][4 * j + 3] = __float_as_uint(fmaf(__uint_as_float(r[cl][4 * j + 3]), sv.w, bv.w));
                                }
                            }
                            if (!FUSED && g.seg_acc) {
                                // the second input tensor's sums, with its own scale
                                uint32_t r2[32];
                                tmem_ld32(t_addr + 2 * BN + (c0 + cl) * 32, r2);
                                tmem_ld_wait();
#pragma unroll
                                for (int j = 0; j < 32; ++j) {
                                    const float sv = nb + j < g.N ? g.x_scale2 * __ldg(g.w_scale + nb + j) : 0.f;
                                    r[cl][j] = __float_as_uint(fmaf(__uint_as_float(r2[j]), sv, __uint_as_float(r[cl][j])));
                                }
                            }
                            if (g.y_tma) {
                                // the buffer is free once the store before the previous one has read it
                                uint8_t* stage = stage0 + (nstore & 1u) * 4096;
                                ++nstore;
                                if (lane == 0)
                                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                                __syncwarp();
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    *reinterpret_cast<uint4*>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                        make_uint4(r[cl][4 * j], r[cl][4 * j + 1], r[cl][4 * j + 2], r[cl][4 * j + 3]);
                                fence_proxy_async();
                                __syncwarp();
                                if (lane == 0) {
                                    asm volatile(
                                        "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                        ::"l"(&tmY), "r"(smem_u32(stage)), "r"(nb), "r"(mt * BM + quarter * 32)
                                        : "memory");
                                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                                }
                            } else if (row_valid) {
                                if (MODE == MODE_ROWS) {
                                    if (full && g.N % 4 == 0) {
                                        uint4* dst = reinterpret_cast<uint4*>(yrow + nb);
#pragma unroll
                                        for (int j = 0; j < 8; ++j)
                                            dst[j] = make_uint4(r[cl][4 * j], r[cl][4 * j + 1], r[cl][4 * j + 2], r[cl][4 * j + 3]);
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 32; ++j)
                                            if (nb + j < g.N)
                                                yrow[nb + j] = __uint_as_float(r[cl][j]);
                                    }
                                } else {
                                    float* dst = yrow + (int64_t)nb * nstride;
                                    if (full) {
#pragma unroll
                                        for (int j = 0; j < 32; j += 4) {
                                            dst[0] = __uint_as_float(r[cl][j]);
                                            dst[nstride] = __uint_as_float(r[cl][j + 1]);
                                            dst[2 * nstride] = __uint_as_float(r[cl][j + 2]);
                                            dst[3 * nstride] = __uint_as_float(r[cl][j + 3]);
                                            dst += 4 * nstride;
                                        }
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 32; ++j)
                                            if (nb + j < g.N)
                                                dst[(int64_t)j * nstride] = __uint_as_float(r[cl][j]);
                                    }
                                }
                            }
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
        if (g.y_tma && lane == 0)
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the staging buffer must outlive its stores
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    } else if (FUSED && warp == 2 + NUM_EPI_WARPS + NUM_XFORM_WARPS) {
        // ---------------- L2 prefetch warp ----------------
        // A transform thread can keep only two rows of loads in flight, so it cannot hide DRAM
        // latency.  This warp runs ahead of them through the CTA's tiles and asks the L2 for every 128-byte line of
        // FP32 activations those tiles will read; it synchronises with nobody.
        const int rows = g.a_chunk_bytes >> 7;
        auto prefetch_tile = [&](int t) {
            int mt, nt;
            decode_tile(t, mt, nt);
            if (MODE == MODE_ROWS) {
                // 128 rows of C floats: one contiguous span
                const int64_t m0 = (int64_t)mt * BM;
                const int64_t m1 = min(m0 + BM, g.M);
                const char* p0 = reinterpret_cast<const char*>(g.x + m0 * g.C);
                const int64_t bytes = (m1 - m0) * g.C * 4;
                for (int64_t o = (int64_t)lane * 128; o < bytes; o += 32 * 128)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p0 + o));
                return;
            }
            const uint32_t f_lo = (uint32_t)mt * BM;
            if ((int64_t)f_lo >= g.M)
                return;
            const uint32_t f_hi = (uint32_t)min((int64_t)f_lo + rows, g.M) - 1u;
            const uint32_t b_lo = fdiv(f_lo, g.div_HpWp), b_hi = fdiv(f_hi, g.div_HpWp);
            const int yp_lo = (int)fdiv(f_lo - b_lo * (uint32_t)g.HpWp, g.div_Wp);
            const int yp_hi = (int)fdiv(f_hi - b_hi * (uint32_t)g.HpWp, g.div_Wp);
            for (int part = 0; part < 2; ++part) {
                if (part == 1 && b_hi == b_lo)
                    break;
                const uint32_t b = part ? b_hi : b_lo;
                const int y0 = part ? 0 : max(yp_lo - g.pad, 0);
                const int y1 = (part || b_hi == b_lo) ? min(yp_hi - g.pad, g.H - 1) : g.H - 1;
                if ((int)b >= g.B || y1 < y0)
                    continue;
                const int bytes = (y1 - y0 + 1) * g.W * 4;        // contiguous per channel
                for (int c = c_lo * BK + lane; c < min(g.C, c_hi * BK); c += 32) {
                    const char* p0 = reinterpret_cast<const char*>(
                        g.x + ((int64_t)(b * (uint32_t)g.C + (uint32_t)c) * g.H + y0) * g.W);
                    for (int o = 0; o < bytes; o += 128)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(p0 + o));
                }
            }
        };
        int last_mt = -1;
        for (int t = t_lo; t < t_hi; t += t_step) {
            int mt, nt;
            decode_tile(t, mt, nt);
            if (mt == last_mt)
                continue;
            last_mt = mt;
            prefetch_tile(t);
        }
    } else if (FUSED) {
        // ---------------- activation-quantize prologue: the transform warps fill the A ring ----------------
        const int tw = warp - (2 + NUM_EPI_WARPS);      // channel group tw % 8, row phase tw / 8
        const int tid = threadIdx.x - 32 * (2 + NUM_EPI_WARPS);
        const int chunks_per_stage = g.a_span / g.taps;
        const int rows = g.a_chunk_bytes >> 7;
        uint32_t sa = 0, pa = 0;
        bool dead = false, nan = false;
        int resident_mt = -1;
        for (int t = t_lo; t < t_hi && !dead; t += t_step) {
            int mt, nt;
            decode_tile(t, mt, nt);
            if (g.a_resident && mt == resident_mt)
                continue;                          // the panel is still in the ring
            resident_mt = mt;
            for (int cc = c_lo; cc < c_hi;) {
                if (!mbar_wait(a_empty + 8 * sa, pa ^ 1)) { dead = true; break; }
                const int nch = min(chunks_per_stage, c_hi - cc);
                uint8_t* dst = smem + sa * g.a_stage_bytes;
                for (int l = 0; l < nch; ++l, dst += g.a_chunk_bytes) {
                    if (MODE == MODE_ROWS)
                        fill_chunk_rows(g, dst, (int64_t)mt * BM, (cc + l) * BK, tid, nan);
                    else
                        fill_chunk_nchw(g, dst, (uint32_t)mt * BM, rows, (cc + l) * BK, tw, lane, nan);
                }
                // make the generic-proxy writes visible to the tensor core's reads, then signal
                fence_proxy_async();
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(a_full + 8 * sa);
                if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                cc += nch;
            }
        }
        if (nan)
            flag_status(g.status, FPQ_ERR_NAN_INPUT);
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    }

    if (ksplit > 1) {
        // every thread of every CTA of the cluster arrives here (all waits above are bounded)
        __syncwarp();
        cluster_sync_all();
        if (warp >= 2 && warp < 2 + NUM_EPI_WARPS) {
            // CTA k adds up the columns k, k + ksplit, ... of the tile over all CTAs of the cluster, in
            // rank order (the same order whatever the timing), then dequantize + bias as usual
            int mt, nt;
            decode_tile(t_lo, mt, nt);
            // a thread owns four consecutive rows (one 16-byte load per peer and column) and every
            // NUM_EPI_WARPS-th of this CTA's columns
            const int e = threadIdx.x - 64;
            const int rg = e & 31, cs = e >> 5;
            bool row_valid[4];
            float* yrow[4];
            int64_t nstride = 1;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                row_target(mt, 4 * rg + q, row_valid[q], yrow[q], nstride);
            // this CTA's staging area as seen in every CTA of the cluster
            uint32_t peer[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                peer[k] = k < ksplit ? peer_smem_addr(smem_base, (uint32_t)k) : 0u;
            // two columns per round: their 2 x ksplit loads are in flight together
            const int cstep = ksplit * NUM_EPI_WARPS;
            for (int c = (int)krank + ksplit * cs; c < BN; c += 2 * cstep) {
                if (nt * BN + c >= g.N)
                    break;
                float4 v[2][8];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int cu = c + u * cstep;
                    const uint32_t off = (uint32_t)(cu * BM + 4 * rg) * 4u;
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        v[u][k] = (k < ksplit && cu < BN) ? ld_cluster_smem4(peer[k] + off) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int cu = c + u * cstep;
                    const int n = nt * BN + cu;
                    if (cu >= BN || n >= g.N)
                        break;
                    float4 acc = v[u][0], acc2 = make_float4(0.f, 0.f, 0.f, 0.f);   // first / second input tensor
                    if (!g.seg_chunk) {
#pragma unroll
                        for (int k = 1; k < 8; ++k)
                            if (k < ksplit) {
                                acc.x += v[u][k].x; acc.y += v[u][k].y; acc.z += v[u][k].z; acc.w += v[u][k].w;
                            }
                    } else {
                        // selects, not branches (v is 0 beyond the cluster)
                        acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const bool one = k < g.seg_ranks;
                            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                            const float4 a1 = one ? v[u][k] : z, a2 = one ? z : v[u][k];
                            acc.x += a1.x; acc.y += a1.y; acc.z += a1.z; acc.w += a1.w;
                            acc2.x += a2.x; acc2.y += a2.y; acc2.z += a2.z; acc2.w += a2.w;
                        }
                    }
                    const float sv = g.stage_scales ? s_scale[n] : g.x_scale * __ldg(g.w_scale + n);
                    const float bv = g.stage_scales ? s_bias[n] : (g.bias ? __ldg(g.bias + n) : 0.f);
                    float out[4] = {fmaf(acc.x, sv, bv), fmaf(acc.y, sv, bv), fmaf(acc.z, sv, bv), fmaf(acc.w, sv, bv)};
                    if (g.seg_chunk) {
                        const float sv2 = g.x_scale2 * __ldg(g.w_scale + n);
                        out[0] = fmaf(acc2.x, sv2, out[0]);
                        out[1] = fmaf(acc2.y, sv2, out[1]);
                        out[2] = fmaf(acc2.z, sv2, out[2]);
                        out[3] = fmaf(acc2.w, sv2, out[3]);
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (row_valid[q])
                            yrow[q][(int64_t)n * nstride] = out[q];
                }
            }
        }
        // nobody leaves (and frees its shared memory) while a peer may still read it
        __syncwarp();
        cluster_sync_all();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (g.seg_acc || pair) ? 4 * BN : 2 * BN);
    }
}

// ---- host side --------------------------------------------------------------------------
static EncodeTiledFn encode_fn() { return tensor_map_encoder(); }

static int pow2_at_least(int v)
{
    int p = 1;
    while (p < v)
        p <<= 1;
    return p;
}

struct DeviceInfo {
    int sms;
    bool smem_set[16];
    int max_clusters[2][4][9];     // [BN == 128][mode][cluster size]: clusters resident at once, 0 = not asked yet, -1 = none
};

static DeviceInfo* device_info()
{
    static DeviceInfo info[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return nullptr;
    if (!info[dev].sms) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
            v = 148;
        info[dev].sms = v;
    }
    return &info[dev];
}

template <int BN, bool FUSED, int MODE>
static bool allow_max_smem(DeviceInfo* di)
{
    const int slot = (BN == 64 ? 0 : 1) + (FUSED ? 2 : 0) + 4 * MODE;
    if (!di->smem_set[slot]) {
        if (cudaFuncSetAttribute(fpq_gemm_kernel<BN, FUSED, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET) !=
            cudaSuccess)
            return false;
        di->smem_set[slot] = true;
    }
    return true;
}

// How many clusters of `size` CTAs of the contraction kernel the GPU holds at once.  Asked of the
// plain kernel for both forms, so that both take the same decision (and add partial sums in the same order).
template <int BN, int MODE>
static int max_clusters(DeviceInfo* di, int size)
{
    int& slot = di->max_clusters[BN == 64 ? 0 : 1][MODE][size];
    if (slot == 0) {
        slot = -1;
        if (allow_max_smem<BN, false, MODE>(di)) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(size * di->sms));
            cfg.blockDim = dim3(num_threads(false));
            cfg.dynamicSmemBytes = SMEM_BUDGET;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)size;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, fpq_gemm_kernel<BN, false, MODE>, &cfg) == cudaSuccess && n > 0)
                slot = n;
            else
                (void)cudaGetLastError();
        }
    }
    return slot;
}

// what the weight tensor map is made from (its box depends on the plan, so it is encoded after planning)
struct WeightSpec {
    const void* w;      // prepared weights [N][taps][Cp]
    int w4, Cp, N;
    const void* a;      // row-major activation codes [M][Ca] (linear layers), else NULL
    int Ca;
    int64_t M;
};

template <int BN, bool FUSED, int MODE>
static fpq_status launch_mode(const CUtensorMap& tmA, const WeightSpec& wspec, const CUtensorMap& tmY, GemmArgs& g,
                                 cudaStream_t st)
{
    // Split the shared-memory budget between the two rings.  A barrier handshake costs the
    // single issuing thread a few hundred cycles, so every stage is made to carry 8-36 MMAs;
    // weights that fit stay resident for all row tiles of a column tile.
    DeviceInfo* di = device_info();
    if (!di)
        return FPQ_ERR_CUDA;
    const int n_pad = (g.N + 31) & ~31;
    g.stage_scales = (n_pad * 8 <= 16384) ? 1 : 0;
    // (without the table of all columns: every epilogue warp's copy of its own columns' scales and biases, 2 * BN floats
    // per group of four warps)
    const int ctl = 512 + 1024 + (g.y_tma ? epi_warps(FUSED) * 8192 : 0) + (g.stage_scales ? n_pad * 8 : 4 * 2 * BN * 4);
    const int budget = SMEM_BUDGET - ctl;
    const int b_block = BN * BK;
    const int a_min_span = (g.mode == MODE_FLAT) ? g.taps : 1;
    const int64_t b_all = (int64_t)g.nblk * b_block;
    g.a_resident = 0;
    // Few tiles and a long reduction (the low-resolution convolutions): a cluster of ksplit CTAs
    // shares each tile.  The split takes the largest cluster that still lets all tiles run at once,
    // then the smallest one with the same longest chunk range.
    g.ksplit = 1;
    const int64_t base_tiles = (int64_t)g.m_tiles * g.n_tiles;
    if (g.pair) {
        // paired row tiles: plain streaming of both operands, no cluster
    } else if (g.seg_chunk) {
        // two input tensors: with few tiles a cluster per tile, at least one CTA per tensor and as
        // many CTAs as keep every tile resident at once; with many tiles no cluster
        if (MODE == MODE_ROWS || FUSED || g.seg_chunk >= g.cchunks)
            return FPQ_ERR_UNSUPPORTED;
        int sp = 2;
        g.seg_acc = 0;
        if (base_tiles * 2 > di->sms) {
            // plenty of tiles: the usual persistent walk, one accumulator per tensor
            sp = 1;
            g.seg_acc = 1;
        } else {
            sp = (int)(di->sms / base_tiles);
            if (sp > 8) sp = 8;
            if (sp > g.cchunks) sp = g.cchunks;
            while (sp > 2 && max_clusters<BN, MODE>(di, sp) < base_tiles)
                --sp;
        }
        if (!g.seg_acc) {
            int r1 = (sp * g.seg_chunk + g.cchunks / 2) / g.cchunks;
            if (r1 < 1) r1 = 1;
            if (r1 > sp - 1) r1 = sp - 1;
            if (r1 > g.seg_chunk) r1 = g.seg_chunk;
            int r2 = sp - r1;
            if (r2 > g.cchunks - g.seg_chunk) r2 = g.cchunks - g.seg_chunk;
            g.seg_ranks = r1;
            g.ksplit = r1 + r2;
        }
    } else if (g.cchunks >= 2 && base_tiles * 2 <= di->sms &&
               (MODE != MODE_ROWS || (g.m_tiles == 1 && (g.cchunks >= 32 || (g.M <= 8 && g.cchunks >= 8))))) {
        // (row-major outputs leave the cluster's reduction column by column, which only pays for a single
        // row tile with a very long reduction or a handful of rows: measured on the SD-v1 linears)
        int s_max = (int)(di->sms / base_tiles);
        if (s_max > 8) s_max = 8;
        if (s_max > g.cchunks) s_max = g.cchunks;
        while (s_max >= 2 && max_clusters<BN, MODE>(di, s_max) < base_tiles)
            --s_max;
        if (s_max >= 2) {
            const int longest = (g.cchunks + s_max - 1) / s_max;
            int sp = s_max;
            while (sp > 2 && (g.cchunks + sp - 2) / (sp - 1) == longest)
                --sp;
            g.ksplit = sp;
        }
    }
    // several column tiles per row tile: try to keep the row tile's whole activation panel in the
    // ring (read / quantized once) and stream the weights
    bool done = false;
    if (g.ksplit == 1 && !g.pair && g.n_tiles > 1 && g.mode != MODE_TAPS) {
        const bool conv9 = g.mode == MODE_FLAT && g.taps == 9 && g.S == 3;
        if (conv9 || g.taps == 1) {
            const int cps = conv9 ? 1 : (g.cchunks >= 3 ? 3 : g.cchunks);      // chunks per A stage
            const int groups = (g.cchunks + cps - 1) / cps;
            const int b_span = conv9 ? 3 : cps;
            const int b_stage = b_span * b_block;
            const int panel = groups * cps * g.a_chunk_bytes;
            if (groups <= 8 && panel + 2 * b_stage <= budget) {
                const int panels = (groups <= 4 && 2 * panel + 2 * b_stage <= budget) ? 2 : 1;
                g.a_resident = 1;
                g.m_fastest = 0;
                g.b_resident = 0;
                g.a_span = cps * a_min_span;
                g.a_stage_bytes = cps * g.a_chunk_bytes;
                g.a_stages = panels * groups;
                g.b_span = b_span;
                g.b_stages = (budget - g.a_stages * g.a_stage_bytes) / b_stage;
                if (g.b_stages > 8) g.b_stages = 8;
                done = true;
            }
        }
    }
    if (done) {
        // configured above
    } else if (g.ksplit == 1 && !g.pair && b_all + 2 * g.a_chunk_bytes <= budget) {
        g.b_resident = 1;
        g.b_span = g.nblk;
        g.b_stages = 1;
        g.m_fastest = 1;
        const int room = budget - (int)b_all;
        int chunks = room / (2 * g.a_chunk_bytes);            // chunks (TAPS: boxes) per stage
        const int want = (g.mode == MODE_FLAT && g.taps >= 4) ? 1 : 4;
        if (chunks > want) chunks = want;
        const int avail = (g.mode == MODE_TAPS) ? g.nblk : g.cchunks;
        if (chunks > avail) chunks = avail;
        if (chunks < 1) chunks = 1;
        g.a_span = chunks * a_min_span;
        g.a_stage_bytes = chunks * g.a_chunk_bytes;
        g.a_stages = room / g.a_stage_bytes;
        if (g.a_stages > 4) g.a_stages = 4;
    } else {
        g.b_resident = 0;
        g.m_fastest = 0;
        int chunks;
        if (g.mode == MODE_FLAT && g.taps > 1) {
            g.b_span = (g.taps == 9 && g.S == 3 && !g.pair) ? 3 : 1;
            g.a_span = g.taps;                                // one chunk per stage serves all taps
            chunks = 1;
            g.a_stages = 2;
        } else {
            g.b_span = (g.mode == MODE_TAPS && g.taps % 3 == 0) ? 3 : 2;
            if (g.b_span > g.nblk) g.b_span = g.nblk;
            g.a_span = g.b_span;
            chunks = g.a_span;
            g.a_stages = 3;
        }
        g.a_stage_bytes = chunks * g.a_chunk_bytes;
        g.b_stages = (budget - g.a_stages * g.a_stage_bytes) / (g.b_span * b_block);
        if (g.b_stages < 2 && g.a_stages > 2) {
            g.a_stages = 2;
            g.b_stages = (budget - g.a_stages * g.a_stage_bytes) / (g.b_span * b_block);
        }
        if (g.b_stages > 8) g.b_stages = 8;
    }
    g.b_stage_bytes = g.b_span * b_block;
    if (g.a_stages < 1 || g.b_stages < 1 || (!g.b_resident && g.b_stages < 2))
        return FPQ_ERR_UNSUPPORTED;
    g.contiguous = (g.a_resident || (g.b_resident && g.n_tiles > 1)) ? 1 : 0;
    g.div_tiles = make_fastdiv((uint32_t)(g.m_fastest ? g.m_tiles : g.n_tiles));
    // the partial sums of a split tile are staged over the rings
    if (g.ksplit > 1 && g.a_stages * g.a_stage_bytes + g.b_stages * g.b_stage_bytes < BN * BM * 4)
        return FPQ_ERR_UNSUPPORTED;
    const int dyn = g.a_stages * g.a_stage_bytes + g.b_stages * g.b_stage_bytes + ctl;
    if (!allow_max_smem<BN, FUSED, MODE>(di))
        return FPQ_ERR_CUDA;
    // Blocks per weight load.  A stage of b_span blocks is a run of taps inside one chunk (3 x 3 layers: three taps) or
    // a run of chunks of a tap-less layer; the resident form holds whole chunks, so one load takes all taps of a chunk.
    g.b_box_t = g.b_box_c = 1;
    if (g.b_resident) {
        if (g.taps > 1 && g.taps <= 16)
            g.b_box_t = g.taps;
        else if (g.taps == 1 && g.cchunks > 1 && g.cchunks <= 8)
            g.b_box_c = g.cchunks;
    } else if (g.taps > 1) {
        if (g.b_span > 1 && g.taps % g.b_span == 0)
            g.b_box_t = g.b_span;
    } else if (g.b_span > 1) {
        g.b_box_c = g.b_span;
    }
    // prepared weights [N][taps][Cp] as (position in chunk, output, tap, chunk): a box lands as [chunk][tap][output][128 B]
    CUtensorMap tmB, tmA2 = tmA;
    g.a_box_c = 1;
    {
        EncodeTiledFn enc = encode_fn();
        if (!enc)
            return FPQ_ERR_CUDA;
        if (MODE == MODE_ROWS && !FUSED && wspec.a && wspec.Ca % BK == 0 && g.taps == 1 && g.a_span > 1 && g.a_span <= 8) {
            // rows of whole chunks: the chunks of a stage as one box, (position in chunk, row, chunk)
            cuuint64_t dimsA[4] = {(cuuint64_t)BK, (cuuint64_t)wspec.M, (cuuint64_t)(wspec.Ca / BK), 1};
            cuuint64_t stridesA[3] = {(cuuint64_t)wspec.Ca, (cuuint64_t)BK, (cuuint64_t)wspec.Ca * (cuuint64_t)wspec.M};
            cuuint32_t boxA[4] = {BK, BM, (cuuint32_t)g.a_span, 1};
            cuuint32_t estrA[4] = {1, 1, 1, 1};
            if (enc(&tmA2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void*)wspec.a, dimsA, stridesA, boxA, estrA,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return FPQ_ERR_CUDA;
            g.a_box_c = g.a_span;
        }
        const cuuint64_t rowB = wspec.w4 ? (cuuint64_t)wspec.Cp / 2 : (cuuint64_t)wspec.Cp;
        cuuint64_t dimsB[4] = {(cuuint64_t)BK, (cuuint64_t)wspec.N, (cuuint64_t)g.taps, (cuuint64_t)(wspec.Cp / BK)};
        cuuint64_t stridesB[3] = {rowB * g.taps, rowB, wspec.w4 ? (cuuint64_t)BK / 2 : (cuuint64_t)BK};
        cuuint32_t boxB[4] = {BK, (cuuint32_t)BN, (cuuint32_t)g.b_box_t, (cuuint32_t)g.b_box_c};
        cuuint32_t estrB[4] = {1, 1, 1, 1};
        if (enc(&tmB, wspec.w4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void*)wspec.w, dimsB,
                stridesB, boxB, estrB, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
    }
    const int64_t tiles = (int64_t)g.m_tiles * g.n_tiles;
    if (g.ksplit > 1 && tiles * g.ksplit > 0x7fffff00ll)
        return FPQ_ERR_SHAPE;
    const int grid = g.ksplit > 1 ? (int)tiles * g.ksplit : (int)(tiles < di->sms ? tiles : di->sms);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(num_threads(FUSED));
    cfg.dynamicSmemBytes = (size_t)dyn;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int nattr = 0;
    if (g.wait_prior_grid) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    if (g.ksplit > 1) {
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = (unsigned)g.ksplit;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)nattr;
    return cudaLaunchKernelEx(&cfg, fpq_gemm_kernel<BN, FUSED, MODE>, tmA2, tmB, tmY, (const GemmArgs)g) == cudaSuccess ? FPQ_OK
                                                                                                      : FPQ_ERR_CUDA;
}

template <int BN, bool FUSED>
static fpq_status launch_variant(const CUtensorMap& tmA, const WeightSpec& wspec, const CUtensorMap& tmY, GemmArgs& g,
                                 cudaStream_t st)
{
    // one instantiation per addressing mode keeps every kernel's code small: the single MMA-issuing
    // thread is sensitive to instruction fetch
    if (g.mode == MODE_ROWS)
        return launch_mode<BN, FUSED, MODE_ROWS>(tmA, wspec, tmY, g, st);
    if (g.mode == MODE_FLAT && g.pair) {
        if (FUSED)
            return FPQ_ERR_UNSUPPORTED;
        return launch_mode<BN, false, MODE_FLAT2>(tmA, wspec, tmY, g, st);
    }
    if (g.mode == MODE_FLAT)
        return launch_mode<BN, FUSED, MODE_FLAT>(tmA, wspec, tmY, g, st);
    if (FUSED)
        return FPQ_ERR_UNSUPPORTED;
    return launch_mode<BN, false, MODE_TAPS>(tmA, wspec, tmY, g, st);
}

fpq_status launch_gemm(const GemmProblem& p, cudaStream_t st)
{
    // the per-device tables behind the plan (SM count, kernel attributes, cluster occupancy) are filled
    // on first use: host threads take turns here
    static std::mutex plan_mutex;
    std::lock_guard<std::mutex> lock(plan_mutex);
    EncodeTiledFn enc = encode_fn();
    if (!enc)
        return FPQ_ERR_CUDA;

    GemmArgs g{};
    g.N = p.N;
    g.cchunks = p.Cp / BK;
    g.taps = p.R * p.S;
    g.nblk = g.cchunks * g.taps;
    g.S = p.S;
    g.stride = p.stride;
    g.Ho = p.Ho;
    g.Wo = p.Wo;
    g.B = p.B;
    g.w_scale = p.w_scale;
    g.x_scale = p.x_scale;
    g.seg_chunk = p.c_seg;
    g.x_scale2 = p.x_scale2;
    g.bias = p.bias;
    g.y = p.y;
    g.status = status_word();
    g.wait_prior_grid = p.after_stage1;

    const int BN = (p.N <= 64) ? 64 : 128;
    g.n_tiles = (p.N + BN - 1) / BN;
    g.idesc = idesc_f8f6f4(p.a_e5m2 ? 1u : 0u, p.w4 ? 5u : (p.w_e5m2 ? 1u : 0u), (uint32_t)BN);
    g.b_block_tx = (uint32_t)(BN * BK) / (p.w4 ? 2 : 1);

    CUtensorMap tmA;
    cuuint64_t dimsA[4], stridesA[3];
    cuuint32_t boxA[4], estrA[4] = {1, 1, 1, 1};
    const int Hp = p.H + 2 * p.pad, Wp = p.W + 2 * p.pad;
    int64_t mtiles;
    g.Wp = 1;
    g.HpWp = 1;
    g.Wt = g.Ht = g.Bt = g.tiles_x = g.tiles_y = 1;
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
        const bool flat_ok = p.stride == 1 && halo_rows <= 2 * 256 - 16 && flat_tiles * 4 <= exact_tiles * 5 + 4 &&
                             framed < 0x7fffff00ll;
        if (flat_ok) {
            g.mode = MODE_FLAT;
            g.M = framed;
            g.Wp = Wp;
            g.HpWp = Hp * Wp;
            mtiles = flat_tiles;
            int rows = halo_rows;
            // Streamed 3 x 3 weights fill shared memory at about half the rate the MMAs of one row tile
            // consume them (measured: ~32 bytes per clock and SM arrive, 64 + 11 are needed).  Two row
            // tiles per unit share every weight block; taken when that beats the loss of parallelism.
            // (measured time per unit in MMA-bound tile times: 2.04 alone, 2 x 1.62 as a pair)
            DeviceInfo* di = device_info();
            const int64_t b_all = (int64_t)g.nblk * BN * BK;
            if (di && p.R == 3 && p.S == 3 && p.x == nullptr && p.c_seg == 0 && b_all > 160 * 1024 &&
                halo_rows + BM <= 2 * 256 - 16) {
                const int64_t alone = flat_tiles * g.n_tiles, pairs = (flat_tiles + 1) / 2 * g.n_tiles;
                const double t_alone = (double)((alone + di->sms - 1) / di->sms) * 2.04;
                const double t_pair = (double)((pairs + di->sms - 1) / di->sms) * 2.0 * 1.62;
                // (a row tile's whole activation panel resident across its column tiles measured a
                // little faster than pairing where it fits)
                const int64_t panel = (int64_t)g.cchunks * round_up(halo_rows, 8) * 128;
                const bool panel_fits = g.n_tiles > 1 && g.cchunks <= 8 && panel + 6 * BN * BK <= SMEM_BUDGET - 12 * 1024;
                if (alone * 2 > di->sms && t_pair < t_alone && !panel_fits) {
                    g.pair = 1;
                    mtiles = (flat_tiles + 1) / 2;
                    rows = halo_rows + BM;
                }
            }
            g.a_boxes = rows > 256 ? 2 : 1;
            g.a_box_rows = (int)round_up((rows + g.a_boxes - 1) / g.a_boxes, 8);
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
    if (mtiles <= 0 || mtiles * g.n_tiles > 0x7fffff00ll)
        return FPQ_ERR_SHAPE;
    g.m_tiles = (int)mtiles;
    g.div_HpWp = make_fastdiv((uint32_t)g.HpWp);
    g.div_Wp = make_fastdiv((uint32_t)g.Wp);
    g.div_Wt = make_fastdiv((uint32_t)g.Wt);
    g.div_Ht = make_fastdiv((uint32_t)g.Ht);
    g.div_tx = make_fastdiv((uint32_t)g.tiles_x);
    g.div_ty = make_fastdiv((uint32_t)g.tiles_y);
    g.a_chunk_bytes = g.a_boxes * g.a_box_rows * 128;
    g.a_chunk_tx = (uint32_t)g.a_chunk_bytes;
    if (enc(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void*)p.a_codes, dimsA, stridesA, boxA, estrA,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return FPQ_ERR_CUDA;

    // (the weight map is encoded once the plan has fixed how many blocks one load covers)
    const WeightSpec wspec = {p.w_prepared, p.w4, p.Cp, p.N, (!p.conv && p.x == nullptr) ? p.a_codes : nullptr, p.Ca, p.M};

    // row-major output through TMA stores
    CUtensorMap tmY = tmA;
    g.y_tma = 0;
    g.vec_scale = ((uintptr_t)p.w_scale % 16 == 0) && (p.bias == nullptr || (uintptr_t)p.bias % 16 == 0);
    if (!p.conv && p.N % 4 == 0 && (uintptr_t)p.y % 16 == 0) {
        cuuint64_t dimsY[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
        cuuint64_t stridesY[1] = {(cuuint64_t)p.N * 4};
        cuuint32_t boxY[2] = {32, 32};
        cuuint32_t estrY[2] = {1, 1};
        if (enc(&tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)p.y, dimsY, stridesY, boxY, estrY,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
        g.y_tma = 1;
    }

    if (p.x != nullptr && p.a_e5m2)
        return FPQ_ERR_UNSUPPORTED;     // the fused forms convert to E4M3
    const bool fused = p.x != nullptr && g.mode != MODE_TAPS;
    if (fused) {
        g.x = p.x;
        g.rinv = 1.0f / p.x_scale;
        g.C = p.C;
        g.H = p.H;
        g.W = p.W;
        g.pad = p.pad;
        g.wait_prior_grid = 0;
        return BN == 64 ? launch_variant<64, true>(tmA, wspec, tmY, g, st) : launch_variant<128, true>(tmA, wspec, tmY, g, st);
    }
    if (p.x != nullptr)
        return FPQ_ERR_UNSUPPORTED;     // the caller falls back to the two-kernel route
    return BN == 64 ? launch_variant<64, false>(tmA, wspec, tmY, g, st) : launch_variant<128, false>(tmA, wspec, tmY, g, st);
}

}  // namespace fpq
