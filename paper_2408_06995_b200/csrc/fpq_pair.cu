// The quantized stride-1 convolution as ONE kernel on CTA pairs: FP32 NCHW activations in, FP32 NCHW
// out, the E4M3 activation codes exist only in shared memory (the layer of Sec. VI-A: quantize ->
// low-bit contraction -> dequantize + bias).
//
// Two CTAs of a cluster share every MMA (tcgen05 cta_group::2, M = 256): each CTA owns 128 output
// pixels (tensor-memory lanes) and HALF of the weight rows, so the layer's whole weight tensor stays
// resident in shared memory at half the footprint per SM, which leaves room for a double-buffered
// activation operand and a deep FP32 staging ring.  Per CTA:
//   warp 0      TMA producer: the CTA's half of the weights once (one box per 128-channel chunk), then FP32
//               activation rows (boxes {W, 128 channels, 1 or 2 image rows}) into the staging ring.  A TMA
//               load costs about one memory latency whatever its size and the loads of a CTA hardly
//               overlap, so the boxes are made large and warp 2 asks the L2 for the rows ahead of time;
//   warp 1      tensor-memory owner; in the pair's first CTA also the MMA issuer for both CTAs;
//   warp 2      L2 prefetch of the FP32 rows the CTA's tiles will read;
//   warps 4-11  epilogue: tcgen05.ld -> acc * (x_scale * w_scale[n]) + bias[n] -> NCHW stores;
//   warps 12-19 transform: staged FP32 rows -> E4M3 codes in the K-major 128-byte-swizzled operand
//               layout, frame positions (zero padding) written as code 0.
// The operand of a tile is the zero-framed channels-last pixel list of the stride-1 scheme: output
// position q reads rows q + r * Wp + s, so all taps read one staged chunk through descriptors moved by
// whole rows.  Every wait is bounded; nothing here uses TMA multicast.
#include <cuda.h>

#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"
#include "fpq_tensormap.h"

namespace fpq {

namespace {

constexpr int BM = 128;
constexpr int BK = 128;
constexpr int EPI_W0 = 4, NUM_EPI = 8;
constexpr int XF_W0 = 12, NUM_XF = 8;
constexpr int NTHREADS = 32 * (XF_W0 + NUM_XF);
constexpr int SMEM_BUDGET = 227 * 1024;
constexpr int MAX_CHUNKS = 16;

struct PairArgs {
    int64_t M;                 // framed pixels B * Hp * Wp
    int N, BN;                 // outputs; MMA N (N rounded up to 64)
    int cchunks, taps, S;      // 128-wide chunks of the channels, taps = R * S
    int nblk;                  // weight blocks = cchunks * taps, each BN/2 rows x 128 bytes per CTA
    int Wp, Hp, HpWp;
    FastDiv div_Wp, div_Hp, div_HpWp, div_W2;
    int B, C, H, W, pad, Ho, Wo;
    int m_tiles, tiles_per_cta; // 128-row tiles; every CTA owns a strip of consecutive tiles (the pair's two strips advance together)
    int reuse;                 // a tile takes the operand rows it shares with the strip's previous tile from that tile's stage
    int rows;                  // operand rows per tile and chunk (128 + halo, multiple of 8)
    int a_stage_bytes, a_stages;
    int x_rows;                // image rows a tile touches
    int x_nr, x_groups;        // image rows per staged box; boxes per tile and chunk
    int x_stage_bytes, x_stages;
    int b_block_bytes;
    uint32_t b_block_tx;
    uint32_t idesc;
    uint32_t tmem_cols;
    const float* x;
    const float* w_scale;
    float x_scale, rinv;
    const float* bias;
    float* y;
    int* status;
};

// The image rows a tile's operand needs: framed rows G_lo .. G_lo + nrow - 1, the first one being row yp_lo of
// image b_lo.  A tile that follows another one in its strip only produces the operand rows from i_lo on.
struct TileRows {
    int i_lo, nrow, ngrp, base_i;
    uint32_t b_lo, yp_lo;
};
__device__ __forceinline__ TileRows tile_rows(const PairArgs& g, int mt, int step)
{
    TileRows t;
    const uint32_t q0 = (uint32_t)mt * BM;
    t.i_lo = (g.reuse && step > 0) ? g.rows - BM : 0;
    const uint32_t G_lo = fdiv(q0 + (uint32_t)t.i_lo, g.div_Wp), G_hi = fdiv(q0 + (uint32_t)g.rows - 1u, g.div_Wp);
    t.nrow = (int)(G_hi - G_lo) + 1;
    t.ngrp = (t.nrow + g.x_nr - 1) / g.x_nr;
    t.b_lo = fdiv(G_lo, g.div_Hp);
    t.yp_lo = G_lo - t.b_lo * (uint32_t)g.Hp;
    t.base_i = (int)(G_lo * (uint32_t)g.Wp) - (int)q0;      // operand row of framed pixel 0 of the first image row
    return t;
}

// two IEEE multiplications in one instruction
__device__ __forceinline__ float2 mul2(float2 a, float r)
{
    unsigned long long ua, ur, ud;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ua) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %1};" : "=l"(ur) : "f"(r));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(ud) : "l"(ua), "l"(ur));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(ud));
    return d;
}

// Sixteen codes for the MMA operand (a minus zero may stay: as an operand it only ever contributes a
// signed zero to the sum; NaN becomes code 0).
__device__ __forceinline__ uint32_t e4m3x4_op(float t0, float t1, float t2, float t3, bool& nan)
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

__global__ void __launch_bounds__(NTHREADS, 1) fpq_pair_conv_kernel(const __grid_constant__ CUtensorMap tmX,
                                                                    const __grid_constant__ CUtensorMap tmB,
                                                                    const PairArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    // layout: [A ring][weights][FP32 staging ring][barriers][x_scale * w_scale | bias]
    const uint32_t a_ring = smem_base;
    const uint32_t b_base = a_ring + g.a_stages * g.a_stage_bytes;
    const uint32_t x_ring = b_base + g.nblk * g.b_block_bytes;
    const uint32_t bars = x_ring + g.x_stages * g.x_stage_bytes;
    const uint32_t x_full = bars, x_empty = bars + 64, a_full = bars + 128, a_empty = bars + 160;
    const uint32_t b_full = bars + 192, acc_full = bars + 320, acc_empty = bars + 336, b_peer = bars + 384;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (bars - smem_base) + 352);
    float* s_scale = reinterpret_cast<float*>(smem + (bars - smem_base) + 512);
    float* s_bias = s_scale + g.BN;

    // launched with programmatic stream serialization: the next kernel in the stream may be set up while this one
    // runs (its CTAs become resident as this kernel's CTAs leave)
    asm volatile("griddepcontrol.launch_dependents;");
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();            // 0: the pair's first CTA (issues the MMAs)
    const int BNh = g.BN >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(x_full + 8 * s, 1);
            mbar_init(x_empty + 8 * s, NUM_XF);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(a_full + 8 * s, 2 * NUM_XF);       // the transform warps of both CTAs
            mbar_init(a_empty + 8 * s, 1);
        }
        for (int s = 0; s < MAX_CHUNKS; ++s) {
            mbar_init(b_full + 8 * s, 1);
            mbar_init(b_peer + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, 2 * NUM_EPI);   // the epilogue warps of both CTAs
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32((const void*)tmem_slot), g.tmem_cols);
        tmem_relinquish_pair();
    }
    // both CTAs' barriers exist before anything arrives on them from the other CTA
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above (barriers, tensor memory) overlapped the tail of the kernel in front; nothing below touches
    // global memory before that kernel has completed and its writes are visible
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // the pair's first CTA's copy of a barrier, as a cluster-space address
    auto leader = [&](uint32_t bar) { return peer_smem_addr(bar, 0u); };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            bool dead = false, b_issued = false;
            uint32_t sx = 0, px = 0, nx = 0;
            auto issue_weights = [&]() {
                // this CTA's half of the weights, one box {128 bytes, BN/2 rows, all taps} per chunk, reported to this
                // CTA's own barrier (a load that reports to a barrier of the other CTA was several times slower);
                // warp 3 of the second CTA passes the news on to the MMA issuer
                for (int cc = 0; cc < g.cchunks; ++cc) {
                    mbar_expect_tx(b_full + 8 * cc, (uint32_t)g.taps * g.b_block_tx);
                    tma_load_3d(b_base + cc * g.taps * g.b_block_bytes, &tmB, b_full + 8 * cc, cc * BK, (int)rank * BNh, 0);
                }
                b_issued = true;
            };
            for (int step = 0; step < g.tiles_per_cta && !dead; ++step) {
                const int mt = (int)blockIdx.x * g.tiles_per_cta + step;
                const TileRows tr = tile_rows(g, mt, step);
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    uint32_t b = tr.b_lo, yp = tr.yp_lo;
                    for (int k = 0; k < tr.ngrp; ++k) {
                        // rows yp .. yp + x_nr - 1 of image b; a row past the image's frame is the top frame row of
                        // the next image (x_nr - 1 <= pad), which the out-of-range fill supplies as zeros too
                        const int y = (int)yp - g.pad;
                        if ((int)b < g.B && y + g.x_nr > 0 && y < g.H) {
                            if (!mbar_wait(x_empty + 8 * sx, px ^ 1)) { dead = true; break; }
                            mbar_expect_tx(x_full + 8 * sx, (uint32_t)g.x_stage_bytes);
                            tma_load_4d(x_ring + sx * g.x_stage_bytes, &tmX, x_full + 8 * sx, 0, cc * BK, y, (int)b);
                            ++nx;
                            if (++sx == (uint32_t)g.x_stages) { sx = 0; px ^= 1; }
                            // the first rows go first so that the transform warps have work while the weights load
                            if (!b_issued && nx == (uint32_t)g.x_stages)
                                issue_weights();
                        }
                        yp += (uint32_t)g.x_nr;
                        if (yp >= (uint32_t)g.Hp) { yp -= (uint32_t)g.Hp; ++b; }
                    }
                }
            }
            if (!b_issued)
                issue_weights();
            if (dead) {
                flag_status(g.status, FPQ_ERR_TIMEOUT);
                for (uint32_t i = (nx > (uint32_t)g.x_stages ? nx - g.x_stages : 0); i < nx; ++i)
                    (void)mbar_wait(x_full + 8 * (i % g.x_stages), (i / g.x_stages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: one thread of the pair's first CTA ----------------
        if (rank == 0 && elect_one()) {
            uint32_t sa = 0, pa = 0, it = 0;
            bool dead = false;
            const uint32_t HI = SMEM_DESC_HI_K_SW128;
            const uint32_t BSTEP = (uint32_t)g.b_block_bytes >> 4;
            const uint32_t b_lo0 = smem_desc_lo(b_base);
            const uint32_t row_wrap8 = (uint32_t)(g.Wp - g.S) * 8u;
            for (int step = 0; step < g.tiles_per_cta && !dead; ++step, ++it) {
                const uint32_t buf = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait_cluster(acc_empty + 8 * buf, aph ^ 1)) { dead = true; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + buf * (uint32_t)g.BN;
                int j = 0;
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    if (!mbar_wait_cluster(a_full + 8 * sa, pa)) { dead = true; break; }
                    tc_fence_after();
                    const uint32_t abase = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                    uint32_t off8 = 0;
                    int sxx = 0;
                    for (int tap = 0; tap < g.taps; ++tap, ++j) {
                        if (it == 0 && tap == 0) {
                            // the weights arrive once, chunk by chunk
                            if (!mbar_wait(b_full + 8 * cc, 0) || !mbar_wait_cluster(b_peer + 8 * cc, 0)) { dead = true; break; }
                            tc_fence_after();
                        }
                        const uint32_t al = abase + off8, bl = b_lo0 + (uint32_t)j * BSTEP;
                        if (j == 0)
                            mma_f8f6f4_pair<false>(d, al, bl, HI, g.idesc);
                        else
                            mma_f8f6f4_pair<true>(d, al, bl, HI, g.idesc);
                        mma_f8f6f4_pair<true>(d, al + 2, bl + 2, HI, g.idesc);
                        mma_f8f6f4_pair<true>(d, al + 4, bl + 4, HI, g.idesc);
                        mma_f8f6f4_pair<true>(d, al + 6, bl + 6, HI, g.idesc);
                        off8 += 8;
                        if (++sxx == g.S) { sxx = 0; off8 += row_wrap8; }
                    }
                    if (dead)
                        break;
                    mma_commit_pair(a_empty + 8 * sa, 3);          // both CTAs' stage is free again
                    if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                }
                if (dead)
                    break;
                mma_commit_pair(acc_full + 8 * buf, 3);
            }
            if (dead)
                flag_status(g.status, FPQ_ERR_TIMEOUT);
        }
    } else if (warp == 3) {
        // ---------------- second CTA: tell the MMA issuer when this CTA's weights have landed ----------------
        if (rank == 1 && lane == 0) {
            const uint32_t rb = leader(b_peer);
            for (int cc = 0; cc < g.cchunks; ++cc) {
                if (!mbar_wait(b_full + 8 * cc, 0)) {
                    flag_status(g.status, FPQ_ERR_TIMEOUT);
                    break;
                }
                mbar_arrive_cluster(rb + 8 * cc);
            }
        }
    } else if (warp == 2) {
        // ---------------- L2 prefetch: every 128-byte line of FP32 activations this CTA's tiles will read ----------------
        // (runs ahead of the producer and synchronises with nobody: a TMA load that hits the L2 takes a third of
        // the time of one that goes to DRAM)
        for (int step = 0; step < g.tiles_per_cta; ++step) {
            const int mt = (int)blockIdx.x * g.tiles_per_cta + step;
            const TileRows tr = tile_rows(g, mt, step);
            uint32_t b = tr.b_lo, yp = tr.yp_lo;
            const int row_bytes = g.W * 4;
            for (int r = 0; r < tr.nrow; ++r) {
                const int y = (int)yp - g.pad;
                if ((int)b < g.B && (unsigned)y < (unsigned)g.H) {
                    for (int c = lane; c < g.C; c += 32) {
                        const char* p0 = reinterpret_cast<const char*>(g.x + (((int64_t)b * g.C + c) * g.H + y) * g.W);
                        for (int o = 0; o < row_bytes; o += 128)
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(p0 + o));
                    }
                }
                if (++yp == (uint32_t)g.Hp) { yp = 0; ++b; }
            }
        }
    } else if (warp >= EPI_W0 && warp < EPI_W0 + NUM_EPI) {
        // ---------------- epilogue: y = acc * (x_scale * w_scale[n]) + bias[n], NCHW ----------------
        const int quarter = warp & 3, half = (warp - EPI_W0) >> 2;
        const int row = quarter * 32 + lane;
        for (int i = threadIdx.x - 32 * EPI_W0; i < g.BN; i += 32 * NUM_EPI) {
            s_scale[i] = (i < g.N) ? g.x_scale * __ldg(g.w_scale + i) : 0.f;
            s_bias[i] = (g.bias && i < g.N) ? __ldg(g.bias + i) : 0.f;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * NUM_EPI) : "memory");
        const uint32_t racc_empty = leader(acc_empty);
        const int64_t nstride = (int64_t)g.Ho * g.Wo;
        uint32_t it = 0;
        bool dead = false;
        for (int step = 0; step < g.tiles_per_cta && !dead; ++step, ++it) {
            const int mt = (int)blockIdx.x * g.tiles_per_cta + step;
            const uint32_t buf = it & 1, aph = (it >> 1) & 1;
            // where this thread's pixel goes
            const uint32_t q = (uint32_t)mt * BM + row;
            const uint32_t b = fdiv(q, g.div_HpWp);
            const uint32_t rem = q - b * (uint32_t)g.HpWp;
            const int oy = (int)fdiv(rem, g.div_Wp);
            const int ox = (int)rem - oy * g.Wp;
            const bool row_valid = ox < g.Wo && oy < g.Ho && (int)b < g.B;
            float* yrow = g.y + ((int64_t)b * g.N * g.Ho + oy) * g.Wo + ox;
            if (!mbar_wait(acc_full + 8 * buf, aph)) { dead = true; break; }
            tc_fence_after();
            const int ncol0 = half * BNh;
            const uint32_t t_addr = tmem_base + buf * (uint32_t)g.BN + (uint32_t)ncol0 + ((uint32_t)(quarter * 32) << 16);
            for (int c = 0; c < BNh; c += 32) {
                const int nb = ncol0 + c;
                if (nb >= g.N)
                    break;
                uint32_t r[32];
                tmem_ld32(t_addr + c, r);
                tmem_ld_wait();
                const float4* s4 = reinterpret_cast<const float4*>(s_scale + nb);
                const float4* b4 = reinterpret_cast<const float4*>(s_bias + nb);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 sv = s4[k], bv = b4[k];
                    r[4 * k + 0] = __float_as_uint(fmaf(__uint_as_float(r[4 * k + 0]), sv.x, bv.x));
                    r[4 * k + 1] = __float_as_uint(fmaf(__uint_as_float(r[4 * k + 1]), sv.y, bv.y));
                    r[4 * k + 2] = __float_as_uint(fmaf(__uint_as_float(r[4 * k + 2]), sv.z, bv.z));
                    r[4 * k + 3] = __float_as_uint(fmaf(__uint_as_float(r[4 * k + 3]), sv.w, bv.w));
                }
                if (row_valid) {
                    float* dst = yrow + (int64_t)nb * nstride;
                    if (nb + 32 <= g.N) {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            dst[(int64_t)k * nstride] = __uint_as_float(r[k]);
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if (nb + k < g.N)
                                dst[(int64_t)k * nstride] = __uint_as_float(r[k]);
                    }
                }
            }
            // hand the accumulator back to the MMA issuer (in the pair's first CTA)
            tc_fence_before();
            __syncwarp();
            if (lane == 0)
                mbar_arrive_cluster(racc_empty + 8 * buf);
        }
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    } else if (warp >= XF_W0) {
        // ---------------- transform: staged FP32 image rows -> E4M3 codes of the operand ----------------
        // Thread item = (pair of neighbouring pixels, 16-channel group): 16 eight-byte loads (half a warp reads
        // 128 contiguous bytes of one channel), 32 conversions, two 16-byte stores (operand rows i and i + 1).
        // The operand rows a tile shares with the previous tile of the strip are copied from that tile's stage.
        constexpr int NT = 32 * NUM_XF;
        const int tid = threadIdx.x - 32 * XF_W0;
        const uint32_t ra_full = leader(a_full);
        uint32_t sa = 0, pa = 0, sx = 0, px = 0;
        bool dead = false, nan = false;
        const int W2 = g.W >> 1;
        const int box_items = g.x_nr * W2 * 8;
        const uint4 zero = make_uint4(0, 0, 0, 0);
        for (int step = 0; step < g.tiles_per_cta; ++step) {
            const int mt = (int)blockIdx.x * g.tiles_per_cta + step;
            const TileRows tr = tile_rows(g, mt, step);
            // every transform warp is done with the previous tile, whose stage the copy below reads (a thread whose
            // wait ran out still comes here, so the barrier always completes)
            asm volatile("bar.sync 2, %0;" ::"n"(NT) : "memory");
            for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                if (!mbar_wait(a_empty + 8 * sa, pa ^ 1)) { dead = true; break; }
                uint8_t* dst = smem + sa * g.a_stage_bytes;
                if (tr.i_lo > 0) {
                    // operand rows [128, rows) of the previous tile are rows [0, rows - 128) of this one; a shift by
                    // 128 rows keeps the swizzle phase, so the 16-byte pieces are copied as they are
                    const uint32_t prev = (sa + (uint32_t)g.a_stages - (uint32_t)g.cchunks) % (uint32_t)g.a_stages;
                    const uint4* src = reinterpret_cast<const uint4*>(smem + prev * g.a_stage_bytes + BM * 128);
                    for (int p = tid; p < tr.i_lo * 8; p += NT)
                        reinterpret_cast<uint4*>(dst)[p] = src[p];
                }
                // zero codes: the frame pixels of the real image rows, all pixels of frame rows and of rows past the
                // batch.  One warp per image row (a thread's own instruction stream is slow: ~6 cycles per dependent
                // instruction, so the rows are not walked one after the other); lane = (pixel slot, 16-channel group)
                for (int r = tid >> 5; r < tr.nrow; r += NUM_XF) {
                    uint32_t yp = tr.yp_lo + (uint32_t)r, b = tr.b_lo;
                    while (yp >= (uint32_t)g.Hp) { yp -= (uint32_t)g.Hp; ++b; }
                    const int y = (int)yp - g.pad;
                    const bool real = (int)b < g.B && (unsigned)y < (unsigned)g.H;
                    const int bi = tr.base_i + r * g.Wp;
                    const int cg = lane & 7;
                    for (int e = lane >> 3; e < (real ? 2 * g.pad : g.Wp); e += 4) {
                        const int xp = real ? (e < g.pad ? e : g.W + e) : e;
                        const int i = bi + xp;
                        if (i >= tr.i_lo && i < g.rows)
                            *reinterpret_cast<uint4*>(dst + i * 128 + ((cg ^ (i & 7)) << 4)) = zero;
                    }
                }
                // the staged boxes
                uint32_t bg = tr.b_lo, ypg = tr.yp_lo;
                int bi = tr.base_i;
                for (int k = 0; k < tr.ngrp && !dead; ++k, bi += g.x_nr * g.Wp) {
                    const int yg = (int)ypg - g.pad;
                    const bool loaded = (int)bg < g.B && yg + g.x_nr > 0 && yg < g.H;   // the producer's own test
                    if (loaded) {
                        if (!mbar_wait(x_full + 8 * sx, px)) { dead = true; break; }
                        const float* xs = reinterpret_cast<const float*>(smem + (x_ring - smem_base) + sx * g.x_stage_bytes);
                        for (int idx = tid; idx < box_items; idx += NT) {
                            const int rest = (int)fdiv((uint32_t)idx, g.div_W2);
                            const int j = idx - rest * W2, cg = rest & 7, jr = rest >> 3;
                            const int y = yg + jr;
                            // (a row of the box past this image's frame belongs to the next image: a frame row, zeroed above)
                            if (k * g.x_nr + jr >= tr.nrow || (unsigned)y >= (unsigned)g.H || (int)ypg + jr >= g.Hp)
                                continue;
                            const int i0 = bi + jr * g.Wp + g.pad + 2 * j;
                            if (i0 + 1 < tr.i_lo || i0 >= g.rows)
                                continue;
                            const float* p = xs + ((jr * BK + cg * 16) * g.W + 2 * j);
                            float2 a[16];
#pragma unroll
                            for (int q = 0; q < 16; ++q)
                                a[q] = mul2(*reinterpret_cast<const float2*>(p + q * g.W), g.rinv);
                            uint4 v0, v1;
                            v0.x = e4m3x4_op(a[0].x, a[1].x, a[2].x, a[3].x, nan);
                            v0.y = e4m3x4_op(a[4].x, a[5].x, a[6].x, a[7].x, nan);
                            v0.z = e4m3x4_op(a[8].x, a[9].x, a[10].x, a[11].x, nan);
                            v0.w = e4m3x4_op(a[12].x, a[13].x, a[14].x, a[15].x, nan);
                            v1.x = e4m3x4_op(a[0].y, a[1].y, a[2].y, a[3].y, nan);
                            v1.y = e4m3x4_op(a[4].y, a[5].y, a[6].y, a[7].y, nan);
                            v1.z = e4m3x4_op(a[8].y, a[9].y, a[10].y, a[11].y, nan);
                            v1.w = e4m3x4_op(a[12].y, a[13].y, a[14].y, a[15].y, nan);
                            if (i0 >= tr.i_lo)
                                *reinterpret_cast<uint4*>(dst + i0 * 128 + ((cg ^ (i0 & 7)) << 4)) = v0;
                            const int i1 = i0 + 1;
                            if (i1 < g.rows)
                                *reinterpret_cast<uint4*>(dst + i1 * 128 + ((cg ^ (i1 & 7)) << 4)) = v1;
                        }
                        // the box has been read: hand the slot back to the producer
                        __syncwarp();
                        if (lane == 0)
                            mbar_arrive(x_empty + 8 * sx);
                        if (++sx == (uint32_t)g.x_stages) { sx = 0; px ^= 1; }
                    }
                    ypg += (uint32_t)g.x_nr;
                    if (ypg >= (uint32_t)g.Hp) { ypg -= (uint32_t)g.Hp; ++bg; }
                }
                if (dead)
                    break;
                // make the generic-proxy writes visible to the tensor cores' reads, then tell the MMA issuer
                fence_proxy_async();
                __syncwarp();
                if (lane == 0)
                    mbar_arrive_cluster(ra_full + 8 * sa);
                if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
            }
        }
        if (nan)
            flag_status(g.status, FPQ_ERR_NAN_INPUT);
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    }

    // nobody leaves while the other CTA may still arrive on this CTA's barriers or read its shared memory,
    // and both CTAs give their tensor memory back together
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, g.tmem_cols);
    }
}

}  // namespace

// FPQ_ERR_UNSUPPORTED: the shape is outside what this kernel covers (the caller takes another route).
// Geometry and shared-memory plan (no CUDA calls, no pointer is followed); FPQ_ERR_UNSUPPORTED outside the kernel's range.
static fpq_status plan_pair(const GemmProblem& p, PairArgs& g, int* dyn_bytes)
{
    if (!p.conv || p.x == nullptr || p.a_e5m2 || p.stride != 1 || p.c_seg != 0 || p.Cp / BK > MAX_CHUNKS || p.R * p.S > 256)
        return FPQ_ERR_UNSUPPORTED;
    if (p.W % 4 != 0 || p.W > 256 || (uintptr_t)p.x % 16 != 0 || p.N > 256 || p.N < 1)
        return FPQ_ERR_UNSUPPORTED;
    const int Hp = p.H + 2 * p.pad, Wp = p.W + 2 * p.pad;
    const int64_t framed = (int64_t)p.B * Hp * Wp;
    const int halo_rows = BM + (p.R - 1) * Wp + (p.S - 1);
    const int64_t flat_tiles = (framed + BM - 1) / BM;
    const int64_t exact_tiles = ((int64_t)p.B * p.Ho * p.Wo + BM - 1) / BM;
    if (halo_rows > 2 * 256 - 16 || flat_tiles * 4 > exact_tiles * 5 + 4 || framed >= 0x7fffff00ll)
        return FPQ_ERR_UNSUPPORTED;

    g = PairArgs{};
    g.M = framed;
    g.N = p.N;
    g.BN = (int)round_up(p.N, 64);
    g.cchunks = p.Cp / BK;
    g.taps = p.R * p.S;
    g.S = p.S;
    g.nblk = g.cchunks * g.taps;
    g.Wp = Wp;
    g.Hp = Hp;
    g.HpWp = Hp * Wp;
    g.div_Wp = make_fastdiv((uint32_t)Wp);
    g.div_Hp = make_fastdiv((uint32_t)Hp);
    g.div_HpWp = make_fastdiv((uint32_t)g.HpWp);
    g.B = p.B; g.C = p.C; g.H = p.H; g.W = p.W; g.pad = p.pad; g.Ho = p.Ho; g.Wo = p.Wo;
    g.m_tiles = (int)flat_tiles;
    g.div_W2 = make_fastdiv((uint32_t)(p.W / 2));
    g.rows = (int)round_up(halo_rows, 8);
    g.a_stage_bytes = g.rows * 128;
    g.x_rows = (Wp - 1 + g.rows - 1) / Wp + 1;
    // two image rows per staged box where the frame allows it (a box may reach one row into the next image
    // only if that row is a frame row) and the box stays within 32 KiB
    g.x_nr = (p.pad >= 1 && 2 * p.W * BK * 4 <= 32 * 1024) ? 2 : 1;
    g.x_groups = (g.x_rows + g.x_nr - 1) / g.x_nr;
    g.x_stage_bytes = g.x_nr * p.W * BK * 4;
    g.b_block_bytes = (g.BN / 2) * BK;
    g.b_block_tx = (uint32_t)g.b_block_bytes / (p.w4 ? 2 : 1);
    g.idesc = idesc_f8f6f4_pair(0u, p.w4 ? 5u : (p.w_e5m2 ? 1u : 0u), (uint32_t)g.BN);
    g.tmem_cols = 32;
    while (g.tmem_cols < 2u * (uint32_t)g.BN)
        g.tmem_cols <<= 1;
    // shared memory: the resident weights, two (or more) operand stages, then as deep a staging ring as fits
    const int ctl = 512 + 2 * g.BN * 4 + 1024;
    const int64_t fixed = (int64_t)g.nblk * g.b_block_bytes + ctl;
    g.a_stages = g.cchunks >= 2 ? 3 : 2;
    int64_t room = SMEM_BUDGET - fixed - (int64_t)g.a_stages * g.a_stage_bytes;
    if (room < 2ll * g.x_stage_bytes && g.x_nr > 1) {
        g.x_nr = 1;
        g.x_groups = g.x_rows;
        g.x_stage_bytes = p.W * BK * 4;
    }
    if (room < 3ll * g.x_stage_bytes && g.a_stages > 2) {
        g.a_stages = 2;
        room = SMEM_BUDGET - fixed - (int64_t)g.a_stages * g.a_stage_bytes;
    }
    if (room < 2ll * g.x_stage_bytes)
        return FPQ_ERR_UNSUPPORTED;
    g.x_stages = (int)(room / g.x_stage_bytes);
    if (g.x_stages > 8)
        g.x_stages = 8;
    *dyn_bytes = (int)(fixed + (int64_t)g.a_stages * g.a_stage_bytes + (int64_t)g.x_stages * g.x_stage_bytes);
    return FPQ_OK;
}

bool pair_conv_applies(const GemmProblem& p)
{
    PairArgs g;
    int dyn = 0;
    return plan_pair(p, g, &dyn) == FPQ_OK;
}

// Shapes on which this kernel measured faster than quantize kernel + contraction kernel on B200: one 128-channel
// chunk (with two chunks the two-kernel route's split reduction still wins).
bool pair_conv_preferred(const GemmProblem& p)
{
    return pair_conv_applies(p) && p.Cp / BK == 1;
}

fpq_status launch_pair_conv(const GemmProblem& p, cudaStream_t st)
{
    static std::mutex mu;
    static EncodeTiledFn enc = nullptr;
    static bool attr_set[64] = {};
    static int sms[64] = {};
    PairArgs g;
    int dyn = 0;
    const fpq_status planned = plan_pair(p, g, &dyn);
    if (planned != FPQ_OK)
        return planned;
    const int Hp = p.H + 2 * p.pad, Wp = p.W + 2 * p.pad;
    (void)Hp;
    (void)Wp;

    g.x = p.x;
    g.w_scale = p.w_scale;
    g.x_scale = p.x_scale;
    g.rinv = 1.0f / p.x_scale;
    g.bias = p.bias;
    g.y = p.y;
    g.status = status_word();
    if (!g.status)
        return FPQ_ERR_CUDA;

    int dev = 0, nsm = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!enc) {
            enc = tensor_map_encoder();
            if (!enc)
                return FPQ_ERR_CUDA;
        }
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
            return FPQ_ERR_CUDA;
        if (!attr_set[dev]) {
            if (cudaFuncSetAttribute(fpq_pair_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET) !=
                cudaSuccess)
                return FPQ_ERR_CUDA;
            int v = 0;
            if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 2)
                v = 148;
            sms[dev] = v;
            attr_set[dev] = true;
        }
        nsm = sms[dev];
    }

    // FP32 activations, NCHW: one box = one image row of 128 channels
    CUtensorMap tmX, tmB;
    {
        // (the channels are the map's second dimension: a box whose rows step through the second dimension
        // loads about twice as fast as one that steps through the third)
        cuuint64_t dims[4] = {(cuuint64_t)p.W, (cuuint64_t)p.C, (cuuint64_t)p.H, (cuuint64_t)p.B};
        cuuint64_t strides[3] = {(cuuint64_t)p.W * 4 * p.H, (cuuint64_t)p.W * 4, (cuuint64_t)p.W * 4 * p.H * p.C};
        cuuint32_t box[4] = {(cuuint32_t)p.W, BK, (cuuint32_t)g.x_nr, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, (void*)p.x, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
    }
    {
        // prepared weights [N][taps][Cp]; a box = this CTA's half of the output channels of one block
        cuuint64_t dims[3] = {(cuuint64_t)p.Cp, (cuuint64_t)p.N, (cuuint64_t)g.taps};
        const cuuint64_t rowB = p.w4 ? (cuuint64_t)p.Cp / 2 : (cuuint64_t)p.Cp;
        cuuint64_t strides[2] = {rowB * g.taps, rowB};
        cuuint32_t box[3] = {BK, (cuuint32_t)(g.BN / 2), (cuuint32_t)g.taps};
        cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&tmB, p.w4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, (void*)p.w_prepared,
                dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
    }

    int nclusters = nsm / 2;
    if (nclusters > (g.m_tiles + 1) / 2)
        nclusters = (g.m_tiles + 1) / 2;
    // every CTA walks a strip of consecutive tiles; the strips of a pair advance in step
    g.tiles_per_cta = (g.m_tiles + 2 * nclusters - 1) / (2 * nclusters);
    g.reuse = (g.a_stages > g.cchunks && g.rows > BM) ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * nclusters));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = (size_t)dyn;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, fpq_pair_conv_kernel, tmX, tmB, (const PairArgs)g) == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq
