// The low-bit contraction of a stride-1 convolution on CTA pairs (tcgen05 cta_group::2, M = 256): the
// wide-MMA form for layers whose time is the tensor cores' (long reductions, many output channels).
// Activation codes come from the quantize kernel (zero-framed channels-last E4M3, as for the general
// contraction), weights from the prepared copy; both are streamed by TMA.
//
// One MMA spans two CTAs: each CTA holds its own 128 output pixels (rows of A and of the accumulator in
// its tensor memory) and HALF of the weight rows of the column tile, so per MMA an SM reads 4 KB of
// activations and 2 KB (BN = 128) or 4 KB (BN = 256) of weights from shared memory instead of 4 + 4 KB
// for half the work, and every weight byte is fetched once per 256 pixels.  Per CTA: warp 0 TMA producer
// (its own activation chunk, its half of the weight blocks, three taps per box: a TMA load costs about
// one memory latency whatever its size), warp 1 tensor-memory owner (and, in the pair's first CTA, the
// MMA issuer for both), warps 2-9 epilogue (tcgen05.ld -> acc * (x_scale * w_scale[n]) + bias[n] -> NCHW).
// Two accumulators: a unit's epilogue overlaps the next unit's MMAs.  Every wait is bounded; no TMA multicast.
#include <cuda.h>

#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"
#include "fpq_tensormap.h"

namespace fpq {

namespace {

constexpr int BM = 128;
constexpr int BK = 128;
constexpr int EPI_W0 = 2, NUM_EPI = 8;
constexpr int NTHREADS = 32 * (EPI_W0 + NUM_EPI);
constexpr int SMEM_BUDGET = 227 * 1024;

struct PGArgs {
    int64_t M;                 // framed pixels B * Hp * Wp
    int N, BN;                 // outputs; column tile (128 or 256), BN / 2 weight rows per CTA
    int cchunks, taps, S;
    int tgroup, ngroups;       // taps per weight stage, weight stages per chunk
    int Wp, HpWp;
    FastDiv div_Wp, div_HpWp, div_nt;
    int B, Ho, Wo;
    int m_tiles, n_tiles, units;   // a unit = (pair of row tiles, column tile), column tile fastest
    int a_boxes, a_box_rows, a_stage_bytes, a_stages;
    int b_tap_bytes, b_stage_bytes, b_stages;
    uint32_t a_tx, b_tx;       // bytes one CTA's loads of a stage report
    uint32_t idesc, tmem_cols;
    int wait_prior_grid;
    int n_pad;                 // N rounded up to the column tile: x_scale * w_scale[n] and bias[n] of all columns sit in shared memory
    const float* w_scale;
    float x_scale;
    const float* bias;
    float* y;
    int* status;
};

__global__ void __launch_bounds__(NTHREADS, 1) fpq_pair_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                    const __grid_constant__ CUtensorMap tmB,
                                                                    const PGArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    // layout: [A ring][B ring][barriers][x_scale * w_scale | bias of the CTA's current column tile, two copies]
    const uint32_t a_ring = smem_base;
    const uint32_t b_ring = a_ring + g.a_stages * g.a_stage_bytes;
    const uint32_t bars = b_ring + g.b_stages * g.b_stage_bytes;
    const uint32_t a_full = bars, a_empty = bars + 64, b_full = bars + 128, b_empty = bars + 192;
    const uint32_t acc_full = bars + 256, acc_empty = bars + 272;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (bars - smem_base) + 288);
    float* s_scale = reinterpret_cast<float*>(smem + (bars - smem_base) + 512);   // [n_pad] x_scale * w_scale, then [n_pad] bias
    float* s_bias = s_scale + g.n_pad;

    asm volatile("griddepcontrol.launch_dependents;");
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int cluster = (int)blockIdx.x >> 1, nclusters = (int)gridDim.x >> 1;
    const int BNh = g.BN >> 1;
    // every cluster walks a contiguous range of units: consecutive units share the pair of row tiles
    const int u_lo = (int)((int64_t)cluster * g.units / nclusters), u_hi = (int)((int64_t)(cluster + 1) * g.units / nclusters);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(a_full + 8 * s, 1);
            mbar_init(a_empty + 8 * s, 1);
            mbar_init(b_full + 8 * s, 1);
            mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, 2 * NUM_EPI);   // the epilogue warps of both CTAs
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32((const void*)tmem_slot), g.tmem_cols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // the activation codes are written by the kernel in front (and the output may alias something it reads)
    asm volatile("griddepcontrol.wait;" ::: "memory");

    auto leader = [&](uint32_t bar) { return peer_smem_addr(bar, 0u); };
    auto decode = [&](int u, int& mu, int& nt) {
        mu = (int)fdiv((uint32_t)u, g.div_nt);
        nt = u - mu * g.n_tiles;
    };

    if (warp == 0) {
        // ---------------- TMA producer: loads in the order the MMAs consume them ----------------
        if (elect_one()) {
            uint32_t sa = 0, pa = 0, sb = 0, pb = 0;
            bool dead = false;
            const uint32_t ra_full = leader(a_full), rb_full = leader(b_full);
            for (int u = u_lo; u < u_hi && !dead; ++u) {
                int mu, nt;
                decode(u, mu, nt);
                const int mt = 2 * mu + (int)rank;
                const int n0 = nt * g.BN + (int)rank * BNh;
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    if (!mbar_wait(a_empty + 8 * sa, pa ^ 1)) { dead = true; break; }
                    if (rank == 0)
                        mbar_expect_tx(a_full + 8 * sa, 2u * g.a_tx);
                    for (int bx = 0; bx < g.a_boxes; ++bx)
                        tma_load_4d_pair(a_ring + sa * g.a_stage_bytes + bx * g.a_box_rows * 128, &tmA, ra_full + 8 * sa,
                                         cc * BK, mt * BM + bx * g.a_box_rows, 0, 0);
                    if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                    for (int tg = 0; tg < g.ngroups; ++tg) {
                        if (!mbar_wait(b_empty + 8 * sb, pb ^ 1)) { dead = true; break; }
                        if (rank == 0)
                            mbar_expect_tx(b_full + 8 * sb, 2u * g.b_tx);
                        tma_load_3d_pair(b_ring + sb * g.b_stage_bytes, &tmB, rb_full + 8 * sb, cc * BK, n0, tg * g.tgroup);
                        if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                    }
                }
            }
            if (dead)
                flag_status(g.status, FPQ_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: one thread of the pair's first CTA ----------------
        if (rank == 0 && elect_one()) {
            uint32_t sa = 0, pa = 0, sb = 0, pb = 0, it = 0;
            bool dead = false;
            const uint32_t HI = SMEM_DESC_HI_K_SW128;
            const uint32_t TSTEP = (uint32_t)g.b_tap_bytes >> 4;
            const uint32_t row_wrap8 = (uint32_t)(g.Wp - g.S) * 8u;
            for (int u = u_lo; u < u_hi && !dead; ++u, ++it) {
                const uint32_t buf = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait_cluster(acc_empty + 8 * buf, aph ^ 1)) { dead = true; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + buf * (uint32_t)g.BN;
                bool first = true;
                for (int cc = 0; cc < g.cchunks && !dead; ++cc) {
                    if (!mbar_wait_cluster(a_full + 8 * sa, pa)) { dead = true; break; }
                    tc_fence_after();
                    const uint32_t abase = smem_desc_lo(a_ring + sa * g.a_stage_bytes);
                    uint32_t off8 = 0;
                    int sxx = 0;
                    for (int tg = 0; tg < g.ngroups && !dead; ++tg) {
                        if (!mbar_wait_cluster(b_full + 8 * sb, pb)) { dead = true; break; }
                        tc_fence_after();
                        const uint32_t bbase = smem_desc_lo(b_ring + sb * g.b_stage_bytes);
                        for (int t = 0; t < g.tgroup; ++t) {
                            const uint32_t al = abase + off8, bl = bbase + (uint32_t)t * TSTEP;
                            if (first)
                                mma_f8f6f4_pair<false>(d, al, bl, HI, g.idesc);
                            else
                                mma_f8f6f4_pair<true>(d, al, bl, HI, g.idesc);
                            first = false;
                            mma_f8f6f4_pair<true>(d, al + 2, bl + 2, HI, g.idesc);
                            mma_f8f6f4_pair<true>(d, al + 4, bl + 4, HI, g.idesc);
                            mma_f8f6f4_pair<true>(d, al + 6, bl + 6, HI, g.idesc);
                            off8 += 8;
                            if (++sxx == g.S) { sxx = 0; off8 += row_wrap8; }
                        }
                        mma_commit_pair(b_empty + 8 * sb, 3);
                        if (++sb == (uint32_t)g.b_stages) { sb = 0; pb ^= 1; }
                    }
                    if (dead)
                        break;
                    mma_commit_pair(a_empty + 8 * sa, 3);
                    if (++sa == (uint32_t)g.a_stages) { sa = 0; pa ^= 1; }
                }
                if (dead)
                    break;
                mma_commit_pair(acc_full + 8 * buf, 3);
            }
            if (dead)
                flag_status(g.status, FPQ_ERR_TIMEOUT);
        }
    } else {
        // ---------------- epilogue: y = acc * (x_scale * w_scale[n]) + bias[n], NCHW ----------------
        const int quarter = warp & 3, half = (warp - EPI_W0) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t racc_empty = leader(acc_empty);
        const int64_t nstride = (int64_t)g.Ho * g.Wo;
        for (int i = threadIdx.x - 32 * EPI_W0; i < g.n_pad; i += 32 * NUM_EPI) {
            s_scale[i] = (i < g.N) ? g.x_scale * __ldg(g.w_scale + i) : 0.f;
            s_bias[i] = (g.bias && i < g.N) ? __ldg(g.bias + i) : 0.f;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * NUM_EPI) : "memory");
        uint32_t it = 0;
        bool dead = false;
        for (int u = u_lo; u < u_hi && !dead; ++u, ++it) {
            int mu, nt;
            decode(u, mu, nt);
            const int mt = 2 * mu + (int)rank;
            const uint32_t buf = it & 1, aph = (it >> 1) & 1;
            const uint32_t q = (uint32_t)mt * BM + row;
            const uint32_t b = fdiv(q, g.div_HpWp);
            const uint32_t rem = q - b * (uint32_t)g.HpWp;
            const int oy = (int)fdiv(rem, g.div_Wp);
            const int ox = (int)rem - oy * g.Wp;
            const bool row_valid = (int64_t)q < g.M && ox < g.Wo && oy < g.Ho && (int)b < g.B;
            float* yrow = g.y + ((int64_t)b * g.N * g.Ho + oy) * g.Wo + ox;
            if (!mbar_wait(acc_full + 8 * buf, aph)) { dead = true; break; }
            tc_fence_after();
            const int ncol0 = half * BNh;                          // first column of this warp within the tile
            const uint32_t t_addr = tmem_base + buf * (uint32_t)g.BN + (uint32_t)ncol0 + ((uint32_t)(quarter * 32) << 16);
            for (int c = 0; c < BNh; c += 32) {
                const int nb = nt * g.BN + ncol0 + c;              // output channel of the chunk's first column
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
            tc_fence_before();
            __syncwarp();
            if (lane == 0)
                mbar_arrive_cluster(racc_empty + 8 * buf);
        }
        if (dead)
            flag_status(g.status, FPQ_ERR_TIMEOUT);
    }

    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, g.tmem_cols);
    }
}

// geometry and shared-memory plan; FPQ_ERR_UNSUPPORTED outside the kernel's range
fpq_status plan_pg(const GemmProblem& p, int nsm, PGArgs& g, int* dyn_bytes)
{
    if (!p.conv || p.x != nullptr || p.stride != 1 || p.c_seg != 0 || p.N < 1 || p.R * p.S > 64)
        return FPQ_ERR_UNSUPPORTED;
    const int Hp = p.H + 2 * p.pad, Wp = p.W + 2 * p.pad;
    const int64_t framed = (int64_t)p.B * Hp * Wp;
    const int halo_rows = BM + (p.R - 1) * Wp + (p.S - 1);
    const int64_t flat_tiles = (framed + BM - 1) / BM;
    const int64_t exact_tiles = ((int64_t)p.B * p.Ho * p.Wo + BM - 1) / BM;
    if (halo_rows > 2 * 256 - 16 || flat_tiles * 4 > exact_tiles * 5 + 4 || framed >= 0x7fffff00ll)
        return FPQ_ERR_UNSUPPORTED;
    g = PGArgs{};
    g.M = framed;
    g.N = p.N;
    g.cchunks = p.Cp / BK;
    g.taps = p.R * p.S;
    g.S = p.S;
    g.tgroup = (g.taps % 3 == 0) ? 3 : 1;
    g.ngroups = g.taps / g.tgroup;
    g.Wp = Wp;
    g.HpWp = Hp * Wp;
    g.div_Wp = make_fastdiv((uint32_t)Wp);
    g.div_HpWp = make_fastdiv((uint32_t)g.HpWp);
    g.B = p.B; g.Ho = p.Ho; g.Wo = p.Wo;
    g.m_tiles = (int)flat_tiles;
    const int m_units = (g.m_tiles + 1) / 2;
    const int nclusters = nsm / 2;
    // 256-wide column tiles halve the weight traffic per MMA, but a cluster needs at least two units for its
    // epilogue to overlap the next unit's MMAs
    g.BN = (p.N > 128 && (int64_t)m_units * ((p.N + 255) / 256) >= 2ll * nclusters) ? 256 : 128;
    g.n_tiles = (p.N + g.BN - 1) / g.BN;
    g.div_nt = make_fastdiv((uint32_t)g.n_tiles);
    g.units = m_units * g.n_tiles;
    g.a_boxes = halo_rows > 256 ? 2 : 1;
    g.a_box_rows = (int)round_up((halo_rows + g.a_boxes - 1) / g.a_boxes, 8);
    g.a_stage_bytes = g.a_boxes * g.a_box_rows * 128;
    g.a_tx = (uint32_t)g.a_stage_bytes;
    g.b_tap_bytes = (g.BN / 2) * BK;
    g.b_stage_bytes = g.tgroup * g.b_tap_bytes;
    g.b_tx = (uint32_t)g.b_stage_bytes / (p.w4 ? 2 : 1);
    g.n_pad = g.n_tiles * g.BN;
    if (g.n_pad * 8 > 32 * 1024)
        return FPQ_ERR_UNSUPPORTED;
    const int ctl = 512 + 1024 + g.n_pad * 8;
    g.a_stages = 2;
    g.b_stages = (SMEM_BUDGET - ctl - g.a_stages * g.a_stage_bytes) / g.b_stage_bytes;
    if (g.b_stages > 8)
        g.b_stages = 8;
    if (g.b_stages < 2)
        return FPQ_ERR_UNSUPPORTED;
    // a third activation stage if the weights still keep three
    if (g.b_stages >= 4 && SMEM_BUDGET - ctl - 3 * g.a_stage_bytes - 3 * g.b_stage_bytes >= 0) {
        g.a_stages = 3;
        g.b_stages = (SMEM_BUDGET - ctl - g.a_stages * g.a_stage_bytes) / g.b_stage_bytes;
        if (g.b_stages > 8)
            g.b_stages = 8;
    }
    g.idesc = idesc_f8f6f4_pair(p.a_e5m2 ? 1u : 0u, p.w4 ? 5u : (p.w_e5m2 ? 1u : 0u), (uint32_t)g.BN);
    g.tmem_cols = 2u * (uint32_t)g.BN;
    g.wait_prior_grid = p.after_stage1;
    *dyn_bytes = ctl + g.a_stages * g.a_stage_bytes + g.b_stages * g.b_stage_bytes;
    return FPQ_OK;
}

}  // namespace

// The layers this kernel is meant for: enough units to fill the GPU's SM pairs and a reduction long enough for the
// tensor cores to be the bound (measured on B200 against the general contraction).
bool pair_gemm_preferred(const GemmProblem& p)
{
    PGArgs g;
    int dyn = 0;
    if (plan_pg(p, 148, g, &dyn) != FPQ_OK)
        return false;
    return g.units >= 60 && g.cchunks * g.taps >= 12;
}

fpq_status launch_pair_gemm(const GemmProblem& p, cudaStream_t st)
{
    static std::mutex mu;
    static EncodeTiledFn enc = nullptr;
    static bool attr_set[64] = {};
    static int sms[64] = {};
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
            if (cudaFuncSetAttribute(fpq_pair_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET) !=
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
    PGArgs g;
    int dyn = 0;
    const fpq_status planned = plan_pg(p, nsm, g, &dyn);
    if (planned != FPQ_OK)
        return planned;
    g.w_scale = p.w_scale;
    g.x_scale = p.x_scale;
    g.bias = p.bias;
    g.y = p.y;
    g.status = status_word();
    if (!g.status)
        return FPQ_ERR_CUDA;

    CUtensorMap tmA, tmB;
    {
        // activation codes: the zero-framed channels-last pixel list [B Hp Wp][Ca]
        cuuint64_t dims[4] = {(cuuint64_t)p.Ca, (cuuint64_t)g.M, 1, 1};
        cuuint64_t strides[3] = {(cuuint64_t)p.Ca, (cuuint64_t)p.Ca * (cuuint64_t)g.M, (cuuint64_t)p.Ca * (cuuint64_t)g.M};
        cuuint32_t box[4] = {BK, (cuuint32_t)g.a_box_rows, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void*)p.a_codes, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
    }
    {
        // prepared weights [N][taps][Cp]; a box = this CTA's half of a column tile for `tgroup` taps of one chunk
        cuuint64_t dims[3] = {(cuuint64_t)p.Cp, (cuuint64_t)p.N, (cuuint64_t)g.taps};
        const cuuint64_t rowB = p.w4 ? (cuuint64_t)p.Cp / 2 : (cuuint64_t)p.Cp;
        cuuint64_t strides[2] = {rowB * g.taps, rowB};
        cuuint32_t box[3] = {BK, (cuuint32_t)(g.BN / 2), (cuuint32_t)g.tgroup};
        cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&tmB, p.w4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, (void*)p.w_prepared,
                dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return FPQ_ERR_CUDA;
    }
    int nclusters = nsm / 2;
    if (nclusters > g.units)
        nclusters = g.units;
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
    return cudaLaunchKernelEx(&cfg, fpq_pair_gemm_kernel, tmA, tmB, (const PGArgs)g) == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq
