// Shared device/host helpers of the fpq CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fpq.h"

namespace fpq {

// ---- format constants resolved on the host, passed to kernels by value --------
struct QFormat {
    int32_t e, m, B;
    int32_t code_max;     // largest magnitude code that may be produced
    uint32_t cmax_bits;   // FP32 bit pattern of the clipping value c
    int32_t sign_shift;   // e + m
    int32_t four_bit;     // 1 if codes are packed two per byte
    int32_t native_e4m3;  // 1 if (4, 3, bias 7, native saturation): hardware convert applies
};

bool resolve_format(fpq_format f, QFormat* q);   // false if the format is impossible
float format_cmax(fpq_format f);

// sticky device status word (defined in fpq_api.cu)
int* status_word();

// The status word holds one bit per kind of device-side event, so that a benign event (a NaN input quantized
// to zero) can never hide a serious one (a bounded wait that ran out, which leaves the output incomplete).
// fpq_read_status reports the most serious bit that is set.
constexpr int STATUS_BIT_NAN = 1, STATUS_BIT_TIMEOUT = 2;
__device__ __forceinline__ void flag_status(int* status, int code)
{
    atomicOr(status, code == FPQ_ERR_TIMEOUT ? STATUS_BIT_TIMEOUT : STATUS_BIT_NAN);
}

__host__ __device__ inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

// ---- the quantizer on one element ---------------------------------------------
// Clip, pick the step of the element's binade, round (nearest-even, or signed
// floor plus the learned decision h), clamp and encode, all on the FP32 bit
// pattern of t = x * (1/scale).  h < 0 selects round to nearest.
__device__ __forceinline__ uint32_t quantize_bits(float t, const QFormat& f, int h, bool& nan)
{
    uint32_t u = __float_as_uint(t);
    uint32_t neg = u >> 31;
    uint32_t au = u & 0x7fffffffu;
    if (au > 0x7f800000u) {
        nan = true;
        return 0;
    }
    au = min(au, f.cmax_bits);                       // clip (Inf included)
    int Eb = (int)(au >> 23);
    uint32_t mant = (au & 0x7fffffu) | (Eb ? 0x800000u : 0u);
    int Ebn = max(Eb, 1);                            // |a| = mant * 2^(Ebn - 150)
    int E = Ebn - 127;
    int e_eff = max(E, 1 - f.B);                     // binade whose step applies
    int shift = min(23 - f.m + (e_eff - E), 31);     // |a| / step = mant / 2^shift
    uint32_t fl = mant >> shift;
    uint32_t rem = mant & ((1u << shift) - 1u);
    uint32_t kmag;
    if (h < 0) {
        uint32_t half = 1u << (shift - 1);
        kmag = fl + ((rem > half) || (rem == half && (fl & 1u)) ? 1u : 0u);
    } else if (!neg) {
        kmag = fl + (uint32_t)h;
    } else {
        uint32_t c = fl + (rem ? 1u : 0u);           // floor of the signed value is -c
        if (c == 0) {                                // minus zero
            kmag = (uint32_t)h;
            neg = 0;
        } else {
            kmag = c - (uint32_t)h;
        }
    }
    int p1 = e_eff + f.B - 1;                        // exponent field - 1 of that binade
    uint32_t code;
    if (p1 >= 1 && kmag < (1u << f.m))               // fell into the finer binade below
        code = ((uint32_t)(p1 - 1) << f.m) + 2u * kmag;
    else
        code = ((uint32_t)p1 << f.m) + kmag;
    code = min(code, (uint32_t)f.code_max);
    if (code == 0)
        neg = 0;
    return code | (neg << f.sign_shift);
}

// Round-to-nearest-even only, any format, in a dozen instructions.  With s the step of the
// element's binade and C = 1.5 * 2^23 * s, the FP32 sum |a| + C is rounded by the hardware to a
// multiple of s (ties to the even multiple), and the multiple k = round(|a| / s) sits in the low
// mantissa bits of the sum.  (exponent field - 1 of the binade) * 2^m + k is the code for normal
// and subnormal results alike; a k of 2^(m+1) carries into the next exponent by itself.
__device__ __forceinline__ uint32_t quantize_rne_bits(float t, const QFormat& f, bool& nan)
{
    const uint32_t u = __float_as_uint(t);
    uint32_t au = u & 0x7fffffffu;
    if (au > 0x7f800000u) {
        nan = true;
        return 0;
    }
    au = min(au, f.cmax_bits);                                   // clip (Inf included)
    const int eb = max((int)(au >> 23), 128 - f.B);              // biased exponent of the binade whose step applies
    const uint32_t cbits = ((uint32_t)(eb - f.m + 23) << 23) | 0x400000u;
    const uint32_t k = __float_as_uint(__fadd_rn(__uint_as_float(au), __uint_as_float(cbits))) - cbits;
    uint32_t code = ((uint32_t)(eb - 128 + f.B) << f.m) + k;
    code = min(code, (uint32_t)f.code_max);
    return code ? code | ((u >> 31) << f.sign_shift) : 0u;
}

// Four E4M3 (bias 7, saturating at 448) codes from four scaled floats with the
// hardware convert; -0 and NaN are mapped to code 0 afterwards.
__device__ __forceinline__ uint32_t e4m3x4_from_scaled(float t0, float t1, float t2, float t3, bool& nan)
{
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(t1), "f"(t0));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(t3), "f"(t2));
    const uint32_t v = (uint32_t)lo | ((uint32_t)hi << 16);
    const uint32_t mag = v & 0x7f7f7f7fu;
    // bytes whose magnitude is not zero keep their sign bit (so -0 becomes +0)
    const uint32_t nonzero = (mag + 0x7f7f7f7fu) & 0x80808080u;
    // a magnitude of 0x7f can only come from a NaN input (finite values saturate at 0x7e)
    const uint32_t nan_bytes = (mag + 0x01010101u) & 0x80808080u;
    if (nan_bytes) {
        nan = true;
        const uint32_t full = (nan_bytes >> 7) * 0xffu;
        return (mag | (v & nonzero)) & ~full;
    }
    return mag | (v & nonzero);
}

// The same for the OCP E5M2 type (bias 15, saturating at 57344): a magnitude above 0x7b can only come from a NaN.
__device__ __forceinline__ uint32_t e5m2x4_from_scaled(float t0, float t1, float t2, float t3, bool& nan)
{
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(t1), "f"(t0));
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(t3), "f"(t2));
    const uint32_t v = (uint32_t)lo | ((uint32_t)hi << 16);
    const uint32_t mag = v & 0x7f7f7f7fu;
    const uint32_t nonzero = (mag + 0x7f7f7f7fu) & 0x80808080u;
    const uint32_t nan_bytes = (mag + 0x04040404u) & 0x80808080u;
    if (nan_bytes) {
        nan = true;
        const uint32_t full = (nan_bytes >> 7) * 0xffu;
        return (mag | (v & nonzero)) & ~full;
    }
    return mag | (v & nonzero);
}

// E5 = false: E4M3 codes; E5 = true: E5M2 codes (the tensor cores' two 8-bit activation types)
template <bool E5>
__device__ __forceinline__ uint32_t fp8x4_from_scaled(float t0, float t1, float t2, float t3, bool& nan)
{
    return E5 ? e5m2x4_from_scaled(t0, t1, t2, t3, nan) : e4m3x4_from_scaled(t0, t1, t2, t3, nan);
}

// ---- PTX wrappers ----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after `limit` SM cycles (by default 4e9, about two seconds) and reports false.
// The cycle counter is only consulted every 1024 unsuccessful polls.
constexpr long long MBAR_WAIT_LIMIT = 4000000000ll;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit = MBAR_WAIT_LIMIT)
{
    if (mbar_try_wait(bar, parity))
        return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 1024; ++i)
            if (mbar_try_wait(bar, parity))
                return true;
        if (clock64() - t0 > limit)
            return false;
    }
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void tma_prefetch_desc(const void* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// One lane of a converged warp (the hardware's pick), as a predicate the compiler knows to be
// true in exactly one thread: code behind it can live on the uniform datapath, which is where the
// MMA and TMA instructions take their descriptors from.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}

__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

__device__ __forceinline__ void tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// D[tmem] (+)= A[smem] * B[smem], 8-bit / 4-bit floating operands, FP32 accumulate.
// The matrix descriptors are passed as their two 32-bit halves (the low half holds the
// start address in 16-byte units and is the only part that moves), so advancing an
// operand costs one 32-bit add in the issuing thread.  ACC = false overwrites D.
template <bool ACC>
__device__ __forceinline__ void mma_f8f6f4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc)
{
    if (ACC) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.eq.u32 p, 1, 1;\n\t"
            "mov.b64 da, {%1, %3};\n\t"
            "mov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.eq.u32 p, 1, 0;\n\t"
            "mov.b64 da, {%1, %3};\n\t"
            "mov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
    }
}

// the barrier gets one arrival once all MMAs issued so far by this thread are done
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive FP32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle,
// groups of 8 rows 1024 bytes apart.  Low half: start address in 16-byte units (14 bits)
// and the (ignored) leading byte offset 1; high half: stride byte offset 1024 >> 4,
// descriptor version 1 (bit 46), layout type 2 = 128-byte swizzle (bits 61-63).
// The swizzle is a function of the shared-memory address itself, so a start address
// moved by whole 128-byte rows stays consistent with TMA-written data (base offset 0).
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr)
{
    return ((addr >> 4) & 0x3fffu) | (1u << 16);
}
constexpr uint32_t SMEM_DESC_HI_K_SW128 = 64u | (1u << 14) | (2u << 29);

// Instruction descriptor: FP32 accumulator, operand formats (0 = E4M3, 1 = E5M2, 5 = E2M1),
// both operands K-major, M = 128, N = n.
__host__ __device__ inline uint32_t idesc_f8f6f4(uint32_t a_fmt, uint32_t b_fmt, uint32_t n)
{
    return (1u << 4) | (a_fmt << 7) | (b_fmt << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// Division of a 31-bit unsigned number by a constant known on the host:
// n / d = (umulhi(n, mul) + n) >> shift.
struct FastDiv {
    uint32_t mul, shift;
};

inline FastDiv make_fastdiv(uint32_t d)
{
    FastDiv f{0, 0};
    if (d > 1) {
        uint32_t s = 0;
        while ((1ull << s) < d)
            ++s;
        f.shift = s;
        f.mul = (uint32_t)((((1ull << 32) * ((1ull << s) - d)) / d) + 1);
    }
    return f;
}

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv& f)
{
    return (uint32_t)(((uint64_t)__umulhi(n, f.mul) + n) >> f.shift);
}

// ---- thread-block cluster: barrier over all threads of all CTAs, and reads of a peer CTA's shared memory
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// address of this CTA's shared-memory location `local_addr` in CTA `peer` of the cluster
__device__ __forceinline__ uint32_t peer_smem_addr(uint32_t local_addr, uint32_t peer)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(peer));
    return remote;
}

__device__ __forceinline__ float4 ld_cluster_smem4(uint32_t cluster_addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(cluster_addr)
                 : "memory");
    return v;
}

// ---- CTA pairs (cta_group::2): one MMA spans the tensor cores and tensor memory of two CTAs of a cluster.
// Both CTAs allocate / free tensor memory with these; the MMAs and commits are issued by one thread of
// the cluster's first CTA, which names both CTAs' shared memory by the same offsets.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}

__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem of both CTAs] (+)= A * B with M = 256: each CTA holds 128 rows of A and of D, and half of B's rows.
template <bool ACC>
__device__ __forceinline__ void mma_f8f6f4_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc)
{
    if (ACC) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.eq.u32 p, 1, 1;\n\t"
            "mov.b64 da, {%1, %3};\n\t"
            "mov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.eq.u32 p, 1, 0;\n\t"
            "mov.b64 da, {%1, %3};\n\t"
            "mov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
    }
}

// one arrival on the barrier at this shared-memory offset in every CTA of `mask`, once all MMAs issued so
// far by this thread are done
__device__ __forceinline__ void mma_commit_pair(uint32_t bar, uint16_t mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}

// TMA load into this CTA's shared memory whose completion is reported to a barrier of the pair's first CTA
// (cluster-space address)
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// arrival on a barrier anywhere in the cluster (cluster-space address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar)
{
    // (default semantics, release at CTA scope: the cluster-scope release form took 1.8 us per arrival here; what
    // the other CTA's MMA reads afterwards is this CTA's own shared memory, already fenced for the async proxy)
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Bounded wait on a barrier of this CTA that other CTAs of the cluster arrive on.  It polls with test_wait:
// a thread suspended in try_wait was not woken by an arrival from another CTA until its time limit ran out
// (about 2 us per wait, measured).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity)
{
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 1024; ++i) {
            uint32_t ok;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(ok)
                : "r"(bar), "r"(parity)
                : "memory");
            if (ok)
                return true;
            __nanosleep(20);
        }
        if (clock64() - t0 > 4000000000ll)
            return false;
    }
}

// Instruction descriptor of the pair form: as idesc_f8f6f4 with M = 256.
__host__ __device__ inline uint32_t idesc_f8f6f4_pair(uint32_t a_fmt, uint32_t b_fmt, uint32_t n)
{
    return (1u << 4) | (a_fmt << 7) | (b_fmt << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}

}  // namespace fpq
