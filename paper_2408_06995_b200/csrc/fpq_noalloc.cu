// fpq_linear_static: the quantized linear layer for callers that cannot hand the
// library a workspace.  The activation codes that fpq_linear keeps in the caller's
// workspace live here in a fixed device array that is part of the library image.
#include "fpq_common.cuh"

namespace {

// Scratch for the activation codes ([M][K rounded up to 16] bytes).  One copy per GPU
// that loads the library, held until the process exits.
static __device__ __align__(256) uint8_t g_static_scratch[FPQ_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device.  In host code the name
// g_static_scratch is only a handle for the runtime, not an address a kernel can
// use, so it is translated once per device with cudaGetSymbolAddress.
void* static_scratch_address()
{
    static void* addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return nullptr;
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess)
            return nullptr;
        addr[dev] = p;
    }
    return addr[dev];
}

}  // namespace

extern "C" fpq_status fpq_linear_static(const float* x, const void* w_prepared, const float* w_scale, float x_scale,
                                        fpq_format fx, fpq_format fw, const float* bias, float* y, int64_t M,
                                        int64_t N, int64_t K, void* stream)
{
    if (M < 0 || N < 0 || K < 0)
        return FPQ_ERR_SHAPE;
    // the size test comes first so that an oversized problem is reported as such
    const int64_t Kp = (K + 15) / 16 * 16;
    if (M > 0 && Kp > 0 && (M > (int64_t)FPQ_STATIC_SCRATCH_BYTES / Kp))
        return FPQ_ERR_TOO_LARGE;
    void* scratch = static_scratch_address();
    if (!scratch)
        return FPQ_ERR_CUDA;
    // Stage 1 rewrites every byte of the [M][Kp] region it later reads (padding
    // columns included), so nothing left over from an earlier call is ever used.
    return fpq_linear(x, w_prepared, w_scale, x_scale, fx, fw, bias, y, M, N, K, scratch,
                      (size_t)FPQ_STATIC_SCRATCH_BYTES, stream);
}
