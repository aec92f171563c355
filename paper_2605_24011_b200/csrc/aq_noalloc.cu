// aq_linear_noalloc: the decode linear (M <= 8) for callers that must not
// allocate.  The float32 accumulation scratch that aq_linear keeps inside the
// handle lives here in a fixed array in device global memory instead, so the
// call itself reserves nothing: no cudaMalloc, no cudaFree, no pool.
#include "aq_internal.h"

namespace aq {

constexpr int64_t NOALLOC_MAX_N = AQ_NOALLOC_MAX_N;          // output features, after padding to 16
constexpr int NOALLOC_MAX_DEVICES = 64;

// [AQ_DECODE_MAX_M][NOALLOC_MAX_N] float32 = 512 KiB, held by every device that loads the library.
static __device__ __align__(256) float g_noalloc_scratch[AQ_DECODE_MAX_M * NOALLOC_MAX_N];

// In host code the symbol above is only a stand-in; kernels need the device
// address, looked up once per device with that device current.
static float* g_scratch_addr[NOALLOC_MAX_DEVICES] = {nullptr};

static cudaError_t scratch_for_current_device(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace aq

using namespace aq;

extern "C" aq_status_t aq_linear_noalloc(aq_handle_t h, const void* x_dev, void* y_dev, int M, aq_dtype_t xy_dtype,
                                         aq_stream_t stream) {
    if (!handle_ok(h) || !x_dev || !y_dev || ((uintptr_t)x_dev & 15u) || ((uintptr_t)y_dev & 15u)) return AQ_ERR_INVALID_ARG;
    if (xy_dtype != AQ_F16 && xy_dtype != AQ_BF16) return (xy_dtype == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    if (M < 1) return AQ_ERR_INVALID_ARG;
    const int64_t ld = (int64_t)h->NT * 16;
    if (M > AQ_DECODE_MAX_M || ld > NOALLOC_MAX_N) return AQ_ERR_UNSUPPORTED;   // beyond the fixed scratch
    float* scratch = nullptr;
    cudaError_t e = scratch_for_current_device(&scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps whatever the last call left: the sums must start from zero
    e = cudaMemsetAsync(scratch, 0, (size_t)M * ld * sizeof(float), s);
    if (e == cudaSuccess) e = launch_gemv(h, x_dev, xy_dtype, M, scratch, ld, s);
    if (e == cudaSuccess) e = launch_finalize(scratch, nullptr, ld, y_dev, xy_dtype, M, h->N, s);
    if (e != cudaSuccess) return cuda_fail(e);
    h->last_stream = s;
    return AQ_OK;
}
