// C-ABI entry points of libaq: argument checks, handle ownership, dispatch.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <new>

#include "aq_internal.h"
#include "aq_layout.cuh"

namespace aq {

static thread_local char g_last_err[256] = "";

aq_status_t cuda_fail(cudaError_t e) {
    snprintf(g_last_err, sizeof(g_last_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return AQ_ERR_CUDA;
}

bool handle_ok(aq_handle_t h) { return h != nullptr && h->magic == AQ_HANDLE_MAGIC; }

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int current_device() {
    int dev = 0;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// SM count of the current device (cached per device).
int sm_count() {
    static PerDeviceValue<int> cache;
    int n = 0;
    const int rc = cache.get(current_device(), &n, [](int dev, int* out) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) { cudaGetLastError(); v = 148; }
        *out = v;
        return 0;
    });
    return rc == 0 ? n : 148;
}

static aq_status_t check_arch(int* dev_out) {
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (major != 10) return AQ_ERR_ARCH;
    if (dev_out) *dev_out = dev;
    return AQ_OK;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static aq_status_t new_handle(int bits, int block, int64_t N, int64_t K, aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (block != 32 || bits < 2 || bits > 4) return AQ_ERR_UNSUPPORTED;
    if (N < 1 || K < 32 || (K % 32) != 0 || N > (int64_t)1 << 24 || K > (int64_t)1 << 24) return AQ_ERR_INVALID_ARG;
    int dev = 0;
    aq_status_t st = check_arch(&dev);
    if (st != AQ_OK) return st;
    aq_handle_s* h = new (std::nothrow) aq_handle_s();
    if (!h) return AQ_ERR_ALLOC;
    h->magic = AQ_HANDLE_MAGIC;
    h->bits = bits; h->device = dev; h->N = N; h->K = K;
    h->NT = (int)((N + 15) / 16);
    h->KP = (int)((K + 255) / 256);
    h->n_frags = (int64_t)h->NT * h->KP * 2;
    h->dev_bytes = (size_t)h->n_frags * frag_bytes(bits);
    h->frags = nullptr; h->acc = nullptr; h->flags = nullptr; h->last_stream = nullptr;
    h->big = nullptr; h->big_bytes = 0; h->sb = nullptr;
    const size_t acc_bytes = (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float);
    if (cudaMalloc(&h->frags, h->dev_bytes) != cudaSuccess || cudaMalloc(&h->acc, acc_bytes) != cudaSuccess ||
        cudaMalloc(&h->flags, 256) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(h->frags); cudaFree(h->acc); cudaFree(h->flags);
        delete h;
        return AQ_ERR_ALLOC;
    }
    *out = h;
    return AQ_OK;
}

static void destroy(aq_handle_s* h) {
    cudaFree(h->frags); cudaFree(h->acc); cudaFree(h->flags); cudaFree(h->big); cudaFree(h->sb);
    h->magic = 0;
    delete h;
}

}  // namespace aq

using namespace aq;

extern "C" {

aq_status_t aq_pack(int bits, int block, const float* W_dev, int64_t N, int64_t K, aq_stream_t stream,
                    aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!W_dev || !aligned16(W_dev)) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_handle(bits, block, N, K, &h);
    if (st != AQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(h->acc, 0, (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->flags, 0, 256, s);
    if (e == cudaSuccess) e = launch_pack(h, W_dev, s);
    if (e != cudaSuccess) { destroy(h); return cuda_fail(e); }
    h->last_stream = s;
    *out = h;
    return AQ_OK;
}

aq_status_t aq_pack_opt(int bits, int block, const float* W_dev, const float* F_dev, int rounds, int64_t N, int64_t K,
                        aq_stream_t stream, aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!W_dev || !aligned16(W_dev) || (F_dev && !aligned16(F_dev)) || rounds < 0 || rounds > 64) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_handle(bits, block, N, K, &h);
    if (st != AQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(h->acc, 0, (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->flags, 0, 256, s);
    if (e == cudaSuccess) e = launch_pack_opt(h, W_dev, F_dev, rounds, s);
    if (e != cudaSuccess) { destroy(h); return cuda_fail(e); }
    h->last_stream = s;
    *out = h;
    return AQ_OK;
}

static size_t sb_nbytes(int bits, int64_t N, int64_t K) { return (size_t)N * (size_t)(K / 256) * (size_t)(18 + 32 * bits); }

static aq_status_t new_sb_handle(int bits, int block, int sblock, int64_t N, int64_t K, aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (sblock != 8) return AQ_ERR_UNSUPPORTED;
    if (K < 256 || K % 256 != 0) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_handle(bits, block, N, K, &h);
    if (st != AQ_OK) return st;
    if (cudaMalloc(&h->sb, (size_t)N * (size_t)(K / 256) * 32) != cudaSuccess) { cudaGetLastError(); destroy(h); return AQ_ERR_ALLOC; }
    *out = h;
    return AQ_OK;
}

aq_status_t aq_pack_sb(int bits, int block, int sblock, const float* W_dev, int64_t N, int64_t K, aq_stream_t stream,
                       aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!W_dev || !aligned16(W_dev)) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_sb_handle(bits, block, sblock, N, K, &h);
    if (st != AQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(h->acc, 0, (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->flags, 0, 256, s);
    if (e == cudaSuccess) e = launch_pack_sb(h, W_dev, s);
    if (e != cudaSuccess) { destroy(h); return cuda_fail(e); }
    h->last_stream = s;
    *out = h;
    return AQ_OK;
}

aq_status_t aq_import_sb(int bits, int block, int sblock, int64_t N, int64_t K, const void* canon_host, size_t nbytes,
                         aq_stream_t stream, aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!canon_host) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_sb_handle(bits, block, sblock, N, K, &h);
    if (st != AQ_OK) return st;
    if (nbytes != sb_nbytes(bits, N, K)) { destroy(h); return AQ_ERR_INVALID_ARG; }
    cudaStream_t s = (cudaStream_t)stream;
    const size_t plain_bytes = (size_t)N * (size_t)(K / 32) * (size_t)(4 + 4 * bits);
    const size_t plain_at = (nbytes + 255) / 256 * 256;
    uint8_t* tmp = nullptr;
    if (cudaMalloc(&tmp, plain_at + plain_bytes) != cudaSuccess) { cudaGetLastError(); destroy(h); return AQ_ERR_ALLOC; }
    cudaError_t e = cudaMemcpyAsync(tmp, canon_host, nbytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->acc, 0, (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->flags, 0, 256, s);
    if (e == cudaSuccess) e = launch_sb_records(h, tmp, tmp + plain_at, true, s);
    if (e == cudaSuccess) e = launch_import(h, tmp + plain_at, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(tmp);
    if (e != cudaSuccess) { destroy(h); return cuda_fail(e); }
    h->last_stream = s;
    *out = h;
    return AQ_OK;
}

aq_status_t aq_import(int bits, int block, int64_t N, int64_t K, const void* canon_host, size_t nbytes,
                      aq_stream_t stream, aq_handle_t* out) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!canon_host) return AQ_ERR_INVALID_ARG;
    aq_handle_t h = nullptr;
    aq_status_t st = new_handle(bits, block, N, K, &h);
    if (st != AQ_OK) return st;
    if (nbytes != (size_t)N * (size_t)(K / 32) * (size_t)(4 + 4 * bits)) { destroy(h); return AQ_ERR_INVALID_ARG; }
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* tmp = nullptr;
    if (cudaMalloc(&tmp, nbytes) != cudaSuccess) { cudaGetLastError(); destroy(h); return AQ_ERR_ALLOC; }
    cudaError_t e = cudaMemcpyAsync(tmp, canon_host, nbytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->acc, 0, (size_t)AQ_DECODE_MAX_M * h->NT * 16 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->flags, 0, 256, s);
    if (e == cudaSuccess) e = launch_import(h, tmp, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(tmp);
    if (e != cudaSuccess) { destroy(h); return cuda_fail(e); }
    h->last_stream = s;
    *out = h;
    return AQ_OK;
}

static aq_status_t range_status(aq_handle_t h) {
    int flag = 0;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    if (e == cudaSuccess) e = cudaMemcpy(&flag, h->flags, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    return (flag & 1) ? AQ_ERR_RANGE : AQ_OK;
}

aq_status_t aq_export(aq_handle_t h, void* canon_host, size_t cap, size_t* nbytes) {
    if (!handle_ok(h)) return AQ_ERR_INVALID_ARG;
    const size_t need = (size_t)h->N * (size_t)(h->K / 32) * (size_t)(4 + 4 * h->bits);
    if (nbytes) *nbytes = need;
    if (!canon_host) return nbytes ? AQ_OK : AQ_ERR_INVALID_ARG;
    if (cap < need) return AQ_ERR_INVALID_ARG;
    uint8_t* tmp = nullptr;
    if (cudaMalloc(&tmp, need) != cudaSuccess) { cudaGetLastError(); return AQ_ERR_ALLOC; }
    cudaStream_t s = h->last_stream;
    cudaError_t e = launch_export(h, tmp, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(canon_host, tmp, need, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(tmp);
    if (e != cudaSuccess) return cuda_fail(e);
    return range_status(h);
}

aq_status_t aq_export_sb(aq_handle_t h, void* canon_host, size_t cap, size_t* nbytes) {
    if (!handle_ok(h) || !h->sb) return AQ_ERR_INVALID_ARG;
    const size_t need = sb_nbytes(h->bits, h->N, h->K);
    if (nbytes) *nbytes = need;
    if (!canon_host) return nbytes ? AQ_OK : AQ_ERR_INVALID_ARG;
    if (cap < need) return AQ_ERR_INVALID_ARG;
    const size_t plain_bytes = (size_t)h->N * (size_t)(h->K / 32) * (size_t)(4 + 4 * h->bits);
    const size_t plain_at = (need + 255) / 256 * 256;
    uint8_t* tmp = nullptr;
    if (cudaMalloc(&tmp, plain_at + plain_bytes) != cudaSuccess) { cudaGetLastError(); return AQ_ERR_ALLOC; }
    cudaStream_t s = h->last_stream;
    cudaError_t e = launch_export(h, tmp + plain_at, s);
    if (e == cudaSuccess) e = launch_sb_records(h, tmp, tmp + plain_at, false, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(canon_host, tmp, need, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(tmp);
    if (e != cudaSuccess) return cuda_fail(e);
    return range_status(h);
}

aq_status_t aq_info(aq_handle_t h, int* bits, int* block, int64_t* N, int64_t* K, size_t* packed_bytes,
                    size_t* device_bytes) {
    if (!handle_ok(h)) return AQ_ERR_INVALID_ARG;
    if (bits) *bits = h->bits;
    if (block) *block = 32;
    if (N) *N = h->N;
    if (K) *K = h->K;
    if (packed_bytes) *packed_bytes = h->sb ? sb_nbytes(h->bits, h->N, h->K) : (size_t)h->N * (size_t)(h->K / 32) * (size_t)(4 + 4 * h->bits);
    if (device_bytes) *device_bytes = h->dev_bytes + (h->sb ? (size_t)h->N * (size_t)(h->K / 256) * 32 : 0);
    return range_status(h);
}

aq_status_t aq_dequant(aq_handle_t h, void* out_dev, aq_dtype_t out_dtype, aq_stream_t stream) {
    if (!handle_ok(h) || !out_dev || !aligned16(out_dev)) return AQ_ERR_INVALID_ARG;
    if (out_dtype != AQ_F16 && out_dtype != AQ_BF16 && out_dtype != AQ_F32) return AQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = launch_dequant(h, out_dev, out_dtype, s);
    if (e != cudaSuccess) return cuda_fail(e);
    h->last_stream = s;
    return AQ_OK;
}

static aq_status_t linear_common(aq_handle_t h, const void* x_dev, void* y_dev, int M, aq_dtype_t xdt,
                                 aq_dtype_t ydt, aq_stream_t stream) {
    if (!handle_ok(h) || !x_dev || !y_dev || !aligned16(x_dev) || !aligned16(y_dev)) return AQ_ERR_INVALID_ARG;
    if (M < 1 || M > AQ_MAX_M) return AQ_ERR_INVALID_ARG;
    if (xdt != AQ_F16 && xdt != AQ_BF16) return (xdt == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (M <= AQ_DECODE_MAX_M) {
        const int64_t ld = (int64_t)h->NT * 16;
        if ((int64_t)M * h->N <= 8192) {   // small outputs: the streaming kernel's last CTA casts them (one launch; one CTA
                                           // alone takes about 0.1 us per 256 outputs, so larger ones get the cast kernel)
            e = launch_gemv(h, x_dev, xdt, M, h->acc, ld, s, y_dev, ydt);
        } else {
            e = launch_gemv(h, x_dev, xdt, M, h->acc, ld, s);
            if (e == cudaSuccess) e = launch_finalize(h->acc, h->acc, ld, y_dev, ydt, M, h->N, s);
        }
    } else {
        // scratch owned by the handle: float32 sums when the output is half precision, the binary16 copy of bfloat16
        // activations with its row scales and flag; allocated on the first such call and when a later one needs more
        auto up = [](size_t v) { return (v + 255) / 256 * 256; };
        const size_t out_bytes = (ydt == AQ_F32) ? 0 : up((size_t)M * h->N * sizeof(float));
        const size_t x16_bytes = (xdt == AQ_BF16) ? up((size_t)M * h->K * 2) : 0;
        const size_t rs_bytes = (xdt == AQ_BF16) ? up((size_t)M * sizeof(float) + 16) : 0;
        const size_t need = out_bytes + x16_bytes + rs_bytes;
        if (need > h->big_bytes) {
            cudaFree(h->big);   // (waits for whatever still uses the old one)
            h->big = nullptr; h->big_bytes = 0;
            if (cudaMalloc(&h->big, need) != cudaSuccess) { cudaGetLastError(); return AQ_ERR_ALLOC; }
            h->big_bytes = need;
        }
        float* sums = (ydt == AQ_F32) ? (float*)y_dev : reinterpret_cast<float*>(h->big);
        const void* xop = x_dev;
        const float* rs = nullptr;
        const int* flag = nullptr;
        e = cudaSuccess;
        if (xdt == AQ_BF16) {
            void* x16 = h->big + out_bytes;
            float* rsw = reinterpret_cast<float*>(h->big + out_bytes + x16_bytes);
            int* fw = reinterpret_cast<int*>(h->big + out_bytes + x16_bytes + (size_t)M * sizeof(float));
            e = launch_rows_to_f16(x_dev, x16, rsw, fw, M, h->K, s);
            xop = x16; rs = rsw; flag = fw;
        }
        if (e == cudaSuccess) e = launch_gemm(h, xop, rs, flag, M, sums, h->N, nullptr, s);
        if (e == cudaSuccess && ydt != AQ_F32) e = launch_finalize(sums, nullptr, h->N, y_dev, ydt, M, h->N, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    h->last_stream = s;
    return AQ_OK;
}

aq_status_t aq_linear(aq_handle_t h, const void* x_dev, void* y_dev, int M, aq_dtype_t xy_dtype,
                      aq_stream_t stream) {
    return linear_common(h, x_dev, y_dev, M, xy_dtype, xy_dtype, stream);
}

aq_status_t aq_linear_f32out(aq_handle_t h, const void* x_dev, float* y_dev, int M, aq_dtype_t x_dtype,
                             aq_stream_t stream) {
    return linear_common(h, x_dev, y_dev, M, x_dtype, AQ_F32, stream);
}

aq_status_t aq_rbf_gram(const void* A_dev, aq_dtype_t dtype, int64_t K, int64_t d, float sigma, float* G_dev, int64_t ldg,
                        aq_stream_t stream) {
    if (!A_dev || !G_dev || !aligned16(A_dev) || (reinterpret_cast<uintptr_t>(G_dev) & 3u)) return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16) return AQ_ERR_UNSUPPORTED;
    if (K < 2 || K > AQ_HSIC_MAX_K || d < 8 || d % 8 != 0 || d > (1 << 24) || ldg < K) return AQ_ERR_INVALID_ARG;
    if (!(sigma > 0.f) || !std::isfinite(sigma) || !std::isfinite(1.0f / (2.0f * sigma * sigma))) return AQ_ERR_INVALID_ARG;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    const cudaError_t e = launch_rbf_gram(A_dev, dtype, K, d, sigma, G_dev, ldg, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

aq_status_t aq_hsic(const float* KA_dev, const float* KB_dev, int64_t K, int64_t ld, double* out_dev, aq_stream_t stream) {
    if (!KA_dev || !KB_dev || !out_dev || (reinterpret_cast<uintptr_t>(out_dev) & 7u)) return AQ_ERR_INVALID_ARG;
    if (K < 2 || K > AQ_HSIC_MAX_K || ld < K) return AQ_ERR_INVALID_ARG;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    const cudaError_t e = launch_hsic(KA_dev, KB_dev, K, ld, ld, out_dev, 0, 0.0, 0.0, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

aq_status_t aq_sensitivity(const float* KX_dev, const float* KZ_dev, const float* KY_dev, int64_t K, int64_t ld, double alpha,
                           double beta, double* out3_dev, aq_stream_t stream) {
    if (!KX_dev || !KZ_dev || !KY_dev || !out3_dev || (reinterpret_cast<uintptr_t>(out3_dev) & 7u)) return AQ_ERR_INVALID_ARG;
    if (K < 2 || K > AQ_HSIC_MAX_K || ld < K || !(alpha >= 0.0) || !(beta >= 0.0) || !std::isfinite(alpha) || !std::isfinite(beta))
        return AQ_ERR_INVALID_ARG;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    cudaError_t e = launch_hsic(KX_dev, KZ_dev, K, ld, ld, out3_dev, 1, alpha, beta, (cudaStream_t)stream);
    if (e == cudaSuccess) e = launch_hsic(KZ_dev, KY_dev, K, ld, ld, out3_dev, 2, alpha, beta, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

size_t aq_attn_scratch_bytes(int n_kv_heads) {
    if (n_kv_heads < 1 || n_kv_heads > 64) return 0;
    return attn_scratch_bytes(n_kv_heads);
}

aq_status_t aq_rope(void* x_dev, int n_heads, int head_dim, int64_t pos, float theta, aq_dtype_t dtype, aq_stream_t stream) {
    if (!x_dev || (reinterpret_cast<uintptr_t>(x_dev) & 3u) || n_heads < 1 || head_dim < 2 || (head_dim & 1) || pos < 0 ||
        (int64_t)n_heads * head_dim > (1 << 24) || !(theta > 1.f) || !std::isfinite(theta))
        return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16 && dtype != AQ_F32) return AQ_ERR_INVALID_ARG;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    const cudaError_t e = launch_rope(x_dev, n_heads, head_dim, pos, theta, dtype, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

aq_status_t aq_kv_append(void* k_cache_dev, void* v_cache_dev, const void* k_dev, const void* v_dev, int n_kv_heads, int head_dim,
                         int64_t pos, int64_t L_max, aq_dtype_t dtype, aq_stream_t stream) {
    if (!k_cache_dev || !v_cache_dev || !k_dev || !v_dev || !aligned16(k_cache_dev) || !aligned16(v_cache_dev) || !aligned16(k_dev) ||
        !aligned16(v_dev) || n_kv_heads < 1 || n_kv_heads > 64 || pos < 0 || pos >= L_max)
        return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16) return (dtype == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    if (head_dim != 128) return AQ_ERR_UNSUPPORTED;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    const cudaError_t e = launch_kv_append(k_cache_dev, v_cache_dev, k_dev, v_dev, n_kv_heads, head_dim, pos, L_max, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

aq_status_t aq_attn_decode(const void* q_dev, const void* k_cache_dev, const void* v_cache_dev, void* out_dev, int M, int n_heads,
                           int n_kv_heads, int head_dim, int64_t L, int64_t L_max, float scale, aq_dtype_t dtype,
                           aq_dtype_t out_dtype, void* scratch_dev, size_t scratch_bytes, aq_stream_t stream) {
    if (!q_dev || !k_cache_dev || !v_cache_dev || !out_dev || !scratch_dev || !aligned16(q_dev) || !aligned16(k_cache_dev) ||
        !aligned16(v_cache_dev) || !aligned16(out_dev) || (reinterpret_cast<uintptr_t>(scratch_dev) & 255u))
        return AQ_ERR_INVALID_ARG;
    if (M < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0 || L < M || L > L_max || L_max > ((int64_t)1 << 31) ||
        !std::isfinite(scale))
        return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16) return (dtype == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    if (out_dtype != AQ_F16 && out_dtype != AQ_BF16 && out_dtype != AQ_F32) return AQ_ERR_INVALID_ARG;
    if (head_dim != 128 || (int64_t)(n_heads / n_kv_heads) * M > 16 || n_kv_heads > 64) return AQ_ERR_UNSUPPORTED;
    aq_status_t st = check_arch(nullptr);
    if (st != AQ_OK) return st;
    if (scratch_bytes < attn_scratch_bytes(n_kv_heads)) return AQ_ERR_INVALID_ARG;
    if (!(scale > 0.f)) scale = 0.08838834764831845f;   // 1 / sqrt(128)
    const cudaError_t e = launch_attn_decode(q_dev, k_cache_dev, v_cache_dev, out_dev, M, n_heads, n_kv_heads, L, L_max, scale, dtype,
                                             out_dtype, scratch_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

aq_status_t aq_allocate_bits(const double* S, const int64_t* numel, const int32_t* layer_of, int64_t n, const int32_t* types,
                             int n_types, double budget, int32_t* bits_out, double* objective_out) {
    if (!S || !numel || !layer_of || !types || !bits_out || n < 1 || n_types < 1 || !std::isfinite(budget)) return AQ_ERR_INVALID_ARG;
    for (int64_t j = 0; j < n; ++j)
        if (!std::isfinite(S[j])) return AQ_ERR_INVALID_ARG;
    const int r = allocate_bits_host(S, numel, layer_of, n, types, n_types, budget, bits_out, objective_out);
    return r == 0 ? AQ_OK : (r == 2 ? AQ_ERR_RANGE : AQ_ERR_INVALID_ARG);
}

aq_status_t aq_check(aq_stream_t stream) {
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    const int g = read_gemm_status(true), d = read_decode_status(true), t = read_stage1_status(true);
    return (g || d || t) ? AQ_ERR_TIMEOUT : AQ_OK;
}

aq_status_t aq_set_wait_limit_ns(uint64_t ns) {
    set_decode_wait_ns(ns);
    return AQ_OK;
}

void aq_debug_decode_hold(int on) { set_decode_hold(on != 0); }

void aq_free(aq_handle_t h) {
    if (!handle_ok(h)) return;
    cudaStreamSynchronize(h->last_stream);
    decode_stack_forget(h);
    destroy(h);
}

const char* aq_status_string(aq_status_t s) {
    switch (s) {
        case AQ_OK: return "AQ_OK";
        case AQ_ERR_INVALID_ARG: return "AQ_ERR_INVALID_ARG";
        case AQ_ERR_UNSUPPORTED: return "AQ_ERR_UNSUPPORTED";
        case AQ_ERR_ALLOC: return "AQ_ERR_ALLOC";
        case AQ_ERR_CUDA: return "AQ_ERR_CUDA";
        case AQ_ERR_TIMEOUT: return "AQ_ERR_TIMEOUT";
        case AQ_ERR_ARCH: return "AQ_ERR_ARCH";
        case AQ_ERR_RANGE: return "AQ_ERR_RANGE";
    }
    return "AQ_ERR_?";
}

const char* aq_last_cuda_error(void) { return g_last_err; }

uint64_t aq_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
