// Decode path (M = 1..8): fused dequantise + mat-vec, y = x W_hat^T, straight
// from the packed fragments (Appendix D: dequantise on the fly inside the
// low-bit kernel; Eq. 1 for the decode).
//
// Bound: HBM, (bits+1)/8 bytes per weight read once.  Every warp streams its
// own contiguous run of units (16 rows x 256 k) through a private cp.async
// ring in shared memory, so several KB per warp are always in flight and no
// block-wide barrier exists.
//
// The arithmetic of one unit is in aq_gemv_core.cuh.
#include <type_traits>

#include "aq_internal.h"
#include "aq_gemv_core.cuh"
#include "aq_layout.cuh"

namespace aq {

constexpr int GEMV_WARPS = 8;     // warps per CTA
constexpr int GEMV_STAGES = 4;    // ring depth per warp (units)

struct GemvArgs {
    const uint8_t* frags;
    const void* x;      // [M][K] fp16 / bf16
    float* acc;         // [M][ldacc] fp32, accumulated with red.add
    int64_t K;          // true K (x row stride)
    int64_t ldacc;
    int64_t n_units;    // KP * NT
    int64_t N;          // true N: rows >= N are padding and are not written
    int NT;
    int M;
    // when y is given the last CTA to finish casts the sums into y[m][n] and zeroes them again (one launch per linear)
    void* y;
    int ydt;
    unsigned int* ticket;   // zero between launches
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t pol) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int BITS, int MT, bool BF16>
__global__ void __launch_bounds__(GEMV_WARPS * 32, 2) gemv_kernel(const GemvArgs a) {
    constexpr int UB = 2 * frag_bytes(BITS);
    constexpr int PIECES = UB / 16 / 32;   // 16-byte pieces per lane per unit
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* ring = smem + (size_t)warp * GEMV_STAGES * UB;
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);

    const int64_t gw = (int64_t)blockIdx.x * GEMV_WARPS + warp;
    const int64_t nw = (int64_t)gridDim.x * GEMV_WARPS;
    const int64_t u0 = (a.n_units * gw) / nw, u1 = (a.n_units * (gw + 1)) / nw;
    if (u0 < u1) {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));

    auto issue = [&](int64_t u, int slot) {
        const uint8_t* src = a.frags + u * UB;
        const uint32_t dst = ring_s + slot * UB;
#pragma unroll
        for (int p = 0; p < PIECES; ++p) cp_async16(dst + (p * 32 + lane) * 16, src + (p * 32 + lane) * 16, pol);
    };
#pragma unroll
    for (int s = 0; s < GEMV_STAGES - 1; ++s) {
        if (u0 + s < u1) issue(u0 + s, s);
        cp_async_commit();
    }

    XOperand<MT> xo;
    int64_t P = u0 / a.NT;
    int R = (int)(u0 - P * a.NT);
    load_x_operand<MT, BF16>(xo, a.x, a.K, a.M, P, lane);
    int slot = 0;
    for (int64_t u = u0; u < u1; ++u) {
        cp_async_wait<GEMV_STAGES - 2>();
        __syncwarp();
        {   // refill the slot freed by the previous iteration
            const int64_t un = u + GEMV_STAGES - 1;
            int ns = slot + GEMV_STAGES - 1; if (ns >= GEMV_STAGES) ns -= GEMV_STAGES;
            if (un < u1) issue(un, ns);
            cp_async_commit();
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        unit_mac<BITS, MT, BF16>(ring + slot * UB, xo, lane, acc);
        unit_commit<MT>(acc, a.acc, a.ldacc, R * 16, a.N, a.M, lane);
        if (++slot == GEMV_STAGES) slot = 0;
        if (++R == a.NT) {
            R = 0; ++P;
            if (u + 1 < u1) load_x_operand<MT, BF16>(xo, a.x, a.K, a.M, P, lane);
        }
    }
    cp_async_wait<0>();
    }
    if (a.y == nullptr) return;
    // last-CTA epilogue: sums of all CTAs are complete once every CTA has taken a ticket after a fence
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1) ? 1 : 0;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int64_t total = (int64_t)a.M * a.N;
    for (int64_t i0 = threadIdx.x; i0 < total; i0 += 4 * blockDim.x) {   // four loads in flight per thread
        float v[4];
        float* p[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + (int64_t)j * blockDim.x;
            const int64_t m = i / a.N, n = i - m * a.N;
            p[j] = a.acc + m * a.ldacc + n;
            v[j] = (i < total) ? __ldcg(p[j]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + (int64_t)j * blockDim.x;
            if (i >= total) break;
            *p[j] = 0.f;
            if (a.ydt == AQ_F32) reinterpret_cast<float*>(a.y)[i] = v[j];
            else if (a.ydt == AQ_F16) reinterpret_cast<__half*>(a.y)[i] = __float2half_rn(v[j]);
            else reinterpret_cast<__nv_bfloat16*>(a.y)[i] = __float2bfloat16_rn(v[j]);
        }
    }
    if (threadIdx.x == 0) *a.ticket = 0u;
}

template <int BITS, int MT, bool BF16>
static cudaError_t launch_one(const GemvArgs& a, cudaStream_t s) {
    constexpr int UB = 2 * frag_bytes(BITS);
    constexpr int SMEM = GEMV_WARPS * GEMV_STAGES * UB;
    static PerDeviceOnce configured;   // per template instance and device: the attribute belongs to the device's context
    auto kern = gemv_kernel<BITS, MT, BF16>;
    {
        const int rc = configured.run(current_device(), [&] {
            return (int)cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        });
        if (rc != 0) return rc < 0 ? cudaErrorInvalidDevice : (cudaError_t)rc;
    }
    const int64_t warps_wanted = a.n_units;
    int grid = 2 * sm_count();
    const int64_t need = (warps_wanted + GEMV_WARPS - 1) / GEMV_WARPS;
    if (need < grid) grid = (int)need;
    kern<<<grid, GEMV_WARPS * 32, SMEM, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

// Small matrices (a few MB: the launch, not HBM, is what counts): one CTA per 16-row tile, its warps share the tile's
// k-slabs, sum in registers along k and meet in shared memory, and the tile's outputs are cast and written by the CTA
// itself: no global atomics, no ticket, no second pass over the sums.
constexpr int ROWS_STAGES = 2;

template <int BITS, int MT, bool BF16>
__global__ void __launch_bounds__(GEMV_WARPS * 32) gemv_rows_kernel(const GemvArgs a) {
    constexpr int UB = 2 * frag_bytes(BITS);
    constexpr int PIECES = UB / 16 / 32;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ float sums[8 * 16];   // [token][row of the tile]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int R = blockIdx.x;
    const int KP = (int)(a.n_units / a.NT);
    uint8_t* ring = smem + (size_t)warp * ROWS_STAGES * UB;
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    auto issue = [&](int P, int slot) {
        const uint8_t* src = a.frags + ((int64_t)P * a.NT + R) * UB;
        const uint32_t dst = ring_s + slot * UB;
#pragma unroll
        for (int p = 0; p < PIECES; ++p) cp_async16(dst + (p * 32 + lane) * 16, src + (p * 32 + lane) * 16, pol);
    };
#pragma unroll
    for (int i = 0; i < ROWS_STAGES; ++i) {
        if (warp + GEMV_WARPS * i < KP) issue(warp + GEMV_WARPS * i, i);
        cp_async_commit();
    }
    if (threadIdx.x < 8 * 16) sums[threadIdx.x] = 0.f;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int slot = 0;
    for (int P = warp; P < KP; P += GEMV_WARPS) {
        XOperand<MT> xo;
        load_x_operand<MT, BF16>(xo, a.x, a.K, a.M, P, lane);
        cp_async_wait<ROWS_STAGES - 1>();
        __syncwarp();
        unit_mac<BITS, MT, BF16>(ring + slot * UB, xo, lane, acc);
        __syncwarp();   // every lane has read the slot
        if (P + GEMV_WARPS * ROWS_STAGES < KP) issue(P + GEMV_WARPS * ROWS_STAGES, slot);
        cp_async_commit();
        slot ^= 1;
    }
    cp_async_wait<0>();
    __syncthreads();   // sums are zero
    if (warp < KP) unit_commit<MT>(acc, sums, 16, 0, 16, a.M, lane);
    __syncthreads();
    if (threadIdx.x < 16 * a.M) {
        const int m = threadIdx.x >> 4, r = threadIdx.x & 15;
        const int64_t row = (int64_t)R * 16 + r;
        if (row < a.N) {
            const float v = sums[m * 16 + r];
            const int64_t i = (int64_t)m * a.N + row;
            if (a.ydt == AQ_F32) reinterpret_cast<float*>(a.y)[i] = v;
            else if (a.ydt == AQ_F16) reinterpret_cast<__half*>(a.y)[i] = __float2half_rn(v);
            else reinterpret_cast<__nv_bfloat16*>(a.y)[i] = __float2bfloat16_rn(v);
        }
    }
}

template <int BITS, int MT, bool BF16>
static cudaError_t launch_rows(const GemvArgs& a, cudaStream_t s) {
    constexpr int SMEM = GEMV_WARPS * ROWS_STAGES * 2 * frag_bytes(BITS);
    static_assert(SMEM <= 48 * 1024, "fits the default dynamic shared memory limit");
    gemv_rows_kernel<BITS, MT, BF16><<<a.NT, GEMV_WARPS * 32, SMEM, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

// True when the row-tile kernel above is the better choice: outputs written by the kernel, one wave of CTAs, every
// warp with a short run along k.
static bool rows_kernel_fits(const GemvArgs& a) {
    const int64_t KP = a.n_units / a.NT;
    return a.y != nullptr && a.NT <= 4 * sm_count() && KP >= 2 && KP <= 8 * GEMV_WARPS;
}

template <int BITS, bool BF16>
static cudaError_t launch_mt(const GemvArgs& a, cudaStream_t s) {
    if (rows_kernel_fits(a)) {
        if (a.M == 1) return launch_rows<BITS, 1, BF16>(a, s);
        if (a.M == 2) return launch_rows<BITS, 2, BF16>(a, s);
        if (a.M <= 4) return launch_rows<BITS, 4, BF16>(a, s);
        return launch_rows<BITS, 8, BF16>(a, s);
    }
    if (a.M == 1) return launch_one<BITS, 1, BF16>(a, s);
    if (a.M == 2) return launch_one<BITS, 2, BF16>(a, s);
    if (a.M <= 4) return launch_one<BITS, 4, BF16>(a, s);
    return launch_one<BITS, 8, BF16>(a, s);
}

cudaError_t launch_gemv(const aq_handle_s* h, const void* x, aq_dtype_t xdt, int M, float* acc, int64_t ldacc,
                        cudaStream_t s, void* y_fused, aq_dtype_t ydt) {
    GemvArgs a;
    a.y = y_fused; a.ydt = (int)ydt; a.ticket = reinterpret_cast<unsigned int*>(h->flags) + 16;
    a.frags = h->frags; a.x = x; a.acc = acc; a.K = h->K; a.ldacc = ldacc;
    a.n_units = (int64_t)h->KP * h->NT; a.NT = h->NT; a.M = M; a.N = h->N;
    const bool bf = (xdt == AQ_BF16);
    switch (h->bits) {
        case 2: return bf ? launch_mt<2, true>(a, s) : launch_mt<2, false>(a, s);
        case 3: return bf ? launch_mt<3, true>(a, s) : launch_mt<3, false>(a, s);
        default: return bf ? launch_mt<4, true>(a, s) : launch_mt<4, false>(a, s);
    }
}

// y = cast(acc) for the first N columns of each row, then acc = 0.
template <typename T>
__global__ void finalize_kernel(const float* __restrict__ acc_in, float* __restrict__ acc_zero, int64_t ld,
                                T* __restrict__ y, int M, int64_t N) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)M * N) return;
    const int64_t m = i / N, n = i - m * N;
    const float v = acc_in[m * ld + n];
    if constexpr (sizeof(T) == 4) y[i] = v;
    else if constexpr (std::is_same<T, __half>::value) y[i] = __float2half_rn(v);
    else y[i] = __float2bfloat16_rn(v);
    if (acc_zero) acc_zero[m * ld + n] = 0.f;
}

cudaError_t launch_finalize(const float* acc_in, float* acc_zero, int64_t ldacc, void* y, aq_dtype_t ydt, int M,
                            int64_t N, cudaStream_t s) {
    const int64_t n = (int64_t)M * N;
    const unsigned grid = (unsigned)((n + 255) / 256);
    if (ydt == AQ_F16) finalize_kernel<__half><<<grid, 256, 0, s>>>(acc_in, acc_zero, ldacc, (__half*)y, M, N);
    else if (ydt == AQ_BF16) finalize_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(acc_in, acc_zero, ldacc, (__nv_bfloat16*)y, M, N);
    else finalize_kernel<float><<<grid, 256, 0, s>>>(acc_in, acc_zero, ldacc, (float*)y, M, N);
    count_launch();
    return cudaGetLastError();
}

}  // namespace aq
