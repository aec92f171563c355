// Decode path (M = 1..8): fused dequantise + mat-vec, y = x W_hat^T, straight
// from the packed fragments (Appendix D: dequantise on the fly inside the
// low-bit kernel; Eq. 1 for the decode).
//
// Bound: HBM, (bits+1)/8 bytes per weight read once.  Every warp streams its
// own contiguous run of units (16 rows x 256 k) through a private cp.async
// ring in shared memory, so several KB per warp are always in flight and no
// block-wide barrier exists.
//
// Arithmetic: with w = d q + m per block,
//     sum_k x w = d * sum (BIAS + q) x  +  (m - BIAS d) * sum x
// The first sum runs on the tensor cores (mma.sync m16n8k16, fp32
// accumulate): the A operand is built two codes per LOP3 by OR-ing the code
// bits into the mantissa of the half-precision constant BIAS (1024 for fp16,
// 128 for bf16), the B operand holds x.  The 8 columns of the instruction are
// (block, token) pairs: with MT tokens per call, 8/MT blocks accumulate side
// by side and the per-block scale is applied to the 4 accumulators only once
// per group of 8/MT blocks.
#include <type_traits>

#include "aq_internal.h"
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
};

template <bool BF16>
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if constexpr (BF16) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    } else {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
}

template <bool BF16>
__device__ __forceinline__ float sum8(const uint4& v) {
    float s = 0.f;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f;
        if constexpr (BF16) f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
        else f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        s += f.x + f.y;
    }
    return s;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t pol) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Per-warp state for the x operand of one pair-slab (256 k).
template <int MT>
struct XOperand {
    static constexpr int BG = 8 / MT;   // blocks that accumulate side by side
    static constexpr int NG = MT / 2;   // groups per fragment (4 blocks)
    uint32_t b[2][4][4];                // [fragment][block][reg]: masked B registers
    float X0[2][NG], X1[2][NG];         // block sums of x for this lane's two accumulator columns
};

template <int MT, bool BF16>
__device__ __forceinline__ void load_x_operand(XOperand<MT>& xo, const void* xv, int64_t K, int M, int64_t P, int lane) {
    constexpr int BG = XOperand<MT>::BG, NG = XOperand<MT>::NG;
    const int g = lane >> 2, t = lane & 3;
    const int tok = g % MT, bs = g / MT;
    const uint16_t* x = reinterpret_cast<const uint16_t*>(xv);
#pragma unroll
    for (int fi = 0; fi < 2; ++fi) {
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
            const int jb = gi * BG + bs;
            const int64_t k = (2 * P + fi) * 128 + 32 * jb + 8 * t;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (tok < M && k < K) v = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)tok * K + k));
            float s = sum8<BF16>(v);
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            // the lane's accumulator columns 2t, 2t+1 are B columns of lanes g' = 2t, 2t+1
            xo.X0[fi][gi] = __shfl_sync(0xffffffffu, s, (2 * t) * 4);
            xo.X1[fi][gi] = __shfl_sync(0xffffffffu, s, (2 * t + 1) * 4);
#pragma unroll
            for (int b2 = 0; b2 < BG; ++b2) {
                const bool on = (b2 == bs);
                xo.b[fi][gi * BG + b2][0] = on ? v.x : 0u;
                xo.b[fi][gi * BG + b2][1] = on ? v.y : 0u;
                xo.b[fi][gi * BG + b2][2] = on ? v.z : 0u;
                xo.b[fi][gi * BG + b2][3] = on ? v.w : 0u;
            }
        }
    }
}

// One unit (two fragments) against the prepared x operand; returns this lane's
// four partial sums: [row g, col 2t], [row g, col 2t+1], [row g+8, col 2t], [row g+8, col 2t+1].
template <int BITS, int MT, bool BF16>
__device__ __forceinline__ void unit_mac(const uint8_t* unit, const XOperand<MT>& xo, int lane, float (&acc)[4]) {
    constexpr int FB = frag_bytes(BITS);
    constexpr int BG = XOperand<MT>::BG, NG = XOperand<MT>::NG;
    constexpr uint32_t MAGIC = BF16 ? 0x43004300u : 0x64006400u;
    constexpr float BIAS = BF16 ? 128.f : 1024.f;
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int fi = 0; fi < 2; ++fi) {
        const uint8_t* fb = unit + fi * FB;
        LaneCodes<BITS> lc;
        load_lane_codes<BITS>(lc, fb, lane);
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int b2 = 0; b2 < BG; ++b2) {
                const int j = gi * BG + b2;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t a[4];
                    a[0] = code_pair<BITS>(lc, j, 0, 2 * h, MAGIC);
                    a[1] = code_pair<BITS>(lc, j, 1, 2 * h, MAGIC);
                    a[2] = code_pair<BITS>(lc, j, 0, 2 * h + 1, MAGIC);
                    a[3] = code_pair<BITS>(lc, j, 1, 2 * h + 1, MAGIC);
                    mma16816<BF16>(c, a, xo.b[fi][j][2 * h], xo.b[fi][j][2 * h + 1]);
                }
            }
            const int jbm = gi * BG + (2 * t) / MT;
            const __half2 dm0 = *reinterpret_cast<const __half2*>(fb + (g * 4 + jbm) * 4);
            const __half2 dm1 = *reinterpret_cast<const __half2*>(fb + ((g + 8) * 4 + jbm) * 4);
            const float d0 = __low2float(dm0), d1 = __low2float(dm1);
            const float mp0 = fmaf(-BIAS, d0, __high2float(dm0)), mp1 = fmaf(-BIAS, d1, __high2float(dm1));
            const float X0 = xo.X0[fi][gi], X1 = xo.X1[fi][gi];
            acc[0] = fmaf(d0, c[0], fmaf(mp0, X0, acc[0]));
            acc[1] = fmaf(d0, c[1], fmaf(mp0, X1, acc[1]));
            acc[2] = fmaf(d1, c[2], fmaf(mp1, X0, acc[2]));
            acc[3] = fmaf(d1, c[3], fmaf(mp1, X1, acc[3]));
        }
    }
}

// Cross-lane reduction and accumulation into out[tok][row] (fp32, red.add).
template <int MT>
__device__ __forceinline__ void unit_commit(float (&acc)[4], float* out, int64_t ld, int row0, int64_t N, int M, int lane) {
    const int g = lane >> 2, t = lane & 3;
    if constexpr (MT == 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 1);
            acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 2);
        }
        // lane t commits one of the four sums: (tok, row half) = (t & 1, t >> 1)
        const float v = (t == 0) ? acc[0] : (t == 1) ? acc[1] : (t == 2) ? acc[2] : acc[3];
        const int tok = t & 1;
        const int row = row0 + g + 8 * (t >> 1);
        if (tok < M && row < N) atomicAdd(out + (int64_t)tok * ld + row, v);
    } else if constexpr (MT == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 2);
        // lanes t = 0,1 hold tokens (2t, 2t+1); lanes 2,3 the same sums: split the four stores
        const int tk = 2 * (t & 1);
        const int hi = t >> 1;   // lanes 0,1 commit row g, lanes 2,3 row g+8
        const float v0 = hi ? acc[2] : acc[0], v1 = hi ? acc[3] : acc[1];
        const int row = row0 + g + 8 * hi;
        if (tk < M && row < N) atomicAdd(out + (int64_t)tk * ld + row, v0);
        if (tk + 1 < M && row < N) atomicAdd(out + (int64_t)(tk + 1) * ld + row, v1);
    } else {
        const int tk = 2 * t;
        const int r0 = row0 + g, r1 = row0 + g + 8;
        if (tk < M) {
            if (r0 < N) atomicAdd(out + (int64_t)tk * ld + r0, acc[0]);
            if (r1 < N) atomicAdd(out + (int64_t)tk * ld + r1, acc[2]);
        }
        if (tk + 1 < M) {
            if (r0 < N) atomicAdd(out + (int64_t)(tk + 1) * ld + r0, acc[1]);
            if (r1 < N) atomicAdd(out + (int64_t)(tk + 1) * ld + r1, acc[3]);
        }
    }
}

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
    if (u0 >= u1) return;

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
    int64_t curP = -1;
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
        const int64_t P = u / a.NT;
        const int R = (int)(u - P * a.NT);
        if (P != curP) { load_x_operand<MT, BF16>(xo, a.x, a.K, a.M, P, lane); curP = P; }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        unit_mac<BITS, MT, BF16>(ring + slot * UB, xo, lane, acc);
        unit_commit<MT>(acc, a.acc, a.ldacc, R * 16, a.N, a.M, lane);
        if (++slot == GEMV_STAGES) slot = 0;
    }
    cp_async_wait<0>();
}

template <int BITS, int MT, bool BF16>
static cudaError_t launch_one(const GemvArgs& a, cudaStream_t s) {
    constexpr int UB = 2 * frag_bytes(BITS);
    constexpr int SMEM = GEMV_WARPS * GEMV_STAGES * UB;
    static bool configured = false;   // per (template instance); attribute is per device context
    auto kern = gemv_kernel<BITS, MT, BF16>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int64_t warps_wanted = a.n_units;
    int grid = 2 * sm_count();
    const int64_t need = (warps_wanted + GEMV_WARPS - 1) / GEMV_WARPS;
    if (need < grid) grid = (int)need;
    kern<<<grid, GEMV_WARPS * 32, SMEM, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

template <int BITS, bool BF16>
static cudaError_t launch_mt(const GemvArgs& a, cudaStream_t s) {
    if (a.M <= 2) return launch_one<BITS, 2, BF16>(a, s);
    if (a.M <= 4) return launch_one<BITS, 4, BF16>(a, s);
    return launch_one<BITS, 8, BF16>(a, s);
}

cudaError_t launch_gemv(const aq_handle_s* h, const void* x, aq_dtype_t xdt, int M, float* acc, int64_t ldacc,
                        cudaStream_t s) {
    GemvArgs a;
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
