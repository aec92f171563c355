// Inter-tensor stage (Section 4.1): RBF kernel matrices of calibration activations on the
// tensor cores, the empirical HSIC of Eq. 2, the sensitivity of Eq. 5, and (host) the greedy
// layer-balanced bit allocation of Eq. 6.
//
// Kernel matrix: |a_i - a_j|^2 = n_i + n_j - 2 <a_i, a_j>.  The inner products are a dense
// K x K x d contraction of half-precision samples (products exact in binary32, binary32
// accumulation in TMEM): tcgen05.mma, both operands tiles of the same matrix brought in by TMA.
// The epilogue turns each accumulator into exp(-D / (2 sigma^2)) and writes the tile and its mirror
// image (only tiles on or above the diagonal are computed).
//
// HSIC: tr(K_A C K_B C) = sum_ij A_ij B_ij - (2/K) sum_i rA_i rB_i + sA sB / K^2 with row sums r and
// totals s, one pass over both matrices, everything in binary64 in a fixed order.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cmath>
#include <cstring>
#include <vector>

#include "aq_internal.h"
#include "aq_tc.cuh"

namespace aq {

constexpr int S1_TILE = 128;       // samples per tile side (UMMA M and N)
constexpr int S1_KSTAGE = 64;      // features per stage (one 128-byte swizzle atom of 16-bit elements)
constexpr int S1_STAGES = 3;       // 3 x (16 + 16) KB: two CTAs fit one SM, so one's epilogue overlaps the other's main loop
constexpr int S1_OP_BYTES = S1_TILE * S1_KSTAGE * 2;
constexpr int S1_THREADS = 192;    // warp 0: TMA, warp 1: MMA, warps 2..5: epilogue
constexpr uint32_t S1_SPIN_LIMIT = 20u * 1000u * 1000u;

__device__ int g_stage1_status = 0;   // nonzero: a bounded wait ran out (code = which)

// scratch of the HSIC reduction: row sums of both matrices and the per-row dot products
__device__ double g_hsic_rows[3][AQ_HSIC_MAX_K];
__device__ float g_sq_norms[AQ_HSIC_MAX_K];

struct GramArgs {
    const float* norms;   // [K] squared norms
    float* out;           // [K][ld]
    int64_t ld;
    int K, d, n_t;
    float c;              // 1 / (2 sigma^2)
};

__device__ __forceinline__ bool s1_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code) {
    for (uint32_t i = 0; i < S1_SPIN_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 2000) {
            __nanosleep(40);
            if (*abort_flag) return false;
        }
    }
    *abort_flag = 1;
    atomicCAS(&g_stage1_status, 0, code);
    return false;
}

// n_i = sum_k a_ik^2: one warp per sample, 8 elements per lane per step, binary32.
template <bool BF16>
__global__ void __launch_bounds__(256) sqnorm_kernel(const void* __restrict__ A, int K, int d, float* __restrict__ norms) {
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= K) return;
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(A) + (int64_t)row * d);
    float s = 0.f;
    for (int v = lane; v < d / 8; v += 32) {
        const uint4 u = __ldg(p + v);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f;
            if constexpr (BF16) f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
            else f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            s = fmaf(f.x, f.x, s);
            s = fmaf(f.y, f.y, s);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) norms[row] = s;
}

template <bool BF16>
__global__ void __launch_bounds__(S1_THREADS, 2) gram_rbf_kernel(const __grid_constant__ CUtensorMap tmap, const GramArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + S1_STAGES * S1_OP_BYTES;
    float* s_nj = reinterpret_cast<float*>(sB + S1_STAGES * S1_OP_BYTES);   // [128] column norms
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_nj + S1_TILE);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * S1_STAGES, bar_accum = bar_empty + 8 * S1_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S1_STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // tile (ti <= tj) of the upper triangle
    int ti = 0, t = (int)blockIdx.x;
    while (t >= a.n_t - ti) { t -= a.n_t - ti; ++ti; }
    const int tj = ti + t;
    const bool diag = (ti == tj);
    const int n_k = (a.d + S1_KSTAGE - 1) / S1_KSTAGE;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S1_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)S1_TILE) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < n_k && ok; ++kb) {
                const uint32_t s = kb % S1_STAGES;
                ok = s1_wait(bar_empty + 8 * s, ((kb / S1_STAGES) & 1) ^ 1, abort_flag, 1);
                if (!ok) break;
                mbar_expect_tx(bar_full + 8 * s, (uint32_t)(diag ? S1_OP_BYTES : 2 * S1_OP_BYTES));
                tma_load_2d(smem_u32(sA + s * S1_OP_BYTES), &tmap, kb * S1_KSTAGE, ti * S1_TILE, bar_full + 8 * s);
                if (!diag) tma_load_2d(smem_u32(sB + s * S1_OP_BYTES), &tmap, kb * S1_KSTAGE, tj * S1_TILE, bar_full + 8 * s);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) |
                                   ((uint32_t)(S1_TILE >> 3) << 17) | ((uint32_t)(S1_TILE >> 4) << 24);
            bool ok = true;
            for (int kb = 0; kb < n_k && ok; ++kb) {
                const uint32_t s = kb % S1_STAGES;
                ok = s1_wait(bar_full + 8 * s, (kb / S1_STAGES) & 1, abort_flag, 2);
                if (!ok) break;
                tc_fence_after();
                const uint64_t ad = make_smem_desc(smem_u32(sA + s * S1_OP_BYTES));
                const uint64_t bd = diag ? ad : make_smem_desc(smem_u32(sB + s * S1_OP_BYTES));
#pragma unroll
                for (int k = 0; k < S1_KSTAGE / 16; ++k)
                    umma_f16(tmem_base, ad + 2 * k, bd + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(bar_empty + 8 * s);
            }
            if (ok) umma_commit(bar_accum);
        }
    } else {
        // epilogue: TMEM lane quarter (warp % 4), lane = row of the tile
        const int lq = warp & 3;
        const int e = threadIdx.x - 64;   // 0..127
        {
            const int jg = tj * S1_TILE + e;
            s_nj[e] = (jg < a.K) ? __ldg(a.norms + jg) : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int i = ti * S1_TILE + lq * 32 + lane;
        const float ni = (i < a.K) ? __ldg(a.norms + i) : 0.f;
        const bool ok = s1_wait(bar_accum, 0, abort_flag, 3);
        if (ok) {
            tc_fence_after();
            const bool vec = (a.ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.out) & 15u) == 0);
            for (int c0 = 0; c0 < S1_TILE; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait();
                const int j0 = tj * S1_TILE + c0;
                float kv[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float dist = fmaxf(ni + s_nj[c0 + j] - 2.f * __uint_as_float(v[j]), 0.f);
                    kv[j] = (i == j0 + j) ? 1.f : expf(-dist * a.c);
                }
                if (i < a.K) {
                    float* row = a.out + (int64_t)i * a.ld + j0;
                    if (vec && j0 + 32 <= a.K) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(row + j) = make_float4(kv[j], kv[j + 1], kv[j + 2], kv[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j0 + j < a.K) row[j] = kv[j];
                    }
                }
                if (!diag && i < a.K) {   // mirror image: lanes are consecutive columns of row j
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j0 + j < a.K) a.out[(int64_t)(j0 + j) * a.ld + i] = kv[j];
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);   // let copies in flight land before the CTA's shared memory goes away
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)S1_TILE) : "memory");
    }
}


// The same computation on CTA pairs: a 256 x 256 tile per pair, tcgen05 cta_group::2.  Each CTA brings in its own 128 rows
// of both operands (half the shared-memory traffic per flop of the kernel above) and keeps its 128 x 256 part of the
// accumulator; the even CTA issues the MMAs and its barriers collect both CTAs' loads.
template <bool BF16>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(S1_THREADS, 2)
gram_rbf_pair_kernel(const __grid_constant__ CUtensorMap tmap, const GramArgs a) {
    constexpr int TW = 2 * S1_TILE;   // tile side
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + S1_STAGES * S1_OP_BYTES;
    float* s_nj = reinterpret_cast<float*>(sB + S1_STAGES * S1_OP_BYTES);   // [256] column norms
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_nj + TW);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * S1_STAGES, bar_accum = bar_empty + 8 * S1_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S1_STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();

    int ti = 0, t = (int)(blockIdx.x >> 1);
    while (t >= a.n_t - ti) { t -= a.n_t - ti; ++ti; }
    const int tj = ti + t;
    const bool diag = (ti == tj);
    const int n_k = (a.d + S1_KSTAGE - 1) / S1_KSTAGE;
    const int rowA0 = ti * TW + (int)rank * S1_TILE, rowB0 = tj * TW + (int)rank * S1_TILE;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S1_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates, with the same destination
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)TW) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the partner's barriers exist before anything is counted on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t per_cta = (uint32_t)(diag ? S1_OP_BYTES : 2 * S1_OP_BYTES);
            bool ok = true;
            for (int kb = 0; kb < n_k && ok; ++kb) {
                const uint32_t s = kb % S1_STAGES;
                ok = s1_wait(bar_empty + 8 * s, ((kb / S1_STAGES) & 1) ^ 1, abort_flag, 4);
                if (!ok) break;
                const uint32_t full0 = cluster_map(bar_full + 8 * s, 0);
                if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * per_cta);
                tma_load_2d_pair(smem_u32(sA + s * S1_OP_BYTES), &tmap, kb * S1_KSTAGE, rowA0, full0);
                if (!diag) tma_load_2d_pair(smem_u32(sB + s * S1_OP_BYTES), &tmap, kb * S1_KSTAGE, rowB0, full0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) |
                                   ((uint32_t)(TW >> 3) << 17) | ((uint32_t)(TW >> 4) << 24);
            bool ok = true;
            for (int kb = 0; kb < n_k && ok; ++kb) {
                const uint32_t s = kb % S1_STAGES;
                ok = s1_wait(bar_full + 8 * s, (kb / S1_STAGES) & 1, abort_flag, 5);
                if (!ok) break;
                tc_fence_after();
                const uint64_t ad = make_smem_desc(smem_u32(sA + s * S1_OP_BYTES));
                const uint64_t bd = diag ? ad : make_smem_desc(smem_u32(sB + s * S1_OP_BYTES));
#pragma unroll
                for (int k = 0; k < S1_KSTAGE / 16; ++k)
                    umma_f16_pair(tmem_base, ad + 2 * k, bd + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit_pair(bar_empty + 8 * s);                    // both CTAs' stage s may be refilled
                umma_commit_pair(cluster_map(bar_empty + 8 * s, 1));
            }
            if (ok) {
                umma_commit_pair(bar_accum);
                umma_commit_pair(cluster_map(bar_accum, 1));
            }
        }
    } else {
        const int lq = warp & 3;
        const int e = threadIdx.x - 64;   // 0..127
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int jg = tj * TW + e + h * S1_TILE;
            s_nj[e + h * S1_TILE] = (jg < a.K) ? __ldg(a.norms + jg) : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int i = rowA0 + lq * 32 + lane;
        const float ni = (i < a.K) ? __ldg(a.norms + i) : 0.f;
        const bool ok = s1_wait(bar_accum, 0, abort_flag, 6);
        if (ok) {
            tc_fence_after();
            const bool vec = (a.ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.out) & 15u) == 0);
            for (int c0 = 0; c0 < TW; c0 += 32) {
                const int j0 = tj * TW + c0;
                if (j0 >= a.K) break;                         // (the same for the whole warp)
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait();
                float kv[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float dist = fmaxf(ni + s_nj[c0 + j] - 2.f * __uint_as_float(v[j]), 0.f);
                    kv[j] = (i == j0 + j) ? 1.f : expf(-dist * a.c);
                }
                if (i < a.K) {
                    float* row = a.out + (int64_t)i * a.ld + j0;
                    if (vec && j0 + 32 <= a.K) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(row + j) = make_float4(kv[j], kv[j + 1], kv[j + 2], kv[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j0 + j < a.K) row[j] = kv[j];
                    }
                    if (!diag) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j0 + j < a.K) a.out[(int64_t)(j0 + j) * a.ld + i] = kv[j];
                    }
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);
    cluster_sync_all();   // nothing of the partner (its operand tiles, its barriers) is in use any more
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TW) : "memory");
    }
}

cudaError_t launch_rbf_gram(const void* A, aq_dtype_t dt, int64_t K, int64_t d, float sigma, float* out, int64_t ld,
                            cudaStream_t s) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return cudaErrorNotSupported;
    float* norms = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&norms), g_sq_norms);
    if (e != cudaSuccess) return e;
    const bool bf = (dt == AQ_BF16);
    if (bf) sqnorm_kernel<true><<<(unsigned)((K + 7) / 8), 256, 0, s>>>(A, (int)K, (int)d, norms);
    else sqnorm_kernel<false><<<(unsigned)((K + 7) / 8), 256, 0, s>>>(A, (int)K, (int)d, norms);
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    CUtensorMap tm;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)K};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {(cuuint32_t)S1_KSTAGE, (cuuint32_t)S1_TILE};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tm, bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(A), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    GramArgs a;
    a.norms = norms; a.out = out; a.ld = ld; a.K = (int)K; a.d = (int)d;
    a.c = 1.0f / (2.0f * sigma * sigma);
    // CTA pairs on 256-wide tiles, or single CTAs on 128-wide tiles: whichever leaves the busiest SM less to do
    // (work in 128 x 128 tiles; the pair kernel gets about 1.25 times as much out of the tensor pipe)
    const int64_t n_t1 = (K + S1_TILE - 1) / S1_TILE, n_t2 = (K + 2 * S1_TILE - 1) / (2 * S1_TILE);
    const int64_t sms = sm_count();
    const int64_t per_sm_pairs = 2 * ((n_t2 * (n_t2 + 1) + sms - 1) / sms);       // n_t2 (n_t2 + 1) CTAs of two tiles each
    const int64_t per_sm_single = (n_t1 * (n_t1 + 1) / 2 + sms - 1) / sms;
    const bool pairs = 4 * per_sm_pairs < 5 * per_sm_single;
    a.n_t = pairs ? (int)n_t2 : (int)n_t1;
    constexpr int SMEM = 1024 + 2 * S1_STAGES * S1_OP_BYTES + 2 * S1_TILE * 4 + 128;
    const unsigned grid = (unsigned)((int64_t)a.n_t * (a.n_t + 1) / 2) * (pairs ? 2u : 1u);
    auto launch = [&](auto kern) -> cudaError_t {
        cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e2 != cudaSuccess) return e2;
        kern<<<grid, S1_THREADS, SMEM, s>>>(tm, a);
        return cudaGetLastError();
    };
    if (pairs) e = bf ? launch(gram_rbf_pair_kernel<true>) : launch(gram_rbf_pair_kernel<false>);
    else e = bf ? launch(gram_rbf_kernel<true>) : launch(gram_rbf_kernel<false>);
    count_launch();
    return e;
}

// ---- HSIC (Eq. 2) -------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Per row i: rA_i = sum_j A_ij, rB_i = sum_j B_ij, p_i = sum_j A_ij B_ij (one warp per row).
__global__ void __launch_bounds__(256) hsic_rows_kernel(const float* __restrict__ KA, const float* __restrict__ KB, int K, int64_t lda,
                                                        int64_t ldb) {
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= K) return;
    const float* pa = KA + (int64_t)row * lda;
    const float* pb = KB + (int64_t)row * ldb;
    double ra = 0.0, rb = 0.0, p = 0.0;
    int j0 = 0;
    if (((lda | ldb) & 3) == 0 && ((reinterpret_cast<uintptr_t>(KA) | reinterpret_cast<uintptr_t>(KB)) & 15u) == 0) {
        // four columns per lane and step, two steps in flight
        const int K4 = K & ~255;
        for (int j = 4 * lane; j < K4; j += 256) {
            const float4 x0 = __ldg(reinterpret_cast<const float4*>(pa + j)), y0 = __ldg(reinterpret_cast<const float4*>(pb + j));
            const float4 x1 = __ldg(reinterpret_cast<const float4*>(pa + j + 128)), y1 = __ldg(reinterpret_cast<const float4*>(pb + j + 128));
            const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
            const float ys[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const double x = (double)xs[q], y = (double)ys[q];
                ra += x; rb += y; p = fma(x, y, p);
            }
        }
        j0 = K4;
    }
    for (int j = j0 + lane; j < K; j += 32) {
        const double x = (double)__ldg(pa + j), y = (double)__ldg(pb + j);
        ra += x; rb += y; p = fma(x, y, p);
    }
    ra = warp_sum(ra); rb = warp_sum(rb); p = warp_sum(p);
    if (lane == 0) { g_hsic_rows[0][row] = ra; g_hsic_rows[1][row] = rb; g_hsic_rows[2][row] = p; }
}

// One CTA: the four totals in a fixed order, then Eq. 2.  With `combine`, out[0] = -alpha out[1] + beta out[2] (Eq. 5).
__global__ void __launch_bounds__(256) hsic_final_kernel(int K, double* out, int combine, double alpha, double beta) {
    __shared__ double sh[4][256];
    double sa = 0.0, sb = 0.0, sp = 0.0, sx = 0.0;
    for (int i = threadIdx.x; i < K; i += 256) {
        const double ra = g_hsic_rows[0][i], rb = g_hsic_rows[1][i];
        sa += ra; sb += rb; sp += g_hsic_rows[2][i]; sx = fma(ra, rb, sx);
    }
    sh[0][threadIdx.x] = sa; sh[1][threadIdx.x] = sb; sh[2][threadIdx.x] = sp; sh[3][threadIdx.x] = sx;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o)
            for (int q = 0; q < 4; ++q) sh[q][threadIdx.x] += sh[q][threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double k = (double)K;
        const double tr = sh[2][0] - 2.0 * sh[3][0] / k + sh[0][0] * sh[1][0] / (k * k);
        const double h = tr / ((k - 1.0) * (k - 1.0));
        if (combine == 0) out[0] = h;
        else {
            out[combine] = h;
            if (combine == 2) out[0] = -alpha * out[1] + beta * h;
        }
    }
}

cudaError_t launch_hsic(const float* KA, const float* KB, int64_t K, int64_t lda, int64_t ldb, double* out, int combine,
                        double alpha, double beta, cudaStream_t s) {
    hsic_rows_kernel<<<(unsigned)((K + 7) / 8), 256, 0, s>>>(KA, KB, (int)K, lda, ldb);
    hsic_final_kernel<<<1, 256, 0, s>>>((int)K, out, combine, alpha, beta);
    count_launch(2);
    return cudaGetLastError();
}

int read_stage1_status(bool clear) {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_stage1_status, sizeof(int));
    if (clear && v) { int z = 0; cudaMemcpyToSymbol(g_stage1_status, &z, sizeof(int)); }
    return v;
}

// ---- bit allocation (Eq. 6; host) -----------------------------------------------------------------
// Greedy: all matrices at types[0]; each step applies, among the single-type upgrades that keep the budget, the one
// with the largest (E_l^2 - E~_l^2) / extra bits; stops when none is left or the best one does not lower the objective.
// Ties go to the lowest index.  Plain binary64, one operation per step of the formulas.
int allocate_bits_host(const double* S, const int64_t* numel, const int32_t* layer_of, int64_t n, const int32_t* types,
                       int n_types, double budget, int32_t* bits_out, double* objective_out) {
    int64_t total = 0;
    int32_t L = 0;
    for (int64_t j = 0; j < n; ++j) {
        if (numel[j] <= 0 || layer_of[j] < 0) return 1;
        total += numel[j];
        if (layer_of[j] + 1 > L) L = layer_of[j] + 1;
    }
    for (int t = 0; t < n_types; ++t)
        if (types[t] < 1 || types[t] > 16 || (t > 0 && types[t] <= types[t - 1])) return 1;
    std::vector<double> eta(n_types), E(L, 0.0);
    for (int t = 0; t < n_types; ++t) eta[t] = std::ldexp(1.0, -2 * types[t]);
    std::vector<int> level(n, 0);
    const double cap = budget * (double)total;
    int64_t used = (int64_t)types[0] * total;
    if ((double)used > cap) return 2;
    for (int64_t j = 0; j < n; ++j) E[layer_of[j]] += S[j] * eta[0];
    for (;;) {
        int64_t best = -1;
        double best_ratio = 0.0, best_E = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            if (level[j] + 1 >= n_types) continue;
            const int64_t extra = (int64_t)(types[level[j] + 1] - types[level[j]]) * numel[j];
            if ((double)(used + extra) > cap) continue;
            const int32_t l = layer_of[j];
            const double E_new = E[l] + S[j] * (eta[level[j] + 1] - eta[level[j]]);
            const double ratio = (E[l] * E[l] - E_new * E_new) / (double)extra;
            if (best < 0 || ratio > best_ratio) { best = j; best_ratio = ratio; best_E = E_new; }
        }
        if (best < 0 || !(best_ratio > 0.0)) break;
        used += (int64_t)(types[level[best] + 1] - types[level[best]]) * numel[best];
        E[layer_of[best]] = best_E;
        ++level[best];
    }
    for (int64_t j = 0; j < n; ++j) bits_out[j] = types[level[j]];
    if (objective_out) {
        std::vector<double> F(L, 0.0);
        for (int64_t j = 0; j < n; ++j) F[layer_of[j]] += S[j] * eta[level[j]];
        double o = 0.0;
        for (int32_t l = 0; l < L; ++l) o += F[l] * F[l];
        *objective_out = o;
    }
    return 0;
}

}  // namespace aq
