// Prefill path (M > 8): dequantise-to-half + tensor-core GEMM on the packed
// weights, out[m][n] (+)= sum_k x[m][k] w_hat[n][k]  (Appendix D: dequantise
// on the fly inside the low-bit kernel; Eq. 1 for the decode).
//
// Bound: tensor cores (dense contraction, 2 M flops per weight).  tcgen05
// UMMA with the accumulator in TMEM:
//   A (M side, 128)  = weight rows, dequantised by four warps from the packed
//                      fragments into the K-major 128-byte-swizzled shared
//                      memory layout the instruction reads,
//   B (N side, <=256) = tokens, fetched by TMA with the same swizzle,
//   D[128 lanes][tokens] fp32 in TMEM, read back with tcgen05.ld.
// Warp roles: 0 = TMA / bulk-copy producer (+ TMEM allocation), 1..4 =
// dequantise then epilogue, 5 = MMA issue.  Every mbarrier wait is bounded;
// when one runs out the CTA raises a status word, drains and returns.
#include <cuda.h>

#include "aq_internal.h"
#include "aq_layout.cuh"

namespace aq {

constexpr int GM_ROWS = 128;       // weight rows per CTA tile (UMMA M)
constexpr int GM_KSTAGE = 64;      // k per pipeline stage (one 128-byte swizzle atom of 16-bit elements)
constexpr int GM_STAGES = 4;       // A/B ring depth
constexpr int GM_PSTAGES = 2;      // packed-fragment ring depth (one k-slab of 128 per slot)
constexpr int GM_THREADS = 192;
constexpr int GM_MAX_TN = 256;     // tokens per CTA tile (UMMA N)
constexpr uint32_t GM_SPIN_LIMIT = 40u * 1000u * 1000u;

__device__ int g_gemm_status = 0;  // nonzero: a bounded wait ran out (code = which)

struct GemmArgs {
    const uint8_t* frags;
    float* out;
    int64_t ldo;
    int64_t N;
    int M;
    int NT;          // 16-row tiles
    int n_slabs;     // k-slabs of 128 (2 * KP)
    int splits;
    int tn;          // token tile = TMA box rows = UMMA N
    int use_red;     // accumulate with red.add instead of plain stores
};

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code) {
    for (uint32_t i = 0; i < GM_SPIN_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 2000) {
            __nanosleep(40);
            if (*abort_flag) return false;
        }
    }
    *abort_flag = 1;
    atomicCAS(&g_gemm_status, 0, code);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128-byte swizzle: 8-row groups of 1024 bytes (stride-dimension byte
// offset), descriptor version 1, layout type 2; the start address advances by
// 32 bytes per 16-element k step inside the swizzle atom.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

template <bool BF16>
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    if constexpr (BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __half2 v = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

template <int BITS, bool BF16>
__global__ void __launch_bounds__(GM_THREADS, 1) gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmArgs a) {
    constexpr int FB = frag_bytes(BITS);
    constexpr int A_BYTES = GM_ROWS * GM_KSTAGE * 2;          // 16 KB
    constexpr int P_BYTES = 8 * FB;                           // packed fragments of one slab
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tn = a.tn;
    const int B_BYTES = tn * 128;
    uint8_t* sA = smem;
    uint8_t* sB = sA + GM_STAGES * A_BYTES;
    uint8_t* sP = sB + GM_STAGES * GM_MAX_TN * 128;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sP + GM_PSTAGES * P_BYTES);
    // bars: full[NS], empty[NS], pfull[NP], pempty[NP], accum
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * GM_STAGES;
    const uint32_t bar_pfull = bar_empty + 8 * GM_STAGES, bar_pempty = bar_pfull + 8 * GM_PSTAGES;
    const uint32_t bar_accum = bar_pempty + 8 * GM_PSTAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * GM_STAGES + 2 * GM_PSTAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tile = blockIdx.x, tok_tile = blockIdx.y, split = blockIdx.z;
    const int slab0 = (int)(((int64_t)a.n_slabs * split) / a.splits);
    const int slab1 = (int)(((int64_t)a.n_slabs * (split + 1)) / a.splits);
    const int n_it = (slab1 - slab0) * 2;                     // k-stages of 64
    const int rt0 = n_tile * 8;                               // first 16-row tile
    const int n_rt = min(8, a.NT - rt0);                      // valid 16-row tiles in this CTA
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < tn) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < GM_STAGES; ++s) { mbar_init(bar_full + 8 * s, 5); mbar_init(bar_empty + 8 * s, 1); }
        for (int s = 0; s < GM_PSTAGES; ++s) { mbar_init(bar_pfull + 8 * s, 1); mbar_init(bar_pempty + 8 * s, 4); }
        mbar_init(bar_accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (n_it > 0) {
        if (warp == 0) {
            // ---------------- producer: packed fragments (bulk copies) + token tiles (TMA) --------------
            if (lane == 0) {
                bool ok = true;
                for (int it = 0; it < n_it && ok; ++it) {
                    if ((it & 1) == 0) {
                        const int pi = it >> 1, ps = pi % GM_PSTAGES;
                        ok = mbar_wait(bar_pempty + 8 * ps, ((pi / GM_PSTAGES) & 1) ^ 1, abort_flag, 1);
                        if (!ok) break;
                        const int slab = slab0 + pi;
                        mbar_expect_tx(bar_pfull + 8 * ps, (uint32_t)(n_rt * FB));
                        for (int ft = 0; ft < n_rt; ++ft) {
                            const int64_t f = (((int64_t)(slab >> 1) * a.NT + rt0 + ft) * 2 + (slab & 1));
                            bulk_load(smem_u32(sP + ps * P_BYTES + ft * FB), a.frags + f * FB, FB, bar_pfull + 8 * ps);
                        }
                    }
                    const int s = it % GM_STAGES;
                    ok = mbar_wait(bar_empty + 8 * s, ((it / GM_STAGES) & 1) ^ 1, abort_flag, 2);
                    if (!ok) break;
                    mbar_expect_tx(bar_full + 8 * s, (uint32_t)B_BYTES);
                    tma_load_2d(smem_u32(sB + s * GM_MAX_TN * 128), &tmap_x, (slab0 * 2 + it) * GM_KSTAGE, tok_tile * tn,
                                bar_full + 8 * s);
                }
            }
        } else if (warp == 5) {
            // ---------------- MMA issue ----------------------------------------------------------------
            if (lane == 0) {
                const uint32_t idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) |
                                       ((uint32_t)(tn >> 3) << 17) | ((uint32_t)(GM_ROWS >> 4) << 24);
                bool ok = true;
                for (int it = 0; it < n_it; ++it) {
                    const int s = it % GM_STAGES;
                    ok = mbar_wait(bar_full + 8 * s, (it / GM_STAGES) & 1, abort_flag, 3);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t ad = make_smem_desc(smem_u32(sA + s * A_BYTES));
                    const uint64_t bd = make_smem_desc(smem_u32(sB + s * GM_MAX_TN * 128));
#pragma unroll
                    for (int k = 0; k < GM_KSTAGE / 16; ++k)
                        umma_f16(tmem_base, ad + 2 * k, bd + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
                    umma_commit(bar_empty + 8 * s);
                }
                if (ok) umma_commit(bar_accum);
            }
        } else {
            // ---------------- dequantise (warps 1..4), then epilogue ------------------------------------
            const int dw = warp - 1, g = lane >> 2, t = lane & 3;
            bool ok = true;
            for (int pi = 0; pi < (n_it >> 1) && ok; ++pi) {
                const int ps = pi % GM_PSTAGES;
                ok = mbar_wait(bar_pfull + 8 * ps, (pi / GM_PSTAGES) & 1, abort_flag, 4);
                if (!ok) break;
                LaneCodes<BITS> lc[2];
                uint32_t dmw[2][2][4];   // [fragment][row half][block]: half2 (scale, min)
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int ft = 2 * dw + q;
                    const uint8_t* fb = sP + ps * P_BYTES + ft * FB;
                    if (ft < n_rt) {
                        load_lane_codes<BITS>(lc[q], fb, lane);
                        const uint4 s0 = *reinterpret_cast<const uint4*>(fb + g * 16);
                        const uint4 s1 = *reinterpret_cast<const uint4*>(fb + (g + 8) * 16);
                        dmw[q][0][0] = s0.x; dmw[q][0][1] = s0.y; dmw[q][0][2] = s0.z; dmw[q][0][3] = s0.w;
                        dmw[q][1][0] = s1.x; dmw[q][1][1] = s1.y; dmw[q][1][2] = s1.z; dmw[q][1][3] = s1.w;
                    } else {
#pragma unroll
                        for (int i = 0; i < 2 * BITS; ++i) lc[q].w[i] = 0;
#pragma unroll
                        for (int i = 0; i < 4; ++i) { dmw[q][0][i] = 0; dmw[q][1][i] = 0; }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pempty + 8 * ps);   // packed bytes are in registers now
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int it = 2 * pi + h, s = it % GM_STAGES;
                    ok = mbar_wait(bar_empty + 8 * s, ((it / GM_STAGES) & 1) ^ 1, abort_flag, 5);
                    if (!ok) break;
                    uint8_t* At = sA + s * A_BYTES;
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            const int j = 2 * h + jj;
#pragma unroll
                            for (int hi = 0; hi < 2; ++hi) {
                                const __half2 dm = *reinterpret_cast<const __half2*>(&dmw[q][hi][j]);
                                const float d = __low2float(dm), m = __high2float(dm);
                                uint32_t o[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const uint32_t p = code_pair<BITS>(lc[q], j, hi, i, 0u);
                                    o[i] = pack2<BF16>(fmaf(d, (float)(p & 0xffffu), m), fmaf(d, (float)(p >> 16), m));
                                }
                                const int row = (2 * dw + q) * 16 + g + 8 * hi;
                                const int chunk = (jj * 4 + t) ^ (row & 7);
                                *reinterpret_cast<uint4*>(At + (row >> 3) * 1024 + (row & 7) * 128 + chunk * 16) =
                                    make_uint4(o[0], o[1], o[2], o[3]);
                            }
                        }
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_full + 8 * s);
                }
            }
            // epilogue: TMEM lane quarter (warp % 4) -> out[token][row]
            if (ok) ok = mbar_wait(bar_accum, 0, abort_flag, 6);
            if (ok) {
                tc_fence_after();
                const int lq = warp & 3;
                const int64_t n = (int64_t)n_tile * GM_ROWS + lq * 32 + lane;
                for (int c0 = 0; c0 < tn; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0, v);
                    tmem_ld_wait();
                    if (n < a.N) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int tok = tok_tile * tn + c0 + j;
                            if (c0 + j < tn && tok < a.M) {
                                float* o = a.out + (int64_t)tok * a.ldo + n;
                                if (a.use_red) atomicAdd(o, __uint_as_float(v[j]));
                                else *o = __uint_as_float(v[j]);
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);   // let copies in flight land before the CTA's shared memory goes away
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ---- host ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <int BITS, bool BF16>
static cudaError_t launch_one(const CUtensorMap& tm, const GemmArgs& a, dim3 grid, cudaStream_t s) {
    constexpr int FB = frag_bytes(BITS);
    constexpr int SMEM = 1024 + GM_STAGES * (GM_ROWS * GM_KSTAGE * 2 + GM_MAX_TN * 128) + GM_PSTAGES * 8 * FB + 256;
    auto kern = gemm_kernel<BITS, BF16>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<grid, GM_THREADS, SMEM, s>>>(tm, a);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gemm(const aq_handle_s* h, const void* x, aq_dtype_t xdt, int M, float* out, int64_t ldo,
                        bool accumulate, cudaStream_t s) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    GemmArgs a;
    a.frags = h->frags; a.out = out; a.ldo = ldo; a.N = h->N; a.M = M; a.NT = h->NT; a.n_slabs = h->KP * 2;
    a.tn = (M >= GM_MAX_TN) ? GM_MAX_TN : ((M + 15) / 16) * 16;
    const int n_tiles = (h->NT + 7) / 8;
    const int tok_tiles = (M + a.tn - 1) / a.tn;
    // split K until the grid covers the SMs (at most one slab-pair per split)
    int splits = 1;
    const int target = sm_count();
    while (n_tiles * tok_tiles * splits < target && splits * 2 <= a.n_slabs / 2) splits *= 2;
    a.splits = splits;
    a.use_red = (accumulate || splits > 1) ? 1 : 0;
    if (splits > 1 && !accumulate) {
        cudaError_t e = cudaMemset2DAsync(out, (size_t)ldo * sizeof(float), 0, (size_t)h->N * sizeof(float), (size_t)M, s);
        if (e != cudaSuccess) return e;
    }
    CUtensorMap tm;
    const cuuint64_t dims[2] = {(cuuint64_t)h->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)h->K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)GM_KSTAGE, (cuuint32_t)a.tn};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(&tm, xdt == AQ_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
                           const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)n_tiles, (unsigned)tok_tiles, (unsigned)splits);
    const bool bf = (xdt == AQ_BF16);
    switch (h->bits) {
        case 2: return bf ? launch_one<2, true>(tm, a, grid, s) : launch_one<2, false>(tm, a, grid, s);
        case 3: return bf ? launch_one<3, true>(tm, a, grid, s) : launch_one<3, false>(tm, a, grid, s);
        default: return bf ? launch_one<4, true>(tm, a, grid, s) : launch_one<4, false>(tm, a, grid, s);
    }
}

int read_gemm_status(bool clear) {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int));
    if (clear && v) { int z = 0; cudaMemcpyToSymbol(g_gemm_status, &z, sizeof(int)); }
    return v;
}

}  // namespace aq
