// Device code shared by the decode kernels (single linear and whole stack):
// the x operand of one 256-k pair-slab, one unit (16 rows x 256 k) of
// multiply-accumulate on the tensor cores, and the commit of a unit's sums.
//
// With w = d q + m per block (Eq. 1),
//     sum_k x w = d * sum (BIAS + q) x  +  (m - BIAS d) * sum x.
// The first sum runs on mma.sync m16n8k16 (fp32 accumulate): the A operand is
// built two codes per LOP3 by OR-ing the code bits into the mantissa of the
// half-precision constant BIAS (1024 for fp16, 128 for bf16); the B operand
// holds x.  The 8 columns of the instruction are (block, token) pairs: with MT
// tokens per call, 8/MT blocks accumulate side by side and the per-block scale
// touches the 4 accumulators once per group of 8/MT blocks.
#pragma once
#include "aq_layout.cuh"

namespace aq {

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
// When `res` is given (same shape as out), res[tok][row] is added as well.
template <int MT>
__device__ __forceinline__ void unit_commit(float (&acc)[4], float* out, int64_t ld, int row0, int64_t N, int M, int lane,
                                            const float* res = nullptr) {
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
        if (tok < M && row < N) {
            const int64_t o = (int64_t)tok * ld + row;
            atomicAdd(out + o, res ? v + __ldcg(res + o) : v);
        }
    } else if constexpr (MT == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 2);
        // lanes t = 0,1 hold tokens (2t, 2t+1); lanes 2,3 the same sums: split the four stores
        const int tk = 2 * (t & 1);
        const int hi = t >> 1;   // lanes 0,1 commit row g, lanes 2,3 row g+8
        const float v0 = hi ? acc[2] : acc[0], v1 = hi ? acc[3] : acc[1];
        const int row = row0 + g + 8 * hi;
        if (tk < M && row < N) {
            const int64_t o = (int64_t)tk * ld + row;
            atomicAdd(out + o, res ? v0 + __ldcg(res + o) : v0);
        }
        if (tk + 1 < M && row < N) {
            const int64_t o = (int64_t)(tk + 1) * ld + row;
            atomicAdd(out + o, res ? v1 + __ldcg(res + o) : v1);
        }
    } else {
        const int tk = 2 * t;
        const int r0 = row0 + g, r1 = row0 + g + 8;
        auto put = [&](int tok, int row, float v) {
            if (tok < M && row < N) {
                const int64_t o = (int64_t)tok * ld + row;
                atomicAdd(out + o, res ? v + __ldcg(res + o) : v);
            }
        };
        put(tk, r0, acc[0]); put(tk, r1, acc[2]);
        put(tk + 1, r0, acc[1]); put(tk + 1, r1, acc[3]);
    }
}

}  // namespace aq
