// Device code shared by the decode kernels (single linear and whole stack):
// the x operand of one 256-k pair-slab, one unit (16 rows x 256 k) of
// multiply-accumulate on the tensor cores, and the commit of a unit's sums.
//
// With w = d q + m per block (Eq. 1),   sum_k x w = d * sum q x  +  m * sum x.
// sum q x runs on mma.sync m16n8k16 (fp32 accumulate) with the codes as the A
// operand and x as the B operand.  The 8 columns of the instruction are
// (block, token) pairs: with MT tokens per call, 8/MT blocks accumulate side
// by side (MT = 1: the 8 blocks of a whole unit) and the per-block scale
// touches the accumulators once per group of 8/MT blocks.
//
// fp16 activations: a code is used where it lies in its word (one AND per A
// register, see InPlace<> in aq_layout.cuh) as the binary16 subnormal
// q 2^(s-24); instructions that read bit position s accumulate into their own
// set of registers and the powers of two are taken out, exactly, when a group
// ends.  The decode kernel is bound by the integer pipe, not by the tensor
// pipe, so what counts is bit operations per weight: here 1/2 AND + 1/16 shift.
//
// bf16 activations: bf16 subnormals would push the products below the fp32
// normal range, so codes are shifted down and OR-ed into the mantissa of 128.0
// (BIAS), and   sum x w = d * sum (BIAS + q) x + (m - BIAS d) * sum x.
#pragma once
#include "aq_layout.cuh"

namespace aq {

// c = a b + c, or c = a b when `first` (the accumulator then needs no zeroing).
template <bool BF16>
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, bool first = false) {
    const float z0 = first ? 0.f : c[0], z1 = first ? 0.f : c[1], z2 = first ? 0.f : c[2], z3 = first ? 0.f : c[3];
    if constexpr (BF16) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                     : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(z0), "f"(z1), "f"(z2), "f"(z3));
    } else {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                     : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(z0), "f"(z1), "f"(z2), "f"(z3));
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

// Where the 16-byte chunk (block bk, quarter t) of a one-token slab staged in shared memory lives: in the
// row of the lane (bk, t) that multiplies it, at a position rotated by the lane
// so that the eight chunks a lane reads never collide on a bank.
__device__ __forceinline__ int ds_spread_offset(int lane, int bk) { return lane * 128 + ((bk ^ (lane & 7)) * 16); }
// The same place as a shared-memory address: with the slab 128-byte aligned, chunk bk of a lane is at
// (slab + lane * 128 + (lane & 7) * 16) ^ (bk * 16), one XOR with a constant per block.
__device__ __forceinline__ uint32_t ds_spread_lane_base(const uint8_t* slab, int lane) {
    return (uint32_t)__cvta_generic_to_shared(slab) + (uint32_t)(lane * 128 + (lane & 7) * 16);
}

// Per-warp state for the x operand of one pair-slab (256 k = the 8 blocks of a unit).
// Lane (g, t) stands for B column g = (block slot g / MT, token g % MT).
template <int MT>
struct XOperand {
    static constexpr int BG = 8 / MT;   // blocks that accumulate side by side
    static constexpr int NG = MT;       // groups per unit
    uint32_t b[8][4];                   // [block][reg]: B registers, zero unless the block sits in this lane's slot
    float X0[NG], X1[NG];               // block sums of x for this lane's two accumulator columns
};

// Fills the operand from 8 halves per group: fetch(tok, k_in_slab) returns the
// lane's 16 bytes x[tok][k .. k+8) (zeros when out of range).
template <int MT, bool BF16, typename Fetch>
__device__ __forceinline__ void fill_x_operand(XOperand<MT>& xo, int lane, Fetch fetch) {
    constexpr int BG = XOperand<MT>::BG, NG = XOperand<MT>::NG;
    const int g = lane >> 2, t = lane & 3;
    const int tok = g % MT, bs = g / MT;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
        const int jb = gi * BG + bs;
        const uint4 v = fetch(tok, 32 * jb + 8 * t);
        float s = sum8<BF16>(v);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        // the lane's accumulator columns 2t, 2t+1 are B columns of lanes g' = 2t, 2t+1
        xo.X0[gi] = __shfl_sync(0xffffffffu, s, (2 * t) * 4);
        xo.X1[gi] = __shfl_sync(0xffffffffu, s, (2 * t + 1) * 4);
#pragma unroll
        for (int b2 = 0; b2 < BG; ++b2) {
            const bool on = (b2 == bs);
            xo.b[gi * BG + b2][0] = on ? v.x : 0u;
            xo.b[gi * BG + b2][1] = on ? v.y : 0u;
            xo.b[gi * BG + b2][2] = on ? v.z : 0u;
            xo.b[gi * BG + b2][3] = on ? v.w : 0u;
        }
    }
}

// x in global memory, row-major [M][K] of half / bf16.
template <int MT, bool BF16>
__device__ __forceinline__ void load_x_operand(XOperand<MT>& xo, const void* xv, int64_t K, int M, int64_t P, int lane) {
    const uint16_t* x = reinterpret_cast<const uint16_t*>(xv);
    fill_x_operand<MT, BF16>(xo, lane, [&](int tok, int kk) {
        const int64_t k = P * 256 + kk;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (tok < M && k < K) v = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)tok * K + k));
        return v;
    });
}

// The factor of sum x: m for in-place codes, m - BIAS d when the codes carry a bias of 128.
template <bool BF16>
__device__ __forceinline__ float min_term(float d, float m) {
    if constexpr (BF16) return fmaf(-128.f, d, m);
    else return m;
}

// True when an instruction f = 2j + h of blocks [b0, b0 + n) reads bit-position class c.
template <int BITS>
__device__ __forceinline__ constexpr bool class_used(int c, int b0, int n) {
    for (int b = b0; b < b0 + n; ++b)
        for (int h = 0; h < 2; ++h)
            if (InPlace<BITS>::cls(2 * (b & 3) + h) == c) return true;
    return false;
}

// True when an instruction of blocks [b0, b) or of block b with half < h reads class c.
template <int BITS>
__device__ __forceinline__ constexpr bool class_used_before(int c, int b0, int b, int h) {
    for (int bb = b0; bb <= b; ++bb)
        for (int hh = 0; hh < 2; ++hh) {
            if (bb == b && hh >= h) break;
            if (InPlace<BITS>::cls(2 * (bb & 3) + hh) == c) return true;
        }
    return false;
}

// One unit (two fragments) against the prepared x operand; adds to this lane's four partial sums:
//   MT >= 2: [row g, col 2t], [row g, col 2t+1], [row g+8, col 2t], [row g+8, col 2t+1]
//            (columns are (block slot, token) pairs, both columns in one slot)
//   MT == 1: the same four, where columns 2t, 2t+1 are two different blocks.
//
// With XS (one token only) the B registers are not taken from xo.b but read, block by block, from the spread-out
// copy of the slab in shared memory (xlane = ds_spread_lane_base of that copy): 32 registers fewer per thread for one
// 16-byte shared load per block.
template <int BITS, int MT, bool BF16, bool XS = false>
__device__ __forceinline__ void unit_mac(const uint8_t* unit, const XOperand<MT>& xo, int lane, float (&acc)[4],
                                         uint32_t xlane = 0) {
    static_assert(!XS || MT == 1, "the shared-memory x operand is the one-token layout");
    using IP = InPlace<BITS>;
    constexpr int FB = frag_bytes(BITS);
    constexpr int BG = XOperand<MT>::BG;
    constexpr int NCLS = BF16 ? 1 : IP::NCLS;
    constexpr uint32_t MAGIC = 0x43004300u;   // bf16 128.0 in both halves
    const int g = lane >> 2, t = lane & 3;
    float cs[NCLS][4];
    LaneCodes<BITS> lc;
    IP ip;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int fi = b >> 2, j = b & 3;
        if (j == 0) {
            load_lane_codes<BITS>(lc, unit + fi * FB, lane);
            if constexpr (!BF16) ip.prepare(lc);
        }
        uint32_t xb[4];
        if constexpr (XS) {
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(xb[0]), "=r"(xb[1]), "=r"(xb[2]), "=r"(xb[3]) : "r"(xlane ^ (uint32_t)(b * 16)));
        } else {
            xb[0] = xo.b[b][0]; xb[1] = xo.b[b][1]; xb[2] = xo.b[b][2]; xb[3] = xo.b[b][3];
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int f = 2 * j + h;
            uint32_t a[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if constexpr (BF16) a[r] = code_pair<BITS>(lc, j, r & 1, 2 * h + (r >> 1), MAGIC);
                else a[r] = ip.reg(f, r);
            }
            // the first instruction of a group that touches an accumulator set starts it from zero
            const int k = BF16 ? 0 : IP::cls(f);
            const bool first = BF16 ? (b % BG == 0 && h == 0) : !class_used_before<BITS>(k, b - b % BG, b, h);
            mma16816<BF16>(cs[k], a, xb[2 * h], xb[2 * h + 1], first);
        }
        if (b % BG == BG - 1) {
            // group of blocks [b - BG + 1, b] done: take the powers of two out, apply scale and min
            const int gi = b / BG;
            float c[4];
            if constexpr (BF16) {
                c[0] = cs[0][0]; c[1] = cs[0][1]; c[2] = cs[0][2]; c[3] = cs[0][3];
            } else {
                c[0] = c[1] = c[2] = c[3] = 0.f;
#pragma unroll
                for (int k = 0; k < NCLS; ++k) {
                    if (class_used<BITS>(k, b - BG + 1, BG)) {
                        const float mul = (float)(1u << (24 - IP::cls_pos(k)));
#pragma unroll
                        for (int x = 0; x < 4; ++x) c[x] = fmaf(cs[k][x], mul, c[x]);
                    }
                }
            }
            if constexpr (MT == 1) {
                // columns 2t, 2t+1 = blocks 2t, 2t+1 of the unit: fragment t >> 1, blocks 2 (t & 1) and the next
                const uint8_t* fb = unit + (t >> 1) * FB;
                const int j0 = 2 * (t & 1);
                const uint2 s0 = *reinterpret_cast<const uint2*>(fb + (g * 4 + j0) * 4);
                const uint2 s1 = *reinterpret_cast<const uint2*>(fb + ((g + 8) * 4 + j0) * 4);
                const __half2 a0 = *reinterpret_cast<const __half2*>(&s0.x), b0 = *reinterpret_cast<const __half2*>(&s0.y);
                const __half2 a1 = *reinterpret_cast<const __half2*>(&s1.x), b1 = *reinterpret_cast<const __half2*>(&s1.y);
                const float X0 = xo.X0[0], X1 = xo.X1[0];
                const float dA0 = __low2float(a0), dB0 = __low2float(b0), dA1 = __low2float(a1), dB1 = __low2float(b1);
                acc[0] = fmaf(dA0, c[0], fmaf(min_term<BF16>(dA0, __high2float(a0)), X0, acc[0]));
                acc[1] = fmaf(dB0, c[1], fmaf(min_term<BF16>(dB0, __high2float(b0)), X1, acc[1]));
                acc[2] = fmaf(dA1, c[2], fmaf(min_term<BF16>(dA1, __high2float(a1)), X0, acc[2]));
                acc[3] = fmaf(dB1, c[3], fmaf(min_term<BF16>(dB1, __high2float(b1)), X1, acc[3]));
            } else {
                const int jbm = gi * BG + (2 * t) / MT;   // the block (0..7) behind this lane's two columns
                const uint8_t* fb = unit + (jbm >> 2) * FB;
                const __half2 dm0 = *reinterpret_cast<const __half2*>(fb + (g * 4 + (jbm & 3)) * 4);
                const __half2 dm1 = *reinterpret_cast<const __half2*>(fb + ((g + 8) * 4 + (jbm & 3)) * 4);
                const float d0 = __low2float(dm0), d1 = __low2float(dm1);
                const float mp0 = min_term<BF16>(d0, __high2float(dm0)), mp1 = min_term<BF16>(d1, __high2float(dm1));
                const float X0 = xo.X0[gi], X1 = xo.X1[gi];
                acc[0] = fmaf(d0, c[0], fmaf(mp0, X0, acc[0]));
                acc[1] = fmaf(d0, c[1], fmaf(mp0, X1, acc[1]));
                acc[2] = fmaf(d1, c[2], fmaf(mp1, X0, acc[2]));
                acc[3] = fmaf(d1, c[3], fmaf(mp1, X1, acc[3]));
            }
        }
    }
}

// Cross-lane reduction and accumulation into out[tok][row] (fp32, red.add).
// When `res` is given (same shape as out), res[tok][row] is added as well.
template <int MT>
__device__ __forceinline__ void unit_commit(float (&acc)[4], float* out, int64_t ld, int row0, int64_t N, int M, int lane,
                                            const float* res = nullptr) {
    const int g = lane >> 2, t = lane & 3;
    auto put = [&](int tok, int row, float v) {
        if (tok < M && row < N) {
            const int64_t o = (int64_t)tok * ld + row;
            atomicAdd(out + o, res ? v + __ldcg(res + o) : v);
        }
    };
    if constexpr (MT == 1) {
        // one token: both columns belong to it.  Lanes t = 0,1 end up with rows g, g+8.
        const float v0 = acc[0] + acc[1], v1 = acc[2] + acc[3];
        float keep = (t & 1) ? v1 : v0;
        const float send = (t & 1) ? v0 : v1;
        keep += __shfl_xor_sync(0xffffffffu, send, 1);
        keep += __shfl_xor_sync(0xffffffffu, keep, 2);
        if (t < 2) put(0, row0 + g + 8 * t, keep);
    } else if constexpr (MT == 2) {
        // four sums over four lanes: lane t ends up with sum t = (tok t & 1, row half t >> 1)
        float kA = (t & 1) ? acc[1] : acc[0], kB = (t & 1) ? acc[3] : acc[2];
        const float sA = (t & 1) ? acc[0] : acc[1], sB = (t & 1) ? acc[2] : acc[3];
        kA += __shfl_xor_sync(0xffffffffu, sA, 1);
        kB += __shfl_xor_sync(0xffffffffu, sB, 1);
        float v = (t & 2) ? kB : kA;
        const float s = (t & 2) ? kA : kB;
        v += __shfl_xor_sync(0xffffffffu, s, 2);
        put(t & 1, row0 + g + 8 * (t >> 1), v);
    } else if constexpr (MT == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 2);
        // lanes t = 0,1 hold tokens (2t, 2t+1); lanes 2,3 the same sums: split the four stores
        const int tk = 2 * (t & 1);
        const int hi = t >> 1;   // lanes 0,1 commit row g, lanes 2,3 row g+8
        put(tk, row0 + g + 8 * hi, hi ? acc[2] : acc[0]);
        put(tk + 1, row0 + g + 8 * hi, hi ? acc[3] : acc[1]);
    } else {
        const int tk = 2 * t;
        put(tk, row0 + g, acc[0]); put(tk, row0 + g + 8, acc[2]);
        put(tk + 1, row0 + g, acc[1]); put(tk + 1, row0 + g + 8, acc[3]);
    }
}

}  // namespace aq
