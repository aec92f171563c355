// aq_pack / aq_import / aq_export kernels: float32 weights or canonical bytes
// <-> the device fragment layout.  Set-up work, not on the timed path.
//
// Quantiser: Eq. 1 (nearest code of the uniform codebook), one correctly
// rounded binary32 operation per step so that the result is reproducible.
#include "aq_internal.h"
#include "aq_layout.cuh"

namespace aq {

template <int BITS>
__device__ __forceinline__ void place_code(uint32_t* words, int j, int hi, int c, uint32_t q) {
#pragma unroll
    for (int tb = 0; tb < BITS; ++tb) {
        int widx, bitpos;
        slot_bit_home(BITS, j, hi, c, tb, widx, bitpos);
        words[widx] |= ((q >> tb) & 1u) << bitpos;
    }
}

template <int BITS>
__device__ __forceinline__ void store_lane_words(uint8_t* fb, int lane, const uint32_t* w) {
    *reinterpret_cast<uint4*>(fb + 256 + lane * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    if constexpr (BITS == 3) *reinterpret_cast<uint2*>(fb + 256 + 512 + lane * 8) = make_uint2(w[4], w[5]);
    if constexpr (BITS == 4) *reinterpret_cast<uint4*>(fb + 256 + 512 + lane * 16) = make_uint4(w[4], w[5], w[6], w[7]);
}

// One warp per fragment.  Lane (g,t) owns elements 8t..8t+7 of each of the 4
// blocks for rows g and g+8.
template <int BITS>
__global__ void __launch_bounds__(128) pack_kernel(const float* __restrict__ W, int64_t N, int64_t K, int NT,
                                                   int64_t n_frags, uint8_t* __restrict__ frags, int* flags) {
    constexpr int FB = frag_bytes(BITS);
    constexpr float L = float((1 << BITS) - 1);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t f = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (f >= n_frags) return;
    const int par = (int)(f & 1);
    const int64_t u = f >> 1;
    const int R = (int)(u % NT);
    const int64_t S = 2 * (u / NT) + par;
    uint8_t* fb = frags + f * FB;

    uint32_t words[2 * BITS];
#pragma unroll
    for (int i = 0; i < 2 * BITS; ++i) words[i] = 0;
    uint32_t my_dm[2] = {0, 0};
    bool bad = false;

    // all 16 loads of the lane first (the fragment's 8 KB are in flight at once), then the arithmetic
    float4 ld[4][2][2];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const int64_t row = (int64_t)R * 16 + g + 8 * hi;
            const int64_t k0 = S * 128 + 32 * j + 8 * t;
            ld[j][hi][0] = ld[j][hi][1] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < N && k0 < K) {
                ld[j][hi][0] = __ldcs(reinterpret_cast<const float4*>(W + row * K + k0));
                ld[j][hi][1] = __ldcs(reinterpret_cast<const float4*>(W + row * K + k0 + 4));
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const float4 a = ld[j][hi][0], b = ld[j][hi][1];
            const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            float mn = v[0], mx = v[0];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                mn = fminf(mn, v[c]); mx = fmaxf(mx, v[c]);
                if (!isfinite(v[c])) bad = true;
            }
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const __half dh = __float2half_rn(__fdiv_rn(__fsub_rn(mx, mn), L));
            const __half mh = __float2half_rn(mn);
            const float d32 = __half2float(dh), m32 = __half2float(mh);
            if (isinf(d32) || isinf(m32)) bad = true;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t q = 0;
                if (d32 != 0.f) {
                    const float tq = __fdiv_rn(__fsub_rn(v[c], m32), d32);
                    q = (uint32_t)fminf(fmaxf(rintf(tq), 0.f), L);
                }
                place_code<BITS>(words, j, hi, c, q);
            }
            if (j == t) my_dm[hi] = (uint32_t)__half_as_ushort(dh) | ((uint32_t)__half_as_ushort(mh) << 16);
        }
    }
    store_lane_words<BITS>(fb, lane, words);
    *reinterpret_cast<uint32_t*>(fb + (g * 4 + t) * 4) = my_dm[0];
    *reinterpret_cast<uint32_t*>(fb + ((g + 8) * 4 + t) * 4) = my_dm[1];
    if (bad) atomicOr(flags, 1);
}

// ---- scale-optimised packing (Section 3.3, Eq. 10 and Eq. 11) -------------------------------
// Sum over a block's 32 values, 8 per lane over the 4 lanes of a block: left to right inside the
// lane, then (l0 + l1) + (l2 + l3); one binary32 rounding per addition.  Called by all 32 lanes.
__device__ __forceinline__ float block_sum32(const float (&x)[8]) {
    float a = x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) a = __fadd_rn(a, x[i]);
    a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, 2));
    return a;
}

// Codes of a block for binary16 parameters (d, m), as pack_kernel chooses them, and
// Phi = sum omega (w - (d q + m))^2 of Eq. 10 for that choice.
__device__ __forceinline__ float code_block(const float (&v)[8], const float (&om)[8], float d32, float m32, float L, float (&q)[8]) {
    float e[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const float t = (d32 != 0.f) ? __fdiv_rn(__fsub_rn(v[c], m32), d32) : 0.f;
        q[c] = fminf(fmaxf(rintf(t), 0.f), L);
        const float r = __fsub_rn(v[c], __fadd_rn(__fmul_rn(d32, q[c]), m32));
        e[c] = __fmul_rn(om[c], __fmul_rn(r, r));
    }
    return block_sum32(e);
}

// As pack_kernel, but the block parameters come from the alternation of Eq. 11 (nearest codes for
// fixed parameters; weighted least squares for (scale, min) with fixed codes), started from the
// round-to-nearest parameters and weighted by omega = F sqrt(sigma^2 + w^2) (Eq. 10; F may be null
// = 1).  Every operation is a single correctly rounded binary32 (the 2 x 2 solve: binary64)
// operation in a fixed order, so that a CPU restatement reproduces the bytes.  A block keeps its
// round-to-nearest form unless the optimised one, after rounding to binary16, lowers Phi.
template <int BITS>
__global__ void __launch_bounds__(128) pack_opt_kernel(const float* __restrict__ W, const float* __restrict__ F, int rounds,
                                                       int64_t N, int64_t K, int NT, int64_t n_frags,
                                                       uint8_t* __restrict__ frags, int* flags) {
    constexpr int FB = frag_bytes(BITS);
    constexpr float L = float((1 << BITS) - 1);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t f = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (f >= n_frags) return;
    const int par = (int)(f & 1);
    const int64_t u = f >> 1;
    const int R = (int)(u % NT);
    const int64_t S = 2 * (u / NT) + par;
    uint8_t* fb = frags + f * FB;

    uint32_t words[2 * BITS];
#pragma unroll
    for (int i = 0; i < 2 * BITS; ++i) words[i] = 0;
    uint32_t my_dm[2] = {0, 0};
    bool bad = false;

#pragma unroll 1
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const int64_t row = (int64_t)R * 16 + g + 8 * hi;
            const int64_t k0 = S * 128 + 32 * j + 8 * t;
            const bool in = row < N && k0 < K;
            float v[8], om[8], ow[8], tmp[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) { v[c] = 0.f; om[c] = 1.f; }
            if (in) {
                const float4 a = *reinterpret_cast<const float4*>(W + row * K + k0);
                const float4 b = *reinterpret_cast<const float4*>(W + row * K + k0 + 4);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            }
            float mn = v[0], mx = v[0];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                mn = fminf(mn, v[c]); mx = fmaxf(mx, v[c]);
                if (!isfinite(v[c])) bad = true;
                tmp[c] = __fmul_rn(v[c], v[c]);
            }
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float sig2 = __fdiv_rn(block_sum32(tmp), 32.f);
#pragma unroll
            for (int c = 0; c < 8; ++c) om[c] = __fsqrt_rn(__fadd_rn(sig2, tmp[c]));
            if (F != nullptr && in) {
                const float4 a = *reinterpret_cast<const float4*>(F + row * K + k0);
                const float4 b = *reinterpret_cast<const float4*>(F + row * K + k0 + 4);
                const float fv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                for (int c = 0; c < 8; ++c) om[c] = __fmul_rn(fv[c], om[c]);
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) ow[c] = __fmul_rn(om[c], v[c]);
            const float S0 = block_sum32(om), Sw = block_sum32(ow);
            const float rtn = __fdiv_rn(__fsub_rn(mx, mn), L);
            float s = rtn, mm = mn;
            bool live = s > 0.f;
            for (int r = 0; r < rounds; ++r) {
                float q[8], oq[8];
                const float den = live ? s : 1.f;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    q[c] = fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(v[c], mm), den)), 0.f), L);
                    oq[c] = __fmul_rn(om[c], q[c]);
                }
                const float S1 = block_sum32(oq);
#pragma unroll
                for (int c = 0; c < 8; ++c) tmp[c] = __fmul_rn(oq[c], q[c]);
                const float S2 = block_sum32(tmp);
#pragma unroll
                for (int c = 0; c < 8; ++c) tmp[c] = __fmul_rn(ow[c], q[c]);
                const float Swq = block_sum32(tmp);
                const double a0 = S0, a1 = S1, a2 = S2, aw = Sw, awq = Swq;
                const double det = __dsub_rn(__dmul_rn(a0, a2), __dmul_rn(a1, a1));
                const double s_new = __ddiv_rn(__dsub_rn(__dmul_rn(a0, awq), __dmul_rn(a1, aw)), det);
                const double m_new = __ddiv_rn(__dsub_rn(aw, __dmul_rn(s_new, a1)), a0);
                live = live && det > 0.0 && isfinite(s_new) && s_new > 0.0;
                if (live) { s = __double2float_rn(s_new); mm = __double2float_rn(m_new); }
            }
            const __half dA = __float2half_rn(rtn), mA = __float2half_rn(mn);
            const __half dB = __float2half_rn(s), mB = __float2half_rn(mm);
            float qA[8], qB[8];
            const float phiA = code_block(v, om, __half2float(dA), __half2float(mA), L, qA);
            const float phiB = code_block(v, om, __half2float(dB), __half2float(mB), L, qB);
            const float dB32 = __half2float(dB), mB32 = __half2float(mB);
            const bool useB = isfinite(dB32) && dB32 != 0.f && isfinite(mB32) && phiB < phiA;
            const __half dh = useB ? dB : dA, mh = useB ? mB : mA;
            if (isinf(__half2float(dh)) || isinf(__half2float(mh))) bad = true;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t q = (uint32_t)(useB ? qB[c] : qA[c]);
                if (j == 0) place_code<BITS>(words, 0, hi, c, q);
                else if (j == 1) place_code<BITS>(words, 1, hi, c, q);
                else if (j == 2) place_code<BITS>(words, 2, hi, c, q);
                else place_code<BITS>(words, 3, hi, c, q);
            }
            if (j == t) my_dm[hi] = (uint32_t)__half_as_ushort(dh) | ((uint32_t)__half_as_ushort(mh) << 16);
        }
    }
    store_lane_words<BITS>(fb, lane, words);
    *reinterpret_cast<uint32_t*>(fb + (g * 4 + t) * 4) = my_dm[0];
    *reinterpret_cast<uint32_t*>(fb + ((g + 8) * 4 + t) * 4) = my_dm[1];
    if (bad) atomicOr(flags, 1);
}

// One warp per fragment, reading block records of the canonical stream.
template <int BITS>
__global__ void __launch_bounds__(128) import_kernel(const uint8_t* __restrict__ canon, int64_t N, int64_t K, int NT,
                                                     int64_t n_frags, uint8_t* __restrict__ frags) {
    constexpr int FB = frag_bytes(BITS);
    constexpr int REC = 4 + 4 * BITS;
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t f = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (f >= n_frags) return;
    const int par = (int)(f & 1);
    const int64_t u = f >> 1;
    const int R = (int)(u % NT);
    const int64_t S = 2 * (u / NT) + par;
    const int64_t nb = K / 32;
    uint8_t* fb = frags + f * FB;
    uint32_t words[2 * BITS];
#pragma unroll
    for (int i = 0; i < 2 * BITS; ++i) words[i] = 0;
    uint32_t my_dm[2] = {0, 0};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const int64_t row = (int64_t)R * 16 + g + 8 * hi;
            const int64_t jb = S * 4 + j;
            if (row < N && jb < nb) {
                const uint8_t* rec = canon + (row * nb + jb) * REC;
                uint32_t val = 0;   // the 8*BITS bits holding codes 8t..8t+7
#pragma unroll
                for (int b = 0; b < BITS; ++b) val |= (uint32_t)rec[4 + t * BITS + b] << (8 * b);
#pragma unroll
                for (int c = 0; c < 8; ++c) place_code<BITS>(words, j, hi, c, (val >> (BITS * c)) & ((1u << BITS) - 1));
                if (j == t) my_dm[hi] = (uint32_t)rec[0] | ((uint32_t)rec[1] << 8) | ((uint32_t)rec[2] << 16) | ((uint32_t)rec[3] << 24);
            }
        }
    }
    store_lane_words<BITS>(fb, lane, words);
    *reinterpret_cast<uint32_t*>(fb + (g * 4 + t) * 4) = my_dm[0];
    *reinterpret_cast<uint32_t*>(fb + ((g + 8) * 4 + t) * 4) = my_dm[1];
}

// One thread per (row, block): gathers the block's bits through code_bit_home().
__global__ void __launch_bounds__(128) export_kernel(const uint8_t* __restrict__ frags, int bits, int64_t N, int64_t K,
                                                     int NT, uint8_t* __restrict__ canon) {
    const int64_t nb = K / 32;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * nb) return;
    const int64_t row = idx / nb, jb = idx % nb;
    const int64_t S = jb >> 2;
    const int j = (int)(jb & 3), r = (int)(row & 15);
    const int64_t R = row >> 4;
    const int FB = frag_bytes(bits);
    const uint8_t* fb = frags + (((S >> 1) * NT + R) * 2 + (S & 1)) * FB;
    const int rec_bytes = 4 + 4 * bits;
    uint8_t* rec = canon + idx * rec_bytes;
    const uint32_t dm = *reinterpret_cast<const uint32_t*>(fb + (r * 4 + j) * 4);
    rec[0] = dm & 0xff; rec[1] = (dm >> 8) & 0xff; rec[2] = (dm >> 16) & 0xff; rec[3] = (dm >> 24) & 0xff;
    uint32_t stream[4] = {0, 0, 0, 0};   // 32*bits bits
    for (int e = 0; e < 32; ++e) {
        for (int tb = 0; tb < bits; ++tb) {
            int wo, bp;
            code_bit_home(bits, r, 32 * j + e, tb, wo, bp);
            const uint32_t bit = (*reinterpret_cast<const uint32_t*>(fb + wo) >> bp) & 1u;
            const int sb = bits * e + tb;
            stream[sb >> 5] |= bit << (sb & 31);
        }
    }
    for (int p = 0; p < 4 * bits; ++p) rec[4 + p] = (stream[p >> 2] >> (8 * (p & 3))) & 0xff;
}

cudaError_t launch_pack(const aq_handle_s* h, const float* W, cudaStream_t s) {
    const unsigned grid = (unsigned)((h->n_frags + 3) / 4);
    switch (h->bits) {
        case 2: pack_kernel<2><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
        case 3: pack_kernel<3><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
        default: pack_kernel<4><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_pack_opt(const aq_handle_s* h, const float* W, const float* F, int rounds, cudaStream_t s) {
    const unsigned grid = (unsigned)((h->n_frags + 3) / 4);
    switch (h->bits) {
        case 2: pack_opt_kernel<2><<<grid, 128, 0, s>>>(W, F, rounds, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
        case 3: pack_opt_kernel<3><<<grid, 128, 0, s>>>(W, F, rounds, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
        default: pack_opt_kernel<4><<<grid, 128, 0, s>>>(W, F, rounds, h->N, h->K, h->NT, h->n_frags, h->frags, h->flags); break;
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_import(const aq_handle_s* h, const uint8_t* canon_dev, cudaStream_t s) {
    const unsigned grid = (unsigned)((h->n_frags + 3) / 4);
    switch (h->bits) {
        case 2: import_kernel<2><<<grid, 128, 0, s>>>(canon_dev, h->N, h->K, h->NT, h->n_frags, h->frags); break;
        case 3: import_kernel<3><<<grid, 128, 0, s>>>(canon_dev, h->N, h->K, h->NT, h->n_frags, h->frags); break;
        default: import_kernel<4><<<grid, 128, 0, s>>>(canon_dev, h->N, h->K, h->NT, h->n_frags, h->frags); break;
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_export(const aq_handle_s* h, uint8_t* canon_dev, cudaStream_t s) {
    const int64_t n = h->N * (h->K / 32);
    const unsigned grid = (unsigned)((n + 127) / 128);
    export_kernel<<<grid, 128, 0, s>>>(h->frags, h->bits, h->N, h->K, h->NT, canon_dev);
    count_launch();
    return cudaGetLastError();
}

}  // namespace aq
