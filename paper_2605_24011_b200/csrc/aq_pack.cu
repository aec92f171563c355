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

#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const int64_t row = (int64_t)R * 16 + g + 8 * hi;
            const int64_t k0 = S * 128 + 32 * j + 8 * t;
            const bool in = row < N && k0 < K;
            float v[8];
            if (in) {
                const float4 a = *reinterpret_cast<const float4*>(W + row * K + k0);
                const float4 b = *reinterpret_cast<const float4*>(W + row * K + k0 + 4);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) v[c] = 0.f;
            }
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
