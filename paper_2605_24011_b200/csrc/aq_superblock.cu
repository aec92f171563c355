// Super-block format (Section 3, "Weight quantization": every S consecutive blocks form a super-block whose own
// scale and zero point compress the per-block parameters).  Reading taken: S = 8 blocks (256 weights); per
// super-block three binary16 values D, Dm, Mn and per block two 6-bit codes u, v with
//     scale_b = f16(D u_b),    min_b = f16(fma(Dm, v_b, Mn)),
// i.e. Eq. 1's rule one level up (symmetric for the scales, asymmetric for the minima), the decoded block parameters
// rounded to binary16.  n + 0.5625 bits per weight in the container instead of n + 1.
//
// On the device a super-block matrix is kept with its DECODED block parameters in the ordinary fragment layout, so
// every kernel of the hot path reads it unchanged; the super-block parameters sit beside the fragments (one 32-byte
// entry per row and super-block) for aq_export_sb.  Set-up work, not on the timed path.
#include "aq_internal.h"
#include "aq_layout.cuh"

namespace aq {

constexpr int SB_BLOCKS = 8;
constexpr float SB_MAX = 63.f;

struct SbEntry {          // one per (row, super-block)
    uint16_t D, Dm, Mn, pad;
    uint8_t u[8], v[8];
    uint8_t pad2[8];
};
static_assert(sizeof(SbEntry) == 32, "SbEntry layout");

template <int BITS>
__device__ __forceinline__ void sb_place_code(uint32_t* words, int j, int hi, int c, uint32_t q) {
#pragma unroll
    for (int tb = 0; tb < BITS; ++tb) {
        int widx, bitpos;
        slot_bit_home(BITS, j, hi, c, tb, widx, bitpos);
        words[widx] |= ((q >> tb) & 1u) << bitpos;
    }
}

// Decoded block parameters from the super-block's.
__device__ __forceinline__ void sb_decode(float D32, float Dm32, float Mn32, uint32_t u, uint32_t v, __half& dh, __half& mh) {
    dh = __float2half_rn(__fmul_rn(D32, (float)u));
    mh = __float2half_rn(__fmaf_rn(Dm32, (float)v, Mn32));
}

// One warp per unit (16 rows x 256 k = one super-block per row).  Lane (g, t) owns elements 8t..8t+7 of each of the
// 8 blocks for rows g and g + 8; the four lanes of a row see all of its blocks' extremes after two shuffles.
template <int BITS>
__global__ void __launch_bounds__(128) pack_sb_kernel(const float* __restrict__ W, int64_t N, int64_t K, int NT, int64_t n_units,
                                                      uint8_t* __restrict__ frags, SbEntry* __restrict__ side, int* flags) {
    constexpr int FB = frag_bytes(BITS);
    constexpr float L = float((1 << BITS) - 1);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t un = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (un >= n_units) return;
    const int R = (int)(un % NT);
    const int64_t P = un / NT;
    bool bad = false;
#pragma unroll 1
    for (int hi = 0; hi < 2; ++hi) {
        const int64_t row = (int64_t)R * 16 + g + 8 * hi;
        float v[8][8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t k0 = P * 256 + 32 * j + 8 * t;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            if (row < N) {
                a = __ldcs(reinterpret_cast<const float4*>(W + row * K + k0));
                b = __ldcs(reinterpret_cast<const float4*>(W + row * K + k0 + 4));
            }
            v[j][0] = a.x; v[j][1] = a.y; v[j][2] = a.z; v[j][3] = a.w; v[j][4] = b.x; v[j][5] = b.y; v[j][6] = b.z; v[j][7] = b.w;
        }
        float s[8], mn[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float lo = v[j][0], up = v[j][0];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                lo = fminf(lo, v[j][c]); up = fmaxf(up, v[j][c]);
                if (!isfinite(v[j][c])) bad = true;
            }
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 1)); up = fmaxf(up, __shfl_xor_sync(0xffffffffu, up, 1));
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 2)); up = fmaxf(up, __shfl_xor_sync(0xffffffffu, up, 2));
            s[j] = __fdiv_rn(__fsub_rn(up, lo), L);
            mn[j] = lo;
        }
        float smax = s[0], mlo = mn[0], mhi = mn[0];
#pragma unroll
        for (int j = 1; j < 8; ++j) { smax = fmaxf(smax, s[j]); mlo = fminf(mlo, mn[j]); mhi = fmaxf(mhi, mn[j]); }
        const __half Dh = __float2half_rn(__fdiv_rn(smax, SB_MAX));
        const __half Mnh = __float2half_rn(mlo);
        const float D32 = __half2float(Dh), Mn32 = __half2float(Mnh);
        const __half Dmh = __float2half_rn(__fdiv_rn(fmaxf(__fsub_rn(mhi, Mn32), 0.f), SB_MAX));
        const float Dm32 = __half2float(Dmh);
        if (isinf(D32) || isinf(Mn32) || isinf(Dm32)) bad = true;
        SbEntry e;
        e.D = __half_as_ushort(Dh); e.Dm = __half_as_ushort(Dmh); e.Mn = __half_as_ushort(Mnh); e.pad = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) e.pad2[i] = 0;
#pragma unroll
        for (int fi = 0; fi < 2; ++fi) {
            uint32_t words[2 * BITS];
#pragma unroll
            for (int i = 0; i < 2 * BITS; ++i) words[i] = 0;
            uint32_t my_dm = 0;
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = fi * 4 + jj;
                uint32_t ub = 0, vb = 0;
                if (D32 != 0.f) ub = (uint32_t)fminf(fmaxf(rintf(__fdiv_rn(s[j], D32)), 0.f), SB_MAX);
                if (Dm32 != 0.f) vb = (uint32_t)fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(mn[j], Mn32), Dm32)), 0.f), SB_MAX);
                e.u[j] = (uint8_t)ub; e.v[j] = (uint8_t)vb;
                __half dh, mh;
                sb_decode(D32, Dm32, Mn32, ub, vb, dh, mh);
                const float d32 = __half2float(dh), m32 = __half2float(mh);
                if (isinf(d32) || isinf(m32)) bad = true;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t q = 0;
                    if (d32 != 0.f) q = (uint32_t)fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(v[j][c], m32), d32)), 0.f), L);
                    sb_place_code<BITS>(words, jj, hi, c, q);
                }
                if (jj == t) my_dm = (uint32_t)__half_as_ushort(dh) | ((uint32_t)__half_as_ushort(mh) << 16);
            }
            // this half of the lane's words: the other row half's bits are OR-ed in by the second pass over hi
            uint8_t* fb = frags + (un * 2 + fi) * FB;
            uint32_t* w0 = reinterpret_cast<uint32_t*>(fb + 256 + lane * 16);
            if (hi == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) w0[i] = words[i];
                if constexpr (BITS == 3) { uint32_t* w1 = reinterpret_cast<uint32_t*>(fb + 256 + 512 + lane * 8); w1[0] = words[4]; w1[1] = words[5]; }
                if constexpr (BITS == 4) { uint32_t* w1 = reinterpret_cast<uint32_t*>(fb + 256 + 512 + lane * 16); for (int i = 0; i < 4; ++i) w1[i] = words[4 + i]; }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) w0[i] |= words[i];
                if constexpr (BITS == 3) { uint32_t* w1 = reinterpret_cast<uint32_t*>(fb + 256 + 512 + lane * 8); w1[0] |= words[4]; w1[1] |= words[5]; }
                if constexpr (BITS == 4) { uint32_t* w1 = reinterpret_cast<uint32_t*>(fb + 256 + 512 + lane * 16); for (int i = 0; i < 4; ++i) w1[i] |= words[4 + i]; }
            }
            *reinterpret_cast<uint32_t*>(fb + ((g + 8 * hi) * 4 + t) * 4) = my_dm;
        }
        if (t == 0 && row < N) side[row * (K / 256) + P] = e;
    }
    if (bad) atomicOr(flags, 1);
}

// Canonical super-block bytes <-> (side entries, plain canonical records with the decoded block parameters).
// One thread per (row, super-block).  to_plain: also writes the side entry (import); else reads it (export).
__global__ void __launch_bounds__(128) sb_records_kernel(uint8_t* sbcanon, uint8_t* plain, SbEntry* side,
                                                         int bits, int64_t N, int64_t K, int to_plain) {
    const int64_t ns = K / 256;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * ns) return;
    const int rec_sb = 18 + 32 * bits, rec_pl = 4 + 4 * bits;
    uint8_t* rs = sbcanon + idx * rec_sb;
    uint8_t* rp = plain + idx * 8 * rec_pl;
    if (to_plain) {
        SbEntry e;
        e.D = (uint16_t)(rs[0] | (rs[1] << 8)); e.Dm = (uint16_t)(rs[2] | (rs[3] << 8)); e.Mn = (uint16_t)(rs[4] | (rs[5] << 8)); e.pad = 0;
        for (int i = 0; i < 8; ++i) e.pad2[i] = 0;
        const float D32 = __half2float(__ushort_as_half(e.D)), Dm32 = __half2float(__ushort_as_half(e.Dm)), Mn32 = __half2float(__ushort_as_half(e.Mn));
        for (int b = 0; b < 8; ++b) {
            const int bit0 = 12 * b;   // 12 bits starting at bit0 of the 96-bit little-endian integer at rs + 6
            const uint32_t w = (uint32_t)rs[6 + (bit0 >> 3)] | ((uint32_t)rs[6 + (bit0 >> 3) + 1] << 8);
            const uint32_t uv = (w >> (bit0 & 7)) & 0xFFFu;
            e.u[b] = (uint8_t)(uv & 63u); e.v[b] = (uint8_t)(uv >> 6);
            __half dh, mh;
            sb_decode(D32, Dm32, Mn32, e.u[b], e.v[b], dh, mh);
            uint8_t* r = rp + b * rec_pl;
            const uint32_t dmw = (uint32_t)__half_as_ushort(dh) | ((uint32_t)__half_as_ushort(mh) << 16);
            *reinterpret_cast<uint32_t*>(r) = dmw;   // (records are 4-byte aligned: the caller aligns `plain`, and 4 + 4n is a multiple of 4)
            for (int p = 0; p < 4 * bits; ++p) r[4 + p] = rs[18 + b * 4 * bits + p];
        }
        side[idx] = e;
    } else {
        const SbEntry e = side[idx];
        rs[0] = e.D & 0xff; rs[1] = e.D >> 8; rs[2] = e.Dm & 0xff; rs[3] = e.Dm >> 8; rs[4] = e.Mn & 0xff; rs[5] = e.Mn >> 8;
        uint32_t acc[3] = {0, 0, 0};
        for (int b = 0; b < 8; ++b) {
            const uint32_t uv = (uint32_t)e.u[b] | ((uint32_t)e.v[b] << 6);
            const int bit0 = 12 * b;
            acc[bit0 >> 5] |= uv << (bit0 & 31);
            if ((bit0 & 31) > 20) acc[(bit0 >> 5) + 1] |= uv >> (32 - (bit0 & 31));
        }
        for (int p = 0; p < 12; ++p) rs[6 + p] = (acc[p >> 2] >> (8 * (p & 3))) & 0xff;
        for (int b = 0; b < 8; ++b)
            for (int p = 0; p < 4 * bits; ++p) rs[18 + b * 4 * bits + p] = rp[b * rec_pl + 4 + p];
    }
}

cudaError_t launch_pack_sb(const aq_handle_s* h, const float* W, cudaStream_t s) {
    const int64_t n_units = h->n_frags / 2;
    const unsigned grid = (unsigned)((n_units + 3) / 4);
    SbEntry* side = reinterpret_cast<SbEntry*>(h->sb);
    switch (h->bits) {
        case 2: pack_sb_kernel<2><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, n_units, h->frags, side, h->flags); break;
        case 3: pack_sb_kernel<3><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, n_units, h->frags, side, h->flags); break;
        default: pack_sb_kernel<4><<<grid, 128, 0, s>>>(W, h->N, h->K, h->NT, n_units, h->frags, side, h->flags); break;
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_sb_records(const aq_handle_s* h, uint8_t* sbcanon_dev, uint8_t* plain_dev, bool to_plain, cudaStream_t s) {
    const int64_t n = h->N * (h->K / 256);
    sb_records_kernel<<<(unsigned)((n + 127) / 128), 128, 0, s>>>(sbcanon_dev, plain_dev, reinterpret_cast<SbEntry*>(h->sb), h->bits, h->N, h->K,
                                                                    to_plain ? 1 : 0);
    count_launch();
    return cudaGetLastError();
}

}  // namespace aq
