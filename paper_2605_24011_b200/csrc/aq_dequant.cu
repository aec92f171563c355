// aq_dequant: the dequantised matrix of Eq. 1, w = scale * q + min, evaluated
// in binary32 (the product is exact, so the sum is the only rounding) and
// rounded once to the output type.
//
// Bound: HBM traffic, (bits+1)/8 bytes read + sizeof(out) bytes written per
// weight.  One warp per fragment (16 rows x 128 k): the warp reads its
// fragment with 16-byte loads, transposes the results through shared memory
// and writes whole 256/512-byte row segments.
#include "aq_internal.h"
#include "aq_layout.cuh"

namespace aq {

template <typename T> struct OutVec;   // 8 consecutive output elements
template <> struct OutVec<__half> {
    uint4 v;
    __device__ __forceinline__ void set(const float* w) {
        __half2 a = __floats2half2_rn(w[0], w[1]), b = __floats2half2_rn(w[2], w[3]);
        __half2 c = __floats2half2_rn(w[4], w[5]), d = __floats2half2_rn(w[6], w[7]);
        v = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                       *reinterpret_cast<uint32_t*>(&c), *reinterpret_cast<uint32_t*>(&d));
    }
};
template <> struct OutVec<__nv_bfloat16> {
    uint4 v;
    __device__ __forceinline__ void set(const float* w) {
        __nv_bfloat162 a = __floats2bfloat162_rn(w[0], w[1]), b = __floats2bfloat162_rn(w[2], w[3]);
        __nv_bfloat162 c = __floats2bfloat162_rn(w[4], w[5]), d = __floats2bfloat162_rn(w[6], w[7]);
        v = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                       *reinterpret_cast<uint32_t*>(&c), *reinterpret_cast<uint32_t*>(&d));
    }
};

// lane (g,t): 8 decoded values of block j, row half hi
template <int BITS>
__device__ __forceinline__ void decode_unit(const LaneCodes<BITS>& lc, const uint8_t* fb, int g, int j, int hi,
                                            float* w) {
    const __half2 dm = *reinterpret_cast<const __half2*>(fb + ((g + 8 * hi) * 4 + j) * 4);
    const float d = __low2float(dm), m = __high2float(dm);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // the two codes as floats without a conversion: 2^23 + q has q in its low mantissa bits, and
        // (2^23 + q) - 2^23 is exact, so the value is the same as (float)q
        const uint32_t p = code_pair<BITS>(lc, j, hi, i, 0u);
        const float q0 = __uint_as_float((p & 0xffffu) | 0x4B000000u) - 8388608.f;
        const float q1 = __uint_as_float(__byte_perm(p, 0x4B000000u, 0x7632)) - 8388608.f;
        w[2 * i] = fmaf(d, q0, m);
        w[2 * i + 1] = fmaf(d, q1, m);
    }
}

template <int BITS, typename T>
__global__ void __launch_bounds__(256) dequant_kernel(const uint8_t* __restrict__ frags, int64_t N, int64_t K, int NT,
                                                      int64_t n_frags, T* __restrict__ out) {
    constexpr int FB = frag_bytes(BITS);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t f = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (f >= n_frags) return;
    const int par = (int)(f & 1);
    const int64_t u = f >> 1;
    const int64_t R = u % NT;
    const int64_t S = 2 * (u / NT) + par;
    const uint8_t* fb = frags + f * FB;
    LaneCodes<BITS> lc;
    load_lane_codes<BITS>(lc, fb, lane);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            float w[8];
            decode_unit<BITS>(lc, fb, g, j, hi, w);
            const int64_t row = R * 16 + g + 8 * hi;
            const int64_t k0 = S * 128 + 32 * j + 8 * t;
            if (row < N && k0 < K) {
                if constexpr (sizeof(T) == 4) {
                    float4* o = reinterpret_cast<float4*>(out + row * K + k0);
                    o[0] = make_float4(w[0], w[1], w[2], w[3]);
                    o[1] = make_float4(w[4], w[5], w[6], w[7]);
                } else {
                    OutVec<T> ov;
                    ov.set(w);
                    *reinterpret_cast<uint4*>(out + row * K + k0) = ov.v;
                }
            }
        }
    }
}

template <int BITS>
static cudaError_t launch_bits(const aq_handle_s* h, void* out, aq_dtype_t dt, cudaStream_t s) {
    const unsigned grid = (unsigned)((h->n_frags + 7) / 8);
    if (dt == AQ_F16)
        dequant_kernel<BITS, __half><<<grid, 256, 0, s>>>(h->frags, h->N, h->K, h->NT, h->n_frags, (__half*)out);
    else if (dt == AQ_BF16)
        dequant_kernel<BITS, __nv_bfloat16><<<grid, 256, 0, s>>>(h->frags, h->N, h->K, h->NT, h->n_frags, (__nv_bfloat16*)out);
    else
        dequant_kernel<BITS, float><<<grid, 256, 0, s>>>(h->frags, h->N, h->K, h->NT, h->n_frags, (float*)out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dequant(const aq_handle_s* h, void* out, aq_dtype_t dt, cudaStream_t s) {
    switch (h->bits) {
        case 2: return launch_bits<2>(h, out, dt, s);
        case 3: return launch_bits<3>(h, out, dt, s);
        default: return launch_bits<4>(h, out, dt, s);
    }
}

}  // namespace aq
