// aq_stack_forward: a program of linears over packed weights with the glue
// between them (Section 3: the matrices of a transformer block; Section 4.3:
// every quantised matmul of the deployed graph runs as a low-bit kernel).
//
// Activations are float32 buffers in the caller's workspace.  Consecutive ops
// that consume the same input vector form a phase; per phase the input is
// formed once (RMS scaling / SiLU*up / plain) and rounded to the activation
// dtype, then each op of the phase accumulates W x into its output buffer.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <vector>

#include "aq_internal.h"

namespace aq {

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static inline bool same_input(const aq_stack_op_t& a, const aq_stack_op_t& b) {
    return a.src == b.src && a.in_op == b.in_op && (a.in_op != AQ_IN_SILU_MUL || a.src2 == b.src2);
}

static bool plan_stack(const aq_stack_t* p, int M, StackPlan& plan) {
    if (!p || !p->ops || !p->buf_width || p->n_ops < 1 || p->n_bufs < 2 || M < 1 || M > AQ_MAX_M) return false;
    plan.buf_off.resize(p->n_bufs);
    size_t off = 0;
    int64_t maxw = 0;
    for (int b = 0; b < p->n_bufs; ++b) {
        if (p->buf_width[b] < 1) return false;
        plan.buf_off[b] = off;
        off += align_up((size_t)M * p->buf_width[b] * sizeof(float), 256);
        if (p->buf_width[b] > maxw) maxw = p->buf_width[b];
    }
    plan.stage_off = off;
    // A buffer that no op writes is an input of the program: buffer 0 is filled from x0, any other one by whoever runs
    // between the ops (the attention of aq_stack_forward_attn) or by the caller, as float32 in the workspace.
    std::vector<char> written(p->n_bufs, 1);
    for (int i = 0; i < p->n_ops; ++i)
        if (p->ops[i].dst >= 1 && p->ops[i].dst < p->n_bufs) written[p->ops[i].dst] = 0;
    plan.external.assign(written.begin(), written.end());
    plan.external[0] = 0;
    for (int i = 0; i < p->n_ops; ++i) {
        const aq_stack_op_t& o = p->ops[i];
        if (!handle_ok(o.w)) return false;
        if (o.src < 0 || o.src >= p->n_bufs || o.dst < 1 || o.dst >= p->n_bufs) return false;
        if (!written[o.src] || written[o.dst]) return false;
        if (o.in_op < AQ_IN_PLAIN || o.in_op > AQ_IN_SILU_MUL || o.out_op < AQ_OUT_STORE || o.out_op > AQ_OUT_ADD) return false;
        if (o.in_op == AQ_IN_SILU_MUL) {
            if (o.src2 < 0 || o.src2 >= p->n_bufs || !written[o.src2] || p->buf_width[o.src2] != p->buf_width[o.src]) return false;
        }
        if (o.out_op == AQ_OUT_ADD) {
            if (o.res < 0 || o.res >= p->n_bufs || !written[o.res] || p->buf_width[o.res] != p->buf_width[o.dst]) return false;
        }
        if (o.w->K != p->buf_width[o.src] || o.w->N != p->buf_width[o.dst]) return false;
        written[o.dst] = 1;
    }
    plan.in_off.resize(p->n_ops);
    for (int i = 0; i < p->n_ops; ++i) {
        if (i > 0 && same_input(p->ops[i], p->ops[i - 1])) { plan.in_off[i] = plan.in_off[i - 1]; continue; }
        plan.phase_first.push_back(i);
        plan.in_off[i] = off;
        off += align_up((size_t)M * p->buf_width[p->ops[i].src] * 2, 256);
    }
    if (M > AQ_DECODE_MAX_M) {   // bfloat16 activations reach the tensor cores as binary16: a second staged vector per phase
        plan.x16_off.assign(p->n_ops, 0);
        plan.rs_off.assign(p->n_ops, 0);
        plan.flag_off.assign(p->n_ops, 0);
        plan.flags_begin = off;          // one int per phase, together: a single memset clears them
        off += align_up((size_t)p->n_ops * sizeof(int), 256);
        plan.flags_end = off;
        for (int i = 0; i < p->n_ops; ++i) {
            if (i > 0 && same_input(p->ops[i], p->ops[i - 1])) {
                plan.x16_off[i] = plan.x16_off[i - 1]; plan.rs_off[i] = plan.rs_off[i - 1]; plan.flag_off[i] = plan.flag_off[i - 1];
                continue;
            }
            plan.flag_off[i] = plan.flags_begin + (size_t)i * sizeof(int);
            plan.x16_off[i] = off;
            off += align_up((size_t)M * p->buf_width[p->ops[i].src] * 2, 256);
            plan.rs_off[i] = off;
            off += align_up((size_t)M * sizeof(float), 256);
        }
    }
    if (M <= AQ_DECODE_MAX_M) {   // the whole-program decode kernel accumulates packed 64-bit sums, one per element
        plan.pk_off.assign(p->n_bufs, 0);
        plan.pk_begin = off;
        for (int b = 1; b < p->n_bufs; ++b) {
            plan.pk_off[b] = off;
            off += align_up((size_t)M * p->buf_width[b] * 8, 256);
        }
        plan.nm_off.assign(p->n_ops, 0);
        for (int i = 0; i < p->n_ops && M >= 3; ++i) {
            if (p->ops[i].in_op != AQ_IN_RMSNORM || (i > 0 && same_input(p->ops[i], p->ops[i - 1]))) continue;
            plan.nm_off[i] = off;
            off += align_up((size_t)AQ_NORM_MAX_CTAS * M * 8, 256);
        }
        plan.pk_end = off;
    }
    plan.total = off;
    (void)maxw;
    return true;
}

// ---- glue kernels ----------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void widen_kernel(const T* __restrict__ x, float* __restrict__ out, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = to_f32<T>(x[i]);
}

template <typename T>
__global__ void narrow_kernel(const float* __restrict__ x, T* __restrict__ out, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = from_f32<T>(x[i]);
}

// Rounds four values and stores them as one 8-byte word.
template <typename T>
__device__ __forceinline__ void store_round4(T* o, const float4& v) {
    const T a = from_f32<T>(v.x), b = from_f32<T>(v.y), c = from_f32<T>(v.z), d = from_f32<T>(v.w);
    uint2 r;
    r.x = (uint32_t)*reinterpret_cast<const uint16_t*>(&a) | ((uint32_t)*reinterpret_cast<const uint16_t*>(&b) << 16);
    r.y = (uint32_t)*reinterpret_cast<const uint16_t*>(&c) | ((uint32_t)*reinterpret_cast<const uint16_t*>(&d) << 16);
    *reinterpret_cast<uint2*>(o) = r;
}

// x[m][k] = round(transform(src[m][k])); K is a multiple of 32, rows are 16-byte aligned.
// RMS scaling: one CTA per token row.  The other two forms have no row-wide term and
// run as a flat grid over groups of four elements (blockIdx.y = 0).
// Outputs the linears of a phase will add into: dst = src (the residual) or zero, n4 groups of four floats each.
struct PresetList {
    float4* dst[8];
    const float4* src[8];
    int64_t n4[8];
    int n;
};

template <typename T>
__global__ void __launch_bounds__(256) stage_kernel(const float* __restrict__ src, const float* __restrict__ src2,
                                                    int in_op, int64_t K, int64_t total4, T* __restrict__ x,
                                                    const PresetList pre) {
    pdl_wait();                 // the buffers read and preset here belong to the kernels before this one
    pdl_launch_dependents();    // the linears of this phase may set themselves up meanwhile
    for (int q = 0; q < pre.n; ++q) {
        float4* d = pre.dst[q];
        const float4* r = pre.src[q];
        for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < pre.n4[q]; i += (int64_t)gridDim.x * 256)
            d[i] = r ? r[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (in_op != AQ_IN_RMSNORM) {
        const float4* s4 = reinterpret_cast<const float4*>(src);
        const float4* t4 = reinterpret_cast<const float4*>(src2);
        for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total4; i += (int64_t)gridDim.x * 256) {
            float4 v = s4[i];
            if (in_op == AQ_IN_SILU_MUL) {
                const float4 u = t4[i];
                v.x = v.x / (1.f + expf(-v.x)) * u.x; v.y = v.y / (1.f + expf(-v.y)) * u.y;
                v.z = v.z / (1.f + expf(-v.z)) * u.z; v.w = v.w / (1.f + expf(-v.w)) * u.w;
            }
            store_round4<T>(x + 4 * i, v);
        }
        return;
    }
    const int64_t m = blockIdx.x;
    const float4* s4 = reinterpret_cast<const float4*>(src + m * K);
    T* o = x + m * K;
    const int64_t q4 = K >> 2;
    __shared__ float red[8];
    float ss = 0.f;
    for (int64_t k = threadIdx.x; k < q4; k += 256) {
        const float4 v = s4[k];
        ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += red[i];
    const float scale = rsqrtf(tot / (float)K + 1e-6f);
    for (int64_t k = threadIdx.x; k < q4; k += 256) {
        const float4 v = s4[k];
        store_round4<T>(o + 4 * k, make_float4(v.x * scale, v.y * scale, v.z * scale, v.w * scale));
    }
}

// The same for bfloat16 activations on the tensor-core path, one CTA per token row: besides the rounded vector x
// (kept for the caller) it writes the binary16 copy x16 the GEMM reads -- exact wherever a bfloat16 value lies
// inside binary16's range; a row with a magnitude of 2^15 or more is divided by the power of two that brings its
// largest one below 2^15, kept in scale[m] (1 otherwise) and undone by the GEMM's epilogue; *flag is raised then.
// The flag must be zero when the kernel starts.
__global__ void __launch_bounds__(256) stage_rows_bf16_kernel(const float* __restrict__ src, const float* __restrict__ src2, int in_op,
                                                              int64_t K, __nv_bfloat16* __restrict__ x, __half* __restrict__ x16,
                                                              float* __restrict__ scale, int* __restrict__ flag, const PresetList pre) {
    pdl_wait();
    pdl_launch_dependents();
    for (int q = 0; q < pre.n; ++q) {
        float4* d = pre.dst[q];
        const float4* r = pre.src[q];
        for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < pre.n4[q]; i += (int64_t)gridDim.x * 256)
            d[i] = r ? r[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int64_t m = blockIdx.x;
    const float4* s4 = reinterpret_cast<const float4*>(src + m * K);
    const float4* t4 = src2 ? reinterpret_cast<const float4*>(src2 + m * K) : nullptr;
    __nv_bfloat16* xr = x + m * K;
    __half* hr = x16 + m * K;
    const int64_t q4 = K >> 2;
    __shared__ float red[8];
    float rms = 1.f;
    if (in_op == AQ_IN_RMSNORM) {
        float ss = 0.f;
        for (int64_t k = threadIdx.x; k < q4; k += 256) {
            const float4 v = s4[k];
            ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += red[i];
        rms = rsqrtf(tot / (float)K + 1e-6f);
        __syncthreads();
    }
    // the rounded vector, its binary16 copy as if no scaling were needed, and the row's largest magnitude
    float mx = 0.f;
    for (int64_t k = threadIdx.x; k < q4; k += 256) {
        float4 v = s4[k];
        if (in_op == AQ_IN_SILU_MUL) {
            const float4 u = t4[k];
            v.x = v.x / (1.f + expf(-v.x)) * u.x; v.y = v.y / (1.f + expf(-v.y)) * u.y;
            v.z = v.z / (1.f + expf(-v.z)) * u.z; v.w = v.w / (1.f + expf(-v.w)) * u.w;
        } else {
            v.x *= rms; v.y *= rms; v.z *= rms; v.w *= rms;
        }
        const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
        uint2 r;
        r.x = *reinterpret_cast<const uint32_t*>(&a); r.y = *reinterpret_cast<const uint32_t*>(&b);
        *reinterpret_cast<uint2*>(xr + 4 * k) = r;
        const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        const __half2 ha = __floats2half2_rn(fa.x, fa.y), hb = __floats2half2_rn(fb.x, fb.y);
        uint2 h;
        h.x = *reinterpret_cast<const uint32_t*>(&ha); h.y = *reinterpret_cast<const uint32_t*>(&hb);
        *reinterpret_cast<uint2*>(hr + 4 * k) = h;
        mx = fmaxf(mx, fmaxf(fmaxf(fabsf(fa.x), fabsf(fa.y)), fmaxf(fabsf(fb.x), fabsf(fb.y))));
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();   // (also: this CTA's writes of x are visible to its own threads below)
    mx = red[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, red[i]);
    float sc = 1.f;
    if (mx >= 32768.f && mx <= 3.0e38f) {
        int e;
        frexpf(mx, &e);
        sc = ldexpf(1.f, e - 15);
        const float inv = 1.f / sc;
        for (int64_t k = threadIdx.x; k < q4; k += 256) {
            const uint2 r = *reinterpret_cast<const uint2*>(xr + 4 * k);
            const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r.x));
            const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r.y));
            const __half2 ha = __floats2half2_rn(fa.x * inv, fa.y * inv), hb = __floats2half2_rn(fb.x * inv, fb.y * inv);
            uint2 h;
            h.x = *reinterpret_cast<const uint32_t*>(&ha); h.y = *reinterpret_cast<const uint32_t*>(&hb);
            *reinterpret_cast<uint2*>(hr + 4 * k) = h;
        }
        if (threadIdx.x == 0) *flag = 1;
    }
    if (threadIdx.x == 0) scale[m] = sc;
}

template <typename T>
static cudaError_t run_stack(const aq_stack_t* p, const StackPlan& plan, const T* x0, T* out, int out_buf, int M,
                             aq_dtype_t dt, uint8_t* ws, cudaStream_t s) {
    cudaError_t e = cudaSuccess;
    const bool decode = (M <= AQ_DECODE_MAX_M);
    auto buf = [&](int b) { return reinterpret_cast<float*>(ws + plan.buf_off[b]); };
    {
        const int64_t n = (int64_t)M * p->buf_width[0];
        widen_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(x0, buf(0), n);
        count_launch();
    }
    if (!decode && dt == AQ_BF16) {   // the "a row was scaled" flags of all phases start at zero
        e = cudaMemsetAsync(ws + plan.flags_begin, 0, plan.flags_end - plan.flags_begin, s);
        if (e != cudaSuccess) return e;
    }
    if (decode) {   // one persistent kernel for the whole program, when it fits
        bool wrote_out = false;
        const int r = launch_decode_stack(p, plan, M, dt, ws, s, &e, out, out_buf, &wrote_out);
        if (r < 0) return e;
        if (r == 0) {
            for (int k = 0; k < p->n_ops; ++k) p->ops[k].w->last_stream = s;
        }
        if (r == 0 && out && !wrote_out) {
            const int64_t n = (int64_t)M * p->buf_width[out_buf];
            narrow_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(buf(out_buf), out, n);
            count_launch();
        }
        if (r == 0) return cudaGetLastError();
        // op by op: the streaming kernel accumulates with red.add, so every output starts at zero (inputs that somebody
        // else has filled are left alone: runs of buffers between them are cleared)
        for (int b = 1; b < p->n_bufs;) {
            if (plan.external[b]) { ++b; continue; }
            int b1 = b;
            while (b1 + 1 < p->n_bufs && !plan.external[b1 + 1]) ++b1;
            const size_t end = (b1 + 1 < p->n_bufs) ? plan.buf_off[b1 + 1] : plan.stage_off;
            e = cudaMemsetAsync(ws + plan.buf_off[b], 0, end - plan.buf_off[b], s);
            if (e != cudaSuccess) return e;
            b = b1 + 1;
        }
    }
    int i = 0;
    while (i < p->n_ops) {
        const aq_stack_op_t& f = p->ops[i];
        const int64_t K = p->buf_width[f.src];
        T* stage = reinterpret_cast<T*>(ws + plan.in_off[i]);
        PresetList pre;
        pre.n = 0;
        bool preset = false;
        if (!decode) {   // the phase's outputs start as residual / zero: written here, in the same launch as x
            float* outs[8];
            int64_t ldos[8];
            int n = 0;
            bool fits = true;
            for (int q = i; q < p->n_ops && same_input(p->ops[q], f); ++q) {
                if (n == 8) { fits = false; break; }
                outs[n] = buf(p->ops[q].dst); ldos[n] = p->buf_width[p->ops[q].dst]; ++n;
            }
            if (fits && gemm_outputs_can_be_preset(outs, ldos, n)) {
                preset = true;
                // launches are made of up to AQ_GEMM_MAX_GROUP matrices: zeros are needed where such a group
                // cannot use the store-first protocol for its split tiles
                for (int q = 0; q < n; ++q) {
                    const aq_stack_op_t& o = p->ops[i + q];
                    const bool has_res = (o.out_op == AQ_OUT_ADD);
                    if (!has_res) {
                        const int g0 = q - q % AQ_GEMM_MAX_GROUP, gn = std::min(AQ_GEMM_MAX_GROUP, n - g0);
                        const aq_handle_s* hs[AQ_GEMM_MAX_GROUP];
                        for (int r = 0; r < gn; ++r) hs[r] = p->ops[i + g0 + r].w;
                        if (gemm_stores_first(hs, gn, M, s)) continue;
                    }
                    pre.dst[pre.n] = reinterpret_cast<float4*>(outs[q]);
                    pre.src[pre.n] = has_res ? reinterpret_cast<const float4*>(buf(o.res)) : nullptr;
                    pre.n4[pre.n] = (int64_t)M * ldos[q] / 4;
                    ++pre.n;
                }
            }
        }
        {
            const int64_t total4 = (int64_t)M * K / 4;
            const unsigned g = (f.in_op == AQ_IN_RMSNORM) ? (unsigned)M : (unsigned)std::min<int64_t>((total4 + 255) / 256, 4 * 148);
            const float* s2 = (f.in_op == AQ_IN_SILU_MUL) ? buf(f.src2) : nullptr;
            if (decode) stage_kernel<T><<<g, 256, 0, s>>>(buf(f.src), s2, (int)f.in_op, K, total4, stage, pre);
            else if (dt == AQ_BF16) {
                int* flag = reinterpret_cast<int*>(ws + plan.flag_off[i]);
                e = launch_pdl(stage_rows_bf16_kernel, dim3((unsigned)M), dim3(256), 0, s, (const float*)buf(f.src), s2, (int)f.in_op, K,
                               reinterpret_cast<__nv_bfloat16*>(stage), reinterpret_cast<__half*>(ws + plan.x16_off[i]),
                               reinterpret_cast<float*>(ws + plan.rs_off[i]), flag, pre);
            } else e = launch_pdl(stage_kernel<T>, dim3(g), dim3(256), 0, s, (const float*)buf(f.src), s2, (int)f.in_op, K, total4, stage, pre);
            if (e != cudaSuccess) return e;
        }
        count_launch();
        int j = i;
        while (j < p->n_ops && same_input(p->ops[j], f)) {
            if (decode) {
                const aq_stack_op_t& o = p->ops[j];
                const int64_t N = p->buf_width[o.dst];
                if (o.out_op == AQ_OUT_ADD) {
                    e = cudaMemcpyAsync(buf(o.dst), buf(o.res), (size_t)M * N * sizeof(float), cudaMemcpyDeviceToDevice, s);
                    if (e != cudaSuccess) return e;
                }
                e = launch_gemv(o.w, stage, dt, M, buf(o.dst), N, s);
                if (e != cudaSuccess) return e;
                o.w->last_stream = s;
                ++j;
            } else {   // the matrices of a phase read the same x: up to AQ_GEMM_MAX_GROUP of them per launch
                const aq_handle_s* hs[AQ_GEMM_MAX_GROUP];
                float* outs[AQ_GEMM_MAX_GROUP];
                const float* ress[AQ_GEMM_MAX_GROUP];
                int64_t ldos[AQ_GEMM_MAX_GROUP];
                int n = 0;
                while (n < AQ_GEMM_MAX_GROUP && j < p->n_ops && same_input(p->ops[j], f)) {
                    const aq_stack_op_t& o = p->ops[j];
                    hs[n] = o.w; outs[n] = buf(o.dst); ldos[n] = p->buf_width[o.dst];
                    ress[n] = (o.out_op == AQ_OUT_ADD) ? buf(o.res) : nullptr;
                    o.w->last_stream = s;
                    ++n; ++j;
                }
                if (dt == AQ_BF16)
                    e = launch_gemm_group(hs, n, ws + plan.x16_off[i], reinterpret_cast<const float*>(ws + plan.rs_off[i]),
                                          reinterpret_cast<const int*>(ws + plan.flag_off[i]), M, outs, ldos, ress,
                                          preset, s);
                else e = launch_gemm_group(hs, n, stage, nullptr, nullptr, M, outs, ldos, ress, preset, s);
                if (e != cudaSuccess) return e;
            }
        }
        i = j;
    }
    if (out) {
        const int64_t n = (int64_t)M * p->buf_width[out_buf];
        narrow_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(buf(out_buf), out, n);
        count_launch();
    }
    return cudaGetLastError();
}

}  // namespace aq

using namespace aq;

extern "C" {

size_t aq_stack_workspace_bytes(const aq_stack_t* prog, int M) {
    StackPlan plan;
    if (!plan_stack(prog, M, plan)) return 0;
    return plan.total;
}

size_t aq_stack_buffer_offset(const aq_stack_t* prog, int M, int b) {
    StackPlan plan;
    if (!plan_stack(prog, M, plan) || b < 0 || b >= prog->n_bufs) return (size_t)-1;
    return plan.buf_off[b];
}

size_t aq_stack_input_offset(const aq_stack_t* prog, int M, int op) {
    StackPlan plan;
    if (!plan_stack(prog, M, plan) || op < 0 || op >= prog->n_ops) return (size_t)-1;
    return plan.in_off[op];
}

aq_status_t aq_stack_forward(const aq_stack_t* prog, const void* x0_dev, void* out_dev, int out_buf, int M,
                             aq_dtype_t dtype, void* workspace_dev, size_t ws_bytes, aq_stream_t stream) {
    StackPlan plan;
    if (!plan_stack(prog, M, plan)) return AQ_ERR_INVALID_ARG;
    if (!x0_dev || !workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) ||
        (reinterpret_cast<uintptr_t>(x0_dev) & 15u) || (reinterpret_cast<uintptr_t>(out_dev) & 15u))
        return AQ_ERR_INVALID_ARG;
    if (ws_bytes < plan.total) return AQ_ERR_INVALID_ARG;
    if (out_dev && (out_buf < 0 || out_buf >= prog->n_bufs)) return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16) return (dtype == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (dtype == AQ_F16)
        e = run_stack<__half>(prog, plan, (const __half*)x0_dev, (__half*)out_dev, out_buf, M, dtype, (uint8_t*)workspace_dev, s);
    else
        e = run_stack<__nv_bfloat16>(prog, plan, (const __nv_bfloat16*)x0_dev, (__nv_bfloat16*)out_dev, out_buf, M, dtype,
                                     (uint8_t*)workspace_dev, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return AQ_OK;
}

size_t aq_stack_attn_scratch_bytes(int n_heads, int n_kv_heads, int M) {
    if (n_heads < 1 || n_kv_heads < 1 || n_kv_heads > 64 || M < 1 || M > AQ_DECODE_MAX_M) return 0;
    return align_up((size_t)M * n_heads * 128 * 2, 256) + attn_scratch_bytes(n_kv_heads);
}

aq_status_t aq_stack_forward_attn(const aq_stack_t* prog, const aq_stack_attn_t* attn, int n_attn, int64_t pos, float theta,
                                  const void* x0_dev, void* out_dev, int out_buf, int M, aq_dtype_t dtype, void* workspace_dev,
                                  size_t ws_bytes, void* attn_scratch_dev, size_t attn_scratch_bytes_given, aq_stream_t stream) {
    StackPlan plan;
    if (!plan_stack(prog, M, plan)) return AQ_ERR_INVALID_ARG;
    if (!x0_dev || !workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) ||
        (reinterpret_cast<uintptr_t>(x0_dev) & 15u) || (reinterpret_cast<uintptr_t>(out_dev) & 15u))
        return AQ_ERR_INVALID_ARG;
    if (ws_bytes < plan.total || n_attn < 0 || (n_attn > 0 && !attn) || pos < 0 || !(theta > 1.f)) return AQ_ERR_INVALID_ARG;
    if (out_dev && (out_buf < 0 || out_buf >= prog->n_bufs)) return AQ_ERR_INVALID_ARG;
    if (dtype != AQ_F16 && dtype != AQ_BF16) return (dtype == AQ_F32) ? AQ_ERR_UNSUPPORTED : AQ_ERR_INVALID_ARG;
    if (M > AQ_DECODE_MAX_M) return AQ_ERR_UNSUPPORTED;
    size_t need = 0;
    int prev = -1;
    for (int i = 0; i < n_attn; ++i) {
        const aq_stack_attn_t& t = attn[i];
        auto buf_ok = [&](int b, int64_t w) { return b >= 1 && b < prog->n_bufs && prog->buf_width[b] == w; };
        if (t.after_op <= prev || t.after_op >= prog->n_ops || t.n_heads < 1 || t.n_kv_heads < 1 || t.n_heads % t.n_kv_heads != 0 ||
            !buf_ok(t.q_buf, (int64_t)t.n_heads * 128) || !buf_ok(t.k_buf, (int64_t)t.n_kv_heads * 128) ||
            !buf_ok(t.v_buf, (int64_t)t.n_kv_heads * 128) || !buf_ok(t.dst_buf, (int64_t)t.n_heads * 128) || !plan.external[t.dst_buf] ||
            !t.k_cache_dev || !t.v_cache_dev || (reinterpret_cast<uintptr_t>(t.k_cache_dev) & 15u) ||
            (reinterpret_cast<uintptr_t>(t.v_cache_dev) & 15u) || pos + M > t.L_max || t.L_max > ((int64_t)1 << 31))
            return AQ_ERR_INVALID_ARG;
        // q, k, v come from ops at or before after_op, and the next op opens a phase (a launch ends where a phase ends)
        bool qw = false, kw = false, vw = false;
        for (int o = 0; o <= t.after_op; ++o) {
            qw |= prog->ops[o].dst == t.q_buf; kw |= prog->ops[o].dst == t.k_buf; vw |= prog->ops[o].dst == t.v_buf;
        }
        if (!qw || !kw || !vw) return AQ_ERR_INVALID_ARG;
        if (t.after_op + 1 < prog->n_ops && same_input(prog->ops[t.after_op + 1], prog->ops[t.after_op])) return AQ_ERR_INVALID_ARG;
        if ((int64_t)(t.n_heads / t.n_kv_heads) * M > 16 || t.n_kv_heads > 64) return AQ_ERR_UNSUPPORTED;
        need = std::max(need, aq_stack_attn_scratch_bytes(t.n_heads, t.n_kv_heads, M));
        prev = t.after_op;
    }
    if (n_attn > 0 && (!attn_scratch_dev || (reinterpret_cast<uintptr_t>(attn_scratch_dev) & 255u) || attn_scratch_bytes_given < need))
        return AQ_ERR_INVALID_ARG;
    {
        int dev = 0, major = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return cuda_fail(cudaGetLastError());
        if (major != 10) return AQ_ERR_ARCH;
    }
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace_dev);
    auto buf = [&](int b) { return reinterpret_cast<float*>(ws + plan.buf_off[b]); };
    cudaError_t e = cudaSuccess;
    {
        const int64_t n = (int64_t)M * prog->buf_width[0];
        if (dtype == AQ_F16) widen_kernel<__half><<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const __half*)x0_dev, buf(0), n);
        else widen_kernel<__nv_bfloat16><<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const __nv_bfloat16*)x0_dev, buf(0), n);
        count_launch();
    }
    int first = 0;
    bool wrote_out = false;
    std::vector<uint8_t> program_key;
    decode_program_key(prog, program_key);
    for (int i = 0; i <= n_attn; ++i) {
        const int end = (i < n_attn) ? attn[i].after_op + 1 : prog->n_ops;
        if (end > first) {
            bool w = false;
            const int r = launch_decode_stack(prog, plan, M, dtype, ws, s, &e, (i == n_attn) ? out_dev : nullptr, out_buf, &w, first, end,
                                              first == 0, &program_key);
            if (r < 0) return cuda_fail(e);
            if (r > 0) return AQ_ERR_UNSUPPORTED;
            wrote_out = wrote_out || w;
        }
        first = end;
        if (i == n_attn) break;
        const aq_stack_attn_t& t = attn[i];
        uint8_t* sc = reinterpret_cast<uint8_t*>(attn_scratch_dev);
        void* q16 = sc;
        void* asc = sc + align_up((size_t)M * t.n_heads * 128 * 2, 256);
        e = launch_attn_prepare(buf(t.q_buf), buf(t.k_buf), buf(t.v_buf), q16, t.k_cache_dev, t.v_cache_dev, M, t.n_heads, t.n_kv_heads, pos,
                                t.L_max, theta, dtype, s);
        if (e == cudaSuccess)
            e = launch_attn_decode(q16, t.k_cache_dev, t.v_cache_dev, buf(t.dst_buf), M, t.n_heads, t.n_kv_heads, pos + M, t.L_max,
                                   0.08838834764831845f, dtype, AQ_F32, asc, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    for (int k = 0; k < prog->n_ops; ++k) prog->ops[k].w->last_stream = s;
    if (out_dev && !wrote_out) {
        const int64_t n = (int64_t)M * prog->buf_width[out_buf];
        if (dtype == AQ_F16) narrow_kernel<__half><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(buf(out_buf), (__half*)out_dev, n);
        else narrow_kernel<__nv_bfloat16><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(buf(out_buf), (__nv_bfloat16*)out_dev, n);
        count_launch();
    }
    e = cudaGetLastError();
    return e == cudaSuccess ? AQ_OK : cuda_fail(e);
}

}  // extern "C"
