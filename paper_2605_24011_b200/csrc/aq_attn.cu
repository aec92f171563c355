// Single-token attention over a key/value cache, rotary embedding and cache append: what sits between the attention
// projections W_Q, W_K, W_V and W_O of a decoder block (Section 2, "Vision-Language-Action models", names the
// projections; the operation between them is the textbook scaled-dot-product attention, which the paper does not restate).
//
// Bound: HBM.  One decoded token reads every cached key and value once: 2 * L * Hkv * D * 2 bytes.  Caches are
// head-major, [Hkv][Lmax][D] of the activation type, so the rows one CTA reads are contiguous.
//
// attn_decode_kernel: grid = (key/value head, split of the positions).  Each of a CTA's four warps streams tiles of 32
// positions (8 KB of keys + 8 KB of values) through its own three-stage cp.async ring (the 16-byte chunks of a row are
// XOR-swizzled by the row, so ldmatrix reads without bank conflicts) and runs the usual online softmax on tensor
// cores: S = Q K^T with the query heads that share the key/value head as the 16 rows of mma.sync.m16n8k16 (unused rows
// are zero), P = exp2(S - max) straight from the accumulator registers into the A operand of O += P V.  The warps'
// running (max, sum, O) are merged in shared memory, each CTA writes one partial per split, and the last CTA of a head to
// arrive (a ticket after a fence; nobody waits) merges the splits and writes the output.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "aq_internal.h"
#include "aq_per_device.h"

namespace aq {

constexpr int AT_D = 128;        // head dimension
constexpr int AT_TILE = 32;      // positions per warp tile
constexpr int AT_WARPS = 4;
constexpr int AT_STAGES = 3;
constexpr int AT_ROW_BYTES = AT_D * 2;
constexpr int AT_TILE_BYTES = AT_TILE * AT_ROW_BYTES;                  // 8 KB
constexpr int AT_SMEM = AT_WARPS * AT_STAGES * 2 * AT_TILE_BYTES;      // 192 KB
constexpr int AT_MAX_SPLITS = 64;

// One ticket per key/value head: zero when the module is loaded, and put back to zero by the CTA that takes the last
// one, so no launch has to clear them.  Shared by every call on the device: calls must not overlap (one stream at a time).
__device__ unsigned int g_attn_tickets[64];

struct AttnArgs {
    const void* q;          // [M][H][D]
    const void* kc;         // [Hkv][Lmax][D]
    const void* vc;
    void* out;              // [M][H][D]
    float* ml;              // [Hkv][splits][16][2]: running maximum (log2 domain) and sum
    float* part;            // [Hkv][splits][16][D]: unnormalised output
    int64_t L, Lmax;
    int G;                  // query heads per key/value head
    int M;                  // new tokens (the last M of the L positions are theirs); G * M <= 16 rows
    int H;                  // query heads in all (row pitch of q and out)
    int chunk;              // positions per split (a multiple of AT_TILE)
    int out_dtype;          // aq_dtype_t of out
    float scale_log2;       // scale * log2(e)
};

__device__ __forceinline__ void at_cp16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void at_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void at_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void at_ldm4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void at_ldm4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
template <bool BF16>
__device__ __forceinline__ void at_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if constexpr (BF16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <bool BF16>
__device__ __forceinline__ uint32_t at_pack(float lo, float hi) {
    if constexpr (BF16) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    } else {
        const __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
}

template <bool BF16>
__global__ void __launch_bounds__(AT_WARPS * 32, 1) attn_decode_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int hk = blockIdx.x, sp = blockIdx.y, n_sp = gridDim.y;
    const int64_t p0 = (int64_t)sp * a.chunk;
    const int64_t p1 = min(a.L, p0 + (int64_t)a.chunk);
    const int n_tiles = (int)((p1 - p0 + AT_TILE - 1) / AT_TILE);          // of the CTA; warp w takes tiles w, w + 4, ...
    const int my_tiles = (n_tiles - warp + AT_WARPS - 1) / AT_WARPS;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem) + (uint32_t)warp * AT_STAGES * 2 * AT_TILE_BYTES;
    const uint8_t* kc = reinterpret_cast<const uint8_t*>(a.kc) + (int64_t)hk * a.Lmax * AT_ROW_BYTES;
    const uint8_t* vc = reinterpret_cast<const uint8_t*>(a.vc) + (int64_t)hk * a.Lmax * AT_ROW_BYTES;

    // copies tile j of this warp (positions pt .. pt + 31) into stage s; rows at or past L are filled with zeros
    auto issue = [&](int j, int s) {
        const int64_t pt = p0 + (int64_t)(warp + AT_WARPS * j) * AT_TILE;
        const int valid = (int)min((int64_t)AT_TILE, a.L - pt);
        const uint32_t dk = ring + (uint32_t)s * 2 * AT_TILE_BYTES, dv = dk + AT_TILE_BYTES;
        const uint8_t* sk = kc + pt * AT_ROW_BYTES;
        const uint8_t* sv = vc + pt * AT_ROW_BYTES;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int idx = i * 32 + lane, row = idx >> 4, c = idx & 15;
            const uint32_t bytes = row < valid ? 16u : 0u;
            const int srow = min(row, valid - 1);
            const uint32_t off = (uint32_t)row * AT_ROW_BYTES + (uint32_t)((c ^ (row & 7)) << 4);
            at_cp16(dk + off, sk + (int64_t)srow * AT_ROW_BYTES + c * 16, bytes);
            at_cp16(dv + off, sv + (int64_t)srow * AT_ROW_BYTES + c * 16, bytes);
        }
    };

    float o[AT_D / 8][4];
#pragma unroll
    for (int nd = 0; nd < AT_D / 8; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g and g + 8: running maximum (log2 domain), sum

    // Launched as a programmatic dependent: the kernel before this one on the stream (the one that rotates q and
    // appends the new rows, when a stack program runs) may still be at work.  Only the last M rows of the cache and q can
    // be its output: a CTA whose positions include those rows waits for it before its first copy, the others start
    // their copies of older rows at once and wait before they read q (and before they write anything).
    const bool has_new_rows = p1 > a.L - a.M;
    if (has_new_rows) pdl_wait();
#pragma unroll
    for (int s = 0; s < AT_STAGES - 1; ++s) {
        if (s < my_tiles) issue(s, s);
        at_commit();
    }
    if (!has_new_rows) pdl_wait();
    // (while the first tiles are on their way) the query heads of this key/value head as the A operand: row r = head
    // hk G + r, rows >= G are zero
    // row r = token r / G, head hk G + r % G of that token; rows >= G M are zero
    const int R = a.G * a.M;
    const int tok0 = g / a.G, tok1 = (g + 8) / a.G;
    uint32_t qf[AT_D / 16][4];
    {
        const uint16_t* q = reinterpret_cast<const uint16_t*>(a.q);
        const uint16_t* q0 = q + ((int64_t)tok0 * a.H + (int64_t)hk * a.G + (g - tok0 * a.G)) * AT_D;
        const uint16_t* q1 = q + ((int64_t)tok1 * a.H + (int64_t)hk * a.G + (g + 8 - tok1 * a.G)) * AT_D;
#pragma unroll
        for (int ks = 0; ks < AT_D / 16; ++ks) {
            const int d0 = 16 * ks + 2 * t;
            qf[ks][0] = g < R ? *reinterpret_cast<const uint32_t*>(q0 + d0) : 0u;
            qf[ks][1] = g + 8 < R ? *reinterpret_cast<const uint32_t*>(q1 + d0) : 0u;
            qf[ks][2] = g < R ? *reinterpret_cast<const uint32_t*>(q0 + d0 + 8) : 0u;
            qf[ks][3] = g + 8 < R ? *reinterpret_cast<const uint32_t*>(q1 + d0 + 8) : 0u;
        }
    }
    // a token sees the positions up to its own: token m of M up to L - M + m (rows past the last one: any limit will do)
    const int64_t lim0 = a.L - (a.M - 1 - min(tok0, a.M - 1)), lim1 = a.L - (a.M - 1 - min(tok1, a.M - 1));
    for (int j = 0; j < my_tiles; ++j) {
        at_wait<AT_STAGES - 2>();
        __syncwarp();   // every lane's copies of tile j have landed, and every lane is through with tile j - 1
        if (j + AT_STAGES - 1 < my_tiles) issue(j + AT_STAGES - 1, (j + AT_STAGES - 1) % AT_STAGES);
        at_commit();
        const uint32_t kt = ring + (uint32_t)(j % AT_STAGES) * 2 * AT_TILE_BYTES, vt = kt + AT_TILE_BYTES;
        const int64_t pt = p0 + (int64_t)(warp + AT_WARPS * j) * AT_TILE;

        // S = Q K^T: 16 x 32
        float sc[4][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int row = 8 * nt + (lane & 7), chunk = 4 * kp + (lane >> 3);
                uint32_t r[4];
                at_ldm4(kt + (uint32_t)row * AT_ROW_BYTES + (uint32_t)((chunk ^ (row & 7)) << 4), r);
                at_mma<BF16>(sc[nt], qf[2 * kp], r[0], r[1]);
                at_mma<BF16>(sc[nt], qf[2 * kp + 1], r[2], r[3]);
            }
        }
        // scale, mask the positions past L, running maximum
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int64_t pc = pt + 8 * nt + 2 * t;
            sc[nt][0] = pc < lim0 ? sc[nt][0] * a.scale_log2 : -INFINITY;
            sc[nt][1] = pc + 1 < lim0 ? sc[nt][1] * a.scale_log2 : -INFINITY;
            sc[nt][2] = pc < lim1 ? sc[nt][2] * a.scale_log2 : -INFINITY;
            sc[nt][3] = pc + 1 < lim1 ? sc[nt][3] * a.scale_log2 : -INFINITY;
            mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
            mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // (a row that has seen nothing yet, its limit lying before this warp's first tiles, keeps -inf: the exponentials
        // below are then taken against 0 and come out as 0)
        const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
        const float b0 = n0 == -INFINITY ? 0.f : n0, b1 = n1 == -INFINITY ? 0.f : n1;
        const float a0 = exp2f(m0 - b0), a1 = exp2f(m1 - b1);
        m0 = n0; m1 = n1;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            sc[nt][0] = exp2f(sc[nt][0] - b0); sc[nt][1] = exp2f(sc[nt][1] - b0);
            sc[nt][2] = exp2f(sc[nt][2] - b1); sc[nt][3] = exp2f(sc[nt][3] - b1);
            s0 += sc[nt][0] + sc[nt][1];
            s1 += sc[nt][2] + sc[nt][3];
        }
        l0 = l0 * a0 + s0;   // (this lane's columns only: the four lanes of a row are added up at the end)
        l1 = l1 * a1 + s1;
#pragma unroll
        for (int nd = 0; nd < AT_D / 8; ++nd) { o[nd][0] *= a0; o[nd][1] *= a0; o[nd][2] *= a1; o[nd][3] *= a1; }
        // O += P V: the accumulators of two neighbouring 8-position tiles are the A operand of one 16-position step
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t pa[4];
            pa[0] = at_pack<BF16>(sc[2 * kk][0], sc[2 * kk][1]);
            pa[1] = at_pack<BF16>(sc[2 * kk][2], sc[2 * kk][3]);
            pa[2] = at_pack<BF16>(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
            pa[3] = at_pack<BF16>(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
#pragma unroll
            for (int ndp = 0; ndp < AT_D / 16; ++ndp) {
                const int mi = lane >> 3;
                const int row = 16 * kk + 8 * (mi & 1) + (lane & 7), chunk = 2 * ndp + (mi >> 1);
                uint32_t r[4];
                at_ldm4_t(vt + (uint32_t)row * AT_ROW_BYTES + (uint32_t)((chunk ^ (row & 7)) << 4), r);
                at_mma<BF16>(o[2 * ndp], pa, r[0], r[1]);
                at_mma<BF16>(o[2 * ndp + 1], pa, r[2], r[3]);
            }
        }
    }
    at_wait<0>();
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- the four warps' results meet in shared memory (the rings are idle now) ----
    __syncthreads();
    float* sm_m = reinterpret_cast<float*>(smem);                  // [warp][16]
    float* sm_l = sm_m + AT_WARPS * 16;                            // [warp][16]
    float* sm_o = sm_l + AT_WARPS * 16;                            // [warp][16][D]
    if (t == 0) {
        sm_m[warp * 16 + g] = m0; sm_m[warp * 16 + g + 8] = m1;
        sm_l[warp * 16 + g] = l0; sm_l[warp * 16 + g + 8] = l1;
    }
#pragma unroll
    for (int nd = 0; nd < AT_D / 8; ++nd) {
        float* r0 = sm_o + ((size_t)warp * 16 + g) * AT_D + 8 * nd + 2 * t;
        float* r1 = sm_o + ((size_t)warp * 16 + g + 8) * AT_D + 8 * nd + 2 * t;
        r0[0] = o[nd][0]; r0[1] = o[nd][1];
        r1[0] = o[nd][2]; r1[1] = o[nd][3];
    }
    __syncthreads();
    const int d = threadIdx.x;   // 128 threads: one output dimension each
    const size_t slot = (size_t)hk * n_sp + sp;
    for (int r = 0; r < R; ++r) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < AT_WARPS; ++w) M = fmaxf(M, sm_m[w * 16 + r]);
        const float Mb = M == -INFINITY ? 0.f : M;   // (a row that saw nothing in this split: all weights 0)
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < AT_WARPS; ++w) {   // (a warp without tiles has maximum -inf and weight 0)
            const float wgt = exp2f(sm_m[w * 16 + r] - Mb);
            acc = fmaf(wgt, sm_o[((size_t)w * 16 + r) * AT_D + d], acc);
            ls = fmaf(wgt, sm_l[w * 16 + r], ls);
        }
        a.part[(slot * 16 + r) * AT_D + d] = acc;
        if (d == 0) { a.ml[(slot * 16 + r) * 2] = M; a.ml[(slot * 16 + r) * 2 + 1] = ls; }
    }

    // ---- the last CTA of this head to get here merges the splits (nobody waits for anybody) ----
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(g_attn_tickets + hk, 1u) == (unsigned)n_sp - 1u) ? 1 : 0;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // all (max, sum) pairs of the head first, in one round of loads; then the partial outputs, eight loads in flight
    float* s_ml = reinterpret_cast<float*>(smem);   // [split][16][2]
    for (int i = threadIdx.x; i < n_sp * 32; i += AT_WARPS * 32) s_ml[i] = __ldcg(a.ml + (size_t)hk * n_sp * 32 + i);
    __syncthreads();
    // one warp per row (rows warp, warp + 4, ...), four output dimensions per lane
    for (int r = warp; r < R; r += AT_WARPS) {
        float M = -INFINITY;   // finite in the end: every token sees position 0, which the first split holds
        for (int s = 0; s < n_sp; ++s) M = fmaxf(M, s_ml[(s * 16 + r) * 2]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float ls = 0.f;
        const float4* pr = reinterpret_cast<const float4*>(a.part + ((size_t)hk * n_sp * 16 + r) * AT_D) + lane;
        for (int s0 = 0; s0 < n_sp; s0 += 8) {
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (s0 + i < n_sp) ? __ldcg(pr + (size_t)(s0 + i) * 16 * (AT_D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (s0 + i < n_sp) {
                    const float wgt = exp2f(s_ml[((s0 + i) * 16 + r) * 2] - M);
                    acc.x = fmaf(wgt, v[i].x, acc.x); acc.y = fmaf(wgt, v[i].y, acc.y);
                    acc.z = fmaf(wgt, v[i].z, acc.z); acc.w = fmaf(wgt, v[i].w, acc.w);
                    ls = fmaf(wgt, s_ml[((s0 + i) * 16 + r) * 2 + 1], ls);
                }
            }
        }
        const float inv = 1.f / ls;
        const float o4[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
        const int tok = r / a.G;
        const size_t oi = ((size_t)tok * a.H + (size_t)hk * a.G + (r - tok * a.G)) * AT_D + 4 * lane;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (a.out_dtype == AQ_F32) reinterpret_cast<float*>(a.out)[oi + i] = o4[i];
            else if (a.out_dtype == AQ_F16) reinterpret_cast<__half*>(a.out)[oi + i] = __float2half_rn(o4[i]);
            else reinterpret_cast<__nv_bfloat16*>(a.out)[oi + i] = __float2bfloat16_rn(o4[i]);
        }
    }
    if (threadIdx.x == 0) g_attn_tickets[hk] = 0u;
}

// ---- rotary embedding and cache append -----------------------------------------------------------------------
// Pair (i, i + D/2) of every head is rotated by pos * theta^(-2 i / D).  The angle is formed in binary64 (a binary32
// angle at position 4096 would already be off by more than the output's rounding), the rotation in binary32.
template <typename T>
__global__ void rope_kernel(T* x, int n_heads, int D, double pos, double log2_theta) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int half = D / 2;
    if (idx >= n_heads * half) return;
    const int h = idx / half, i = idx - h * half;
    const double ang = pos * exp2(-2.0 * (double)i / (double)D * log2_theta);
    double s, c;
    sincos(ang, &s, &c);
    T* p = x + (size_t)h * D;
    float a, b;
    if constexpr (sizeof(T) == 4) { a = p[i]; b = p[i + half]; }
    else if constexpr (std::is_same<T, __half>::value) { a = __half2float(p[i]); b = __half2float(p[i + half]); }
    else { a = __bfloat162float(p[i]); b = __bfloat162float(p[i + half]); }
    const float fc = (float)c, fs = (float)s;
    const float ra = fmaf(a, fc, -b * fs), rb = fmaf(b, fc, a * fs);
    if constexpr (sizeof(T) == 4) { p[i] = ra; p[i + half] = rb; }
    else if constexpr (std::is_same<T, __half>::value) { p[i] = __float2half_rn(ra); p[i + half] = __float2half_rn(rb); }
    else { p[i] = __float2bfloat16_rn(ra); p[i + half] = __float2bfloat16_rn(rb); }
}

// cache[hk][pos][:] = row[hk][:] for keys and values (16-bit elements, 16 bytes per thread).
__global__ void kv_append_kernel(uint4* kc, uint4* vc, const uint4* k, const uint4* v, int n_kv, int row_vec, int64_t pos, int64_t Lmax) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_kv * row_vec) return;
    const int hk = idx / row_vec, c = idx - hk * row_vec;
    const size_t o = ((size_t)hk * Lmax + pos) * row_vec + c;
    kc[o] = k[idx];
    vc[o] = v[idx];
}

// What a stack program's attention step does with the float32 q, k, v rows of its M new tokens before the attention
// itself: rotates q and k for their positions, rounds q to the activation type into a staging array [M][H][D], and puts
// the rounded k and v into rows pos .. pos + M - 1 of the caches.  One CTA of D/2 threads per (token, head).
template <typename T>
__global__ void attn_prepare_kernel(const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v, T* __restrict__ q16,
                                    T* __restrict__ kc, T* __restrict__ vc, int H, int Hkv, int D, int64_t pos, int64_t Lmax, double log2_theta) {
    const int m = blockIdx.y, hh = blockIdx.x, i = threadIdx.x, half = D / 2;
    pdl_launch_dependents();   // the attention kernel may set itself up and read older cache rows meanwhile
    auto cast = [](float x) -> T {
        if constexpr (std::is_same<T, __half>::value) return __float2half_rn(x);
        else return __float2bfloat16_rn(x);
    };
    if (hh >= H + Hkv) {   // a value head: rounded as it is
        const int hk = hh - H - Hkv;
        const float* src = v + ((size_t)m * Hkv + hk) * D;
        T* dst = vc + ((size_t)hk * Lmax + pos + m) * D;
        dst[i] = cast(src[i]);
        dst[i + half] = cast(src[i + half]);
        return;
    }
    const double ang = (double)(pos + m) * exp2(-2.0 * (double)i / (double)D * log2_theta);
    double sn, cs;
    sincos(ang, &sn, &cs);
    const float fc = (float)cs, fs = (float)sn;
    const bool is_q = hh < H;
    const float* src = is_q ? q + ((size_t)m * H + hh) * D : k + ((size_t)m * Hkv + (hh - H)) * D;
    T* dst = is_q ? q16 + ((size_t)m * H + hh) * D : kc + ((size_t)(hh - H) * Lmax + pos + m) * D;
    const float a = src[i], b = src[i + half];
    dst[i] = cast(fmaf(a, fc, -b * fs));
    dst[i + half] = cast(fmaf(b, fc, a * fs));
}

cudaError_t launch_attn_prepare(const float* q, const float* k, const float* v, void* q16, void* kc, void* vc, int M, int H, int Hkv,
                                int64_t pos, int64_t Lmax, float theta, aq_dtype_t dt, cudaStream_t s) {
    const dim3 grid((unsigned)(H + 2 * Hkv), (unsigned)M);
    const double l2t = log2((double)theta);
    if (dt == AQ_F16)
        attn_prepare_kernel<__half><<<grid, AT_D / 2, 0, s>>>(q, k, v, reinterpret_cast<__half*>(q16), reinterpret_cast<__half*>(kc),
                                                             reinterpret_cast<__half*>(vc), H, Hkv, AT_D, pos, Lmax, l2t);
    else
        attn_prepare_kernel<__nv_bfloat16><<<grid, AT_D / 2, 0, s>>>(q, k, v, reinterpret_cast<__nv_bfloat16*>(q16),
                                                                    reinterpret_cast<__nv_bfloat16*>(kc), reinterpret_cast<__nv_bfloat16*>(vc), H,
                                                                    Hkv, AT_D, pos, Lmax, l2t);
    count_launch();
    return cudaGetLastError();
}

// ---- host ---------------------------------------------------------------------------------------------------
static int attn_max_splits(int n_kv) {
    // one CTA per SM fits (its rings take most of the shared memory), so one wave: as many splits as keep the grid
    // inside the SM count
    int want = sm_count() / n_kv;
    if (want < 1) want = 1;
    return want > AT_MAX_SPLITS ? AT_MAX_SPLITS : want;
}
static void attn_geometry(int n_kv, int64_t L, int* splits, int* chunk) {
    // ... but never less than one tile per warp in a split
    int64_t ch = (L + attn_max_splits(n_kv) - 1) / attn_max_splits(n_kv);
    const int64_t min_ch = (int64_t)AT_WARPS * AT_TILE;
    if (ch < min_ch) ch = min_ch;
    ch = (ch + AT_TILE - 1) / AT_TILE * AT_TILE;
    *chunk = (int)ch;
    *splits = (int)((L + ch - 1) / ch);
}

// Scratch for any context length with this many key/value heads: tickets, (max, sum) pairs, partial outputs.
size_t attn_scratch_bytes(int n_kv) {
    return 256 + (size_t)n_kv * AT_MAX_SPLITS * 16 * 2 * sizeof(float) + (size_t)n_kv * attn_max_splits(n_kv) * 16 * AT_D * sizeof(float) + 256;
}

cudaError_t launch_attn_decode(const void* q, const void* kc, const void* vc, void* out, int M, int n_heads, int n_kv, int64_t L,
                               int64_t Lmax, float scale, aq_dtype_t dt, aq_dtype_t out_dt, void* scratch, cudaStream_t s) {
    int splits, chunk;
    attn_geometry(n_kv, L, &splits, &chunk);
    AttnArgs a;
    a.q = q; a.kc = kc; a.vc = vc; a.out = out;
    uint8_t* sc = reinterpret_cast<uint8_t*>(scratch);
    a.ml = reinterpret_cast<float*>(sc + 256);
    a.part = reinterpret_cast<float*>(sc + 256 + (size_t)n_kv * AT_MAX_SPLITS * 16 * 2 * sizeof(float));
    a.L = L; a.Lmax = Lmax; a.G = n_heads / n_kv; a.M = M; a.H = n_heads; a.chunk = chunk; a.out_dtype = (int)out_dt;
    a.scale_log2 = scale * 1.4426950408889634f;
    const bool bf = (dt == AQ_BF16);
    static PerDeviceOnce configured[2];
    {
        const int rc = configured[bf ? 1 : 0].run(current_device(), [&] {
            return bf ? (int)cudaFuncSetAttribute(attn_decode_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM)
                      : (int)cudaFuncSetAttribute(attn_decode_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM);
        });
        if (rc != 0) return rc < 0 ? cudaErrorInvalidDevice : (cudaError_t)rc;
    }
    const dim3 grid((unsigned)n_kv, (unsigned)splits);
    const cudaError_t e = bf ? launch_pdl(attn_decode_kernel<true>, grid, dim3(AT_WARPS * 32), AT_SMEM, s, a)
                             : launch_pdl(attn_decode_kernel<false>, grid, dim3(AT_WARPS * 32), AT_SMEM, s, a);
    count_launch();
    return e;
}

cudaError_t launch_rope(void* x, int n_heads, int D, int64_t pos, float theta, aq_dtype_t dt, cudaStream_t s) {
    const int n = n_heads * (D / 2);
    const unsigned grid = (unsigned)((n + 127) / 128);
    const double l2t = log2((double)theta);
    if (dt == AQ_F16) rope_kernel<__half><<<grid, 128, 0, s>>>(reinterpret_cast<__half*>(x), n_heads, D, (double)pos, l2t);
    else if (dt == AQ_BF16) rope_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(reinterpret_cast<__nv_bfloat16*>(x), n_heads, D, (double)pos, l2t);
    else rope_kernel<float><<<grid, 128, 0, s>>>(reinterpret_cast<float*>(x), n_heads, D, (double)pos, l2t);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_kv_append(void* kc, void* vc, const void* k, const void* v, int n_kv, int D, int64_t pos, int64_t Lmax, cudaStream_t s) {
    const int row_vec = D * 2 / 16;
    const int n = n_kv * row_vec;
    kv_append_kernel<<<(unsigned)((n + 127) / 128), 128, 0, s>>>(reinterpret_cast<uint4*>(kc), reinterpret_cast<uint4*>(vc),
                                                                 reinterpret_cast<const uint4*>(k), reinterpret_cast<const uint4*>(v), n_kv,
                                                                 row_vec, pos, Lmax);
    count_launch();
    return cudaGetLastError();
}

}  // namespace aq
