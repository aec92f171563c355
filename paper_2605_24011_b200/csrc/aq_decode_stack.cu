// Decode path for a whole program of linears (M = 1..8) in ONE persistent
// kernel launch (Section 4.3: the deployed forward pass dispatches every
// quantised matmul to a low-bit kernel; Appendix D: dequantise on the fly).
//
// Bound: HBM -- every packed byte of every matrix is read once per pass.  A
// 4096 x 4096 matrix is about a microsecond of HBM time, less than a kernel
// launch, so the pass runs as one cooperative grid of one CTA per SM:
//
//   * Work.  Consecutive ops that read the same input vector form a phase.
//     The units (16 rows x 256 k) of a phase's matrices are concatenated and
//     dealt as contiguous runs: first to CTAs, then to the 15 consumer warps
//     of a CTA.
//   * Weight stream.  Which bytes a warp will need does not depend on any
//     activation, so a 16th warp (lane w serves consumer warp w) keeps every
//     consumer's private ring of bulk copies (cp.async.bulk + mbarrier, L2
//     evict-first) full, running ahead across op and phase boundaries.
//   * Dependencies.  Sums leave the warps as fp32 red.add into the output
//     buffer.  Every op has an arrival counter in global memory; a CTA arrives
//     once all its warps have committed their share of the op.  The arrival is
//     a gpu-scope release, which waits for L2 to acknowledge the CTA's sums
//     (about two microseconds under load): with one token a 17th warp does it,
//     so that no consumer warp starts its next op late.  Before a phase
//     a CTA waits (bounded) until the ops that wrote the buffers it reads have
//     been arrived at by every CTA.  Ops nobody waits for soon (k and v of an
//     attention block) therefore overlap the wait of the ops that follow.
//   * Glue.  At the start of a phase each CTA forms, in shared memory, the
//     rounded input vector for the k-slabs its warps will touch (RMS scaling /
//     SiLU(g)*u / plain) with one round trip to L2, and writes its share of the
//     vector to the caller's workspace, where every op's input stays readable.
//     For one token the vector is stored already spread out as the B operand of
//     the tensor-core instruction (non-zero only in the column of its block),
//     so a warp picks its operand up with eight 16-byte loads.
//
// Every wait is bounded: when one runs out the kernel raises a status word,
// gives copies in flight time to land and returns.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

#include "aq_gemv_core.cuh"
#include "aq_internal.h"

namespace aq {

constexpr int DS_WARPS = 15;                // consumer warps
constexpr int DS_CTHREADS = DS_WARPS * 32;  // consumer threads
constexpr int DS_OPBARS = 32;               // ring of per-op arrival barriers
// One or two tokens: a release warp besides the copy warp (17 warps put 5 on one scheduler, so the kernel must stay at 96 registers:
// the launch bound of 640 makes the compiler do that).  More tokens need the registers: 16 warps, and the consumer warp
// that completes an op publishes it itself.
__host__ __device__ constexpr bool ds_release_warp(int MT) { return MT <= 2; }
__host__ __device__ constexpr int ds_threads(int MT) { return DS_CTHREADS + (ds_release_warp(MT) ? 64 : 32); }
__host__ __device__ constexpr int ds_reg_bound(int MT) { return ds_release_warp(MT) ? 640 : 512; }
constexpr int DS_SLOTS = 5;                 // ring depth per warp (units)
constexpr int DS_SLOT_BYTES = 2560;         // the largest unit (4-bit: 2 fragments of 1280 B)
constexpr int DS_MAX_SLOTS = 6;             // staged slabs per phase per CTA (one token; fewer with more tokens)
constexpr int DS_XS_BYTES = DS_MAX_SLOTS * 4224;   // staged input (see ds_slab_bytes)
constexpr int DS_MAX_PHASE_OPS = 8;
constexpr int DS_MAX_DEPS = 12;
constexpr int DS_RMS_HOLD = 4;              // float4 per thread kept in registers by the one-token RMS path
constexpr uint64_t DS_WAIT_NS = 2000000000ull;   // every wait gives up after two seconds

// Shared-memory bytes of one staged slab (256 k): one token is stored spread out
// as B operands (32 lanes x 8 blocks x 16 B) plus 8 block sums, padded to a multiple of 128 bytes (the readers form
// addresses with an XOR); several tokens are stored plainly, [token][256] halves.
__host__ __device__ constexpr int ds_slab_bytes(int M) { return M == 1 ? 4096 + 128 : M * 512; }

__device__ int g_decode_status = 0;   // nonzero: a bounded wait ran out (1 = counter, 2 = copy)

struct DsOp {
    const uint8_t* frags;
    float* dst;            // float32 [M][N]
    const float* res;      // float32 [M][N] added once (by the k-slab-0 units), or null
    int32_t N;             // true rows
    int32_t NT;            // 16-row tiles
    int32_t n_units;       // KP * NT = units_q * (number of CTAs) + units_r
    int32_t bits;
    int32_t units_q;
    int32_t units_r_rot;   // units_r | rot << 16: CTA c takes the run of slot (c + rot) mod (number of CTAs)
};

struct DsPhase {
    const float* src;      // float32 [M][K]
    const float* src2;     // second input of AQ_IN_SILU_MUL, else null
    void* stage;           // [M][K] of the activation dtype: the rounded input, kept for the caller
    int32_t K;
    int32_t in_op;
    int32_t op_first;      // index of ops[0] in the program (names its arrival counter)
    int32_t op_count;
    int32_t units_total;
    int32_t n_deps;
    int16_t deps[DS_MAX_DEPS];   // ops that must be complete before this phase reads its inputs
    int32_t pad_[2];
    DsOp ops[DS_MAX_PHASE_OPS];
};
static_assert(sizeof(DsOp) == 48, "DsOp layout");
static_assert(sizeof(DsPhase) % 16 == 0, "a phase record is fetched with one bulk copy");

// What the copy stream needs to know of an op / a phase, small enough to keep the
// whole program's worth in shared memory (a cursor then advances in tens of cycles).
struct DsMiniOp {
    const uint8_t* frags;
    uint32_t q_bits;       // units_q | bits << 28
    uint32_t r_rot;        // units_r | rot << 16
};
struct DsMiniPhase {
    int32_t op_first;      // index into the mini-op table
    int32_t op_count;
    int32_t pad_[2];
};
static_assert(sizeof(DsMiniOp) == 16 && sizeof(DsMiniPhase) == 16, "mini tables are copied as 16-byte items");
constexpr int DS_MINI_BYTES = 8192;

struct DsArgs {
    const DsPhase* phases;
    const DsMiniPhase* mini_phases;   // n_phases entries, followed by
    const DsMiniOp* mini_ops;         // n_mini_ops entries (contiguous: one copy brings both)
    uint32_t* cnt;         // per-op arrival counters, zero at launch
    int n_phases;
    int n_mini_ops;
    int M;
};

// ---- small PTX wrappers ---------------------------------------------------------
__device__ __forceinline__ uint32_t ds_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ds_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void ds_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ds_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool ds_mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool ds_mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void ds_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ uint64_t ds_now_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait on a shared-memory barrier; false when DS_WAIT_NS passed.
__device__ __forceinline__ bool ds_mbar_wait(uint32_t bar, uint32_t parity) {
    if (ds_mbar_try(bar, parity)) return true;
    const uint64_t t0 = ds_now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (ds_mbar_try(bar, parity)) return true;
        if (ds_now_ns() - t0 > DS_WAIT_NS) return false;
    }
}
__device__ __forceinline__ uint32_t ds_ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Barrier among the consumer warps only (the copy warp never joins).
__device__ __forceinline__ void ds_consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(DS_CTHREADS) : "memory"); }

// ---- the warp's position in its stream of units ---------------------------------
struct DsCursor {
    int ph;                // phase (n_phases: past the end)
    int oi;                // op inside the phase
    int u, u_end;          // position inside the current op
    const uint8_t* base;   // the op's fragments
    int ub;                // bytes per unit
};

// Every op's units are dealt on their own: with n = q G + r units and G CTAs, slot
// s takes q + 1 units if s < r, else q; CTA c takes slot (c + rot) mod G, where rot
// moves on from op to op so that the odd units do not always land on the same CTAs.
__device__ __forceinline__ void ds_cta_run(int q, int r_rot, int& a, int& b) {
    const int r = r_rot & 0xFFFF, rot = r_rot >> 16;
    int s = (int)blockIdx.x + rot;
    if (s >= (int)gridDim.x) s -= (int)gridDim.x;
    a = q * s + min(s, r);
    b = a + q + (s < r ? 1 : 0);
}
// ... and the run of one of its consumer warps (the warps too take turns with the short shares).
__device__ __forceinline__ void ds_warp_run(int q, int r_rot, int warp, int& wa, int& wb) {
    int a, b;
    ds_cta_run(q, r_rot, a, b);
    const int n = b - a;
    int w = warp + ((r_rot >> 16) * 7) % DS_WARPS;
    if (w >= DS_WARPS) w -= DS_WARPS;
    wa = a + (n * w) / DS_WARPS;
    wb = a + (n * (w + 1)) / DS_WARPS;
}

// Moves the cursor to the next op (from (ph, oi) on) in which the warp owns units.
// mp / mo: the mini tables (in shared memory when they fit, else in global memory).
__device__ __forceinline__ void ds_seek(DsCursor& c, const DsMiniPhase* mp, const DsMiniOp* mo, int n_phases, int warp) {
    while (c.ph < n_phases) {
        const DsMiniPhase P = mp[c.ph];
        while (c.oi < P.op_count) {
            const DsMiniOp op = mo[P.op_first + c.oi];
            int u0, u1;
            ds_warp_run((int)(op.q_bits & 0x0FFFFFFFu), (int)op.r_rot, warp, u0, u1);
            if (u0 < u1) {
                c.u = u0; c.u_end = u1;
                c.ub = 2 * frag_bytes((int)(op.q_bits >> 28));
                c.base = op.frags;
                return;
            }
            ++c.oi;
        }
        ++c.ph;
        c.oi = 0;
    }
}

// ---- glue arithmetic --------------------------------------------------------------
__device__ __forceinline__ float ds_silu_mul(float g, float u) { return g / (1.f + expf(-g)) * u; }

// Rounds four values to the activation dtype; *sum gets the sum of the rounded values.
template <bool BF16>
__device__ __forceinline__ uint2 ds_round4(const float4& v, float* sum) {
    uint2 r;
    if constexpr (BF16) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
        r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
        const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        *sum = (fa.x + fa.y) + (fb.x + fb.y);
    } else {
        __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
        r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
        const float2 fa = __half22float2(a), fb = __half22float2(b);
        *sum = (fa.x + fa.y) + (fb.x + fb.y);
    }
    return r;
}

// Four consecutive elements of the input vector of token m at k (k % 4 == 0, k < K), before rounding.
__device__ __forceinline__ float4 ds_form4(const DsPhase& P, int m, int k, float scale) {
    const float4 s = __ldcg(reinterpret_cast<const float4*>(P.src + (int64_t)m * P.K + k));
    if (P.in_op == AQ_IN_SILU_MUL) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(P.src2 + (int64_t)m * P.K + k));
        return make_float4(ds_silu_mul(s.x, t.x), ds_silu_mul(s.y, t.y), ds_silu_mul(s.z, t.z), ds_silu_mul(s.w, t.w));
    }
    return make_float4(s.x * scale, s.y * scale, s.z * scale, s.w * scale);
}

// ---- shared memory ------------------------------------------------------------------
struct DsShared {
    alignas(128) uint8_t ring[DS_WARPS][DS_SLOTS][DS_SLOT_BYTES];
    alignas(128) uint8_t xs[DS_XS_BYTES];   // staged input slabs
    alignas(16) uint8_t mini[DS_MINI_BYTES];   // [DsMiniPhase x n_phases][DsMiniOp x n_mini_ops] when they fit
    alignas(16) DsPhase rec[2];             // descriptors of the current and the next phase
    alignas(8) uint64_t full[DS_WARPS][DS_SLOTS];    // copy landed
    alignas(8) uint64_t empty[DS_WARPS][DS_SLOTS];   // consumer has read the slot
    alignas(8) uint64_t rec_bar[2];
    float red[AQ_DECODE_MAX_M][DS_WARPS];
    float scale[AQ_DECODE_MAX_M];
    int seg_slab_lo[2][DS_MAX_PHASE_OPS];   // per op of the phase: first pair-slab this CTA reads for it
    int seg_slot_lo[2][DS_MAX_PHASE_OPS];   // ... and the slot in xs where that slab is staged (the next slabs follow)
    int slab_of_slot[2][DS_MAX_SLOTS];      // the slabs staged for this phase, ascending
    int n_slots[2];
    int4 run[DS_MAX_PHASE_OPS][DS_WARPS];   // per op of the phase and consumer warp: first unit, end, its slab, its row tile
    int run_xslot[DS_MAX_PHASE_OPS][DS_WARPS];   // ... and the slot in xs of that slab
    alignas(8) uint64_t opbar[DS_OPBARS];   // op (index % DS_OPBARS): the consumer warps that are through with it
    int released;                           // ops whose arrival the release warp has published
    int done[32];                           // (no release warp) warps of this CTA that finished op (index & 31)
    int abort_flag;
};


// Writes 4 rounded elements (k .. k+3 of slab-local index) of the staged vector.
template <int MT>
__device__ __forceinline__ void ds_store4(uint8_t* slab, int M, int m, int kl, uint2 r) {
    if constexpr (MT == 1) {
        const int bk = kl >> 5, t = (kl >> 3) & 3;
        *reinterpret_cast<uint2*>(slab + ds_spread_offset(bk * 4 + t, bk) + (kl & 7) * 2) = r;
    } else {
        *reinterpret_cast<uint2*>(slab + ((size_t)m * 256 + kl) * 2) = r;
    }
}

// The x operand of one pair-slab from its staged copy in shared memory.
template <int MT, bool BF16>
__device__ __forceinline__ void ds_load_x_operand(XOperand<MT>& xo, const uint8_t* slab, int M, int lane) {
    if constexpr (MT == 1) {   // (the B registers are read from the slab where they are used)
        const float2 xs = *reinterpret_cast<const float2*>(slab + 4096 + (lane & 3) * 8);
        xo.X0[0] = xs.x; xo.X1[0] = xs.y;
    } else {
        const uint16_t* x = reinterpret_cast<const uint16_t*>(slab);
        fill_x_operand<MT, BF16>(xo, lane, [&](int tok, int kk) {
            uint4 v = make_uint4(0, 0, 0, 0);
            if (tok < M) v = *reinterpret_cast<const uint4*>(x + tok * 256 + kk);
            return v;
        });
    }
}

// ---- the kernel ---------------------------------------------------------------------
template <int MT, bool BF16>
__global__ void __launch_bounds__(ds_reg_bound(MT), 1) decode_stack_kernel(const DsArgs a) {
    constexpr bool RELW = ds_release_warp(MT);
    extern __shared__ __align__(128) uint8_t ds_smem_raw[];
    DsShared& sh = *reinterpret_cast<DsShared*>(ds_smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int M = a.M;
    const int slab_bytes = ds_slab_bytes(M);

    if (threadIdx.x < DS_OPBARS) { ds_mbar_init(ds_smem(&sh.opbar[threadIdx.x]), DS_WARPS); sh.done[threadIdx.x] = 0; }
    if (threadIdx.x == 0) {
        sh.abort_flag = 0;
        sh.released = 0;
        ds_mbar_init(ds_smem(&sh.rec_bar[0]), 1);
        ds_mbar_init(ds_smem(&sh.rec_bar[1]), 1);
    }
    if (warp < DS_WARPS && lane == 0) {
#pragma unroll
        for (int s = 0; s < DS_SLOTS; ++s) {
            ds_mbar_init(ds_smem(&sh.full[warp][s]), 1);
            ds_mbar_init(ds_smem(&sh.empty[warp][s]), 1);
        }
    }
    // one-token slabs keep zeros everywhere but in the chunks the stagers rewrite every phase
    for (int i = threadIdx.x; i < DS_XS_BYTES / 16; i += (int)blockDim.x)
        reinterpret_cast<uint4*>(sh.xs)[i] = make_uint4(0, 0, 0, 0);
    // the copy stream's tables: into shared memory when they fit
    const int mini_items = a.n_phases + a.n_mini_ops;
    const bool mini_in_smem = mini_items * 16 <= DS_MINI_BYTES;
    if (mini_in_smem)
        for (int i = threadIdx.x; i < mini_items; i += (int)blockDim.x)
            reinterpret_cast<uint4*>(sh.mini)[i] = __ldg(reinterpret_cast<const uint4*>(a.mini_phases) + i);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const DsMiniPhase* mp = mini_in_smem ? reinterpret_cast<const DsMiniPhase*>(sh.mini) : a.mini_phases;
    const DsMiniOp* mo = mini_in_smem ? reinterpret_cast<const DsMiniOp*>(sh.mini + (size_t)a.n_phases * 16) : a.mini_ops;

    uint64_t pol, pol_keep;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));

    if (warp == DS_WARPS) {
        // ================= the copy warp: lane w keeps consumer warp w's ring full =================
        DsCursor c;
        c.ph = a.n_phases; c.oi = 0; c.u = c.u_end = 0; c.base = nullptr; c.ub = 0;
        if (lane < DS_WARPS) { c.ph = 0; ds_seek(c, mp, mo, a.n_phases, lane); }
        uint32_t iseq = 0;   // copies issued for this consumer
        uint64_t t_progress = ds_now_ns();
        uint32_t idle = 0;
        for (;;) {
            const bool active = c.ph < a.n_phases;
            bool moved = false;
            if (active) {
                // the n-th copy into a slot (n >= 1) waits for the consumer's arrival after its (n-1)-th read
                const uint32_t slot = iseq % DS_SLOTS, n = iseq / DS_SLOTS;
                const bool is_free = (n == 0) || ds_mbar_test(ds_smem(&sh.empty[lane][slot]), (n - 1) & 1u);
                if (is_free) {
                    const uint32_t bar = ds_smem(&sh.full[lane][slot]);
                    ds_expect_tx(bar, (uint32_t)c.ub);
                    ds_bulk_load(ds_smem(&sh.ring[lane][slot][0]), c.base + (int64_t)c.u * c.ub, (uint32_t)c.ub, bar, pol);
                    ++iseq;
                    if (++c.u == c.u_end) { ++c.oi; ds_seek(c, mp, mo, a.n_phases, lane); }
                    moved = true;
                }
            }
            if (!__any_sync(0xffffffffu, active)) break;
            if (__any_sync(0xffffffffu, moved)) { idle = 0; continue; }
            __nanosleep(200);   // a consumer needs about a microsecond per unit: no need to spin on its barriers
            if ((++idle & 255u) == 0) {   // nothing to do for a while: stop if the CTA gave up, or after the time limit
                if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) break;
                const uint64_t t = ds_now_ns();
                if (idle == 256u) t_progress = t;
                else if (t - t_progress > 2 * DS_WAIT_NS) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; break; }
            }
        }
        return;
    }

    if (RELW && warp == DS_WARPS + 1) {
        // ================= the release warp: publishes, op by op, that this CTA's sums are in place =================
        // The gpu-scope release waits until the CTA's additions have been acknowledged by L2 (microseconds): here it
        // holds up nobody, whereas a consumer warp doing it would start its next op that much later.
        if (lane == 0) {
            for (int opx = 0; opx < a.n_mini_ops; ++opx) {
                const uint32_t bar = ds_smem(&sh.opbar[opx % DS_OPBARS]), parity = (uint32_t)(opx / DS_OPBARS) & 1u;
                const uint64_t t0 = ds_now_ns();
                bool ok = ds_mbar_try(bar, parity);
                while (!ok) {
#pragma unroll 1
                    for (int i = 0; i < 32 && !ok; ++i) {   // (sleeping between tries: this warp shares a scheduler with consumers)
                        __nanosleep(100);
                        ok = ds_mbar_try(bar, parity);
                    }
                    if (ok) break;
                    if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) break;
                    if (ds_now_ns() - t0 > 2 * DS_WAIT_NS) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; break; }
                }
                if (!ok) break;
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.cnt + opx) : "memory");
                *reinterpret_cast<volatile int*>(&sh.released) = opx + 1;
            }
        }
        return;
    }

    // ================= consumer warps =================
    auto fetch_record = [&](int q) {
        const uint32_t bar = ds_smem(&sh.rec_bar[q & 1]);
        ds_expect_tx(bar, (uint32_t)sizeof(DsPhase));
        ds_bulk_load(ds_smem(&sh.rec[q & 1]), a.phases + q, (uint32_t)sizeof(DsPhase), bar, pol_keep);
    };
    if (threadIdx.x == 0) {
        fetch_record(0);
        if (a.n_phases > 1) fetch_record(1);
    }

    uint32_t cslot = 0, cparity = 0;   // next ring slot to consume and the parity of its `full` barrier
    bool dead = false;                 // this warp gave up on a wait
    XOperand<MT> xo;

#pragma unroll 1
    for (int ph = 0; ph < a.n_phases; ++ph) {
        const int pb = ph & 1;
        const DsPhase& P = sh.rec[pb];
        // -- the phase's descriptors (fetched one phase ahead) --
        if (!ds_mbar_wait(ds_smem(&sh.rec_bar[pb]), (uint32_t)(ph >> 1) & 1u)) {
            atomicCAS(&g_decode_status, 0, 2);
            sh.abort_flag = 1;
        }
        if (*reinterpret_cast<volatile int*>(&sh.abort_flag) == 0) {
            // -- which slabs of the input this CTA's warps will read (independent of the data) --
            if (threadIdx.x == DS_CTHREADS - 1) {
                int lo[DS_MAX_PHASE_OPS], hi[DS_MAX_PHASE_OPS];
                for (int oi = 0; oi < P.op_count; ++oi) {
                    int u0, u1;
                    ds_cta_run(P.ops[oi].units_q, P.ops[oi].units_r_rot, u0, u1);
                    lo[oi] = (u0 < u1) ? u0 / P.ops[oi].NT : 0;
                    hi[oi] = (u0 < u1) ? (u1 - 1) / P.ops[oi].NT : -1;
                    sh.seg_slab_lo[pb][oi] = lo[oi];
                }
                // ascending list of the distinct slabs: repeatedly take the smallest one above the last
                int n = 0, last = -1;
                for (;;) {
                    int nxt = 0x7fffffff;
                    for (int oi = 0; oi < P.op_count; ++oi) {
                        if (hi[oi] > last) nxt = min(nxt, max(lo[oi], last + 1));
                    }
                    if (nxt == 0x7fffffff || n == DS_MAX_SLOTS) break;
                    sh.slab_of_slot[pb][n++] = nxt;
                    last = nxt;
                }
                sh.n_slots[pb] = n;
                for (int oi = 0; oi < P.op_count; ++oi) {
                    int sl = 0;
                    while (sl < n && sh.slab_of_slot[pb][sl] != lo[oi]) ++sl;
                    sh.seg_slot_lo[pb][oi] = sl;
                }
            }
            // -- wait for the writers of what this phase reads --
            if ((int)threadIdx.x < P.n_deps) {
                const uint32_t* c = a.cnt + P.deps[threadIdx.x];
                uint32_t i = 0;
                uint64_t t0 = 0;
                while (ds_ld_acquire(c) < gridDim.x) {
                    if ((++i & 63u) == 0) {   // now and then: did another CTA give up, or has this wait run out?
                        if (*reinterpret_cast<volatile int*>(&g_decode_status) != 0) { sh.abort_flag = 1; break; }
                        const uint64_t t = ds_now_ns();
                        if (t0 == 0) t0 = t;
                        if (t - t0 > DS_WAIT_NS) { atomicCAS(&g_decode_status, 0, 1); sh.abort_flag = 1; break; }
                    }
                }
            }
        }
        ds_consumer_sync();
        if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) break;
        // every warp is past phase ph - 1: its record slot is free for phase ph + 1
        if (threadIdx.x == 0 && ph >= 1 && ph + 1 < a.n_phases) fetch_record(ph + 1);
        // every warp's run in every op of the phase, worked out by one thread each (the warps then switch ops with one load)
        if ((int)threadIdx.x < P.op_count * DS_WARPS) {
            const int oi = (int)threadIdx.x / DS_WARPS, w = (int)threadIdx.x - oi * DS_WARPS;
            const DsOp& op = P.ops[oi];
            int u0, u1;
            ds_warp_run(op.units_q, op.units_r_rot, w, u0, u1);
            const int Pk = (u0 < u1) ? u0 / op.NT : 0;
            sh.run[oi][w] = make_int4(u0, u1, Pk, u0 - Pk * op.NT);
            sh.run_xslot[oi][w] = sh.seg_slot_lo[pb][oi] + Pk - sh.seg_slab_lo[pb][oi];
        }

        // -- form the rounded input vector: slabs this CTA reads -> shared memory, its share -> workspace --
        {
            const int n_slots = sh.n_slots[pb];
            const int q4 = P.K >> 2;                                  // groups of 4 elements per token
            const int g0 = (int)(((int64_t)q4 * blockIdx.x) / gridDim.x), g1 = (int)(((int64_t)q4 * (blockIdx.x + 1)) / gridDim.x);
            uint16_t* rec_out = reinterpret_cast<uint16_t*>(P.stage);
            // the staged copy of slab `slab`, or null when this CTA does not read it
            auto slot_of = [&](int slab) -> uint8_t* {
                for (int sl = 0; sl < n_slots; ++sl)
                    if (sh.slab_of_slot[pb][sl] == slab) return sh.xs + (size_t)sl * slab_bytes;
                return nullptr;
            };
            // stores group i4 (elements 4 i4 ..) of token m into slab copy `sl`; whole warps call this together
            auto place = [&](uint8_t* sl, int m, int i4, float4 v, bool rec) {
                float sum;
                const uint2 r = ds_round4<BF16>(v, &sum);   // v is zero past the end of the row: padding stages zeros
                if constexpr (MT == 1) {   // block sums: 8 consecutive groups = 8 consecutive lanes
                    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                }
                const int kl = (i4 * 4) & 255;
                if (sl) {
                    ds_store4<MT>(sl, M, m, kl, r);
                    if constexpr (MT == 1) {
                        if ((lane & 7) == 0) *reinterpret_cast<float*>(sl + 4096 + (kl >> 5) * 4) = sum;
                    }
                }
                if (rec) *reinterpret_cast<uint2*>(rec_out + (int64_t)m * P.K + i4 * 4) = r;
            };
            if (P.in_op == AQ_IN_RMSNORM && MT == 1 && q4 <= DS_RMS_HOLD * DS_CTHREADS) {
                // one token, row held in registers: one trip to L2, destinations worked out while it is under way
                float4 v[DS_RMS_HOLD];
                uint8_t* dest[DS_RMS_HOLD];
#pragma unroll
                for (int n = 0; n < DS_RMS_HOLD; ++n) {
                    const int i4 = threadIdx.x + n * DS_CTHREADS;
                    v[n] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (i4 < q4) v[n] = __ldcg(reinterpret_cast<const float4*>(P.src) + i4);
                }
#pragma unroll
                for (int n = 0; n < DS_RMS_HOLD; ++n) dest[n] = slot_of((threadIdx.x + n * DS_CTHREADS) >> 6);
                float ss = 0.f;
#pragma unroll
                for (int n = 0; n < DS_RMS_HOLD; ++n) {
                    ss = fmaf(v[n].x, v[n].x, ss); ss = fmaf(v[n].y, v[n].y, ss);
                    ss = fmaf(v[n].z, v[n].z, ss); ss = fmaf(v[n].w, v[n].w, ss);
                }
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
                if (lane == 0) sh.red[0][warp] = ss;
                ds_consumer_sync();
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < DS_WARPS; ++w) tot += sh.red[0][w];
                const float scale = rsqrtf(tot / (float)P.K + 1e-6f);
#pragma unroll
                for (int n = 0; n < DS_RMS_HOLD; ++n) {
                    const int i4 = threadIdx.x + n * DS_CTHREADS;
                    if (n * DS_CTHREADS < q4)   // the same for every thread: warps stay whole
                        place(dest[n], 0, i4, make_float4(v[n].x * scale, v[n].y * scale, v[n].z * scale, v[n].w * scale),
                              i4 >= g0 && i4 < g1);
                }
            } else {
                if (P.in_op == AQ_IN_RMSNORM) {
                    for (int m = 0; m < M; ++m) {
                        const float4* s4 = reinterpret_cast<const float4*>(P.src + (int64_t)m * P.K);
                        float ss = 0.f;
                        for (int i = threadIdx.x; i < q4; i += DS_CTHREADS) {
                            const float4 v = __ldcg(s4 + i);
                            ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
                        }
#pragma unroll
                        for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
                        if (lane == 0) sh.red[m][warp] = ss;
                    }
                    ds_consumer_sync();
                    if ((int)threadIdx.x < M) {
                        float tot = 0.f;
#pragma unroll
                        for (int w = 0; w < DS_WARPS; ++w) tot += sh.red[threadIdx.x][w];
                        sh.scale[threadIdx.x] = rsqrtf(tot / (float)P.K + 1e-6f);
                    }
                    ds_consumer_sync();
                }
                // one list of work: first the slabs this CTA reads, then its share of the record
                const int per_slab = 64 * M;
                const int n_a = n_slots * per_slab;
                const int n_b = (g1 - g0) * M;
                const int n_all = n_a + n_b;
                for (int it0 = 0; it0 < n_all; it0 += DS_CTHREADS) {
                    const int it = it0 + threadIdx.x;
                    int m = 0, i4 = 0;
                    bool valid = false;
                    uint8_t* sl = nullptr;
                    if (it < n_a) {
                        const int s_ = it / per_slab, w = it - s_ * per_slab;
                        m = w >> 6;
                        i4 = sh.slab_of_slot[pb][s_] * 64 + (w & 63);
                        sl = sh.xs + (size_t)s_ * slab_bytes;
                        valid = i4 < q4;
                    } else if (it < n_all) {
                        const int w = it - n_a;
                        m = w / (g1 - g0);
                        i4 = g0 + w - m * (g1 - g0);
                        valid = true;
                    }
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (valid) v = ds_form4(P, m, i4 * 4, P.in_op == AQ_IN_RMSNORM ? sh.scale[m] : 1.f);
                    if (it0 + (int)(threadIdx.x - lane) < n_a) {
                        place(sl, m, i4, v, false);              // n_a is a multiple of 32: the whole warp is inside the slab items
                    } else if (valid) {
                        float sum;
                        const uint2 r = ds_round4<BF16>(v, &sum);
                        *reinterpret_cast<uint2*>(rec_out + (int64_t)m * P.K + i4 * 4) = r;
                    }
                }
            }
        }
        ds_consumer_sync();

        // -- consume this warp's units of the phase --
#pragma unroll 1
        for (int oi = 0; oi < P.op_count; ++oi) {
            const int opx = P.op_first + oi;
            const DsOp& op = P.ops[oi];
            const int NT = op.NT, bits = op.bits;
            const int4 rn = sh.run[oi][warp];
            const int u0 = rn.x, u1 = rn.y;
            if (u0 < u1 && !dead) {
                int Pk = rn.z, R = rn.w;
                const uint8_t* xseg = sh.xs + (size_t)sh.run_xslot[oi][warp] * slab_bytes;
                ds_load_x_operand<MT, BF16>(xo, xseg, M, lane);
                uint32_t xlane = ds_spread_lane_base(xseg, lane);
                float* dst = op.dst;
                const float* res = op.res;
                const int N = op.N;
                // the unit loop, one copy per code width (the width is the op's, not the unit's)
                auto run_units = [&](auto bits_tag) {
                    constexpr int BITS = decltype(bits_tag)::value;
#pragma unroll 1
                    for (int u = u0; u < u1; ++u) {
                        dead = __any_sync(0xffffffffu, !ds_mbar_wait(ds_smem(&sh.full[warp][cslot]), cparity));
                        if (dead) {
                            if (lane == 0) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; }
                            break;
                        }
                        const uint8_t* unit = &sh.ring[warp][cslot][0];
                        float acc[4] = {0.f, 0.f, 0.f, 0.f};
                        unit_mac<BITS, MT, BF16, MT == 1>(unit, xo, lane, acc, xlane);
                        __syncwarp();        // every lane has read its part of the slot
                        if (lane == 0) ds_mbar_arrive(ds_smem(&sh.empty[warp][cslot]));
                        if (++cslot == DS_SLOTS) { cslot = 0; cparity ^= 1u; }
                        unit_commit<MT>(acc, dst, N, R * 16, N, M, lane, Pk == 0 ? res : nullptr);
                        if (++R == NT) {
                            R = 0; ++Pk;
                            xseg += slab_bytes;
                            xlane += (uint32_t)slab_bytes;
                            if (u + 1 < u1) ds_load_x_operand<MT, BF16>(xo, xseg, M, lane);
                        }
                    }
                };
                if (bits == 2) run_units(std::integral_constant<int, 2>{});
                else if (bits == 3) run_units(std::integral_constant<int, 3>{});
                else run_units(std::integral_constant<int, 4>{});
            }
            __syncwarp();
            if constexpr (RELW) {
                // arrive: this warp is through with the op (its additions are ordered before the arrival); the release
                // warp publishes the op once all consumer warps have arrived
                if (lane == 0) {
                    // the barriers are a ring: do not lap the release warp
                    uint32_t spins = 0;
                    uint64_t t0 = 0;
                    while (opx - *reinterpret_cast<volatile int*>(&sh.released) >= DS_OPBARS) {
                        if ((++spins & 255u) == 0) {
                            if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) break;
                            const uint64_t t = ds_now_ns();
                            if (t0 == 0) t0 = t;
                            if (t - t0 > DS_WAIT_NS) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; break; }
                        }
                    }
                    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(ds_smem(&sh.opbar[opx % DS_OPBARS])) : "memory");
                }
            } else {
                // arrive: the CTA's last warp to finish the op publishes it (the warps' commits are ordered before the
                // release below through the acq_rel counter in shared memory)
                if (lane == 0) {
                    int old;
                    asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(ds_smem(&sh.done[opx & 31])) : "memory");
                    if (old == DS_WARPS - 1) {
                        sh.done[opx & 31] = 0;
                        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.cnt + opx) : "memory");
                    }
                }
            }
        }
    }

    // after a failed wait copies may still be on their way into this CTA's shared memory: give them time
    if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) __nanosleep(500000);
}

// ---- host: plan, cache, launch -----------------------------------------------------
namespace {

struct DecodePlan {
    std::vector<uint8_t> key;
    std::vector<aq_handle_t> handles;
    uint8_t* dev = nullptr;       // [phase records][mini phases, mini ops][arrival counters]
    size_t phases_bytes = 0, mini_bytes = 0, cnt_bytes = 0;
    int n_mini_ops = 0;
    int n_phases = 0;
    int device = 0;
    uint64_t stamp = 0;
};

std::mutex g_plan_mutex;
std::vector<DecodePlan*> g_plans;
uint64_t g_plan_clock = 0;
constexpr size_t MAX_PLANS = 16;

void drop_plan(DecodePlan* p) {
    if (p->dev) cudaFree(p->dev);
    delete p;
}

template <typename T> void key_put(std::vector<uint8_t>& k, const T& v) {
    const uint8_t* b = reinterpret_cast<const uint8_t*>(&v);
    k.insert(k.end(), b, b + sizeof(T));
}

}  // namespace

// Device tables of a program: one record per phase (at most DS_MAX_PHASE_OPS ops that
// read the same input vector).  False when the program does not fit this kernel.
bool build_decode_tables(const aq_stack_t* p, const StackPlan& plan, int M, int n_cta, uint8_t* ws,
                         std::vector<DsPhase>& phases) {
    if (M < 1 || M > AQ_DECODE_MAX_M || p->n_ops > 32000) return false;
    phases.clear();
    std::vector<int> writer(p->n_bufs, -1);
    std::vector<char> waited(p->n_ops, 0);
    int rot = 0;   // where the next op's odd units start
    const int n_ph = (int)plan.phase_first.size();
    for (int ph = 0; ph < n_ph; ++ph) {
        const int pfirst = plan.phase_first[ph];
        const int plast = (ph + 1 < n_ph) ? plan.phase_first[ph + 1] : p->n_ops;
        for (int first = pfirst; first < plast;) {
            // as many of the phase's ops (at most DS_MAX_PHASE_OPS) as leave every CTA's staged slabs inside the
            // shared-memory buffer; the rest of them form a further phase with the same input
            const aq_stack_op_t& f = p->ops[first];
            const int64_t K = p->buf_width[f.src];
            if (K > (int64_t)1 << 24 || n_cta > 32767) return false;
            DsPhase P;
            int count = std::min(plast - first, DS_MAX_PHASE_OPS), rot_after = rot;
            for (; count >= 1; --count) {
                memset(&P, 0, sizeof(P));
                int r2 = rot;
                int64_t off = 0;
                bool ok = true;
                for (int i = first; i < first + count && ok; ++i) {
                    const aq_handle_s* h = p->ops[i].w;
                    DsOp& d = P.ops[i - first];
                    const int64_t nu = (int64_t)h->KP * h->NT;
                    if (off + nu > (int64_t)1 << 26) { ok = false; break; }
                    d.N = (int32_t)h->N; d.NT = h->NT; d.n_units = (int32_t)nu; d.bits = h->bits;
                    d.units_q = (int32_t)(nu / n_cta);
                    d.units_r_rot = (int32_t)(nu % n_cta) | (r2 << 16);
                    r2 = (int)((r2 + nu % n_cta) % n_cta);
                    off += nu;
                }
                for (int c = 0; c < n_cta && ok; ++c) {
                    std::vector<int64_t> need;
                    for (int i = 0; i < count; ++i) {
                        const int64_t q = P.ops[i].units_q, r = P.ops[i].units_r_rot & 0xFFFF, ro = P.ops[i].units_r_rot >> 16;
                        const int64_t sl = (c + ro) % n_cta;
                        const int64_t u0 = q * sl + std::min(sl, r), u1 = u0 + q + (sl < r ? 1 : 0);
                        if (u0 < u1)
                            for (int64_t x = u0 / P.ops[i].NT; x <= (u1 - 1) / P.ops[i].NT; ++x) need.push_back(x);
                    }
                    std::sort(need.begin(), need.end());
                    const int64_t slabs = std::unique(need.begin(), need.end()) - need.begin();
                    if (slabs > DS_MAX_SLOTS || slabs * ds_slab_bytes(M) > DS_XS_BYTES) ok = false;
                }
                if (ok) { P.units_total = (int32_t)off; rot_after = r2; break; }
            }
            if (count < 1) return false;
            const int last = first + count;
            rot = rot_after;
            P.src = reinterpret_cast<const float*>(ws + plan.buf_off[f.src]);
            P.src2 = (f.in_op == AQ_IN_SILU_MUL) ? reinterpret_cast<const float*>(ws + plan.buf_off[f.src2]) : nullptr;
            P.stage = ws + plan.in_off[first];
            P.K = (int32_t)K; P.in_op = f.in_op; P.op_first = first; P.op_count = count;
            std::vector<int> deps;
            auto need = [&](int buf) {
                const int w = writer[buf];
                if (w >= 0 && !waited[w]) { waited[w] = 1; deps.push_back(w); }
            };
            need(f.src);
            if (f.in_op == AQ_IN_SILU_MUL) need(f.src2);
            for (int i = first; i < last; ++i) {
                const aq_stack_op_t& o = p->ops[i];
                DsOp& d = P.ops[i - first];
                d.frags = o.w->frags;
                d.dst = reinterpret_cast<float*>(ws + plan.buf_off[o.dst]);
                d.res = (o.out_op == AQ_OUT_ADD) ? reinterpret_cast<const float*>(ws + plan.buf_off[o.res]) : nullptr;
                if (o.out_op == AQ_OUT_ADD) need(o.res);
            }
            if ((int)deps.size() > DS_MAX_DEPS) return false;
            P.n_deps = (int)deps.size();
            for (size_t j = 0; j < deps.size(); ++j) P.deps[j] = (int16_t)deps[j];
            for (int i = first; i < last; ++i) writer[p->ops[i].dst] = i;
            phases.push_back(P);
            first = last;
        }
    }
    return true;
}

template <int MT, bool BF16>
static cudaError_t launch_ds(const DsArgs& a, int grid, cudaStream_t s) {
    auto kern = decode_stack_kernel<MT, BF16>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DsShared));
        if (e != cudaSuccess) return e;
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, ds_threads(MT), sizeof(DsShared));
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
        configured = true;
    }
    DsArgs args = a;
    void* params[1] = {&args};
    cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3((unsigned)grid), dim3(ds_threads(MT)), params,
                                                sizeof(DsShared), s);
    if (e == cudaSuccess) count_launch();
    return e;
}

int launch_decode_stack(const aq_stack_t* p, const StackPlan& plan, int M, aq_dtype_t dt, uint8_t* ws, cudaStream_t s,
                        cudaError_t* err) {
    *err = cudaSuccess;
    const int grid = sm_count();
    int dev = 0;
    cudaGetDevice(&dev);
    // key: everything the device tables are computed from
    std::vector<uint8_t> key;
    key_put(key, M); key_put(key, dev); key_put(key, grid); key_put(key, ws);
    key_put(key, p->n_ops); key_put(key, p->n_bufs);
    for (int i = 0; i < p->n_ops; ++i) {
        key_put(key, p->ops[i]);
        key_put(key, p->ops[i].w->frags);
    }
    for (int b = 0; b < p->n_bufs; ++b) key_put(key, p->buf_width[b]);

    std::lock_guard<std::mutex> lock(g_plan_mutex);
    DecodePlan* dp = nullptr;
    for (DecodePlan* q : g_plans)
        if (q->key == key) { dp = q; break; }
    if (!dp) {
        std::vector<DsPhase> phases;
        if (!build_decode_tables(p, plan, M, grid, ws, phases)) return 1;
        dp = new DecodePlan();
        dp->key = key;
        dp->device = dev;
        for (int i = 0; i < p->n_ops; ++i) dp->handles.push_back(p->ops[i].w);
        dp->phases_bytes = (phases.size() * sizeof(DsPhase) + 255) / 256 * 256;
        std::vector<uint8_t> mini(phases.size() * sizeof(DsMiniPhase));
        for (size_t i = 0; i < phases.size(); ++i) {
            DsMiniPhase mph;
            memset(&mph, 0, sizeof(mph));
            mph.op_first = dp->n_mini_ops; mph.op_count = phases[i].op_count;
            memcpy(mini.data() + i * sizeof(DsMiniPhase), &mph, sizeof(mph));
            dp->n_mini_ops += phases[i].op_count;
        }
        for (size_t i = 0; i < phases.size(); ++i)
            for (int j = 0; j < phases[i].op_count; ++j) {
                DsMiniOp mop;
                mop.frags = phases[i].ops[j].frags;
                mop.q_bits = (uint32_t)phases[i].ops[j].units_q | ((uint32_t)phases[i].ops[j].bits << 28);
                mop.r_rot = (uint32_t)phases[i].ops[j].units_r_rot;
                const uint8_t* b = reinterpret_cast<const uint8_t*>(&mop);
                mini.insert(mini.end(), b, b + sizeof(mop));
            }
        dp->mini_bytes = (mini.size() + 255) / 256 * 256;
        dp->cnt_bytes = ((size_t)p->n_ops * sizeof(uint32_t) + 255) / 256 * 256;
        dp->n_phases = (int)phases.size();
        cudaError_t e = cudaMalloc(&dp->dev, dp->phases_bytes + dp->mini_bytes + dp->cnt_bytes);
        if (e == cudaSuccess) e = cudaMemcpy(dp->dev, phases.data(), phases.size() * sizeof(DsPhase), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(dp->dev + dp->phases_bytes, mini.data(), mini.size(), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { cudaGetLastError(); drop_plan(dp); *err = e; return -1; }
        if (g_plans.size() >= MAX_PLANS) {
            size_t oldest = 0;
            for (size_t i = 1; i < g_plans.size(); ++i)
                if (g_plans[i]->stamp < g_plans[oldest]->stamp) oldest = i;
            drop_plan(g_plans[oldest]);
            g_plans.erase(g_plans.begin() + oldest);
        }
        g_plans.push_back(dp);
    }
    dp->stamp = ++g_plan_clock;

    DsArgs a;
    a.phases = reinterpret_cast<const DsPhase*>(dp->dev);
    a.mini_phases = reinterpret_cast<const DsMiniPhase*>(dp->dev + dp->phases_bytes);
    a.mini_ops = reinterpret_cast<const DsMiniOp*>(dp->dev + dp->phases_bytes + (size_t)dp->n_phases * sizeof(DsMiniPhase));
    a.n_mini_ops = dp->n_mini_ops;
    a.cnt = reinterpret_cast<uint32_t*>(dp->dev + dp->phases_bytes + dp->mini_bytes);
    a.n_phases = dp->n_phases;
    a.M = M;
    cudaError_t e = cudaMemsetAsync(a.cnt, 0, dp->cnt_bytes, s);
    if (e == cudaSuccess) {
        const bool bf = (dt == AQ_BF16);
        if (M == 1) e = bf ? launch_ds<1, true>(a, grid, s) : launch_ds<1, false>(a, grid, s);
        else if (M == 2) e = bf ? launch_ds<2, true>(a, grid, s) : launch_ds<2, false>(a, grid, s);
        else if (M <= 4) e = bf ? launch_ds<4, true>(a, grid, s) : launch_ds<4, false>(a, grid, s);
        else e = bf ? launch_ds<8, true>(a, grid, s) : launch_ds<8, false>(a, grid, s);
    }
    if (e != cudaSuccess) { *err = e; return -1; }
    return 0;
}

void decode_stack_forget(aq_handle_t h) {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    for (size_t i = 0; i < g_plans.size();) {
        bool uses = false;
        for (aq_handle_t x : g_plans[i]->handles)
            if (x == h) { uses = true; break; }
        if (uses) { drop_plan(g_plans[i]); g_plans.erase(g_plans.begin() + i); }
        else ++i;
    }
}

int read_decode_status(bool clear) {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_decode_status, sizeof(int));
    if (clear && v) { int z = 0; cudaMemcpyToSymbol(g_decode_status, &z, sizeof(int)); }
    return v;
}

}  // namespace aq
