// Decode path for a whole program of linears (M = 1..8) in ONE persistent
// kernel launch (Section 4.3: the deployed forward pass dispatches every
// quantised matmul to a low-bit kernel; Appendix D: dequantise on the fly).
//
// Bound: HBM -- every packed byte of every matrix is read once per pass.  A
// 4096 x 4096 matrix is about a microsecond of HBM time, less than a kernel
// launch, so the pass runs as one cooperative grid of one CTA per SM:
//
//   * Work.  Consecutive ops that read the same input vector form a phase.
//     Every op's units (16 rows x 256 k) are dealt as contiguous runs to the
//     CTAs; inside a CTA the runs of a phase are concatenated into one list
//     and consumer warp w takes positions w, w + 15, w + 30 ... of it, so all
//     warps of a CTA reach the end of a phase within one unit of each other
//     and a warp never "switches ops": every unit comes with a descriptor.
//   * Weight stream.  Which bytes a warp will need does not depend on any
//     activation, so a 16th warp (lane w serves consumer warp w) keeps every
//     consumer's private ring of bulk copies (cp.async.bulk + mbarrier, L2
//     evict-first) full, running ahead across op and phase boundaries, and
//     writes each unit's descriptor (op, unit index) beside it.
//   * Sums and dependencies.  A unit's 16 row sums leave the warp as ONE
//     64-bit red.add each: the sum in 2^-24 fixed point in the upper 52 bits
//     plus 1 in the lower 12 bits.  A row is complete when its count equals the
//     number of k-slabs of the matrix, so whoever needs a value polls the value
//     itself: no arrival counters, no fences, no release, and the result does
//     not depend on the order of the additions.  A CTA starts a phase as soon
//     as the elements IT reads are complete, not when the whole op is.
//   * Glue.  At the start of a phase each CTA forms, in shared memory, the
//     rounded input vector for the k-slabs its warps will touch (RMS scaling /
//     SiLU(g)*u / plain) with one round trip to L2, and writes its share of the
//     float32 buffer and of the rounded vector to the caller's workspace,
//     where every op's input and output stay readable.  For one token the
//     vector is stored already spread out as the B operand of the tensor-core
//     instruction (non-zero only in the column of its block), so a warp picks
//     its operand up with eight 16-byte loads.
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

typedef unsigned long long u64;

constexpr int DS_WARPS = 15;                // consumer warps
constexpr int DS_CTHREADS = DS_WARPS * 32;  // consumer threads
constexpr int DS_THREADS = DS_CTHREADS + 32;   // + the copy warp
constexpr int DS_SLOTS = 5;                 // ring depth per warp (units)
constexpr int DS_SLOT_BYTES = 2560;         // the largest unit (4-bit: 2 fragments of 1280 B)
constexpr int DS_MAX_SLOTS = 6;             // staged slabs per phase per CTA (one token; fewer with more tokens)
constexpr int DS_XS_BYTES = DS_MAX_SLOTS * 4224;   // staged input (see ds_slab_bytes)
constexpr int DS_MAX_PHASE_OPS = 8;
constexpr int DS_RMS_HOLD = 4;              // groups of four elements per thread kept in registers by the one-token RMS path
constexpr int DS_DESC_BITS_SHIFT = 8;       // descriptor word 0: op inside the phase | code width << 8
constexpr u64 DS_WAIT_NS_DEFAULT = 2000000000ull;   // every wait gives up after two seconds

// A packed sum: bits [12, 64) hold the value in units of 2^-24 (two's complement), bits [0, 12) the number of
// contributions added so far.
constexpr int DS_CNT_BITS = 12;
constexpr u64 DS_CNT_MASK = (1ull << DS_CNT_BITS) - 1;
constexpr int DS_MAX_CONTRIB = (1 << DS_CNT_BITS) - 1;
constexpr float DS_FIX_ONE = 16777216.f;            // 2^24
constexpr float DS_FIX_MAX = 134217600.f;           // just below 2^27: what the 52-bit field holds with room to add
constexpr int DS_RES_PLAIN = 0x100;

// Shared-memory bytes of one staged slab (256 k): one token is stored spread out
// as B operands (32 lanes x 8 blocks x 16 B) plus 8 block sums, padded to a multiple of 128 bytes (the readers form
// addresses with an XOR); several tokens are stored plainly, [token][256] halves.
__host__ __device__ constexpr int ds_slab_bytes(int M) { return M == 1 ? 4096 + 128 : M * 512; }

__device__ int g_decode_status = 0;   // nonzero: a bounded wait ran out (1 = an input never completed, 2 = a copy)

struct DsOp {
    const uint8_t* frags;
    u64* dst;              // packed sums [M][N]
    const void* res;       // [M][N] added once (by the k-slab-0 units), or null: packed sums that are complete before the
                           // phase starts, or plain float32 when bit 8 of `bits` is set (the program input)
    int32_t N;             // true rows
    int32_t NT;            // 16-row tiles
    uint32_t nt_magic;     // floor(2^32 / NT) + 1: u / NT = umulhi(u, magic) or one more (u < 2^26); 0 when NT = 1
    int32_t bits;          // code width | DS_RES_PLAIN
    int32_t units_q;       // KP * NT = units_q * (number of CTAs) + units_r
    int32_t units_r_rot;   // units_r | rot << 16: CTA c takes the run of slot (c + rot) mod (number of CTAs)
};

struct DsPhase {
    const u64* src;        // packed [M][K], or null when the source is plain float32
    const u64* src2;       // second input of AQ_IN_SILU_MUL (packed), else null
    const float* src_f;    // plain float32 [M][K] source (the program input), used when src is null
    const float* src2_f;
    float* rec;            // float32 [M][K]: the caller's copy of src, written share by share (null: nothing to write)
    float* rec2;
    void* stage;           // [M][K] of the activation dtype: the rounded input, kept for the caller
    int32_t K;
    int32_t in_op;
    int32_t op_count;
    uint32_t expect;       // contributions that complete an element of src
    uint32_t expect2;
    int32_t pad_[1];
    u64* norm;             // [CTAs][M] (sum of squares over the CTA's share of the row | 1 << 32), zero before the
                           // pass; null: every CTA reads whole rows for the norm itself
    u64 pad2_;
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
    int32_t NT;
    uint32_t nt_magic;
    int32_t pad_[2];
};
struct DsMiniPhase {
    int32_t op_first;      // index into the mini-op table
    int32_t op_count;
    int32_t pad_[2];
};
static_assert(sizeof(DsMiniOp) == 32 && sizeof(DsMiniPhase) == 16, "mini tables are copied as 16-byte items");
constexpr int DS_MINI_BYTES = 10240;

// What one CTA needs to know of one phase besides the phase record: worked out on the host, since it depends on
// nothing but the shapes (a single thread doing this in the kernel sat on every phase's critical path).
struct DsCtaPhase {
    int32_t total;                          // units of the phase dealt to this CTA
    int32_t n_slots;                        // staged slabs
    int32_t slab_of_slot[DS_MAX_SLOTS];     // the pair-slabs staged for the phase, ascending
    int32_t xoff[DS_MAX_PHASE_OPS];         // per op: (slot of its first slab) - (that slab): slab P sits in slot xoff + P
};
static_assert(sizeof(DsCtaPhase) == 64, "DsCtaPhase layout");

// A stretch of a buffer no phase reads: converted to float32 for the caller once the last phase is done.
struct DsTail {
    const u64* src;
    float* out;
    int32_t n;
    uint32_t expect;
    int32_t pad_[2];
};
static_assert(sizeof(DsTail) == 32, "DsTail layout");
constexpr int DS_TAIL_CHUNK = 2048;

struct DsArgs {
    const DsPhase* phases;
    const DsMiniPhase* mini_phases;   // n_phases entries, followed by
    const DsMiniOp* mini_ops;         // n_mini_ops entries (contiguous: one copy brings both)
    const DsTail* tails;
    const DsCtaPhase* ctab;           // [phase][CTA]
    u64 wait_ns;
    int n_phases;
    int n_mini_ops;
    int n_tails;
    int M;
    // the caller's rounded output: the tail chunks that convert [out_src, out_src + out_n) also write it (null: nobody does)
    void* out;
    const u64* out_src;
    int64_t out_n;
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
// Bounded wait on a shared-memory barrier; false when wait_ns passed.
__device__ __forceinline__ bool ds_mbar_wait(uint32_t bar, uint32_t parity, u64 wait_ns) {
    if (ds_mbar_try(bar, parity)) return true;
    const uint64_t t0 = ds_now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (ds_mbar_try(bar, parity)) return true;
        if (ds_now_ns() - t0 > wait_ns) return false;
    }
}
// Barrier among the consumer warps only (the copy warp never joins).
__device__ __forceinline__ void ds_consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(DS_CTHREADS) : "memory"); }
// The same barrier, returning the OR of `flag` over all consumer threads: every thread gets the same answer, so a
// decision to leave the phase loop is taken by all warps or by none (a flag read after a plain barrier could change
// between two threads' reads).
__device__ __forceinline__ bool ds_consumer_sync_or(int flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"(flag), "n"(DS_CTHREADS) : "memory");
    return r != 0;
}

// ---- packed sums ------------------------------------------------------------------
__device__ __forceinline__ u64 ds_pack(float v) {
    v = fminf(fmaxf(v, -DS_FIX_MAX), DS_FIX_MAX);
    return ((u64)__float2ll_rn(v * DS_FIX_ONE) << DS_CNT_BITS) + 1ull;
}
__device__ __forceinline__ float ds_unpack(u64 w) { return __ll2float_rn((long long)w >> DS_CNT_BITS) * (1.f / DS_FIX_ONE); }
__device__ __forceinline__ void ds_ld2(const u64* p, u64& a, u64& b) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ u64 ds_ld1(const u64* p) {
    u64 a;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(a) : "l"(p) : "memory");
    return a;
}
__device__ __forceinline__ void ds_red_add(u64* p, u64 v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
struct DsQuad { u64 w[4]; };
__device__ __forceinline__ void ds_ld_quad(const u64* p, DsQuad& q) { ds_ld2(p, q.w[0], q.w[1]); ds_ld2(p + 2, q.w[2], q.w[3]); }
__device__ __forceinline__ bool ds_quad_ready(const DsQuad& q, uint32_t expect) {
    return (uint32_t)(q.w[0] & DS_CNT_MASK) == expect && (uint32_t)(q.w[1] & DS_CNT_MASK) == expect &&
           (uint32_t)(q.w[2] & DS_CNT_MASK) == expect && (uint32_t)(q.w[3] & DS_CNT_MASK) == expect;
}
__device__ __forceinline__ float4 ds_quad_value(const DsQuad& q) {
    return make_float4(ds_unpack(q.w[0]), ds_unpack(q.w[1]), ds_unpack(q.w[2]), ds_unpack(q.w[3]));
}
// Re-reads four packed sums until all are complete; false (status raised) when the wait runs out or the grid gave up.
__device__ __noinline__ bool ds_quad_wait(const u64* p, DsQuad& q, uint32_t expect, u64 wait_ns, int* abort_flag) {
    const uint64_t t0 = ds_now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 16; ++i) {
            ds_ld_quad(p, q);
            if (ds_quad_ready(q, expect)) return true;
        }
        if (*reinterpret_cast<volatile int*>(&g_decode_status) != 0) { *abort_flag = 1; return false; }
        if (ds_now_ns() - t0 > wait_ns) { atomicCAS(&g_decode_status, 0, 1); *abort_flag = 1; return false; }
    }
}

// q holds a first reading of the four sums at p: true once they are complete (re-read as long as needed, into a
// copy of its own so that q itself can stay in registers).
__device__ __forceinline__ bool ds_quad_complete(const u64* p, DsQuad& q, uint32_t expect, u64 wait_ns, int* abort_flag) {
    if (ds_quad_ready(q, expect)) return true;
    DsQuad t;
    const bool ok = ds_quad_wait(p, t, expect, wait_ns, abort_flag);
    q = t;
    return ok;
}

// ---- the CTA's share of an op --------------------------------------------------------
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

// The copy stream's position: consumer w reads positions w, w + DS_WARPS, ... of the list made of the CTA's runs
// of the phase's ops, one after the other.
struct DsCursor {
    int ph, oi;            // phase (n_phases: past the end) and op inside it
    int pos, base;         // position in the phase's list; position at which op oi's run starts
    int a, len;            // op oi's run: first unit, number of units
    const uint8_t* frags;
    int ub;                // bytes per unit
    int NT;                // the op's row tiles and the magic number that divides by them
    uint32_t magic;
    uint32_t word0;        // op inside the phase | bits << 8, for the unit's descriptor
};
__device__ __forceinline__ void ds_cursor_load(DsCursor& c, const DsMiniPhase* mp, const DsMiniOp* mo) {
    const DsMiniOp op = mo[mp[c.ph].op_first + c.oi];
    int a, b;
    ds_cta_run((int)(op.q_bits & 0x0FFFFFFFu), (int)op.r_rot, a, b);
    c.a = a; c.len = b - a;
    c.frags = op.frags;
    c.ub = 2 * frag_bytes((int)(op.q_bits >> 28));
    c.NT = op.NT; c.magic = op.nt_magic;
    c.word0 = (uint32_t)c.oi | ((op.q_bits >> 28) << DS_DESC_BITS_SHIFT);
}
// Moves (ph, oi, base) on until op oi's run contains pos; a new phase starts again at position `lane`.
__device__ __forceinline__ void ds_cursor_settle(DsCursor& c, const DsMiniPhase* mp, const DsMiniOp* mo, int n_phases, int lane) {
    while (c.ph < n_phases && c.pos - c.base >= c.len) {
        c.base += c.len;
        if (++c.oi >= mp[c.ph].op_count) {
            ++c.ph; c.oi = 0; c.base = 0; c.pos = lane;
            if (c.ph >= n_phases) return;
        }
        ds_cursor_load(c, mp, mo);
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

// ---- shared memory ------------------------------------------------------------------
struct DsShared {
    alignas(128) uint8_t ring[DS_WARPS][DS_SLOTS][DS_SLOT_BYTES];
    alignas(128) uint8_t xs[DS_XS_BYTES];   // staged input slabs
    alignas(16) uint8_t mini[DS_MINI_BYTES];   // [DsMiniPhase x n_phases][DsMiniOp x n_mini_ops] when they fit
    alignas(16) DsPhase rec[2];             // descriptors of the current and the next phase
    alignas(8) uint64_t full[DS_WARPS][DS_SLOTS];    // copy landed
    alignas(8) uint64_t empty[DS_WARPS][DS_SLOTS];   // consumer has read the slot
    alignas(8) uint64_t rec_bar[2];
    alignas(16) uint4 desc[DS_WARPS][DS_SLOTS];      // the unit in the slot: (op | bits << 8, pair-slab, row tile, -)
    alignas(16) DsCtaPhase ctab[2];         // this CTA's tables of the current and the next phase
    float red[AQ_DECODE_MAX_M][DS_WARPS];
    float scale[AQ_DECODE_MAX_M];
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

// Cross-lane reduction of a unit's partial sums and one packed red.add per (token, row).  When `res` is given its
// value (complete, same shape as out) rides along.  Free of branches when res is null (bounds are predicates), so
// that the compiler can weave it into the next unit's arithmetic.
__device__ __forceinline__ void ds_red_add_if(u64* p, u64 v, bool on) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "@p red.relaxed.gpu.global.add.u64 [%0], %1;\n\t}"
        ::"l"(p), "l"(v), "r"((uint32_t)on) : "memory");
}
template <int MT>
__device__ __forceinline__ void ds_unit_commit(const float (&acc)[4], u64* out, const void* res, bool res_plain, int64_t ld, int row0,
                                               int N, int M, int lane) {
    const int g = lane >> 2, t = lane & 3;
    auto put = [&](int tok, int row, float v, bool lane_on) {
        const bool on = lane_on && tok < M && row < N;
        const int64_t o = (int64_t)tok * ld + row;
        u64 w = ds_pack(v);
        if (res != nullptr && on) {
            if (res_plain) w += ds_pack(__ldcg(reinterpret_cast<const float*>(res) + o)) - 1ull;
            else w += ds_ld1(reinterpret_cast<const u64*>(res) + o) & ~DS_CNT_MASK;
        }
        ds_red_add_if(out + o, w, on);
    };
    if constexpr (MT == 1) {
        const float v0 = acc[0] + acc[1], v1 = acc[2] + acc[3];
        float keep = (t & 1) ? v1 : v0;
        const float send = (t & 1) ? v0 : v1;
        keep += __shfl_xor_sync(0xffffffffu, send, 1);
        keep += __shfl_xor_sync(0xffffffffu, keep, 2);
        put(0, row0 + g + 8 * (t & 1), keep, t < 2);
    } else if constexpr (MT == 2) {
        float kA = (t & 1) ? acc[1] : acc[0], kB = (t & 1) ? acc[3] : acc[2];
        const float sA = (t & 1) ? acc[0] : acc[1], sB = (t & 1) ? acc[2] : acc[3];
        kA += __shfl_xor_sync(0xffffffffu, sA, 1);
        kB += __shfl_xor_sync(0xffffffffu, sB, 1);
        float v = (t & 2) ? kB : kA;
        const float s = (t & 2) ? kA : kB;
        v += __shfl_xor_sync(0xffffffffu, s, 2);
        put(t & 1, row0 + g + 8 * (t >> 1), v, true);
    } else if constexpr (MT == 4) {
        float c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) c[i] = acc[i] + __shfl_xor_sync(0xffffffffu, acc[i], 2);
        const int tk = 2 * (t & 1);
        const int hi = t >> 1;
        put(tk, row0 + g + 8 * hi, hi ? c[2] : c[0], true);
        put(tk + 1, row0 + g + 8 * hi, hi ? c[3] : c[1], true);
    } else {
        const int tk = 2 * t;
        put(tk, row0 + g, acc[0], true); put(tk, row0 + g + 8, acc[2], true);
        put(tk + 1, row0 + g, acc[1], true); put(tk + 1, row0 + g + 8, acc[3], true);
    }
}

// A unit whose sums have not left the warp yet: they do at the start of the next unit's arithmetic, where the
// shuffles, the conversion and the red.add hide behind tensor-core work instead of standing between two units.
struct DsPending {
    float acc[4];
    u64* out;
    int row0, N;
    bool on;
};
template <int MT>
__device__ __forceinline__ void ds_flush(DsPending& pd, int M, int lane) {
    if (pd.on) ds_unit_commit<MT>(pd.acc, pd.out, nullptr, false, pd.N, pd.row0, pd.N, M, lane);   // (pd.on is the same in every lane)
    pd.on = false;
}

// One unit: the previous unit's commit, then this unit's multiply-accumulate.
template <int BITS, int MT, bool BF16>
__device__ __forceinline__ void ds_unit_body(const uint8_t* unit, const uint8_t* xseg, XOperand<MT>& xo, DsPending& pd, int M, int lane,
                                             float (&acc)[4]) {
    ds_load_x_operand<MT, BF16>(xo, xseg, M, lane);
    const uint32_t xlane = ds_spread_lane_base(xseg, lane);
    ds_flush<MT>(pd, M, lane);
    unit_mac<BITS, MT, BF16, MT == 1>(unit, xo, lane, acc, xlane);
}

// ---- the kernel ---------------------------------------------------------------------
template <int MT, bool BF16>
__global__ void __launch_bounds__(DS_THREADS, 1) decode_stack_kernel(const DsArgs a) {
    extern __shared__ __align__(128) uint8_t ds_smem_raw[];
    DsShared& sh = *reinterpret_cast<DsShared*>(ds_smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int M = a.M;
    const int slab_bytes = ds_slab_bytes(M);
    const u64 wait_ns = a.wait_ns;

    if (threadIdx.x == 0) {
        sh.abort_flag = 0;
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
    const int mini_items = a.n_phases + 2 * a.n_mini_ops;   // in 16-byte pieces
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
        c.ph = a.n_phases; c.oi = 0; c.pos = 0; c.base = 0; c.a = 0; c.len = 0; c.frags = nullptr; c.ub = 0;
        c.NT = 1; c.magic = 0; c.word0 = 0;
        if (lane < DS_WARPS && a.n_phases > 0) {
            c.ph = 0; c.pos = lane;
            ds_cursor_load(c, mp, mo);
            ds_cursor_settle(c, mp, mo, a.n_phases, lane);
        }
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
                    const uint32_t u = (uint32_t)(c.a + (c.pos - c.base));
                    int Pk = c.magic ? (int)__umulhi(u, c.magic) : (int)u;   // u / NT (no magic: NT = 1)
                    int R = (int)u - Pk * c.NT;
                    if (R < 0) { --Pk; R += c.NT; }
                    // (ordered before the copy's arrival by the release of expect_tx)
                    sh.desc[lane][slot] = make_uint4(c.word0, (uint32_t)Pk, (uint32_t)R, 0u);
                    const uint32_t bar = ds_smem(&sh.full[lane][slot]);
                    ds_expect_tx(bar, (uint32_t)c.ub);
                    ds_bulk_load(ds_smem(&sh.ring[lane][slot][0]), c.frags + (int64_t)u * c.ub, (uint32_t)c.ub, bar, pol);
                    ++iseq;
                    c.pos += DS_WARPS;
                    ds_cursor_settle(c, mp, mo, a.n_phases, lane);
                    moved = true;
                }
            }
            if (!__any_sync(0xffffffffu, active)) break;
            if (__any_sync(0xffffffffu, moved)) { idle = 0; continue; }
            __nanosleep(200);   // a consumer needs about half a microsecond per unit: no need to spin on its barriers
            if ((++idle & 255u) == 0) {   // nothing to do for a while: stop if the CTA gave up, or after the time limit
                if (*reinterpret_cast<volatile int*>(&sh.abort_flag)) break;
                const uint64_t t = ds_now_ns();
                if (idle == 256u) t_progress = t;
                else if (t - t_progress > 2 * wait_ns) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; break; }
            }
        }
        return;
    }

    // ================= consumer warps =================
    auto fetch_record = [&](int q) {   // the phase's record and this CTA's tables for it, on one barrier
        const uint32_t bar = ds_smem(&sh.rec_bar[q & 1]);
        ds_expect_tx(bar, (uint32_t)(sizeof(DsPhase) + sizeof(DsCtaPhase)));
        ds_bulk_load(ds_smem(&sh.rec[q & 1]), a.phases + q, (uint32_t)sizeof(DsPhase), bar, pol_keep);
        ds_bulk_load(ds_smem(&sh.ctab[q & 1]), a.ctab + (size_t)q * gridDim.x + blockIdx.x, (uint32_t)sizeof(DsCtaPhase), bar, pol_keep);
    };
    if (threadIdx.x == 0) {
        if (a.n_phases > 0) fetch_record(0);
        if (a.n_phases > 1) fetch_record(1);
    }

    uint32_t cslot = 0, cparity = 0;   // next ring slot to consume and the parity of its `full` barrier
    bool dead = false;                 // this warp gave up on a wait
    XOperand<MT> xo;
    DsPending pd;
    pd.on = false; pd.out = nullptr; pd.row0 = 0; pd.N = 0;
    pd.acc[0] = pd.acc[1] = pd.acc[2] = pd.acc[3] = 0.f;

#pragma unroll 1
    for (int ph = 0; ph < a.n_phases; ++ph) {
        const int pb = ph & 1;
        const DsPhase& P = sh.rec[pb];
        const DsCtaPhase& C = sh.ctab[pb];
        // -- the phase's descriptors (fetched one phase ahead) --
        if (!ds_mbar_wait(ds_smem(&sh.rec_bar[pb]), (uint32_t)(ph >> 1) & 1u, wait_ns)) {
            atomicCAS(&g_decode_status, 0, 2);
            sh.abort_flag = 1;
        }
        // every warp is through with phase ph - 1: the staged slabs and its record slot are free
        if (ds_consumer_sync_or(*reinterpret_cast<volatile int*>(&sh.abort_flag))) break;
        if (threadIdx.x == 0 && ph >= 1 && ph + 1 < a.n_phases) fetch_record(ph + 1);

        // -- form the rounded input vector: slabs this CTA reads -> shared memory, its share -> workspace --
        {
            const int n_slots = C.n_slots;
            const int q4 = P.K >> 2;                                  // groups of 4 elements per token
            const int g0 = (int)(((int64_t)q4 * blockIdx.x) / gridDim.x), g1 = (int)(((int64_t)q4 * (blockIdx.x + 1)) / gridDim.x);
            uint16_t* stage_out = reinterpret_cast<uint16_t*>(P.stage);
            const uint32_t expect = P.expect, expect2 = P.expect2;
            uint32_t spins = 0;
            uint64_t t_wait0 = 0;
            // after a round of readings that found something incomplete: true when the wait has to end
            auto give_up = [&]() -> bool {
                if ((++spins & 7u) != 0) return false;
                if (*reinterpret_cast<volatile int*>(&g_decode_status) != 0) { sh.abort_flag = 1; return true; }
                const uint64_t t = ds_now_ns();
                if (t_wait0 == 0) t_wait0 = t;
                if (t - t_wait0 > wait_ns) { atomicCAS(&g_decode_status, 0, 1); sh.abort_flag = 1; return true; }
                return false;
            };
            // four consecutive source elements (group i4 of token m), complete; zeros after a failed wait
            auto source4 = [&](const u64* p, const float* pf, uint32_t ex, int m, int i4) -> float4 {
                const int64_t o = (int64_t)m * P.K + 4 * (int64_t)i4;
                if (p == nullptr) return __ldcg(reinterpret_cast<const float4*>(pf + o));
                DsQuad q;
                for (;;) {
                    ds_ld_quad(p + o, q);
                    if (ds_quad_ready(q, ex)) return ds_quad_value(q);
                    if (give_up()) return make_float4(0.f, 0.f, 0.f, 0.f);
                }
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
                if (rec) *reinterpret_cast<uint2*>(stage_out + (int64_t)m * P.K + i4 * 4) = r;
            };
            if (P.in_op == AQ_IN_RMSNORM && MT == 1 && q4 <= DS_RMS_HOLD * DS_CTHREADS) {
                // one token, row held in registers: one trip to L2 once the row is complete (all of a thread's readings
                // go out together and are repeated together until every one of them is complete)
                float4 v[DS_RMS_HOLD];
                int slabs[DS_MAX_SLOTS];
#pragma unroll
                for (int x = 0; x < DS_MAX_SLOTS; ++x) slabs[x] = C.slab_of_slot[x];
                if (P.src != nullptr) {
                    DsQuad q[DS_RMS_HOLD];
                    for (;;) {
                        bool ready = true;
#pragma unroll
                        for (int n = 0; n < DS_RMS_HOLD; ++n) {
                            const int i4 = threadIdx.x + n * DS_CTHREADS;
                            if (i4 < q4) ds_ld_quad(P.src + 4 * (int64_t)i4, q[n]);
                        }
#pragma unroll
                        for (int n = 0; n < DS_RMS_HOLD; ++n) {
                            const int i4 = threadIdx.x + n * DS_CTHREADS;
                            if (i4 < q4) ready = ready && ds_quad_ready(q[n], expect);
                        }
                        if (ready || give_up()) break;
                    }
                    const bool failed = *reinterpret_cast<volatile int*>(&sh.abort_flag) != 0;
#pragma unroll
                    for (int n = 0; n < DS_RMS_HOLD; ++n) {
                        const int i4 = threadIdx.x + n * DS_CTHREADS;
                        v[n] = (i4 < q4 && !failed) ? ds_quad_value(q[n]) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                } else {
#pragma unroll
                    for (int n = 0; n < DS_RMS_HOLD; ++n) {
                        const int i4 = threadIdx.x + n * DS_CTHREADS;
                        v[n] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (i4 < q4) v[n] = __ldcg(reinterpret_cast<const float4*>(P.src_f) + i4);
                    }
                }
                __syncwarp();
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
                    if (n * DS_CTHREADS < q4) {   // the same for every thread: warps stay whole
                        const bool mine = i4 >= g0 && i4 < g1;
                        if (mine && P.rec) reinterpret_cast<float4*>(P.rec)[i4] = v[n];
                        const int slab = i4 >> 6;
                        int sl = -1;
#pragma unroll
                        for (int x = 0; x < DS_MAX_SLOTS; ++x) sl = (x < n_slots && slabs[x] == slab) ? x : sl;
                        // most of the row is read for its sum of squares only: a warp (its 32 groups are half a slab)
                        // whose groups are neither staged nor part of this CTA's share of the caller's copy rounds nothing
                        const int wg = i4 - lane;
                        if (sl >= 0 || (wg < g1 && wg + 32 > g0))
                            place(sl >= 0 ? sh.xs + (size_t)sl * slab_bytes : nullptr, 0, i4,
                                  make_float4(v[n].x * scale, v[n].y * scale, v[n].z * scale, v[n].w * scale), mine);
                    }
                }
            } else {
                bool normed = false;
                if constexpr (MT > 1) {
                if (P.in_op == AQ_IN_RMSNORM && P.norm != nullptr) {
                    // Row norms from shares: this CTA sums the squares of its share of every token row (one group of
                    // four per thread, one trip to L2), publishes the M partial sums as (float | 1 << 32) words, and
                    // gathers every CTA's words; all sums run in a fixed order, so every CTA gets the same norms.
                    float* part = &sh.red[0][0];
                    float* gathered = reinterpret_cast<float*>(sh.xs);   // [CTA][M]: the slab area is not in use yet
                    const int share = g1 - g0, n_items = share * M;      // (the host made sure n_items fits sh.red)
                    if ((int)threadIdx.x < n_items) {
                        const int m = (int)threadIdx.x / share, i4 = g0 + (int)threadIdx.x - m * share;
                        const float4 v = source4(P.src, P.src_f, expect, m, i4);
                        part[threadIdx.x] = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, v.w * v.w)));
                    }
                    ds_consumer_sync();
                    if ((int)threadIdx.x < M) {
                        float ss = 0.f;
                        for (int j = 0; j < share; ++j) ss += part[threadIdx.x * share + j];
                        const u64 w = (u64)__float_as_uint(ss) | (1ull << 32);
                        asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(P.norm + (size_t)blockIdx.x * M + threadIdx.x), "l"(w) : "memory");
                    }
                    const int n_words = (int)gridDim.x * M;
                    for (int it = threadIdx.x; it < n_words; it += DS_CTHREADS) {
                        u64 w;
                        for (;;) {
                            w = ds_ld1(P.norm + it);
                            if ((w >> 32) != 0 || give_up()) break;
                        }
                        gathered[it] = __uint_as_float((uint32_t)w);
                    }
                    ds_consumer_sync();
                    if ((int)threadIdx.x < M) {
                        float tot = 0.f;
                        for (int c = 0; c < (int)gridDim.x; ++c) tot += gathered[c * M + threadIdx.x];
                        sh.scale[threadIdx.x] = rsqrtf(tot / (float)P.K + 1e-6f);
                    }
                    ds_consumer_sync();
                    normed = true;
                }
                }
                if (P.in_op == AQ_IN_RMSNORM && !normed) {
                    for (int m = 0; m < M; ++m) {
                        float ss = 0.f;
                        for (int i = threadIdx.x; i < q4; i += DS_CTHREADS) {
                            const float4 v = source4(P.src, P.src_f, expect, m, i);
                            ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
                        }
                        __syncwarp();
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
                // one list of work: first the slabs this CTA reads, then its share of the caller's copies
                const int per_slab = 64 * M;
                const int n_a = n_slots * per_slab;
                const int n_b = (g1 - g0) * M;
                const int n_all = n_a + n_b;
                const bool two = (P.in_op == AQ_IN_SILU_MUL);
                for (int it0 = 0; it0 < n_all; it0 += DS_CTHREADS) {
                    const int it = it0 + threadIdx.x;
                    int m = 0, i4 = 0;
                    bool valid = false;
                    uint8_t* sl = nullptr;
                    if (it < n_a) {
                        const int s_ = it / per_slab, w = it - s_ * per_slab;
                        m = w >> 6;
                        i4 = C.slab_of_slot[s_] * 64 + (w & 63);
                        sl = sh.xs + (size_t)s_ * slab_bytes;
                        valid = i4 < q4;
                    } else if (it < n_all) {
                        const int w = it - n_a;
                        m = w / (g1 - g0);
                        i4 = g0 + w - m * (g1 - g0);
                        valid = true;
                    }
                    const bool share = it >= n_a;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (valid) {
                        // both sources' readings go out together and are repeated together until complete
                        const int64_t o = (int64_t)m * P.K + 4 * (int64_t)i4;
                        float4 s = make_float4(0.f, 0.f, 0.f, 0.f), t = s;
                        DsQuad qa, qb;
                        for (;;) {
                            if (P.src) ds_ld_quad(P.src + o, qa);
                            else s = __ldcg(reinterpret_cast<const float4*>(P.src_f + o));
                            if (two) {
                                if (P.src2) ds_ld_quad(P.src2 + o, qb);
                                else t = __ldcg(reinterpret_cast<const float4*>(P.src2_f + o));
                            }
                            bool ready = true;
                            if (P.src) ready = ds_quad_ready(qa, expect);
                            if (two && P.src2) ready = ready && ds_quad_ready(qb, expect2);
                            if (ready) {
                                if (P.src) s = ds_quad_value(qa);
                                if (two && P.src2) t = ds_quad_value(qb);
                                break;
                            }
                            if (give_up()) { s = t = make_float4(0.f, 0.f, 0.f, 0.f); break; }
                        }
                        if (share && P.rec) *reinterpret_cast<float4*>(P.rec + o) = s;
                        if (two) {
                            if (share && P.rec2) *reinterpret_cast<float4*>(P.rec2 + o) = t;
                            v = make_float4(ds_silu_mul(s.x, t.x), ds_silu_mul(s.y, t.y), ds_silu_mul(s.z, t.z), ds_silu_mul(s.w, t.w));
                        } else {
                            const float sc = (P.in_op == AQ_IN_RMSNORM) ? sh.scale[m] : 1.f;
                            v = make_float4(s.x * sc, s.y * sc, s.z * sc, s.w * sc);
                        }
                    }
                    __syncwarp();
                    if (it0 + (int)(threadIdx.x - lane) < n_a) {
                        place(sl, m, i4, v, false);              // n_a is a multiple of 32: the whole warp is inside the slab items
                    } else if (valid) {
                        float sum;
                        const uint2 r = ds_round4<BF16>(v, &sum);
                        *reinterpret_cast<uint2*>(stage_out + (int64_t)m * P.K + i4 * 4) = r;
                    }
                }
            }
        }
        if (ds_consumer_sync_or(*reinterpret_cast<volatile int*>(&sh.abort_flag))) break;

        // -- consume this warp's units of the phase: positions warp, warp + 15, ... of the CTA's list --
        const int total = C.total;
#pragma unroll 1
        for (int pos = warp; pos < total && !dead; pos += DS_WARPS) {
            dead = __any_sync(0xffffffffu, !ds_mbar_wait(ds_smem(&sh.full[warp][cslot]), cparity, wait_ns));
            if (dead) {
                if (lane == 0) { atomicCAS(&g_decode_status, 0, 2); sh.abort_flag = 1; }
                break;
            }
            const uint4 ds = sh.desc[warp][cslot];
            const uint8_t* xseg = sh.xs + (size_t)(C.xoff[ds.x & 0xFFu] + (int)ds.y) * slab_bytes;
            const uint8_t* unit = &sh.ring[warp][cslot][0];
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const int bits = (int)(ds.x >> DS_DESC_BITS_SHIFT);
            if (bits == 2) ds_unit_body<2, MT, BF16>(unit, xseg, xo, pd, M, lane, acc);
            else if (bits == 3) ds_unit_body<3, MT, BF16>(unit, xseg, xo, pd, M, lane, acc);
            else ds_unit_body<4, MT, BF16>(unit, xseg, xo, pd, M, lane, acc);
            __syncwarp();        // every lane has read its part of the slot
            if (lane == 0) ds_mbar_arrive(ds_smem(&sh.empty[warp][cslot]));
            if (++cslot == DS_SLOTS) { cslot = 0; cparity ^= 1u; }
            const DsOp& op = P.ops[ds.x & 0xFFu];
            if (ds.y == 0 && op.res != nullptr) {   // (rare: the residual rides along with the first k-slab's sums)
                ds_unit_commit<MT>(acc, op.dst, op.res, (op.bits & DS_RES_PLAIN) != 0, op.N, (int)ds.z * 16, op.N, M, lane);
            } else {
                pd.acc[0] = acc[0]; pd.acc[1] = acc[1]; pd.acc[2] = acc[2]; pd.acc[3] = acc[3];
                pd.out = op.dst; pd.N = op.N; pd.row0 = (int)ds.z * 16; pd.on = true;
            }
        }
        ds_flush<MT>(pd, M, lane);   // nothing of this phase stays behind: other CTAs wait for these sums
    }

    // -- buffers no phase reads (and the last outputs): float32 copies for the caller, one chunk per warp --
    if (*reinterpret_cast<volatile int*>(&sh.abort_flag) == 0) {
#pragma unroll 1
        for (int e = (int)blockIdx.x * DS_WARPS + warp; e < a.n_tails; e += (int)gridDim.x * DS_WARPS) {
            const DsTail T = a.tails[e];
            bool ok = true;
            for (int i = lane * 4; i < T.n && ok; i += 128) {      // n is a multiple of 4
                DsQuad q;
                ds_ld_quad(T.src + i, q);
                if (!ds_quad_complete(T.src + i, q, T.expect, wait_ns, &sh.abort_flag)) ok = false;
                else {
                    const float4 v = ds_quad_value(q);
                    *reinterpret_cast<float4*>(T.out + i) = v;
                    if (a.out != nullptr) {
                        const int64_t o = (T.src - a.out_src) + i;
                        float unused;
                        if (o >= 0 && o < a.out_n) *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.out) + o) = ds_round4<BF16>(v, &unused);
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
    uint8_t* dev = nullptr;       // [phase records][mini phases, mini ops][tail chunks][per-CTA phase tables]
    size_t phases_bytes = 0, mini_bytes = 0, tail_bytes = 0, ctab_bytes = 0;
    int n_mini_ops = 0;
    int n_phases = 0;
    int n_tails = 0;
    int device = 0;
    bool pinned = false;          // recorded into a CUDA graph: its device tables must outlive the plan cache's turnover
    std::vector<char> in_tails;   // per buffer: the tail chunks convert it (no phase reads it)
    uint64_t stamp = 0;
};

std::mutex g_plan_mutex;
std::vector<DecodePlan*> g_plans;
uint64_t g_plan_clock = 0;
constexpr size_t MAX_PLANS = 256;   // (a program with attention between its linears is one plan per stretch of linears)
u64 g_wait_ns = DS_WAIT_NS_DEFAULT;
bool g_hold = false;          // testing: the first packed input of a program expects one contribution too many

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
// read the same input vector) and the list of buffers nobody reads.  False when the program
// does not fit this kernel.
bool build_decode_tables(const aq_stack_t* p, const StackPlan& plan, int M, int n_cta, uint8_t* ws,
                         std::vector<DsPhase>& phases, std::vector<DsTail>& tails, std::vector<DsCtaPhase>& ctab,
                         std::vector<char>& in_tails, int op_first, int op_end) {
    if (M < 1 || M > AQ_DECODE_MAX_M || p->n_ops > 32000 || plan.pk_off.empty()) return false;
    phases.clear();
    tails.clear();
    ctab.clear();
    std::vector<int> writer(p->n_bufs, -1);         // op that writes the buffer
    std::vector<char> whole(p->n_bufs, 0);          // every CTA has seen the whole buffer complete (a normalised input)
    std::vector<char> recorded(p->n_bufs, 0);       // some phase writes the caller's float32 copy
    auto packed = [&](int b) { return reinterpret_cast<u64*>(ws + plan.pk_off[b]); };
    auto plain = [&](int b) { return reinterpret_cast<float*>(ws + plan.buf_off[b]); };
    auto expect_of = [&](int b) { return (uint32_t)p->ops[writer[b]].w->KP; };
    // a launch that runs ops [op_first, op_end) of the program: what earlier launches of the pass wrote is complete (as
    // packed sums and as the caller's float32 copy) before this one starts
    for (int i = 0; i < op_first; ++i) {
        writer[p->ops[i].dst] = i;
        whole[p->ops[i].dst] = 1;
        recorded[p->ops[i].dst] = 1;
    }
    int rot = 0;   // where the next op's odd units start
    bool hold = g_hold;
    const int n_ph = (int)plan.phase_first.size();
    for (int ph = 0; ph < n_ph; ++ph) {
        const int pfirst = plan.phase_first[ph];
        const int plast = (ph + 1 < n_ph) ? plan.phase_first[ph + 1] : p->n_ops;
        if (pfirst < op_first || pfirst >= op_end) continue;
        if (plast > op_end) return false;   // (a launch ends where a phase ends)
        for (int first = pfirst; first < plast;) {
            // as many of the phase's ops (at most DS_MAX_PHASE_OPS) as leave every CTA's staged slabs inside the
            // shared-memory buffer; the rest of them form a further phase with the same input
            const aq_stack_op_t& f = p->ops[first];
            const int64_t K = p->buf_width[f.src];
            if (K > (int64_t)1 << 24 || n_cta > 32767) return false;
            DsPhase P;
            std::vector<DsCtaPhase> ctab_phase;
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
                    if (off + nu > (int64_t)1 << 26 || h->KP > DS_MAX_CONTRIB) { ok = false; break; }
                    d.N = (int32_t)h->N; d.NT = h->NT; d.bits = h->bits;
                    d.nt_magic = h->NT > 1 ? (uint32_t)(((uint64_t)1 << 32) / (uint64_t)h->NT + 1) : 0u;
                    d.units_q = (int32_t)(nu / n_cta);
                    d.units_r_rot = (int32_t)(nu % n_cta) | (r2 << 16);
                    r2 = (int)((r2 + nu % n_cta) % n_cta);
                    off += nu;
                }
                std::vector<DsCtaPhase> tab(ok ? n_cta : 0);
                for (int c = 0; c < n_cta && ok; ++c) {
                    // the slabs CTA c reads for the phase, ascending, and where each op's first slab sits among them
                    DsCtaPhase& T = tab[c];
                    memset(&T, 0, sizeof(T));
                    std::vector<int64_t> need;
                    int64_t lo[DS_MAX_PHASE_OPS];
                    for (int i = 0; i < count; ++i) {
                        const int64_t q = P.ops[i].units_q, r = P.ops[i].units_r_rot & 0xFFFF, ro = P.ops[i].units_r_rot >> 16;
                        const int64_t sl = (c + ro) % n_cta;
                        const int64_t u0 = q * sl + std::min(sl, r), u1 = u0 + q + (sl < r ? 1 : 0);
                        T.total += (int32_t)(u1 - u0);
                        lo[i] = -1;
                        if (u0 < u1) {
                            lo[i] = u0 / P.ops[i].NT;
                            for (int64_t x = u0 / P.ops[i].NT; x <= (u1 - 1) / P.ops[i].NT; ++x) need.push_back(x);
                        }
                    }
                    std::sort(need.begin(), need.end());
                    need.erase(std::unique(need.begin(), need.end()), need.end());
                    const int64_t slabs = (int64_t)need.size();
                    if (slabs > DS_MAX_SLOTS || slabs * ds_slab_bytes(M) > DS_XS_BYTES) { ok = false; break; }
                    T.n_slots = (int32_t)slabs;
                    for (int64_t x = 0; x < slabs; ++x) T.slab_of_slot[x] = (int32_t)need[x];
                    for (int i = 0; i < count; ++i) {
                        if (lo[i] < 0) continue;
                        const int64_t slot = std::lower_bound(need.begin(), need.end(), lo[i]) - need.begin();
                        T.xoff[i] = (int32_t)(slot - lo[i]);   // (the op's slabs are consecutive, so are their slots)
                    }
                }
                if (ok) ctab_phase = tab;
                if (ok) { rot_after = r2; break; }
            }
            if (count < 1) return false;
            const int last = first + count;
            rot = rot_after;
            auto source = [&](int b, const u64*& sp, const float*& sf, float*& rec, uint32_t& ex) {
                if (writer[b] < 0) { sp = nullptr; sf = plain(b); rec = nullptr; ex = 0; return; }   // the program input
                sp = packed(b); sf = nullptr; ex = expect_of(b);
                rec = recorded[b] ? nullptr : plain(b);
                recorded[b] = 1;
            };
            source(f.src, P.src, P.src_f, P.rec, P.expect);
            if (hold && P.src) { P.expect += 1; hold = false; }   // (a count no row reaches: every CTA's wait runs out)
            if (f.in_op == AQ_IN_SILU_MUL) source(f.src2, P.src2, P.src2_f, P.rec2, P.expect2);
            if (f.in_op == AQ_IN_RMSNORM) whole[f.src] = 1;
            P.stage = ws + plan.in_off[first];
            P.K = (int32_t)K; P.in_op = f.in_op; P.op_count = count;
            // several tokens: the row norms come from per-CTA partial sums exchanged through the workspace (whole
            // rows read by every CTA are 8 M K bytes per CTA from the same lines of L2); the partial sums of a CTA's
            // share are added up through sh.red, hence the bound on the share
            P.norm = nullptr;
            if (f.in_op == AQ_IN_RMSNORM && M >= 3 && !plan.nm_off.empty() && plan.nm_off[pfirst] != 0 && n_cta <= AQ_NORM_MAX_CTAS &&
                (int64_t)M * ((K / 4 + n_cta - 1) / n_cta + 1) <= (int64_t)AQ_DECODE_MAX_M * DS_WARPS)
                P.norm = reinterpret_cast<u64*>(ws + plan.nm_off[pfirst]);
            for (int i = first; i < last; ++i) {
                const aq_stack_op_t& o = p->ops[i];
                DsOp& d = P.ops[i - first];
                d.frags = o.w->frags;
                d.dst = packed(o.dst);
                d.res = nullptr;
                if (o.out_op == AQ_OUT_ADD) {
                    // the residual is read without a wait: it must be complete for every CTA when the phase starts,
                    // i.e. the program input (plain float32) or an input that every CTA has already read as a whole
                    // (a normalised one)
                    if (writer[o.res] < 0) { d.res = plain(o.res); d.bits |= DS_RES_PLAIN; }
                    else if (whole[o.res]) d.res = packed(o.res);
                    else return false;
                }
            }
            for (int i = first; i < last; ++i) writer[p->ops[i].dst] = i;
            phases.push_back(P);
            ctab.insert(ctab.end(), ctab_phase.begin(), ctab_phase.end());
            first = last;
        }
    }
    // what no phase has copied out for the caller
    in_tails.assign(p->n_bufs, 0);
    for (int b = 1; b < p->n_bufs; ++b) {
        if (writer[b] < op_first || recorded[b]) continue;   // (written by this launch, read by none of its phases)
        const int64_t n = (int64_t)M * p->buf_width[b];
        if (n % 4) return false;
        in_tails[b] = 1;
        for (int64_t i = 0; i < n; i += DS_TAIL_CHUNK) {
            DsTail t;
            memset(&t, 0, sizeof(t));
            t.src = packed(b) + i; t.out = plain(b) + i;
            t.n = (int32_t)std::min<int64_t>(DS_TAIL_CHUNK, n - i);
            t.expect = expect_of(b);
            tails.push_back(t);
        }
    }
    return true;
}

template <int MT, bool BF16>
static cudaError_t launch_ds(const DsArgs& a, int grid, cudaStream_t s) {
    auto kern = decode_stack_kernel<MT, BF16>;
    static PerDeviceOnce configured;
    {
        const int rc = configured.run(current_device(), [&] {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DsShared));
            if (e != cudaSuccess) return (int)e;
            int per_sm = 0;
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, DS_THREADS, sizeof(DsShared));
            if (e != cudaSuccess) return (int)e;
            return per_sm < 1 ? (int)cudaErrorCooperativeLaunchTooLarge : 0;
        });
        if (rc != 0) return rc < 0 ? cudaErrorInvalidDevice : (cudaError_t)rc;
    }
    DsArgs args = a;
    void* params[1] = {&args};
    cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3((unsigned)grid), dim3(DS_THREADS), params,
                                                sizeof(DsShared), s);
    if (e == cudaSuccess) count_launch();
    return e;
}

// The part of a plan's key that depends on the program alone (ops, their matrices, buffer widths).
void decode_program_key(const aq_stack_t* p, std::vector<uint8_t>& key) {
    key.reserve(key.size() + (size_t)p->n_ops * (sizeof(aq_stack_op_t) + 8) + (size_t)p->n_bufs * 8 + 16);
    key_put(key, p->n_ops); key_put(key, p->n_bufs);
    for (int i = 0; i < p->n_ops; ++i) {
        key_put(key, p->ops[i]);
        key_put(key, p->ops[i].w->frags);
    }
    for (int b = 0; b < p->n_bufs; ++b) key_put(key, p->buf_width[b]);
}

int launch_decode_stack(const aq_stack_t* p, const StackPlan& plan, int M, aq_dtype_t dt, uint8_t* ws, cudaStream_t s,
                        cudaError_t* err, void* out, int out_buf, bool* wrote_out, int op_first, int op_end, bool clear,
                        const std::vector<uint8_t>* program_key) {
    *err = cudaSuccess;
    *wrote_out = false;
    if (op_end < 0) op_end = p->n_ops;
    const int grid = sm_count();
    const int dev = current_device();
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
    const bool capturing = (cap != cudaStreamCaptureStatusNone);
    // key: everything the device tables are computed from
    std::vector<uint8_t> key;
    key_put(key, M); key_put(key, dev); key_put(key, grid); key_put(key, ws); key_put(key, op_first); key_put(key, op_end);
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    key_put(key, g_hold);
    if (program_key) key.insert(key.end(), program_key->begin(), program_key->end());   // (built once for all the launches of a pass)
    else decode_program_key(p, key);

    DecodePlan* dp = nullptr;
    for (DecodePlan* q : g_plans)
        if (q->key == key) { dp = q; break; }
    if (!dp) {
        if (capturing) return 1;   // tables are built (allocation, synchronous copies) by an eager call only
        std::vector<DsPhase> phases;
        std::vector<DsTail> tails;
        std::vector<DsCtaPhase> ctab;
        std::vector<char> in_tails;
        if (!build_decode_tables(p, plan, M, grid, ws, phases, tails, ctab, in_tails, op_first, op_end)) return 1;
        if (g_plans.size() >= MAX_PLANS) {   // make room: the oldest plan no graph refers to
            size_t oldest = g_plans.size();
            for (size_t i = 0; i < g_plans.size(); ++i)
                if (!g_plans[i]->pinned && (oldest == g_plans.size() || g_plans[i]->stamp < g_plans[oldest]->stamp)) oldest = i;
            if (oldest == g_plans.size()) return 1;   // all pinned: this program runs op by op
            drop_plan(g_plans[oldest]);
            g_plans.erase(g_plans.begin() + oldest);
        }
        dp = new DecodePlan();
        dp->key = key;
        dp->device = dev;
        for (int i = 0; i < p->n_ops; ++i) dp->handles.push_back(p->ops[i].w);
        dp->in_tails = in_tails;
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
                memset(&mop, 0, sizeof(mop));
                mop.NT = phases[i].ops[j].NT; mop.nt_magic = phases[i].ops[j].nt_magic;
                mop.frags = phases[i].ops[j].frags;
                mop.q_bits = (uint32_t)phases[i].ops[j].units_q | ((uint32_t)(phases[i].ops[j].bits & 0xFF) << 28);
                mop.r_rot = (uint32_t)phases[i].ops[j].units_r_rot;
                const uint8_t* b = reinterpret_cast<const uint8_t*>(&mop);
                mini.insert(mini.end(), b, b + sizeof(mop));
            }
        dp->mini_bytes = (mini.size() + 255) / 256 * 256;
        dp->tail_bytes = (tails.size() * sizeof(DsTail) + 255) / 256 * 256;
        dp->n_phases = (int)phases.size();
        dp->n_tails = (int)tails.size();
        dp->ctab_bytes = (ctab.size() * sizeof(DsCtaPhase) + 255) / 256 * 256;
        cudaError_t e = cudaMalloc(&dp->dev, dp->phases_bytes + dp->mini_bytes + dp->tail_bytes + dp->ctab_bytes + 256);
        if (e == cudaSuccess) e = cudaMemcpy(dp->dev, phases.data(), phases.size() * sizeof(DsPhase), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(dp->dev + dp->phases_bytes, mini.data(), mini.size(), cudaMemcpyHostToDevice);
        if (e == cudaSuccess && !tails.empty())
            e = cudaMemcpy(dp->dev + dp->phases_bytes + dp->mini_bytes, tails.data(), tails.size() * sizeof(DsTail), cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(dp->dev + dp->phases_bytes + dp->mini_bytes + dp->tail_bytes, ctab.data(), ctab.size() * sizeof(DsCtaPhase),
                           cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { cudaGetLastError(); drop_plan(dp); *err = e; return -1; }
        g_plans.push_back(dp);
    }
    dp->stamp = ++g_plan_clock;
    if (capturing) dp->pinned = true;

    DsArgs a;
    a.phases = reinterpret_cast<const DsPhase*>(dp->dev);
    a.mini_phases = reinterpret_cast<const DsMiniPhase*>(dp->dev + dp->phases_bytes);
    a.mini_ops = reinterpret_cast<const DsMiniOp*>(dp->dev + dp->phases_bytes + (size_t)dp->n_phases * sizeof(DsMiniPhase));
    a.tails = reinterpret_cast<const DsTail*>(dp->dev + dp->phases_bytes + dp->mini_bytes);
    a.ctab = reinterpret_cast<const DsCtaPhase*>(dp->dev + dp->phases_bytes + dp->mini_bytes + dp->tail_bytes);
    a.n_mini_ops = dp->n_mini_ops;
    a.n_phases = dp->n_phases;
    a.n_tails = dp->n_tails;
    a.M = M;
    a.wait_ns = g_wait_ns;
    a.out = nullptr; a.out_src = nullptr; a.out_n = 0;
    if (out != nullptr && out_buf >= 1 && out_buf < p->n_bufs && dp->in_tails[out_buf] &&
        (reinterpret_cast<uintptr_t>(out) & 7u) == 0) {
        a.out = out;
        a.out_src = reinterpret_cast<const u64*>(ws + plan.pk_off[out_buf]);
        a.out_n = (int64_t)M * p->buf_width[out_buf];
        *wrote_out = true;
    }
    // the packed sums start from zero (once per pass: a later launch of the same pass reads what the earlier ones left)
    cudaError_t e = clear ? cudaMemsetAsync(ws + plan.pk_begin, 0, plan.pk_end - plan.pk_begin, s) : cudaSuccess;
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

void set_decode_hold(bool on) {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    g_hold = on;
}

void set_decode_wait_ns(unsigned long long ns) {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    g_wait_ns = ns ? ns : DS_WAIT_NS_DEFAULT;
}

}  // namespace aq
