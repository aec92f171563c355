// Prefill path (M > 8): dequantise-to-half + tensor-core GEMM on the packed
// weights, out[m][n] = (res[m][n]) + sum_k x[m][k] w_hat[n][k]  (Appendix D:
// dequantise on the fly inside the low-bit kernel; Eq. 1 for the decode).
//
// Both operands enter the tensor core as binary16: a dequantised weight is
// fp16(scale * q + min) (one half-precision FMA, 11 significant bits, so the
// worst case of the product sum is 2^-11 sum|x w|).  bfloat16 activations are
// widened to binary16 by the caller of this kernel (exact wherever the value is
// inside binary16's range; a token row that is not comes scaled by a power of
// two, undone in the epilogue through tok_scale).
//
// Bound: tensor cores (dense contraction, 2 M flops per weight).  tcgen05
// UMMA with the accumulators in TMEM:
//   A (M side, 128)   = weight rows, dequantised by eight warps from the packed
//                       fragments into the K-major 128-byte-swizzled shared
//                       memory layout the instruction reads,
//   B (N side, <=256) = tokens, fetched by TMA with the same swizzle,
//   D[128 lanes][tokens] fp32 in TMEM: two accumulators of up to 256 tokens, so
//                       a weight is dequantised once per 512 tokens.
// One persistent CTA per SM.  The work -- (row tile, token super-tile, 128-k
// slab) triples, weighted by their accumulators -- is cut into contiguous
// runs, one per CTA, balanced for MMA work plus a fixed cost per piece of a
// tile; a run that covers a tile's whole K stores its sums, any other run
// adds them (reduce-add copies; see the store-first protocol below).
// Warp roles: 0..7 = dequantise then epilogue, 8 = token-tile TMA producer
// (+ TMEM allocation), 9 = MMA issue, 10 = packed-fragment bulk-copy producer.
// Epilogue: TMEM -> registers -> 32 x 32 fp32 chunks in shared memory (the idle
// A ring) -> TMA tensor store, or TMA reduce-add when the tile is split.  Every mbarrier wait is bounded; when one
// runs out the CTA raises a status word, drains and returns.
#include <cuda.h>

#include <atomic>
#include <cstring>

#include "aq_gemm_runs.h"
#include "aq_internal.h"
#include "aq_layout.cuh"
#include "aq_tc.cuh"

namespace aq {

constexpr int GM_ROWS = 128;       // weight rows per CTA tile (UMMA M)
constexpr int GM_KSTAGE = 64;      // k per A stage (one 128-byte swizzle atom of 16-bit elements)
constexpr int GM_ASTAGES = 4;      // dequantised-weight ring (16 KB each)
constexpr int GM_BSLOTS = 4;       // token ring: 256 tokens x 64 k = 32 KB each (one accumulator's share of a stage)
constexpr int GM_PSTAGES = 3;      // packed-fragment ring (one k-slab of 128 per slot)
constexpr int GM_DQ_WARPS = 8;
constexpr int GM_THREADS = (GM_DQ_WARPS + 3) * 32;
constexpr int GM_MAX_TN = 256;     // tokens per accumulator (UMMA N)
constexpr int GM_B_BYTES = GM_MAX_TN * 128;
constexpr int GM_A_BYTES = GM_ROWS * GM_KSTAGE * 2;
constexpr uint32_t GM_SPIN_LIMIT = 40u * 1000u * 1000u;

__device__ int g_gemm_status = 0;  // nonzero: a bounded wait ran out (code = which)

// Split tiles without zeroing the output first: the run that holds a tile's last k-slab is the first thing its CTA
// does; it STORES its sums and then writes the launch's epoch into the tile's flag; the other runs of the tile add
// theirs once they see it.  Flags are never reset: every launch has its own epoch and takes the next of a few arrays.
constexpr int GM_FLAG_SLOTS = 8;
constexpr int GM_MAX_TILES = 8192;
__device__ uint32_t g_tile_flags[GM_FLAG_SLOTS][GM_MAX_TILES];

constexpr int GM_MAX_OPS = 4;      // matrices that share one input (q|k|v, gate|up) run as one launch

struct GemmOp {
    const uint8_t* frags;
    float* out;            // float32 [M][ldo]
    const float* res;      // float32 [M][ldo] added once, or null
    int64_t ldo;
    int N;
    int NT;                // 16-row tiles
    int R;                 // row tiles of 128
    int bits;
};

struct GemmArgs {
    GemmOp op[GM_MAX_OPS];
    int n_ops;
    int Rtot;              // row tiles of 128 over all ops
    int M;
    int n_slabs;           // 128-k slabs (K padded to 256)
    int n_st;              // token super-tiles
    int n2;                // the first n2 of them hold two accumulators, the others one
    int st_tokens;         // tokens per super-tile (512 when M > 256)
    int tn;                // TMA box rows: 256 when M > 256, else M rounded up to 16
    int tma_out;           // 1: the epilogue writes through the output tensor maps (needs ldo % 4 == 0)
    int store_first;       // 1: split tiles of matrices without a residual use the store-then-add protocol above
    int flag_slot;
    uint32_t epoch;
    const float* tok_scale;    // per token: the power of two its row of x was divided by, or null
    const int* scaled_flag;    // nonzero when some entry of tok_scale is not 1 (null: none is)
    int bounds[GM_MAX_GRID + 1];   // CTA c works on slab-accumulators [bounds[c], bounds[c + 1]) (even numbers)
};

struct GemmOutMaps { CUtensorMap m[GM_MAX_OPS]; };

// One contiguous piece of a CTA's run: slabs [s0, s1) of tile (rt, st).
struct GemmSeg {
    int op, rt, st, na, s0, s1;   // rt: row tile inside matrix op
    int tile;                     // index of the tile in the launch
    int w0, w1;            // tokens (rounded up to 16) of the two accumulators
};

// Work is measured in slab-accumulators: a slab of a tile with two accumulators
// counts 2.  Tiles are ordered super-tile-major, so the two-accumulator tiles come
// first; run boundaries are even, hence whole slabs everywhere.
__device__ __forceinline__ bool gemm_next_seg(long long& pos, long long hi, const GemmArgs& a, GemmSeg& sg) {
    if (pos >= hi) return false;
    const long long c2 = 2LL * a.n_slabs, reg2 = c2 * a.n2 * a.Rtot;
    long long t, end;
    if (pos < reg2) {
        t = pos / c2;
        end = min(hi, (t + 1) * c2);
        sg.na = 2; sg.s0 = (int)((pos - t * c2) >> 1); sg.s1 = (int)((end - t * c2) >> 1);
    } else {
        const long long t1 = (pos - reg2) / a.n_slabs, base = reg2 + t1 * a.n_slabs;
        t = (long long)a.n2 * a.Rtot + t1;
        end = min(hi, base + a.n_slabs);
        sg.na = 1; sg.s0 = (int)(pos - base); sg.s1 = (int)(end - base);
    }
    pos = end;
    sg.tile = (int)t;
    sg.st = (int)(t / a.Rtot);
    int r = (int)(t - (long long)sg.st * a.Rtot);
    sg.op = 0;
    while (sg.op + 1 < a.n_ops && r >= a.op[sg.op].R) { r -= a.op[sg.op].R; ++sg.op; }
    sg.rt = r;
    const int rem = a.M - sg.st * a.st_tokens;
    if (sg.na == 2) { sg.w0 = GM_MAX_TN; sg.w1 = min(GM_MAX_TN, (rem - GM_MAX_TN + 15) & ~15); }
    else { sg.w0 = min(a.tn, (rem + 15) & ~15); sg.w1 = 0; }
    return true;
}

// Bounded wait.  Returns false when the limit ran out or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code) {
    for (uint32_t i = 0; i < GM_SPIN_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 2000) {
            __nanosleep(40);
            if (*abort_flag) return false;
        }
    }
    *abort_flag = 1;
    atomicCAS(&g_gemm_status, 0, code);
    return false;
}

// Two dequantised weights (k-adjacent, one row) as the 32-bit A-tile element.  p holds the two codes OR-ed into
// the mantissa of the binary16 constant 1024.0 in each half: subtract 1024 (exact), one half2 FMA with scale and min.
__device__ __forceinline__ uint32_t dequant_pair(uint32_t p, __half2 d2, __half2 m2) {
    const __half2 q = __hsub2(*reinterpret_cast<const __half2*>(&p), __float2half2_rn(1024.f));
    const __half2 w = __hfma2(q, d2, m2);
    return *reinterpret_cast<const uint32_t*>(&w);
}

// One dequantise warp's share of a k-slab: its fragment (16 rows x 128 k) becomes
// rows 16 dw .. 16 dw + 15 of two A stages.  `have` is false for row tiles past the
// end of the matrix (zeros are written).  Returns false when a wait ran out.
template <int BITS>
__device__ __forceinline__ bool dequant_slab(const uint8_t* slab, bool have, int dw, int lane, uint8_t* sA, uint32_t bar_pempty_slot,
                                             uint32_t bar_aempty, uint32_t bar_afull, uint32_t& ai, volatile int* abort_flag) {
    constexpr int FB = frag_bytes(BITS);
    constexpr uint32_t MAGIC = 0x64006400u;
    const int g = lane >> 2, t = lane & 3;
    LaneCodes<BITS> lc;
    uint32_t dmw[2][4];   // [row half][block]: half2 (scale, min)
    {
        const uint8_t* fb = slab + dw * FB;
        if (have) {
            load_lane_codes<BITS>(lc, fb, lane);
            const uint4 s0 = *reinterpret_cast<const uint4*>(fb + g * 16);
            const uint4 s1 = *reinterpret_cast<const uint4*>(fb + (g + 8) * 16);
            dmw[0][0] = s0.x; dmw[0][1] = s0.y; dmw[0][2] = s0.z; dmw[0][3] = s0.w;
            dmw[1][0] = s1.x; dmw[1][1] = s1.y; dmw[1][2] = s1.z; dmw[1][3] = s1.w;
        } else {
#pragma unroll
            for (int i = 0; i < 2 * BITS; ++i) lc.w[i] = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) { dmw[0][i] = 0; dmw[1][i] = 0; }
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_pempty_slot);   // packed bytes are in registers now
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t as = ai % GM_ASTAGES;
        if (!mbar_wait(bar_aempty + 8 * as, ((ai / GM_ASTAGES) & 1) ^ 1, abort_flag, 6)) return false;
        ++ai;
        uint8_t* At = sA + as * GM_A_BYTES;
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            // the two 16-byte chunks of this lane (blocks 2h and 2h + 1 of the row)
            uint32_t o[2][4];
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int j = 2 * h + jj;
                const __half2 dm = *reinterpret_cast<const __half2*>(&dmw[hi][j]);
                const __half2 d2 = __low2half2(dm), m2 = __high2half2(dm);
#pragma unroll
                for (int i = 0; i < 4; ++i) o[jj][i] = dequant_pair(code_pair<BITS>(lc, j, hi, i, MAGIC), d2, m2);
            }
            // Rows with odd g store block 2h + 1 first: the eight lanes that a 16-byte store serves together (g = 2q,
            // 2q + 1; t = 0..3) then hit eight different chunks of the swizzle atom instead of four twice.
            const int row = dw * 16 + g + 8 * hi;
            const bool odd = (g & 1) != 0;
            uint8_t* rp = At + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const int jj = odd ? 1 - st : st;
                const uint4 v = (st == 0) == !odd ? make_uint4(o[0][0], o[0][1], o[0][2], o[0][3]) : make_uint4(o[1][0], o[1][1], o[1][2], o[1][3]);
                *reinterpret_cast<uint4*>(rp + (((jj * 4 + t) ^ (row & 7)) * 16)) = v;
            }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_afull + 8 * as);
    }
    return true;
}

__global__ void __launch_bounds__(GM_THREADS, 1) gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ GemmOutMaps tmap_out, const GemmArgs a) {
    constexpr int P_BYTES = 8 * frag_bytes(4);                // packed fragments of one slab (largest width)
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + GM_ASTAGES * GM_A_BYTES;
    uint8_t* sP = sB + GM_BSLOTS * GM_B_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sP + GM_PSTAGES * P_BYTES);
    const uint32_t bar_afull = smem_u32(bars), bar_aempty = bar_afull + 8 * GM_ASTAGES;
    const uint32_t bar_bfull = bar_aempty + 8 * GM_ASTAGES, bar_bempty = bar_bfull + 8 * GM_BSLOTS;
    const uint32_t bar_pfull = bar_bempty + 8 * GM_BSLOTS, bar_pempty = bar_pfull + 8 * GM_PSTAGES;
    const uint32_t bar_accum = bar_pempty + 8 * GM_PSTAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * GM_ASTAGES + 2 * GM_BSLOTS + 2 * GM_PSTAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tmem_cols = (a.n2 > 0) ? 512u : (a.tn <= 32 ? 32u : a.tn <= 64 ? 64u : a.tn <= 128 ? 128u : 256u);

    if (threadIdx.x == 0) {
        for (int s = 0; s < GM_ASTAGES; ++s) { mbar_init(bar_afull + 8 * s, GM_DQ_WARPS); mbar_init(bar_aempty + 8 * s, 1); }
        for (int s = 0; s < GM_BSLOTS; ++s) { mbar_init(bar_bfull + 8 * s, 1); mbar_init(bar_bempty + 8 * s, 1); }
        for (int s = 0; s < GM_PSTAGES; ++s) { mbar_init(bar_pfull + 8 * s, 1); mbar_init(bar_pempty + 8 * s, GM_DQ_WARPS); }
        mbar_init(bar_accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == GM_DQ_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The packed weights never change, so their copies and the dequantisation start at once, under the tail of the
    // kernel before this one; the roles that read or write activations (token tiles, epilogue) call pdl_wait() first.
    pdl_launch_dependents();

    // this CTA's run, in slab-accumulators (even bounds)
    const long long run_lo = a.bounds[blockIdx.x], run_hi = a.bounds[blockIdx.x + 1];
    GemmSeg sg;
    long long pos = run_lo;

    if (warp == GM_DQ_WARPS) {
        // ---------------- producer: token tiles (TMA) ---------------------------------------------
        if (lane == 0) {
            uint32_t bi = 0;
            bool ok = true;
            pdl_wait();   // x is the predecessor's output
            while (ok && gemm_next_seg(pos, run_hi, a, sg)) {
                for (int it = 2 * sg.s0; it < 2 * sg.s1 && ok; ++it) {
                    for (int j = 0; j < sg.na; ++j) {
                        const uint32_t bs = bi % GM_BSLOTS;
                        ok = mbar_wait(bar_bempty + 8 * bs, ((bi / GM_BSLOTS) & 1) ^ 1, abort_flag, 2);
                        if (!ok) break;
                        mbar_expect_tx(bar_bfull + 8 * bs, (uint32_t)(a.tn * 128));
                        tma_load_2d(smem_u32(sB + bs * GM_B_BYTES), &tmap_x, it * GM_KSTAGE,
                                    sg.st * a.st_tokens + j * GM_MAX_TN, bar_bfull + 8 * bs);
                        ++bi;
                    }
                }
            }
        }
    } else if (warp == GM_DQ_WARPS + 2) {
        // ---------------- producer: packed fragments (bulk copies) ----------------------------------
        if (lane == 0) {
            uint32_t pi = 0;
            bool ok = true;
            while (ok && gemm_next_seg(pos, run_hi, a, sg)) {
                const GemmOp& op = a.op[sg.op];
                const int rt0 = sg.rt * 8, n_rt = min(8, op.NT - rt0);
                const int FB = frag_bytes(op.bits);
                for (int s = sg.s0; s < sg.s1; ++s) {
                    const uint32_t ps = pi % GM_PSTAGES;
                    ok = mbar_wait(bar_pempty + 8 * ps, ((pi / GM_PSTAGES) & 1) ^ 1, abort_flag, 1);
                    if (!ok) break;
                    mbar_expect_tx(bar_pfull + 8 * ps, (uint32_t)(n_rt * FB));
                    for (int ft = 0; ft < n_rt; ++ft) {
                        const int64_t f = (((int64_t)(s >> 1) * op.NT + rt0 + ft) * 2 + (s & 1));
                        bulk_load(smem_u32(sP + ps * P_BYTES + ft * FB), op.frags + f * FB, FB, bar_pfull + 8 * ps);
                    }
                    ++pi;
                }
            }
        }
    } else if (warp == GM_DQ_WARPS + 1) {
        // ---------------- MMA issue ----------------------------------------------------------------
        if (lane == 0) {
            uint32_t ai = 0, bi = 0;
            bool ok = true;
            while (ok && gemm_next_seg(pos, run_hi, a, sg)) {
                uint32_t idesc[2];
                for (int j = 0; j < 2; ++j) {
                    const uint32_t w = (j == 0) ? sg.w0 : sg.w1;
                    idesc[j] = (1u << 4) | ((w >> 3) << 17) | ((uint32_t)(GM_ROWS >> 4) << 24);   // f16 x f16 -> f32
                }
                for (int it = 2 * sg.s0; it < 2 * sg.s1 && ok; ++it) {
                    const uint32_t as = ai % GM_ASTAGES;
                    ok = mbar_wait(bar_afull + 8 * as, (ai / GM_ASTAGES) & 1, abort_flag, 3);
                    if (!ok) break;
                    const uint64_t ad = make_smem_desc(smem_u32(sA + as * GM_A_BYTES));
                    for (int j = 0; j < sg.na; ++j) {
                        const uint32_t bs = bi % GM_BSLOTS;
                        ok = mbar_wait(bar_bfull + 8 * bs, (bi / GM_BSLOTS) & 1, abort_flag, 4);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t bd = make_smem_desc(smem_u32(sB + bs * GM_B_BYTES));
#pragma unroll
                        for (int k = 0; k < GM_KSTAGE / 16; ++k)
                            umma_f16(tmem_base + (uint32_t)(j * GM_MAX_TN), ad + 2 * k, bd + 2 * k, idesc[j],
                                     (it > 2 * sg.s0 || k > 0) ? 1u : 0u);
                        umma_commit(bar_bempty + 8 * bs);
                        ++bi;
                    }
                    if (!ok) break;
                    umma_commit(bar_aempty + 8 * as);
                    ++ai;
                }
                if (ok) umma_commit(bar_accum);
            }
        }
    } else {
        // ---------------- dequantise (warps 0..7), then epilogue -----------------------------------
        const int dw = warp;
        uint32_t pi = 0, ai = 0, segc = 0;
        bool ok = true;
        while (gemm_next_seg(pos, run_hi, a, sg)) {   // (every warp walks every run, also after a failed wait: see the barrier below)
            const GemmOp& op = a.op[sg.op];
            const int n_rt = min(8, op.NT - sg.rt * 8);
            for (int s = sg.s0; s < sg.s1 && ok; ++s) {
                const uint32_t ps = pi % GM_PSTAGES;
                ok = mbar_wait(bar_pfull + 8 * ps, (pi / GM_PSTAGES) & 1, abort_flag, 5);
                if (!ok) break;
                ++pi;
                const uint8_t* slab = sP + ps * P_BYTES;
                if (op.bits == 2) ok = dequant_slab<2>(slab, dw < n_rt, dw, lane, sA, bar_pempty + 8 * ps, bar_aempty, bar_afull, ai, abort_flag);
                else if (op.bits == 3) ok = dequant_slab<3>(slab, dw < n_rt, dw, lane, sA, bar_pempty + 8 * ps, bar_aempty, bar_afull, ai, abort_flag);
                else ok = dequant_slab<4>(slab, dw < n_rt, dw, lane, sA, bar_pempty + 8 * ps, bar_aempty, bar_afull, ai, abort_flag);
            }
            // epilogue: TMEM lane quarter (warp % 4) x this warp group's columns -> out[token][row]
            if (ok) ok = mbar_wait(bar_accum, segc & 1, abort_flag, 7);
            ++segc;
            pdl_wait();   // outputs, residuals and tile flags belong to the stream's order (returns at once after the first time)
            if (ok) {
                tc_fence_after();
                const int lq = dw & 3, grp = dw >> 2;
                int c_lo, c_hi, acc;
                if (sg.na == 2) { acc = grp; c_lo = 0; c_hi = grp ? sg.w1 : sg.w0; }
                else {
                    const int half = ((sg.w0 / 2 + 31) / 32) * 32;
                    acc = 0; c_lo = grp ? min(half, sg.w0) : 0; c_hi = grp ? sg.w0 : min(half, sg.w0);
                }
                // with a residual the launcher has copied it into out: every run then adds on top of it
                const bool first_mode = a.store_first && op.res == nullptr;
                const bool entire = (sg.s0 == 0 && sg.s1 == a.n_slabs);
                const bool whole = (entire && (op.res == nullptr || !a.tma_out)) || (first_mode && sg.s1 == a.n_slabs);
                const bool raise_flag = first_mode && whole && !entire;
                if (first_mode && !whole) {   // the tile's last-slab run has to have stored before anything is added
                    const uint32_t* fl = &g_tile_flags[a.flag_slot][sg.tile];
                    uint32_t seen = 0, spins = 0;
                    if (lane == 0) {
                        while ((seen = ld_acquire_u32(fl)) != a.epoch) {
                            if (++spins > (1u << 22) || *abort_flag) break;
                            __nanosleep(100);
                        }
                        if (seen != a.epoch) { *abort_flag = 1; atomicCAS(&g_gemm_status, 0, 8); }
                    }
                    seen = __shfl_sync(0xffffffffu, seen, 0);
                    ok = (seen == a.epoch);
                }
                if (ok) {
                const bool add_res = (op.res != nullptr && sg.s0 == 0 && !a.tma_out);
                const CUtensorMap* tmo = &tmap_out.m[sg.op];
                const int n0 = sg.rt * GM_ROWS + lq * 32;
                const int64_t n = (int64_t)n0 + lane;
                const int tok0 = sg.st * a.st_tokens + acc * GM_MAX_TN;
                // token rows whose input was divided by a power of two get it back here (rare: a flag says whether any)
                const bool scaled = a.scaled_flag != nullptr && __ldcg(a.scaled_flag) != 0;
                if (a.tma_out) {
                    // the A ring is idle now (every MMA of the run has completed): two 4 KB chunks per warp
                    float* stg = reinterpret_cast<float*>(sA + dw * 8192);
                    // two register sets: the TMEM load of the next 32 columns is in flight while this one is staged
                    const uint32_t t_addr = tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(acc * GM_MAX_TN);
                    auto emit = [&](uint32_t (&v)[32], int c0, int buf) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) asm volatile("" : "+r"(v[j]));   // (read only after the wait above)
                        if (lane == 0) bulk_wait_read<1>();   // the copy that last read this chunk has left shared memory
                        __syncwarp();
                        float* chunk = stg + buf * 1024;      // [32 tokens][32 rows]
                        if (scaled) {
                            const float sc = __ldcg(a.tok_scale + min(tok0 + c0 + lane, a.M - 1));
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * __shfl_sync(0xffffffffu, sc, j));
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) chunk[j * 32 + lane] = __uint_as_float(v[j]);
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0) {   // rows / tokens past the end of the tensor are clipped by the copy
                            if (whole) tma_store_2d(tmo, smem_u32(chunk), n0, tok0 + c0);
                            else tma_reduce_add_2d(tmo, smem_u32(chunk), n0, tok0 + c0);
                            bulk_commit();
                        }
                    };
                    uint32_t va[32], vb[32];
                    int n_chunks = 0;   // (the two staging chunks alternate; the copies are drained at the end of the piece)
                    if (c_lo < c_hi) tmem_ld32(t_addr + (uint32_t)c_lo, va);
                    for (int c0 = c_lo; c0 < c_hi; c0 += 64) {
                        tmem_ld_wait();
                        if (c0 + 32 < c_hi) tmem_ld32(t_addr + (uint32_t)(c0 + 32), vb);
                        emit(va, c0, n_chunks++ & 1);
                        if (c0 + 32 < c_hi) {
                            tmem_ld_wait();
                            if (c0 + 64 < c_hi) tmem_ld32(t_addr + (uint32_t)(c0 + 64), va);
                            emit(vb, c0 + 32, n_chunks++ & 1);
                        }
                    }
                    if (lane == 0) {
                        if (raise_flag) bulk_wait_all<0>();   // the stores must have landed before the flag goes up
                        else bulk_wait_read<0>();             // the A ring is written again right after
                    }
                    __syncwarp();
                } else {
                    for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(acc * GM_MAX_TN + c0), v);
                        tmem_ld_wait();
                        if (n < op.N) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int tok = tok0 + c0 + j;
                                if (c0 + j < c_hi && tok < a.M) {
                                    const int64_t o = (int64_t)tok * op.ldo + n;
                                    float val = __uint_as_float(v[j]);
                                    if (scaled) val *= __ldcg(a.tok_scale + tok);
                                    if (add_res) val += __ldg(op.res + o);
                                    if (whole) op.out[o] = val;
                                    else atomicAdd(op.out + o, val);
                                }
                            }
                        }
                    }
                }
                }
                tc_fence_before();   // the next run's first MMA may overwrite the accumulators
            }
            // the chunks staged above live in the A ring: nobody refills it before everybody has left the epilogue
            asm volatile("bar.sync 1, %0;" ::"n"(GM_DQ_WARPS * 32) : "memory");
            if (threadIdx.x == 0 && ok && a.store_first && a.op[sg.op].res == nullptr && sg.s1 == a.n_slabs && sg.s0 != 0)
                st_release_u32(&g_tile_flags[a.flag_slot][sg.tile], a.epoch);
        }
    }
    if (warp < GM_DQ_WARPS && lane == 0) bulk_wait_all<0>();   // this thread's output copies are complete
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);   // let copies in flight land before the CTA's shared memory goes away
    if (warp == GM_DQ_WARPS) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ---- host ---------------------------------------------------------------------
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

static cudaError_t launch_one(const CUtensorMap& tm, const GemmOutMaps& tmo, const GemmArgs& a, int grid, cudaStream_t s) {
    constexpr int SMEM = 1024 + GM_ASTAGES * GM_A_BYTES + GM_BSLOTS * GM_B_BYTES + GM_PSTAGES * 8 * frag_bytes(4) + 256;
    auto kern = gemm_kernel;
    static PerDeviceOnce configured;
    {
        const int rc = configured.run(current_device(), [&] {
            return (int)cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        });
        if (rc != 0) return rc < 0 ? cudaErrorInvalidDevice : (cudaError_t)rc;
    }
    cudaError_t e = launch_pdl(kern, dim3((unsigned)grid), dim3(GM_THREADS), SMEM, s, tm, tmo, a);
    count_launch();
    return e;
}

bool gemm_stores_first(const aq_handle_s* const* hs, int n, int M, cudaStream_t s);

// n (<= GM_MAX_OPS) matrices with the same K against one x: out[i] = (res[i]) + x W_i^T.
// outs_ready: the caller has already put the residual (or zeros) into every output.
cudaError_t launch_gemm_group(const aq_handle_s* const* hs, int n, const void* x16, const float* tok_scale, const int* scaled_flag,
                              int M, float* const* outs, const int64_t* ldos, const float* const* ress, bool outs_ready,
                              cudaStream_t s) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc || n < 1 || n > GM_MAX_OPS) return cudaErrorNotSupported;
    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.n_ops = n; a.M = M; a.n_slabs = hs[0]->KP * 2;
    a.tok_scale = tok_scale; a.scaled_flag = tok_scale ? scaled_flag : nullptr;
    for (int i = 0; i < n; ++i) {
        if (hs[i]->K != hs[0]->K) return cudaErrorInvalidValue;
        GemmOp& o = a.op[i];
        o.frags = hs[i]->frags; o.out = outs[i]; o.res = ress ? ress[i] : nullptr; o.ldo = ldos[i];
        o.N = (int)hs[i]->N; o.NT = hs[i]->NT; o.R = (hs[i]->NT + 7) / 8; o.bits = hs[i]->bits;
        a.Rtot += o.R;
    }
    if (M > GM_MAX_TN) {
        a.tn = GM_MAX_TN; a.st_tokens = 2 * GM_MAX_TN;
        a.n_st = (M + a.st_tokens - 1) / a.st_tokens;
        a.n2 = (M - a.st_tokens * (a.n_st - 1) > GM_MAX_TN) ? a.n_st : a.n_st - 1;
    } else {
        a.tn = ((M + 15) / 16) * 16; a.st_tokens = a.tn; a.n_st = 1; a.n2 = 0;
    }
    const long long total = (long long)a.n_slabs * a.Rtot * (2LL * a.n2 + (a.n_st - a.n2));
    int grid = sm_count() < GM_MAX_GRID ? sm_count() : GM_MAX_GRID;
    if (total / 2 < grid) grid = (int)(total / 2);
    if (total > 0x7fffffffLL) return cudaErrorInvalidValue;
    cut_runs(total, (long long)a.n2 * a.Rtot, 2LL * a.n_slabs, a.n_slabs, grid, a.bounds);
    CUtensorMap tm;
    const cuuint64_t dims[2] = {(cuuint64_t)hs[0]->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)hs[0]->K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)GM_KSTAGE, (cuuint32_t)a.tn};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x16), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    // the outputs as tensors [M][N] of float32 for the epilogue's 32 x 32 copies (row pitch must be 16-byte aligned)
    GemmOutMaps tmo;
    memset(&tmo, 0, sizeof(tmo));
    a.tma_out = 1;
    for (int i = 0; i < n && a.tma_out; ++i) {
        const GemmOp& o = a.op[i];
        if (o.ldo % 4 != 0 || (reinterpret_cast<uintptr_t>(o.out) & 15u) != 0) { a.tma_out = 0; break; }
        const cuuint64_t odims[2] = {(cuuint64_t)o.N, (cuuint64_t)M};
        const cuuint64_t ostrides[1] = {(cuuint64_t)o.ldo * 4};
        const cuuint32_t obox[2] = {32, 32};
        if (enc(&tmo.m[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, o.out, odims, ostrides, obox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            a.tma_out = 0;
    }
    // What an output holds before the kernel: the residual when there is one (every run then adds to it);
    // else zeros when some run does not cover a whole tile; else nothing.
    bool all_whole = true;
    {
        const long long c2 = 2LL * a.n_slabs, reg2 = c2 * a.n2 * a.Rtot;
        for (int c = 1; c < grid && all_whole; ++c) {
            const long long b = a.bounds[c];
            all_whole = (b <= reg2) ? (b % c2 == 0) : ((b - reg2) % a.n_slabs == 0);
        }
    }
    if (outs_ready && !a.tma_out) return cudaErrorInvalidValue;   // (the caller checks gemm_outputs_can_be_preset first)
    static std::atomic<uint32_t> epoch_counter{0};
    a.store_first = (a.tma_out && gemm_stores_first(hs, n, M, s)) ? 1 : 0;
    a.epoch = epoch_counter.fetch_add(1) + 1;
    if (a.epoch == 0) a.epoch = epoch_counter.fetch_add(1) + 1;   // flags start out as zero: never use that value
    a.flag_slot = (int)(a.epoch % GM_FLAG_SLOTS);
    // What an output holds before the kernel: the residual when there is one (every run then adds to it); zeros
    // when runs add without the store-first protocol; else nothing.  With outs_ready the caller has done this.
    for (int i = 0; i < n && !outs_ready; ++i) {
        const GemmOp& o = a.op[i];
        cudaError_t e = cudaSuccess;
        if (o.res && a.tma_out)
            e = cudaMemcpy2DAsync(o.out, (size_t)o.ldo * sizeof(float), o.res, (size_t)o.ldo * sizeof(float),
                                  (size_t)o.N * sizeof(float), (size_t)M, cudaMemcpyDeviceToDevice, s);
        else if (!all_whole && !(a.store_first && !o.res))
            e = cudaMemset2DAsync(o.out, (size_t)o.ldo * sizeof(float), 0, (size_t)o.N * sizeof(float), (size_t)M, s);
        if (e != cudaSuccess) return e;
    }
    return launch_one(tm, tmo, a, grid, s);
}

cudaError_t launch_gemm(const aq_handle_s* h, const void* x16, const float* tok_scale, const int* scaled_flag, int M, float* out,
                        int64_t ldo, const float* res, cudaStream_t s) {
    return launch_gemm_group(&h, 1, x16, tok_scale, scaled_flag, M, &out, &ldo, &res, false, s);
}

// ---- bfloat16 activations -> binary16 operand ---------------------------------------------------------------
// One CTA per token row.  A bfloat16 value has 8 significant bits, so it is a binary16 value whenever it is inside
// binary16's range (magnitudes below 2^-17 land on the subnormal grid, an absolute error below 2^-25).  A row that
// holds a magnitude of 2^15 or more is divided by the power of two that brings its largest one below 2^15 (exact for
// everything that stays normal); scale[m] is that power of two, 1 otherwise, and *flag is raised when any row has one.
__global__ void __launch_bounds__(256) rows_to_f16_kernel(const __nv_bfloat16* __restrict__ x, __half* __restrict__ x16,
                                                          float* __restrict__ scale, int* __restrict__ flag, int64_t K) {
    const int64_t m = blockIdx.x;
    const __nv_bfloat16* xr = x + m * K;
    __half* o = x16 + m * K;
    float mx = 0.f;
    for (int64_t k = threadIdx.x * 8; k < K; k += 256 * 8) {   // K is a multiple of 32
        const uint4 v = *reinterpret_cast<const uint4*>(xr + k);
        const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&v);
        uint4 r;
        __half2* h = reinterpret_cast<__half2*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(b[i]);
            h[i] = __floats2half2_rn(f.x, f.y);
            mx = fmaxf(mx, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
        *reinterpret_cast<uint4*>(o + k) = r;
    }
    __shared__ float red[8];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, red[i]);
    float sc = 1.f;
    if (mx >= 32768.f && mx <= 3.0e38f) {   // (non-finite input stays non-finite: nothing to rescue)
        int e;
        frexpf(mx, &e);                       // mx = f 2^e, f in [0.5, 1)
        sc = ldexpf(1.f, e - 15);             // mx / sc in [2^14, 2^15)
        const float inv = 1.f / sc;
        for (int64_t k = threadIdx.x * 8; k < K; k += 256 * 8) {
            const uint4 v = *reinterpret_cast<const uint4*>(xr + k);
            const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&v);
            uint4 r;
            __half2* h = reinterpret_cast<__half2*>(&r);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(b[i]);
                h[i] = __floats2half2_rn(f.x * inv, f.y * inv);
            }
            *reinterpret_cast<uint4*>(o + k) = r;
        }
        if (threadIdx.x == 0) *flag = 1;
    }
    if (threadIdx.x == 0) scale[m] = sc;
}

cudaError_t launch_rows_to_f16(const void* x_bf16, void* x16, float* scale, int* flag, int M, int64_t K, cudaStream_t s) {
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    rows_to_f16_kernel<<<(unsigned)M, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(x_bf16), reinterpret_cast<__half*>(x16), scale,
                                                   flag, K);
    count_launch();
    return cudaGetLastError();
}

// True when outputs without a residual need no zeroing before launch_gemm_group (split tiles store first).
bool gemm_stores_first(const aq_handle_s* const* hs, int n, int M, cudaStream_t s) {
    // The protocol tells launches apart by a fresh epoch per launch.  A launch recorded into a CUDA graph would run
    // again with the epoch it was recorded with, so while a stream is being captured outputs are zeroed and added to.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { cudaGetLastError(); return false; }
    if (cap != cudaStreamCaptureStatusNone) return false;
    long long R = 0;
    for (int i = 0; i < n; ++i) R += (hs[i]->NT + 7) / 8;
    const long long n_st = (M > GM_MAX_TN) ? (M + 2 * GM_MAX_TN - 1) / (2 * GM_MAX_TN) : 1;
    return R * n_st <= GM_MAX_TILES;
}

// True when launch_gemm_group accepts outputs preset by the caller (they are written through tensor maps).
bool gemm_outputs_can_be_preset(float* const* outs, const int64_t* ldos, int n) {
    if (!tensor_map_encoder()) return false;
    for (int i = 0; i < n; ++i)
        if (ldos[i] % 4 != 0 || (reinterpret_cast<uintptr_t>(outs[i]) & 15u) != 0) return false;
    return true;
}

int read_gemm_status(bool clear) {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int));
    if (clear && v) { int z = 0; cudaMemcpyToSymbol(g_gemm_status, &z, sizeof(int)); }
    return v;
}

}  // namespace aq
