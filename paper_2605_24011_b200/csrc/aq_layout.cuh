// Device-private weight layout ("fragment layout") and the bit tricks that read it.
//
// The canonical container (Appendix D) is row-major block records; on the
// device the same bits are regrouped so that one warp reads what one tensor
// core instruction needs with 16-byte accesses:
//
//   fragment = 16 rows x 128 k (4 blocks of 32), FB = 256 (bits+1) bytes
//     bytes [0,256)  : half2 (scale, min) at [row r][block j] -> (r*4 + j)*4
//     bytes [256,FB) : codes.  Slot s = g*4 + t (g = row mod 8, t = 0..3) owns,
//                      for rows g and g+8 and each block j, the 8 codes
//                      8t .. 8t+7 of that block (a "unit" of 8 codes).
//   unit pair = fragments of k-slabs 2P and 2P+1 for one row tile, contiguous.
//   order     = [pair-slab P][row tile R][slab parity] ; N padded to 16, K to 256.
//
// Code placement inside a slot is chosen so that (w >> sh) & mask yields two
// k-adjacent codes of one row in the two 16-bit halves of a register:
//   4-bit: slot = 2 pieces of 16 B (piece p at 256 + p*512 + s*16): words
//          [unit(g,2p), unit(g+8,2p), unit(g,2p+1), unit(g+8,2p+1)];
//          in a word nibble i holds code 2i, nibble i+4 holds code 2i+1.
//   2-bit: slot = 16 B at 256 + s*16: words [row g blocks 0,1], [row g+8
//          blocks 0,1], [row g blocks 2,3], [row g+8 blocks 2,3]; in a word the
//          low half holds the even codes (crumb i + 4*(j&1) = code 2i of block
//          j), the high half the odd codes.
//   3-bit: slot = 24 B: per row three words hold 16 code pairs; pair P = 4j+i
//          (codes 2i, 2i+1 of block j) sits, for P < 15, in word P/5 at bits
//          3(P%5) of the low half (even code) and high half (odd code); pair
//          15 is spread over bit 15 / bit 31 of the three words.  Words of row
//          g and word 0 of row g+8 are at 256 + s*16, words 1,2 of row g+8 at
//          256 + 512 + s*8.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace aq {

constexpr int ROWS = 16;        // rows per fragment
constexpr int SLAB = 128;       // k per fragment
constexpr int SCALE_BYTES = 256;

__host__ __device__ constexpr int frag_bytes(int bits) { return 256 * (bits + 1); }

// One code bit's home: byte offset of a 32-bit word inside the fragment and the
// bit position in it.  r in 0..15, kk in 0..127, tb = bit of the code.
__host__ __device__ inline void code_bit_home(int bits, int r, int kk, int tb, int& word_off, int& bitpos) {
    const int j = kk >> 5, e = kk & 31, t = e >> 3, c = e & 7;
    const int g = r & 7, hi = r >> 3, s = g * 4 + t;
    const int half = c & 1, i = c >> 1;
    if (bits == 4) {
        word_off = 256 + (j >> 1) * 512 + s * 16 + ((j & 1) * 2 + hi) * 4;
        bitpos = 4 * (i + 4 * half) + tb;
    } else if (bits == 2) {
        word_off = 256 + s * 16 + ((j >> 1) * 2 + hi) * 4;
        bitpos = 16 * half + 2 * (i + 4 * (j & 1)) + tb;
    } else {
        const int P = 4 * j + i;
        int w;
        if (P < 15) { w = P / 5; bitpos = 16 * half + 3 * (P % 5) + tb; }
        else        { w = tb;    bitpos = 16 * half + 15; }
        const int rw = hi * 3 + w;
        word_off = (rw < 4) ? (256 + s * 16 + rw * 4) : (256 + 512 + s * 8 + (rw - 4) * 4);
    }
}

// ---- register-level extraction -------------------------------------------
// A lane's code words for one fragment.
template <int BITS> struct LaneCodes;
template <> struct LaneCodes<2> { uint32_t w[4]; };
template <> struct LaneCodes<3> { uint32_t w[6]; };   // [0..2] row g, [3..5] row g+8
template <> struct LaneCodes<4> { uint32_t w[8]; };   // piece p at [4p .. 4p+3]

template <int BITS>
__device__ __forceinline__ void load_lane_codes(LaneCodes<BITS>& lc, const uint8_t* frag, int lane) {
    const uint4 a = *reinterpret_cast<const uint4*>(frag + 256 + lane * 16);
    lc.w[0] = a.x; lc.w[1] = a.y; lc.w[2] = a.z; lc.w[3] = a.w;
    if constexpr (BITS == 3) {
        const uint2 b = *reinterpret_cast<const uint2*>(frag + 256 + 512 + lane * 8);
        lc.w[4] = b.x; lc.w[5] = b.y;
    }
    if constexpr (BITS == 4) {
        const uint4 b = *reinterpret_cast<const uint4*>(frag + 256 + 512 + lane * 16);
        lc.w[4] = b.x; lc.w[5] = b.y; lc.w[6] = b.z; lc.w[7] = b.w;
    }
}

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t orv) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(orv));   // (a & mask) | orv
    return d;
}

// Pair i (codes 2i, 2i+1) of block j, row half hi (0: row g, 1: row g+8): the
// two codes land in bits [0,BITS) and [16,16+BITS) of the result, OR-ed with
// `orv` (0 for plain integers, a floating-point exponent pattern otherwise).
template <int BITS>
__device__ __forceinline__ uint32_t code_pair(const LaneCodes<BITS>& lc, int j, int hi, int i, uint32_t orv) {
    if constexpr (BITS == 4) {
        const uint32_t w = lc.w[(j >> 1) * 4 + (j & 1) * 2 + hi];
        return lop3_and_or(w >> (4 * i), 0x000F000Fu, orv);
    } else if constexpr (BITS == 2) {
        const uint32_t w = lc.w[(j >> 1) * 2 + hi];
        return lop3_and_or(w >> (2 * (i + 4 * (j & 1))), 0x00030003u, orv);
    } else {
        const uint32_t* R = lc.w + hi * 3;
        const int P = 4 * j + i;
        if (P < 15) return lop3_and_or(R[P / 5] >> (3 * (P % 5)), 0x00070007u, orv);
        uint32_t v = lop3_and_or(R[0] >> 15, 0x00010001u, orv);
        v = lop3_and_or(R[1] >> 14, 0x00020002u, v);
        v = lop3_and_or(R[2] >> 13, 0x00040004u, v);
        return v;
    }
}

}  // namespace aq
