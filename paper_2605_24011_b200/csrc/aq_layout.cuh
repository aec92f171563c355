// Device-private weight layout ("fragment layout") and the bit tricks that read it.
//
// The canonical container (Appendix D) is row-major block records; on the
// device the same bits are regrouped so that one warp reads what one tensor
// core instruction needs with 16-byte accesses, and so that a code can be used
// as a tensor-core operand WHERE IT LIES, with one AND and no shift:
//
//   fragment = 16 rows x 128 k (4 blocks of 32), FB = 256 (bits+1) bytes
//     bytes [0,256)  : half2 (scale, min) at [row r][block j] -> (r*4 + j)*4
//     bytes [256,FB) : codes.  Slot s = g*4 + t (g = row mod 8, t = 0..3) owns,
//                      for rows g and g+8 and each block j, the 8 codes
//                      8t .. 8t+7 of that block.
//   unit     = fragments of k-slabs 2P and 2P+1 for one row tile, contiguous.
//   order    = [pair-slab P][row tile R][slab parity] ; N padded to 16, K to 256.
//
// A slot's 64 codes are 32 pairs (two k-adjacent codes of one row: the even
// one in the low half of a 32-bit word, the odd one in the high half, at the
// same bit position).  Pair (j, hi, i) -- block j, row half hi, codes 2i, 2i+1
// of the slot -- feeds tensor-core instruction f = 2j + (i >> 1) as A register
// r = hi + 2 (i & 1).  The four registers of one instruction sit in four
// different words at the SAME bit position, so the instruction sees
// 2^pos * q in every element and the power of two is taken out afterwards:
//   2-bit: word r (4 words at 256 + s*16), field f at bit 2f of each half.
//   4-bit: word (f >> 2)*4 + r (piece p = f >> 2 at 256 + p*512 + s*16), field
//          f & 3 at bit 4 (f & 3).
//   3-bit: words 0..3 ("r-words", at 256 + s*16) hold f = 0..4 at bit 3f of
//          word r; words 4,5 ("e-words", at 768 + s*8) hold f = 5,6,7: register
//          r of f = 5 at bit 3 (r >> 1) of e-word r & 1, of f = 6 at bit
//          6 + 3 (r >> 1), of f = 7 (r < 2) at bit 12; registers 2,3 of f = 7
//          are spread over bit 15 of words {0,1,2} and {3,4,5} (code bit b in
//          the b-th word of the triple).
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace aq {

constexpr int ROWS = 16;        // rows per fragment
constexpr int SLAB = 128;       // k per fragment
constexpr int SCALE_BYTES = 256;

__host__ __device__ constexpr int frag_bytes(int bits) { return 256 * (bits + 1); }

// Home of bit tb of code c (0..7) of the slot's block j, row half hi: the index
// of the slot's 32-bit word and the bit position in it.
__host__ __device__ inline void slot_bit_home(int bits, int j, int hi, int c, int tb, int& widx, int& bitpos) {
    const int half = c & 1, i = c >> 1;
    const int f = 2 * j + (i >> 1), r = hi + 2 * (i & 1);
    if (bits == 2) {
        widx = r; bitpos = 16 * half + 2 * f + tb;
    } else if (bits == 4) {
        widx = (f >> 2) * 4 + r; bitpos = 16 * half + 4 * (f & 3) + tb;
    } else {
        if (f <= 4) { widx = r; bitpos = 16 * half + 3 * f + tb; }
        else if (f == 5) { widx = 4 + (r & 1); bitpos = 16 * half + 3 * (r >> 1) + tb; }
        else if (f == 6) { widx = 4 + (r & 1); bitpos = 16 * half + 6 + 3 * (r >> 1) + tb; }
        else if (r < 2) { widx = 4 + r; bitpos = 16 * half + 12 + tb; }
        else { widx = (r == 2 ? 0 : 3) + tb; bitpos = 16 * half + 15; }
    }
}

// Byte offset, inside the fragment, of word widx of slot s.
__host__ __device__ inline int slot_word_offset(int bits, int s, int widx) {
    if (bits == 2) return 256 + s * 16 + widx * 4;
    if (bits == 4) return 256 + (widx >> 2) * 512 + s * 16 + (widx & 3) * 4;
    return widx < 4 ? 256 + s * 16 + widx * 4 : 256 + 512 + s * 8 + (widx - 4) * 4;
}

// One code bit's home: byte offset of a 32-bit word inside the fragment and the
// bit position in it.  r in 0..15, kk in 0..127, tb = bit of the code.
__host__ __device__ inline void code_bit_home(int bits, int r, int kk, int tb, int& word_off, int& bitpos) {
    const int j = kk >> 5, e = kk & 31, t = e >> 3, c = e & 7;
    const int g = r & 7, hi = r >> 3;
    int widx;
    slot_bit_home(bits, j, hi, c, tb, widx, bitpos);
    word_off = slot_word_offset(bits, g * 4 + t, widx);
}

// ---- register-level extraction -------------------------------------------
// A lane's code words for one fragment.
template <int BITS> struct LaneCodes { uint32_t w[2 * BITS]; };

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
// The general (shift + mask) reader; the fp16 decode path reads in place instead.
template <int BITS>
__device__ __forceinline__ uint32_t code_pair(const LaneCodes<BITS>& lc, int j, int hi, int i, uint32_t orv) {
    const int f = 2 * j + (i >> 1), r = hi + 2 * (i & 1);
    if constexpr (BITS == 2) {
        return lop3_and_or(lc.w[r] >> (2 * f), 0x00030003u, orv);
    } else if constexpr (BITS == 4) {
        return lop3_and_or(lc.w[(f >> 2) * 4 + r] >> (4 * (f & 3)), 0x000F000Fu, orv);
    } else {
        if (f <= 4) return lop3_and_or(lc.w[r] >> (3 * f), 0x00070007u, orv);
        if (f == 5) return lop3_and_or(lc.w[4 + (r & 1)] >> (3 * (r >> 1)), 0x00070007u, orv);
        if (f == 6) return lop3_and_or(lc.w[4 + (r & 1)] >> (6 + 3 * (r >> 1)), 0x00070007u, orv);
        if (r < 2) return lop3_and_or(lc.w[4 + r] >> 12, 0x00070007u, orv);
        const uint32_t* T = lc.w + (r == 2 ? 0 : 3);
        uint32_t v = lop3_and_or(T[0] >> 15, 0x00010001u, orv);
        v = lop3_and_or(T[1] >> 14, 0x00020002u, v);
        v = lop3_and_or(T[2] >> 13, 0x00040004u, v);
        return v;
    }
}

// ---- in-place reader (fp16 operands) ----------------------------------------
// A code left at bit position s of a half-word, everything else masked away,
// IS the binary16 subnormal q * 2^(s - 24) as long as s + BITS <= 10.  One AND
// per A register; a byte shift of the whole word brings the upper fields into
// the mantissa.  InPlace<BITS> holds a lane's words and their shifted copies.
template <int BITS> struct InPlace;

template <> struct InPlace<2> {
    static constexpr int NCLS = 5;                           // bit positions 0,2,4,6,8
    uint32_t w[4], w8[4];
    __device__ __forceinline__ void prepare(const LaneCodes<2>& lc) {
#pragma unroll
        for (int r = 0; r < 4; ++r) { w[r] = lc.w[r]; w8[r] = lc.w[r] >> 8; }
    }
    static __device__ __forceinline__ constexpr int pos(int f) { return f <= 4 ? 2 * f : 2 * f - 8; }
    static __device__ __forceinline__ constexpr int cls(int f) { return pos(f) / 2; }
    static __device__ __forceinline__ constexpr int cls_pos(int c) { return 2 * c; }
    __device__ __forceinline__ uint32_t reg(int f, int r) const {
        return (f <= 4 ? w[r] : w8[r]) & (0x00030003u << pos(f));
    }
};

template <> struct InPlace<4> {
    static constexpr int NCLS = 2;                           // bit positions 0,4
    uint32_t w[8], w8[8];
    __device__ __forceinline__ void prepare(const LaneCodes<4>& lc) {
#pragma unroll
        for (int r = 0; r < 8; ++r) { w[r] = lc.w[r]; w8[r] = lc.w[r] >> 8; }
    }
    static __device__ __forceinline__ constexpr int pos(int f) { return 4 * (f & 1); }
    static __device__ __forceinline__ constexpr int cls(int f) { return f & 1; }
    static __device__ __forceinline__ constexpr int cls_pos(int c) { return 4 * c; }
    __device__ __forceinline__ uint32_t reg(int f, int r) const {
        const int k = (f >> 2) * 4 + r;
        return ((f & 2) ? w8[k] : w[k]) & (0x000F000Fu << pos(f));
    }
};

template <> struct InPlace<3> {
    static constexpr int NCLS = 5;                           // bit positions 0,1,3,4,6
    uint32_t w[4], w8[4], e[2], e3[2], e8[2], sc[2];
    __device__ __forceinline__ void prepare(const LaneCodes<3>& lc) {
#pragma unroll
        for (int r = 0; r < 4; ++r) { w[r] = lc.w[r]; w8[r] = lc.w[r] >> 8; }
#pragma unroll
        for (int x = 0; x < 2; ++x) { e[x] = lc.w[4 + x]; e3[x] = lc.w[4 + x] >> 3; e8[x] = lc.w[4 + x] >> 8; }
        // the two pairs spread over bit 15 of three words each, gathered at bit position 4
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint32_t* T = lc.w + 3 * x;
            uint32_t v = (T[0] >> 11) & 0x00100010u;
            v = lop3_and_or(T[1] >> 10, 0x00200020u, v);
            v = lop3_and_or(T[2] >> 9, 0x00400040u, v);
            sc[x] = v;
        }
    }
    static __device__ __forceinline__ constexpr int pos(int f) {
        return f <= 2 ? 3 * f : f == 3 ? 1 : f == 4 ? 4 : f == 5 ? 0 : f == 6 ? 6 : 4;
    }
    static __device__ __forceinline__ constexpr int cls(int f) {
        return pos(f) == 0 ? 0 : pos(f) == 1 ? 1 : pos(f) == 3 ? 2 : pos(f) == 4 ? 3 : 4;
    }
    static __device__ __forceinline__ constexpr int cls_pos(int c) { return c == 0 ? 0 : c == 1 ? 1 : c == 2 ? 3 : c == 3 ? 4 : 6; }
    __device__ __forceinline__ uint32_t reg(int f, int r) const {
        const uint32_t m = 0x00070007u << pos(f);
        if (f <= 2) return w[r] & m;
        if (f <= 4) return w8[r] & m;
        if (f <= 6) return (r < 2 ? e[r] : e3[r - 2]) & m;
        return r < 2 ? (e8[r] & m) : sc[r - 2];
    }
};

}  // namespace aq
