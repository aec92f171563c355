"""Per-element pure-Python restatement of the block format, for tiny matrices.

No NumPy arithmetic: roundings to binary32 / binary16 go through `struct`,
the bit stream through Python big integers.  Used only to pin the oracle.
"""
import math
import struct


def f32(x: float) -> float:
    return struct.unpack("<f", struct.pack("<f", x))[0]


def f16(x: float) -> float:
    return struct.unpack("<e", struct.pack("<e", x))[0]


def f16_bytes(x: float) -> bytes:
    return struct.pack("<e", x)


def rint_even(t: float) -> int:
    fl = math.floor(t)
    r = t - fl
    if r > 0.5:
        return fl + 1
    if r < 0.5:
        return fl
    return fl if fl % 2 == 0 else fl + 1


def quantize_block(w, bits):
    """w: 32 python floats (binary32 values).  Returns (d, m, codes)."""
    L = (1 << bits) - 1
    mn, mx = min(w), max(w)
    d = f16(f32(f32(mx - mn) / float(L)))
    m = f16(mn)
    codes = []
    for v in w:
        if d == 0.0:
            codes.append(0)
            continue
        t = f32(f32(v - m) / d)
        codes.append(max(0, min(L, rint_even(t))))
    return d, m, codes


def pack_block(d, m, codes, bits) -> bytes:
    big = 0
    for i, c in enumerate(codes):
        big |= c << (bits * i)
    return f16_bytes(d) + f16_bytes(m) + big.to_bytes(4 * bits, "little")


def unpack_block(rec: bytes, bits):
    d = struct.unpack("<e", rec[0:2])[0]
    m = struct.unpack("<e", rec[2:4])[0]
    big = int.from_bytes(rec[4:], "little")
    codes = [(big >> (bits * i)) & ((1 << bits) - 1) for i in range(32)]
    return d, m, codes


def dequant_elem_f32(d, m, c) -> float:
    return f32(f32(d * c) + m)


def matrix(W, bits):
    """W: list of rows of python floats.  Returns per-row lists of
    (d, m, codes) blocks and the canonical byte string."""
    out, raw = [], b""
    for row in W:
        blocks = []
        for j in range(0, len(row), 32):
            d, m, codes = quantize_block(row[j:j + 32], bits)
            blocks.append((d, m, codes))
            raw += pack_block(d, m, codes, bits)
        out.append(blocks)
    return out, raw


def linear_row(blocks, x):
    """sum_k x[k] * (d*q+m) with exact products summed by math.fsum."""
    terms, mags = [], []
    k = 0
    for d, m, codes in blocks:
        for c in codes:
            w = d * c + m          # exact in binary64
            terms.append(x[k] * w)
            mags.append(abs(x[k]) * abs(w))
            k += 1
    return math.fsum(terms), math.fsum(mags)
