"""Plain NumPy oracle for the low-bit block-quantised linear layer.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU baseline.  It shares no code with the CUDA path and is never
tuned for speed.

What it states (paper passages in brackets):

* block format [Section 3, "Weight quantization", Eq. 1]: every B = 32
  consecutive elements of a weight row share one scale and one zero point and
  are coded with the same n bits; a matrix has one bit-width [Section 1,
  "a single bit-width per matrix"].  Eq. 1 writes the decode as
  s_b (q_i - z_b); here it is stored as  scale * q + min  with
  min = -s_b z_b, which names the same set of representable values.
* quantiser: round to the nearest code of the uniform codebook {0..2^n-1}
  [Eq. 1's argmin; the "RTN block quantization" row of the ablation table].
* container [Appendix D]: per tensor the packed integer codes, per-block
  scales and zero points.  The byte order below (little-endian, LSB first) is
  this build's reading; the paper does not print one.
* linear: y = x W_hat^T, activations in half precision [Limitations:
  weight-only quantisation], evaluated here in float64.

Pins: tests/test_oracle_*.py (brute force, closed forms, hand-derived bytes
in tests/golden/).  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BLOCK = 32


def code_max(bits: int) -> int:
    """Largest code L = 2^n - 1 of the uniform n-bit codebook [Eq. 1, Q_n]."""
    if bits not in (2, 3, 4):
        raise ValueError("bits must be 2, 3 or 4")
    return (1 << bits) - 1


# --------------------------------------------------------------------------
# Eq. 1, quantise: per block min/max -> fp16 scale and min -> nearest code
# --------------------------------------------------------------------------
def quantize(W: np.ndarray, bits: int):
    """Round-to-nearest block quantiser [Eq. 1 argmin; RTN ablation row].

    W: float32 [N][K], K % 32 == 0.  Returns (d, m, q): d, m float16
    [N][K/32] (scale, min) and q uint8 [N][K] (codes).

    Each arithmetic step is one correctly rounded IEEE binary32 operation:
        d = f16( f32( f32(max - min) / f32(L) ) )      (ties to even)
        m = f16( min )
        t = f32( f32(w - f32(m)) / f32(d) );  q = clamp(rint(t), 0, L)
    A block whose scale rounds to zero gets all-zero codes.
    """
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    if K % BLOCK:
        raise ValueError("K must be a multiple of 32")
    L = np.float32(code_max(bits))
    Wb = W.reshape(N, K // BLOCK, BLOCK)
    mn = Wb.min(axis=2)
    mx = Wb.max(axis=2)
    rng = (mx - mn).astype(np.float32)            # one fp32 subtraction
    d = (rng / L).astype(np.float32).astype(np.float16)
    m = mn.astype(np.float16)
    d32 = d.astype(np.float32)[:, :, None]
    m32 = m.astype(np.float32)[:, :, None]
    num = (Wb - m32).astype(np.float32)           # one fp32 subtraction
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (num / d32).astype(np.float32)        # one fp32 division
    t = np.where(d32 == 0, np.float32(0), t)
    q = np.clip(np.rint(t), 0, L)                 # rint: ties to even
    return d, m, q.astype(np.uint8).reshape(N, K)


def quantize_ideal(W: np.ndarray, d: np.ndarray, m: np.ndarray, bits: int):
    """Nearest code in exact (float64) arithmetic for given (d, m) [Eq. 1].

    Returns (q_star, frac): q_star = clamp(floor(t + 1/2)) and frac = t -
    floor(t), with t = (w - m)/d in float64; used only to show that the fp32
    quantiser departs from the exact argmin at near-ties alone.
    """
    W = np.asarray(W, dtype=np.float64)
    N, K = W.shape
    Wb = W.reshape(N, K // BLOCK, BLOCK)
    d64 = d.astype(np.float64)[:, :, None]
    m64 = m.astype(np.float64)[:, :, None]
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(d64 == 0, 0.0, (Wb - m64) / d64)
    q = np.clip(np.floor(t + 0.5), 0, code_max(bits))
    return q.astype(np.uint8).reshape(N, K), (t - np.floor(t)).reshape(N, K)


# --------------------------------------------------------------------------
# Appendix D container: canonical bytes
# --------------------------------------------------------------------------
def packed_nbytes(N: int, K: int, bits: int) -> int:
    """Closed form: N * K/32 * (4 + 4n) bytes, i.e. n + 1 bits per weight."""
    return N * (K // BLOCK) * (4 + 4 * bits)


def pack(d: np.ndarray, m: np.ndarray, q: np.ndarray, bits: int) -> np.ndarray:
    """Canonical byte stream [Appendix D: codes + per-block scale + zero point].

    Blocks in row-major order over (row, block); each record is
    [scale fp16 LE][min fp16 LE][codes], the codes forming one little-endian
    integer of 32*n bits in which code i sits at bits [n*i, n*i + n).
    """
    N, nb = d.shape
    assert q.shape == (N, nb * BLOCK)
    L = code_max(bits)
    assert int(q.max(initial=0)) <= L
    # bit t of code i -> stream bit n*i + t; byte p holds stream bits 8p..8p+7
    codebits = np.unpackbits(q.reshape(N, nb, BLOCK, 1), axis=3, bitorder="little")[..., :bits]
    stream = np.packbits(codebits.reshape(N, nb, BLOCK * bits), axis=2, bitorder="little")
    rec = np.empty((N, nb, 4 + 4 * bits), dtype=np.uint8)
    rec[:, :, 0:2] = d.astype("<f2").view(np.uint8).reshape(N, nb, 2)
    rec[:, :, 2:4] = m.astype("<f2").view(np.uint8).reshape(N, nb, 2)
    rec[:, :, 4:] = stream
    return rec.reshape(-1)


def unpack(buf: np.ndarray, bits: int, N: int, K: int):
    """Inverse of pack(): canonical bytes -> (d, m, q)."""
    nb = K // BLOCK
    buf = np.asarray(buf, dtype=np.uint8)
    assert buf.size == packed_nbytes(N, K, bits)
    rec = buf.reshape(N, nb, 4 + 4 * bits)
    d = np.ascontiguousarray(rec[:, :, 0:2]).view("<f2").reshape(N, nb).astype(np.float16)
    m = np.ascontiguousarray(rec[:, :, 2:4]).view("<f2").reshape(N, nb).astype(np.float16)
    sbits = np.unpackbits(np.ascontiguousarray(rec[:, :, 4:]), axis=2, bitorder="little")
    sbits = sbits.reshape(N, nb, BLOCK, bits)
    weights = (1 << np.arange(bits)).astype(np.uint8)
    q = (sbits * weights).sum(axis=3).astype(np.uint8)
    return d, m, q.reshape(N, K)


# --------------------------------------------------------------------------
# Eq. 1, dequantise
# --------------------------------------------------------------------------
def dequant_f32(d: np.ndarray, m: np.ndarray, q: np.ndarray) -> np.ndarray:
    """w_hat = scale * q + min in binary32 [Eq. 1].

    f32(d) * f32(q) is exact (an 11-bit by a 4-bit significand), so the sum is
    the only rounding and a fused multiply-add gives the same bits.
    """
    N, nb = d.shape
    qf = q.reshape(N, nb, BLOCK).astype(np.float32)
    prod = d.astype(np.float32)[:, :, None] * qf
    return (prod + m.astype(np.float32)[:, :, None]).astype(np.float32).reshape(N, nb * BLOCK)


def dequant_f64(d: np.ndarray, m: np.ndarray, q: np.ndarray) -> np.ndarray:
    """w_hat = scale * q + min with no rounding at all (float64 holds it)."""
    N, nb = d.shape
    qf = q.reshape(N, nb, BLOCK).astype(np.float64)
    return (d.astype(np.float64)[:, :, None] * qf + m.astype(np.float64)[:, :, None]).reshape(N, nb * BLOCK)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """binary32 -> bfloat16 bit pattern, round to nearest even (NaN kept quiet)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    nan = np.isnan(x)
    r = np.where(nan, 0x7FC0, r)
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit pattern -> float64 (exact)."""
    u = np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def dequant(d, m, q, dtype: str) -> np.ndarray:
    """Dequantised matrix as bit patterns: 'f16' or 'bf16' -> uint16 [N][K],
    'f32' -> uint32.  One fp32 evaluation, then one round-to-nearest-even cast."""
    w32 = dequant_f32(d, m, q)
    if dtype == "f32":
        return w32.view(np.uint32)
    if dtype == "f16":
        return w32.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        return f32_to_bf16_bits(w32)
    raise ValueError(dtype)


# --------------------------------------------------------------------------
# the linear layer
# --------------------------------------------------------------------------
def linear(d, m, q, x: np.ndarray):
    """y[t][n] = sum_k x[t][k] * w_hat[n][k] in float64, and the magnitude sum
    T[t][n] = sum_k |x[t][k]| |w_hat[n][k]| the tolerance is stated against.

    x: [M][K], already converted exactly from its half-precision storage.
    """
    What = dequant_f64(d, m, q)
    x = np.asarray(x, dtype=np.float64)
    y = np.matmul(x, What.T)
    T = np.matmul(np.abs(x), np.abs(What).T)
    return y, T


def linear_excess(y_test: np.ndarray, y: np.ndarray, T: np.ndarray) -> np.ndarray:
    """|y_test - y| / (2e-3 T + 1e-5): a value <= 1 everywhere passes."""
    return np.abs(np.asarray(y_test, dtype=np.float64) - y) / (2e-3 * T + 1e-5)


# --------------------------------------------------------------------------
# glue between the linears of a transformer block [Section 3: the MLP holds
# gate, up and down matrices]
# --------------------------------------------------------------------------
def silu(g: np.ndarray) -> np.ndarray:
    """SiLU(g) = g / (1 + exp(-g)) in float64."""
    g = np.asarray(g, dtype=np.float64)
    return g / (1.0 + np.exp(-g))


def silu_mul(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    """h = SiLU(g) * u in float64 (the gated-MLP activation)."""
    return silu(g) * np.asarray(u, dtype=np.float64)


def rms_scale(h: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """Per-row scalar 1 / sqrt(mean(h^2) + eps) of a gain-free RMS norm, float64."""
    h = np.asarray(h, dtype=np.float64)
    return 1.0 / np.sqrt((h * h).mean(axis=-1, keepdims=True) + eps)
