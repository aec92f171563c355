"""Plain NumPy oracle for the low-bit block-quantised linear layer.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU baseline.  It shares no code with the CUDA path and is never
tuned for speed.

What it states (paper passages in brackets):

* block format [Section 3, "Weight quantization", Eq. 1]: every B = 32
  consecutive elements of a weight row share one scale and one zero point and
  are coded with the same n bits; every matrix has one bit-width [Section 1 and
  Section 4.1: the inter-tensor stage assigns a width per matrix].  Eq. 1 writes the decode as
  s_b (q_i - z_b); here it is stored as  scale * q + min  with
  min = -s_b z_b, which names the same set of representable values.
* quantiser: round to the nearest code of the uniform codebook {0..2^n-1}
  [Eq. 1's argmin; the "RTN block quantization" row of the ablation table].
* container [Appendix D]: per tensor the packed integer codes, per-block
  scales and zero points.  The byte order below (little-endian, LSB first) is
  this library's reading; the paper does not print one.
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


# --------------------------------------------------------------------------
# Intra-tensor scale optimisation [Section 3.3, Eq. 10 and Eq. 11]
# --------------------------------------------------------------------------
# Eq. 10: per block, minimise Phi_b = sum_i omega_i (w_i - w_hat_i)^2 with
# omega_i = F_ii sqrt(sigma_b^2 + w_i^2), sigma_b^2 the block's mean squared weight and F the
# diagonal Fisher scores (F = 1: the magnitude-weighted row of the ablation table).
# Eq. 11 alternates nearest codes for a fixed scale with the closed-form scale for fixed codes.
# The paper writes the symmetric decode s_b q_i; this container decodes scale * q + min
# (Eq. 1 with a zero point), so the least-squares step here solves for the pair (scale, min):
# the same stationarity condition with two unknowns.  Reading taken where the paper is silent:
# start from the round-to-nearest parameters; stop when the normal equations are singular or the
# scale is not positive; keep the round-to-nearest block when the optimised one, after rounding
# its parameters to binary16, does not lower Phi_b.

def _omega(Wb: np.ndarray, Fb) -> np.ndarray:
    """Eq. 10 weights in float64; Wb [..., 32]."""
    Wb = Wb.astype(np.float64)
    sig2 = (Wb * Wb).mean(axis=-1, keepdims=True)
    om = np.sqrt(sig2 + Wb * Wb)
    return om if Fb is None else om * Fb.astype(np.float64)


def block_phi(W: np.ndarray, d, m, q, F=None) -> np.ndarray:
    """Phi_b of Eq. 10 in float64 for decoded values d q + m; returns [N][K/32]."""
    N, K = W.shape
    Wb = np.asarray(W, dtype=np.float64).reshape(N, K // BLOCK, BLOCK)
    Fb = None if F is None else np.asarray(F).reshape(N, K // BLOCK, BLOCK)
    what = (np.asarray(d, dtype=np.float64)[:, :, None] * np.asarray(q, dtype=np.float64).reshape(N, K // BLOCK, BLOCK)
            + np.asarray(m, dtype=np.float64)[:, :, None])
    return (_omega(Wb, Fb) * (Wb - what) ** 2).sum(axis=2)


def scale_opt_ideal(W: np.ndarray, bits: int, F=None, rounds: int = 4):
    """Eq. 11 in float64 from the round-to-nearest start.  Returns (s, m, q, trace): unrounded
    parameters [N][K/32], codes [N][K] and Phi_b after every half step (q step, then
    least-squares step), which Eq. 11 says never goes up."""
    N, K = W.shape
    L = float(code_max(bits))
    Wb = np.asarray(W, dtype=np.float64).reshape(N, K // BLOCK, BLOCK)
    Fb = None if F is None else np.asarray(F).reshape(N, K // BLOCK, BLOCK)
    om = _omega(Wb, Fb)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    s = (mx - mn) / L
    m = mn.copy()
    live = s > 0
    q = np.zeros_like(Wb)
    trace = []
    phi = lambda: (om * (Wb - (s[:, :, None] * q + m[:, :, None])) ** 2).sum(axis=2)
    for _ in range(rounds):
        with np.errstate(divide="ignore", invalid="ignore"):
            t = np.where(live[:, :, None], (Wb - m[:, :, None]) / np.where(live, s, 1.0)[:, :, None], 0.0)
        q = np.clip(np.floor(t + 0.5), 0, L)
        trace.append(phi())
        S0, S1, S2 = om.sum(axis=2), (om * q).sum(axis=2), (om * q * q).sum(axis=2)
        Sw, Swq = (om * Wb).sum(axis=2), (om * Wb * q).sum(axis=2)
        det = S0 * S2 - S1 * S1
        with np.errstate(divide="ignore", invalid="ignore"):
            s_new = (S0 * Swq - S1 * Sw) / det
            m_new = (Sw - s_new * S1) / S0
        ok = live & (det > 0) & np.isfinite(s_new) & (s_new > 0)
        s = np.where(ok, s_new, s)
        m = np.where(ok, m_new, m)
        trace.append(phi())
    return s, m, q.astype(np.uint8).reshape(N, K), trace


def _sum32(x: np.ndarray) -> np.ndarray:
    """Sum of the last axis (32 float32 values) in the stated order: eight at a time left to
    right, then (g0 + g1) + (g2 + g3).  One binary32 rounding per addition."""
    g = x.reshape(x.shape[:-1] + (4, 8)).astype(np.float32)
    a = g[..., 0]
    for i in range(1, 8):
        a = (a + g[..., i]).astype(np.float32)
    return ((a[..., 0] + a[..., 1]).astype(np.float32) + (a[..., 2] + a[..., 3]).astype(np.float32)).astype(np.float32)


def quantize_opt(W: np.ndarray, bits: int, F=None, rounds: int = 4):
    """Scale-optimised block quantiser [Eq. 10, Eq. 11], same outputs as quantize().

    Every step is one correctly rounded binary32 operation in a stated order (sums: _sum32),
    except the 2 x 2 solve, done in binary64 from the binary32 sums, one rounding per operation.
    The paper fixes neither the precision nor the order of the sums; both are a reading taken so
    that two implementations can agree byte for byte.  What ties this function to the plain
    statement (scale_opt_ideal, float64) is tests/test_oracle_scale_opt.py: same parameters in
    all but the blocks where a near-tie parts the two runs, and a Phi_b no worse than the better
    plain candidate.
        sigma2 = sum32(w w) / 32;  omega = F * sqrt(sigma2 + w w)            (F omitted when None)
        s = (max - min) / L, mm = min
        repeat `rounds` times, while s > 0:
            q = clamp(rint((w - mm) / s), 0, L)
            S0 = sum32(omega), S1 = sum32(omega q), S2 = sum32((omega q) q),
            Sw = sum32(omega w), Swq = sum32((omega w) q)
            det = S0 S2 - S1 S1; stop unless det > 0
            s' = (S0 Swq - S1 Sw) / det; stop unless s' is finite and > 0
            mm = f32((Sw - s' S1) / S0), s = f32(s')
    Two candidates are then coded exactly as quantize() codes a block from its binary16
    parameters: (f16((max - min)/L), f16(min)) and (f16(s), f16(mm)); the second is kept when its
    Phi = sum32(omega (w - (d q + m))^2) is smaller, its scale is finite and non-zero.
    """
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    if K % BLOCK:
        raise ValueError("K must be a multiple of 32")
    L = np.float32(code_max(bits))
    f32 = np.float32
    Wb = W.reshape(N, K // BLOCK, BLOCK)
    ww = (Wb * Wb).astype(f32)
    sig2 = (_sum32(ww) / f32(32)).astype(f32)
    om = np.sqrt((sig2[:, :, None] + ww).astype(f32)).astype(f32)
    if F is not None:
        om = (np.ascontiguousarray(F, dtype=f32).reshape(N, K // BLOCK, BLOCK) * om).astype(f32)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    s = ((mx - mn).astype(f32) / L).astype(f32)
    mm = mn.copy()
    live = s > 0
    ow = (om * Wb).astype(f32)
    S0, Sw = _sum32(om), _sum32(ow)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        for _ in range(rounds):
            t = ((Wb - mm[:, :, None]).astype(f32) / np.where(live, s, f32(1))[:, :, None]).astype(f32)
            q = np.clip(np.rint(t), 0, L).astype(f32)
            oq = (om * q).astype(f32)
            S1, S2, Swq = _sum32(oq), _sum32((oq * q).astype(f32)), _sum32((ow * q).astype(f32))
            a0, a1, a2, aw, awq = (v.astype(np.float64) for v in (S0, S1, S2, Sw, Swq))
            det = a0 * a2 - a1 * a1
            s_new = (a0 * awq - a1 * aw) / det
            m_new = (aw - s_new * a1) / a0
            ok = live & (det > 0) & np.isfinite(s_new) & (s_new > 0)
            live = ok
            s = np.where(ok, s_new.astype(f32), s)
            mm = np.where(ok, m_new.astype(f32), mm)

        def code(dh, mh):
            d32, m32 = dh.astype(f32)[:, :, None], mh.astype(f32)[:, :, None]
            t = ((Wb - m32).astype(f32) / d32).astype(f32)
            t = np.where(d32 == 0, f32(0), t)
            q = np.clip(np.rint(t), 0, L).astype(f32)
            what = ((d32 * q).astype(f32) + m32).astype(f32)
            r = (Wb - what).astype(f32)
            return q, _sum32((om * (r * r).astype(f32)).astype(f32))

        dA, mA = ((mx - mn).astype(f32) / L).astype(f32).astype(np.float16), mn.astype(np.float16)
        dB, mB = s.astype(np.float16), mm.astype(np.float16)
        qA, phiA = code(dA, mA)
        qB, phiB = code(dB, mB)
    dB32 = dB.astype(f32)
    useB = np.isfinite(dB32) & (dB32 != 0) & np.isfinite(mB.astype(f32)) & (phiB < phiA)
    d = np.where(useB, dB, dA)
    m = np.where(useB, mB, mA)
    q = np.where(useB[:, :, None], qB, qA)
    return d, m, q.astype(np.uint8).reshape(N, K)


# --------------------------------------------------------------------------
# Super-blocks: two-level block parameters [Section 3, "Weight quantization"]
# --------------------------------------------------------------------------
# The paper's format is a block / super-block hierarchy: S consecutive blocks form a super-block
# whose own scale and zero point compress the per-block (s_b, z_b).  It prints neither S nor the
# width of the compressed parameters.  Reading taken here: S = 8 blocks (256 weights); the block
# scales and the block minima of a super-block are each coded with Eq. 1's rule one level up,
# with 6-bit codes u_b, v_b in {0..63}:
#     scale_b = D u_b                     (symmetric special case: zero point 0; D binary16)
#     min_b   = Mn + Dm v_b               (asymmetric: Mn, Dm binary16; Mn plays the zero point)
# and the decoded block parameters are rounded to binary16, so that a super-block matrix decodes
# exactly like a plain one with those parameters: w_hat = f16(scale_b) q + f16(min_b).
# Stored bits per weight: n + (3 * 16 + 8 * 12) / 256 = n + 0.5625 (against n + 1).
SUPER = 8
SUB_MAX = 63


def sb_block_params(D, Dm, Mn, u, v):
    """Decoded per-block (scale, min) as binary16 [N][K/32] from the super-block parameters
    D, Dm, Mn [N][K/256] (binary16) and the 6-bit codes u, v [N][K/32].  One rounding each:
    scale = f16(D u) (the product is exact in binary32), min = f16(fma(Dm, v, Mn))."""
    D32 = np.repeat(np.asarray(D, dtype=np.float16).astype(np.float32), SUPER, axis=1)
    Dm64 = np.repeat(np.asarray(Dm, dtype=np.float16).astype(np.float64), SUPER, axis=1)
    Mn64 = np.repeat(np.asarray(Mn, dtype=np.float16).astype(np.float64), SUPER, axis=1)
    with np.errstate(over="ignore", invalid="ignore"):
        d = (D32 * u.astype(np.float32)).astype(np.float32).astype(np.float16)
        # fused multiply-add: the exact value (float64 holds it) rounded once to binary32, then to binary16
        m = (Dm64 * v.astype(np.float64) + Mn64).astype(np.float32).astype(np.float16)
    return d, m


def quantize_sb(W: np.ndarray, bits: int):
    """Round-to-nearest quantiser with super-block parameters.  W float32 [N][K], K % 256 == 0.
    Returns (D, Dm, Mn, u, v, q).  Every step is one correctly rounded binary32 operation:
        per block:        s = (max - min) / L,  mn = min                         (as quantize(), before binary16)
        per super-block:  D  = f16(max_b s / 63);              u_b = clamp(rint(s_b / D), 0, 63)   (0 when D = 0)
                          Mn = f16(min_b mn_b);  Dm = f16(max(0, max_b mn_b - Mn) / 63)
                          v_b = clamp(rint((mn_b - Mn) / Dm), 0, 63)                               (0 when Dm = 0)
        codes:            q = clamp(rint((w - min_b) / scale_b), 0, L) with the DECODED block parameters
                          (sb_block_params), 0 everywhere when scale_b = 0."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    if K % (BLOCK * SUPER):
        raise ValueError("K must be a multiple of 256")
    f32 = np.float32
    L = f32(code_max(bits))
    Wb = W.reshape(N, K // BLOCK, BLOCK)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    s = ((mx - mn).astype(f32) / L).astype(f32)
    sS, mnS = s.reshape(N, -1, SUPER), mn.reshape(N, -1, SUPER)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        D = (sS.max(axis=2) / f32(SUB_MAX)).astype(f32).astype(np.float16)
        D32 = D.astype(f32)[:, :, None]
        u = np.where(D32 == 0, f32(0), np.clip(np.rint((sS / D32).astype(f32)), 0, SUB_MAX))
        Mn = mnS.min(axis=2).astype(np.float16)
        Mn32 = Mn.astype(f32)
        Dm = (np.maximum((mnS.max(axis=2) - Mn32).astype(f32), f32(0)) / f32(SUB_MAX)).astype(f32).astype(np.float16)
        Dm32 = Dm.astype(f32)[:, :, None]
        t = ((mnS - Mn32[:, :, None]).astype(f32) / Dm32).astype(f32)
        v = np.where(Dm32 == 0, f32(0), np.clip(np.rint(t), 0, SUB_MAX))
    u = np.nan_to_num(u).astype(np.uint8).reshape(N, K // BLOCK)
    v = np.nan_to_num(v).astype(np.uint8).reshape(N, K // BLOCK)
    d, m = sb_block_params(D, Dm, Mn, u, v)
    d32, m32 = d.astype(f32)[:, :, None], m.astype(f32)[:, :, None]
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        tq = ((Wb - m32).astype(f32) / d32).astype(f32)
    tq = np.where(d32 == 0, f32(0), tq)
    q = np.clip(np.rint(tq), 0, L)
    return D, Dm, Mn, u, v, q.astype(np.uint8).reshape(N, K)


def packed_nbytes_sb(N: int, K: int, bits: int) -> int:
    """Closed form: per super-block 6 + 12 + 8 * 4n bytes, i.e. n + 0.5625 bits per weight."""
    return N * (K // (BLOCK * SUPER)) * (18 + 32 * bits)


def pack_sb(D, Dm, Mn, u, v, q, bits: int) -> np.ndarray:
    """Canonical bytes of a super-block matrix: super-blocks in row-major order over (row, super-block); a record is
    [D f16 LE][Dm f16 LE][Mn f16 LE][12 bytes: one little-endian integer of 96 bits in which block b's u sits at bits
    [12 b, 12 b + 6) and its v at [12 b + 6, 12 b + 12)][codes of the 8 blocks: 8 x 4n bytes, each block as in pack()]."""
    N, ns = D.shape
    nb = ns * SUPER
    assert u.shape == (N, nb) and v.shape == (N, nb) and q.shape == (N, nb * BLOCK)
    assert int(u.max(initial=0)) <= SUB_MAX and int(v.max(initial=0)) <= SUB_MAX and int(q.max(initial=0)) <= code_max(bits)
    rec = np.empty((N, ns, 18 + 32 * bits), dtype=np.uint8)
    for a, off in ((D, 0), (Dm, 2), (Mn, 4)):
        rec[:, :, off:off + 2] = np.asarray(a).astype("<f2").view(np.uint8).reshape(N, ns, 2)
    uv = u.astype(np.uint16) | (v.astype(np.uint16) << 6)                      # 12 bits per block
    uvbits = np.unpackbits(uv.reshape(N, ns, SUPER, 1).view(np.uint8), axis=3, bitorder="little")[..., :12]
    rec[:, :, 6:18] = np.packbits(uvbits.reshape(N, ns, SUPER * 12), axis=2, bitorder="little")
    codebits = np.unpackbits(q.reshape(N, ns, SUPER * BLOCK, 1), axis=3, bitorder="little")[..., :bits]
    rec[:, :, 18:] = np.packbits(codebits.reshape(N, ns, SUPER * BLOCK * bits), axis=2, bitorder="little")
    return rec.reshape(-1)


def unpack_sb(buf: np.ndarray, bits: int, N: int, K: int):
    """Inverse of pack_sb(): canonical bytes -> (D, Dm, Mn, u, v, q)."""
    ns = K // (BLOCK * SUPER)
    buf = np.asarray(buf, dtype=np.uint8)
    assert buf.size == packed_nbytes_sb(N, K, bits)
    rec = buf.reshape(N, ns, 18 + 32 * bits)
    f = lambda off: np.ascontiguousarray(rec[:, :, off:off + 2]).view("<f2").reshape(N, ns).astype(np.float16)
    D, Dm, Mn = f(0), f(2), f(4)
    uvbits = np.unpackbits(np.ascontiguousarray(rec[:, :, 6:18]), axis=2, bitorder="little").reshape(N, ns, SUPER, 12)
    w6 = (1 << np.arange(6)).astype(np.uint8)
    u = (uvbits[..., :6] * w6).sum(axis=3).astype(np.uint8).reshape(N, ns * SUPER)
    v = (uvbits[..., 6:] * w6).sum(axis=3).astype(np.uint8).reshape(N, ns * SUPER)
    cb = np.unpackbits(np.ascontiguousarray(rec[:, :, 18:]), axis=2, bitorder="little").reshape(N, ns, SUPER * BLOCK, bits)
    q = (cb * (1 << np.arange(bits)).astype(np.uint8)).sum(axis=3).astype(np.uint8).reshape(N, K)
    return D, Dm, Mn, u, v, q
