"""ctypes binding over libaq.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used by
callers for device memory and streams.  Importing this module loads the
library and raises if it is missing (there is no fallback path).
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AQ_LIBRARY") or os.path.join(_HERE, "libaq.so")   # AQ_LIBRARY: another build of the same library

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_2605_24011_b200.build` "
        "(libaq has no CPU or PyTorch fallback)")

_lib = C.CDLL(LIB_PATH)

AQ_OK, AQ_ERR_INVALID_ARG, AQ_ERR_UNSUPPORTED, AQ_ERR_ALLOC, AQ_ERR_CUDA, AQ_ERR_TIMEOUT, AQ_ERR_ARCH, AQ_ERR_RANGE = range(8)
AQ_F16, AQ_BF16, AQ_F32 = 0, 1, 2
AQ_IN_PLAIN, AQ_IN_RMSNORM, AQ_IN_SILU_MUL = 0, 1, 2
AQ_OUT_STORE, AQ_OUT_ADD = 0, 1
AQ_MAX_M, AQ_DECODE_MAX_M = 4096, 8

SYMBOLS = ("aq_pack", "aq_pack_opt", "aq_pack_sb", "aq_import_sb", "aq_export_sb", "aq_import", "aq_export", "aq_info", "aq_dequant", "aq_linear", "aq_linear_f32out", "aq_linear_noalloc",
           "aq_rbf_gram", "aq_hsic", "aq_sensitivity", "aq_allocate_bits",
           "aq_attn_scratch_bytes", "aq_rope", "aq_kv_append", "aq_attn_decode", "aq_stack_attn_scratch_bytes", "aq_stack_forward_attn",
           "aq_stack_workspace_bytes", "aq_stack_forward", "aq_stack_buffer_offset", "aq_stack_input_offset", "aq_check", "aq_free",
           "aq_set_wait_limit_ns", "aq_debug_decode_hold", "aq_status_string", "aq_last_cuda_error", "aq_kernel_launches")

_H = C.c_void_p


class StackOp(C.Structure):
    _fields_ = [("w", _H), ("src", C.c_int32), ("src2", C.c_int32), ("dst", C.c_int32), ("res", C.c_int32),
                ("in_op", C.c_int32), ("out_op", C.c_int32)]


class Stack(C.Structure):
    _fields_ = [("n_ops", C.c_int32), ("n_bufs", C.c_int32), ("ops", C.POINTER(StackOp)),
                ("buf_width", C.POINTER(C.c_int64))]


_lib.aq_pack.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.POINTER(_H)]
_lib.aq_pack_opt.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.POINTER(_H)]
_lib.aq_pack_opt.restype = C.c_int
_lib.aq_rbf_gram.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_float, C.c_void_p, C.c_int64, C.c_void_p]
_lib.aq_rbf_gram.restype = C.c_int
_lib.aq_attn_scratch_bytes.argtypes = [C.c_int]
_lib.aq_attn_scratch_bytes.restype = C.c_size_t
_lib.aq_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_float, C.c_int, C.c_void_p]
_lib.aq_rope.restype = C.c_int
_lib.aq_kv_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_void_p]
_lib.aq_kv_append.restype = C.c_int
_lib.aq_attn_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int64,
                                C.c_float, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.aq_attn_decode.restype = C.c_int
_lib.aq_hsic.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
_lib.aq_hsic.restype = C.c_int
_lib.aq_sensitivity.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_double, C.c_double, C.c_void_p, C.c_void_p]
_lib.aq_sensitivity.restype = C.c_int
_lib.aq_allocate_bits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.c_double, C.c_void_p,
                                  C.POINTER(C.c_double)]
_lib.aq_allocate_bits.restype = C.c_int
_lib.aq_import.argtypes = [C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(_H)]
_lib.aq_pack_sb.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.POINTER(_H)]
_lib.aq_pack_sb.restype = C.c_int
_lib.aq_import_sb.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(_H)]
_lib.aq_import_sb.restype = C.c_int
_lib.aq_export_sb.argtypes = [_H, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
_lib.aq_export_sb.restype = C.c_int
_lib.aq_export.argtypes = [_H, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
_lib.aq_info.argtypes = [_H, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                         C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
_lib.aq_dequant.argtypes = [_H, C.c_void_p, C.c_int, C.c_void_p]
_lib.aq_linear.argtypes = [_H, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
_lib.aq_linear_f32out.argtypes = [_H, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
_lib.aq_linear_noalloc.argtypes = [_H, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
_lib.aq_linear_noalloc.restype = C.c_int
_lib.aq_stack_workspace_bytes.argtypes = [C.POINTER(Stack), C.c_int]
_lib.aq_stack_workspace_bytes.restype = C.c_size_t
_lib.aq_stack_buffer_offset.argtypes = [C.POINTER(Stack), C.c_int, C.c_int]
_lib.aq_stack_buffer_offset.restype = C.c_size_t
_lib.aq_stack_input_offset.argtypes = [C.POINTER(Stack), C.c_int, C.c_int]
_lib.aq_stack_input_offset.restype = C.c_size_t
_lib.aq_stack_forward.argtypes = [C.POINTER(Stack), C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                  C.c_size_t, C.c_void_p]
_lib.aq_check.argtypes = [C.c_void_p]
_lib.aq_check.restype = C.c_int
_lib.aq_set_wait_limit_ns.argtypes = [C.c_uint64]
_lib.aq_set_wait_limit_ns.restype = C.c_int
_lib.aq_debug_decode_hold.argtypes = [C.c_int]
_lib.aq_debug_decode_hold.restype = None
_lib.aq_free.argtypes = [_H]
_lib.aq_free.restype = None
_lib.aq_status_string.argtypes = [C.c_int]
_lib.aq_status_string.restype = C.c_char_p
_lib.aq_kernel_launches.argtypes = []
_lib.aq_kernel_launches.restype = C.c_uint64
_lib.aq_last_cuda_error.argtypes = []
_lib.aq_last_cuda_error.restype = C.c_char_p
for _n in ("aq_pack", "aq_import", "aq_export", "aq_info", "aq_dequant", "aq_linear", "aq_linear_f32out",
           "aq_stack_forward"):
    getattr(_lib, _n).restype = C.c_int


class AqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = f"{where}: {status_string(status)}"
        if status == AQ_ERR_CUDA:
            msg += f" ({_lib.aq_last_cuda_error().decode()})"
        super().__init__(msg)


def status_string(status: int) -> str:
    return _lib.aq_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != AQ_OK:
        raise AqError(status, where)


def _ptr(t) -> int:
    """Address of a torch tensor's storage (0 for None)."""
    return 0 if t is None else int(t.data_ptr())


def _stream(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    return int(getattr(stream, "cuda_stream", stream))


_DT = {"f16": AQ_F16, "bf16": AQ_BF16, "f32": AQ_F32}


def dtype_code(t) -> int:
    """aq_dtype_t of a torch tensor / dtype / short name."""
    if isinstance(t, str):
        return _DT[t]
    import torch
    dt = t.dtype if hasattr(t, "data_ptr") else t
    return {torch.float16: AQ_F16, torch.bfloat16: AQ_BF16, torch.float32: AQ_F32}[dt]


class Handle:
    """Owns one aq_handle_t."""

    def __init__(self, raw: int):
        self._h = raw

    @property
    def raw(self):
        return self._h

    def free(self):
        if self._h:
            _lib.aq_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def aq_pack(bits: int, block: int, W, stream=None) -> Handle:
    """W: CUDA float32 tensor [N][K] (contiguous)."""
    N, K = W.shape
    h = _H()
    _check(_lib.aq_pack(bits, block, _ptr(W), N, K, _stream(stream), C.byref(h)), "aq_pack")
    return Handle(h.value)


def aq_pack_opt(bits: int, block: int, W, F=None, rounds: int = 4, stream=None) -> Handle:
    """W: CUDA float32 [N][K]; F: CUDA float32 [N][K] Fisher scores or None (= 1)."""
    N, K = W.shape
    h = _H()
    _check(_lib.aq_pack_opt(bits, block, _ptr(W), _ptr(F), rounds, N, K, _stream(stream), C.byref(h)), "aq_pack_opt")
    return Handle(h.value)


def aq_rbf_gram(A, sigma: float, G=None, stream=None):
    """A: CUDA float16 / bfloat16 [K][d]; returns (or fills) the float32 [K][K] RBF kernel matrix."""
    import torch
    K, d = A.shape
    if G is None:
        G = torch.empty((K, K), dtype=torch.float32, device=A.device)
    _check(_lib.aq_rbf_gram(_ptr(A), dtype_code(A), K, d, float(sigma), _ptr(G), G.stride(0), _stream(stream)), "aq_rbf_gram")
    return G


def aq_attn_scratch_bytes(n_kv_heads: int) -> int:
    return int(_lib.aq_attn_scratch_bytes(int(n_kv_heads)))


def aq_rope(x, pos: int, theta: float = 10000.0, stream=None):
    """x: CUDA [n_heads][head_dim] (float16 / bfloat16 / float32), rotated in place for position pos."""
    H, D = x.shape
    _check(_lib.aq_rope(_ptr(x), H, D, int(pos), float(theta), dtype_code(x), _stream(stream)), "aq_rope")
    return x


def aq_kv_append(k_cache, v_cache, k, v, pos: int, stream=None):
    """k_cache, v_cache: CUDA [n_kv_heads][L_max][head_dim]; k, v: CUDA [n_kv_heads][head_dim] of the same type."""
    Hkv, Lmax, D = k_cache.shape
    _check(_lib.aq_kv_append(_ptr(k_cache), _ptr(v_cache), _ptr(k), _ptr(v), Hkv, D, int(pos), Lmax, dtype_code(k_cache),
                             _stream(stream)), "aq_kv_append")


def aq_attn_decode(q, k_cache, v_cache, L: int, out, scratch, scale: float = 0.0, stream=None):
    """q: CUDA [n_heads][head_dim] (one new token) or [M][n_heads][head_dim] (M new tokens, the last M of the L cached
    positions, each seeing the positions up to its own); caches [n_kv_heads][L_max][head_dim]; out: CUDA, the shape of
    q, any of the three types; scratch: CUDA uint8 tensor of at least aq_attn_scratch_bytes(n_kv_heads) bytes."""
    M = 1 if q.dim() == 2 else q.shape[0]
    H, D = q.shape[-2], q.shape[-1]
    Hkv, Lmax, _ = k_cache.shape
    _check(_lib.aq_attn_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), M, H, Hkv, D, int(L), Lmax, float(scale),
                               dtype_code(q), dtype_code(out), _ptr(scratch), scratch.numel() * scratch.element_size(),
                               _stream(stream)), "aq_attn_decode")
    return out


def aq_hsic(KA, KB, out=None, stream=None):
    """KA, KB: CUDA float32 [K][K] (same row pitch); returns a CUDA float64 tensor of one element."""
    import torch
    K = KA.shape[0]
    if out is None:
        out = torch.empty(1, dtype=torch.float64, device=KA.device)
    if KA.stride(0) != KB.stride(0):
        raise ValueError("aq_hsic: the two matrices need the same row pitch")
    _check(_lib.aq_hsic(_ptr(KA), _ptr(KB), K, KA.stride(0), _ptr(out), _stream(stream)), "aq_hsic")
    return out


def aq_sensitivity(KX, KZ, KY, alpha: float, beta: float, out=None, stream=None):
    """Returns a CUDA float64 tensor [S, HSIC(X, Z), HSIC(Z, Y)]."""
    import torch
    K = KZ.shape[0]
    if out is None:
        out = torch.empty(3, dtype=torch.float64, device=KZ.device)
    if not (KX.stride(0) == KZ.stride(0) == KY.stride(0)):
        raise ValueError("aq_sensitivity: the three matrices need the same row pitch")
    _check(_lib.aq_sensitivity(_ptr(KX), _ptr(KZ), _ptr(KY), K, KZ.stride(0), float(alpha), float(beta), _ptr(out), _stream(stream)),
           "aq_sensitivity")
    return out


def aq_allocate_bits(S, numel, layer_of, types, budget: float):
    """Host call: returns (bits per matrix as a numpy int32 array, objective)."""
    import numpy as np
    S = np.ascontiguousarray(S, dtype=np.float64)
    numel = np.ascontiguousarray(numel, dtype=np.int64)
    layer_of = np.ascontiguousarray(layer_of, dtype=np.int32)
    types = np.ascontiguousarray(types, dtype=np.int32)
    n = S.shape[0]
    if numel.shape[0] != n or layer_of.shape[0] != n:
        raise ValueError("aq_allocate_bits: arrays of different length")
    bits = np.empty(n, dtype=np.int32)
    obj = C.c_double()
    _check(_lib.aq_allocate_bits(S.ctypes.data, numel.ctypes.data, layer_of.ctypes.data, n, types.ctypes.data, types.shape[0],
                                 float(budget), bits.ctypes.data, C.byref(obj)), "aq_allocate_bits")
    return bits, obj.value


def aq_pack_raw(bits, block, w_ptr, N, K, stream_ptr=0):
    """Direct call with raw addresses; returns (status, handle value or None)."""
    h = _H()
    st = _lib.aq_pack(bits, block, w_ptr, N, K, stream_ptr, C.byref(h))
    return st, h.value


def aq_import(bits: int, block: int, N: int, K: int, canon, stream=None) -> Handle:
    """canon: host bytes / numpy uint8 array holding the canonical stream."""
    import numpy as np
    buf = np.ascontiguousarray(np.frombuffer(canon, dtype=np.uint8) if isinstance(canon, (bytes, bytearray)) else canon,
                               dtype=np.uint8)
    h = _H()
    _check(_lib.aq_import(bits, block, N, K, buf.ctypes.data, buf.size, _stream(stream), C.byref(h)), "aq_import")
    return Handle(h.value)


def aq_pack_sb(bits: int, W, block: int = 32, sblock: int = 8, stream=None) -> Handle:
    """Super-block form: W CUDA float32 [N][K] (contiguous), K % 256 == 0."""
    N, K = W.shape
    h = _H()
    _check(_lib.aq_pack_sb(bits, block, sblock, _ptr(W), N, K, _stream(stream), C.byref(h)), "aq_pack_sb")
    return Handle(h.value)


def aq_import_sb(bits: int, N: int, K: int, canon, block: int = 32, sblock: int = 8, stream=None) -> Handle:
    """canon: host bytes / numpy uint8 array holding the canonical super-block stream."""
    import numpy as np
    buf = np.ascontiguousarray(np.frombuffer(canon, dtype=np.uint8) if isinstance(canon, (bytes, bytearray)) else canon,
                               dtype=np.uint8)
    h = _H()
    _check(_lib.aq_import_sb(bits, block, sblock, N, K, buf.ctypes.data, buf.size, _stream(stream), C.byref(h)), "aq_import_sb")
    return Handle(h.value)


def aq_export_sb(h: Handle, allow_range_error: bool = False):
    """Canonical super-block bytes as a numpy uint8 array."""
    import numpy as np
    n = C.c_size_t()
    _check(_lib.aq_export_sb(h.raw, None, 0, C.byref(n)), "aq_export_sb(size)")
    out = np.empty(n.value, dtype=np.uint8)
    st = _lib.aq_export_sb(h.raw, out.ctypes.data, out.size, C.byref(n))
    if not (allow_range_error and st == AQ_ERR_RANGE):
        _check(st, "aq_export_sb")
    return out


def aq_export(h: Handle, allow_range_error: bool = False):
    """Canonical bytes as a numpy uint8 array."""
    import numpy as np
    n = C.c_size_t()
    _check(_lib.aq_export(h.raw, None, 0, C.byref(n)), "aq_export(size)")
    out = np.empty(n.value, dtype=np.uint8)
    st = _lib.aq_export(h.raw, out.ctypes.data, out.size, C.byref(n))
    if not (allow_range_error and st == AQ_ERR_RANGE):
        _check(st, "aq_export")
    return out


def aq_info(h: Handle):
    bits, block = C.c_int(), C.c_int()
    N, K = C.c_int64(), C.c_int64()
    pb, db = C.c_size_t(), C.c_size_t()
    st = _lib.aq_info(h.raw, C.byref(bits), C.byref(block), C.byref(N), C.byref(K), C.byref(pb), C.byref(db))
    return {"status": st, "bits": bits.value, "block": block.value, "N": N.value, "K": K.value,
            "packed_bytes": pb.value, "device_bytes": db.value}


def aq_dequant(h: Handle, out, stream=None):
    """out: CUDA tensor [N][K] of float16 / bfloat16 / float32."""
    _check(_lib.aq_dequant(h.raw, _ptr(out), dtype_code(out), _stream(stream)), "aq_dequant")
    return out


def aq_linear(h: Handle, x, y, M: int | None = None, stream=None):
    """x: CUDA [M][K] float16/bfloat16; y: CUDA [M][N] of the same dtype, or float32."""
    M = int(x.shape[0]) if M is None else M
    if dtype_code(y) == AQ_F32:
        _check(_lib.aq_linear_f32out(h.raw, _ptr(x), _ptr(y), M, dtype_code(x), _stream(stream)), "aq_linear_f32out")
    else:
        if dtype_code(y) != dtype_code(x):
            raise AqError(AQ_ERR_INVALID_ARG, "aq_linear: y dtype must equal x dtype (or float32)")
        _check(_lib.aq_linear(h.raw, _ptr(x), _ptr(y), M, dtype_code(x), _stream(stream)), "aq_linear")
    return y


def aq_linear_noalloc(h: Handle, x, y, M: int | None = None, stream=None):
    """aq_linear for M <= 8 that reserves no memory: the sums are built in a fixed
    512 KiB array inside the library instead of scratch owned by the handle.  For
    callers that may not allocate on the device (deadline loops, fixed memory
    budgets).  x, y: CUDA tensors of the same half-precision dtype.  Calls on one
    GPU share the array, so they must not overlap."""
    M = int(x.shape[0]) if M is None else M
    _check(_lib.aq_linear_noalloc(h.raw, _ptr(x), _ptr(y), M, dtype_code(x), _stream(stream)), "aq_linear_noalloc")
    return y


class Program:
    """Host-side aq_stack_t builder.  ops: dicts with keys w (Handle), src, dst
    and optionally src2, res, in_op, out_op."""

    def __init__(self, buf_width, ops):
        self.handles = [o["w"] for o in ops]           # keep alive
        self._ops = (StackOp * len(ops))()
        for i, o in enumerate(ops):
            self._ops[i] = StackOp(o["w"].raw, o["src"], o.get("src2", -1), o["dst"], o.get("res", -1),
                                   o.get("in_op", AQ_IN_PLAIN), o.get("out_op", AQ_OUT_STORE))
        self._w = (C.c_int64 * len(buf_width))(*buf_width)
        self.c = Stack(len(ops), len(buf_width), self._ops, self._w)
        self.buf_width = list(buf_width)
        self.ops = ops

    def workspace_bytes(self, M: int) -> int:
        return int(_lib.aq_stack_workspace_bytes(C.byref(self.c), M))

    def buffer_offset(self, M: int, b: int) -> int:
        return int(_lib.aq_stack_buffer_offset(C.byref(self.c), M, b))

    def input_offset(self, M: int, op: int) -> int:
        return int(_lib.aq_stack_input_offset(C.byref(self.c), M, op))


def aq_stack_workspace_bytes(prog: Program, M: int) -> int:
    return prog.workspace_bytes(M)


def aq_stack_forward(prog: Program, x0, out, out_buf: int, M: int, workspace, stream=None):
    """x0: CUDA [M][width0] f16/bf16; out: CUDA [M][width[out_buf]] same dtype or None;
    workspace: CUDA uint8 tensor of at least workspace_bytes(M)."""
    _check(_lib.aq_stack_forward(C.byref(prog.c), _ptr(x0), _ptr(out), out_buf, M, dtype_code(x0), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)), "aq_stack_forward")
    return out


class StackAttn(C.Structure):
    _fields_ = [("after_op", C.c_int32), ("q_buf", C.c_int32), ("k_buf", C.c_int32), ("v_buf", C.c_int32), ("dst_buf", C.c_int32),
                ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("pad_", C.c_int32),
                ("k_cache_dev", C.c_void_p), ("v_cache_dev", C.c_void_p), ("L_max", C.c_int64)]


def aq_stack_attn_scratch_bytes(n_heads: int, n_kv_heads: int, M: int) -> int:
    _lib.aq_stack_attn_scratch_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
    _lib.aq_stack_attn_scratch_bytes.restype = C.c_size_t
    return int(_lib.aq_stack_attn_scratch_bytes(n_heads, n_kv_heads, M))


def aq_stack_forward_attn(prog: Program, attn, pos: int, x0, out, out_buf: int, M: int, workspace, scratch, theta: float = 10000.0,
                          stream=None):
    """aq_stack_forward with attention over key/value caches between the linears.  attn: list of dicts with keys
    after_op, q_buf, k_buf, v_buf, dst_buf, n_heads, n_kv_heads, k_cache, v_cache (CUDA [n_kv_heads][L_max][128] of x0's
    type); pos: position of the first of the M new tokens; scratch: CUDA uint8 tensor (aq_stack_attn_scratch_bytes)."""
    arr = (StackAttn * max(1, len(attn)))()
    for i, t in enumerate(attn):
        arr[i] = StackAttn(t["after_op"], t["q_buf"], t["k_buf"], t["v_buf"], t["dst_buf"], t["n_heads"], t["n_kv_heads"], 0,
                           _ptr(t["k_cache"]), _ptr(t["v_cache"]), t["k_cache"].shape[1])
    _lib.aq_stack_forward_attn.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                           C.c_int, C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
    _lib.aq_stack_forward_attn.restype = C.c_int
    _check(_lib.aq_stack_forward_attn(C.byref(prog.c), arr, len(attn), int(pos), float(theta), _ptr(x0), _ptr(out), out_buf, M,
                                      dtype_code(x0), _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(scratch),
                                      scratch.numel() * scratch.element_size(), _stream(stream)), "aq_stack_forward_attn")
    return out


def stack_buffer(prog: Program, workspace, M: int, b: int):
    """float32 view [M][width[b]] of buffer b inside the workspace."""
    import torch
    off = prog.buffer_offset(M, b)
    n = M * prog.buf_width[b]
    return workspace[off:off + 4 * n].view(torch.float32).view(M, prog.buf_width[b])


def aq_check(stream=None) -> int:
    """Synchronise the stream; raise if a device-side wait timed out or CUDA failed."""
    _check(_lib.aq_check(_stream(stream)), "aq_check")
    return AQ_OK


def stack_input(prog: Program, workspace, M: int, op: int, dtype):
    """[M][K] view (activation dtype) of the rounded input vector op `op` consumed."""
    off = prog.input_offset(M, op)
    K = prog.buf_width[prog.ops[op]["src"]]
    return workspace[off:off + 2 * M * K].view(dtype).view(M, K)


def aq_set_wait_limit_ns(ns: int) -> int:
    """Limit of every device-side wait of the decode-stack kernel (0: the default)."""
    _check(_lib.aq_set_wait_limit_ns(int(ns)), "aq_set_wait_limit_ns")
    return AQ_OK


def aq_debug_decode_hold(on: bool) -> None:
    """Testing only: decode tables built while on wait for a contribution that never comes."""
    _lib.aq_debug_decode_hold(1 if on else 0)


def aq_kernel_launches() -> int:
    return int(_lib.aq_kernel_launches())


def raw_lib():
    """The ctypes library object (tests of the ABI itself)."""
    return _lib
