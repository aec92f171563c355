"""The C-ABI library loads, exports every symbol the header declares, and its
host-side argument checks answer without touching a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "aq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(aq_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_exported():
    from paper_2605_24011_b200 import aq
    lib = aq.raw_lib()
    names = _declared()
    assert "aq_pack" in names and "aq_dequant" in names and "aq_linear" in names and "aq_stack_forward" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(aq.SYMBOLS) <= set(names)


def test_status_strings():
    from paper_2605_24011_b200 import aq
    assert aq.status_string(0) == "AQ_OK"
    assert aq.status_string(aq.AQ_ERR_RANGE) == "AQ_ERR_RANGE"
    assert aq.status_string(aq.AQ_ERR_TIMEOUT) == "AQ_ERR_TIMEOUT"


def test_host_side_argument_checks_need_no_gpu():
    from paper_2605_24011_b200 import aq
    lib = aq.raw_lib()
    fake = 0x1000  # never dereferenced: these calls fail in validation
    st, h = aq.aq_pack_raw(5, 32, fake, 16, 32)
    assert st == aq.AQ_ERR_UNSUPPORTED and h is None
    st, h = aq.aq_pack_raw(4, 64, fake, 16, 32)
    assert st == aq.AQ_ERR_UNSUPPORTED
    st, h = aq.aq_pack_raw(4, 32, fake, 16, 33)
    assert st == aq.AQ_ERR_INVALID_ARG
    st, h = aq.aq_pack_raw(4, 32, fake, 0, 32)
    assert st == aq.AQ_ERR_INVALID_ARG
    st, h = aq.aq_pack_raw(4, 32, 0, 16, 32)
    assert st == aq.AQ_ERR_INVALID_ARG
    st, h = aq.aq_pack_raw(4, 32, fake + 4, 16, 32)     # misaligned
    assert st == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_dequant(None, fake, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_linear(None, fake, fake, 1, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_stack_workspace_bytes(None, 1) == 0
    n = C.c_size_t()
    assert lib.aq_export(None, None, 0, C.byref(n)) == aq.AQ_ERR_INVALID_ARG
    lib.aq_free(None)   # no-op
    # attention entry points: the same order of checks (arguments first, the device last)
    assert lib.aq_attn_scratch_bytes(0) == 0 and lib.aq_attn_scratch_bytes(65) == 0
    big = 0x10000
    assert lib.aq_attn_decode(None, big, big, big, 1, 32, 32, 128, 10, 64, 0.0, 0, 2, big, 1 << 30, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_attn_decode(big, big, big, big, 1, 32, 32, 64, 10, 64, 0.0, 0, 2, big, 1 << 30, None) == aq.AQ_ERR_UNSUPPORTED
    assert lib.aq_attn_decode(big, big, big, big, 9, 32, 16, 128, 10, 64, 0.0, 0, 2, big, 1 << 30, None) == aq.AQ_ERR_UNSUPPORTED
    assert lib.aq_attn_decode(big, big, big, big, 1, 32, 32, 128, 65, 64, 0.0, 0, 2, big, 1 << 30, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_rope(None, 32, 128, 0, 10000.0, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_rope(big, 32, 128, 0, 0.5, 0, None) == aq.AQ_ERR_INVALID_ARG          # theta must exceed 1
    assert lib.aq_kv_append(big, big, big, big, 32, 128, 64, 64, 0, None) == aq.AQ_ERR_INVALID_ARG   # pos == L_max
    assert lib.aq_kv_append(big, big, big, big, 32, 64, 0, 64, 0, None) == aq.AQ_ERR_UNSUPPORTED


def test_binding_has_no_fallback():
    """The binding names only the library: no oracle, no torch math."""
    src = open(os.path.join(ROOT, "paper_2605_24011_b200", "aq.py")).read()
    assert "oracle" not in src.replace("no CPU or PyTorch fallback", "")
    for bad in ("torch.matmul", "torch.mm", "F.linear", "@ "):
        assert bad not in src
