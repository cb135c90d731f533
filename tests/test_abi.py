"""The shared library loads without a GPU and exports every entry point that include/dq.h declares."""
import ctypes
import os
import re

import paper_1805_10111_b200 as dq
from paper_1805_10111_b200 import build as dq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dq_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    dq_build.build()
    names = _declared()
    assert len(names) >= 15 and "dq_round" in names and "dq_quantize_sparsify_pack" in names
    L = ctypes.CDLL(dq.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(dq.EXPORTS) == names                      # the Python binding covers the same set
    for n in names:
        assert callable(getattr(dq, n))


def test_host_only_helpers():
    assert dq.dq_packed_bytes(1, 2) == 16 and dq.dq_packed_bytes(128, 2) == 32 and dq.dq_packed_bytes(1000, 4) == 512
    assert dq.dq_packed_bytes(1 << 27, 8) == 1 << 27
    assert "bit width" in dq.dq_strerror(dq.DQ_ERR_BITS)
    assert dq.dq_strerror(0) == "ok"
