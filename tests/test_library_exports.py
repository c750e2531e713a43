"""CPU-side checks of the boundary: the shared library builds, loads and exports every function
include/goq.h declares; size queries behave; no compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def goq():
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq as g
    g.lib()
    return g


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "goq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(goq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(goq):
    names = _declared_functions()
    assert {"goq_pack", "goq_unpack", "goq_gemv", "goq_gemm", "goq_packed_bytes"} <= set(names)
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2605_26092_b200", "libgoq.so"))
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(goq.EXPORTS) == names


def test_size_queries(goq):
    d = goq.desc(4096, 4096, 128, 3)
    # 3 code bits + 0.75 record bits per weight + one fp16 pair per 128 weights = 4.00 bits per weight
    assert goq.algorithmic_bytes(d) == 4096 * 4096 * 4 // 8
    # packed: one 32-bit word per 8 weights + 4 bytes per (row, group)
    assert goq.packed_bytes(d) == 4096 * 4096 // 2 + 4096 * 32 * 4
    assert goq.algorithmic_bytes(goq.desc(256, 256, 64, 3)) == 256 * 256 * 15 // 32 + 256 * 4 * 4
    # padding to 16 rows x 128 k
    d2 = goq.desc(40, 192, 64, 3)
    assert goq.packed_bytes(d2) == 48 * 256 // 2 + 48 * 4 * 4
    assert goq.packed_bytes(goq.desc(40, 192, 64, 4)) > goq.packed_bytes(d2)
    for bad in [goq.desc(0, 128, 64, 3), goq.desc(16, 100, 64, 3), goq.desc(16, 128, 24, 3),
                goq.desc(16, 128, 64, 5), goq.desc(16, 128, 64, 3, layout=7), goq.desc(16, 128, 256, 3)]:
        assert goq.packed_bytes(bad) == 0 and goq.algorithmic_bytes(bad) == 0


def test_status_strings(goq):
    seen = {goq.status_string(s) for s in range(9)}
    assert len(seen) == 9 and "ok" in seen


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2605_26092_b200 import goq as g
    monkeypatch.setattr(g, "_lib", None)
    monkeypatch.setattr(g, "_LIB_PATH", "/nonexistent/libgoq.so")
    with pytest.raises(ImportError):
        g.lib()
