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


class _FakeBuffer:
    """Stands in for a device tensor in make_sequence: goq_sequence_order only compares addresses."""
    def __init__(self, addr):
        self.addr = addr

    def data_ptr(self):
        return self.addr


def test_sequence_order_is_decided_from_the_address_ranges(goq):
    """goq_sequence_order runs on the host and dereferences nothing: items are described with made-up addresses.
    Cases: nothing shared; the whole bf16 output of the previous item; a slice of it (batch 1) at a multiple of 8
    channels and at an odd start; an fp32 producer; an input that spans two outputs; an output buffer written twice; a
    flagged item; batch 2 reading all of a batch-2 output and reading a slice of it."""
    d44 = goq.desc(4096, 4096, 128, 3)
    d_half = goq.desc(256, 2048, 128, 3)     # reads 2048 channels
    d_two = goq.desc(256, 8192, 128, 3)      # reads 8192 channels
    B = 1 << 20
    X0, Y0, Y1, Y2, Y3, Y4 = (_FakeBuffer(0x10000000 + i * B) for i in range(6))
    pk = _FakeBuffer(0x70000000)
    def order(items):
        kinds, sources = goq.sequence_order(goq.make_sequence(items))
        return list(zip(kinds, sources))
    N, D, Bar = goq.ORDER_NONE, goq.ORDER_DATA, goq.ORDER_BARRIER
    # independent items
    assert order([(d44, pk, X0, 1, Y0, goq.BF16, False), (d44, pk, X0, 1, Y1, goq.BF16, False)]) == [(N, -1), (N, -1)]
    # a chain through whole outputs, then an fp32 producer, then a flagged item
    got = order([(d44, pk, X0, 1, Y0, goq.BF16, False), (d44, pk, Y0, 1, Y1, goq.BF16, False),
                 (d44, pk, Y1, 1, Y2, goq.F32, False), (d44, pk, Y2, 1, Y3, goq.BF16, False),
                 (d44, pk, X0, 1, Y4, goq.BF16, True)])
    assert got == [(N, -1), (D, 0), (D, 1), (Bar, -1), (Bar, -1)]
    # slices of a batch-1 output: channel 2048 (a multiple of 8) is data flow, channel 2052 is not
    s_ok, s_odd = _FakeBuffer(Y0.addr + 2048 * 2), _FakeBuffer(Y0.addr + 2052 * 2)
    got = order([(d44, pk, X0, 1, Y0, goq.BF16, False), (d_half, pk, s_ok, 1, Y1, goq.BF16, False),
                 (d_half, pk, s_odd, 1, Y2, goq.BF16, False)])
    assert got == [(N, -1), (D, 0), (Bar, -1)]
    # one input spanning two outputs that lie side by side; then an output buffer written a second time
    y_lo, y_hi = _FakeBuffer(Y0.addr), _FakeBuffer(Y0.addr + 4096 * 2)
    got = order([(d44, pk, X0, 1, y_lo, goq.BF16, False), (d44, pk, X0, 1, y_hi, goq.BF16, False),
                 (d_two, pk, y_lo, 1, Y1, goq.BF16, False), (d44, pk, X0, 1, y_lo, goq.BF16, False)])
    assert got == [(N, -1), (N, -1), (Bar, -1), (Bar, -1)]
    # batch 2: the whole output is data flow, a narrower view of it is not
    got = order([(d44, pk, X0, 2, Y0, goq.BF16, False), (d44, pk, Y0, 2, Y1, goq.BF16, False),
                 (d_half, pk, Y0, 2, Y2, goq.BF16, False)])
    assert got == [(N, -1), (D, 0), (Bar, -1)]
