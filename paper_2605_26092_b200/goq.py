"""ctypes binding of libgoq.so with the same names as include/goq.h.

Arguments are torch CUDA tensors (device memory) or plain integers; the functions pass
`tensor.data_ptr()` and the current CUDA stream to the C ABI and raise GoqError on a non-zero
status. No arithmetic of the method happens here.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_int, c_int32, c_size_t, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgoq.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_OVERFLOW_BOUND, ERR_ARCH, ERR_CUDA, \
    ERR_TIMEOUT = range(9)
BF16, F32, I8 = 0, 1, 2
OP_GEMV, OP_GEMM = 0, 1
LAYOUT_TILE16 = 1
LAYOUT_TILE16_K1 = 2

EXPORTS = (
    "goq_status_string", "goq_packed_bytes", "goq_algorithmic_bytes", "goq_workspace_bytes", "goq_pack",
    "goq_unpack", "goq_gemv", "goq_gemm", "goq_gemv_host", "goq_set_gemv_variant", "goq_sequence_order", "goq_workspace_init",
    "goq_workspace_status", "goq_gemv_static", "goq_last_cuda_error", "goq_sequence_workspace_bytes",
    "goq_gemv_sequence", "goq_gemv_sequence_host", "goq_set_wait_limit", "goq_gemv_static_status", "goq_quantize_activations", "goq_gemm_i8_requant",
    "goq_quantize_geo", "goq_solve_ref",
)


class GoqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        extra = f", cudaError {lib().goq_last_cuda_error()}" if status == ERR_CUDA else ""
        super().__init__(f"{where}: status {status} ({status_string(status)}{extra})")


class Desc(Structure):
    _fields_ = [("n_out", c_int32), ("k_in", c_int32), ("group", c_int32), ("wbits", c_int32), ("layout", c_int32)]


class GemvItem(Structure):
    _fields_ = [("desc", Desc), ("packed", c_void_p), ("x_bf16", c_void_p), ("y", c_void_p), ("batch", c_int32),
                ("y_dtype", c_int32), ("depends", c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libgoq.so (built in-tree by build.py). Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} not found: run `python -m paper_2605_26092_b200.build` first")
        L = ctypes.CDLL(_LIB_PATH)
        L.goq_status_string.restype = c_char_p
        L.goq_status_string.argtypes = [c_int]
        for name in ("goq_packed_bytes", "goq_algorithmic_bytes"):
            getattr(L, name).restype = c_size_t
            getattr(L, name).argtypes = [POINTER(Desc)]
        L.goq_workspace_bytes.restype = c_size_t
        L.goq_workspace_bytes.argtypes = [POINTER(Desc), c_int, c_int]
        L.goq_pack.restype = c_int
        L.goq_pack.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.goq_unpack.restype = c_int
        L.goq_unpack.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.goq_gemv.restype = c_int
        L.goq_gemv.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p, c_size_t, c_void_p]
        L.goq_gemm.restype = c_int
        L.goq_gemm.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p,
                               c_void_p, c_int, c_void_p, c_void_p, c_size_t, c_void_p]
        L.goq_gemv_host.restype = c_int
        L.goq_gemv_host.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p,
                                    c_void_p, c_size_t, c_void_p]
        L.goq_workspace_init.restype = c_int
        L.goq_workspace_init.argtypes = [c_void_p, c_size_t, c_void_p]
        L.goq_workspace_status.restype = c_int
        L.goq_workspace_status.argtypes = [c_void_p, c_void_p, POINTER(c_int)]
        L.goq_gemv_static.restype = c_int
        L.goq_gemv_static.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p]
        L.goq_quantize_activations.restype = c_int
        L.goq_quantize_activations.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
        L.goq_gemm_i8_requant.restype = c_int
        L.goq_gemm_i8_requant.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p,
                                          c_void_p, c_void_p, c_void_p, c_void_p]
        L.goq_quantize_geo.restype = c_int
        L.goq_quantize_geo.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.goq_solve_ref.restype = c_int
        L.goq_solve_ref.argtypes = [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_int, ctypes.c_double, c_void_p,
                                    c_void_p, c_void_p]
        L.goq_gemv_static_status.restype = c_int
        L.goq_gemv_static_status.argtypes = [c_void_p, POINTER(c_int)]
        L.goq_last_cuda_error.restype = c_int
        L.goq_last_cuda_error.argtypes = []
        L.goq_sequence_workspace_bytes.restype = ctypes.c_size_t
        L.goq_sequence_workspace_bytes.argtypes = [c_int]
        L.goq_gemv_sequence.restype = c_int
        L.goq_gemv_sequence.argtypes = [POINTER(GemvItem), c_int, c_void_p, ctypes.c_size_t, c_void_p]
        L.goq_sequence_order.restype = c_int
        L.goq_sequence_order.argtypes = [POINTER(GemvItem), c_int, POINTER(c_int32), POINTER(c_int32)]
        L.goq_gemv_sequence_host.restype = c_int
        L.goq_gemv_sequence_host.argtypes = [POINTER(GemvItem), c_int, c_void_p, c_void_p, ctypes.c_size_t, c_void_p,
                                             c_void_p, ctypes.c_size_t, c_void_p, ctypes.c_size_t, c_void_p]
        L.goq_set_gemv_variant.restype = c_int
        L.goq_set_gemv_variant.argtypes = [c_int]
        L.goq_set_wait_limit.restype = c_int
        L.goq_set_wait_limit.argtypes = [c_int]
        _lib = L
    return _lib


def desc(n_out: int, k_in: int, group: int, wbits: int, layout: int = LAYOUT_TILE16) -> Desc:
    return Desc(n_out, k_in, group, wbits, layout)


def status_string(status: int) -> str:
    return lib().goq_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr() if hasattr(t, "data_ptr") else int(t))


def _stream(stream=None):
    if stream is not None:
        return c_void_p(int(stream))
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != OK:
        raise GoqError(status, where)


def packed_bytes(d: Desc) -> int:
    return lib().goq_packed_bytes(ctypes.byref(d))


def algorithmic_bytes(d: Desc) -> int:
    return lib().goq_algorithmic_bytes(ctypes.byref(d))


def workspace_bytes(d: Desc, op: int, m: int) -> int:
    return lib().goq_workspace_bytes(ctypes.byref(d), op, m)


def workspace_init(ws, stream=None):
    _check(lib().goq_workspace_init(_ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "goq_workspace_init")


def workspace_status(ws, stream=None) -> int:
    out = c_int(0)
    _check(lib().goq_workspace_status(_ptr(ws), _stream(stream), ctypes.byref(out)), "goq_workspace_status")
    return out.value


def new_workspace(d: Desc, op: int, m: int):
    """Allocate (torch) and initialise a scratch buffer large enough for the call; None if none is needed."""
    import torch
    n = workspace_bytes(d, op, m)
    if n == 0:
        return None
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    workspace_init(ws)
    return ws


def set_gemv_variant(variant: int) -> int:
    return lib().goq_set_gemv_variant(variant)


def set_wait_limit(polls: int) -> int:
    """goq_set_wait_limit: bound of the device-side waits of goq_gemv_sequence (tests only; 0 = the kernel's own)."""
    return lib().goq_set_wait_limit(polls)


def pack(d: Desc, codes, meta, coef_f16, packed, stream=None):
    _check(lib().goq_pack(ctypes.byref(d), _ptr(codes), _ptr(meta), _ptr(coef_f16), _ptr(packed),
                          packed.numel() * packed.element_size(), _stream(stream)), "goq_pack")


def unpack(d: Desc, packed, codes_b1=None, codes_b2=None, coef_f16=None, stream=None):
    _check(lib().goq_unpack(ctypes.byref(d), _ptr(packed), _ptr(codes_b1), _ptr(codes_b2), _ptr(coef_f16),
                            _stream(stream)), "goq_unpack")


def gemv(d: Desc, packed, x_bf16, batch: int, y, y_dtype: int, ws=None, stream=None):
    wsb = 0 if ws is None else ws.numel() * ws.element_size()
    _check(lib().goq_gemv(ctypes.byref(d), _ptr(packed), _ptr(x_bf16), batch, _ptr(y), y_dtype, _ptr(ws), wsb,
                          _stream(stream)), "goq_gemv")


def gemv_static(d: Desc, packed, x_bf16, batch: int, y, y_dtype: int, stream=None):
    """goq_gemv_static: the decode GEMV with the library's built-in scratch array (no scratch argument).
    For callers that cannot allocate device memory; calls that may overlap on the GPU must not share it."""
    _check(lib().goq_gemv_static(ctypes.byref(d), _ptr(packed), _ptr(x_bf16), batch, _ptr(y), y_dtype,
                                 _stream(stream)), "goq_gemv_static")


def quantize_activations(x, x_dtype: int, m: int, k: int, xq, sx, amax=None, abits: int = 8, stream=None):
    _check(lib().goq_quantize_activations(_ptr(x), x_dtype, m, k, abits, _ptr(amax), _ptr(xq), _ptr(sx), _stream(stream)),
           "goq_quantize_activations")


def gemm_i8_requant(d: Desc, packed, x, m: int, sx, cq, sc, y, amax, yq=None, sy=None, stream=None):
    _check(lib().goq_gemm_i8_requant(ctypes.byref(d), _ptr(packed), _ptr(x), m, _ptr(sx), _ptr(cq), _ptr(sc), _ptr(y),
                                     _ptr(amax), _ptr(yq), _ptr(sy), _stream(stream)), "goq_gemm_i8_requant")


def quantize_geo(d: Desc, w, codes, meta, coef_f16, stream=None):
    _check(lib().goq_quantize_geo(ctypes.byref(d), _ptr(w), _ptr(codes), _ptr(meta), _ptr(coef_f16), _stream(stream)),
           "goq_quantize_geo")


def solve_ref(d: Desc, w, codes, meta, x_calib, m: int, lam: float, coef_f16, c_f64=None, stream=None):
    _check(lib().goq_solve_ref(ctypes.byref(d), _ptr(w), _ptr(codes), _ptr(meta), _ptr(x_calib), m, float(lam),
                               _ptr(coef_f16), _ptr(c_f64), _stream(stream)), "goq_solve_ref")


def gemv_static_status(stream=None) -> int:
    """goq_gemv_static_status: status word of the library's built-in scratch array (synchronises the stream)."""
    out = c_int(0)
    _check(lib().goq_gemv_static_status(_stream(stream), ctypes.byref(out)), "goq_gemv_static_status")
    return out.value


def sequence_workspace_bytes(n_items: int) -> int:
    return lib().goq_sequence_workspace_bytes(n_items)


def make_sequence(items):
    """items: iterable of (desc, packed, x_bf16, batch, y, y_dtype, depends). Returns the ctypes array
    goq_gemv_sequence takes (it holds raw device pointers: keep the tensors alive)."""
    items = list(items)
    arr = (GemvItem * len(items))()
    for a, (d, packed, x, batch, y, y_dtype, depends) in zip(arr, items):
        a.desc = d
        a.packed, a.x_bf16, a.y = _ptr(packed), _ptr(x), _ptr(y)
        a.batch, a.y_dtype, a.depends = batch, y_dtype, 1 if depends else 0
    return arr


ORDER_NONE, ORDER_DATA, ORDER_BARRIER = 0, 1, 2


def sequence_order(seq):
    """goq_sequence_order: (kinds, sources) - how goq_gemv_sequence will order each item of `seq` (host only)."""
    n = len(seq)
    kinds, sources = (c_int32 * n)(), (c_int32 * n)()
    _check(lib().goq_sequence_order(seq, n, kinds, sources), "goq_sequence_order")
    return list(kinds), list(sources)


def gemv_sequence(seq, ws, stream=None):
    """goq_gemv_sequence: a chain of decode GEMVs in one persistent kernel. `seq` comes from make_sequence."""
    _check(lib().goq_gemv_sequence(seq, len(seq), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "goq_gemv_sequence")


def gemv_sequence_host(seq, x_host, x_stage, y_host, y_stage, ws, stream=None):
    """goq_gemv_sequence_host: one copy of the activation block in, the sequence kernel, one copy of the output
    block out. x_host / y_host are (pinned) host tensors, x_stage / y_stage the device blocks the items point into."""
    xb, yb = x_stage.numel() * x_stage.element_size(), y_stage.numel() * y_stage.element_size()
    _check(lib().goq_gemv_sequence_host(seq, len(seq), _ptr(x_host), _ptr(x_stage), xb, _ptr(y_host), _ptr(y_stage), yb,
                                        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "goq_gemv_sequence_host")


def gemm(d: Desc, packed, x, m: int, x_dtype: int, y=None, y_dtype: int = F32, sx=None, cq=None, sc=None,
         acc=None, ws=None, stream=None):
    wsb = 0 if ws is None else ws.numel() * ws.element_size()
    _check(lib().goq_gemm(ctypes.byref(d), _ptr(packed), _ptr(x), m, x_dtype, _ptr(sx), _ptr(cq), _ptr(sc),
                          _ptr(y), y_dtype, _ptr(acc), _ptr(ws), wsb, _stream(stream)), "goq_gemm")


def gemv_host(d: Desc, packed, x_host, batch: int, y_host, y_dtype: int, x_stage, y_stage, ws=None, stream=None):
    wsb = 0 if ws is None else ws.numel() * ws.element_size()
    _check(lib().goq_gemv_host(ctypes.byref(d), _ptr(packed), _ptr(x_host), batch, _ptr(y_host), y_dtype,
                               _ptr(x_stage), _ptr(y_stage), _ptr(ws), wsb, _stream(stream)), "goq_gemv_host")
