"""Helpers for the GPU parity tests: move oracle-side numpy arrays to the device and call the C ABI."""
import numpy as np
import torch

from paper_2605_26092_b200 import goq


def elementwise_rel_err(y: np.ndarray, y_ref: np.ndarray) -> float:
    """max |y - y_ref| / max |y_ref| over all outputs: one wrong output among thousands shows here, not in a norm."""
    return float(np.max(np.abs(y - y_ref)) / np.max(np.abs(y_ref)))


def check_parity(y, y_ref, norm_tol, elem_tol, what=""):
    """Both acceptance metrics of an A16 comparison: per-token 2-norm ratio (max over tokens) and the largest
    element-wise deviation relative to the largest reference magnitude."""
    y = np.asarray(y, dtype=np.float64)
    num = np.linalg.norm(y - y_ref, axis=-1)
    den = np.linalg.norm(y_ref, axis=-1)
    nerr = float(np.max(num / np.where(den > 0, den, 1.0)))
    eerr = elementwise_rel_err(y, y_ref)
    assert nerr <= norm_tol, "%s normwise %.3e > %.1e" % (what, nerr, norm_tol)
    assert eerr <= elem_tol, "%s element-wise %.3e > %.1e" % (what, eerr, elem_tol)
    return nerr, eerr


def check_bf16_output(y16, y_ref, elem_tol, what=""):
    """A bf16 output is the kernel's fp32 result rounded once. bf16 keeps 8 significant bits: the rounding moves an
    element by at most half a unit in the last place, 2^-8 of its magnitude (2^-9 only at the top of a binade), which
    alone is ~1.5e-3 in the 2-norm for outputs spread over their binades and up to 2^-8 = 3.9e-3 in the worst case.
    So the check is per element: within 2^-8 |y_ref| of the fp64 reference, plus the bound the fp32 output is held to
    (elem_tol of the largest reference magnitude). Returns the normwise error for the record."""
    y16 = np.asarray(y16, dtype=np.float64)
    slack = 2.0 ** -8 * np.abs(y_ref) + elem_tol * np.max(np.abs(y_ref))
    worst = float(np.max(np.abs(y16 - y_ref) / slack))
    assert worst <= 1.0, "%s bf16 output off by %.3f of the rounding bound" % (what, worst)
    den = np.linalg.norm(y_ref, axis=-1)
    return float(np.max(np.linalg.norm(y16 - y_ref, axis=-1) / np.where(den > 0, den, 1.0)))


def dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    if a.dtype == np.float16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


def pack_weights(n, k, g, b, codes, meta, coef):
    d = goq.desc(n, k, g, b)
    nbytes = goq.packed_bytes(d)
    assert nbytes > 0
    packed = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    goq.pack(d, dev(codes), dev(meta), dev(coef), packed)
    torch.cuda.synchronize()
    return d, packed


def run_gemv(d, packed, x_bits: np.ndarray, y_dtype=goq.F32, variant=0):
    batch = x_bits.shape[0]
    x = dev(x_bits)
    y = torch.empty((batch, d.n_out), dtype=torch.float32 if y_dtype == goq.F32 else torch.bfloat16, device="cuda")
    ws = goq.new_workspace(d, goq.OP_GEMV, batch)
    prev = goq.set_gemv_variant(variant)
    try:
        goq.gemv(d, packed, x, batch, y, y_dtype, ws=ws)
    finally:
        goq.set_gemv_variant(prev)
    torch.cuda.synchronize()
    if ws is not None:
        assert goq.workspace_status(ws) == goq.OK
    return y.float().cpu().numpy().astype(np.float64)


def run_gemm_bf16(d, packed, x_bits: np.ndarray, y_dtype=goq.F32, variant=0):
    m = x_bits.shape[0]
    x = dev(x_bits)
    y = torch.empty((m, d.n_out), dtype=torch.float32 if y_dtype == goq.F32 else torch.bfloat16, device="cuda")
    ws = goq.new_workspace(d, goq.OP_GEMM, m)
    prev = goq.set_gemv_variant(variant)
    try:
        goq.gemm(d, packed, x, m, goq.BF16, y=y, y_dtype=y_dtype, ws=ws)
    finally:
        goq.set_gemv_variant(prev)
    torch.cuda.synchronize()
    if ws is not None:
        assert goq.workspace_status(ws) == goq.OK
    return y.float().cpu().numpy().astype(np.float64)


def run_gemm_i8(d, packed, xq, sx, cq, sc, want_y=True):
    m = xq.shape[0]
    acc = torch.empty((2, m, d.n_out), dtype=torch.int32, device="cuda")
    y = torch.empty((m, d.n_out), dtype=torch.float32, device="cuda") if want_y else None
    goq.gemm(d, packed, dev(xq), m, goq.I8, y=y, y_dtype=goq.F32, sx=dev(sx), cq=dev(cq), sc=dev(sc), acc=acc)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), (None if y is None else y.cpu().numpy().astype(np.float64))
