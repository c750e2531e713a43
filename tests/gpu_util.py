"""Helpers for the GPU parity tests: move oracle-side numpy arrays to the device and call the C ABI."""
import numpy as np
import torch

from paper_2605_26092_b200 import goq


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
