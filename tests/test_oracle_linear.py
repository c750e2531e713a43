"""Pins for the oracle's reference linear layers (float and integer)."""
import numpy as np
import pytest

import synth_inputs as si
from oracle import goq_oracle as O


def _small(n=12, k=128, g=64, b=3, seed=0):
    w = si.gaussian_weights(n, k, seed=seed)
    return O.quantize_geo(w, g, b)


@pytest.mark.parametrize("b,g", [(3, 64), (4, 64), (2, 32)])
def test_linear_f64_equals_library_matmul_on_reconstructed_weights(b, g):
    codes, meta, coef = _small(b=b, g=g, seed=1)
    x = si.bf16_bits_to_f64(si.bf16_activations(5, 128, seed=2))
    y = O.linear_f64(codes, meta, coef, x, g, b)
    y_lib = x @ O.reconstruct(codes, meta, coef, g, b).T
    assert np.max(np.abs(y - y_lib)) <= 1e-13 * np.max(np.abs(y_lib))


def test_linear_f64_equals_scalar_loops():
    codes, meta, coef = _small(n=6, k=128, g=64, seed=3)
    x = si.bf16_bits_to_f64(si.bf16_activations(2, 128, seed=4))
    y = O.linear_f64(codes, meta, coef, x, 64, 3)
    y_loop = O.linear_f64_loops(codes, meta, coef, x, 64, 3)
    assert np.max(np.abs(y - y_loop)) <= 1e-13 * np.max(np.abs(y_loop))


def test_linear_f64_hand_example():
    """One row, one group of 8: values worked out by hand from the definitions."""
    # codes (b=3): +1, +.5, 0, -.25, -1, -.125, +.25, +.5
    codes = np.array([[0, 1, 3, 6, 4, 7, 2, 1]], dtype=np.uint8)
    # record: s = 3 -> pairs (0,3),(1,2),(4,7),(5,6); eta = (+1, -1, -1, +1)
    meta = np.array([[2 | (0b0110 << 2)]], dtype=np.uint8)
    coef = np.array([[[0.5, 0.25]]], dtype=np.float16)
    b1 = [1, .5, 0, -.25, -1, -.125, .25, .5]
    # y0=-x3, y3=x0 ; y1=+x2, y2=-x1 ; y4=+x7, y7=-x4 ; y5=-x6, y6=x5
    b2 = [.25, 0, -.5, 1, .5, -.25, -.125, 1]
    assert O.decode_b1(codes, 3)[0].tolist() == b1
    assert O.decode_b2(codes, meta, 3)[0].tolist() == b2
    x = np.array([[1.0, 2.0, -3.0, 4.0, 0.5, -8.0, 16.0, -2.0]])
    s1 = 1 + 1 + 0 - 1 - .5 + 1 + 4 - 1       # = 4.5
    s2 = .25 + 0 + 1.5 + 4 + .25 + 2 - 2 - 2   # = 4.0
    y = O.linear_f64(codes, meta, coef, x, 8, 3)
    assert y[0, 0] == 0.5 * s1 + 0.25 * s2


def test_row_subset_matches_full():
    codes, meta, coef = _small(n=20, k=256, g=128, seed=5)
    x = si.bf16_bits_to_f64(si.bf16_activations(3, 256, seed=6))
    rows = si.sample_rows(20, 5, seed=1)
    full = O.linear_f64(codes, meta, coef, x, 128, 3)
    assert np.array_equal(O.linear_f64(codes, meta, coef, x, 128, 3, rows=rows), full[:, rows])


def test_single_basis_special_case_is_pot_rtn_with_least_squares_scale():
    """With c2 forced to 0 the layer is the classic one-basis PoT layer: y = sum_j c1_j <b1_j, x_j>."""
    w = si.gaussian_weights(4, 128, seed=7)
    codes, meta, coef, aux = O.quantize_geo(w, 64, 3, return_aux=True)
    coef1 = coef.copy()
    coef1[..., 1] = 0
    x = si.bf16_bits_to_f64(si.bf16_activations(2, 128, seed=8))
    y = O.linear_f64(codes, meta, coef1, x, 64, 3)
    b1 = O.decode_b1(codes, 3)
    ref = sum((x[:, j * 64:(j + 1) * 64] @ b1[:, j * 64:(j + 1) * 64].T) * coef1[:, j, 0].astype(np.float64)
              for j in range(2))
    assert np.allclose(y, ref, rtol=1e-14, atol=0)
    # and c1 is the least-squares scale of the rounded block
    wg = w.reshape(4, 2, 64).astype(np.float64)
    b1g = b1.reshape(4, 2, 64)
    assert np.allclose(aux["c"][..., 0], np.sum(wg * b1g, -1) / np.sum(b1g * b1g, -1), rtol=1e-14)


# ---------------------------------------------------------------- integer path
def test_int8_quantizers():
    x = si.f32_activations(7, 64, seed=9)
    xq, sx = O.quantize_activations_int8(x)
    assert xq.dtype == np.int8 and np.abs(xq.astype(int)).max() == 127
    assert np.all(np.abs(xq.astype(np.float64) * sx[:, None] - x) <= 0.5 * sx[:, None] * (1 + 1e-6))
    _, _, coef = _small(seed=10)
    cq, sc = O.quantize_coefficients_int8(coef)
    assert cq.shape == coef.shape and sc.shape == (coef.shape[0], 2)
    c = coef.astype(np.float64)
    assert np.all(np.abs(cq.astype(np.float64) * sc[:, None, :] - c) <= 0.5 * sc[:, None, :] * (1 + 1e-6))


@pytest.mark.parametrize("b,g", [(3, 64), (4, 32)])
def test_linear_i32_equals_python_integer_shift_add(b, g):
    codes, meta, coef = _small(n=5, k=128, g=g, b=b, seed=11)
    cq, sc = O.quantize_coefficients_int8(coef)
    xq, sx = O.quantize_activations_int8(si.f32_activations(3, 128, seed=12))
    acc1, acc2, y, s1, s2 = O.linear_i32(codes, meta, cq, sc, xq, sx, g, b, return_groups=True)
    l1, l2 = O.linear_i32_loops(codes, meta, cq, xq, g, b)
    assert np.array_equal(acc1, l1) and np.array_equal(acc2, l2)
    # int64 matmul of the integer operands gives the same group sums
    b1i, b2i = O.int_weights(codes, meta, b)
    for j in range(128 // g):
        sl = slice(j * g, (j + 1) * g)
        assert np.array_equal(s1[j], xq[:, sl].astype(np.int64) @ b1i[:, sl].T)
        assert np.array_equal(s2[j], xq[:, sl].astype(np.int64) @ b2i[:, sl].T)
    # the dequantised output approximates the float layer on the dequantised operands
    xdq = xq.astype(np.float64) * sx[:, None].astype(np.float64)
    c_dq = (cq.astype(np.float64) * sc[:, None, :].astype(np.float64)).astype(np.float64)
    b1, b2 = O.decode_b1(codes, b), O.decode_b2(codes, meta, b)
    ref = np.zeros_like(y)
    for j in range(128 // g):
        sl = slice(j * g, (j + 1) * g)
        ref += (xdq[:, sl] @ b1[:, sl].T) * c_dq[None, :, j, 0] + (xdq[:, sl] @ b2[:, sl].T) * c_dq[None, :, j, 1]
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-18)


def test_integer_operands_are_shifts():
    codes = np.arange(8, dtype=np.uint8)[None, :]
    meta = np.zeros((1, 1), dtype=np.uint8)
    b1i, _ = O.int_weights(codes, meta, 3)
    assert b1i[0].tolist() == [8, 4, 2, 0, -8, -4, -2, -1]


def test_linear_i32_overflow_is_detected():
    codes = np.zeros((1, 64 * 400), dtype=np.uint8)           # all +1 -> operand 8
    meta = np.zeros((1, 8 * 400), dtype=np.uint8)
    cq = np.full((1, 400, 2), 127, dtype=np.int8)
    sc = np.ones((1, 2), dtype=np.float32)
    xq = np.full((1, 64 * 400), 127, dtype=np.int8)
    with pytest.raises(OverflowError):
        O.linear_i32(codes, meta, cq, sc, xq, np.ones(1, np.float32), 64, 3)


def test_normwise_error_measure():
    ref = np.array([[3.0, 4.0], [0.0, 1.0]])
    y = np.array([[3.0, 4.5], [0.0, 1.0]])
    assert O.normwise_rel_err(y, ref) == pytest.approx(0.1)


def test_bf16_helpers_roundtrip():
    bits = si.bf16_activations(4, 32, seed=13)
    x = si.bf16_bits_to_f64(bits)
    assert np.array_equal(si.f32_to_bf16_bits(x.astype(np.float32)), bits)
    import torch
    t = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)
    assert np.array_equal(t.view(torch.int16).numpy().view(np.uint16), bits)
    y = np.array([1.00390625, 1.01171875], dtype=np.float32)    # ties: round to even
    assert si.f32_to_bf16_bits(y).tolist() == [0x3F80, 0x3F82]


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_narrow_activation_integers_in_byte_containers(bits):
    """b_a-bit activations (Section 3.5): the 8-bit case is the int8 quantizer; every width reaches +-q_max, stays inside
    it, and is off by at most half a step (the grid is uniform, so round-to-nearest means |x - s q| <= s / 2)."""
    x = si.f32_activations(9, 300, seed=bits)
    x[3] = 0.0
    xq, sx = O.quantize_activations_int(x, bits)
    qmax = (1 << (bits - 1)) - 1
    if bits == 8:
        xq8, sx8 = O.quantize_activations_int8(x)
        assert np.array_equal(xq, xq8) and np.array_equal(sx, sx8)
    assert xq.dtype == np.int8 and np.abs(xq.astype(int)).max() == qmax and not xq[3].any() and sx[3] == 1.0
    s64 = np.where(np.max(np.abs(x), 1) == 0, 1.0, np.max(np.abs(x), 1) / qmax)
    assert np.all(np.abs(x - s64[:, None] * xq) <= 0.5 * s64[:, None] * (1 + 1e-12))
