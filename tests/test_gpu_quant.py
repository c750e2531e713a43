"""GPU parity of the steps either side of the inner product: the single-basis (K = 1) form, the activation quantizer
and requantising epilogue (Section 3.5), the GEO quantizer (Sections 3.2-3.4) and the REF-mode solve (Eq. 3),
each called through the C ABI and held to the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import goq_oracle as O

pytestmark = pytest.mark.gpu
TIGHT = 2e-5


@pytest.fixture(scope="module")
def goq():
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq as g
    g.lib()
    assert torch.cuda.is_available()
    return g


def _pack(goq, n, k, g, b, codes, meta, coef, layout):
    from tests.gpu_util import dev
    d = goq.desc(n, k, g, b, layout)
    packed = torch.zeros(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
    goq.pack(d, dev(codes), dev(meta), dev(coef), packed)
    torch.cuda.synchronize()
    return d, packed


# --------------------------------------------------------------------------------------------- K = 1
@pytest.mark.parametrize("n,k,g,b", [(300, 1152, 128, 3), (64, 512, 32, 2), (1000, 4224, 64, 3)])
def test_single_basis_layout_evaluates_c1_b1_on_every_path(goq, n, k, g, b):
    """w_hat = c1 b1 (Section 3.1). The K = 1 layout is fed (a) the oracle's K = 1 quantization and (b) a dual-basis
    quantization, whose records and c2 goq_pack must then drop: both evaluate c1 b1. Decode GEMV at batch 1 and 3 (the
    chain kernel skips the second operand), batch 9 (streaming kernel) and the GEMM at 70 tokens."""
    from tests.gpu_util import run_gemv, run_gemm_bf16, check_parity
    w = si.weights_with_outlier_channels(n, k, seed=n + b)
    c1, m1, f1 = O.quantize_k1(w, g, b)
    c2, m2, f2 = O.quantize_geo(w, g, b)
    assert np.array_equal(c1, c2) and m2.any() and f2[..., 1].any()
    assert goq.algorithmic_bytes(goq.desc(n, k, g, b, goq.LAYOUT_TILE16_K1)) == n * k * b // 8 + n * (k // g) * 2
    for codes, meta, coef in ((c1, m1, f1), (c2, m2, f2)):
        d, packed = _pack(goq, n, k, g, b, codes, meta, coef, goq.LAYOUT_TILE16_K1)
        for batch in (1, 3, 9):
            xb = si.bf16_activations(batch, k, seed=batch)
            y_ref = O.linear_f64(c1, m1, f1, si.bf16_bits_to_f64(xb), g, b)
            check_parity(run_gemv(d, packed, xb, goq.F32), y_ref, TIGHT, 1e-4, "K=1 gemv batch %d" % batch)
        xb = si.bf16_activations(70, k, seed=7)
        y_ref = O.linear_f64(c1, m1, f1, si.bf16_bits_to_f64(xb), g, b)
        check_parity(run_gemm_bf16(d, packed, xb), y_ref, 5e-4, 2e-3, "K=1 gemm")


# --------------------------------------------------------------------------------------------- activation quantizer
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_activation_quantizer_bit_equal_to_oracle(goq, dtype):
    """Per-token symmetric int8 (Section 3.5): integers and scales equal to the oracle's bit for bit, with and without the
    largest magnitudes handed in; an all-zero token, one of tiny and one of huge magnitude, and exact half-way cases."""
    m, k = 37, 1000
    x = si.f32_activations(m, k, seed=3).astype(np.float32)
    x[4] = 0.0
    x[5] *= np.float32(2.0 ** -100)
    x[6] *= np.float32(2.0 ** 100)
    x[7, :] = np.float32(127.0)
    x[7, ::2] = np.float32(0.5)      # x / s_x lands exactly on .5: round half to even
    x[7, 1::4] = np.float32(-2.5)
    if dtype == "bf16":
        bits = si.f32_to_bf16_bits(x)
        x = si.bf16_bits_to_f64(bits).astype(np.float32)
        xd = torch.from_numpy(bits.view(np.int16)).cuda()
        code = goq.BF16
    else:
        xd = torch.from_numpy(x).cuda()
        code = goq.F32
    xq_ref, sx_ref = O.quantize_activations_int8(x)
    for given in (False, True):
        xq = torch.full((m, k), 99, dtype=torch.int8, device="cuda")
        sx = torch.zeros(m, dtype=torch.float32, device="cuda")
        amax = torch.from_numpy(np.max(np.abs(x), axis=1).astype(np.float32)).cuda() if given else None
        goq.quantize_activations(xd, code, m, k, xq, sx, amax=amax)
        torch.cuda.synchronize()
        assert np.array_equal(xq.cpu().numpy(), xq_ref)
        assert np.array_equal(sx.cpu().numpy(), sx_ref)


@pytest.mark.parametrize("abits,b,g,k", [(4, 3, 64, 768), (6, 3, 128, 1024), (8, 4, 64, 768), (4, 4, 32, 512), (8, 4, 16, 256)])
def test_narrow_activations_and_w4_on_the_integer_path(goq, abits, b, g, k):
    """A4 / A6 activations in int8 containers (quantised on the device, bit-equal to the oracle) through the integer
    layer, and W4 weights (2^emax = 128 split over two signed bytes): ACC_1, ACC_2 bit-exact against the oracle."""
    from tests.gpu_util import pack_weights, run_gemm_i8
    n, m = 72, 150
    codes, meta, coef = O.quantize_geo(si.weights_with_outlier_channels(n, k, seed=abits + b), g, b)
    cq, sc = O.quantize_coefficients_int8(coef)
    x = si.f32_activations(m, k, seed=abits).astype(np.float32)
    xq_ref, sx_ref = O.quantize_activations_int(x, abits)
    xq = torch.empty((m, k), dtype=torch.int8, device="cuda")
    sx = torch.empty((m,), dtype=torch.float32, device="cuda")
    goq.quantize_activations(torch.from_numpy(x).cuda(), goq.F32, m, k, xq, sx, abits=abits)
    torch.cuda.synchronize()
    assert np.array_equal(xq.cpu().numpy(), xq_ref) and np.array_equal(sx.cpu().numpy(), sx_ref)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    acc, y = run_gemm_i8(d, packed, xq_ref, sx_ref, cq, sc)
    a1, a2, y_ref = O.linear_i32(codes, meta, cq, sc, xq_ref, sx_ref, g, b)
    assert np.array_equal(acc[0], a1) and np.array_equal(acc[1], a2)
    assert O.normwise_rel_err(y, y_ref) <= TIGHT


def test_integer_layer_with_requantising_epilogue(goq):
    """goq_gemm_i8_requant: y equals goq_gemm's y bit for bit, the recorded per-token maxima equal max |y| exactly, and
    the requantised output equals the oracle's quantizer applied to the y actually produced (Section 3.5)."""
    from tests.gpu_util import dev, pack_weights
    n, k, g, b, m = 200, 768, 64, 3, 333
    codes, meta, coef = O.quantize_geo(si.gaussian_weights(n, k, seed=8), g, b)
    cq, sc = O.quantize_coefficients_int8(coef)
    xq, sx = O.quantize_activations_int8(si.f32_activations(m, k, seed=9))
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    args = (dev(xq), m, dev(sx), dev(cq), dev(sc))
    y0 = torch.empty((m, n), dtype=torch.float32, device="cuda")
    goq.gemm(d, packed, args[0], m, goq.I8, y=y0, y_dtype=goq.F32, sx=args[2], cq=args[3], sc=args[4])
    y = torch.empty((m, n), dtype=torch.float32, device="cuda")
    amax = torch.full((m,), 7.0, dtype=torch.float32, device="cuda")
    yq = torch.empty((m, n), dtype=torch.int8, device="cuda")
    sy = torch.empty((m,), dtype=torch.float32, device="cuda")
    goq.gemm_i8_requant(d, packed, args[0], m, args[2], args[3], args[4], y, amax, yq, sy)
    torch.cuda.synchronize()
    assert torch.equal(y, y0)
    yh = y.cpu().numpy()
    assert np.array_equal(amax.cpu().numpy(), np.max(np.abs(yh), axis=1))
    yq_ref, sy_ref = O.quantize_activations_int8(yh)
    assert np.array_equal(yq.cpu().numpy(), yq_ref) and np.array_equal(sy.cpu().numpy(), sy_ref)
    # and y itself against the exact integer evaluation
    _, _, y_ref = O.linear_i32(codes, meta, cq, sc, xq, sx, g, b)
    assert O.normwise_rel_err(yh.astype(np.float64), y_ref) <= TIGHT


# --------------------------------------------------------------------------------------------- GEO quantizer
def _objective(w, codes, meta, g, b):
    """Reconstruction error per macro-block with least-squares coefficients for the given discrete choice, and the
    alignment <r, b2> per micro-block (Section 3.3's objective)."""
    n, k = w.shape
    wg = w.reshape(n, k // g, g)
    b1 = O.decode_b1(codes, b).reshape(n, k // g, g)
    b2 = O.decode_b2(codes, meta, b).reshape(n, k // g, g)
    nb1, nb2 = np.sum(b1 * b1, -1), np.sum(b2 * b2, -1)
    c1 = np.where(nb1 > 0, np.sum(wg * b1, -1) / np.where(nb1 > 0, nb1, 1), 0.0)
    c2 = np.where(nb2 > 0, np.sum(wg * b2, -1) / np.where(nb2 > 0, nb2, 1), 0.0)
    r = wg - c1[..., None] * b1
    align = np.sum((r * b2).reshape(n, k // 8, 8), -1)
    err = np.sum((r - c2[..., None] * b2) ** 2, -1)
    return err, align, np.stack([c1, c2], -1)


@pytest.mark.parametrize("n,k,g,b", [(64, 1024, 128, 3), (33, 256, 64, 2), (40, 384, 128, 4), (16, 128, 8, 3), (20, 192, 32, 3)])
def test_geo_quantizer_matches_oracle_objective(goq, n, k, g, b):
    """goq_quantize_geo against oracle.quantize_geo. Primary codes: equal (same float64 arithmetic). Records: several
    encodings can be equally good (a zero sign argument, equal pattern scores) and sums are added in another order, so
    the comparison is on what is unique - the alignment reached per micro-block and the reconstruction error per
    macro-block - never on raw record bits; the fp16 coefficients must be those of the device's own discrete choice."""
    w = si.weights_with_outlier_channels(n, k, seed=n + k + b).astype(np.float32)
    w[3, :g] = 0.0                                   # an all-zero macro-block
    w[5, g:2 * g] = np.float32(0.25)                 # constant block: every pattern ties
    codes_o, meta_o, coef_o = O.quantize_geo(w, g, b)
    d = goq.desc(n, k, g, b)
    codes = torch.full((n, k), 0xEE, dtype=torch.uint8, device="cuda")
    meta = torch.full((n, k // 8), 0xEE, dtype=torch.uint8, device="cuda")
    coef = torch.zeros((n, k // g, 2), dtype=torch.int16, device="cuda")
    goq.quantize_geo(d, torch.from_numpy(w).cuda(), codes, meta, coef)
    torch.cuda.synchronize()
    codes_g, meta_g = codes.cpu().numpy(), meta.cpu().numpy()
    coef_g = coef.cpu().numpy().view(np.float16)
    assert np.array_equal(codes_g, codes_o)
    assert meta_g.max() < 64
    w64 = w.astype(np.float64)
    err_o, al_o, _ = _objective(w64, codes_o, meta_o, g, b)
    err_g, al_g, c_g = _objective(w64, codes_g, meta_g, g, b)
    scale = np.sum(w64.reshape(n, k // g, g) ** 2, -1) + 1e-300
    assert np.all(np.abs(err_g - err_o) <= 1e-12 * scale)
    assert np.allclose(al_g, al_o, rtol=1e-10, atol=1e-14 * np.sqrt(scale.max()))
    assert np.mean(meta_g == meta_o) > 0.99
    assert np.array_equal(coef_g.view(np.uint16), c_g.astype(np.float16).view(np.uint16))
    assert not meta_g[3, :g // 8].any() and not coef_g[3, 0].any()
    # the device's own quantization through pack and the decode GEMV, against the oracle's layer on the same fields
    from tests.gpu_util import run_gemv, check_parity
    dd, packed = _pack(goq, n, k, g, b, codes_g, meta_g, coef_g, goq.LAYOUT_TILE16)
    xb = si.bf16_activations(2, k, seed=1)
    check_parity(run_gemv(dd, packed, xb, goq.F32), O.linear_f64(codes_g, meta_g, coef_g, si.bf16_bits_to_f64(xb), g, b), TIGHT, 1e-4)


def test_geo_quantizer_single_basis_layout(goq):
    n, k, g, b = 48, 512, 128, 3
    w = si.gaussian_weights(n, k, seed=4).astype(np.float32)
    c_o, m_o, f_o = O.quantize_k1(w, g, b)
    d = goq.desc(n, k, g, b, goq.LAYOUT_TILE16_K1)
    codes = torch.empty((n, k), dtype=torch.uint8, device="cuda")
    meta = torch.full((n, k // 8), 0xEE, dtype=torch.uint8, device="cuda")
    coef = torch.zeros((n, k // g, 2), dtype=torch.int16, device="cuda")
    goq.quantize_geo(d, torch.from_numpy(w).cuda(), codes, meta, coef)
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy(), c_o) and not meta.cpu().numpy().any()
    assert np.array_equal(coef.cpu().numpy().view(np.uint16), f_o.view(np.uint16))


# --------------------------------------------------------------------------------------------- REF solve
@pytest.mark.parametrize("n,k,g,b,m", [(40, 512, 128, 3, 100), (17, 256, 64, 2, 33), (24, 128, 32, 4, 7)])
def test_ref_solve_matches_oracle(goq, n, k, g, b, m):
    """Eq. 3 on synthetic calibration inputs (N(0,1) with a few outlier channels): the unrounded pairs agree with the
    oracle's ridge solution to float64 accuracy, the stored fp16 pairs are their roundings."""
    w = si.gaussian_weights(n, k, seed=n + m).astype(np.float32)
    codes, meta, _ = O.quantize_geo(w, g, b)
    x = si.f32_activations(m, k, seed=m).astype(np.float32)
    x[:, ::37] *= np.float32(8.0)
    c_ref = O.solve_ref(w, codes, meta, x, g, b, lam=1e-4)
    from tests.gpu_util import dev
    d = goq.desc(n, k, g, b)
    coef = torch.zeros((n, k // g, 2), dtype=torch.int16, device="cuda")
    c64 = torch.zeros((n, k // g, 2), dtype=torch.float64, device="cuda")
    goq.solve_ref(d, torch.from_numpy(w).cuda(), dev(codes), dev(meta), torch.from_numpy(x).cuda(), m, 1e-4, coef, c64)
    torch.cuda.synchronize()
    got = c64.cpu().numpy()
    assert np.allclose(got, c_ref, rtol=1e-9, atol=1e-12)
    assert np.array_equal(coef.cpu().numpy().view(np.uint16), got.astype(np.float16).view(np.uint16))
    # REF differs from GEO (the calibration covariance is not the identity) but stays a small correction of it
    _, _, c_geo = _objective(w.astype(np.float64), codes, meta, g, b)
    assert not np.allclose(got, c_geo, rtol=1e-3)
