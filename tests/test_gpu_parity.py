"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Tolerances: float-activation outputs within 2e-3 normwise relative error of the fp64 oracle (the stated
bar); the fp32-accumulating kernels are expected far inside it, so a second, tight bound (2e-5) guards
against errors that the loose bar would hide. Integer accumulators: bit-exact.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import goq_oracle as O

pytestmark = pytest.mark.gpu

TOL = 2e-3
TIGHT = 2e-5
GEMM_TC_TOL = 5e-4   # fp16 weight operand of the tcgen05 GEMM (derivation in test_gemm_bf16_small_full_parity)
# Element-wise bounds, max |y - y_ref| / max |y_ref|. fp32-accumulating kernels: exact products, so the error of one
# output is fp32 summation (~sqrt(K) 2^-24 of the partial sums) plus, in the integer-operand form, the 2^-15 rounding
# of small activations: ~1e-5 of the largest output at K = 4096; 1e-4 leaves a factor 10 and still catches one wrong
# output (which would be off by a sizeable fraction of max |y_ref|). tcgen05 GEMM: independent 2^-12 roundings of the
# weights, ~2e-4 of a typical output, a few e-4 of the largest in the tail: 2e-3. bf16 outputs are checked against their
# rounding bound element by element (gpu_util.check_bf16_output).
ELEM_TIGHT = 1e-4
ELEM_TC = 2e-3


@pytest.fixture(scope="module")
def goq():
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq as g
    g.lib()
    assert torch.cuda.is_available()
    return g


def b2_reference_bytes(codes, meta, b):
    """Oracle b2 values in the byte format goq_unpack emits: (sign << 3) | e, 0x80 for zero."""
    b2 = O.decode_b2(codes, meta, b)
    out = np.full(b2.shape, 0x80, dtype=np.uint8)
    nz = b2 != 0
    e = np.zeros(b2.shape, dtype=np.int64)
    e[nz] = np.round(-np.log2(np.abs(b2[nz]))).astype(np.int64)
    out[nz] = (((b2[nz] < 0).astype(np.uint8) << 3) | e[nz].astype(np.uint8))
    return out


# ------------------------------------------------------------------------------------- pack / unpack
@pytest.mark.parametrize("n,k,g,b", [(256, 256, 64, 3), (40, 192, 64, 3), (17, 384, 128, 3), (33, 256, 32, 2),
                                     (24, 128, 16, 4), (16, 128, 8, 3)])
def test_pack_unpack_roundtrip_and_b2_derivation(goq, n, k, g, b):
    from tests.gpu_util import pack_weights
    w = si.gaussian_weights(n, k, seed=n + k)
    codes, meta, coef = O.quantize_geo(w, g, b)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    b1 = torch.full((n, k), 0xEE, dtype=torch.uint8, device="cuda")
    b2 = torch.full((n, k), 0xEE, dtype=torch.uint8, device="cuda")
    cf = torch.zeros((n, k // g, 2), dtype=torch.int16, device="cuda")
    goq.unpack(d, packed, b1, b2, cf)
    torch.cuda.synchronize()
    assert np.array_equal(b1.cpu().numpy(), codes)
    assert np.array_equal(b2.cpu().numpy(), b2_reference_bytes(codes, meta, b))
    assert np.array_equal(cf.cpu().numpy().view(np.uint16), coef.view(np.uint16))


def test_unpack_covers_all_64_records_and_all_codes(goq):
    from tests.gpu_util import pack_weights
    rng = np.random.default_rng(0)
    n, k = 64, 512
    codes = rng.integers(0, 8, size=(n, k), dtype=np.uint8)
    meta = (np.arange(n * k // 8) % 64).astype(np.uint8).reshape(n, k // 8)
    coef = rng.standard_normal((n, k // 128, 2)).astype(np.float16)
    d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
    b2 = torch.empty((n, k), dtype=torch.uint8, device="cuda")
    goq.unpack(d, packed, None, b2, None)
    torch.cuda.synchronize()
    assert np.array_equal(b2.cpu().numpy(), b2_reference_bytes(codes, meta, 3))


# ------------------------------------------------------------------------------------- decode GEMV
def _quantized(n, k, g, b, seed, outliers=False):
    w = si.weights_with_outlier_channels(n, k, seed=seed) if outliers else si.gaussian_weights(n, k, seed=seed)
    return O.quantize_geo(w, g, b)


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
@pytest.mark.parametrize("batch", [1, 8])
def test_config1_single_layer_256(goq, variant, batch):
    """K = N = 256, W3, group 64, fp16 coefficients, bf16 activations, batch 1 and 8, seed 0."""
    from tests.gpu_util import pack_weights, run_gemv
    codes, meta, coef = _quantized(256, 256, 64, 3, seed=0)
    d, packed = pack_weights(256, 256, 64, 3, codes, meta, coef)
    xb = si.bf16_activations(batch, 256, seed=0)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 64, 3)
    from tests.gpu_util import check_parity
    y = run_gemv(d, packed, xb, goq.F32, variant)
    check_parity(y, y_ref, TIGHT, ELEM_TIGHT, "fp32 out")
    y16 = run_gemv(d, packed, xb, goq.BF16, variant)
    from tests.gpu_util import check_bf16_output
    nerr = check_bf16_output(y16, y_ref, ELEM_TIGHT)   # one extra rounding of the output, checked element by element
    print("bf16 output: normwise error %.3e" % nerr)
    assert 0 < nerr <= 2.0 ** -8


@pytest.mark.parametrize("n,k,g,b,batch,variant", [
    (40, 192, 64, 3, 3, 1), (40, 192, 64, 3, 3, 2), (17, 384, 128, 3, 16, 2), (17, 384, 128, 3, 16, 1),
    (33, 256, 32, 2, 5, 2), (33, 256, 32, 2, 5, 1), (24, 128, 16, 4, 2, 1), (16, 128, 8, 3, 1, 1),
    (48, 256, 64, 4, 9, 2), (48, 256, 64, 4, 9, 1), (16, 128, 128, 3, 1, 2), (300, 1152, 128, 3, 12, 2),
    (40, 192, 64, 3, 3, 3), (17, 384, 128, 3, 16, 3), (33, 256, 32, 2, 5, 3), (16, 128, 128, 3, 1, 3),
    (300, 1152, 128, 3, 12, 3), (64, 512, 32, 3, 7, 3),
    (40, 192, 64, 3, 3, 0), (17, 384, 128, 3, 4, 0), (16, 128, 128, 3, 1, 0), (300, 1152, 128, 3, 2, 0),
    (48, 256, 64, 2, 4, 0), (130, 640, 128, 2, 1, 0), (129, 200 * 64, 64, 3, 2, 0),
])
def test_gemv_ragged_shapes_bit_widths_and_groups(goq, n, k, g, b, batch, variant):
    from tests.gpu_util import pack_weights, run_gemv
    codes, meta, coef = _quantized(n, k, g, b, seed=n * 7 + k, outliers=True)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    xb = si.bf16_activations(batch, k, seed=k)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, b)
    from tests.gpu_util import check_parity
    y = run_gemv(d, packed, xb, goq.F32, variant)
    check_parity(y, y_ref, TIGHT, ELEM_TIGHT)


@pytest.mark.parametrize("n,k,g,b,batch,variant", [(1000, 2048, 128, 3, 1, 0), (2100, 4224, 64, 3, 4, 0), (4096, 1024, 128, 3, 16, 3),
                                                   (1000, 2048, 128, 2, 9, 3), (72, 8192, 128, 3, 2, 0), (5000, 128, 32, 3, 3, 0)])
def test_gemv_tiles_split_across_ctas(goq, n, k, g, b, batch, variant):
    """Shapes whose 16-row tiles are shared by several CTAs (each CTA takes a contiguous range of unit records; partial
    sums meet in scratch and are added in CTA order), from one tile spread over 30 CTAs to 40 tiles per CTA; every
    output is compared, twice, and the two runs must agree bit for bit."""
    from tests.gpu_util import pack_weights, run_gemv, check_parity
    codes, meta, coef = si.random_quantized(n, k, g, b, seed=n + k + batch)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    xb = si.bf16_activations(batch, k, seed=batch)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, b)
    y = run_gemv(d, packed, xb, goq.F32, variant)
    nerr, eerr = check_parity(y, y_ref, TIGHT, ELEM_TIGHT)
    print("split tiles, variant %d: normwise %.3e element-wise %.3e" % (variant, nerr, eerr))
    assert np.array_equal(y, run_gemv(d, packed, xb, goq.F32, variant))


def test_two_kernel_variants_agree_closely_and_runs_are_deterministic(goq):
    from tests.gpu_util import pack_weights, run_gemv
    codes, meta, coef = si.random_quantized(512, 1024, 128, 3, seed=3)
    d, packed = pack_weights(512, 1024, 128, 3, codes, meta, coef)
    xb = si.bf16_activations(4, 1024, seed=4)
    y1 = run_gemv(d, packed, xb, goq.F32, 1)
    y2 = run_gemv(d, packed, xb, goq.F32, 2)
    assert O.normwise_rel_err(y1, y2) < 1e-5
    y3 = run_gemv(d, packed, xb, goq.F32, 3)
    assert O.normwise_rel_err(y3, y2) < 1e-5
    y0 = run_gemv(d, packed, xb, goq.F32, 0)   # batch 4: the chain kernel's integer operands
    assert O.normwise_rel_err(y0, y2) < 2e-5
    for v in (0, 1, 2, 3):
        a = run_gemv(d, packed, xb, goq.F32, v)
        b = run_gemv(d, packed, xb, goq.F32, v)
        assert np.array_equal(a, b)


def test_extreme_activations_keep_exponent_arithmetic_right(goq):
    """Zeros, tiny and huge bf16 values: the exponent-shift product must equal the true product."""
    from tests.gpu_util import pack_weights, run_gemv
    codes, meta, coef = si.random_quantized(32, 256, 64, 3, seed=5)
    d, packed = pack_weights(32, 256, 64, 3, codes, meta, coef)
    x = si.bf16_bits_to_f64(si.bf16_activations(2, 256, seed=6))
    x[0, ::3] = 0.0
    x[0, 1::7] *= 2.0 ** -120
    x[1, ::5] *= 2.0 ** 100
    xb = si.f32_to_bf16_bits(x.astype(np.float32))
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 64, 3)
    for v in (0, 1, 2, 3):
        assert O.normwise_rel_err(run_gemv(d, packed, xb, goq.F32, v), y_ref) <= TIGHT


@pytest.mark.parametrize("name,n,k", si.LLAMA2_7B_LINEARS[3:])
@pytest.mark.parametrize("batch", [1, 4, 16])
def test_config2_llama7b_shapes_sampled_rows(goq, name, n, k, batch):
    """7B-shaped linears, W3 group 128, full-size launch; the oracle evaluates a seeded sample of rows."""
    from tests.gpu_util import pack_weights, run_gemv
    codes, meta, coef = si.random_quantized(n, k, 128, 3, seed=n + k)
    rows = si.sample_rows(n, 96, seed=1)
    # rows quantized by the oracle from outlier-channel weights replace the random fields in the sample
    w = si.weights_with_outlier_channels(len(rows), k, seed=7)
    codes[rows], meta[rows], coef[rows] = O.quantize_geo(w, 128, 3)
    d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
    xb = si.bf16_activations(batch, k, seed=batch)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 128, 3, rows=rows)
    from tests.gpu_util import check_parity
    y = run_gemv(d, packed, xb, goq.F32)
    check_parity(y[:, rows], y_ref, TIGHT, ELEM_TIGHT)


_CFG5 = {name: (n, k) for name, n, k in si.LLAMA2_70B_LINEARS}


@pytest.mark.parametrize("name,b,batch", [("mlp_gate_up", 2, 1), ("mlp_down", 3, 16), ("attn_qo", 4, 1),
                                          ("gqa_kv", 2, 16), ("attn_qo", 3, 4)])
def test_config5_llama70b_shapes_bit_width_sweep_sampled_rows(goq, name, b, batch):
    """70B-shaped linears at W2/W3/W4, group 128, full-size launch; the oracle evaluates sampled rows."""
    from tests.gpu_util import pack_weights, run_gemv
    n, k = _CFG5[name]
    codes, meta, coef = si.random_quantized(n, k, 128, b, seed=n + k + b)
    rows = si.sample_rows(n, 48, seed=3)
    w = si.weights_with_student_t_channels(len(rows), k, seed=9)
    codes[rows], meta[rows], coef[rows] = O.quantize_geo(w, 128, b)
    d, packed = pack_weights(n, k, 128, b, codes, meta, coef)
    xb = si.bf16_activations(batch, k, seed=batch + b)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 128, b, rows=rows)
    from tests.gpu_util import check_parity
    y = run_gemv(d, packed, xb, goq.F32)
    check_parity(y[:, rows], y_ref, TIGHT, ELEM_TIGHT)


@pytest.mark.parametrize("name,b,m", [("gqa_kv", 4, 256), ("attn_qo", 2, 64), ("attn_qo", 4, 700), ("attn_qo", 3, 64),
                                      ("mlp_gate_up", 3, 256), ("mlp_down", 3, 64)])
def test_config5_llama70b_shapes_crossover_batches_on_the_gemm(goq, name, b, m):
    """The batch sweep's upper end (64, 256 tokens and beyond) goes through goq_gemm: 70B-shaped linears at W2 / W4
    on the tensor-core kernel (split-K at 64 and 256 tokens), sampled rows against the oracle."""
    from tests.gpu_util import pack_weights, run_gemm_bf16
    n, k = _CFG5[name]
    codes, meta, coef = si.random_quantized(n, k, 128, b, seed=n + k + b + 1)
    rows = si.sample_rows(n, 32, seed=5)
    w = si.weights_with_student_t_channels(len(rows), k, seed=10)
    codes[rows], meta[rows], coef[rows] = O.quantize_geo(w, 128, b)
    d, packed = pack_weights(n, k, 128, b, codes, meta, coef)
    xb = si.bf16_activations(m, k, seed=m + b)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 128, b, rows=rows)
    from tests.gpu_util import check_parity
    y = run_gemm_bf16(d, packed, xb)
    check_parity(y[:, rows], y_ref, GEMM_TC_TOL, ELEM_TC)


# ------------------------------------------------------------------------------------- prefill GEMM
@pytest.mark.parametrize("n,k,g,b,m,variant", [
    (80, 384, 128, 3, 150, 0), (80, 384, 128, 3, 150, 2), (256, 512, 64, 3, 600, 0), (40, 192, 32, 2, 17, 0),
    (130, 256, 8, 3, 513, 0), (16, 128, 16, 3, 1, 0), (300, 1152, 128, 3, 1030, 0), (96, 256, 64, 3, 60, 0),
    (64, 256, 64, 3, 256, 0), (64, 256, 64, 3, 257, 0), (80, 384, 128, 4, 150, 0), (40, 256, 32, 4, 20, 0), (300, 1152, 64, 4, 600, 0), (130, 256, 8, 4, 513, 0),
])
def test_gemm_bf16_small_full_parity(goq, n, k, g, b, m, variant):
    """Prefill GEMM, every output compared. variant 2: the two-operand mma.sync kernel, held to the tight bound.
    variant 0: from 65 tokens on the tcgen05 kernel, whose weight operand is w_hat rounded once to fp16: a relative
    error uniform in +-2^-12 per weight, rms 2^-12/sqrt(3) = 1.4e-4, independent between weights, so the normwise
    output error is of that size; bound 5e-4. (Up to 32 tokens and group >= 32, variant 0 is the streaming GEMV: tight bound.)"""
    from tests.gpu_util import pack_weights, run_gemm_bf16
    codes, meta, coef = _quantized(n, k, g, b, seed=11 + n, outliers=True)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    xb = si.bf16_activations(m, k, seed=12)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, b)
    y = run_gemm_bf16(d, packed, xb, variant=variant)
    err = O.normwise_rel_err(y, y_ref)
    print("gemm variant %d: normwise error %.3e" % (variant, err))
    # up to 32 tokens the streaming GEMV (W <= 3, group >= 32) or the exact mma.sync kernel (W4) takes the call
    on_tc = variant == 0 and (m > 32 or (g < 32 and b <= 3))
    assert err <= TOL and err <= (GEMM_TC_TOL if on_tc else TIGHT), err
    from tests.gpu_util import elementwise_rel_err
    assert elementwise_rel_err(y, y_ref) <= (ELEM_TC if on_tc else ELEM_TIGHT)


@pytest.mark.parametrize("n,k", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_config4_prefill_2048_tokens_sampled_rows(goq, n, k):
    """The three linear shapes of the 7B layer at M = 2048, full-size launches (11008 x 4096: 296 full tiles and a
    tail wave of half tiles; 4096 x 11008: the longest fp16 accumulation, 172 k-chunks), sampled rows, all tokens."""
    from tests.gpu_util import pack_weights, run_gemm_bf16, check_parity
    m = 2048
    codes, meta, coef = si.random_quantized(n, k, 128, 3, seed=21 + n + k)
    rows = si.sample_rows(n, 48, seed=2)
    w = si.gaussian_weights(len(rows), k, seed=22)
    codes[rows], meta[rows], coef[rows] = O.quantize_geo(w, 128, 3)
    d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
    xb = si.bf16_activations(m, k, seed=23)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 128, 3, rows=rows)
    y = run_gemm_bf16(d, packed, xb)
    nerr, eerr = check_parity(y[:, rows], y_ref, GEMM_TC_TOL, ELEM_TC)
    print("M=2048 %dx%d: normwise %.3e element-wise %.3e" % (n, k, nerr, eerr))


@pytest.mark.parametrize("b", [3, 4])
def test_gemm_small_and_mixed_weight_magnitudes(goq, b):
    """The tcgen05 GEMM forms w_hat in fp16. Weights of standard deviation 2e-2 .. 1.2e-6 (coefficients down into fp16's
    subnormal range) and a layer whose channels differ by 2^12 in scale must all come out at the kernel's usual accuracy:
    every channel's coefficients are scaled by a power of two before w_hat is formed and the epilogue undoes it."""
    from tests.gpu_util import pack_weights, run_gemm_bf16, check_parity
    n, k, g, m = 256, 1024, 128, 200
    xb = si.bf16_activations(m, k, seed=6)
    for exp in (0, -8, -12, -14):
        w = si.gaussian_weights(n, k, seed=5) * 2.0 ** exp
        if exp == -8:
            w[::3] *= 2.0 ** -12   # channels of very different scale inside one 128-channel tile
        codes, meta, coef = O.quantize_geo(w, g, b)
        d, packed = pack_weights(n, k, g, b, codes, meta, coef)
        y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, b)
        y = run_gemm_bf16(d, packed, xb)
        # per channel: a channel 2^12 below its neighbours must be as accurate as they are
        err = np.linalg.norm(y - y_ref, axis=0) / np.maximum(np.linalg.norm(y_ref, axis=0), 1e-300)
        live = np.linalg.norm(y_ref, axis=0) > 0
        assert np.max(err[live]) <= 4 * GEMM_TC_TOL, (exp, float(np.max(err[live])))
        assert O.normwise_rel_err(y, y_ref) <= GEMM_TC_TOL, (exp, O.normwise_rel_err(y, y_ref))


def test_gemm_token_scaling_extreme_activations(goq):
    """The tcgen05 GEMM feeds fp16 activations scaled per token by a power of two. Tokens of very different
    magnitude (2^100, 2^-100), an all-zero token, a token whose elements span 2^24 and one with many zeros must
    all come out at the kernel's usual accuracy, each token judged on its own norm."""
    from tests.gpu_util import pack_weights, run_gemm_bf16
    n, k, m, g, b = 144, 512, 200, 64, 3
    codes, meta, coef = _quantized(n, k, g, b, seed=51)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    x = si.bf16_bits_to_f64(si.bf16_activations(m, k, seed=52))
    x[3] *= 2.0 ** 100
    x[4] *= 2.0 ** -100
    x[5] = 0.0
    x[6, ::2] *= 2.0 ** 24       # half of the token 2^24 above the rest: the small half is still above 2^-28 of the largest
    x[7, 1::3] = 0.0
    x[8, :] = 0.0
    x[8, 17] = -3.0              # a single non-zero element
    xb = si.f32_to_bf16_bits(x.astype(np.float32))
    xr = si.bf16_bits_to_f64(xb)
    y_ref = O.linear_f64(codes, meta, coef, xr, g, b)
    y = run_gemm_bf16(d, packed, xb)
    assert np.all(np.isfinite(y))
    assert np.all(y[5] == 0.0)
    for tok in range(m):
        if tok == 5:
            continue
        e = np.linalg.norm(y[tok] - y_ref[tok]) / np.linalg.norm(y_ref[tok])
        assert e <= GEMM_TC_TOL, (tok, e)


@pytest.mark.parametrize("n,k,g,m", [(200, 2048, 128, 100), (130, 1152, 64, 256), (520, 4096, 128, 49)])
def test_gemm_split_k_few_tokens(goq, n, k, g, m):
    """At most 256 tokens and few channel tiles: several CTAs share a tile along k (4, 2 and 4 splits here, the last
    one ragged), park partial tiles in the scratch buffer and the last to arrive adds them in split order. Every output
    compared; a second call on the same scratch buffer must give the same bits (the counters are left zero)."""
    from tests.gpu_util import pack_weights, dev
    codes, meta, coef = _quantized(n, k, g, 3, seed=61 + n)
    d, packed = pack_weights(n, k, g, 3, codes, meta, coef)
    xb = si.bf16_activations(m, k, seed=62)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, 3)
    x = dev(xb)
    ws = goq.new_workspace(d, goq.OP_GEMM, m)
    outs = []
    for _ in range(2):
        y = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        goq.gemm(d, packed, x, m, goq.BF16, y=y, y_dtype=goq.F32, ws=ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        outs.append(y)
    assert torch.equal(outs[0], outs[1])
    err = O.normwise_rel_err(outs[0].cpu().numpy().astype(np.float64), y_ref)
    assert err <= GEMM_TC_TOL, err


def test_one_scratch_buffer_serves_calls_of_different_shapes_and_kernels(goq):
    """Every kernel keeps its counters in the same leading area of the scratch buffer and leaves them zero, and
    nothing else is carried between calls: a buffer sized for the largest call, initialised once, must give the same
    bits as a fresh buffer per call - streaming GEMV (tiles that straddle CTAs park partial sums), the sequence
    kernel behind goq_gemv, the tensor-core GEMM with and without split-K, interleaved and repeated."""
    from tests.gpu_util import pack_weights, dev
    layers = []
    for i, (n, k, g) in enumerate([(1000, 1152, 128), (300, 4224, 64), (130, 2048, 128)]):
        codes, meta, coef = si.random_quantized(n, k, g, 3, seed=70 + i)
        d, packed = pack_weights(n, k, g, 3, codes, meta, coef)
        layers.append((d, packed, n, k))
    calls = []   # (layer index, op, m)
    for rep in range(2):
        for li in range(3):
            calls += [(li, "gemv", 16), (li, "gemm", 100), (li, "gemv", 1), (li, "gemm", 300), (li, "gemv", 5)]
    xs = {m: {li: dev(si.bf16_activations(m, layers[li][3], seed=80 + m + li)) for li in range(3)} for m in (1, 5, 16, 100, 300)}
    need = max(goq.workspace_bytes(layers[li][0], goq.OP_GEMV if op == "gemv" else goq.OP_GEMM, m) for li, op, m in calls)
    shared = torch.empty(need, dtype=torch.uint8, device="cuda")
    goq.workspace_init(shared)

    def run(li, op, m, ws):
        d, packed, n, k = layers[li]
        y = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        if op == "gemv":
            goq.gemv(d, packed, xs[m][li], m, y, goq.F32, ws=ws)
        else:
            goq.gemm(d, packed, xs[m][li], m, goq.BF16, y=y, y_dtype=goq.F32, ws=ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        return y

    for li, op, m in calls:
        fresh = goq.new_workspace(layers[li][0], goq.OP_GEMV if op == "gemv" else goq.OP_GEMM, m)
        want = run(li, op, m, fresh)
        got = run(li, op, m, shared)
        assert torch.isfinite(got).all()
        assert torch.equal(want, got), (li, op, m)


@pytest.mark.parametrize("m", [100, 700])
def test_gemm_output_alignment_does_not_change_the_result(goq, m):
    """The GEMM epilogue stores 16 bytes per thread when the output allows it and element by element otherwise:
    an output that starts 4 (fp32) or 2 (bf16) bytes off a 16-byte boundary must hold the same bits."""
    from tests.gpu_util import pack_weights, dev
    n, k = 256, 1024
    codes, meta, coef = si.random_quantized(n, k, 128, 3, seed=91)
    d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
    x = dev(si.bf16_activations(m, k, seed=92))
    ws = goq.new_workspace(d, goq.OP_GEMM, m)
    for dtype, code in ((torch.float32, goq.F32), (torch.bfloat16, goq.BF16)):
        flat = torch.zeros(m * n + 8, dtype=dtype, device="cuda")
        aligned = flat[:m * n].view(m, n)
        goq.gemm(d, packed, x, m, goq.BF16, y=aligned, y_dtype=code, ws=ws)
        torch.cuda.synchronize()
        want = aligned.clone()
        flat2 = torch.zeros(m * n + 8, dtype=dtype, device="cuda")
        shifted = flat2[1:m * n + 1].view(m, n)
        assert shifted.data_ptr() % 16 != 0
        goq.gemm(d, packed, x, m, goq.BF16, y=shifted, y_dtype=code, ws=ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        assert torch.equal(want, shifted)
        assert float(flat2[0]) == 0.0 and float(flat2[m * n + 1:].abs().sum()) == 0.0


def test_gemm_tail_wave_runs_as_half_tiles(goq):
    """160 output tiles (20 channel tiles x 8 token tiles) on 148 SMs: the 12 tiles of the last wave are scheduled
    as 24 half tiles of 256 tokens; 3900 tokens make the last token tile ragged. Sampled channels, all tokens."""
    from tests.gpu_util import pack_weights, run_gemm_bf16
    n, k, m = 2560, 256, 3900
    codes, meta, coef = si.random_quantized(n, k, 64, 3, seed=41)
    rows = np.unique(np.concatenate([si.sample_rows(n, 48, seed=4), np.arange(n - 130, n)]))   # the split tiles are the last ones
    d, packed = pack_weights(n, k, 64, 3, codes, meta, coef)
    xb = si.bf16_activations(m, k, seed=42)
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 64, 3, rows=rows)
    y = run_gemm_bf16(d, packed, xb)
    assert O.normwise_rel_err(y[:, rows], y_ref) <= GEMM_TC_TOL
    # every token of the ragged last tile, channel by channel
    assert np.max(np.abs(y[3584:, rows] - y_ref[3584:])) <= 5e-3 * np.max(np.abs(y_ref))


# ------------------------------------------------------------------------------------- integer path
@pytest.mark.parametrize("n,k,g,b,m", [(48, 256, 64, 3, 200), (20, 192, 32, 2, 130), (16, 128, 128, 3, 1),
                                       (40, 128, 16, 3, 70), (200, 384, 128, 3, 333)])
def test_int8_path_bit_exact_small(goq, n, k, g, b, m):
    from tests.gpu_util import pack_weights, run_gemm_i8
    codes, meta, coef = _quantized(n, k, g, b, seed=31)
    cq, sc = O.quantize_coefficients_int8(coef)
    xq, sx = O.quantize_activations_int8(si.f32_activations(m, k, seed=32))
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    acc, y = run_gemm_i8(d, packed, xq, sx, cq, sc)
    a1, a2, y_ref = O.linear_i32(codes, meta, cq, sc, xq, sx, g, b)
    assert np.array_equal(acc[0], a1) and np.array_equal(acc[1], a2)
    assert O.normwise_rel_err(y, y_ref) <= TIGHT


@pytest.mark.parametrize("name,n,k", si.VIT_B16_LINEARS)
def test_config3_vit_b16_int8_bit_exact(goq, name, n, k):
    """ViT-B/16-shaped linears, 197 x 64 tokens, W3 group 64, per-token int8 activations:
    full-size launch, int32 accumulators compared bit for bit on a seeded sample of output channels
    (all tokens) - and on every channel for the extreme activations of the first 64 tokens."""
    from tests.gpu_util import pack_weights, run_gemm_i8
    m = si.VIT_B16_TOKENS
    w = si.gaussian_weights(n, k, seed=n + k)
    codes, meta, coef = O.quantize_geo(w, 64, 3)
    cq, sc = O.quantize_coefficients_int8(coef)
    xq, sx = O.quantize_activations_int8(si.f32_activations(m, k, seed=41))
    xq[:32] = 127
    xq[32:64] = -127
    d, packed = pack_weights(n, k, 64, 3, codes, meta, coef)
    acc, y = run_gemm_i8(d, packed, xq, sx, cq, sc)
    rows = si.sample_rows(n, 48, seed=3)
    a1, a2, y_ref = O.linear_i32(codes, meta, cq, sc, xq, sx, 64, 3, rows=rows)
    assert np.array_equal(acc[0][:, rows], a1) and np.array_equal(acc[1][:, rows], a2)
    assert O.normwise_rel_err(y[:, rows], y_ref) <= TIGHT
    b1, b2, _ = O.linear_i32(codes, meta, cq, sc, xq[:64], sx[:64], 64, 3)
    assert np.array_equal(acc[0][:64], b1) and np.array_equal(acc[1][:64], b2)


# ------------------------------------------------------------------------------------- boundary behaviour
def test_argument_errors_return_status_without_launching(goq):
    d = goq.desc(32, 256, 64, 3)
    packed = torch.zeros(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
    x = torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 32), dtype=torch.float32, device="cuda")

    def status(fn, *a, **kw):
        try:
            fn(*a, **kw)
        except goq.GoqError as e:
            return e.status
        return goq.OK

    assert status(goq.gemv, d, packed, x, 0, y, goq.F32) == goq.ERR_INVALID_ARG
    assert status(goq.gemv, d, packed, x, 17, y, goq.F32) == goq.ERR_INVALID_ARG
    assert status(goq.gemv, d, packed, x, 1, y, 5) == goq.ERR_INVALID_ARG
    assert status(goq.gemv, d, None, x, 1, y, goq.F32) == goq.ERR_INVALID_ARG
    assert status(goq.gemv, goq.desc(32, 250, 64, 3), packed, x, 1, y, goq.F32) == goq.ERR_INVALID_ARG
    xo = torch.zeros(2 * 256 + 8, dtype=torch.bfloat16, device="cuda")[1:]
    assert status(goq.gemv, d, packed, xo, 1, y, goq.F32) == goq.ERR_ALIGNMENT
    assert status(goq.gemv, d, packed[16:], x, 1, y, goq.F32) == goq.ERR_ALIGNMENT
    assert goq.workspace_bytes(d, goq.OP_GEMV, 1) > 0
    assert status(goq.gemv, d, packed, x, 1, y, goq.F32) == goq.ERR_WORKSPACE          # scratch missing
    tiny = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert status(goq.gemv, d, packed, x, 1, y, goq.F32, ws=tiny) == goq.ERR_WORKSPACE  # scratch too small
    small = torch.zeros(64, dtype=torch.uint8, device="cuda")
    z = torch.zeros(32 * 256, dtype=torch.uint8, device="cuda")
    assert status(goq.pack, d, z, z, z, small) == goq.ERR_WORKSPACE
    # integer path: static overflow bound and missing operands
    big = goq.desc(16, 16768, 128, 3)
    pb = torch.zeros(goq.packed_bytes(big), dtype=torch.uint8, device="cuda")
    xi = torch.zeros((1, 16768), dtype=torch.int8, device="cuda")
    cqz = torch.zeros((16, 131, 2), dtype=torch.int8, device="cuda")
    acc = torch.zeros((2, 1, 16), dtype=torch.int32, device="cuda")
    assert status(goq.gemm, big, pb, xi, 1, goq.I8, cq=cqz, acc=acc) == goq.ERR_OVERFLOW_BOUND
    assert status(goq.gemm, d, packed, xi, 1, goq.I8, acc=acc) == goq.ERR_INVALID_ARG
    assert status(goq.gemm, d, packed, x, 1, 9, y=y) == goq.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(y.abs().sum()) == 0.0


def test_outputs_do_not_spill_past_their_buffers(goq):
    from tests.gpu_util import pack_weights, dev
    n, k, batch = 40, 192, 3
    codes, meta, coef = _quantized(n, k, 64, 3, seed=51)
    d, packed = pack_weights(n, k, 64, 3, codes, meta, coef)
    x = dev(si.bf16_activations(batch, k, seed=52))
    ws = goq.new_workspace(d, goq.OP_GEMV, batch)
    for variant in (1, 2, 3):
        buf = torch.full((batch * n + 64,), 7.5, dtype=torch.float32, device="cuda")
        y = buf[32:32 + batch * n]
        prev = goq.set_gemv_variant(variant)
        goq.gemv(d, packed, x, batch, y, goq.F32, ws=ws)
        goq.set_gemv_variant(prev)
        torch.cuda.synchronize()
        h = buf.cpu().numpy()
        assert np.all(h[:32] == 7.5) and np.all(h[-32:] == 7.5) and not np.any(h[32:-32] == 7.5)


def test_host_buffer_entry_point(goq):
    from tests.gpu_util import pack_weights
    n, k, batch = 64, 256, 4
    codes, meta, coef = _quantized(n, k, 64, 3, seed=61)
    d, packed = pack_weights(n, k, 64, 3, codes, meta, coef)
    xb = si.bf16_activations(batch, k, seed=62)
    xh = torch.from_numpy(xb.view(np.int16)).pin_memory()
    yh = torch.zeros((batch, n), dtype=torch.float32).pin_memory()
    xs = torch.empty((batch, k), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((batch, n), dtype=torch.float32, device="cuda")
    ws = goq.new_workspace(d, goq.OP_GEMV, batch)
    goq.gemv_host(d, packed, xh, batch, yh, goq.F32, xs, ys, ws=ws)
    torch.cuda.synchronize()
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 64, 3)
    assert O.normwise_rel_err(yh.numpy().astype(np.float64), y_ref) <= TIGHT


def test_weights_packed_just_before_the_call_on_the_same_stream(goq):
    """Stream order without a synchronise in between: goq_pack writes the packed image, and the very next calls on the same
    stream are goq_gemv (batch 1, the chain kernel), goq_gemm at 300 tokens (tcgen05 kernel, launched as a programmatic
    dependent of its pre-pass) and goq_gemv_sequence. Each must give the bits of the same call made after a synchronise:
    none of these kernels reads the weights before the preceding work on the stream is complete. (The streaming kernel
    behind goq_gemv at batch 5..16 prefetches weights ahead of its dependency wait; its rule is stated in goq.h.)"""
    from tests.gpu_util import dev
    n, k, g, b, m = 2048, 1024, 128, 3, 300
    codes, meta, coef = si.random_quantized(n, k, g, b, seed=77)
    d = goq.desc(n, k, g, b)
    x1, xm = dev(si.bf16_activations(1, k, seed=78)), dev(si.bf16_activations(m, k, seed=79))
    cd, md, fd = dev(codes), dev(meta), dev(coef)
    ws_v, ws_m = goq.new_workspace(d, goq.OP_GEMV, 1), goq.new_workspace(d, goq.OP_GEMM, m)
    ws_s = torch.empty(goq.sequence_workspace_bytes(2), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws_s)
    torch.cuda.synchronize()

    def run(sync_between):
        packed = torch.full((goq.packed_bytes(d),), 0x5A, dtype=torch.uint8, device="cuda")   # stale contents
        y1 = torch.zeros((1, n), dtype=torch.float32, device="cuda")
        ym = torch.zeros((m, n), dtype=torch.float32, device="cuda")
        ya = torch.zeros((1, n), dtype=torch.bfloat16, device="cuda")
        yb = torch.zeros((1, n), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        goq.pack(d, cd, md, fd, packed)
        if sync_between:
            torch.cuda.synchronize()
        goq.gemv(d, packed, x1, 1, y1, goq.F32, ws=ws_v)
        if sync_between:
            torch.cuda.synchronize()
        goq.gemm(d, packed, xm, m, goq.BF16, y=ym, y_dtype=goq.F32, ws=ws_m)
        if sync_between:
            torch.cuda.synchronize()
        seq = goq.make_sequence([(d, packed, x1, 1, ya, goq.BF16, False), (d, packed, ya[:, :k], 1, yb, goq.F32, False)])
        goq.gemv_sequence(seq, ws_s)
        torch.cuda.synchronize()
        for w in (ws_v, ws_m, ws_s):
            assert goq.workspace_status(w) == goq.OK
        return y1.clone(), ym.clone(), ya.clone(), yb.clone()

    ref = run(True)
    for rep in range(3):
        got = run(False)
        for a, r in zip(got, ref):
            assert torch.equal(a, r), rep
    y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(x1.view(torch.int16).cpu().numpy().view(np.uint16)), g, b)
    assert O.normwise_rel_err(ref[0].cpu().numpy().astype(np.float64), y_ref) <= TIGHT
