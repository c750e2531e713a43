"""Pins for the oracle's quantizer: each check ties it to something the paper or the
mathematics fixes, not to the oracle itself."""
import itertools

import numpy as np
import pytest

import synth_inputs as si
from oracle import goq_oracle as O


# ---------------------------------------------------------------- lattice and pair tables
def test_lattice_3bit_matches_printed_set(golden):
    printed = sorted(float(t) for t in golden("lattice_3bit.txt")[0])
    assert sorted(O.lattice_values(3).tolist()) == printed
    # the code convention: c = sign<<2 | e, the positive smallest bin is the zero
    assert O.lattice_values(3).tolist() == [1.0, 0.5, 0.25, 0.0, -1.0, -0.5, -0.25, -0.125]


@pytest.mark.parametrize("b", [2, 3, 4])
def test_lattice_rule_general(b):
    vals = O.lattice_values(b)
    emax = O.emax_of(b)
    assert len(set(vals.tolist())) == 2 ** b          # all states distinct
    assert 0.0 in vals and +2.0 ** -emax not in vals   # smallest positive bin repurposed as zero
    assert -2.0 ** -emax in vals
    mags = sorted(set(np.abs(vals[vals != 0]).tolist()))
    assert mags == [2.0 ** -e for e in range(emax, -1, -1)]


def test_pair_tables_match_printed_sets(golden):
    for row in golden("pair_sets.txt"):
        s = int(row[0])
        printed = [tuple(int(v) for v in t.split(",")) for t in row[1:]]
        assert O.pair_table(s) == printed
        # sigma_s is an involution without fixed points and the pairs cover every lane once
        lanes = sorted(i for p in printed for i in p)
        assert lanes == list(range(8))


def test_storage_arithmetic(golden):
    pat_bits, sign_bits, bits, g, per_w, n_micro, n_terms = golden("storage_overhead.txt")[0]
    assert int(pat_bits) + int(sign_bits) == int(bits) == 6
    assert int(bits) / int(g) == float(per_w) == 0.75
    assert 128 // O.MICRO == int(n_micro)
    assert sum(len(O.pair_table(s)) for s in (1, 2, 3, 4)) == int(n_terms)
    # the record byte uses exactly 6 bits
    w = si.gaussian_weights(8, 256, seed=3)
    _, meta, _ = O.quantize_geo(w, 128, 3)
    assert meta.max() < 64 and meta.shape == (8, 256 // 8)


# ---------------------------------------------------------------- round to nearest
@pytest.mark.parametrize("b", [2, 3, 4])
def test_rtn_is_nearest_by_brute_force(b):
    rng = np.random.default_rng(1)
    v = rng.uniform(-1, 1, size=4000)
    codes = O.rtn_codes(v, b)
    vals = O.lattice_values(b)
    for x, c in zip(v, codes):
        d = np.abs(x - vals)
        assert d[c] == d.min()


def test_rtn_thresholds_and_ties_3bit():
    vals = O.lattice_values(3)
    eps = 1e-9
    # thresholds between neighbouring states
    for thr, lo, hi in [(-0.75, -1, -0.5), (-0.375, -0.5, -0.25), (-0.1875, -0.25, -0.125),
                        (-0.0625, -0.125, 0.0), (0.125, 0.0, 0.25), (0.375, 0.25, 0.5), (0.75, 0.5, 1.0)]:
        assert vals[O.rtn_codes(np.array([thr - eps]), 3)[0]] == lo
        assert vals[O.rtn_codes(np.array([thr + eps]), 3)[0]] == hi
        tie = vals[O.rtn_codes(np.array([thr]), 3)[0]]
        assert tie == (lo if abs(lo) < abs(hi) else hi)  # exact tie -> smaller magnitude


@pytest.mark.parametrize("b", [2, 4])
def test_rtn_ties_go_to_the_smaller_magnitude_at_other_widths(b):
    """The midpoint between any two neighbouring states of the b-bit lattice maps to the one of smaller magnitude,
    and a hair to either side maps to that side (the 3-bit case is spelt out threshold by threshold above)."""
    vals = np.sort(O.lattice_values(b))
    for lo, hi in zip(vals[:-1], vals[1:]):
        mid = 0.5 * (lo + hi)   # dyadic: exact in float64
        got = O.lattice_values(b)[O.rtn_codes(np.array([mid]), b)[0]]
        assert got == (lo if abs(lo) < abs(hi) else hi)
        assert O.lattice_values(b)[O.rtn_codes(np.array([mid - 1e-9]), b)[0]] == lo
        assert O.lattice_values(b)[O.rtn_codes(np.array([mid + 1e-9]), b)[0]] == hi


def test_largest_element_maps_to_unit():
    w = si.gaussian_weights(16, 256, seed=5)
    codes, _, _ = O.quantize_geo(w, 64, 3)
    b1 = O.decode_b1(codes, 3).reshape(16, 4, 64)
    wg = w.reshape(16, 4, 64)
    idx = np.argmax(np.abs(wg), axis=-1)
    top = np.take_along_axis(b1, idx[..., None], -1)[..., 0]
    assert np.array_equal(top, np.sign(np.take_along_axis(wg, idx[..., None], -1)[..., 0]))


# ---------------------------------------------------------------- Theorem 1
@pytest.mark.parametrize("b", [3, 4])
def test_orthogonality_exact_for_all_64_configurations(b):
    rng = np.random.default_rng(2)
    vals = O.lattice_values(b)
    for _ in range(50):
        x = vals[rng.integers(0, len(vals), size=8)]
        for s in (1, 2, 3, 4):
            for eta in itertools.product((1.0, -1.0), repeat=4):
                y = O.dual_exchange(x, s, np.array(eta))
                assert float(np.dot(x, y)) == 0.0                      # exact (dyadic rationals)
                assert sorted(np.abs(y).tolist()) == sorted(np.abs(x).tolist())  # signed permutation


def test_exchange_is_the_printed_rotation():
    x = np.arange(1.0, 9.0)
    # s = 2, pair (0,2) with eta=+1: y0 = -x2, y2 = +x0 ; pair (1,3) with eta=-1: y1 = +x3, y3 = -x1
    y = O.dual_exchange(x, 2, np.array([1.0, -1.0, 1.0, 1.0]))
    assert y.tolist() == [-3.0, 4.0, 1.0, -2.0, -7.0, -8.0, 5.0, 6.0]


def test_b2_from_record_matches_definition_and_b1_perp_b2():
    w = si.weights_with_outlier_channels(32, 512, seed=7)
    codes, meta, _ = O.quantize_geo(w, 128, 3)
    b1 = O.decode_b1(codes, 3)
    b2 = O.decode_b2(codes, meta, 3)
    # per micro-block orthogonality, exactly
    assert np.all(np.sum((b1 * b2).reshape(32, -1, 8), axis=-1) == 0.0)
    assert np.array_equal(np.sum(b1 * b1, 1), np.sum(b2 * b2, 1))
    # spot-check one micro-block by hand from its record byte
    n, t = 5, 9
    s = int(meta[n, t] & 3) + 1
    x = b1[n, 8 * t:8 * t + 8]
    y = np.zeros(8)
    for p, (i, j) in enumerate(O.pair_table(s)):
        eta = -1.0 if (meta[n, t] >> (2 + p)) & 1 else 1.0
        y[i], y[j] = -eta * x[j], eta * x[i]
    assert np.array_equal(y + 0.0, b2[n, 8 * t:8 * t + 8])
    # the zero state stays zero under a sign flip; +2^-emax may appear in b2 but never in b1
    assert not np.any(b1 == 0.125)
    assert np.array_equal(b2 == 0.0, np.isin(np.abs(b2), [0.0]))


# ---------------------------------------------------------------- residual, solver, coefficients
def _blocks(w, g):
    return w.reshape(w.shape[0], -1, g).astype(np.float64)


def test_residual_orthogonal_to_b1():
    w = si.gaussian_weights(8, 512, seed=11)
    codes, _, _, aux = O.quantize_geo(w, 128, 3, return_aux=True)
    b1 = O.decode_b1(codes, 3).reshape(8, 4, 128)
    wg = _blocks(w, 128)
    r = wg - aux["c"][..., 0:1] * b1
    dots = np.abs(np.sum(r * b1, -1))
    bound = 1e-12 * np.linalg.norm(wg, axis=-1) * np.linalg.norm(b1, axis=-1)
    assert np.all(dots <= bound)


@pytest.mark.parametrize("wb", [2, 3, 4])
def test_alignment_is_optimal_over_all_64_candidates(wb):
    """Per micro-block exhaustive search over (s, eta) gives the same best alignment."""
    w = si.gaussian_weights(4, 128, seed=13)
    codes, meta, _, aux = O.quantize_geo(w, 64, wb, return_aux=True)
    b1 = O.decode_b1(codes, wb).reshape(4, 2, 64)
    wg = _blocks(w, 64)
    r = wg - aux["c"][..., 0:1] * b1
    x = b1.reshape(4, 2, 8, 8)
    rho = r.reshape(4, 2, 8, 8)
    b2 = O.decode_b2(codes, meta, wb).reshape(4, 2, 8, 8)
    for idx in np.ndindex(4, 2, 8):
        best = -np.inf
        for s in (1, 2, 3, 4):
            for eta in itertools.product((1.0, -1.0), repeat=4):
                best = max(best, float(np.dot(O.dual_exchange(x[idx], s, np.array(eta)), rho[idx])))
        got = float(np.dot(b2[idx], rho[idx]))
        assert got == pytest.approx(best, rel=1e-12, abs=1e-15)
        assert got == pytest.approx(aux["alignment"].reshape(4, 2, 8)[idx], rel=1e-12, abs=1e-15)


@pytest.mark.parametrize("g,wb", [(8, 3), (16, 3), (8, 2), (8, 4), (16, 2)])
def test_joint_brute_force_over_dual_lattice_on_tiny_groups(g, wb):
    """Minimum reconstruction error over every (s, eta) assignment of every micro-block,
    with least-squares coefficients, equals what the analytical solver reaches."""
    rng = np.random.default_rng(17)
    for trial in range(6 if g == 8 else 2):
        w = rng.standard_normal((1, g)) * 0.02
        codes, meta, _, aux = O.quantize_geo(w, g, wb, return_aux=True)
        b1 = O.decode_b1(codes, wb)[0]
        b2 = O.decode_b2(codes, meta, wb)[0]
        c1, c2 = aux["c"][0, 0]
        err = float(np.sum((w[0] - c1 * b1 - c2 * b2) ** 2))
        configs = [(s, eta) for s in (1, 2, 3, 4) for eta in itertools.product((1.0, -1.0), repeat=4)]
        best = np.inf
        for combo in itertools.product(configs, repeat=g // 8):
            cand = np.concatenate([O.dual_exchange(b1[8 * t:8 * t + 8], s, np.array(eta))
                                   for t, (s, eta) in enumerate(combo)])
            a = np.stack([b1, cand], 1)
            sol, *_ = np.linalg.lstsq(a, w[0], rcond=None)
            best = min(best, float(np.sum((w[0] - a @ sol) ** 2)))
        assert err == pytest.approx(best, rel=1e-9, abs=1e-18)


def test_coefficients_decoupled_equal_general_2x2_solve_and_pythagoras():
    w = si.weights_with_outlier_channels(16, 512, seed=19)
    codes, meta, _, aux = O.quantize_geo(w, 128, 3, return_aux=True)
    b1 = O.decode_b1(codes, 3).reshape(16, 4, 128)
    b2 = O.decode_b2(codes, meta, 3).reshape(16, 4, 128)
    wg = _blocks(w, 128)
    for idx in np.ndindex(16, 4):
        a = np.stack([b1[idx], b2[idx]], 1)
        gram = a.T @ a
        assert gram[0, 1] == 0.0
        sol = np.linalg.solve(gram, a.T @ wg[idx])           # Eq. 2 without using orthogonality
        assert np.allclose(sol, aux["c"][idx], rtol=1e-11, atol=0)
        c1, c2 = aux["c"][idx]
        assert c2 >= 0.0                                        # c2 = sum of |alignments| / ||b1||^2
        assert c2 == pytest.approx(aux["alignment"].reshape(16, 4, 16)[idx].sum() / gram[0, 0], rel=1e-10)
        err2 = np.sum((wg[idx] - a @ sol) ** 2)
        pyth = np.sum(wg[idx] ** 2) - c1 * c1 * gram[0, 0] - c2 * c2 * gram[1, 1]
        assert err2 == pytest.approx(pyth, rel=1e-8, abs=1e-16)
        err1 = np.sum((wg[idx] - c1 * b1[idx]) ** 2)            # single-basis error
        assert err2 <= err1 + 1e-18


def test_power_of_two_scaling_invariance():
    w = si.gaussian_weights(8, 256, seed=23)
    c0, m0, f0, a0 = O.quantize_geo(w, 64, 3, return_aux=True)
    c1, m1, f1, a1 = O.quantize_geo(w * np.float32(2.0 ** -5), 64, 3, return_aux=True)
    assert np.array_equal(c0, c1) and np.array_equal(m0, m1)
    assert np.array_equal(a0["c"] * 2.0 ** -5, a1["c"])


def test_lattice_vector_is_reproduced_exactly():
    """w = alpha * b with alpha > 0 and b on the lattice with a +-1 entry: b1 = b, c2 = 0, w_hat = w."""
    rng = np.random.default_rng(29)
    vals = O.lattice_values(3)
    b = vals[rng.integers(0, 8, size=(4, 64))]
    b[:, 0] = [1.0, -1.0, 1.0, -1.0]
    alpha = 0.03125 * 3
    w = alpha * b
    codes, meta, coef, aux = O.quantize_geo(w, 64, 3, return_aux=True)
    assert np.array_equal(O.decode_b1(codes, 3), b)
    assert np.allclose(aux["c"][..., 0], alpha, rtol=1e-15) and np.all(np.abs(aux["c"][..., 1]) < 1e-17)


def test_planted_dual_basis_solution_is_recovered():
    """w = c1*b + c2*exchange(b) with a known record and small c2: the solver must reach zero error,
    which pins the sign rule, the pair order and the coefficient formulas together."""
    rng = np.random.default_rng(31)
    vals = O.lattice_values(3)
    for trial in range(20):
        b = vals[rng.integers(0, 8, size=64)]
        b[rng.integers(0, 64)] = 1.0
        s_true = rng.integers(1, 5, size=8)
        eta_true = rng.choice([1.0, -1.0], size=(8, 4))
        b2 = np.concatenate([O.dual_exchange(b[8 * t:8 * t + 8], int(s_true[t]), eta_true[t]) for t in range(8)])
        c1, c2 = 0.04, 0.04 * 0.02   # c2*|b2| <= 0.02*c1 keeps every element inside its rounding cell
        w = (c1 * b + c2 * b2)[None, :]
        codes, meta, _, aux = O.quantize_geo(w, 64, 3, return_aux=True)
        assert np.array_equal(O.decode_b1(codes, 3)[0], b)
        w_hat = aux["c"][0, 0, 0] * O.decode_b1(codes, 3)[0] + aux["c"][0, 0, 1] * O.decode_b2(codes, meta, 3)[0]
        assert np.max(np.abs(w_hat - w[0])) < 1e-16
        assert aux["c"][0, 0, 0] == pytest.approx(c1, rel=1e-12)
        assert aux["c"][0, 0, 1] == pytest.approx(c2, rel=1e-9)


def test_zero_block_bypass_and_input_checks():
    w = si.gaussian_weights(2, 128, seed=37)
    w[0, :64] = 0.0
    codes, meta, coef = O.quantize_geo(w, 64, 3)
    assert np.all(O.decode_b1(codes, 3)[0, :64] == 0.0) and np.all(meta[0, :8] == 0)
    assert np.all(coef[0, 0].astype(np.float64) == 0.0)
    with pytest.raises(ValueError):
        O.quantize_geo(np.array([[np.nan] * 64]), 64, 3)
    with pytest.raises(ValueError):
        O.quantize_geo(np.zeros((1, 100)), 64, 3)


def test_reconstruction_is_the_sum_of_two_signed_pot_terms_exactly():
    w = si.gaussian_weights(8, 256, seed=41)
    for b in (2, 3, 4):
        codes, meta, coef = O.quantize_geo(w, 64, b)
        w_hat = O.reconstruct(codes, meta, coef, 64, b)
        b1, b2 = O.decode_b1(codes, b), O.decode_b2(codes, meta, b)
        c = coef.astype(np.float64)
        for n, k in [(0, 0), (3, 77), (7, 255), (5, 128)]:
            j = k // 64
            t1 = c[n, j, 0] * b1[n, k]
            t2 = c[n, j, 1] * b2[n, k]
            for t, bv in ((t1, b1[n, k]), (t2, b2[n, k])):
                if bv != 0.0:   # each term is a signed power of two times the coefficient: mantissa unchanged
                    assert np.frexp(t)[0] in (np.frexp(c[n, j, 0])[0] * np.sign(bv), np.frexp(c[n, j, 1])[0] * np.sign(bv))
            assert w_hat[n, k] == t1 + t2
        # fp16-rounded coefficients stay close to the unrounded solve
        assert np.max(np.abs(w_hat - w)) < np.max(np.abs(w))
        # two bases never lose to one
        c1_only = c[..., 0].repeat(64, axis=1) * b1
        assert np.sum((w_hat - w) ** 2) <= np.sum((c1_only - w) ** 2) * (1 + 1e-3)


# ---------------------------------------------------------------------------------------------
# K = 1 (Section 3.1) and REF-mode coefficients (Section 3.4, Eq. 3)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("b", [2, 3, 4])
def test_k1_is_the_first_basis_of_the_dual_form_and_never_better(b):
    """Eq. 2 decouples, so the K = 1 scale is the dual form's c1; by Pythagoras the K = 2 error is the K = 1 error
    minus c2^2 ||b2||^2 (the K = 1 / K = 2 comparison of the basis-dimension ablation, here per block)."""
    w = si.gaussian_weights(24, 256, seed=70 + b).astype(np.float64)
    c1k, m1k, cf1 = O.quantize_k1(w, 64, b)
    c2k, m2k, cf2, aux = O.quantize_geo(w, 64, b, return_aux=True)
    assert np.array_equal(c1k, c2k) and not m1k.any()
    assert np.array_equal(cf1[..., 0], cf2[..., 0]) and not cf1[..., 1].any()
    wg = w.reshape(24, 4, 64)
    b1 = O.decode_b1(c2k, b).reshape(24, 4, 64)
    b2 = O.decode_b2(c2k, m2k, b).reshape(24, 4, 64)
    e1 = np.sum((wg - aux["c"][..., :1] * b1) ** 2, axis=-1)
    e2 = np.sum((wg - aux["c"][..., :1] * b1 - aux["c"][..., 1:] * b2) ** 2, axis=-1)
    assert np.all(e2 <= e1 + 1e-15)
    assert np.allclose(e1 - e2, aux["c"][..., 1] ** 2 * np.sum(b2 * b2, axis=-1), rtol=1e-9, atol=1e-18)
    # the K = 1 record evaluates to c1 b1 in the reference layer: the second term is multiplied by c2 = 0
    x = si.bf16_bits_to_f64(si.bf16_activations(3, 256, seed=1))
    y = O.linear_f64(c1k, m1k, cf1, x, 64, b)
    ref = x @ (O.coef_to_f64(cf1)[..., :1].repeat(64, axis=1).reshape(24, 256) * O.decode_b1(c1k, b)).T
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-15)


def test_ref_solve_against_library_least_squares_and_its_limits():
    """Eq. 3 pinned three ways: (1) ridge = ordinary least squares on the augmented system [A; sqrt(lam) I] c = [Y; 0]
    (library lstsq); (2) with orthonormal calibration rows spanning the block (X_q^T X_q = I) and lam -> 0 the
    activation-space problem is the weight-space one, so REF returns the GEO coefficients of Eq. 2; (3) the
    regulariser only shrinks: ||c(lam)|| decreases in lam."""
    rng = np.random.default_rng(5)
    n, k, g, b = 6, 128, 64, 3
    w = si.gaussian_weights(n, k, seed=91).astype(np.float64)
    codes, meta, coef, aux = O.quantize_geo(w, g, b, return_aux=True)
    x = rng.standard_normal((40, k))
    c = O.solve_ref(w, codes, meta, x, g, b, lam=1e-4)
    b1, b2 = O.decode_b1(codes, b), O.decode_b2(codes, meta, b)
    for r in range(n):
        for j in range(k // g):
            sl = slice(j * g, (j + 1) * g)
            a = np.stack([x[:, sl] @ b1[r, sl], x[:, sl] @ b2[r, sl]], axis=1)
            aug = np.vstack([a, np.sqrt(1e-4) * np.eye(2)])
            rhs = np.concatenate([x[:, sl] @ w[r, sl], np.zeros(2)])
            ref = np.linalg.lstsq(aug, rhs, rcond=None)[0]
            assert np.allclose(c[r, j], ref, rtol=1e-9, atol=1e-12)
    q, _ = np.linalg.qr(rng.standard_normal((g, g)))
    xo = np.zeros((g, k))
    xo[:, :g] = q
    xo[:, g:] = q[::-1]
    c0 = O.solve_ref(w, codes, meta, xo, g, b, lam=1e-13)
    assert np.allclose(c0, aux["c"], rtol=1e-8, atol=1e-11)
    norms = [np.linalg.norm(O.solve_ref(w, codes, meta, x, g, b, lam=l)) for l in (1e-6, 1e-2, 1e2)]
    assert norms[0] > norms[1] > norms[2]
