"""CPU oracle for the GoQuant dual-basis Power-of-Two linear layer (arxiv 2605.26092).

THIS IS TEST INFRASTRUCTURE. It is a plain, slow, float64 / exact-integer restatement of
what the paper defines, written to be checked against the paper by eye. Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import it; the CUDA library never
does, and the two share no code.

What is here, with the passage each part follows:

  lattice_values        Section 3.2, the asymmetric lattice L_3bit, generalised to b bits by
                        the rule stated there (the smallest positive bin becomes zero).
  rtn_codes             Section 3.2, b1 = Q(w / ||w||_inf), element-wise round to nearest.
  pair_table            Section 3.3, Theorem 1: sigma_s(i) = i XOR s, P_s = {(i, sigma_s(i)) : i < sigma_s(i)}.
  dual_exchange         Section 3.3, Theorem 1: (y_i, y_j) = (-eta x_j, eta x_i) for each pair.
  quantize_geo          Section 3.2 (Eq. 1 residual), Section 3.3 steps 1-3 (eta*, A_s, s*,
                        6-bit record per micro-block), Section 3.4 GEO mode (Eq. 2, decoupled c1, c2).
  decode_b1 / decode_b2 / reconstruct
                        Section 3.1: w_hat = c1 b1 + c2 b2; Section 3.3 on carrying the PoT
                        magnitude and the sign separately (a flipped zero stays zero; +2^-emax may appear in b2).
  quantize_k1           Section 3.1, the single-basis form w_hat = c1 b1 (the K = 1 row of the basis-dimension
                        ablation): b1 as in Section 3.2, c1 the least-squares scale, no second basis.
  solve_ref             Section 3.4, REF mode (Eq. 3): c* = (A^T A + lambda I)^-1 A^T Y per macro-block with
                        A = [X_q b1, X_q b2], Y = X_q w, lambda = 1e-4.
  linear_f64            Section 3.5, Eq. 4, float activations: per-group dot products against
                        b1 and b2, coefficients applied to the group sums.
  quantize_activations_int8 / quantize_activations_int / quantize_coefficients_int8 / linear_i32
                        Section 3.5, Eq. 4 with integer X~ and c~: exact integer S1, S2, ACC1, ACC2.

Readings taken where the paper is silent (each is also listed in the design notes):
  * b-bit lattice for b != 3: magnitudes 2^0 .. 2^-emax with emax = 2^(b-1) - 1, every negative,
    every positive except +2^-emax, plus 0.
  * round-to-nearest ties go to the state of smaller magnitude.
  * eta = +1 when the sign argument is exactly 0; the smallest s among equal A_s wins.
  * a real layer has K/g macro-blocks per output channel: coefficients multiply per-group sums.
  * coefficients are stored as fp16 (round to nearest even); the rounded values are "the" coefficients.
  * integer path: left shifts x~ << (emax - e) (lossless) with 2^-emax folded into the output
    scale; 8-bit symmetric coefficient integers with one scale per output channel and basis;
    per-token symmetric int8 activations.

Code convention: code c in [0, 2^b): sign = c >> (b-1), e = c & emax,
value = (-1)^sign * 2^-e, except c == emax (sign 0, e = emax) which is 0.
Record byte per micro-block: bits[1:0] = s - 1, bit (2 + p) = 1 iff eta of the p-th pair of
P_s (pairs in ascending order of their lower index) is -1.

Parity pins for every function live in tests/test_oracle_*.py. Accuracy figures of the paper
(perplexity, top-1) need its models and datasets: parity unpinned, not attempted.
"""
from __future__ import annotations

import numpy as np

MICRO = 8  # micro-block size G (Section 3.3)


# ----------------------------------------------------------------------------------------
# Lattice and codes (Section 3.2)
# ----------------------------------------------------------------------------------------
def emax_of(wbits: int) -> int:
    return (1 << (wbits - 1)) - 1


def lattice_values(wbits: int) -> np.ndarray:
    """value[c] for every code c of the b-bit asymmetric PoT lattice."""
    emax = emax_of(wbits)
    vals = np.zeros(1 << wbits, dtype=np.float64)
    for c in range(1 << wbits):
        sign = c >> (wbits - 1)
        e = c & emax
        if sign == 0 and e == emax:
            vals[c] = 0.0
        else:
            vals[c] = (-1.0) ** sign * 2.0 ** (-e)
    return vals


def rtn_codes(v: np.ndarray, wbits: int) -> np.ndarray:
    """Nearest lattice state to each element of v (linear distance); ties -> smaller magnitude."""
    vals = lattice_values(wbits)
    order = np.argsort(np.abs(vals), kind="stable")  # candidates by ascending magnitude
    cand = vals[order]
    v = np.asarray(v, dtype=np.float64)
    dist = np.abs(v[..., None] - cand)
    pick = np.argmin(dist, axis=-1)  # first minimum = smallest magnitude among ties
    return order[pick].astype(np.uint8)


# ----------------------------------------------------------------------------------------
# Strided Dual-Exchange (Section 3.3, Theorem 1)
# ----------------------------------------------------------------------------------------
def pair_table(s: int):
    """P_s: the disjoint pairs (i, i XOR s) with i < i XOR s, ascending in i."""
    return [(i, i ^ s) for i in range(MICRO) if i < (i ^ s)]


def dual_exchange(x: np.ndarray, s: int, eta) -> np.ndarray:
    """Apply the signed exchange of pattern s with pair signs eta (4 values of +-1) to x[..., 8]."""
    x = np.asarray(x, dtype=np.float64)
    y = np.zeros_like(x)
    for p, (i, j) in enumerate(pair_table(s)):
        e = np.asarray(eta)[..., p]
        y[..., i] = -e * x[..., j]
        y[..., j] = e * x[..., i]
    return y


def meta_fields(meta: np.ndarray):
    """Split record bytes into (s in 1..4, eta[..., 4] in {+1,-1})."""
    meta = np.asarray(meta, dtype=np.uint8)
    s = (meta & 3).astype(np.int64) + 1
    flags = (meta[..., None] >> (2 + np.arange(4))) & 1
    eta = np.where(flags == 1, -1.0, 1.0)
    return s, eta


# ----------------------------------------------------------------------------------------
# Decode (Sections 3.1, 3.3)
# ----------------------------------------------------------------------------------------
def decode_b1(codes: np.ndarray, wbits: int) -> np.ndarray:
    return lattice_values(wbits)[np.asarray(codes, dtype=np.int64)]


def decode_b2(codes: np.ndarray, meta: np.ndarray, wbits: int) -> np.ndarray:
    """b2[n, k]: the recorded exchange applied to b1 inside every micro-block."""
    b1 = decode_b1(codes, wbits)
    n, k = b1.shape
    x = b1.reshape(n, k // MICRO, MICRO)
    s, eta = meta_fields(meta)
    y = np.zeros_like(x)
    for pat in (1, 2, 3, 4):
        sel = s == pat
        if not sel.any():
            continue
        y[sel] = dual_exchange(x[sel], pat, eta[sel])
    return y.reshape(n, k) + 0.0  # +0.0 turns -0.0 into +0.0


def coef_to_f64(coef_f16: np.ndarray) -> np.ndarray:
    return np.asarray(coef_f16, dtype=np.float16).astype(np.float64)


def reconstruct(codes, meta, coef_f16, group: int, wbits: int) -> np.ndarray:
    """W_hat[n, k] = c1[n, j] * b1[n, k] + c2[n, j] * b2[n, k], j = k // group (Section 3.1)."""
    b1 = decode_b1(codes, wbits)
    b2 = decode_b2(codes, meta, wbits)
    c = coef_to_f64(coef_f16)
    c1 = np.repeat(c[..., 0], group, axis=1)
    c2 = np.repeat(c[..., 1], group, axis=1)
    return c1 * b1 + c2 * b2


# ----------------------------------------------------------------------------------------
# GEO quantizer (Sections 3.2 - 3.4)
# ----------------------------------------------------------------------------------------
def quantize_geo(w: np.ndarray, group: int, wbits: int, return_aux: bool = False,
                 row_chunk: int = 256):
    """Quantize W [N][K] (macro-blocks of `group` consecutive k inside a row).

    Returns codes u8 [N][K], meta u8 [N][K/8], coef fp16 [N][K/group][2].
    With return_aux also a dict of the unrounded float64 c1, c2 and the alignment scores.
    """
    w = np.asarray(w)
    if not np.all(np.isfinite(w)):
        raise ValueError("weights must be finite")
    n, k = w.shape
    if k % group or group % MICRO:
        raise ValueError("K must be a multiple of group and group a multiple of 8")
    codes = np.empty((n, k), dtype=np.uint8)
    meta = np.empty((n, k // MICRO), dtype=np.uint8)
    c_all = np.empty((n, k // group, 2), dtype=np.float64)
    a_best = np.empty((n, k // MICRO), dtype=np.float64)
    for r0 in range(0, n, row_chunk):
        r1 = min(n, r0 + row_chunk)
        cd, mt, cc, ab = _quantize_rows(w[r0:r1].astype(np.float64), group, wbits)
        codes[r0:r1], meta[r0:r1], c_all[r0:r1], a_best[r0:r1] = cd, mt, cc, ab
    coef = c_all.astype(np.float16)
    if return_aux:
        return codes, meta, coef, {"c": c_all, "alignment": a_best}
    return codes, meta, coef


def _quantize_rows(w: np.ndarray, group: int, wbits: int):
    n, k = w.shape
    nj = k // group
    nt = group // MICRO
    wg = w.reshape(n, nj, group)
    emax = emax_of(wbits)

    # Section 3.2: s_norm = ||w||_inf, v = w / s_norm, b1 = Q(v).
    s_norm = np.max(np.abs(wg), axis=-1, keepdims=True)
    zero_blk = s_norm[..., 0] == 0.0
    v = wg / np.where(s_norm == 0.0, 1.0, s_norm)
    codes = rtn_codes(v, wbits)
    codes[zero_blk] = emax  # the zero code
    b1 = lattice_values(wbits)[codes]

    # Eq. 1: r = w - (<w, b1> / ||b1||^2) b1, with the zero-norm bypass.
    nb1 = np.sum(b1 * b1, axis=-1)
    safe = np.where(nb1 == 0.0, 1.0, nb1)
    c1 = np.where(nb1 == 0.0, 0.0, np.sum(wg * b1, axis=-1) / safe)
    r = wg - c1[..., None] * b1

    # Section 3.3 steps 1-2 per micro-block: d = x_i r_j - x_j r_i, eta* = sgn d, A_s = sum |d|.
    x = b1.reshape(n, nj, nt, MICRO)
    rho = r.reshape(n, nj, nt, MICRO)
    a_s = np.empty((4,) + x.shape[:-1], dtype=np.float64)
    d_s = np.empty((4,) + x.shape[:-1] + (4,), dtype=np.float64)
    for s in (1, 2, 3, 4):
        for p, (i, j) in enumerate(pair_table(s)):
            d_s[s - 1, ..., p] = x[..., i] * rho[..., j] - x[..., j] * rho[..., i]
        a_s[s - 1] = np.sum(np.abs(d_s[s - 1]), axis=-1)
    s_star = np.argmax(a_s, axis=0)  # first maximiser; value is s - 1
    d_star = np.take_along_axis(d_s, s_star[None, ..., None], axis=0)[0]
    a_star = np.take_along_axis(a_s, s_star[None], axis=0)[0]
    flags = (d_star < 0.0).astype(np.uint8)  # eta = -1 iff d < 0
    meta = s_star.astype(np.uint8)
    for p in range(4):
        meta |= flags[..., p] << (2 + p)
    meta[zero_blk] = 0

    # Step 3: assemble b2 from the recorded exchanges.
    eta = np.where(flags == 1, -1.0, 1.0)
    y = np.zeros_like(x)
    for s in (1, 2, 3, 4):
        sel = s_star == (s - 1)
        if sel.any():
            y[sel] = dual_exchange(x[sel], s, eta[sel])
    b2 = y.reshape(n, nj, group)

    # Eq. 2 (diagonal normal equations): c2 = <w, b2> / ||b2||^2.
    nb2 = np.sum(b2 * b2, axis=-1)
    safe2 = np.where(nb2 == 0.0, 1.0, nb2)
    c2 = np.where(nb2 == 0.0, 0.0, np.sum(wg * b2, axis=-1) / safe2)

    c = np.stack([c1, c2], axis=-1)
    return (codes.reshape(n, k), meta.reshape(n, k // MICRO), c, a_star.reshape(n, k // MICRO))


# ----------------------------------------------------------------------------------------
# Single-basis form (Section 3.1: w_hat = c1 b1) and REF-mode coefficients (Section 3.4, Eq. 3)
# ----------------------------------------------------------------------------------------
def quantize_k1(w: np.ndarray, group: int, wbits: int):
    """K = 1: b1 = Q(w / ||w||_inf) (Section 3.2) and c1 = <w, b1> / ||b1||^2, the least-squares scale of
    w_hat = c1 b1 (Section 3.1). Returned in the dual-basis format with an empty second basis:
    record bytes 0 and c2 = 0, so every consumer of (codes, meta, coef) evaluates c1 b1."""
    w = np.asarray(w, dtype=np.float64)
    if not np.all(np.isfinite(w)):
        raise ValueError("weights must be finite")
    n, k = w.shape
    if k % group or group % MICRO:
        raise ValueError("K must be a multiple of group and group a multiple of 8")
    wg = w.reshape(n, k // group, group)
    s_norm = np.max(np.abs(wg), axis=-1, keepdims=True)
    v = wg / np.where(s_norm == 0.0, 1.0, s_norm)
    codes = rtn_codes(v, wbits)
    codes[s_norm[..., 0] == 0.0] = emax_of(wbits)
    b1 = lattice_values(wbits)[codes]
    nb1 = np.sum(b1 * b1, axis=-1)
    c1 = np.where(nb1 == 0.0, 0.0, np.sum(wg * b1, axis=-1) / np.where(nb1 == 0.0, 1.0, nb1))
    coef = np.stack([c1, np.zeros_like(c1)], axis=-1).astype(np.float16)
    return codes.reshape(n, k), np.zeros((n, k // MICRO), dtype=np.uint8), coef


def solve_ref(w: np.ndarray, codes, meta, x_calib: np.ndarray, group: int, wbits: int, lam: float = 1e-4) -> np.ndarray:
    """REF mode (Eq. 3). For every row n and macro-block j, with X_q = x_calib[:, j*g:(j+1)*g] (M observations),
    A = [X_q b1, X_q b2] (M x 2), Y = X_q w:  c* = (A^T A + lam I)^-1 A^T Y.  Returns float64 [N][K/g][2]."""
    w = np.asarray(w, dtype=np.float64)
    x = np.asarray(x_calib, dtype=np.float64)
    n, k = w.shape
    nj = k // group
    b1 = decode_b1(codes, wbits)
    b2 = decode_b2(codes, meta, wbits)
    out = np.empty((n, nj, 2), dtype=np.float64)
    for j in range(nj):
        xq = x[:, j * group:(j + 1) * group]                      # M x g
        y = xq @ w[:, j * group:(j + 1) * group].T                # M x N : column n is X_q w_n
        a1 = xq @ b1[:, j * group:(j + 1) * group].T              # M x N : X_q b1
        a2 = xq @ b2[:, j * group:(j + 1) * group].T
        for r in range(n):
            a = np.stack([a1[:, r], a2[:, r]], axis=1)            # M x 2
            out[r, j] = np.linalg.solve(a.T @ a + lam * np.eye(2), a.T @ y[:, r])
    return out


# ----------------------------------------------------------------------------------------
# Reference linear layer, float activations (Section 3.5, Eq. 4)
# ----------------------------------------------------------------------------------------
def linear_f64(codes, meta, coef_f16, x: np.ndarray, group: int, wbits: int, rows=None) -> np.ndarray:
    """y[m, n] = sum_j ( c1[n,j] * sum_{k in j} b1[n,k] x[m,k] + c2[n,j] * sum_{k in j} b2[n,k] x[m,k] ).

    x is float64 [M][K] (the bf16 inputs widened exactly). `rows` restricts the output channels.
    """
    if rows is not None:
        codes, meta, coef_f16 = codes[rows], meta[rows], coef_f16[rows]
    b1 = decode_b1(codes, wbits)
    b2 = decode_b2(codes, meta, wbits)
    c = coef_to_f64(coef_f16)
    x = np.asarray(x, dtype=np.float64)
    m, k = x.shape
    y = np.zeros((m, codes.shape[0]), dtype=np.float64)
    for j in range(k // group):
        sl = slice(j * group, (j + 1) * group)
        s1 = x[:, sl] @ b1[:, sl].T
        s2 = x[:, sl] @ b2[:, sl].T
        y += s1 * c[None, :, j, 0] + s2 * c[None, :, j, 1]
    return y


def linear_f64_loops(codes, meta, coef_f16, x, group: int, wbits: int) -> np.ndarray:
    """The same sum written with scalar Python loops (tiny inputs only)."""
    b1 = decode_b1(codes, wbits)
    b2 = decode_b2(codes, meta, wbits)
    c = coef_to_f64(coef_f16)
    m, k = x.shape
    n = codes.shape[0]
    y = np.zeros((m, n))
    for mi in range(m):
        for ni in range(n):
            tot = 0.0
            for j in range(k // group):
                s1 = 0.0
                s2 = 0.0
                for kk in range(j * group, (j + 1) * group):
                    s1 += b1[ni, kk] * float(x[mi, kk])
                    s2 += b2[ni, kk] * float(x[mi, kk])
                tot += c[ni, j, 0] * s1 + c[ni, j, 1] * s2
            y[mi, ni] = tot
    return y


# ----------------------------------------------------------------------------------------
# Integer path (Section 3.5, Eq. 4 with integer activations and coefficients)
# ----------------------------------------------------------------------------------------
def _rne(x):
    return np.rint(x)  # numpy rounds half to even


def quantize_activations_int8(x: np.ndarray):
    """Per-token symmetric int8: s_x[m] = max_k |x[m,k]| / 127, x~ = clamp(rne(x / s_x), +-127)."""
    x = np.asarray(x, dtype=np.float64)
    amax = np.max(np.abs(x), axis=1)
    sx = np.where(amax == 0.0, 1.0, amax / 127.0)
    xq = np.clip(_rne(x / sx[:, None]), -127, 127).astype(np.int8)
    return xq, sx.astype(np.float32)


def quantize_activations_int(x: np.ndarray, bits: int):
    """Per-token symmetric b_a-bit integers in int8 containers (Section 3.5's b_a; the A4 / A6 settings of the accuracy
    tables): q_max = 2^(bits-1) - 1, s_x[m] = max_k |x[m,k]| / q_max, x~ = clamp(rne(x / s_x), +-q_max)."""
    if not 2 <= bits <= 8:
        raise ValueError("bits must be in 2..8")
    qmax = float((1 << (bits - 1)) - 1)
    x = np.asarray(x, dtype=np.float64)
    amax = np.max(np.abs(x), axis=1)
    sx = np.where(amax == 0.0, 1.0, amax / qmax)
    xq = np.clip(_rne(x / sx[:, None]), -qmax, qmax).astype(np.int8)
    return xq, sx.astype(np.float32)


def quantize_coefficients_int8(coef_f16: np.ndarray):
    """Per-output-channel, per-basis symmetric int8 of the fp16 coefficients.

    Returns cq int8 [N][J][2] and sc fp32 [N][2] with c ~= sc * cq.
    """
    c = coef_to_f64(coef_f16)
    amax = np.max(np.abs(c), axis=1)  # [N][2]
    sc = np.where(amax == 0.0, 1.0, amax / 127.0)
    cq = np.clip(_rne(c / sc[:, None, :]), -127, 127).astype(np.int8)
    return cq, sc.astype(np.float32)


def int_weights(codes, meta, wbits: int):
    """Integer operands B1int, B2int = 2^emax * b1, 2^emax * b2 (each +-2^(emax-e) or 0)."""
    scale = float(1 << emax_of(wbits))
    b1 = decode_b1(codes, wbits) * scale
    b2 = decode_b2(codes, meta, wbits) * scale
    b1i = b1.astype(np.int64)
    b2i = b2.astype(np.int64)
    assert np.array_equal(b1i, b1) and np.array_equal(b2i, b2)
    return b1i, b2i


def linear_i32(codes, meta, cq, sc, xq, sx, group: int, wbits: int, rows=None, return_groups=False):
    """Exact integer evaluation.

    S1[m,j,n] = sum_{k in j} x~[m,k] * B1int[n,k]   (a shift-and-add: +-(x~ << (emax - e)))
    ACC1[m,n] = sum_j c~1[n,j] * S1[m,j,n]          (same for the second basis)
    y[m,n]    = s_x[m] * 2^-emax * ( s_c1[n] * ACC1 + s_c2[n] * ACC2 )

    Returns (ACC1 int32 [M][N], ACC2 int32 [M][N], y float64 [M][N]) and, on request, the
    per-group sums S1, S2 as int64 [J][M][N]. Raises if an accumulator leaves int32.
    """
    if rows is not None:
        codes, meta, cq, sc = codes[rows], meta[rows], cq[rows], sc[rows]
    b1i, b2i = int_weights(codes, meta, wbits)
    xq = np.asarray(xq)
    m, k = xq.shape
    n = codes.shape[0]
    nj = k // group
    xf = xq.astype(np.float64)  # every product and sum below is far under 2^53: float64 is exact
    acc1 = np.zeros((m, n), dtype=np.int64)
    acc2 = np.zeros((m, n), dtype=np.int64)
    s_keep = ([], [])
    cq64 = np.asarray(cq, dtype=np.int64)
    for j in range(nj):
        sl = slice(j * group, (j + 1) * group)
        s1 = (xf[:, sl] @ b1i[:, sl].T.astype(np.float64)).astype(np.int64)
        s2 = (xf[:, sl] @ b2i[:, sl].T.astype(np.float64)).astype(np.int64)
        if np.abs(s1).max(initial=0) >= 2 ** 31 or np.abs(s2).max(initial=0) >= 2 ** 31:
            raise OverflowError("group sum leaves int32")
        acc1 += s1 * cq64[None, :, j, 0]
        acc2 += s2 * cq64[None, :, j, 1]
        if return_groups:
            s_keep[0].append(s1)
            s_keep[1].append(s2)
        if np.abs(acc1).max(initial=0) >= 2 ** 31 or np.abs(acc2).max(initial=0) >= 2 ** 31:
            raise OverflowError("accumulator leaves int32")
    sc64 = np.asarray(sc, dtype=np.float64)
    sx64 = np.asarray(sx, dtype=np.float64)
    y = sx64[:, None] * 2.0 ** (-emax_of(wbits)) * (sc64[None, :, 0] * acc1 + sc64[None, :, 1] * acc2)
    out = (acc1.astype(np.int32), acc2.astype(np.int32), y)
    if return_groups:
        return out + (np.stack(s_keep[0]), np.stack(s_keep[1]))
    return out


def linear_i32_loops(codes, meta, cq, xq, group: int, wbits: int):
    """ACC1, ACC2 with Python integers and explicit shifts (tiny inputs only)."""
    emax = emax_of(wbits)
    n, k = codes.shape
    m = xq.shape[0]
    s_fld, eta = meta_fields(meta)
    acc1 = [[0] * n for _ in range(m)]
    acc2 = [[0] * n for _ in range(m)]
    for ni in range(n):
        # integer (sign, shift) pairs of b1 and b2; shift None means the zero state
        t1 = []
        for kk in range(k):
            c = int(codes[ni, kk])
            sign = c >> (wbits - 1)
            e = c & emax
            t1.append((0, None) if (sign == 0 and e == emax) else (sign, emax - e))
        t2 = [None] * k
        for t in range(k // MICRO):
            for p, (i, j) in enumerate(pair_table(int(s_fld[ni, t]))):
                neg = 1 if eta[ni, t, p] < 0 else 0
                si, shi = t1[t * MICRO + i]
                sj, shj = t1[t * MICRO + j]
                t2[t * MICRO + i] = (sj ^ 1 ^ neg, shj)  # y_i = -eta x_j
                t2[t * MICRO + j] = (si ^ neg, shi)      # y_j =  eta x_i
        for mi in range(m):
            for jg in range(k // group):
                s1 = 0
                s2 = 0
                for kk in range(jg * group, (jg + 1) * group):
                    xv = int(xq[mi, kk])
                    sg, sh = t1[kk]
                    if sh is not None:
                        s1 += -(xv << sh) if sg else (xv << sh)
                    sg, sh = t2[kk]
                    if sh is not None:
                        s2 += -(xv << sh) if sg else (xv << sh)
                acc1[mi][ni] += int(cq[ni, jg, 0]) * s1
                acc2[mi][ni] += int(cq[ni, jg, 1]) * s2
    return np.array(acc1, dtype=np.int64), np.array(acc2, dtype=np.int64)


# ----------------------------------------------------------------------------------------
# Error measures used by the parity tests
# ----------------------------------------------------------------------------------------
def normwise_rel_err(y: np.ndarray, y_ref: np.ndarray) -> float:
    """max over batch rows of ||y[m] - y_ref[m]||_2 / ||y_ref[m]||_2."""
    y = np.asarray(y, dtype=np.float64)
    num = np.linalg.norm(y - y_ref, axis=1)
    den = np.linalg.norm(y_ref, axis=1)
    return float(np.max(num / np.where(den == 0.0, 1.0, den)))
