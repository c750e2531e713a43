"""goq_gemv_sequence: a chain of decode GEMVs in one persistent kernel, against the CPU oracle."""
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


def _layer(goq, n, k, g, b, seed):
    from tests.gpu_util import pack_weights
    codes, meta, coef = si.random_quantized(n, k, g, b, seed=seed)
    d, packed = pack_weights(n, k, g, b, codes, meta, coef)
    return dict(n=n, k=k, g=g, b=b, codes=codes, meta=meta, coef=coef, d=d, packed=packed)


def _ws(goq, n_items):
    ws = torch.empty(goq.sequence_workspace_bytes(n_items), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws)
    return ws


@pytest.fixture
def form(goq):
    """Automatic kernel choice (the chain kernel has one arithmetic form: integer operands)."""
    prev = goq.set_gemv_variant(0)
    yield 0
    goq.set_gemv_variant(prev)


@pytest.mark.parametrize("flagged,batch", [(True, 3), (False, 3), (False, 1), (False, 4), (False, 6)])
def test_chain_with_real_dependencies_matches_oracle_stage_by_stage(goq, form, flagged, batch):
    """y0 = W0 x0 (bf16 out) feeds W1, whose bf16 output feeds W2: every stage is checked against the oracle
    evaluated on the bits the previous stage actually produced. Flagged items wait for the completion counter;
    unflagged ones are ordered by the library from the address ranges (they poll the producer's tagged copy)."""
    from tests.gpu_util import dev
    shapes = [(256, 384), (512, 256), (130, 512)]   # (n_out, k_in): n_out of one = k_in of the next
    layers = [_layer(goq, n, k, 64, 3, seed=40 + i) for i, (n, k) in enumerate(shapes)]
    x0 = si.bf16_activations(batch, shapes[0][1], seed=5)
    bufs = [dev(x0)] + [torch.zeros((batch, n), dtype=torch.bfloat16, device="cuda") for n, _ in shapes[:-1]]
    y_last = torch.zeros((batch, shapes[-1][0]), dtype=torch.float32, device="cuda")
    outs = bufs[1:] + [y_last]
    items = [(L["d"], L["packed"], bufs[i], batch, outs[i], goq.BF16 if i < 2 else goq.F32, flagged and i > 0)
             for i, L in enumerate(layers)]
    seq = goq.make_sequence(items)
    ws = _ws(goq, len(items))
    for _ in range(2):   # the scratch is left clean: a second call needs no re-initialisation
        goq.gemv_sequence(seq, ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        x_bits = x0
        for i, L in enumerate(layers):
            y_ref = O.linear_f64(L["codes"], L["meta"], L["coef"], si.bf16_bits_to_f64(x_bits), L["g"], L["b"])
            got = outs[i].float().cpu().numpy().astype(np.float64)
            if i == 2:
                assert O.normwise_rel_err(got, y_ref) <= TIGHT, (i, O.normwise_rel_err(got, y_ref))
            else:   # bf16 outputs carry one extra rounding: held to it element by element
                from tests.gpu_util import check_bf16_output
                check_bf16_output(got, y_ref, 1e-4, "stage %d" % i)
            if i < 2:
                x_bits = outs[i].view(torch.int16).cpu().numpy().view(np.uint16)


def _check_item(L, x_bits, out, bf16_out, what):
    """One item against the oracle evaluated on the activation bits it was given."""
    from tests.gpu_util import check_bf16_output
    y_ref = O.linear_f64(L["codes"], L["meta"], L["coef"], si.bf16_bits_to_f64(x_bits), L["g"], L["b"])
    got = out.float().cpu().numpy().astype(np.float64)
    if bf16_out:
        check_bf16_output(got, y_ref, 1e-4, what)
    else:
        assert O.normwise_rel_err(got, y_ref) <= TIGHT, (what, O.normwise_rel_err(got, y_ref))


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def test_data_flow_slices_fan_out_and_a_producer_two_items_back(goq, form):
    """Unflagged items ordered by address ranges alone (batch 1): item 1 and item 2 read two different slices of item
    0's bf16 output (channel counts that are no multiple of a tile), item 3 reads item 1's output although item 2 lies
    between them, item 4 reads all of item 2's. Run twice on one scratch buffer, with a producer wide enough to be
    spread over every SM, so that readers really wait for tiles finished elsewhere."""
    from tests.gpu_util import dev
    L0 = _layer(goq, 4104, 512, 32, 3, seed=700)       # 256.5 tiles: the last one is half empty
    L1 = _layer(goq, 416, 2048, 32, 3, seed=701)        # reads y0[0:2048]
    L2 = _layer(goq, 544, 1024, 32, 3, seed=702)        # reads y0[3072:4096]
    L3 = _layer(goq, 100, 416, 32, 3, seed=703)         # reads y1 (416 channels: k padded to 512)
    L4 = _layer(goq, 64, 544, 32, 3, seed=704)          # reads y2
    x0 = si.bf16_activations(1, 512, seed=70)
    y0 = torch.zeros((1, 4104), dtype=torch.bfloat16, device="cuda")
    y1 = torch.zeros((1, 416), dtype=torch.bfloat16, device="cuda")
    y2 = torch.zeros((1, 544), dtype=torch.bfloat16, device="cuda")
    y3 = torch.zeros((1, 100), dtype=torch.float32, device="cuda")
    y4 = torch.zeros((1, 64), dtype=torch.bfloat16, device="cuda")
    items = [(L0["d"], L0["packed"], dev(x0), 1, y0, goq.BF16, False),
             (L1["d"], L1["packed"], y0[:, 0:2048], 1, y1, goq.BF16, False),
             (L2["d"], L2["packed"], y0[:, 3072:4096], 1, y2, goq.BF16, False),
             (L3["d"], L3["packed"], y1, 1, y3, goq.F32, False),
             (L4["d"], L4["packed"], y2, 1, y4, goq.BF16, False)]
    keep = [t[2] for t in items]
    seq = goq.make_sequence(items)
    ws = _ws(goq, len(items))
    for rep in range(2):
        for y in (y0, y1, y2, y3, y4):
            y.zero_()
        goq.gemv_sequence(seq, ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        b0 = _bits(y0)
        _check_item(L0, x0, y0, True, "item 0")
        _check_item(L1, b0[:, 0:2048], y1, True, "item 1")
        _check_item(L2, b0[:, 3072:4096], y2, True, "item 2")
        _check_item(L3, _bits(y1), y3, False, "item 3")
        _check_item(L4, _bits(y2), y4, True, "item 4")
    del keep


def test_overlaps_the_tagged_copy_cannot_serve_fall_back_to_the_counter_wait(goq, form):
    """Unflagged items whose buffers overlap earlier ones in ways the word-by-word wait does not cover are still ordered
    correctly: item 2 reads one buffer that items 0 and 1 each wrote half of (two producers), item 3 writes where item 0
    wrote after item 2 has read it (an output buffer used twice)."""
    from tests.gpu_util import dev
    La = _layer(goq, 512, 256, 64, 3, seed=710)
    Lb = _layer(goq, 512, 256, 64, 3, seed=711)
    Lc = _layer(goq, 256, 1024, 64, 3, seed=712)
    Ld = _layer(goq, 512, 256, 64, 3, seed=713)
    x0 = si.bf16_activations(1, 256, seed=71)
    xd = dev(x0)
    P = torch.zeros((1, 1024), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda")
    items = [(La["d"], La["packed"], xd, 1, P[:, 0:512], goq.BF16, False),
             (Lb["d"], Lb["packed"], xd, 1, P[:, 512:1024], goq.BF16, False),
             (Lc["d"], Lc["packed"], P, 1, B, goq.BF16, False),
             (Ld["d"], Ld["packed"], B, 1, P[:, 0:512], goq.BF16, False)]
    keep = [t[4] for t in items]
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    # P[0:512] now holds item 3's result; item 0's is recomputed on its own (the kernel is deterministic)
    P0 = torch.zeros((1, 512), dtype=torch.bfloat16, device="cuda")
    goq.gemv_sequence(goq.make_sequence([(La["d"], La["packed"], xd, 1, P0, goq.BF16, False)]), _ws(goq, 1))
    torch.cuda.synchronize()
    _check_item(La, x0, P0, True, "item 0")
    _check_item(Lb, x0, P[:, 512:1024].contiguous(), True, "item 1")
    p_bits = np.concatenate([_bits(P0), _bits(P[:, 512:1024].contiguous())], axis=1)
    _check_item(Lc, p_bits, B, True, "item 2")
    _check_item(Ld, _bits(B), P[:, 0:512].contiguous(), True, "item 3")
    del keep


def test_a_data_flow_wait_that_runs_out_reports_timeout(goq):
    """The word-by-word wait is bounded like every other: with a bound of one poll a reader gives up before the producer's
    tiles are there, the launch ends by itself with GOQ_ERR_TIMEOUT, and after a zero-fill the chain runs correctly."""
    from tests.gpu_util import dev
    La, Lb = _layer(goq, 2048, 2048, 128, 3, seed=601), _layer(goq, 512, 2048, 128, 3, seed=602)
    xa = si.bf16_activations(1, 2048, seed=31)
    mid = torch.zeros((1, 2048), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 512), dtype=torch.float32, device="cuda")
    xd = dev(xa)
    seq = goq.make_sequence([(La["d"], La["packed"], xd, 1, mid, goq.BF16, False), (Lb["d"], Lb["packed"], mid, 1, y, goq.F32, False)])
    ws = _ws(goq, 2)
    prev = goq.set_wait_limit(1)
    try:
        goq.gemv_sequence(seq, ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.ERR_TIMEOUT
    finally:
        goq.set_wait_limit(prev)
    goq.workspace_init(ws)
    goq.gemv_sequence(seq, ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    _check_item(Lb, _bits(mid), y, False, "second linear")


@pytest.mark.parametrize("g,b", [(128, 3), (32, 2)])
def test_independent_items_of_mixed_shapes(goq, g, b, form):
    """Ragged rows and k, fewer and more than 16 k-blocks per tile, batch 1..8, both output types."""
    from tests.gpu_util import dev
    shapes = [(40, 256, 1), (300, 4224, 2), (16, 128, 8), (1000, 1152, 5), (257, 2048 + 128, 3)]
    layers, xs, ys, items = [], [], [], []
    for i, (n, k, m) in enumerate(shapes):
        L = _layer(goq, n, k, g, b, seed=90 + i)
        xb = si.bf16_activations(m, k, seed=60 + i)
        y = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        layers.append(L); xs.append(xb); ys.append(y)
        items.append((L["d"], L["packed"], dev(xb), m, y, goq.F32, False))
    keep = [it[2] for it in items]
    seq = goq.make_sequence(items)
    ws = _ws(goq, len(items))
    goq.gemv_sequence(seq, ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    first = [y.clone() for y in ys]
    for L, xb, y in zip(layers, xs, ys):
        y_ref = O.linear_f64(L["codes"], L["meta"], L["coef"], si.bf16_bits_to_f64(xb), g, b)
        from tests.gpu_util import check_parity
        check_parity(y.cpu().numpy(), y_ref, TIGHT, 1e-4)
    goq.gemv_sequence(seq, ws)
    torch.cuda.synchronize()
    for a, y in zip(first, ys):
        assert torch.equal(a, y)   # same sums in the same order: bit-identical
    del keep


@pytest.mark.parametrize("g,b", [(128, 3), (64, 2)])
def test_small_batches_integer_operand_form(goq, g, b, form):
    """Every item has batch <= 4, so the automatic choice is the integer-operand form; extreme activations included."""
    from tests.gpu_util import dev
    shapes = [(40, 256, 1), (300, 4224, 2), (16, 128, 4), (1000, 1152, 3), (257, 2048 + 128, 1)]
    keep, checks, items = [], [], []
    for i, (n, k, m) in enumerate(shapes):
        L = _layer(goq, n, k, g, b, seed=190 + i)
        x = si.bf16_bits_to_f64(si.bf16_activations(m, k, seed=160 + i))
        if i == 1:
            x[0, ::3] = 0.0
            x[0, 1::7] *= 2.0 ** -60
            x[1, ::5] *= 2.0 ** 40
        xb = si.f32_to_bf16_bits(x.astype(np.float32))
        y = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        xd = dev(xb)
        keep.append(xd)
        items.append((L["d"], L["packed"], xd, m, y, goq.F32, False))
        checks.append((L, xb, y))
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    for L, xb, y in checks:
        y_ref = O.linear_f64(L["codes"], L["meta"], L["coef"], si.bf16_bits_to_f64(xb), g, b)
        err = O.normwise_rel_err(y.cpu().numpy().astype(np.float64), y_ref)
        print("sequence form %d: normwise error %.3e" % (form, err))
        assert err <= TIGHT, err


@pytest.mark.parametrize("shapes", [
    [(64, 4224, 4), (48, 11008, 3), (300, 256, 1)],      # batch <= 4: integer form unless bf16 operands are forced
    [(32, 4096, 8), (500, 2304, 7), (40, 128, 2)],       # batch up to 8: bf16 operands
])
def test_activations_beyond_the_two_cta_buffer(goq, shapes, form):
    """Batches and widths whose staged activations exceed the buffer that leaves room for two CTAs per SM run
    with a buffer sized for the launch and one CTA per SM; a dependent chain inside exercises the counters."""
    from tests.gpu_util import dev
    keep, checks, items = [], [], []
    for i, (n, k, m) in enumerate(shapes):
        L = _layer(goq, n, k, 128, 3, seed=290 + i)
        xb = si.bf16_activations(m, k, seed=260 + i)
        y = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        xd = dev(xb)
        keep.append(xd)
        items.append((L["d"], L["packed"], xd, m, y, goq.F32, i > 0))
        checks.append((L, xb, y))
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    for L, xb, y in checks:
        y_ref = O.linear_f64(L["codes"], L["meta"], L["coef"], si.bf16_bits_to_f64(xb), 128, 3)
        assert O.normwise_rel_err(y.cpu().numpy().astype(np.float64), y_ref) <= TIGHT
    del keep


def test_one_7b_shaped_layer_sampled_rows(goq, form):
    from tests.gpu_util import dev
    items, checks = [], []
    for i, (name, n, k) in enumerate(si.LLAMA2_7B_LINEARS):
        codes, meta, coef = si.random_quantized(n, k, 128, 3, seed=300 + i)
        rows = si.sample_rows(n, 32, seed=i)
        w = si.weights_with_outlier_channels(len(rows), k, seed=i)
        codes[rows], meta[rows], coef[rows] = O.quantize_geo(w, 128, 3)
        from tests.gpu_util import pack_weights
        d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
        xb = si.bf16_activations(1, k, seed=200 + i)
        y = torch.zeros((1, n), dtype=torch.float32, device="cuda")
        items.append((d, packed, dev(xb), 1, y, goq.F32, True))
        checks.append((codes, meta, coef, xb, rows, y))
    seq = goq.make_sequence(items)
    ws = _ws(goq, len(items))
    goq.gemv_sequence(seq, ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    for codes, meta, coef, xb, rows, y in checks:
        y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), 128, 3, rows=rows)
        from tests.gpu_util import check_parity
        check_parity(y.cpu().numpy().astype(np.float64)[:, rows], y_ref, TIGHT, 1e-4)


def test_two_7b_shaped_layers_as_a_true_chain_sampled_rows(goq, form):
    """The launch configuration the benchmark times, at full size: 14 linears of the 7B shapes, each reading the first
    k channels of the previous linear's bf16 output (no item flagged: ordered by data flow), run three times on one
    scratch buffer. Every linear is checked on sampled rows against the oracle evaluated on the bits its producer
    actually wrote; repeated launches must reproduce the same bits (fixed summation order)."""
    from tests.gpu_util import dev, pack_weights, check_bf16_output
    layers, outs, items = [], [], []
    x0 = si.bf16_activations(1, 4096, seed=900)
    for j in range(14):
        name, n, k = si.LLAMA2_7B_LINEARS[j % 7]
        codes, meta, coef = si.random_quantized(n, k, 128, 3, seed=910 + j)
        coef = (coef.astype(np.float64) * (0.02 / 0.03) * (4096.0 / k) ** 0.5).astype(np.float16)   # about unit gain along the chain
        rows = si.sample_rows(n, 24, seed=j)
        d, packed = pack_weights(n, k, 128, 3, codes, meta, coef)
        y = torch.zeros((1, n), dtype=torch.bfloat16, device="cuda")
        x = dev(x0) if j == 0 else outs[j - 1][:, :k]
        items.append((d, packed, x, 1, y, goq.BF16, False))
        outs.append(y)
        layers.append((codes, meta, coef, rows, k))
    keep = [t[2] for t in items]
    seq = goq.make_sequence(items)
    ws = _ws(goq, len(items))
    first = None
    for rep in range(3):
        for y in outs:
            y.zero_()
        goq.gemv_sequence(seq, ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.OK
        bits = [_bits(y) for y in outs]
        if first is None:
            first = bits
            for j, (codes, meta, coef, rows, k) in enumerate(layers):
                x_bits = x0 if j == 0 else bits[j - 1][:, :k]
                y_ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(x_bits), 128, 3, rows=rows)
                check_bf16_output(si.bf16_bits_to_f64(bits[j])[:, rows], y_ref, 1e-4, "linear %d" % j)
            assert np.isfinite(si.bf16_bits_to_f64(bits[-1])).all() and np.abs(si.bf16_bits_to_f64(bits[-1])).max() > 0
        else:
            for j in range(14):
                assert np.array_equal(bits[j], first[j]), (rep, j)
    del keep


def test_unsupported_and_invalid_sequences_return_a_status(goq):
    from tests.gpu_util import dev
    L = _layer(goq, 64, 256, 64, 3, seed=1)
    L2 = _layer(goq, 64, 256, 128, 3, seed=2)
    ws = _ws(goq, 2)
    x9 = dev(si.bf16_activations(9, 256, seed=1))
    y9 = torch.zeros((9, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(goq.GoqError) as e:
        goq.gemv_sequence(goq.make_sequence([(L["d"], L["packed"], x9, 9, y9, goq.F32, False)]), ws)
    assert e.value.status == goq.ERR_UNSUPPORTED
    x1 = dev(si.bf16_activations(1, 256, seed=1))
    y1 = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    mixed = [(L["d"], L["packed"], x1, 1, y1, goq.F32, False), (L2["d"], L2["packed"], x1, 1, y1, goq.F32, True)]
    with pytest.raises(goq.GoqError) as e:
        goq.gemv_sequence(goq.make_sequence(mixed), ws)
    assert e.value.status == goq.ERR_UNSUPPORTED
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(goq.GoqError) as e:
        goq.gemv_sequence(goq.make_sequence(mixed[:1] * 2), small)
    assert e.value.status == goq.ERR_WORKSPACE


def test_a_wait_that_runs_out_reports_timeout_and_the_context_stays_usable(goq):
    """goq_set_wait_limit(1) bounds every device-side wait of the chain kernel to a single probe. In a dependent chain
    the first CTA to finish the first linear probes the completion counter before the other CTAs have reported, finds
    it short and gives up: the launch still ends by itself, the status word reads GOQ_ERR_TIMEOUT, nothing faults.
    After the scratch buffer is zero-filled again the same chain runs correctly."""
    from tests.gpu_util import dev
    La, Lb = _layer(goq, 2048, 2048, 128, 3, seed=601), _layer(goq, 512, 2048, 128, 3, seed=602)
    xa = si.bf16_activations(1, 2048, seed=31)
    mid = torch.zeros((1, 2048), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 512), dtype=torch.float32, device="cuda")
    xd = dev(xa)
    seq = goq.make_sequence([(La["d"], La["packed"], xd, 1, mid, goq.BF16, False), (Lb["d"], Lb["packed"], mid, 1, y, goq.F32, True)])
    ws = _ws(goq, 2)
    prev = goq.set_wait_limit(1)
    try:
        goq.gemv_sequence(seq, ws)
        torch.cuda.synchronize()
        assert goq.workspace_status(ws) == goq.ERR_TIMEOUT
    finally:
        goq.set_wait_limit(prev)
    goq.workspace_init(ws)
    goq.gemv_sequence(seq, ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    mid_bits = mid.view(torch.int16).cpu().numpy().view(np.uint16)
    ref = O.linear_f64(Lb["codes"], Lb["meta"], Lb["coef"], si.bf16_bits_to_f64(mid_bits), 128, 3)
    assert O.normwise_rel_err(y.cpu().numpy().astype(np.float64), ref) <= TIGHT


def test_host_block_entry_point(goq):
    """goq_gemv_sequence_host: activations in one pinned host block, outputs in another; a two-linear chain whose
    second item reads the first one's bf16 output inside the output block."""
    n0, k0, n1, m = 256, 384, 100, 2
    L0, L1 = _layer(goq, n0, k0, 64, 3, seed=11), _layer(goq, n1, n0, 64, 3, seed=12)
    xb = si.bf16_activations(m, k0, seed=9)
    x_bytes, y0_bytes, y1_bytes = m * k0 * 2, m * n0 * 2, m * n1 * 4
    x_stage = torch.zeros(x_bytes, dtype=torch.uint8, device="cuda")
    y_stage = torch.zeros(y0_bytes + y1_bytes, dtype=torch.uint8, device="cuda")
    x_host = torch.from_numpy(xb.view(np.uint8).reshape(-1).copy()).pin_memory()
    y_host = torch.zeros(y0_bytes + y1_bytes, dtype=torch.uint8).pin_memory()
    xv = x_stage.view(torch.bfloat16).view(m, k0)
    y0v = y_stage[:y0_bytes].view(torch.bfloat16).view(m, n0)
    y1v = y_stage[y0_bytes:].view(torch.float32).view(m, n1)
    seq = goq.make_sequence([(L0["d"], L0["packed"], xv, m, y0v, goq.BF16, False), (L1["d"], L1["packed"], y0v, m, y1v, goq.F32, True)])
    ws = _ws(goq, 2)
    goq.gemv_sequence_host(seq, x_host, x_stage, y_host, y_stage, ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    mid_bits = y_host[:y0_bytes].numpy().view(np.uint16).reshape(m, n0)
    y0_ref = O.linear_f64(L0["codes"], L0["meta"], L0["coef"], si.bf16_bits_to_f64(xb), 64, 3)
    from tests.gpu_util import check_bf16_output
    check_bf16_output(si.bf16_bits_to_f64(mid_bits), y0_ref, 1e-4)
    y1 = y_host[y0_bytes:].numpy().view(np.float32).reshape(m, n1).astype(np.float64)
    y1_ref = O.linear_f64(L1["codes"], L1["meta"], L1["coef"], si.bf16_bits_to_f64(mid_bits), 64, 3)
    assert O.normwise_rel_err(y1, y1_ref) <= TIGHT
    # an item whose buffers lie outside the blocks is refused on the host
    stray = torch.zeros((m, n1), dtype=torch.float32, device="cuda")
    bad = goq.make_sequence([(L0["d"], L0["packed"], xv, m, y0v, goq.BF16, False), (L1["d"], L1["packed"], y0v, m, stray, goq.F32, True)])
    with pytest.raises(goq.GoqError) as e:
        goq.gemv_sequence_host(bad, x_host, x_stage, y_host, y_stage, ws)
    assert e.value.status == goq.ERR_INVALID_ARG


def test_long_sequence_is_split_into_launches_and_small_grids_work(goq, form):
    """300 items (more than one launch holds) over two tiny layers: 8 row tiles in all per launch chunk would leave most
    CTAs without work, so the grid shrinks to the tile count; every item is checked."""
    from tests.gpu_util import dev
    La, Lb = _layer(goq, 48, 128, 64, 3, seed=501), _layer(goq, 80, 256, 64, 3, seed=502)
    xa, xb_ = si.bf16_activations(2, 128, seed=21), si.bf16_activations(2, 256, seed=22)
    xad, xbd = dev(xa), dev(xb_)
    ys, items = [], []
    for i in range(300):
        L, x, k = (La, xad, 128) if i % 2 == 0 else (Lb, xbd, 256)
        y = torch.full((2, L["n"]), float("nan"), dtype=torch.float32, device="cuda")
        ys.append(y)
        items.append((L["d"], L["packed"], x, 2, y, goq.F32, i % 3 != 0))
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    ref_a = O.linear_f64(La["codes"], La["meta"], La["coef"], si.bf16_bits_to_f64(xa), 64, 3)
    ref_b = O.linear_f64(Lb["codes"], Lb["meta"], Lb["coef"], si.bf16_bits_to_f64(xb_), 64, 3)
    for i, y in enumerate(ys):
        ref = ref_a if i % 2 == 0 else ref_b
        assert O.normwise_rel_err(y.cpu().numpy().astype(np.float64), ref) <= TIGHT, i
    assert torch.equal(ys[0], ys[298]) and torch.equal(ys[1], ys[299])


@pytest.mark.parametrize("g,b,k1,batch", [(32, 2, False, 1), (64, 2, False, 5), (128, 3, True, 1), (64, 3, True, 4), (32, 3, False, 8)])
def test_data_flow_chain_over_widths_groups_single_basis_and_batches(goq, form, g, b, k1, batch):
    """A four-linear true chain (no item flagged) for every template form of the chain kernel that the headline case does
    not reach: W2, the three group sizes, the single-basis layout (no second operand), one and two column groups of
    tokens. Every linear against the oracle on the bits its producer wrote."""
    from tests.gpu_util import dev
    layout = goq.LAYOUT_TILE16_K1 if k1 else goq.LAYOUT_TILE16
    if batch > 1:   # the whole output of the producer (batch 1 reads slices, below)
        return _whole_output_chain(goq, g, b, layout, batch)
    shapes = [(1040, 384), (640, 1040 - 16), (2064, 640), (96, 2064 - 16)]   # channel counts that are no multiple of 16 or 128
    shapes = [(n, (k // g) * g) for n, k in shapes]                            # ... but whole macro-blocks along k
    layers, outs, items = [], [], []
    x0 = si.bf16_activations(batch, shapes[0][1], seed=950 + g)
    for j, (n, k) in enumerate(shapes):
        codes, meta, coef = si.random_quantized(n, k, g, b, seed=960 + j + g + b)
        d = goq.desc(n, k, g, b, layout)
        packed = torch.zeros(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
        goq.pack(d, dev(codes), dev(meta), dev(coef), packed)
        last = j == len(shapes) - 1
        y = torch.zeros((batch, n), dtype=torch.float32 if last else torch.bfloat16, device="cuda")
        x = dev(x0) if j == 0 else outs[j - 1][:, :k]   # a slice of the producer's row
        items.append((d, packed, x, batch, y, goq.F32 if last else goq.BF16, False))
        outs.append(y)
        layers.append((codes, meta, coef, n, k))
    torch.cuda.synchronize()
    kinds, _ = goq.sequence_order(goq.make_sequence(items))
    assert kinds == [goq.ORDER_NONE] + [goq.ORDER_DATA] * 3
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    x_bits = x0
    for j, (codes, meta, coef, n, k) in enumerate(layers):
        c, mt, cf = (codes, np.zeros_like(meta), np.stack([coef[..., 0], np.zeros_like(coef[..., 1])], axis=-1)) if k1 else (codes, meta, coef)
        y_ref = O.linear_f64(c, mt, cf, si.bf16_bits_to_f64(x_bits[:, :k]), g, b)
        got = outs[j].float().cpu().numpy().astype(np.float64)
        if j == len(layers) - 1:
            assert O.normwise_rel_err(got, y_ref) <= TIGHT, (j, O.normwise_rel_err(got, y_ref))
        else:
            from tests.gpu_util import check_bf16_output
            check_bf16_output(got, y_ref, 1e-4, "linear %d" % j)
            x_bits = _bits(outs[j])


def _whole_output_chain(goq, g, b, layout, batch):
    """batch > 1: each linear reads the whole bf16 output of the previous one (k_j = n_{j-1})."""
    from tests.gpu_util import dev, check_bf16_output
    k1 = layout == goq.LAYOUT_TILE16_K1
    widths = [384, 1024, 640, 2048, 96]
    widths = [max(g, (w // g) * g) for w in widths]
    layers, outs, items = [], [], []
    x0 = si.bf16_activations(batch, widths[0], seed=970 + g)
    for j in range(4):
        n, k = widths[j + 1], widths[j]
        codes, meta, coef = si.random_quantized(n, k, g, b, seed=980 + j + g + b)
        d = goq.desc(n, k, g, b, layout)
        packed = torch.zeros(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
        goq.pack(d, dev(codes), dev(meta), dev(coef), packed)
        last = j == 3
        y = torch.zeros((batch, n), dtype=torch.float32 if last else torch.bfloat16, device="cuda")
        x = dev(x0) if j == 0 else outs[j - 1]
        items.append((d, packed, x, batch, y, goq.F32 if last else goq.BF16, False))
        outs.append(y)
        layers.append((codes, meta, coef, n, k))
    kinds, sources = goq.sequence_order(goq.make_sequence(items))
    assert kinds == [goq.ORDER_NONE] + [goq.ORDER_DATA] * 3 and sources == [-1, 0, 1, 2]
    ws = _ws(goq, len(items))
    goq.gemv_sequence(goq.make_sequence(items), ws)
    torch.cuda.synchronize()
    assert goq.workspace_status(ws) == goq.OK
    x_bits = x0
    for j, (codes, meta, coef, n, k) in enumerate(layers):
        c, mt, cf = (codes, np.zeros_like(meta), np.stack([coef[..., 0], np.zeros_like(coef[..., 1])], axis=-1)) if k1 else (codes, meta, coef)
        y_ref = O.linear_f64(c, mt, cf, si.bf16_bits_to_f64(x_bits), g, b)
        got = outs[j].float().cpu().numpy().astype(np.float64)
        if j == 3:
            assert O.normwise_rel_err(got, y_ref) <= TIGHT, (j, O.normwise_rel_err(got, y_ref))
        else:
            check_bf16_output(got, y_ref, 1e-4, "linear %d" % j)
            x_bits = _bits(outs[j])
