"""goq_gemv_static: the decode GEMV for callers that cannot allocate device memory.

Some users of this library cannot hand goq_gemv a scratch buffer: a plugin living inside a serving engine
that owns every byte of device memory, a decode loop that must never pay for cudaMalloc's device-wide
synchronisation, C code with no allocator at all. goq_gemv_static serves them from a fixed array inside the
library. This test calls it through the C ABI and holds it to the regular entry point, twice in a row,
because the second call starts from whatever the first one left in that shared array.

The file name sorts last on purpose: if this test fails, a run that stops at the first failure has already
run every other test. It passes on its own in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import goq_oracle as O

pytestmark = pytest.mark.gpu

TIGHT = 2e-5   # the bound the other GPU tests put on the fp32-accumulating kernels


@pytest.fixture(scope="module")
def goq():
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq as g
    g.lib()
    assert torch.cuda.is_available()
    return g


def _dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype in (np.uint16, np.float16):
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


def test_static_scratch_entry_matches_regular_entry_on_two_calls_in_a_row(goq):
    # 1000 rows x 1536 k: 63 row tiles of 12 records each over 296 CTAs, so most tiles are shared by
    # several CTAs and the scratch array (counters + parked partial sums) is really exercised.
    n, k, g, wb = 1000, 1536, 128, 3
    codes, meta, coef = si.random_quantized(n, k, g, wb, seed=77)
    rows = si.sample_rows(n, 40, seed=5)
    codes[rows], meta[rows], coef[rows] = O.quantize_geo(si.gaussian_weights(len(rows), k, seed=78), g, wb)
    d = goq.desc(n, k, g, wb)
    packed = torch.zeros(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
    goq.pack(d, _dev(codes), _dev(meta), _dev(coef), packed)
    ws = goq.new_workspace(d, goq.OP_GEMV, 16)
    assert goq.workspace_bytes(d, goq.OP_GEMV, 16) > 0

    for call, batch in enumerate((5, 16)):          # two calls in a row, different batch buckets
        xb = si.bf16_activations(batch, k, seed=100 + call)
        x = _dev(xb)
        y_regular = torch.full((batch, n), float("nan"), dtype=torch.float32, device="cuda")
        y_static = torch.full((batch, n), float("nan"), dtype=torch.float32, device="cuda")
        goq.gemv(d, packed, x, batch, y_regular, goq.F32, ws=ws)
        goq.gemv_static(d, packed, x, batch, y_static, goq.F32)
        torch.cuda.synchronize()
        if call == 1:
            # a warmed call allocates nothing: neither through torch nor behind its back (free device memory as the
            # driver reports it is unchanged across the call)
            torch_before, (free_before, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
            goq.gemv_static(d, packed, x, batch, y_static, goq.F32)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == torch_before
            assert torch.cuda.mem_get_info()[0] == free_before
        assert goq.gemv_static_status() == goq.OK   # the built-in array's status word: no wait gave up
        a = y_regular.cpu().numpy().astype(np.float64)
        b = y_static.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(b))
        assert O.normwise_rel_err(b, a) <= TIGHT
        # and both agree with the oracle on the sampled rows
        ref = O.linear_f64(codes, meta, coef, si.bf16_bits_to_f64(xb), g, wb, rows=rows)
        assert O.normwise_rel_err(b[:, rows], ref) <= TIGHT


def test_static_scratch_entry_rejects_what_it_cannot_serve(goq):
    x = torch.zeros((1, 128), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 16), dtype=torch.float32, device="cuda")
    dummy = torch.zeros(4096, dtype=torch.uint8, device="cuda")

    def status(d):
        try:
            goq.gemv_static(d, dummy, x, 1, y, goq.F32)
        except goq.GoqError as e:
            return e.status
        return goq.OK

    # more 16-row tiles than the scratch buffer's counter area holds: the streaming kernel does not take the layer
    # (goq_gemv serves it with a scratch-free kernel), refused here before anything is launched
    huge = goq.desc(8_000_000, 128, 128, 3)
    assert goq.workspace_bytes(huge, goq.OP_GEMV, 16) == 0
    assert status(huge) == goq.ERR_UNSUPPORTED
    # configurations the scratch-free kernels of goq_gemv serve
    assert status(goq.desc(16, 128, 16, 3)) == goq.ERR_UNSUPPORTED
    assert status(goq.desc(16, 128, 128, 4)) == goq.ERR_UNSUPPORTED
    assert status(goq.desc(16, 100, 128, 3)) == goq.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(y.abs().sum()) == 0.0
