"""The give-up path of the bounded device-side waits, made to run for real.

Every tensor-core kernel of the library waits on mbarriers through tc::mbar_wait / tc::warp_wait,
which give up after a time limit, latch DC_ERR_TIMEOUT in the caller's workspace header and let the
kernel return.  dc_selftest_bounded_wait runs exactly those routines on a barrier that nothing ever
completes (one CTA, no copies or tensor-core work in flight, a limit of a few milliseconds), so the
whole path is exercised without any fault: the wait runs out, the other role leaves through the
abort flag, the status is reported once and cleared, and the same workspace then serves an ordinary
convolution whose result is checked against the oracle."""
import time

import numpy as np
import pytest

from oracle import dc_oracle as O
from paper_2301_12187_b200 import inputs as I
from parity_util import assert_close

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_workspace_stays_usable():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")
    assert dc.workspace_status(ws) == dc.OK
    limit_us = 3000
    torch.cuda.synchronize()
    t0 = time.time()
    dc.selftest_bounded_wait(ws, limit_us)
    st, where, detail = dc.workspace_status_where(ws)          # synchronises
    dt = time.time() - t0
    assert st == dc.ERR_TIMEOUT
    assert where == 0x90000, hex(where)                        # the converged-warp wait ran out first
    assert detail == 2                                         # both roles left their wait
    assert limit_us * 1e-6 <= dt < 1.0                         # gave up after the limit, not at once, not never
    # reported once, then clear
    assert dc.workspace_status_where(ws) == (dc.OK, 0, 0)
    # the context and the workspace are still good: an ordinary launch on it matches the oracle
    spec = I.make_layer(61, 0, 24, 24, 3, 1, 1)
    lay = dc.DeviceLayer(spec)
    wf = torch.empty_like(lay.weight)
    bf = torch.empty(24, device="cuda")
    dc.fold_bn(lay, wf, bf)
    g = dc.geom(24, 24, 1, 3, 1, 1)
    assert dc.conv_kernel_name(2, 20, 20, g, dc.BF16) == "k_conv_tc_pairrows"
    packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    dc.pack_weights(wf, g, dc.BF16, packed)
    x = I.make_input(62, (2, 20, 20, 24), bf16=True)
    y = torch.full((2, 20, 20, 24), float("nan"), dtype=torch.bfloat16, device="cuda")
    dc.conv_forward(torch.from_numpy(x).to("cuda", dtype=torch.bfloat16), g, packed, bf, dc.ACT_IDENTITY, None, y, ws)
    assert dc.workspace_status(ws) == dc.OK
    Wf, bfo = O.fold_bn(spec)
    ref = O.conv_direct(x.transpose(0, 3, 1, 2), Wf, bfo, 3, 1, 1)
    assert_close(y.float().cpu().numpy().astype(np.float64).transpose(0, 3, 1, 2), ref, 2e-2)


def test_selftest_argument_errors():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")
    for limit in (0, 100001):
        with pytest.raises(dc.DcError) as e:
            dc.selftest_bounded_wait(ws, limit)
        assert e.value.status == dc.ERR_INVALID_ARG
    with pytest.raises(dc.DcError) as e:
        dc.selftest_bounded_wait(ws[:64], 1000)
    assert e.value.status == dc.ERR_WORKSPACE
    assert dc.workspace_status(ws) == dc.OK
