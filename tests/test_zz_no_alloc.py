"""dc_merge_chain_static: the merge for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (inside an allocator callback, in a
plug-in after its host's initialisation phase, next to an allocator that owns the whole device).
For them the library carries its own fixed scratch array.  This test calls that entry point
through the C ABI several times in a row, with different runs, and checks each result against the
regular dc_merge_chain, which works in a caller-provided workspace (and is itself held to the
oracle in test_gpu_parity.py, so agreement with it is agreement with the oracle at the same
tolerance).  It also checks that the device's free memory is the same before and after the call.
The file name sorts last on purpose: if this addition ever fails, every other test has already run.
"""
import numpy as np
import pytest

from paper_2301_12187_b200 import inputs as I

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_W = 1e-5


def rel(a, b):
    a, b = a.double().flatten(), b.double().flatten()
    return float((a - b).norm() / b.norm().clamp_min(1e-30))


def merge_both(dc, specs, residuals):
    layers = [dc.DeviceLayer(s) for s in specs]
    g, ws_bytes = dc.merge_query(layers, residuals)
    out = {}
    for name in ("workspace", "static"):
        wm = torch.full((g.c_out, g.c_in, g.k, g.k), float("nan"), dtype=torch.float32, device="cuda")
        bm = torch.full((g.c_out,), float("nan"), dtype=torch.float32, device="cuda")
        packed = torch.zeros(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
        if name == "workspace":
            ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
            dc.merge_chain(layers, residuals, wm, bm, packed, dc.BF16, ws)
        else:
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            dc.merge_chain_static(layers, residuals, wm, bm, packed, dc.BF16)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        torch.cuda.synchronize()
        out[name] = (wm, bm, packed)
    return out


def test_static_scratch_merge_matches_workspace_merge_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    assert dc.merge_chain_static_capacity() == 4 << 20
    # two different runs back to back: the second call finds the first call's leftovers in the scratch
    mk = I.make_layer
    dense = ([mk(51, 0, 32, 48, 3, 1, 1), mk(51, 1, 48, 32, 3, 1, 1)], [])                 # dense o dense composition
    dw_first = ([mk(52, 0, 16, 16, 3, 1, 1, depthwise=True), mk(52, 1, 16, 16, 3, 1, 1, depthwise=True),
                 mk(52, 2, 16, 8, 1, 1, 0)], [(0, 0)])                                      # diagonal compositions
    cases = [(c.layers, c.residuals) for c in (I.chain_case(3), I.chain_case(1), I.chain_case(3))] + [dense, dw_first]
    # the first call on a device looks up the scratch array's address (and may load the module):
    # make it before the calls whose effect on free memory is measured
    dc.merge_chain_static([dc.DeviceLayer(s) for s in dense[0]], dense[1], torch.empty((32, 32, 5, 5), device="cuda"),
                          torch.empty((32,), device="cuda"), None, dc.F32)
    torch.cuda.synchronize()
    for layers_, res_ in cases:
        out = merge_both(dc, layers_, res_)
        (w0, b0, p0), (w1, b1, p1) = out["workspace"], out["static"]
        assert not torch.isnan(w1).any() and not torch.isnan(b1).any()
        assert rel(w1, w0) <= TOL_W and rel(b1, b0) <= TOL_W
        assert torch.equal(p0, p1)


def test_static_scratch_merge_inside_a_captured_graph():
    """After a first call outside capture (it looks up the scratch array's address), the call only queues
    kernels on the stream: captured in a CUDA graph and replayed, it gives the same bits every time."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    case = I.chain_case(1)
    layers = [dc.DeviceLayer(s) for s in case.layers]
    g, ws_bytes = dc.merge_query(layers, case.residuals)
    ref_w = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
    ref_b = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
    ref_p = torch.zeros(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    dc.merge_chain(layers, case.residuals, ref_w, ref_b, ref_p, dc.BF16, torch.empty(ws_bytes, dtype=torch.uint8, device="cuda"))
    wm, bm, packed = torch.empty_like(ref_w), torch.empty_like(ref_b), torch.zeros_like(ref_p)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        dc.merge_chain_static(layers, case.residuals, wm, bm, packed, dc.BF16)       # warm-up, outside capture
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            dc.merge_chain_static(layers, case.residuals, wm, bm, packed, dc.BF16)
        for _ in range(2):
            wm.fill_(float("nan")); bm.fill_(float("nan")); packed.zero_()
            graph.replay()
            st.synchronize()
            assert rel(wm, ref_w) <= TOL_W and rel(bm, ref_b) <= TOL_W
            assert torch.equal(packed, ref_p)


def test_static_scratch_merge_refuses_runs_beyond_its_capacity():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    specs = I.inverted_residual(0, 0, 160, 160, 6, 1, block=0, acts=(None, None))   # 160 -> 960 -> 160
    layers = [dc.DeviceLayer(s) for s in specs]
    g, ws_bytes = dc.merge_query(layers, [(0, 2)])
    assert ws_bytes > dc.merge_chain_static_capacity()
    wm = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
    bm = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
    with pytest.raises(dc.DcError) as e:
        dc.merge_chain_static(layers, [(0, 2)], wm, bm, None, dc.F32)
    assert e.value.status == dc.ERR_WORKSPACE
