"""CPU-only checks of the C-ABI library: it loads, exports every symbol include/dc.h declares,
and its host-side validation and geometry need no GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2301_12187_b200 import dc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # a 16-byte aligned, never dereferenced "device pointer"


def L(c_in, c_out, k=1, s=1, p=0, dw=False, bn=True):
    b = FAKE if bn else None
    return dc.Layer(c_in, c_out, c_in if dw else 1, k, s, p, FAKE, None, b, b, b, b, 1e-5)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = dc.lib()
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(dc.EXPORTS)


def test_status_strings():
    assert dc.status_string(dc.OK) == "ok"
    assert "timed out" in dc.status_string(dc.ERR_TIMEOUT)


@pytest.mark.parametrize("layers,res,expect", [
    ([L(16, 96), L(96, 96, 3, 1, 1, dw=True), L(96, 24)], [], (16, 24, 1, 3, 1, 1)),
    ([L(24, 144), L(144, 144, 3, 1, 1, dw=True), L(144, 24)], [(0, 2)], (24, 24, 1, 3, 1, 1)),
    ([L(24, 144), L(144, 144, 3, 2, 1, dw=True), L(144, 32)], [], (24, 32, 1, 3, 2, 1)),
    ([L(32, 192), L(192, 192, 3, 1, 1, dw=True), L(192, 32)] * 2, [(0, 2), (3, 5)], (32, 32, 1, 5, 1, 2)),
    ([L(3, 8, 3, 2, 1), L(8, 8, 3, 1, 1), L(8, 4, 5, 2, 2)], [], (3, 4, 1, 3 + 2 * 2 + 4 * 2, 4, 1 + 2 + 2 * 2)),
])
def test_merge_query_geometry(layers, res, expect):
    g, nbytes = dc.merge_query(layers, res)
    assert g.as_tuple() == expect
    assert nbytes > 0 and nbytes % 256 == 0


def status_of(fn, *a):
    try:
        fn(*a)
    except dc.DcError as e:
        return e.status
    return dc.OK


def test_merge_query_rejects_bad_chains():
    q = dc.merge_query
    assert status_of(q, [L(16, 96), L(95, 24)], []) == dc.ERR_SHAPE
    assert status_of(q, [L(16, 16, 2)], []) == dc.ERR_UNSUPPORTED                       # even kernel
    assert status_of(q, [dc.Layer(16, 16, 4, 3, 1, 1, FAKE, None, None, None, None, None, 0)], []) == dc.ERR_UNSUPPORTED
    assert status_of(q, [L(24, 144), L(144, 144, 3, 2, 1, dw=True), L(144, 24)], [(0, 2)]) == dc.ERR_NOT_MERGEABLE
    assert status_of(q, [L(24, 144), L(144, 144, 3, 1, 1, dw=True), L(144, 32)], [(0, 2)]) == dc.ERR_NOT_MERGEABLE
    assert status_of(q, [L(24, 24, 3, 1, 0)], [(0, 0)]) == dc.ERR_NOT_MERGEABLE          # 2p != k-1
    assert status_of(q, [L(8, 8)], [(0, 3)]) == dc.ERR_INVALID_ARG
    assert status_of(q, [L(8, 8), L(8, 8)], [(0, 1), (1, 1)]) == dc.ERR_INVALID_ARG      # overlapping groups
    assert status_of(q, [dc.Layer(8, 8, 1, 1, 1, 0, None, None, None, None, None, None, 0)], []) == dc.ERR_INVALID_ARG
    assert status_of(q, [dc.Layer(8, 8, 1, 1, 1, 0, FAKE, None, FAKE, None, None, None, 0)], []) == dc.ERR_INVALID_ARG


def test_packed_bytes():
    assert dc.packed_bytes(dc.geom(24, 24, 1, 3, 1, 1), dc.F32) == 24 * 24 * 9 * 4
    assert dc.packed_bytes(dc.geom(96, 96, 96, 3, 1, 1), dc.BF16) == 96 * 9 * 4
    # fold order: 3 chunks x 3 tap rows = 9 entries padded to 10; rows = 3 tap columns x 24 channels,
    # padded to 80; 16 bytes per (entry, row)
    # pair order: 2 parities x 3 chunks x 3 rows x 2 column pairs = 36 entries, N = 2 x 24
    assert dc.packed_bytes(dc.geom(24, 24, 1, 3, 1, 1), dc.BF16) == 36 * 48 * 16
    # pair rows, 5x5: 5 tap rows x 3 pair shifts x 8 chunks of the 64-channel line, N = 2 x 32
    assert dc.packed_bytes(dc.geom(32, 32, 1, 5, 1, 2), dc.BF16) == 120 * 64 * 16
    # fold order (c_in too wide for a 128-byte pixel pair): 5 chunks x 5 tap rows (+1 padding entry), N = 5 x 32
    assert dc.packed_bytes(dc.geom(40, 32, 1, 5, 1, 2), dc.BF16) == 26 * 160 * 16
    # general order: 18 chunks x 9 taps in 3 groups of 6 chunks, 64 output channels
    assert dc.packed_bytes(dc.geom(144, 64, 1, 3, 1, 1), dc.BF16) == 3 * 54 * 64 * 16
    assert dc.packed_bytes(dc.geom(3, 32, 1, 3, 2, 1), dc.BF16) == 10 * 32 * 16
    assert status_of(dc.packed_bytes, dc.geom(24, 24, 1, 4, 1, 1), dc.BF16) == dc.ERR_UNSUPPORTED


def test_kernel_name_query_follows_the_dispatch_rules():
    # few input channels: pair rows; many channels and >= 48 outputs, stride 1: rows; 40-64 channels, few outputs: fold; wide or strided: general tensor-core kernel;
    # channel counts that are no multiple of 8: CUDA cores
    assert dc.conv_kernel_name(64, 56, 56, dc.geom(24, 24, 1, 3, 1, 1), dc.BF16) == "k_conv_tc_pairrows"
    assert dc.conv_kernel_name(128, 28, 28, dc.geom(32, 32, 1, 5, 1, 2), dc.BF16) == "k_conv_tc_pairrows"
    assert dc.conv_kernel_name(128, 14, 14, dc.geom(40, 32, 1, 5, 1, 2), dc.BF16) == "k_conv_tc_fold"
    assert dc.conv_kernel_name(128, 56, 56, dc.geom(24, 32, 1, 3, 2, 1), dc.BF16) == "k_conv_tc_pairrows"
    assert dc.conv_kernel_name(128, 56, 56, dc.geom(96, 144, 1, 5, 2, 2), dc.BF16) == "k_conv_tc"
    assert dc.conv_kernel_name(128, 14, 14, dc.geom(96, 576, 1, 1, 1, 0), dc.BF16) == "k_conv_tc_rows"
    assert dc.conv_kernel_name(128, 7, 7, dc.geom(160, 960, 1, 3, 1, 1), dc.BF16) == "k_conv_tc_rows"
    assert dc.conv_kernel_name(128, 28, 28, dc.geom(144, 32, 1, 3, 1, 1), dc.BF16) == "k_conv_tc_rows"
    assert dc.conv_kernel_name(128, 28, 28, dc.geom(144, 24, 1, 3, 1, 1), dc.BF16) == "k_conv_tc"
    assert dc.conv_kernel_name(128, 224, 224, dc.geom(3, 32, 1, 3, 2, 1), dc.BF16) == "k_conv_stem_s2"
    assert dc.conv_kernel_name(2, 17, 33, dc.geom(3, 40, 1, 3, 2, 1), dc.BF16) == "k_conv_stem_tc"
    assert dc.conv_kernel_name(1, 20, 20, dc.geom(3, 264, 1, 3, 2, 1), dc.BF16) == "k_conv_smallcin_bf16"
    assert dc.conv_kernel_name(128, 56, 56, dc.geom(20, 12, 1, 3, 1, 1), dc.BF16) == "k_conv_dense_bf16"
    assert dc.conv_kernel_name(2, 16, 16, dc.geom(16, 24, 1, 3, 1, 1), dc.F32) == "k_conv_dense_f32"
    assert dc.conv_kernel_name(2, 16, 16, dc.geom(16, 16, 16, 3, 1, 1), dc.BF16) is None
    assert dc.conv_kernel_name(0, 16, 16, dc.geom(16, 24, 1, 3, 1, 1), dc.BF16) is None


def test_entry_points_validate_before_touching_the_device():
    lib = dc.lib()
    g = dc.geom(24, 24, 1, 3, 1, 1)
    ws = dc.conv_workspace_bytes()
    f = lib.dc_conv_forward
    assert f(None, 1, 8, 8, C.byref(g), FAKE, None, 0, None, FAKE, dc.BF16, FAKE, ws, None) == dc.ERR_INVALID_ARG
    assert f(FAKE, 1, 8, 8, C.byref(g), FAKE, None, 0, None, FAKE, dc.BF16, None, 0, None) == dc.ERR_WORKSPACE
    assert f(FAKE + 4, 1, 8, 8, C.byref(g), FAKE, None, 0, None, FAKE, dc.BF16, FAKE, ws, None) == dc.ERR_ALIGNMENT
    assert f(FAKE, 1, 1, 1, C.byref(dc.geom(8, 8, 1, 5, 1, 0)), FAKE, None, 0, None, FAKE, dc.F32, FAKE, ws, None) == dc.ERR_SHAPE
    assert f(FAKE, 1, 8, 8, C.byref(g), FAKE, None, 7, None, FAKE, dc.BF16, FAKE, ws, None) == dc.ERR_INVALID_ARG
    d = lib.dc_dwconv_forward
    assert d(FAKE, 1, 8, 8, 16, 2, 1, 0, FAKE, None, 0, FAKE, dc.F32, None) == dc.ERR_UNSUPPORTED
    assert d(FAKE, 1, 8, 8, 16, 3, 1, 1, FAKE + 8, None, 0, FAKE, dc.F32, None) == dc.ERR_ALIGNMENT
    m = lib.dc_merge_chain
    arr = dc.layer_array([L(8, 8)])
    res, _ = dc._res_array([])
    assert m(arr, 1, res, 0, FAKE, FAKE, None, dc.F32, FAKE, 16, None) == dc.ERR_WORKSPACE
    assert m(arr, 1, res, 0, FAKE, FAKE, None, dc.F32, None, 1 << 20, None) == dc.ERR_WORKSPACE
    assert m(arr, 1, res, 0, None, FAKE, None, dc.F32, FAKE, 1 << 20, None) == dc.ERR_INVALID_ARG
    blk = dc.Block(24, 144, 24, 1, 3, 2, 1, 1, 1, 1, FAKE, None, FAKE, None, FAKE, None)
    n = C.c_size_t(0)
    assert lib.dc_block_workspace_bytes(1, 8, 8, C.byref(blk), dc.BF16, C.byref(n)) == dc.ERR_NOT_MERGEABLE
    blk.dw_stride = 1
    assert lib.dc_block_workspace_bytes(2, 8, 8, C.byref(blk), dc.BF16, C.byref(n)) == dc.OK
    assert n.value == 256 + 2 * (2 * 8 * 8 * 144 * 2)


def test_host_entry_reports_its_workspace():
    arr = dc.layer_array([L(24, 144), L(144, 144, 3, 1, 1, dw=True), L(144, 24)])
    n = dc.chain_host_workspace_bytes(arr, 3, [(0, 2)], 4, 16, 16, dc.BF16)
    assert n > 2 * 4 * 16 * 16 * 24 * 2


def test_host_parameter_layout_offsets():
    """dc_chain_host_param_layout: 256-byte-rounded slots, six per layer, in layer order."""
    import ctypes as C
    from paper_2301_12187_b200 import dc, inputs as I
    specs = [I.make_layer(0, 0, 24, 144, 1, 1, 0), I.make_layer(0, 1, 144, 144, 3, 1, 1, depthwise=True)]
    arr, keep = dc.host_layer_array(specs)
    offs = (C.c_size_t * 12)()
    total = C.c_size_t(0)
    assert dc.lib().dc_chain_host_param_layout(arr, 2, offs, C.byref(total)) == dc.OK
    r = lambda b: (b + 255) // 256 * 256
    want, o = [], 0
    for s in specs:
        for j in range(6):
            want.append(o)
            o += r(s.weight.size * 4 if j == 0 else s.c_out * 4)
    assert list(offs) == want and total.value == o
    assert dc.lib().dc_chain_host_param_layout(arr, 0, offs, C.byref(total)) == dc.ERR_INVALID_ARG


def test_vgg_style_cases_have_the_shapes_of_their_stage():
    """Host logic of the bench's VGG-style workload: two dense 3x3 layers of equal width with no activation
    between them, on the map of that width's stage; by the oracle's geometry rule they merge into a 5x5
    layer with padding 2 (two 3x3 -> 5x5)."""
    from oracle import dc_oracle as O
    from paper_2301_12187_b200 import inputs as I
    assert sorted(I.VGG_MAPS) == [64, 128, 256, 512]
    for c, hw in I.VGG_MAPS.items():
        case = I.vgg_case(c, seed=3, batch=2)
        assert case.x_shape == (2, hw, hw, c) and case.dtype == "bf16" and case.residuals == []
        assert [(s.c_in, s.c_out, s.k, s.stride, s.pad, s.groups, s.act) for s in case.layers] == [(c, c, 3, 1, 1, 1, None)] * 2
        assert O.compose_geometry(case.layers) == (5, 1, 2)
