"""GPU parity: every C-ABI entry point against the fp64 oracle on the same seeded inputs.

Tolerances (rel-L2 = ||a-b||/||b||, b the oracle): merged weights and bias 1e-5 (fp32 FMA merge);
conv outputs 1e-4 in fp32 and 2e-2 in bf16 (bf16 rounding of the merged weights, of the input and
of the output; fp32 accumulation).  Every output is also held to the element-wise bound of
parity_util (a localised fault cannot hide under a whole-tensor norm), and every buffer the library
writes sits between sentinel bands that must come back untouched."""
import numpy as np
import pytest

from oracle import dc_oracle as O
from paper_2301_12187_b200 import inputs as I
from parity_util import Guarded, assert_close

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_W, TOL_F32, TOL_BF16 = 1e-5, 1e-4, 2e-2


@pytest.fixture(scope="module")
def dc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc as _dc
    _dc.lib()
    return _dc


def dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda", dtype=dtype).contiguous()


def nchw(t):
    return t.float().cpu().numpy().astype(np.float64).transpose(0, 3, 1, 2)


def new_ws(dc, nbytes=None):
    return torch.zeros(max(nbytes or 0, dc.conv_workspace_bytes()), dtype=torch.uint8, device="cuda")


def run_merge(dc, specs, residuals, packed_dtype=None, algo=0):
    layers = [dc.DeviceLayer(s) for s in specs]
    g, ws_bytes = dc.merge_query(layers, residuals)
    bufs = [Guarded(torch, (g.c_out, g.c_in, g.k, g.k), torch.float32, fill=float("nan")),
            Guarded(torch, (g.c_out,), torch.float32, fill=float("nan")),
            Guarded(torch, (ws_bytes,), torch.uint8)]
    wm, bm, ws = (b.t for b in bufs)
    packed = None
    if packed_dtype is not None:
        bufs.append(Guarded(torch, (dc.packed_bytes(g, packed_dtype),), torch.uint8))
        packed = bufs[-1].t
    dc.merge_chain(layers, residuals, wm, bm, packed, packed_dtype if packed_dtype is not None else dc.F32, ws,
                   algo=algo)
    torch.cuda.synchronize()
    for b, name in zip(bufs, ("merged weights", "merged bias", "merge workspace", "packed weights")):
        b.check(name)
    assert not torch.isnan(wm).any() and not torch.isnan(bm).any()
    return g, wm, bm, packed


def run_conv(dc, x, g, packed, bias, act, residual=None, algo=0):
    n, h, w, _ = x.shape
    ho, wo = O.out_extent(h, g.k, g.stride, g.pad), O.out_extent(w, g.k, g.stride, g.pad)
    gy = Guarded(torch, (n, ho, wo, g.c_out), x.dtype, fill=float("nan"))
    gws = Guarded(torch, (dc.conv_workspace_bytes(),), torch.uint8, fill=0)
    y, ws = gy.t, gws.t
    dc.conv_forward(x, g, packed, bias, act, residual, y, ws, algo=algo)
    assert dc.workspace_status(ws) == dc.OK
    gy.check("conv output")
    gws.check("conv workspace")
    assert not torch.isnan(y.float()).any(), "an output element was never written"
    return y


def small_chain(name, rng_seed=0):
    """Reduced-size versions of the four single-span topologies plus harder ones."""
    mk = I.make_layer
    s = rng_seed
    if name == "t0":
        return [mk(s, 0, 16, 96, 1, 1, 0), mk(s, 1, 96, 96, 3, 1, 1, depthwise=True), mk(s, 2, 96, 24, 1, 1, 0)], []
    if name == "t1":
        return [mk(s, 0, 24, 144, 1, 1, 0), mk(s, 1, 144, 144, 3, 1, 1, depthwise=True), mk(s, 2, 144, 24, 1, 1, 0)], [(0, 2)]
    if name == "t2":
        return [mk(s, 0, 24, 144, 1, 1, 0), mk(s, 1, 144, 144, 3, 2, 1, depthwise=True), mk(s, 2, 144, 32, 1, 1, 0)], []
    if name == "t3":
        L = []
        for b in range(2):
            L += [mk(s, 3 * b, 32, 192, 1, 1, 0), mk(s, 3 * b + 1, 192, 192, 3, 1, 1, depthwise=True),
                  mk(s, 3 * b + 2, 192, 32, 1, 1, 0)]
        return L, [(0, 2), (3, 5)]
    if name == "dense_pair":
        return [mk(s, 0, 8, 16, 3, 1, 1), mk(s, 1, 16, 8, 3, 1, 1, with_bn=False)], []
    if name == "s2_first":
        return [mk(s, 0, 8, 16, 3, 2, 1), mk(s, 1, 16, 16, 1, 1, 0), mk(s, 2, 16, 24, 1, 1, 0)], []
    if name == "dw_first":
        return [mk(s, 0, 16, 16, 3, 1, 1, depthwise=True), mk(s, 1, 16, 16, 3, 1, 1, depthwise=True),
                mk(s, 2, 16, 8, 1, 1, 0)], [(0, 0)]
    if name == "dw_only":
        return [mk(s, 0, 8, 8, 3, 1, 1, depthwise=True), mk(s, 1, 8, 8, 3, 2, 1, depthwise=True)], []
    if name == "single":
        return [mk(s, 0, 8, 24, 3, 1, 1)], []
    if name == "skip_mid":
        return [mk(s, 0, 8, 16, 1, 1, 0), mk(s, 1, 16, 16, 3, 1, 1, depthwise=True), mk(s, 2, 16, 40, 1, 1, 0)], [(1, 1)]
    raise KeyError(name)


CHAINS = ["t0", "t1", "t2", "t3", "dense_pair", "s2_first", "dw_first", "dw_only", "single", "skip_mid"]


def test_fold_bn(dc):
    for spec in (I.make_layer(3, 0, 24, 40, 3, 1, 1), I.make_layer(3, 1, 32, 32, 3, 1, 1, depthwise=True),
                 I.make_layer(3, 2, 8, 8, 1, 1, 0, with_bn=False)):
        lay = dc.DeviceLayer(spec)
        w = torch.empty_like(lay.weight)
        b = torch.empty(spec.c_out, device="cuda")
        dc.fold_bn(lay, w, b)
        Wo, bo = O.fold_bn(spec)
        assert O.rel_l2(w.cpu().numpy(), Wo) < 1e-6 and O.rel_l2(b.cpu().numpy(), bo) < 1e-6 or \
            (spec.bn is None and np.all(bo == 0) and float(b.abs().max()) == 0)


@pytest.mark.parametrize("name", CHAINS)
def test_merge_chain_weights(dc, name):
    specs, res = small_chain(name)
    g, wm, bm, _ = run_merge(dc, specs, res)
    W, b, k, s, p = O.merge_formula(specs, res)
    assert (g.k, g.stride, g.pad, g.c_in, g.c_out) == (k, s, p, W.shape[1], W.shape[0])
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W
    assert O.rel_l2(bm.cpu().numpy(), b) <= TOL_W


def wide_chain(name, s=5):
    """Runs with more arithmetic than `small_chain`: two skip blocks in a row at three widths, a
    dense 3x3 o 3x3 o 3x3 run (7x7 result) and a stride-2 run with a 5x5 depthwise layer."""
    mk = I.make_layer
    if name in ("two_blocks_32", "two_blocks_64", "two_blocks_48"):
        c = int(name.rsplit("_", 1)[1])
        L = []
        for b in range(2):
            L += [mk(s, 3 * b, c, 6 * c, 1, 1, 0), mk(s, 3 * b + 1, 6 * c, 6 * c, 3, 1, 1, depthwise=True),
                  mk(s, 3 * b + 2, 6 * c, c, 1, 1, 0)]
        return L, [(0, 2), (3, 5)]
    if name == "dense_7x7":
        return [mk(s, 0, 16, 24, 3, 1, 1), mk(s, 1, 24, 24, 3, 1, 1), mk(s, 2, 24, 16, 3, 1, 1)], [(1, 1)]
    if name == "s2_dw5":
        return [mk(s, 0, 40, 240, 1, 1, 0), mk(s, 1, 240, 240, 5, 2, 2, depthwise=True), mk(s, 2, 240, 48, 1, 1, 0)], []
    raise KeyError(name)


WIDE = ["two_blocks_32", "two_blocks_64", "two_blocks_48", "dense_7x7", "s2_dw5"]


@pytest.mark.parametrize("algo", ["steps", "auto"])
@pytest.mark.parametrize("name", CHAINS + WIDE)
def test_merge_chain_both_walks(dc, name, algo):
    """The pairwise walk and the walk that merges inverted-residual blocks in one step, each
    against the oracle's formula (weights, bias, and the bf16 packed copy through the fp32 result)."""
    specs, res = small_chain(name) if name in CHAINS else wide_chain(name)
    code = dc.MERGE_STEPS if algo == "steps" else dc.MERGE_AUTO
    g, wm, bm, packed = run_merge(dc, specs, res, packed_dtype=dc.BF16, algo=code)
    W, b, k, s, p = O.merge_formula(specs, res)
    assert (g.k, g.stride, g.pad) == (k, s, p)
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W
    assert O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    # the packed copy must be what dc_pack_weights makes of the delivered fp32 kernel, bit for bit
    again = torch.empty_like(packed)
    dc.pack_weights(wm, g, dc.BF16, again)
    torch.cuda.synchronize()
    assert torch.equal(packed, again)


@pytest.mark.parametrize("case", ["no_bn", "bias_no_bn", "wide_hidden", "block_inside_run", "fold_order", "rows_order",
                                  "block_after_1x1", "skip_1x1_then_3x3"])
def test_block_step_edge_cases(dc, case):
    """Blocks without BN, with plain biases, with a hidden width that is staged in several passes,
    and a block in the middle of a longer run (neighbours composed pairwise around it)."""
    mk = I.make_layer
    if case == "no_bn":
        specs = [mk(11, 0, 8, 48, 1, 1, 0, with_bn=False), mk(11, 1, 48, 48, 3, 1, 1, depthwise=True, with_bn=False),
                 mk(11, 2, 48, 8, 1, 1, 0, with_bn=False)]
        res = [(0, 2)]
    elif case == "bias_no_bn":
        specs = [mk(12, 0, 16, 96, 1, 1, 0, with_bn=False, with_bias=True),
                 mk(12, 1, 96, 96, 5, 2, 2, depthwise=True), mk(12, 2, 96, 24, 1, 1, 0, with_bias=True)]
        res = []
    elif case == "wide_hidden":
        specs = [mk(13, 0, 160, 960, 1, 1, 0), mk(13, 1, 960, 960, 3, 1, 1, depthwise=True), mk(13, 2, 960, 160, 1, 1, 0)]
        res = [(0, 2)]
    elif case == "block_after_1x1":  # a k x k piece composed after a 1x1 layer: one term per tap sum
        specs = [mk(17, 0, 40, 16, 1, 1, 0), mk(17, 1, 16, 96, 1, 1, 0), mk(17, 2, 96, 96, 3, 1, 1, depthwise=True),
                 mk(17, 3, 96, 16, 1, 1, 0)]
        res = [(1, 3)]
    elif case == "skip_1x1_then_3x3":  # (W1 + I) under a dense 3x3
        specs = [mk(18, 0, 24, 24, 1, 1, 0), mk(18, 1, 24, 40, 3, 1, 1)]
        res = [(0, 0)]
    elif case == "fold_order":      # 40-64 input channels, narrow output: packed copy in the fold order
        specs = [mk(15, 0, 48, 288, 1, 1, 0), mk(15, 1, 288, 288, 3, 1, 1, depthwise=True), mk(15, 2, 288, 24, 1, 1, 0)]
        res = []
    elif case == "rows_order":      # wide input and output: packed copy in 64-channel planes
        specs = [mk(16, 0, 64, 384, 1, 1, 0), mk(16, 1, 384, 384, 3, 1, 1, depthwise=True), mk(16, 2, 384, 64, 1, 1, 0)]
        res = [(0, 2)]
    else:
        specs = [mk(14, 0, 16, 8, 3, 1, 1), mk(14, 1, 8, 48, 1, 1, 0), mk(14, 2, 48, 48, 3, 1, 1, depthwise=True),
                 mk(14, 3, 48, 8, 1, 1, 0), mk(14, 4, 8, 24, 1, 1, 0)]
        res = [(1, 3)]
    g, wm, bm, packed = run_merge(dc, specs, res, packed_dtype=dc.BF16)
    W, b, *_ = O.merge_formula(specs, res)
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W
    assert O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    again = torch.empty_like(packed)
    dc.pack_weights(wm, g, dc.BF16, again)
    torch.cuda.synchronize()
    assert torch.equal(packed, again)
    g2, wm2, bm2, _ = run_merge(dc, specs, res, algo=dc.MERGE_STEPS)
    assert O.rel_l2(wm2.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm2.cpu().numpy(), b) <= TOL_W


@pytest.mark.parametrize("c,n,h,w", [(64, 2, 28, 28), (128, 2, 14, 14), (256, 1, 14, 14), (512, 1, 14, 14)])
def test_vgg_style_dense_merge(dc, c, n, h, w):
    """Two dense 3x3 layers (VGG-style, c -> c -> c) merged into one 5x5 layer: merged weights against
    the formula, and the bf16 forward of the merged layer (tensor-bound for these widths) against the
    sequential chain."""
    mk = I.make_layer
    specs = [mk(31, 0, c, c, 3, 1, 1), mk(31, 1, c, c, 3, 1, 1)]
    g, wm, bm, packed = run_merge(dc, specs, [], packed_dtype=dc.BF16)
    assert (g.k, g.stride, g.pad) == (5, 1, 2)
    W, b, *_ = O.merge_formula(specs, [])
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    assert dc.conv_kernel_name(n, h, w, g, dc.BF16) == "k_conv_tc_rows"
    x = I.make_input(32, (n, h, w, c), bf16=True)
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bm, dc.ACT_IDENTITY)
    ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), specs, [])
    assert_close(nchw(y), ref, TOL_BF16)


def width14_chain(name, s=41):
    """Spans with the channel counts of MobileNetV2 at width 1.4 (Fig. 4: 48, 24, 32, 144, ...)."""
    mk = I.make_layer
    if name == "first_block":      # depthwise 48 + projection to 24 (t = 1 block after the 48-channel stem)
        return [mk(s, 0, 48, 48, 3, 1, 1, depthwise=True), mk(s, 1, 48, 24, 1, 1, 0)], []
    if name == "block_s2":         # 24 -> 144 -> 32, stride 2
        return [mk(s, 0, 24, 144, 1, 1, 0), mk(s, 1, 144, 144, 3, 2, 1, depthwise=True), mk(s, 2, 144, 32, 1, 1, 0)], []
    if name == "block_res_32":     # 32 -> 192 -> 32 with its skip folded
        return [mk(s, 0, 32, 192, 1, 1, 0), mk(s, 1, 192, 192, 3, 1, 1, depthwise=True), mk(s, 2, 192, 32, 1, 1, 0)], [(0, 2)]
    if name == "block_res_88":     # 88 -> 528 -> 88 (64 x 1.4 rounded to 8)
        return [mk(s, 0, 88, 528, 1, 1, 0), mk(s, 1, 528, 528, 3, 1, 1, depthwise=True), mk(s, 2, 528, 88, 1, 1, 0)], [(0, 2)]
    if name == "cross_block_48":   # two 48-channel blocks merged across their boundary: 5x5, 48 -> 48
        L = []
        for b in range(2):
            L += [mk(s, 3 * b, 48, 288, 1, 1, 0), mk(s, 3 * b + 1, 288, 288, 3, 1, 1, depthwise=True),
                  mk(s, 3 * b + 2, 288, 48, 1, 1, 0)]
        return L, [(0, 2), (3, 5)]
    if name == "project_expand":   # projection of one block and expansion of the next: 144 -> 32 -> 192
        return [mk(s, 0, 144, 32, 1, 1, 0), mk(s, 1, 32, 192, 1, 1, 0)], []
    raise KeyError(name)


@pytest.mark.parametrize("name,n,h,w", [("first_block", 2, 28, 28), ("block_s2", 2, 28, 28), ("block_res_32", 2, 28, 28),
                                        ("block_res_88", 2, 14, 14), ("cross_block_48", 2, 14, 14),
                                        ("project_expand", 1, 14, 14)])
def test_width_1p4_spans(dc, name, n, h, w):
    """Merge and bf16 forward of spans at MobileNetV2-1.4 widths, both walks of the merge."""
    specs, res = width14_chain(name)
    W, b, k, s, p = O.merge_formula(specs, res)
    for algo in (dc.MERGE_AUTO, dc.MERGE_STEPS):
        g, wm, bm, packed = run_merge(dc, specs, res, packed_dtype=dc.BF16, algo=algo)
        assert (g.k, g.stride, g.pad) == (k, s, p)
        assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    x = I.make_input(42, (n, h, w, specs[0].c_in), bf16=True)
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bm, dc.ACT_RELU6)
    ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), specs, res, final_act="relu6")
    assert_close(nchw(y), ref, TOL_BF16, what=name)


@pytest.mark.parametrize("stride", [1, 2])
def test_large_packed_copy_is_written_chunk_by_chunk(dc, stride):
    """Merged kernels whose packed copy has 262 144 elements or more are packed one 16-byte chunk per
    thread (rows order for stride 1, general order for stride 2): same bits as dc_pack_weights."""
    mk = I.make_layer
    specs = [mk(21, 0, 192, 192, 1, 1, 0), mk(21, 1, 192, 192, 3, stride, 1)]
    g, wm, bm, packed = run_merge(dc, specs, [], packed_dtype=dc.BF16)
    assert packed.numel() // 2 >= 262144
    W, b, *_ = O.merge_formula(specs, [])
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    again = torch.empty_like(packed)
    dc.pack_weights(wm, g, dc.BF16, again)
    torch.cuda.synchronize()
    assert torch.equal(packed, again)


@pytest.mark.parametrize("name", CHAINS)
def test_merged_conv_fp32_equals_sequential_chain(dc, name):
    specs, res = small_chain(name, rng_seed=1)
    g, wm, bm, packed = run_merge(dc, specs, res, packed_dtype=dc.F32)
    x = I.make_input(1, (2, 13, 11, specs[0].c_in))
    y = run_conv(dc, dev(x), g, packed, bm, dc.ACT_IDENTITY)
    ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), specs, res)
    assert y.shape[1:3] == ref.shape[2:]
    assert_close(nchw(y), ref, TOL_F32, bf16=False)


def test_config0_tiny_fp32(dc):
    case = I.chain_case(0)
    g, wm, bm, packed = run_merge(dc, case.layers, case.residuals, packed_dtype=dc.F32)
    W, b, k, s, p = O.merge_formula(case.layers, case.residuals)
    assert (g.c_in, g.c_out, g.k, g.stride, g.pad) == (16, 24, 3, 1, 1)
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    x = case.x()
    y = run_conv(dc, dev(x), g, packed, bm, dc.ACT_IDENTITY)
    ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), case.layers, case.residuals)
    assert_close(nchw(y), ref, TOL_F32, bf16=False)
    # the chain with its original per-layer padding agrees inside and differs on the border ring
    orig = O.chain_forward_original(x.transpose(0, 3, 1, 2), case.layers, case.residuals)
    assert O.rel_l2(nchw(y)[:, :, 1:-1, 1:-1], orig[:, :, 1:-1, 1:-1]) <= TOL_F32
    assert O.rel_l2(nchw(y), orig) > 1e-3


BF16_SHAPES = [
    # (name, n, h, w) -- spatial sizes that span several tiles and leave ragged tails
    ("t1", 3, 19, 23), ("t2", 2, 22, 18), ("t3", 2, 17, 21), ("t0", 1, 9, 40), ("s2_first", 2, 30, 14),
    ("dense_pair", 2, 12, 70), ("single", 3, 8, 8), ("skip_mid", 1, 33, 9),
]


@pytest.mark.parametrize("algo", ["simt", "auto"])
@pytest.mark.parametrize("name,n,h,w", BF16_SHAPES)
def test_merged_conv_bf16_equals_sequential_chain(dc, name, n, h, w, algo):
    specs, res = small_chain(name, rng_seed=2)
    g, wm, bm, packed = run_merge(dc, specs, res, packed_dtype=dc.BF16)
    x = I.make_input(2, (n, h, w, specs[0].c_in), bf16=True)
    for act in (dc.ACT_IDENTITY, dc.ACT_RELU6):
        y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bm, act,
                     algo=dc.ALGO_SIMT if algo == "simt" else dc.ALGO_AUTO)
        ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), specs, res,
                                        final_act="relu6" if act else None)
        assert not torch.isnan(y.float()).any()
        assert_close(nchw(y), ref, TOL_BF16)


@pytest.mark.parametrize("algo", ["simt", "auto"])
@pytest.mark.parametrize("c_in,c_out,k,s,p,n,h,w", [
    (32, 16, 1, 1, 0, 2, 14, 14), (96, 24, 1, 1, 0, 1, 20, 12), (160, 320, 1, 1, 0, 2, 7, 7),
    (320, 1280, 1, 1, 0, 1, 7, 7), (3, 32, 3, 2, 1, 2, 32, 32), (16, 96, 1, 1, 0, 1, 24, 24),
    (96, 144, 5, 2, 2, 1, 20, 20), (64, 384, 1, 1, 0, 3, 14, 14), (24, 40, 7, 1, 3, 1, 16, 16),
    (40, 24, 3, 1, 0, 1, 12, 12), (20, 12, 3, 1, 1, 1, 10, 10),
])
def test_single_conv_bf16_with_explicit_skip(dc, c_in, c_out, k, s, p, n, h, w, algo):
    spec = I.make_layer(5, 0, c_in, c_out, k, s, p)
    lay = dc.DeviceLayer(spec)
    wf = torch.empty_like(lay.weight)
    bf = torch.empty(c_out, device="cuda")
    dc.fold_bn(lay, wf, bf)
    g = dc.geom(c_in, c_out, 1, k, s, p)
    packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    dc.pack_weights(wf, g, dc.BF16, packed)
    x = I.make_input(6, (n, h, w, c_in), bf16=True)
    ho, wo = O.out_extent(h, k, s, p), O.out_extent(w, k, s, p)
    r = I.round_bf16(I.normal(7, 99, (n, ho, wo, c_out)))
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bf, dc.ACT_RELU6, residual=dev(r, torch.bfloat16),
                 algo=dc.ALGO_SIMT if algo == "simt" else dc.ALGO_AUTO)
    Wf, bfo = O.fold_bn(spec)
    ref = O.relu6(O.conv_direct(x.transpose(0, 3, 1, 2), Wf, bfo, k, s, p) + r.transpose(0, 3, 1, 2))
    assert_close(nchw(y), ref, TOL_BF16)


# One case per branch of the forward kernels: the expected kernel is asserted, so a change of the
# dispatch rules cannot silently drop a kernel from the parity suite.
@pytest.mark.parametrize("c_in,c_out,k,s,p,n,h,w,kernel", [
    (24, 24, 3, 1, 1, 3, 30, 22, "k_conv_tc_pairrows"),     # odd padding: pairs (2j-1, 2j), masked ends
    (32, 32, 5, 1, 2, 2, 28, 28, "k_conv_tc_pairrows"),     # 5x5, even padding, full 128-byte lines
    (16, 8, 3, 1, 0, 1, 18, 40, "k_conv_tc_pairrows"),      # no padding, 16 of 64 channels of a line used
    (8, 16, 3, 1, 1, 1, 6, 300, "k_conv_tc_pairrows"),      # three column strips: per-pixel stores, strip halos
    (16, 16, 7, 1, 3, 1, 20, 20, "k_conv_tc_pairrows"),     # 7x7: 56 instructions per block
    (24, 24, 3, 1, 1, 1, 9, 15, "k_conv_dense_bf16"),       # odd width: pair-order weights read by the CUDA-core kernel
    (40, 32, 5, 1, 2, 2, 14, 14, "k_conv_tc_fold"),         # odd entry count (padding entry), 5 tap columns
    (48, 24, 3, 1, 1, 2, 20, 20, "k_conv_tc_fold"),
    (64, 32, 3, 1, 1, 1, 12, 70, "k_conv_tc_fold"),         # two column strips
    (4, 16, 5, 1, 2, 1, 9, 200, "k_conv_stem_tc"),          # two row segments per output row, 26 chunk planes
    (3, 40, 3, 2, 1, 2, 17, 33, "k_conv_stem_tc"),          # 40 output channels (48 operand rows), odd sizes
    (3, 32, 3, 2, 1, 3, 40, 300, "k_conv_stem_tc"),         # the stem's geometry, ragged second segment
    (1, 8, 3, 1, 1, 2, 20, 20, "k_conv_stem_tc"),           # one input channel
    (3, 24, 5, 2, 2, 2, 21, 304, "k_conv_stem_tc"),         # 16-byte row chunks with a shifted second segment
    (3, 32, 3, 2, 1, 2, 224, 224, "k_conv_stem_s2"),        # the stem itself: image rows as the operand, bands of 4 rows
    (3, 32, 3, 2, 1, 3, 41, 304, "k_conv_stem_s2"),         # two segments per output row (the second ragged), odd height
    (3, 40, 3, 2, 1, 2, 17, 32, "k_conv_stem_s2"),          # 40 output channels (48 operand rows), last band partial
    (4, 16, 3, 2, 0, 2, 20, 40, "k_conv_stem_s2"),          # no padding, four channels: pixels already 8 bytes
    (1, 8, 3, 2, 1, 2, 21, 24, "k_conv_stem_s2"),           # one input channel
    (2, 128, 3, 2, 1, 1, 12, 16, "k_conv_stem_s2"),         # 128 output channels: one output row per band
    (3, 32, 3, 2, 1, 64, 66, 64, "k_conv_stem_s2"),         # more bands than resident CTAs: one or two bands per CTA
    (3, 264, 3, 2, 1, 1, 20, 20, "k_conv_smallcin_bf16"),   # too many outputs for one accumulator: CUDA cores
    (24, 32, 3, 2, 1, 2, 28, 28, "k_conv_tc_pairrows"),     # stride 2: one output per line, even/odd row boxes
    (32, 16, 5, 2, 2, 1, 30, 44, "k_conv_tc_pairrows"),     # stride 2, even padding, 5x5
    (16, 24, 3, 2, 0, 2, 17, 36, "k_conv_tc_pairrows"),     # stride 2, no padding, odd height
    (40, 32, 3, 2, 1, 2, 28, 28, "k_conv_tc"),              # stride 2 on parity planes (more than 32 channels)
    (96, 144, 5, 2, 2, 1, 56, 56, "k_conv_tc"),             # the widest stride-2 merged layer of the network: several tiles per image
    (48, 64, 7, 2, 3, 1, 31, 44, "k_conv_tc"),              # 7x7 stride 2, odd height: four even and three odd tap rows
    (48, 24, 5, 2, 1, 2, 22, 26, "k_conv_tc"),              # 5x5 stride 2 with padding 1: odd tap columns lead
    (72, 48, 3, 2, 0, 1, 17, 150, "k_conv_tc"),             # stride 2 without padding, two column strips
    (32, 16, 1, 1, 0, 2, 20, 24, "k_conv_tc_pairrows"),     # 1x1: one instruction per 32-byte K step
    (32, 96, 1, 1, 0, 2, 20, 24, "k_conv_tc_rows"),         # 1x1 expansion from few channels: one half-filled plane
    (16, 96, 1, 1, 0, 1, 40, 112, "k_conv_tc_rows"),        # 1x1 expansion from 16 channels, row tiles
    (32, 192, 3, 1, 1, 2, 28, 28, "k_conv_tc_rows"),        # 3x3 from few channels to more outputs than the pair rows take: two column strips, 110 KB of resident weights
    (16, 136, 5, 1, 2, 1, 12, 20, "k_conv_tc_rows"),        # the same with 16 channels and a 5x5 kernel, two passes
    (32, 40, 1, 1, 0, 2, 20, 24, "k_conv_tc"),              # 1x1 with 40 outputs: general kernel
    (16, 128, 3, 1, 1, 1, 12, 16, "k_conv_tc_pairrows"),    # N = 256: two accumulator slots, run-time channel loop
    (32, 64, 3, 2, 1, 1, 28, 28, "k_conv_tc_pairrows"),     # stride 2, 64 output channels
    (160, 200, 3, 1, 1, 5, 7, 7, "k_conv_tc_rows"),         # three planes (the last half full), two passes; few images: one per tile
    (96, 64, 1, 1, 0, 7, 7, 7, "k_conv_tc_rows"),           # 1x1 at 7 x 7, few images: one per tile
    (96, 64, 1, 1, 0, 733, 7, 7, "k_conv_tc_rows"),         # 1x1, a machine's worth of images: five per tile (147 tiles), the last group of three
    (160, 200, 3, 1, 1, 300, 7, 7, "k_conv_tc_rows"),       # 3x3 at 7 x 7 with more items than CTAs: three images per tile, two passes, runs cut by blocks (items shared by two CTAs)
    (960, 160, 1, 1, 0, 128, 7, 7, "k_conv_tc_rows"),       # deep projection of the network: two images per tile fill the machine (five would leave two thirds idle)
    (512, 512, 1, 1, 0, 6, 7, 7, "k_conv_tc_rows"),          # deep 1x1 with more than 256 outputs: two passes of 256 channels, one accumulator set
    (64, 48, 5, 1, 2, 1, 20, 70, "k_conv_tc_rows"),         # 5x5, two column strips, row tiles
    (384, 64, 3, 1, 1, 2, 14, 14, "k_conv_tc_rows"),        # six planes, whole image per tile
    (128, 128, 5, 1, 2, 2, 14, 14, "k_conv_tc_rows"),       # 5x5 with 128 outputs: two passes of 64 (weight stage limit)
    (96, 96, 7, 1, 3, 1, 14, 14, "k_conv_tc_rows"),         # 7x7: passes of at most 80 output channels
    (144, 32, 3, 1, 1, 1, 28, 28, "k_conv_tc_rows"),        # many channels, 32 outputs: rows kernel with resident weights, two strips of 14 x 14
    (80, 48, 3, 1, 1, 2, 14, 27, "k_conv_tc_rows"),         # ragged strips (14 + 13 columns), whole height per tile
    (64, 64, 3, 1, 1, 1, 33, 45, "k_conv_tc_rows"),         # three strips of 15 columns, row tiles of 13, 13 and 7
    (200, 24, 3, 1, 1, 2, 14, 14, "k_conv_tc"),             # many channels, fewer than 32 outputs: general kernel
    (192, 32, 1, 1, 0, 2, 28, 28, "k_conv_tc_rows"),        # 1x1 projection to 32 channels
])
def test_each_forward_kernel_against_the_oracle(dc, c_in, c_out, k, s, p, n, h, w, kernel):
    g = dc.geom(c_in, c_out, 1, k, s, p)
    assert dc.conv_kernel_name(n, h, w, g, dc.BF16) == kernel
    spec = I.make_layer(11, 0, c_in, c_out, k, s, p)
    lay = dc.DeviceLayer(spec)
    wf = torch.empty_like(lay.weight)
    bf = torch.empty(c_out, device="cuda")
    dc.fold_bn(lay, wf, bf)
    packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    dc.pack_weights(wf, g, dc.BF16, packed)
    x = I.make_input(12, (n, h, w, c_in), bf16=True)
    ho, wo = O.out_extent(h, k, s, p), O.out_extent(w, k, s, p)
    r = I.round_bf16(I.normal(13, 99, (n, ho, wo, c_out)))
    Wf, bfo = O.fold_bn(spec)
    lin = O.conv_direct(x.transpose(0, 3, 1, 2), Wf, bfo, k, s, p)
    # plain, and with skip input + ReLU6
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bf, dc.ACT_IDENTITY)
    assert_close(nchw(y), lin, TOL_BF16)
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bf, dc.ACT_RELU6, residual=dev(r, torch.bfloat16))
    assert_close(nchw(y), O.relu6(lin + r.transpose(0, 3, 1, 2)), TOL_BF16)


@pytest.mark.parametrize("c,k,s,p,n,h,w", [(64, 3, 1, 1, 2, 19, 21), (48, 3, 2, 1, 1, 20, 30), (32, 5, 1, 2, 1, 11, 13)])
def test_dwconv_stencil_without_activation(dc, c, k, s, p, n, h, w):
    """The stencil's instantiations without ReLU6 (tile widths 32 and 16, widths that are no multiple of a
    thread's item): negative and large outputs must come through unclamped."""
    spec = I.make_layer(18, 0, c, c, k, s, p, depthwise=True)
    lay = dc.DeviceLayer(spec)
    wf = torch.empty_like(lay.weight)
    bf = torch.empty(c, device="cuda")
    dc.fold_bn(lay, wf, bf)
    g = dc.geom(c, c, c, k, s, p)
    packed = torch.empty(dc.packed_bytes(g, dc.F32) // 4, dtype=torch.float32, device="cuda")
    dc.pack_weights(wf, g, dc.F32, packed)
    x = 4.0 * I.make_input(19, (n, h, w, c), bf16=True)
    x = I.round_bf16(x)
    ho, wo = O.out_extent(h, k, s, p), O.out_extent(w, k, s, p)
    gy = Guarded(torch, (n, ho, wo, c), torch.bfloat16, fill=float("nan"))
    dc.dwconv_forward(dev(x, torch.bfloat16), k, s, p, packed, bf, dc.ACT_IDENTITY, gy.t)
    assert dc.dwconv_status() == dc.OK
    gy.check("depthwise output")
    Wf, bfo = O.fold_bn(spec)
    ref = O.conv_direct(x.transpose(0, 3, 1, 2), Wf, bfo, k, s, p, groups=c)
    assert ref.min() < -1.0 and ref.max() > 6.5        # the case does exercise what ReLU6 would have cut
    assert_close(nchw(gy.t), ref, TOL_BF16, bf16=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("c,k,s,p,n,h,w", [(32, 3, 1, 1, 2, 12, 12), (96, 3, 2, 1, 1, 15, 17),
                                           (144, 3, 1, 1, 1, 9, 30), (20, 5, 1, 2, 1, 8, 8),
                                           (6, 3, 2, 1, 2, 7, 7), (960, 3, 1, 1, 2, 7, 7),
                                           # the shared-memory stencil: several row tiles with a ragged last one,
                                           # stride 2 with an odd height, 5x5 both strides, several images per tile
                                           (32, 3, 1, 1, 3, 150, 112), (96, 3, 2, 1, 2, 41, 112), (240, 5, 2, 2, 2, 28, 28),
                                           (384, 3, 1, 1, 21, 14, 14), (576, 5, 1, 2, 3, 14, 14), (24, 3, 1, 0, 2, 9, 20)])
def test_dwconv(dc, dtype, c, k, s, p, n, h, w):
    spec = I.make_layer(8, 0, c, c, k, s, p, depthwise=True)
    lay = dc.DeviceLayer(spec)
    wf = torch.empty_like(lay.weight)
    bf = torch.empty(c, device="cuda")
    dc.fold_bn(lay, wf, bf)
    g = dc.geom(c, c, c, k, s, p)
    packed = torch.empty(dc.packed_bytes(g, dc.F32) // 4, dtype=torch.float32, device="cuda")
    dc.pack_weights(wf, g, dc.F32, packed)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    x = I.make_input(9, (n, h, w, c), bf16=(dtype == "bf16"))
    ho, wo = O.out_extent(h, k, s, p), O.out_extent(w, k, s, p)
    gy = Guarded(torch, (n, ho, wo, c), tdt, fill=float("nan"))
    y = gy.t
    dc.dwconv_forward(dev(x, tdt), k, s, p, packed, bf, dc.ACT_RELU6, y)
    assert dc.dwconv_status() == dc.OK
    gy.check("depthwise output")
    Wf, bfo = O.fold_bn(spec)
    ref = O.relu6(O.conv_direct(x.transpose(0, 3, 1, 2), Wf, bfo, k, s, p, groups=c))
    assert_close(nchw(y), ref, TOL_F32 if dtype == "f32" else TOL_BF16, bf16=(dtype == "bf16"))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("c_in,c_out,t,s,n,h,w", [(24, 24, 6, 1, 2, 14, 14), (16, 24, 6, 2, 1, 16, 16),
                                                  (32, 16, 1, 1, 1, 12, 12)])
def test_block_forward(dc, dtype, c_in, c_out, t, s, n, h, w):
    specs = I.inverted_residual(10, 0, c_in, c_out, t, s, block=0)
    code = dc.F32 if dtype == "f32" else dc.BF16
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    keep, packed, biases = [], [], []
    for spec in specs:
        lay = dc.DeviceLayer(spec)
        wf = torch.empty_like(lay.weight)
        bf = torch.empty(spec.c_out, device="cuda")
        dc.fold_bn(lay, wf, bf)
        g = dc.geom(spec.c_in, spec.c_out, spec.groups, spec.k, spec.stride, spec.pad)
        pk = torch.empty(dc.packed_bytes(g, code), dtype=torch.uint8, device="cuda")
        dc.pack_weights(wf, g, code, pk)
        packed.append(pk)
        biases.append(bf)
        keep.append((lay, wf))
    has_exp = t != 1
    res = s == 1 and c_in == c_out
    if has_exp:
        pe, pd, pp = packed
        be, bd, bp = biases
    else:
        (pd, pp), (bd, bp) = packed, biases
        pe = be = None
    blk = dc.Block(c_in, c_in * t, c_out, int(has_exp), 3, s, 1, int(res), dc.ACT_RELU6, dc.ACT_RELU6,
                   pe.data_ptr() if has_exp else None, be.data_ptr() if has_exp else None,
                   pd.data_ptr(), bd.data_ptr(), pp.data_ptr(), bp.data_ptr())
    x = I.make_input(11, (n, h, w, c_in), bf16=(dtype == "bf16"))
    ho = O.out_extent(h, 3, s, 1)
    wo = O.out_extent(w, 3, s, 1)
    gy = Guarded(torch, (n, ho, wo, c_out), tdt, fill=float("nan"))
    gws = Guarded(torch, (max(dc.block_workspace_bytes(n, h, w, blk, code), dc.conv_workspace_bytes()),), torch.uint8,
                  fill=0)
    y, ws = gy.t, gws.t
    dc.block_forward(dev(x, tdt), blk, y, ws)
    assert dc.workspace_status(ws) == dc.OK
    gy.check("block output")
    gws.check("block workspace")
    cur = x.transpose(0, 3, 1, 2).astype(np.float64)
    skip = cur
    for spec in specs:
        Wf, bfo = O.fold_bn(spec)
        cur = O.conv_direct(cur, Wf, bfo, spec.k, spec.stride, spec.pad, spec.groups)
        if spec.act == "relu6":
            cur = O.relu6(cur)
    if res:
        cur = cur + skip
    # bf16: three roundings of the intermediate maps on the GPU side -> 3x the single-layer budget
    if dtype == "f32":
        assert_close(nchw(y), cur, TOL_F32, bf16=False)
    else:
        assert_close(nchw(y), cur, 3 * TOL_BF16, scale=3.0)


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_full_size_configs_on_every_image(dc, idx):
    """The batch-64/128 workloads in the launch configuration the benchmark times, every image
    against the oracle's sequential chain (each CTA owns a run of tiles somewhere in the batch, so a
    sample of images would leave most CTAs unchecked)."""
    case = I.chain_case(idx)
    g, wm, bm, packed = run_merge(dc, case.layers, case.residuals, packed_dtype=dc.BF16)
    W, b, k, s, p = O.merge_formula(case.layers, case.residuals)
    assert O.rel_l2(wm.cpu().numpy(), W) <= TOL_W and O.rel_l2(bm.cpu().numpy(), b) <= TOL_W
    x = case.x()
    y = run_conv(dc, dev(x, torch.bfloat16), g, packed, bm, dc.ACT_IDENTITY)
    ref = O.chain_forward_reordered(x.transpose(0, 3, 1, 2), case.layers, case.residuals)
    r, worst, max_abs = assert_close(nchw(y), ref, TOL_BF16, what=case.name)
    print("%s: rel-L2 %.3e, worst element at %.2f of its bound, max abs error %.3e" % (case.name, r, worst, max_abs))
    # per image as well: no single image may carry the whole error budget
    yn = nchw(y)
    for i in range(x.shape[0]):
        assert O.rel_l2(yn[i], ref[i]) <= TOL_BF16, (case.name, i)


def test_host_entry_point_matches_device_path(dc):
    case = I.chain_case(1, batch=4)
    arr, keep = dc.host_layer_array(case.layers)
    n, h, w, c = case.x_shape
    nbytes = dc.chain_host_workspace_bytes(arr, len(case.layers), case.residuals, n, h, w, dc.BF16)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    xh = torch.from_numpy(case.x()).to(torch.bfloat16).pin_memory()
    yh = torch.empty((n, h, w, 24), dtype=torch.bfloat16).pin_memory()
    dc.chain_forward_host(arr, len(case.layers), case.residuals, xh, dc.ACT_IDENTITY, yh, ws)
    assert dc.workspace_status(ws) == dc.OK
    ref = O.chain_forward_reordered(case.x().transpose(0, 3, 1, 2), case.layers, case.residuals)
    assert_close(yh.float().numpy().transpose(0, 3, 1, 2), ref, TOL_BF16)


def test_async_host_entry_point_overlaps_streams_and_matches_the_oracle(dc):
    # three batches in flight on three streams, each with its own workspace and pinned buffers
    arrs, outs, streams, cases = [], [], [], []
    for slot in range(3):
        case = I.chain_case(1, seed=20 + slot, batch=3)
        # slots 0 and 1: one pinned parameter block in the library's layout (a single transfer); slot 2: loose arrays
        arr, keep = dc.host_layer_array(case.layers, pinned=(slot < 2))
        n, h, w, c = case.x_shape
        nbytes = dc.chain_host_workspace_bytes(arr, len(case.layers), case.residuals, n, h, w, dc.BF16)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        xh = torch.from_numpy(case.x()).to(torch.bfloat16).pin_memory()
        yh = torch.zeros((n, h, w, 24), dtype=torch.bfloat16).pin_memory()
        st = torch.cuda.Stream()
        arrs.append((arr, keep, ws, xh))
        outs.append(yh); streams.append(st); cases.append(case)
    torch.cuda.synchronize()
    for slot in range(3):
        arr, keep, ws, xh = arrs[slot]
        dc.chain_forward_host_async(arr, len(cases[slot].layers), cases[slot].residuals, xh, dc.ACT_IDENTITY,
                                    outs[slot], ws, streams[slot])
    for slot in range(3):
        streams[slot].synchronize()
        assert dc.workspace_status(arrs[slot][2], streams[slot]) == dc.OK
        case = cases[slot]
        ref = O.chain_forward_reordered(case.x().transpose(0, 3, 1, 2), case.layers, case.residuals)
        assert_close(outs[slot].float().numpy().transpose(0, 3, 1, 2), ref, TOL_BF16)


def test_empty_and_degenerate_inputs_are_rejected_or_handled(dc):
    g = dc.geom(8, 8, 1, 3, 1, 1)
    packed = torch.zeros(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    x = torch.zeros((1, 1, 1, 8), dtype=torch.bfloat16, device="cuda")
    y = run_conv(dc, x, g, packed, None, dc.ACT_IDENTITY)            # 1x1 image, all taps but one in the padding
    assert y.shape == (1, 1, 1, 8) and float(y.float().abs().max()) == 0.0
    with pytest.raises(dc.DcError) as e:
        dc.conv_forward(torch.zeros((1, 2, 2, 8), dtype=torch.bfloat16, device="cuda"), dc.geom(8, 8, 1, 5, 1, 0),
                        packed, None, 0, None, y, new_ws(dc))
    assert e.value.status == dc.ERR_SHAPE
