"""Pins for the fp64 oracle: closed forms, brute force, and the shapes the paper states.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign or index, transposed operand, wrong tap offset) fails at least one of them.
None of the expected values comes from the oracle's own formulas re-typed: they
are textbook identities (matrix product, polynomial product), facts printed in
the paper (tests/golden/paper_facts.txt) or brute force by pure-Python loops.
"""
import itertools
import os
from types import SimpleNamespace

import numpy as np
import pytest

from oracle import dc_oracle as O
from paper_2301_12187_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")


def facts():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


def L(c_in, c_out, k, s=1, p=0, dw=False, rng=None, bn=True, bias=False):
    rng = rng or np.random.default_rng(0)
    g = c_in if dw else 1
    w = rng.standard_normal((c_out, c_in // g, k, k))
    b = rng.standard_normal(c_out) if bias else None
    bnp = None
    if bn:
        bnp = (rng.uniform(0.5, 1.5, c_out), rng.standard_normal(c_out) * 0.3,
               rng.standard_normal(c_out) * 0.3, rng.uniform(0.5, 1.5, c_out))
    return SimpleNamespace(c_in=c_in, c_out=c_out, groups=g, k=k, stride=s, pad=p, weight=w,
                           bias=b, bn=bnp, eps=1e-5)


def brute_conv(x, W, b, k, s, p, groups):
    """Seven nested Python loops straight from the definition (tiny inputs only)."""
    n, ci, h, w = x.shape
    co = W.shape[0]
    ho = (h + 2 * p - k) // s + 1
    wo = (w + 2 * p - k) // s + 1
    cgi, cgo = ci // groups, co // groups
    y = np.zeros((n, co, ho, wo))
    for a in range(n):
        for o in range(co):
            for Y in range(ho):
                for X in range(wo):
                    acc = 0.0 if b is None else b[o]
                    for i in range(cgi):
                        for u in range(k):
                            for v in range(k):
                                yy, xx = Y * s + u - p, X * s + v - p
                                if 0 <= yy < h and 0 <= xx < w:
                                    acc += W[o, i, u, v] * x[a, (o // cgo) * cgi + i, yy, xx]
                    y[a, o, Y, X] = acc
    return y


# ---- P13: the forward definition -----------------------------------------------------------


@pytest.mark.parametrize("k,s,p,groups", [(1, 1, 0, 1), (3, 1, 1, 1), (3, 2, 1, 1), (5, 1, 2, 1),
                                          (3, 1, 1, 4), (3, 2, 1, 4), (3, 2, 0, 2), (5, 2, 1, 1)])
def test_conv_direct_matches_python_loops(k, s, p, groups):
    rng = np.random.default_rng(k * 100 + s * 10 + p + groups)
    x = rng.standard_normal((2, 4, 7, 6))
    W = rng.standard_normal((4 if groups > 1 else 3, 4 // groups, k, k))
    b = rng.standard_normal(W.shape[0])
    assert np.allclose(O.conv_direct(x, W, b, k, s, p, groups), brute_conv(x, W, b, k, s, p, groups),
                       rtol=0, atol=1e-13)


def test_conv_1x1_is_a_matrix_product():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 5, 4, 3))
    W = rng.standard_normal((7, 5, 1, 1))
    b = rng.standard_normal(7)
    ref = np.einsum("oi,nihw->nohw", W[:, :, 0, 0], x) + b[None, :, None, None]
    assert np.allclose(O.conv_direct(x, W, b, 1, 1, 0), ref, atol=1e-13)


def test_conv_of_ones_sums_the_kernel_inside_and_less_on_the_border():
    W = np.arange(1, 10, dtype=float).reshape(1, 1, 3, 3)
    y = O.conv_direct(np.ones((1, 1, 5, 5)), W, np.array([0.5]), 3, 1, 1)
    assert y[0, 0, 2, 2] == 45.5
    assert y[0, 0, 0, 0] == 0.5 + 5 + 6 + 8 + 9          # taps that look at the padding drop out
    assert y[0, 0, 4, 4] == 0.5 + 1 + 2 + 4 + 5


def test_no_kernel_flip_cross_correlation():
    x = np.zeros((1, 1, 5, 5))
    x[0, 0, 1, 3] = 1.0                                   # impulse up-right of the centre
    W = np.arange(9, dtype=float).reshape(1, 1, 3, 3)
    y = O.conv_direct(x, W, None, 3, 1, 1)
    # output (2,2) looks at input (2+u-1, 2+v-1): the impulse is at u=0, v=2
    assert y[0, 0, 2, 2] == W[0, 0, 0, 2]


def test_depthwise_with_delta_kernel_is_a_copy_and_lift_is_exact():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 3, 6, 6))
    Wd = np.zeros((3, 1, 3, 3))
    Wd[:, 0, 1, 1] = 1.0
    assert np.array_equal(O.conv_direct(x, Wd, None, 3, 1, 1, groups=3), x)
    Wd = rng.standard_normal((3, 1, 3, 3))
    dense = O.lift_depthwise(Wd)
    assert dense.shape == (3, 3, 3, 3) and dense[0, 1].max() == 0 and np.array_equal(dense[2, 2], Wd[2, 0])
    assert np.allclose(O.conv_direct(x, Wd, None, 3, 2, 1, groups=3),
                       O.conv_direct(x, dense, None, 3, 2, 1), atol=1e-13)      # P6


def test_relu6():
    assert list(O.relu6(np.array([-1.0, 0.0, 3.5, 6.0, 7.0]))) == [0.0, 0.0, 3.5, 6.0, 6.0]


# ---- P12: BN fold ----------------------------------------------------------------------------


def test_fold_bn_equals_literal_bn():
    rng = np.random.default_rng(3)
    lay = L(3, 5, 3, 1, 1, rng=rng, bias=True)
    x = rng.standard_normal((2, 3, 6, 6))
    lit = O.batchnorm(O.conv_direct(x, lay.weight, lay.bias, 3, 1, 1), lay.bn, lay.eps)
    Wf, bf = O.fold_bn(lay)
    assert np.allclose(O.conv_direct(x, Wf, bf, 3, 1, 1), lit, atol=1e-12)
    # hand value for one channel: g = gamma/sqrt(var+eps)
    g = lay.bn[0][1] / np.sqrt(lay.bn[3][1] + lay.eps)
    assert np.isclose(bf[1], lay.bn[1][1] + (lay.bias[1] - lay.bn[2][1]) * g, atol=1e-15)
    assert np.allclose(Wf[1], g * lay.weight[1], atol=1e-15)


def test_fold_bn_identity_statistics():
    lay = L(2, 2, 1, bn=False)
    lay.bn = (np.ones(2), np.zeros(2), np.zeros(2), np.ones(2) - 1e-5)
    Wf, bf = O.fold_bn(lay)
    assert np.allclose(Wf, lay.weight, atol=1e-15) and np.allclose(bf, 0)


def test_batchnorm_literal_values():
    x = np.array([1.0, 3.0]).reshape(1, 1, 1, 2)
    y = O.batchnorm(x, (np.array([2.0]), np.array([0.5]), np.array([1.0]), np.array([4.0 - 1e-5])), 1e-5)
    assert np.allclose(y.ravel(), [0.5, 2.5], atol=1e-14)


# ---- P1/P2: geometry -------------------------------------------------------------------------


def test_geometry_closed_form_and_extents():
    rng = np.random.default_rng(4)
    for _ in range(200):
        n = rng.integers(1, 6)
        ks = rng.choice([1, 3, 5], n)
        ss = rng.choice([1, 2], n)
        ps = rng.integers(0, 3, n)
        lays = [SimpleNamespace(k=int(k), stride=int(s), pad=int(p)) for k, s, p in zip(ks, ss, ps)]
        k, s, p = O.compose_geometry(lays)
        cum = np.concatenate([[1], np.cumprod(ss)[:-1]])
        assert k - 1 == int(((ks - 1) * cum).sum())
        assert p == int((ps * cum).sum())
        assert s == int(np.prod(ss))
        # reordered chain (pad once by p', then pad 0) and merged conv agree on the output extent
        for h in range(k, k + 12):
            e = h + 2 * p
            for lay in lays:
                e = O.out_extent(e, lay.k, lay.stride, 0)
            assert e == O.out_extent(h, k, s, p)


def test_paper_shapes():
    f = facts()
    rng = np.random.default_rng(5)
    for K in (1, 3, 5):
        W = O.merge_pair(rng.standard_normal((5, 4, K, K)), 1, rng.standard_normal((3, 5, K, K)))
        assert W.shape[2] == 2 * K - 1 == eval(f["two_KxK_stride1_merged_kernel"], {"K": K})
        assert [W.shape[1], W.shape[0]] == [int(t) for t in f["fig1_merged_channels_in_out"].split()]
    assert O.compose_geometry([SimpleNamespace(k=3, stride=1, pad=1)] * 2)[0] == int(f["two_3x3_merged_kernel"])
    a, m, c = (int(t) for t in f["pointwise_pair_channels"].split())
    W1, W2 = rng.standard_normal((m, a, 1, 1)), rng.standard_normal((c, m, 1, 1))
    W = O.merge_pair(W1, 1, W2)
    assert W.shape == (c, a, 1, 1)
    assert np.linalg.matrix_rank(W[:, :, 0, 0]) == 1                     # 100 -> 1 -> 100 is rank one


def test_mobilenet_table_matches_paper_flops():
    net = I.mobilenet_v2(batch=1)
    h = 224
    macs = 0
    for lay in net.layers:
        h = O.out_extent(h, lay.k, lay.stride, lay.pad) if lay.role != "project" and lay.role != "expand" \
            and lay.role != "head" else h
        macs += h * h * lay.c_out * (lay.c_in // lay.groups) * lay.k * lay.k
    macs += 1280 * 1000                                                  # classifier, not built here
    assert abs(macs / 1e6 - float(facts()["mbv2_1_0_mflops_bn_fused"])) < 3.0
    assert len(net.layers) == 52 and sum(1 for l in net.layers if l.act == "relu6") == 35


# ---- P3/P4/P5/P11: the pairwise formula ----------------------------------------------------------


def test_pointwise_pair_is_matrix_product_with_bias():
    rng = np.random.default_rng(6)
    W1, W2 = rng.standard_normal((6, 4, 1, 1)), rng.standard_normal((5, 6, 1, 1))
    b1, b2 = rng.standard_normal(6), rng.standard_normal(5)
    assert np.allclose(O.merge_pair(W1, 1, W2)[:, :, 0, 0], W2[:, :, 0, 0] @ W1[:, :, 0, 0], atol=1e-13)
    assert np.allclose(O.merge_bias(b1, W2, b2), W2[:, :, 0, 0] @ b1 + b2, atol=1e-13)


def test_single_channel_3x3_pair_is_polynomial_product():
    ones = np.ones((1, 1, 3, 3))
    tri = np.array([1, 2, 3, 2, 1.0])
    assert np.array_equal(O.merge_pair(ones, 1, ones)[0, 0], np.outer(tri, tri))
    rng = np.random.default_rng(7)
    a, b = rng.standard_normal((3, 3)), rng.standard_normal((3, 3))
    full = np.zeros((5, 5))
    for u in range(3):
        for v in range(3):
            full[u:u + 3, v:v + 3] += b[u, v] * a                         # 2-D polynomial product
    assert np.allclose(O.merge_pair(a.reshape(1, 1, 3, 3), 1, b.reshape(1, 1, 3, 3))[0, 0], full, atol=1e-14)


def test_stride_dilates_the_second_kernel():
    rng = np.random.default_rng(8)
    W1 = rng.standard_normal((2, 2, 1, 1))
    W2 = rng.standard_normal((2, 2, 3, 3))
    W = O.merge_pair(W1, 2, W2)                                           # 1x1 stride 2, then 3x3
    assert W.shape[2:] == (5, 5)
    mask = np.zeros((5, 5), bool)
    mask[::2, ::2] = True
    assert np.all(W[:, :, ~mask] == 0) and np.all(W[:, :, mask] != 0)
    assert np.allclose(W[:, :, ::2, ::2], np.einsum("ocuv,ci->oiuv", W2, W1[:, :, 0, 0]), atol=1e-13)
    W3 = O.merge_pair(rng.standard_normal((2, 2, 3, 3)), 2, W1)           # 3x3 stride 2, then 1x1
    assert W3.shape[2:] == (3, 3)


def test_bias_uses_sum_over_taps():
    W2 = np.arange(18, dtype=float).reshape(1, 2, 3, 3)
    out = O.merge_bias(np.array([2.0, -1.0]), W2, np.array([0.25]))
    assert out[0] == 0.25 + 2.0 * W2[0, 0].sum() - 1.0 * W2[0, 1].sum()


def test_linearity_and_associativity():
    rng = np.random.default_rng(9)
    A, B, C = (rng.standard_normal(s) for s in [(3, 2, 3, 3), (4, 3, 1, 1), (2, 4, 3, 3)])
    assert np.allclose(O.merge_pair(2.5 * A, 1, B), 2.5 * O.merge_pair(A, 1, B), atol=1e-13)
    left = O.merge_pair(O.merge_pair(A, 2, B), 2, C)                      # A has stride 2
    right = O.merge_pair(A, 2, O.merge_pair(B, 1, C))
    assert np.allclose(left, right, atol=1e-12)


# ---- P7: identity / skip ------------------------------------------------------------------------


def test_identity_kernel_and_skip_fold():
    rng = np.random.default_rng(10)
    delta = np.zeros((3, 3, 3, 3))
    for c in range(3):
        delta[c, c, 1, 1] = 1.0
    A = rng.standard_normal((3, 3, 3, 3))
    assert np.allclose(O.merge_pair(A, 1, delta)[:, :, 1:4, 1:4], A) and np.allclose(O.merge_pair(delta, 1, A)[:, :, 1:4, 1:4], A)
    zero = L(3, 3, 3, 1, 1, bn=False)
    zero.weight = np.zeros_like(zero.weight)
    W, b, k, s, p = O.merge_formula([zero], [(0, 0)])
    assert np.array_equal(W, delta) and np.all(b == 0)
    lays = [L(3, 6, 1, rng=rng), L(6, 6, 3, 1, 1, dw=True, rng=rng), L(6, 3, 1, rng=rng)]
    x = rng.standard_normal((1, 3, 6, 6))
    W, b, k, s, p = O.merge_formula(lays, [(0, 2)])
    Wn, bn_, *_ = O.merge_formula(lays, [])
    assert np.allclose(W - Wn, delta, atol=1e-14) and np.allclose(b, bn_)
    assert np.allclose(O.conv_direct(x, W, b, k, s, p),
                       O.conv_direct(x, Wn, bn_, k, s, p) + x, atol=1e-12)  # f(x) + x, App. E.1


# ---- P8/P9/P10: exactness, impulse brute force, the padding contract -------------------------


TOPOLOGIES = {
    "cfg0": (lambda r: [L(4, 12, 1, rng=r), L(12, 12, 3, 1, 1, dw=True, rng=r), L(12, 5, 1, rng=r)], []),
    "cfg1": (lambda r: [L(4, 12, 1, rng=r), L(12, 12, 3, 1, 1, dw=True, rng=r), L(12, 4, 1, rng=r)], [(0, 2)]),
    "cfg2": (lambda r: [L(4, 12, 1, rng=r), L(12, 12, 3, 2, 1, dw=True, rng=r), L(12, 6, 1, rng=r)], []),
    "cfg3": (lambda r: [L(4, 8, 1, rng=r), L(8, 8, 3, 1, 1, dw=True, rng=r), L(8, 4, 1, rng=r),
                        L(4, 8, 1, rng=r), L(8, 8, 3, 1, 1, dw=True, rng=r), L(8, 4, 1, rng=r)], [(0, 2), (3, 5)]),
    "dense3x3_pair": (lambda r: [L(3, 4, 3, 1, 1, rng=r, bias=True), L(4, 2, 3, 1, 1, rng=r, bias=True)], []),
    "s2_then_1x1_then_dw": (lambda r: [L(3, 4, 3, 2, 1, rng=r), L(4, 4, 1, rng=r), L(4, 4, 3, 1, 1, dw=True, rng=r)], []),
    "skip_in_the_middle": (lambda r: [L(3, 4, 3, 2, 1, rng=r), L(4, 4, 3, 1, 1, dw=True, rng=r), L(4, 2, 1, rng=r)], [(1, 1)]),
}


@pytest.mark.parametrize("name", sorted(TOPOLOGIES))
def test_merged_conv_equals_reordered_chain(name):
    make, res = TOPOLOGIES[name]
    rng = np.random.default_rng(11)
    lays = make(rng)
    x = rng.standard_normal((2, lays[0].c_in, 11, 9))
    W, b, k, s, p = O.merge_formula(lays, res)
    assert O.rel_l2(O.conv_direct(x, W, b, k, s, p), O.chain_forward_reordered(x, lays, res)) < 1e-12


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "dense3x3_pair", "skip_in_the_middle"])
def test_impulse_probing_recovers_the_formula(name):
    make, res = TOPOLOGIES[name]
    rng = np.random.default_rng(12)
    lays = make(rng)
    if name.startswith("cfg"):                                            # keep the brute force tiny
        lays = [L(2, 4, 1, rng=rng), L(4, 4, 3, 2 if name == "cfg2" else 1, 1, dw=True, rng=rng),
                L(4, 2 if name != "cfg2" else 3, 1, rng=rng)]
    Wf, bf, k, s, p = O.merge_formula(lays, res)
    Wi, bi, ki, si, pi = O.merge_by_impulse(lays, res)
    assert (k, s, p) == (ki, si, pi)
    assert O.rel_l2(Wi, Wf) < 1e-12 and O.rel_l2(bi, bf) < 1e-12


def test_padding_contract_two_3x3():
    """Fig. 5 / App. E.2: pad 1 + 1 differs from the merged 5x5 on the border, pad 2 first is equal."""
    f = facts()
    rng = np.random.default_rng(13)
    p_each, p_first = int(f["two_3x3_pad_each"]), int(f["two_3x3_pad_first"])
    lays = [L(2, 3, 3, 1, p_each, rng=rng, bn=False), L(3, 2, 3, 1, p_each, rng=rng, bn=False)]
    x = rng.standard_normal((1, 2, 8, 8))
    W, b, k, s, p = O.merge_formula(lays)
    assert (k, p) == (5, p_first)
    merged = O.conv_direct(x, W, b, k, s, p)
    orig = O.chain_forward_original(x, lays)
    reord = O.chain_forward_reordered(x, lays)
    assert np.allclose(merged, reord, atol=1e-12)
    assert np.allclose(merged[:, :, 1:-1, 1:-1], orig[:, :, 1:-1, 1:-1], atol=1e-12)
    ring = np.ones(merged.shape, bool)
    ring[:, :, 1:-1, 1:-1] = False
    assert np.abs(merged - orig)[ring].max() > 1e-3
    # "pad 2 on the first conv" written with plain calls
    two = O.conv_direct(O.conv_direct(x, lays[0].weight, None, 3, 1, p_first), lays[1].weight, None, 3, 1, 0)
    assert np.allclose(two, merged, atol=1e-12)


def test_border_differs_when_first_pointwise_has_a_shift():
    rng = np.random.default_rng(14)
    lays = TOPOLOGIES["cfg0"][0](rng)
    x = rng.standard_normal((1, 4, 8, 8))
    W, b, k, s, p = O.merge_formula(lays)
    merged, orig = O.conv_direct(x, W, b, k, s, p), O.chain_forward_original(x, lays)
    assert np.allclose(merged[:, :, 1:-1, 1:-1], orig[:, :, 1:-1, 1:-1], atol=1e-12)
    assert np.abs(merged - orig).max() > 1e-3


def test_planted_mistakes_are_caught():
    """A dropped bias term, a transposed tap and a wrong stride each break exactness."""
    rng = np.random.default_rng(15)
    lays = TOPOLOGIES["cfg2"][0](rng)
    x = rng.standard_normal((1, 4, 9, 9))
    W, b, k, s, p = O.merge_formula(lays)
    ref = O.chain_forward_reordered(x, lays)
    assert O.rel_l2(O.conv_direct(x, W, b, k, s, p), ref) < 1e-12
    assert O.rel_l2(O.conv_direct(x, W.transpose(0, 1, 3, 2), b, k, s, p), ref) > 1e-3
    assert O.rel_l2(O.conv_direct(x, W, 0 * b, k, s, p), ref) > 1e-3
    assert O.conv_direct(x, W, b, k, 1, p).shape != ref.shape


# ---- the data module itself ------------------------------------------------------------------------


def test_generator_is_counter_based_and_has_the_stated_moments():
    a = I.normal(0, 5, (1000,))
    b = I.normal(0, 5, (2000,))
    assert np.array_equal(a, b[:1000])
    big = I.normal(1, 6, (200000,), std=0.5)
    assert abs(big.mean()) < 0.01 and abs(big.std() - 0.5) < 0.01
    u = I.uniform(2, 7, (200000,), 0.5, 1.5)
    assert u.min() >= 0.5 and u.max() < 1.5 and abs(u.mean() - 1.0) < 0.01
    lay = I.chain_case(1).layers[1]
    assert abs(lay.weight.std() - (1 / 9) ** 0.5) < 0.02                 # depthwise fan_in = 9


def test_round_bf16_ties_to_even():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -(1.0 + 2 ** -8 + 2 ** -20)],
                 dtype=np.float32)
    r = I.round_bf16(v)
    assert list(r) == [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -(1.0 + 2 ** -7)]
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)


def test_plan_is_deterministic_and_respects_the_rules():
    net = I.mobilenet_v2(batch=1)
    acts, ops = I.plan_spans(net, seed=0)
    acts2, ops2 = I.plan_spans(net, seed=0)
    assert acts == acts2 and [o.layers for o in ops] == [o.layers for o in ops2]
    assert sum(1 for a in acts if a == "relu6") == 35 - 17 and acts[-1] == "relu6"
    covered = list(itertools.chain.from_iterable(o.layers for o in ops))
    assert covered == list(range(52))
    for o in ops:
        lays = [net.layers[i] for i in o.layers]
        assert all(acts[i] is None for i in o.layers[:-1])
        seen_s2 = False
        for lay in lays:
            assert not (seen_s2 and lay.k > 1)                            # App. B.2
            seen_s2 = seen_s2 or lay.stride > 1
        assert O.compose_geometry(lays)[0] <= 7
        for f, l in o.residuals:
            blk = net.blocks[lays[f].block]
            assert blk["residual"] and o.layers[f] == blk["first"] and o.layers[l] == blk["last"]
    assert any(o.add_from >= -1 for o in ops) and any(o.residuals for o in ops)
    assert I.plan_spans(net, seed=1)[0] != acts
