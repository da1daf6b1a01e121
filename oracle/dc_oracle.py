"""fp64 CPU oracle for convolution merging -- TEST INFRASTRUCTURE, not product code.

What the hot path of arXiv 2301.12187 computes, written out plainly: fold each
batch-norm into its convolution, compose a run of convolutions whose
intermediate activations are identities into one convolution (Sec. 3, Eq. 1),
fold a skip addition in as an identity kernel (App. E.1), and run the result.
The reference semantics of "the sequential chain" is the padding-reordered
chain of App. E.2: all zero padding of a run is applied before its first
convolution.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares no code with the CUDA library and never imports it.
The heavy loops live in dc_oracle.c (plain C, fp64); this file sequences them.

Layout: feature maps are NCHW float64 numpy arrays, kernels are
[c_out][c_in/groups][k][k].  A layer is any object with the attributes
  c_in, c_out, groups, k, stride, pad, weight, bias (or None),
  bn (None or a tuple gamma, beta, mean, var), eps.
A residual group is a pair (first, last) of layer indices:
  y = chain[first..last](x) + x.

Pinned by tests/test_oracle_pins.py (closed forms, brute force, the paper's
worked shapes).  No function here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dc_oracle.c")
_LIB = os.path.join(_HERE, "libdc_oracle.so")

_D = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile dc_oracle.c into libdc_oracle.so next to it (gcc, -O2, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.dco_num_threads.restype = ctypes.c_int
        lib.dco_out_extent.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(_D)


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def num_threads() -> int:
    return int(_c().dco_num_threads())


def set_num_threads(t: int) -> None:
    _c().dco_set_num_threads(ctypes.c_int(int(t)))


# --------------------------------------------------------------------------- elementary steps


def out_extent(h: int, k: int, s: int, p: int) -> int:
    """floor((h + 2p - k)/s) + 1 (0 if the kernel does not fit)."""
    return int(_c().dco_out_extent(int(h), int(k), int(s), int(p)))


def fold_bn(layer):
    """O1 -- BN fusion (Sec. 2 'TensorRT', Sec. 5.1 'Evaluation').  Returns (W~, b~) in fp64."""
    W = _f64(layer.weight)
    b = _f64(layer.bias)
    c_out = W.shape[0]
    if layer.bn is None:
        return W.copy(), (b.copy() if b is not None else np.zeros(c_out))
    gamma, beta, mean, var = (_f64(t) for t in layer.bn)
    Wo = np.empty_like(W)
    bo = np.empty(c_out)
    _c().dco_fold_bn(_p(W), _p(b), _p(gamma), _p(beta), _p(mean), _p(var),
                     ctypes.c_double(float(layer.eps)), c_out, int(W.size // c_out), _p(Wo), _p(bo))
    return Wo, bo


def batchnorm(x, bn, eps):
    """Eval-mode BN applied literally to an NCHW map (what fold_bn is checked against)."""
    x = _f64(x).copy()
    gamma, beta, mean, var = (_f64(t) for t in bn)
    n, c, h, w = x.shape
    _c().dco_batchnorm(_p(x), n, c, h * w, _p(gamma), _p(beta), _p(mean), _p(var),
                       ctypes.c_double(float(eps)))
    return x


def conv_direct(x, W, bias, k, s, p, groups=1):
    """O2 -- direct convolution by the definition (Sec. 3, f_theta); NCHW fp64."""
    x = _f64(x)
    W = _f64(W)
    bias = _f64(bias)
    n, c_in, h, w = x.shape
    c_out = W.shape[0]
    assert W.shape == (c_out, c_in // groups, k, k), (W.shape, c_in, groups, k)
    ho, wo = out_extent(h, k, s, p), out_extent(w, k, s, p)
    y = np.zeros((n, c_out, ho, wo))
    _c().dco_conv_direct(_p(x), n, c_in, h, w, _p(W), _p(bias), c_out, k, s, p, groups, _p(y))
    return y


def relu6(x):
    """O7 -- min(max(v, 0), 6), the MobileNetV2 activation."""
    return np.minimum(np.maximum(x, 0.0), 6.0)


def lift_depthwise(Wdw):
    """Depthwise [c][1][k][k] as the dense kernel delta(o,i)*Wdw[o]."""
    Wdw = _f64(Wdw)
    c, one, k, _ = Wdw.shape
    assert one == 1
    W = np.empty((c, c, k, k))
    _c().dco_lift_depthwise(_p(Wdw), c, k, _p(W))
    return W


def merge_pair(W1, s1, W2):
    """theta2 (*) theta1 for dense operands (Sec. 3; Eq. 1): k' = k1 + (k2-1)*s1."""
    W1 = _f64(W1)
    W2 = _f64(W2)
    c1, c0, k1, _ = W1.shape
    c2, c1b, k2, _ = W2.shape
    assert c1 == c1b, (W1.shape, W2.shape)
    kk = k1 + (k2 - 1) * s1
    out = np.empty((c2, c0, kk, kk))
    _c().dco_merge_pair(_p(W1), c0, c1, k1, int(s1), _p(W2), c2, k2, _p(out))
    return out


def merge_bias(b1, W2, b2):
    """b'[o] = b2[o] + sum_c (sum_taps W2[o,c]) b1[c]."""
    W2 = _f64(W2)
    b1 = _f64(b1)
    b2 = _f64(b2)
    c2, c1, k2, _ = W2.shape
    out = np.empty(c2)
    _c().dco_merge_bias(_p(b1), c1, _p(W2), _p(b2), c2, k2, _p(out))
    return out


# --------------------------------------------------------------------------- geometry


def compose_geometry(layers):
    """Fold (k, s, p) pairwise along the chain: k' = k1+(k2-1)s1, s' = s1 s2, p' = p1+p2 s1."""
    k, s, p = layers[0].k, layers[0].stride, layers[0].pad
    for L in layers[1:]:
        k, p, s = k + (L.k - 1) * s, p + L.pad * s, s * L.stride
    return k, s, p


def _group_starting_at(residuals, idx):
    for first, last in residuals or ():
        if first == idx:
            return first, last
    return None


# --------------------------------------------------------------------------- sequential chains


def _apply_layer(x, L, pad):
    """One conv with the given zero padding, then its BN applied literally."""
    y = conv_direct(x, L.weight, L.bias, L.k, L.stride, pad, L.groups)
    if L.bn is not None:
        y = batchnorm(y, L.bn, L.eps)
    return y


def chain_forward_reordered(x, layers, residuals=(), final_act=None):
    """O3 -- the sequential chain after padding reordering (App. E.2).

    x is zero-padded once by p' = sum_i p_i prod_{j<i} s_j, then every layer
    runs with no padding, BN literal, identities in between.  A skip addition
    adds the input of the group's first layer, centre-cropped to the group's
    output size (App. E.1: f(x) + x).
    """
    x = _f64(x)
    _, _, p_tot = compose_geometry(layers)
    cur = np.pad(x, ((0, 0), (0, 0), (p_tot, p_tot), (p_tot, p_tot)))
    i = 0
    while i < len(layers):
        grp = _group_starting_at(residuals, i)
        if grp is None:
            cur = _apply_layer(cur, layers[i], 0)
            i += 1
            continue
        first, last = grp
        skip = cur
        for j in range(first, last + 1):
            cur = _apply_layer(cur, layers[j], 0)
        ch = (skip.shape[2] - cur.shape[2]) // 2
        cw = (skip.shape[3] - cur.shape[3]) // 2
        assert skip.shape[2] - cur.shape[2] == 2 * ch and skip.shape[1] == cur.shape[1]
        cur = cur + skip[:, :, ch:ch + cur.shape[2], cw:cw + cur.shape[3]]
        i = last + 1
    if final_act == "relu6":
        cur = relu6(cur)
    return cur


def chain_forward_original(x, layers, residuals=(), final_act=None):
    """O4 -- the chain before padding reordering: each layer pads for itself."""
    cur = _f64(x)
    i = 0
    while i < len(layers):
        grp = _group_starting_at(residuals, i)
        if grp is None:
            cur = _apply_layer(cur, layers[i], layers[i].pad)
            i += 1
            continue
        first, last = grp
        skip = cur
        for j in range(first, last + 1):
            cur = _apply_layer(cur, layers[j], layers[j].pad)
        assert skip.shape == cur.shape
        cur = cur + skip
        i = last + 1
    if final_act == "relu6":
        cur = relu6(cur)
    return cur


# --------------------------------------------------------------------------- merging


def _dense_folded(L):
    """BN-folded kernel of one layer as a dense [c_out][c_in][k][k] kernel plus bias."""
    W, b = fold_bn(L)
    if L.groups != 1:
        assert L.groups == L.c_in == L.c_out, "only dense or depthwise layers"
        W = lift_depthwise(W)
    return W, b


def _merge_run(layers):
    """Left-to-right pairwise merge of a run without skip additions."""
    W, b = _dense_folded(layers[0])
    s = layers[0].stride
    for L in layers[1:]:
        W2, b2 = _dense_folded(L)
        b = merge_bias(b, W2, b2)
        W = merge_pair(W, s, W2)
        s *= L.stride
    return W, b, s


def merge_formula(layers, residuals=()):
    """O5 -- merged conv (W', b', k', s', p') by the pairwise formula (Sec. 3; Eq. 1).

    Each residual group is merged to a single conv first and receives its
    identity kernel at tap ((k_blk-1)/2, (k_blk-1)/2) (App. E.1); the pieces are
    then composed left to right.
    """
    W = b = None
    s = 1
    i = 0
    while i < len(layers):
        grp = _group_starting_at(residuals, i)
        if grp is None:
            Wp, bp = _dense_folded(layers[i])
            sp = layers[i].stride
            i += 1
        else:
            first, last = grp
            Wp, bp, sp = _merge_run(layers[first:last + 1])
            kb = Wp.shape[2]
            assert sp == 1 and Wp.shape[0] == Wp.shape[1] and kb % 2 == 1, "skip needs f(x) ~ x"
            c = (kb - 1) // 2
            for o in range(Wp.shape[0]):
                Wp[o, o, c, c] += 1.0
            i = last + 1
        if W is None:
            W, b, s = Wp, bp, sp
        else:
            b = merge_bias(b, Wp, bp)
            W = merge_pair(W, s, Wp)
            s *= sp
    k, s_chk, p = compose_geometry(layers)
    assert W.shape[2] == k and s == s_chk
    return W, b, k, s, p


def merge_by_impulse(layers, residuals=()):
    """O6 -- merged conv read off impulse responses of the reordered chain (brute force).

    Independent of merge_formula: with every bias and BN shift zeroed the chain
    is linear, so W'[o,i,u',v'] is the response at one interior output position
    to a unit impulse in input channel i at the position tap (u',v') looks at;
    b' is the response to x = 0 with the shifts restored.  Tiny chains only.
    """
    k, s, p = compose_geometry(layers)
    lin = []
    for L in layers:
        bn = None
        if L.bn is not None:
            g, _, _, v = L.bn
            bn = (g, np.zeros_like(np.asarray(g, dtype=np.float64)),
                  np.zeros_like(np.asarray(g, dtype=np.float64)), v)
        lin.append(SimpleNamespace(c_in=L.c_in, c_out=L.c_out, groups=L.groups, k=L.k,
                                   stride=L.stride, pad=L.pad, weight=L.weight, bias=None, bn=bn,
                                   eps=L.eps))
    y0 = -(-p // s)                      # first output row whose window starts inside the image
    base = y0 * s - p
    hc = base + k + s                    # canvas: window of output y0 fits with room to spare
    c_in, c_out = layers[0].c_in, layers[-1].c_out
    W = np.zeros((c_out, c_in, k, k))
    for i in range(c_in):
        for u in range(k):
            for v in range(k):
                x = np.zeros((1, c_in, hc, hc))
                x[0, i, base + u, base + v] = 1.0
                y = chain_forward_reordered(x, lin, residuals)
                W[:, i, u, v] = y[0, :, y0, y0]
    yb = chain_forward_reordered(np.zeros((1, c_in, hc, hc)), layers, residuals)
    b = yb[0, :, y0, y0].copy()
    return W, b, k, s, p


def rel_l2(a, b):
    """||a-b||_2 / ||b||_2 with b the reference."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    nb = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / (nb if nb > 0 else 1.0)
