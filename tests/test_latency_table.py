"""Latency table T[i][j] and the latency-optimal merge pattern (Sec. 4.1, Algorithm 1): the span
rules on CPU, the measured table and the pattern on a GPU."""
import pytest

from oracle import dp_oracle as P
from paper_2301_12187_b200 import inputs as I
from paper_2301_12187_b200 import latency as LT


def test_span_rules_on_mobilenet_v2():
    net = I.mobilenet_v2(seed=0, batch=2, res=32)
    L = len(net.layers)
    assert L == 52
    assert all(LT.span_residuals(net, i, i + 1) == [] for i in range(L))
    blocks = [b for b in net.blocks if b["residual"]]
    assert len(blocks) == 10
    f, l = blocks[0]["first"], blocks[0]["last"]
    assert LT.span_residuals(net, f, l + 1) == [(0, l - f)]              # the whole skip block: one group
    assert LT.span_residuals(net, f + 1, l + 1) is None                   # cuts through the skip
    assert LT.span_residuals(net, f - 1, l) is None
    assert LT.span_residuals(net, f - 1, l + 1) == [(1, l - f + 1)]       # a neighbour plus the whole block
    # stem (stride 2) followed by the first depthwise 3x3: a k > 1 layer after a stride-2 layer
    assert LT.span_residuals(net, 0, 2) is None
    # two consecutive skip blocks (3x3 twice -> 5x5) are fine, four would exceed k' = 7
    f2 = blocks[1]["first"] if blocks[1]["first"] == l + 1 else None
    three = [b for b in net.blocks if b["residual"]][1:4]                  # the 32-channel and 64-channel stages
    a, b = three[0]["first"], three[1]["last"]
    if three[1]["first"] == three[0]["last"] + 1:
        assert LT.span_residuals(net, a, b + 1) == [(0, 2), (3, 5)]
    shapes = LT.boundary_shapes(net)
    assert shapes[0] == (2, 32, 32, 3) and shapes[1] == (2, 16, 16, 32) and shapes[-1] == (2, 1, 1, 1280)
    assert f2 is None or f2 == l + 1


@pytest.mark.gpu
def test_measured_table_and_optimal_pattern():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    dc.lib()
    net = I.mobilenet_v2(seed=0, batch=8, res=64)
    L = len(net.layers)
    T, us = LT.measure_latency_table(net, unit_us=0.1, reps=5, max_span=4)
    for i in range(L):
        assert T[i][i + 1] < dc.DP_INF and us[i][i + 1] > 0
        for j in range(i + 2, L + 1):
            valid = j - i <= 4 and LT.span_residuals(net, i, j) is not None
            assert (T[i][j] < dc.DP_INF) == valid
    total, S, t_opt, split = LT.optimal_pattern(T, L)
    assert total == P.alg1(T, L)[0][0][L]
    assert total <= sum(T[i][i + 1] for i in range(L))
    bounds = [0] + S + [L]
    assert sum(T[a][b] for a, b in zip(bounds[:-1], bounds[1:])) == total
    assert all(T[a][b] < dc.DP_INF for a, b in zip(bounds[:-1], bounds[1:]))
    # a merged inverted-residual block replaces three launches over 6x wider maps: it must be in the table
    blk = [b for b in net.blocks if b["residual"]][0]
    assert T[blk["first"]][blk["last"] + 1] < dc.DP_INF
