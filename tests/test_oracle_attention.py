"""Pins of the fixed-order decode attention in the oracle (an extension: the paper keeps vendor attention
and names fixed-order attention as the outstanding source of residual divergence).  The C oracle is
checked against things other than itself: hand-derived values that separate candidate orders, closed
forms, an exact-rational re-implementation (oracle/exact.py, Python fractions), the mathematical
definition in FP64, and the exponential against the correctly rounded one within a stated bound."""
import math

import numpy as np
import pytest

from oracle import exact, oracle

T24 = float(2 ** 24)


def f32(x):
    return float(np.float32(x))


# ---- the exponential ---------------------------------------------------------------------------------
def test_exp_special_values():
    assert oracle.exp_det(0.0) == 1.0 and oracle.exp_det(-0.0) == 1.0
    assert oracle.exp_det(-104.5) == 0.0 and oracle.exp_det(-1000.0) == 0.0
    assert oracle.exp_det(-103.9) == 2.0 ** -149          # the smallest subnormal
    # n * ln2 exactly representable cases: exp(-ln2 * n) is close to 2^-n
    for n in (1, 10, 25, 100, 126, 127, 140):
        x = f32(-n * math.log(2.0))
        assert abs(oracle.exp_det(x) / math.exp(x) - 1.0) < 1e-5 or n > 126


def test_exp_within_two_ulp_of_the_real_exponential():
    xs = np.concatenate([-np.linspace(0, 87.3, 200001), -np.logspace(-30, 1.9, 5000)]).astype(np.float32)
    worst = 0.0
    for x in xs[::7]:
        got = oracle.exp_det(float(x))
        want = math.exp(float(x))
        ulp = 2.0 ** (math.floor(math.log2(want)) - 23)
        worst = max(worst, abs(got - want) / ulp)
    assert worst < 2.0, worst
    # subnormal results: within one subnormal spacing
    for x in np.linspace(-103.9, -87.4, 500).astype(np.float32):
        assert abs(oracle.exp_det(float(x)) - math.exp(float(x))) <= 2.0 ** -149


def test_exp_equals_the_exact_rational_replay():
    rng = np.random.default_rng(5)
    xs = np.concatenate([-rng.random(300) * 104.0, -rng.random(100) * 1e-3, [-87.33654, -88.0, -103.97, -0.34657359]])
    for x in xs.astype(np.float32):
        assert oracle.exp_det(float(x)) == exact.exp_det(float(x)), float(x)


def test_exp_is_monotone_on_a_fine_grid():
    xs = -np.linspace(0, 30, 60001).astype(np.float32)
    vals = [oracle.exp_det(float(x)) for x in xs]
    assert all(a >= b for a, b in zip(vals, vals[1:]))


# ---- the reductions: hand-derived values that separate candidate orders ------------------------------
def test_lane_sum_hand_traces():
    """T = 128 values: e[0] = 1 and 127 copies of 2^-25.  Lane l owns e[4l .. 4l+3] and adds them in ascending
    order from +0: lane 0 = 1 (each 2^-25 is below half an ulp of 1 and is absorbed); every other lane =
    4 * 2^-25 = 2^-23 exactly.  Adjacent-first tree: 1 + 2^-23, then + 2^-22, ... all exact (multiples of
    2^-23 below 2): 1 + 31 * 2^-23.  A single ascending chain over the 128 values would give 1."""
    e = np.full(128, 2.0 ** -25, dtype=np.float32)
    e[0] = 1.0
    assert oracle.lane_sum(e) == 1.0 + 31 * 2.0 ** -23
    # 256 values, T24 first: lane 0 = T24 (absorbs 1 three times in chunk 0 and four times in chunk 1), the other
    # lanes 8 each: T24 + 8 = T24+8 exactly, then + 16, + 32, ...: T24 + 31 * 8
    e = np.ones(256, dtype=np.float32)
    e[0] = T24
    assert oracle.lane_sum(e) == T24 + 248.0
    # tail: 130 values -> chunk 1 holds keys 128, 129 in lane 0 only
    e = np.ones(130, dtype=np.float32)
    assert oracle.lane_sum(e) == 130.0
    # lane 0 = 1+1+1+1 = 4, + e[128] = 5, + e[129] = T24 + 5 = 16777221: a tie between 16777220 and 16777222,
    # resolved to the even significand 16777220; the other 31 lanes hold 4 each: + 124
    e[129] = T24
    assert oracle.lane_sum(e) == 16777220.0 + 124.0
    assert oracle.lane_sum(e) == exact.lane_sum([float(v) for v in e])


def test_lane_dot_hand_traces():
    """The dot product over D uses the lane order too: q = ones, k = [T24, 1, 1, 1, -T24, 1, ...] (D = 128):
    lane 0 = T24 (absorbs three ones), lane 1 = -T24 + 3, tree: T24 + (-T24+3) = 3, other lanes 4 each: 3 + 30*4."""
    q = np.ones(128, dtype=np.float32)
    k = np.ones(128, dtype=np.float32)
    k[0], k[4] = T24, -T24
    assert oracle.lane_dot(q, k) == 3.0 + 120.0
    # fused single rounding in the chain (same operands as the linear layer's pin): 2^-30 survives
    q = np.zeros(8, dtype=np.float32)
    k = np.zeros(8, dtype=np.float32)
    q[0], k[0] = np.float32(-(1 + 2.0 ** -7 + 2.0 ** -23)), 1.0
    q[1], k[1] = np.float32(1 + 2.0 ** -23), np.float32(1 + 2.0 ** -7)
    assert oracle.lane_dot(q, k) == 2.0 ** -30


def _uniform_case(T, D, vcol):
    """q = 0: every score is 0, every weight exp_det(0) = 1, l = T; o[d] = (segment-ordered sum of v[:, d]) / T."""
    q = np.zeros((1, 1, D), dtype=np.float32)
    k = np.ones((1, 1, T, D), dtype=np.float32)
    v = np.zeros((1, 1, T, D), dtype=np.float32)
    v[0, 0, :, 0] = vcol
    return oracle.attention_decode(q, k, v, 0.125)[0, 0]


def test_pv_order_hand_traces():
    """T = 512 = two segments of 256 keys, all weights 1.
    (a) v = [T24, 1 x 255 | 1 x 256]: segment 0 is one ascending chain: T24 absorbs 255 ones -> T24; segment 1 =
        256; fold T24 + 256 (exact); o = (T24 + 256) / 512 = 32768.5.  One chain over all 512 keys would give
        T24 / 512 = 32768; a lane-split sum inside the segment would keep most of the ones.
    (b) v = [1 x 256 | T24, 1 x 254, -T24]: segment 0 = 256; segment 1: T24 absorbs 254 ones, -T24 -> 0; fold
        256 + 0; o = 0.5.  (A descending fold or chain would give other values.)"""
    v = np.ones(512, dtype=np.float32)
    v[0] = T24
    assert _uniform_case(512, 4, v)[0] == 32768.5
    v = np.ones(512, dtype=np.float32)
    v[256], v[511] = T24, -T24
    assert _uniform_case(512, 4, v)[0] == 0.5
    # three segments, left fold ((P0 + P1) + P2) with P = T24, 1, 1 -> T24 (each 1 absorbed); a tree or a right fold
    # gives T24 + 2
    v = np.zeros(768, dtype=np.float32)
    v[0], v[256], v[512] = T24, 1.0, 1.0
    assert _uniform_case(768, 4, v)[0] == np.float32(T24 / 768.0)


def test_closed_forms():
    rng = np.random.default_rng(0)
    # T = 1: the output is the value row itself
    q = rng.standard_normal((2, 4, 16)).astype(np.float32)
    k = rng.standard_normal((2, 2, 1, 16)).astype(np.float32)
    v = rng.standard_normal((2, 2, 1, 16)).astype(np.float32)
    o = oracle.attention_decode(q, k, v, 0.25)
    for h in range(4):
        assert np.array_equal(o[:, h], v[:, h // 2, 0])
    # uniform weights over small integers: exact mean, one rounding
    T, D = 300, 8
    vv = rng.integers(-8, 9, size=(T, D)).astype(np.float32)
    qz = np.zeros((1, 1, D), dtype=np.float32)
    o = oracle.attention_decode(qz, np.ones((1, 1, T, D), np.float32), vv[None, None], 1.0)[0, 0]
    want = (vv.astype(np.float64).sum(axis=0) / T).astype(np.float32)
    assert np.array_equal(o, want)


def test_layout_heads_and_accuracy_against_fp64():
    """Random data, grouped-query heads: the oracle against softmax(q k^T scale) v in FP64.  A wrong head
    mapping, a transposed operand or a missing scale is an O(1) error; the order only moves the last bits."""
    rng = np.random.default_rng(1)
    B, Hq, Hkv, T, D = 2, 8, 2, 333, 128
    q = rng.standard_normal((B, Hq, D)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, T, D)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, T, D)).astype(np.float32)
    scale = f32(1.0 / math.sqrt(D))
    o = oracle.attention_decode(q, k, v, scale)
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            s = (k[b, h // G].astype(np.float64) @ q[b, h].astype(np.float64)) * scale
            p = np.exp(s - s.max())
            want = (p[:, None] * v[b, h // G].astype(np.float64)).sum(axis=0) / p.sum()
            assert np.abs(o[b, h] - want).max() < 2e-6


@pytest.mark.parametrize("T,D", [(5, 8), (130, 4), (300, 8), (40, 132), (257, 12)])
def test_c_oracle_equals_exact_rational_replay(T, D):
    rng = np.random.default_rng(T * 1000 + D)
    q = rng.standard_normal(D).astype(np.float32)
    k = rng.standard_normal((T, D)).astype(np.float32)
    v = (rng.standard_normal((T, D)) * 3).astype(np.float32)
    k[0] = q * 4                                   # one dominant key: weights span many orders of magnitude
    scale = f32(0.7)
    got = oracle.attention_decode(q[None, None], k[None, None], v[None, None], scale)[0, 0]
    want = exact.attention_row([float(t) for t in q], [[float(t) for t in row] for row in k],
                               [[float(t) for t in row] for row in v], scale)
    assert [float(t) for t in got] == want
