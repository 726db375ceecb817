"""Pins of the fixed-order RMSNorm oracle against things other than itself: hand-derived sums of
squares (tests/golden/rmsnorm_examples.txt), an exact-rational re-implementation, closed forms,
the power-of-two scaling invariance and an FP64 evaluation of the definition."""
import os

import numpy as np
import pytest

from oracle import exact, oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "rmsnorm_examples.txt")


def _pattern(name, H):
    x = np.zeros(H, dtype=np.float32)
    if name == "ones":
        x[:] = 1.0
    elif name == "big0_then_ones":
        x[:] = 1.0
        x[0] = 4096.0
    else:
        x[0] = 4096.0
        for tok in name.split("_")[1:]:
            assert tok.startswith("one")
            x[int(tok[3:])] = 1.0
    return x


def _examples():
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, H, pat, ss, _why = [f.strip() for f in line.split("|")]
        yield name, int(H), pat, int(ss)


@pytest.mark.parametrize("name,H,pat,ss", list(_examples()))
def test_hand_derived_sum_of_squares(name, H, pat, ss):
    x = _pattern(pat, H)
    assert oracle.sum_squares(x) == float(ss), name
    assert exact.sum_squares([float(v) for v in x]) == float(ss), name


def test_order_matters_for_these_examples():
    """The examples are chosen so that other plausible orders give other sums."""
    x = _pattern("big0_then_ones", 256)
    seq = np.float32(0)
    for v in x:
        seq = np.float32(seq + v * v)
    assert float(seq) == 16777216.0 and oracle.sum_squares(x) == 16777464.0
    x = _pattern("big0_one4_one8", 128)
    assert float(np.float32(np.float32(1) + np.float32(1)) + np.float32(2 ** 24)) == 16777218.0
    assert oracle.sum_squares(x) == 16777216.0


def test_closed_forms():
    g = np.linspace(-2, 2, 256, dtype=np.float32)
    for c in (1.0, -1.0, 3.0, 0.5, -1024.0):
        x = np.full((1, 256), c, dtype=np.float32)
        y = oracle.rmsnorm(x, g, 0.0)
        # ss = 256 c^2 exactly, mean = c^2, root = |c|, r = fl(1/|c|), fl(c * r) = +-1 for these c
        assert np.array_equal(y[0], np.sign(c) * g), c
    # eps only: x = 0 -> y = +-0 * g = 0
    y = oracle.rmsnorm(np.zeros((2, 130), np.float32), np.ones(130, np.float32), 1e-5)
    assert not y.any()


def test_matches_exact_rational_micro_oracle():
    rng = np.random.default_rng(5)
    for H in (1, 3, 5, 127, 128, 129, 260, 515):
        for eps in (0.0, 1e-5, 1e-6):
            x = rng.standard_normal((2, H)).astype(np.float32)
            x[1] *= np.float32(1e-3)
            g = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
            y = oracle.rmsnorm(x, g, eps)
            e32 = float(np.float32(eps))
            for m in range(2):
                want = exact.rmsnorm_row([float(v) for v in x[m]], [float(v) for v in g], e32)
                assert np.array_equal(y[m].view(np.uint32), np.array(want, dtype=np.float32).view(np.uint32)), (H, eps, m)


def test_sqrt32_is_correctly_rounded():
    rng = np.random.default_rng(9)
    vals = np.concatenate([rng.uniform(0, 4, 2000), rng.uniform(0, 1e-30, 200), rng.uniform(1e20, 1e30, 200),
                           np.array([1.0, 4.0, 2.25, 2.0, 3.0, 1e-45, 16777216.0])]).astype(np.float32)
    for v in vals:
        want = np.float32(np.sqrt(np.float64(v)))          # double sqrt then one rounding is exact for binary32 inputs
        assert exact.sqrt32(float(v)) == float(want), v


def test_power_of_two_scaling_invariance():
    """With eps = 0, scaling a row by 2^k scales ss by 4^k, the root by 2^k and r by 2^-k, all
    exactly, so y is unchanged bit for bit (absent overflow / underflow)."""
    rng = np.random.default_rng(11)
    x = rng.standard_normal((4, 1000)).astype(np.float32)
    g = rng.standard_normal(1000).astype(np.float32)
    base = oracle.rmsnorm(x, g, 0.0)
    for k in (-20, -3, 1, 7, 30):
        y = oracle.rmsnorm(x * np.float32(2.0 ** k), g, 0.0)
        assert np.array_equal(y.view(np.uint32), base.view(np.uint32)), k


def test_close_to_fp64_definition():
    rng = np.random.default_rng(13)
    for H in (64, 4096, 5000):
        x = rng.standard_normal((3, H)).astype(np.float32)
        g = rng.standard_normal(H).astype(np.float32)
        y = oracle.rmsnorm(x, g, 1e-5)
        xd, gd = x.astype(np.float64), g.astype(np.float64)
        ref = xd / np.sqrt((xd * xd).mean(axis=1, keepdims=True) + np.float64(np.float32(1e-5))) * gd
        # ss carries at most ~(H/128 + 5 + 4) roundings per chain, then 5 more operations
        assert np.abs(y - ref).max() <= 8 * 2.0 ** -24 * np.abs(ref).max() + 1e-30, H


def test_rows_are_independent_and_rejects_bad_arguments():
    rng = np.random.default_rng(17)
    x = rng.standard_normal((5, 300)).astype(np.float32)
    g = rng.standard_normal(300).astype(np.float32)
    y = oracle.rmsnorm(x, g, 1e-6)
    for m in range(5):
        assert np.array_equal(oracle.rmsnorm(x[m:m + 1], g, 1e-6)[0], y[m])
    with pytest.raises((ValueError, AssertionError)):
        oracle.rmsnorm(x, g[:10], 1e-6)
