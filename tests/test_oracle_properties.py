"""Pins for the CPU oracle that hold for any correct implementation of the method: the FP64 error
bound, the exact-integer special case (a library integer matmul), structural invariants (batch
invariance R4, permutation, sign symmetry, power-of-two scaling), the argmax tie rule, and the
shape -> parameter rule."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import inputs


def _up_np(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (2, 8, 64), (4, 8, 256), (3, 5, 512), (2, 4, 1000),
                                   (65, 6, 640), (70, 3, 1000)])
def test_fp64_error_bound(M, N, K):
    """|y_oracle - y_exact| <= 4*K*2^-24 * sum_k |x_k||w_k| per element (the stated accuracy bound;
    the paper reports an error at the 1e-7-relative level, supplement C on R1)."""
    x, W, b = inputs.make_case(M, N, K, seed=11)
    xb, Wb = x.numpy(), inputs.bf16_bits(W)
    y = oracle.linear(xb, Wb, None)
    wf = _up_np(Wb).astype(np.float64)
    xd = xb.astype(np.float64)
    worst = 0.0
    for m in range(M):
        for n in range(N):
            prods = xd[m] * wf[n]                       # exact: 24-bit x 8-bit significands
            ref = math.fsum(prods.tolist())
            bound = 4 * K * 2.0 ** -24 * float(np.abs(prods).sum())
            err = abs(float(y[m, n]) - ref)
            assert err <= bound, (m, n, err, bound)
            worst = max(worst, err / max(float(np.abs(prods).sum()), 1e-30))
    assert worst < 1e-5


@pytest.mark.parametrize("M,N,K", [(1, 1024, 512), (8, 300, 4096), (32, 64, 14336), (5, 37, 1000),
                                   (130, 200, 1792), (65, 129, 1000)])
def test_exact_integer_case_equals_int64_matmul(M, N, K):
    """Integer inputs in [-8, 8]: |sum| <= 64*K < 2^24, so every order is exact and must equal the
    integer matrix product computed by a library routine."""
    x, W, b = inputs.make_int_case(M, N, K, seed=5)
    want = (x.to(torch.int64) @ W.to(torch.float32).to(torch.int64).T + b.to(torch.int64)).numpy()
    y = oracle.linear(x.numpy(), inputs.bf16_bits(W), b.numpy())
    assert np.array_equal(y.astype(np.int64), want)
    assert np.array_equal(y, want.astype(np.float32))


def test_batch_invariance_in_decode_bucket():
    """R4: row m of a batch-M problem equals the M = 1 result of that row for every M <= 64."""
    N, K = 48, 1536
    x, W, b = inputs.make_case(64, N, K, seed=3)
    Wb = inputs.bf16_bits(W)
    full = oracle.linear(x.numpy(), Wb, b.numpy())
    for M in (1, 2, 3, 8, 17, 32, 33, 64):
        part = oracle.linear(x[:M].numpy(), Wb, b.numpy())
        assert np.array_equal(part.view(np.uint32), full[:M].view(np.uint32))
    one = oracle.linear(x[5:6].numpy(), Wb, b.numpy())
    assert np.array_equal(one.view(np.uint32), full[5:6].view(np.uint32))


def test_bucket_edge_changes_the_order():
    """Row 0 changes at M = 65 because the shape crosses into the prefill configuration
    (supplement C on R4)."""
    assert oracle.order_params(64, 128, 2048)["bucket"] == "decode"
    assert oracle.order_params(65, 128, 2048)["bucket"] == "prefill"
    x, W, _ = inputs.make_case(65, 128, 2048, seed=9)
    Wb = inputs.bf16_bits(W)
    a = oracle.linear(x[:64].numpy(), Wb, None)
    c = oracle.linear(x.numpy(), Wb, None)
    assert not np.array_equal(a[0].view(np.uint32), c[0].view(np.uint32))


@pytest.mark.parametrize("M", [4, 80])
def test_permutation_sign_and_scaling_invariants(M):
    N, K = 24, 768
    x, W, _ = inputs.make_case(M, N, K, seed=21)
    xb, Wb = x.numpy(), inputs.bf16_bits(W)
    prm = oracle.order_params(M, N, K)
    y = oracle.linear(xb, Wb, None, params=prm)
    rng = np.random.default_rng(0)
    pm, pn = rng.permutation(M), rng.permutation(N)
    yp = oracle.linear(xb[pm], Wb[pn], None, params=prm)
    assert np.array_equal(yp.view(np.uint32), y[pm][:, pn].view(np.uint32))
    yn = oracle.linear(-xb, Wb, None, params=prm)                  # round-to-nearest-even is symmetric
    assert np.array_equal(yn.view(np.uint32), (-y).view(np.uint32))
    ys = oracle.linear(xb * np.float32(2.0 ** 7), Wb, None, params=prm)   # exact scaling, no over/underflow
    assert np.array_equal(ys.view(np.uint32), (y * np.float32(2.0 ** 7)).view(np.uint32))


def test_sampled_outputs_match_full():
    x, W, b = inputs.make_case(6, 50, 1280, seed=2)
    Wb = inputs.bf16_bits(W)
    y = oracle.linear(x.numpy(), Wb, b.numpy())
    ms = np.array([0, 5, 3, 3], dtype=np.int64)
    ns = np.array([0, 49, 7, 8], dtype=np.int64)
    s = oracle.linear_sampled(x.numpy(), Wb, b.numpy(), ms, ns)
    assert np.array_equal(s.view(np.uint32), y[ms, ns].view(np.uint32))


def test_argmax_lower_index_wins_ties():
    """The tie is resolved toward the lower index (end-to-end determinism section)."""
    y = np.array([[1.0, 3.0, 3.0, 2.0],
                  [-0.0, 0.0, -1.0, 0.0],
                  [-5.0, -5.0, -5.0, -5.0],
                  [1.0, 2.0, 7.0, 7.0]], dtype=np.float32)
    assert list(oracle.argmax_rows(y)) == [1, 0, 0, 2]
    rng = np.random.default_rng(1)
    z = rng.standard_normal((5, 1000)).astype(np.float32)
    z[2, 900] = z[2, 100] = z[2].max() + 1
    want = torch.from_numpy(z).argmax(dim=1).numpy()
    want[2] = 100
    assert list(oracle.argmax_rows(z)) == list(want)
    z[4, 77] = np.nan
    assert oracle.argmax_rows(z)[4] == 77


def test_order_params_rule():
    # decode parameters never depend on M (R4)
    for (N, K) in [(1024, 512), (4096, 4096), (6144, 4096), (28672, 4096), (4096, 14336), (128256, 4096),
                   (1000, 1000), (7, 100)]:
        ref = oracle.order_params(1, N, K)
        for M in (2, 8, 31, 32, 33, 64):
            assert oracle.order_params(M, N, K) == ref
    # benchmark shapes
    assert oracle.order_params(1, 1024, 512) == dict(bucket="decode", V=4, L=32, P=1, seg_len=256, S=2,
                                                     order_version=2)
    for (N, K) in [(4096, 4096), (6144, 4096), (28672, 4096), (4096, 14336), (128256, 4096)]:
        p = oracle.order_params(8, N, K)
        assert (p["S"], p["seg_len"]) == ((1, K) if N >= 16384 else (2, K // 2))
    # every segment non-empty, boundaries on multiples of 256, all of K covered
    for M in (1, 64, 65, 128, 2048):
        for N in (1, 100, 1000, 4096, 28672):
            for K in (1, 8, 255, 256, 257, 1000, 4096, 14336):
                p = oracle.order_params(M, N, K)
                assert p["seg_len"] % 256 == 0
                assert (p["S"] - 1) * p["seg_len"] < K <= p["S"] * p["seg_len"]
