"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (automatic
kernel choice, default grid): sampled outputs against the oracle one by one, the exact-integer
special case against a library matrix product on every element, and the LM-head argmax cases."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import assert_bits_equal, run_gpu

pytestmark = pytest.mark.gpu


def sample_points(M, N, rng, count=1500):
    ms = rng.integers(0, M, size=count)
    ns = rng.integers(0, N, size=count)
    # always include the corners and the last rows/columns of tiles of every size used
    edge_n = [0, 1, 7, 8, 15, 16, 31, 32, 63, 64, 127, 128, N - 129, N - 128, N - 65, N - 33, N - 17, N - 9, N - 2, N - 1]
    edge_m = [0, M - 1, M // 2, min(M - 1, 127), min(M - 1, 128)]
    for m in edge_m:
        for n in edge_n:
            if 0 <= n < N:
                ms = np.append(ms, m)
                ns = np.append(ns, n)
    return ms.astype(np.int64), ns.astype(np.int64)


@pytest.mark.parametrize("name,K,N", inputs.LLAMA3_8B_LAYER)
@pytest.mark.parametrize("M", inputs.DECODE_MS)
def test_decode_full_size_sampled(name, K, N, M):
    x, W, b = inputs.make_case(M, N, K)
    got = run_gpu(x, W, b)
    assert not np.isnan(got).any()
    ms, ns = sample_points(M, N, np.random.default_rng(M + N))
    want = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns)
    assert_bits_equal(got[ms, ns], want, f"{name} M={M}")


@pytest.mark.parametrize("name,K,N", inputs.PREFILL_SHAPES)
@pytest.mark.parametrize("M", inputs.PREFILL_MS)
def test_prefill_full_size_sampled(name, K, N, M):
    x, W, b = inputs.make_case(M, N, K)
    got = run_gpu(x, W, b)
    assert not np.isnan(got).any()
    ms, ns = sample_points(M, N, np.random.default_rng(M + N))
    want = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns)
    assert_bits_equal(got[ms, ns], want, f"{name} M={M}")


@pytest.mark.parametrize("M,N,K", [(4, 6144, 4096), (16, 4096, 14336), (32, 28672, 4096), (64, 4096, 4096),
                                   (128, 4096, 14336), (512, 28672, 4096), (2048, 4096, 14336)])
def test_exact_integer_case_every_element(M, N, K):
    """Integer inputs in [-8, 8]: every order is exact, so every element must equal the integer
    matrix product (computed here by the FP64 library GEMM, exact for these magnitudes)."""
    x, W, b = inputs.make_int_case(M, N, K, seed=M + N + K)
    got = run_gpu(x, W, b)
    want = (x.cuda().double() @ W.cuda().double().T + b.cuda().double()).float().cpu().numpy()
    assert_bits_equal(got, want, "integer case")


def _lm_head_case(M):
    name, K, N = inputs.LLAMA3_8B_LM_HEAD
    W = inputs.make_weight(N, K, inputs.named_seed("lm_head"))
    g = torch.Generator().manual_seed(inputs.shape_seed(M, N, K))
    x = torch.randn(M, K, generator=g)
    return x, W


def _gpu_logits_and_argmax(x, W):
    M, K = x.shape
    N = W.shape[0]
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    plan = B.det_linear_plan(M, N, K)
    B.det_linear_run(plan, x.cuda(), W.cuda(), None, y)
    B.det_argmax_rows(y, idx)
    B.det_linear_plan_check(plan)
    plan.close()
    return y.cpu().numpy(), idx.cpu().numpy()


@pytest.mark.parametrize("M", [1, 8, 32])
def test_lm_head_logits_and_argmax(M):
    x, W = _lm_head_case(M)
    got, idx = _gpu_logits_and_argmax(x, W)
    want = oracle.linear(x.numpy(), inputs.bf16_bits(W), None)
    assert_bits_equal(got, want, f"lm_head M={M}")
    assert idx.tolist() == oracle.argmax_rows(want).tolist()


@pytest.mark.parametrize("n_positions", [16, 0])
def test_lm_head_near_tie_and_exact_tie(n_positions):
    """Two weight rows that differ by one BF16 ulp in 16 positions (or not at all): the logits must
    still be bit-equal to the oracle's and the argmax must be the oracle's; an exact tie returns
    the lower row index."""
    M = 8
    x, W = _lm_head_case(M)
    base = oracle.linear(x[:1].numpy(), inputs.bf16_bits(W), None)
    r1 = int(oracle.argmax_rows(base)[0])
    r2 = int(np.random.default_rng(3).integers(0, W.shape[0]))
    if r2 == r1:
        r2 = (r1 + 1) % W.shape[0]
    W2 = inputs.make_near_tie(W, r1, r2, n_positions=n_positions, seed=11)
    want = oracle.linear(x.numpy(), inputs.bf16_bits(W2), None)
    want_idx = oracle.argmax_rows(want)
    got, idx = _gpu_logits_and_argmax(x, W2)
    assert_bits_equal(got, want, "near-tie logits")
    assert idx.tolist() == want_idx.tolist()
    top2 = np.argsort(want[0])[-2:]
    assert set(top2.tolist()) == {r1, r2}
    if n_positions == 0:
        assert want[0, r1] == want[0, r2]
        assert idx[0] == min(r1, r2)
    # repeated runs give the same argmax and the same logits
    for _ in range(3):
        g2, i2 = _gpu_logits_and_argmax(x, W2)
        assert_bits_equal(g2, got, "repeat")
        assert i2.tolist() == idx.tolist()
