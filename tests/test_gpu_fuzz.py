"""Seeded random shapes through every entry point against the oracle: bit-exact.  Complements the
hand-picked shapes of the other files (ragged tails, tiny and odd sizes, every weight format,
column shards, forced kernels and tilings)."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from paper_2609_25624_b200.sharded import shard_range
from tests.gpu_util import KERNEL_DECODE, KERNEL_GENERIC, KERNEL_PREFILL, assert_bits_equal, oracle_y, run_gpu

pytestmark = pytest.mark.gpu


def _shapes(seed, n, m_hi):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        M = int(rng.integers(1, m_hi + 1))
        N = int(rng.choice([rng.integers(1, 40), rng.integers(40, 700), 8 * rng.integers(1, 120)]))
        K = int(rng.choice([rng.integers(1, 60), 8 * rng.integers(1, 400), 4 * rng.integers(1, 300), rng.integers(60, 2000)]))
        out.append((M, N, K))
    return out


@pytest.mark.parametrize("M,N,K", _shapes(2024, 40, 64))
def test_random_decode_shapes(M, N, K):
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    wfmt = ("bf16", "fp16", "fp32")[int(rng.integers(0, 3))]
    bias = bool(rng.integers(0, 2))
    x, W, b = inputs.make_case_w(M, N, K, wfmt, bias=bias)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b), want, f"auto {wfmt}")
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, f"generic {wfmt}")
    k_align = 4 if wfmt == "fp32" else 8
    if K % k_align == 0 and K % 4 == 0:
        v = int(rng.integers(1, 5))
        assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_DECODE, variant=v), want, f"decode variant {v} {wfmt}")


@pytest.mark.parametrize("M,N,K", _shapes(77, 16, 300))
def test_random_prefill_and_shards(M, N, K):
    M = max(M, 65)
    rng = np.random.default_rng(M * 7919 + N * 104729 + K)
    wfmt = ("bf16", "fp16", "fp32")[int(rng.integers(0, 3))]
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b), want, f"auto {wfmt}")
    k_align = 4 if wfmt == "fp32" else 8
    if K % k_align == 0 and K % 4 == 0:
        tr = int(rng.integers(5, 9))
        assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_PREFILL, variant=tr), want, f"tile {16 * tr} {wfmt}")
    # the same layer as column shards written in place
    world = int(rng.integers(2, 5))
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for r in range(world):
        n0, cnt = shard_range(N, r, world)
        if cnt == 0:
            continue
        plan = B.det_linear_plan_shard(M, N, K, n0, cnt, N, wfmt)
        B.det_linear_run_shard(plan, xd, Wd[n0:n0 + cnt], bd[n0:n0 + cnt], y[:, n0:n0 + cnt])
        B.det_linear_plan_check(plan)
        plan.close()
    torch.cuda.synchronize()
    assert_bits_equal(y.cpu().numpy(), want, f"{world} shards {wfmt}")


@pytest.mark.parametrize("seed", range(12))
def test_random_rmsnorm(seed):
    rng = np.random.default_rng(seed)
    M = int(rng.integers(1, 70))
    H = int(rng.choice([rng.integers(1, 300), 4 * rng.integers(1, 1100), 128 * rng.integers(1, 40), rng.integers(300, 9000)]))
    eps = float(rng.choice([0.0, 1e-6, 1e-5, 1e-3]))
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(M, H, generator=g) * float(10.0 ** rng.integers(-3, 4))
    gain = torch.randn(H, generator=g)
    y = torch.full((M, H), float("nan"), device="cuda")
    B.det_rmsnorm(x.cuda(), gain.cuda(), eps, y)
    torch.cuda.synchronize()
    assert_bits_equal(y.cpu().numpy(), oracle.rmsnorm(x.numpy(), gain.numpy(), eps), f"{M}x{H} eps={eps}")
