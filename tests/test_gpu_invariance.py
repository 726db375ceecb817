"""Invariance of the bits: repeated runs, streams, concurrent streams, CUDA-graph replay, grid size
and SM-count limits (green contexts) must all give one and the same output (rule R3: the result is
"independent of the device, its SM count, and grid scheduling"; the run-to-run ablation reports
exactly one distinct output in 50 runs)."""
import hashlib

import numpy as np
import pytest
import torch

from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import assert_bits_equal, oracle_y, run_gpu

pytestmark = pytest.mark.gpu

# decode (M <= 64) and prefill; the prefill cases cover the combine launch (S = 9) and the in-kernel fold, where the
# block that folds a tile is whichever finishes last (S = 4, 3, 2)
CASES = [(1, 1024, 512), (8, 4096, 4096), (32, 1000, 2048), (130, 520, 2304), (200, 1024, 1024), (300, 1152, 768),
         (512, 640, 512)]


def digest(t):
    return hashlib.sha256(t.detach().cpu().numpy().tobytes()).hexdigest()


@pytest.mark.parametrize("M,N,K", CASES)
def test_fifty_runs_one_output(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    plan = B.det_linear_plan(M, N, K)
    seen = set()
    for i in range(50):
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        B.det_linear_run(plan, xd, Wd, bd, y)
        seen.add(digest(y))
    B.det_linear_plan_check(plan)
    plan.close()
    assert len(seen) == 1
    if M * N * K <= 40_000_000:
        assert seen == {hashlib.sha256(oracle_y(x, W, b).tobytes()).hexdigest()}


@pytest.mark.parametrize("M,N,K", CASES)
def test_streams_and_concurrency(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    ref = run_gpu(x, W, b)
    streams = [torch.cuda.Stream() for _ in range(3)]
    plans = [B.det_linear_plan(M, N, K) for _ in streams]
    ys = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in streams]
    torch.cuda.synchronize()
    for rep in range(5):                       # the three streams run concurrently, each with its own plan
        for s, p, y in zip(streams, plans, ys):
            B.det_linear_run(p, xd, Wd, bd, y, stream=s)
    torch.cuda.synchronize()
    for p, y in zip(plans, ys):
        B.det_linear_plan_check(p)
        assert_bits_equal(y.cpu().numpy(), ref, "stream")
        p.close()


@pytest.mark.parametrize("M,N,K", CASES)
def test_grid_size_does_not_matter(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    ref = run_gpu(x, W, b)
    for blocks in (1, 7, 64, 147):
        assert_bits_equal(run_gpu(x, W, b, max_blocks=blocks), ref, f"max_blocks={blocks}")


@pytest.mark.parametrize("M,N,K", CASES)
def test_cuda_graph_replay_equals_eager(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    ref = run_gpu(x, W, b)
    plan = B.det_linear_plan(M, N, K)
    y = torch.empty(M, N, dtype=torch.float32, device="cuda")
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        B.det_linear_run(plan, xd, Wd, bd, y)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for _ in range(3):
                B.det_linear_run(plan, xd, Wd, bd, y)
        for _ in range(3):
            y.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert_bits_equal(y.cpu().numpy(), ref, "graph replay")
    plan.close()


def _green_or_skip(sm):
    try:
        return B.det_test_green_stream_create(sm)
    except B.DetLinearError as e:
        pytest.skip(f"green contexts refused by the driver: {e}")


@pytest.mark.parametrize("M,N,K", CASES)
def test_sm_count_limits_green_contexts(M, N, K):
    """The same call on 8, 32 and 64 SMs (green contexts) and on the whole device."""
    x, W, b = inputs.make_case(M, N, K)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    ref = run_gpu(x, W, b)
    granted = []
    for sm in (8, 32, 64):
        stream, handle, got_sm = _green_or_skip(sm)
        try:
            granted.append(got_sm)
            plan = B.det_linear_plan(M, N, K)
            y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            B.det_linear_run(plan, xd, Wd, bd, y, stream=stream)
            B.det_linear_plan_check(plan, stream=stream)
            torch.cuda.synchronize()
            assert_bits_equal(y.cpu().numpy(), ref, f"{got_sm} SMs")
            plan.close()
        finally:
            B.det_test_green_stream_destroy(handle)
    assert granted[0] < 148
