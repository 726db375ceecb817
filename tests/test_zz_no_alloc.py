"""det_linear_run_noalloc, the entry point for callers that cannot allocate (a host that owns all
device memory through its own pool, a plugin after initialisation, a latency-critical loop): it
must give the same bits as det_linear_plan + det_linear_run, on two calls in a row (the built-in
scratch keeps the previous call's contents), and reject shapes whose split-K partials exceed the
built-in scratch.  Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import assert_bits_equal, oracle_y, run_gpu

pytestmark = pytest.mark.gpu

# (M, N, K): decode with two segments, twice (folded inside the kernel: no scratch), ragged K,
# prefill with split (S = 8: the partials go through the built-in scratch)
CASES = [(1, 1024, 512), (8, 4096, 1024), (5, 300, 1001), (130, 200, 4096)]


@pytest.mark.parametrize("M,N,K", CASES)
def test_noalloc_matches_planned_run_twice_in_a_row(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    want = run_gpu(x, W, b)                     # existing entry point: det_linear_plan + det_linear_run
    assert_bits_equal(want, oracle_y(x, W, b), "planned run vs oracle")
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.det_linear_run_noalloc(xd, Wd, bd, y)     # first call on the device: resolves the scratch address
    torch.cuda.synchronize()
    for call in range(2):
        y.fill_(float("nan"))
        B.det_linear_run_noalloc(xd, Wd, bd, y)
        torch.cuda.synchronize()
        assert_bits_equal(y.cpu().numpy(), want, f"call {call}")
    # the entry point allocates nothing: the device's free memory does not shrink across calls (device-wide
    # figure, so allow for another process allocating at the same moment by looking more than once)
    for attempt in range(3):
        free_before = torch.cuda.mem_get_info()[0]
        for _ in range(4):
            B.det_linear_run_noalloc(xd, Wd, bd, y)
        torch.cuda.synchronize()
        if torch.cuda.mem_get_info()[0] >= free_before:
            break
    else:
        raise AssertionError("free device memory shrank across det_linear_run_noalloc calls")
    # a different problem in between must not disturb the next call (shared scratch, stale contents)
    x2, W2, b2 = inputs.make_case(3, 512, 768, seed=5)
    y2 = torch.empty(3, 512, dtype=torch.float32, device="cuda")
    B.det_linear_run_noalloc(x2.cuda(), W2.cuda(), b2.cuda(), y2)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.det_linear_run_noalloc(xd, Wd, None, y)
    torch.cuda.synchronize()
    assert_bits_equal(y.cpu().numpy(), run_gpu(x, W, None), "no bias, after another problem")
    assert_bits_equal(y2.cpu().numpy(), run_gpu(x2, W2, b2), "interleaved problem")


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    M, N, K = 128, 4096, 14336                  # S = 14: 14 * 128 * 4096 * 4 bytes = 29 MB of partials
    prm = B.det_linear_plan_params(M, N, K)
    assert prm.workspace_bytes > (4 << 20)
    x = torch.zeros(M, K, device="cuda")
    W = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(M, N, device="cuda")
    with pytest.raises(B.DetLinearError) as ei:
        B.det_linear_run_noalloc(x, W, None, y)
    assert ei.value.status == 2
    msg = B.det_last_error()
    assert str(prm.workspace_bytes) in msg and str(4 << 20) in msg
    rc = B.lib().det_linear_run_noalloc(1, 8, 8, None, None, None, None, None)
    assert rc == 1
