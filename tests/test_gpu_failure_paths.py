"""Failure paths, exercised in forms that never fault, trap or hang the device:

* a device allocation made to fail on the HOST (a countdown in the library's allocation wrapper):
  plan creation must return NULL with DET_ERR_ALLOC and leak nothing;
* a bounded device-side wait made to run out: thread block 0 of the decode kernel is told not to request
  one activation copy, so the consumers' wait for that stage reaches a (shortened) time limit, records
  it in the plan's status word and the kernel returns by itself; det_linear_plan_check must report
  DET_ERR_DEVICE_TIMEOUT, and the next ordinary run on the same plan must be bit-exact again.
"""
import time

import pytest
import torch

from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import assert_bits_equal, oracle_y

pytestmark = pytest.mark.gpu

DET_ERR_ALLOC, DET_ERR_DEVICE_TIMEOUT = 4, 6


def test_plan_allocation_failure_is_reported_and_leaks_nothing():
    torch.cuda.synchronize()
    B.det_linear_plan(8, 64, 512).close()                       # context and library warmed up
    free0 = torch.cuda.mem_get_info()[0]
    # prefill plan with split-K: two device allocations (status word, then the 2 MB workspace)
    M, N, K = 128, 256, 4096
    assert B.det_linear_plan_params(M, N, K).workspace_bytes > 0
    for nth in (1, 2):
        B.det_test_fail_next_alloc(nth)
        try:
            with pytest.raises(B.DetLinearError) as ei:
                B.det_linear_plan(M, N, K)
        finally:
            B.det_test_fail_next_alloc(0)
        assert ei.value.status == DET_ERR_ALLOC
        assert B.det_last_status() == DET_ERR_ALLOC
        assert "allocation" in B.det_last_error()
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free0                 # the status word of the nth = 2 case was freed
    # the hook is one-shot: the next plan is fine and computes the right bits
    x, W, b = inputs.make_case(4, 96, 512)
    plan = B.det_linear_plan(4, 96, 512)
    assert B.det_last_status() == 0
    y = torch.empty(4, 96, device="cuda")
    B.det_linear_run(plan, x.cuda(), W.cuda(), b.cuda(), y)
    B.det_linear_plan_check(plan)
    plan.close()
    assert_bits_equal(y.cpu().numpy(), oracle_y(x, W, b), "after the injected failures")


def test_host_staging_allocation_failure():
    x, W, b = inputs.make_case(2, 64, 512)
    plan = B.det_linear_plan(2, 64, 512)
    xh, yh = x.pin_memory(), torch.empty(2, 64).pin_memory()
    B.det_test_fail_next_alloc(2)                               # x staging succeeds, y staging fails
    try:
        with pytest.raises(B.DetLinearError) as ei:
            B.det_linear_run_host(plan, xh, W.cuda(), b.cuda(), yh)
    finally:
        B.det_test_fail_next_alloc(0)
    assert ei.value.status == DET_ERR_ALLOC
    B.det_linear_run_host(plan, xh, W.cuda(), b.cuda(), yh)      # the retry allocates both and works
    plan.close()
    assert_bits_equal(yh.numpy(), oracle_y(x, W, b), "after the failed staging allocation")


@pytest.mark.parametrize("M,N,K", [(8, 4096, 4096), (1, 1024, 512), (32, 600, 2048)])
def test_bounded_wait_expires_and_the_kernel_returns(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    plan = B.det_linear_plan(M, N, K)
    assert B.det_linear_plan_describe(plan)["kernel"] == "decode"
    B.det_linear_run(plan, xd, Wd, bd, y)
    B.det_linear_plan_check(plan)
    assert_bits_equal(y.cpu().numpy(), want, "before")

    B.det_test_plan_set_wait(plan, 5_000_000, withhold_first_copy=True)     # 5 ms per wait
    t0 = time.perf_counter()
    B.det_linear_run(plan, xd, Wd, bd, y)
    with pytest.raises(B.DetLinearError) as ei:
        B.det_linear_plan_check(plan)                            # synchronises: the kernel has returned
    elapsed = time.perf_counter() - t0
    assert ei.value.status == DET_ERR_DEVICE_TIMEOUT
    # site 2 = a consumer's wait for a full stage, site 1 = the producer finding no free slot for as long;
    # both run out here and the later one is the one on record
    assert "site 2" in B.det_last_error() or "site 1" in B.det_last_error()
    assert elapsed < 5.0, f"the stalled kernel took {elapsed:.2f} s to give up"

    # the record is cleared by the check; the context is intact and the plan usable again
    B.det_test_plan_set_wait(plan, 2_000_000_000, withhold_first_copy=False)
    y.fill_(float("nan"))
    B.det_linear_run(plan, xd, Wd, bd, y)
    B.det_linear_plan_check(plan)
    plan.close()
    assert_bits_equal(y.cpu().numpy(), want, "after the expired wait")


def test_bounded_wait_expires_in_the_prefill_kernel():
    """The TMA-fed prefill kernel bounds its waits too: block 0 is made to miss its first activation tile,
    gives up after the limit and returns; the plan reports it and works again afterwards."""
    M, N, K = 128, 256, 1024
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    plan = B.det_linear_plan(M, N, K)
    d = B.det_linear_plan_describe(plan)
    assert d["kernel"] == "prefill" and d["prefill_tile"]["feed"] == "tma"
    B.det_test_plan_set_wait(plan, 5_000_000, withhold_first_copy=True)     # 5 ms per wait
    t0 = time.perf_counter()
    B.det_linear_run(plan, xd, Wd, bd, y)
    with pytest.raises(B.DetLinearError) as ei:
        B.det_linear_plan_check(plan)
    elapsed = time.perf_counter() - t0
    assert ei.value.status == DET_ERR_DEVICE_TIMEOUT
    assert "site 4" in B.det_last_error() or "site 3" in B.det_last_error()
    assert elapsed < 5.0, f"the stalled kernel took {elapsed:.2f} s to give up"
    B.det_test_plan_set_wait(plan, 2_000_000_000, withhold_first_copy=False)
    # other activations: nothing of the abandoned run (partial tiles, tile counts of the in-kernel fold) may leak in
    x2, _, _ = inputs.make_case(M, N, K + 8)
    x2 = x2[:, :K].contiguous()
    for rep in range(2):
        y.fill_(float("nan"))
        B.det_linear_run(plan, x2.cuda(), Wd, bd, y)
        B.det_linear_plan_check(plan)
        assert_bits_equal(y.cpu().numpy(), oracle_y(x2, W, b), f"after the expired wait, run {rep}")
    plan.close()


@pytest.mark.parametrize("M,N,K,nth", [(128, 256, 4096, 3), (96, 136, 256, 2)])
def test_prefill_without_its_activation_workspace(M, N, K, nth):
    """The transposed-activation workspace is optional: when its allocation fails the plan is still created,
    runs the register-staged kernel and produces the same bits."""
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert (B.det_linear_plan_params(M, N, K).workspace_bytes > 0) == (nth == 3)
    B.det_test_fail_next_alloc(nth)                 # status word, (partials,) then the workspace
    try:
        plan = B.det_linear_plan(M, N, K)
    finally:
        B.det_test_fail_next_alloc(0)
    assert B.det_linear_plan_describe(plan)["prefill_tile"]["feed"] == "registers"
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.det_linear_run(plan, x.cuda(), W.cuda(), b.cuda(), y)
    B.det_linear_plan_check(plan)
    plan.close()
    assert_bits_equal(y.cpu().numpy(), want, "register-staged fallback")
    plan = B.det_linear_plan(M, N, K)
    assert B.det_linear_plan_describe(plan)["prefill_tile"]["feed"] == "tma"
    plan.close()
