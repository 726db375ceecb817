"""Helpers for the GPU parity tests: run the CUDA path through the C ABI and fetch bits."""
import numpy as np
import torch

from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs

KERNEL_GENERIC, KERNEL_DECODE, KERNEL_PREFILL = 0, 1, 2


def to_dev(t):
    return None if t is None else t.cuda()


def run_gpu(x, W, b, kernel=None, variant=0, max_blocks=0, stream=None, y_fill=float("nan"), two_pass_combine=False):
    """x [M,K] f32, W [N,K] bf16 / fp16 / fp32 (the plan's weight format follows the dtype), b [N] f32 or
    None (CPU or CUDA tensors) -> y as numpy float32 [M,N].
    The output buffer is pre-filled with NaN so that an element the kernel never wrote is caught."""
    M, K = x.shape
    N = W.shape[0]
    xd, Wd, bd = x.cuda(), W.cuda(), to_dev(b)
    y = torch.full((M, N), y_fill, dtype=torch.float32, device="cuda")
    plan = B.det_linear_plan_w(M, N, K, inputs.weight_format_of(W))
    try:
        if kernel is not None:
            B.det_test_plan_force_kernel(plan, kernel)
        if variant:
            B.det_test_plan_set_variant(plan, variant)
        if max_blocks:
            B.det_test_plan_set_max_blocks(plan, max_blocks)
        if two_pass_combine:
            B.det_test_plan_set_wait(plan, 2_000_000_000, two_pass_combine=True)
        B.det_linear_run(plan, xd, Wd, bd, y, stream=stream)
        B.det_linear_plan_check(plan, stream=stream)
        torch.cuda.synchronize()
    finally:
        plan.close()
    return y.cpu().numpy()


def oracle_y(x, W, b):
    from oracle import oracle
    return oracle.linear(x.numpy(), inputs.weight_bits(W), None if b is None else b.numpy(),
                         wfmt=inputs.weight_format_of(W))


def assert_bits_equal(got, want, what=""):
    got = np.ascontiguousarray(got, dtype=np.float32)
    want = np.ascontiguousarray(want, dtype=np.float32)
    assert got.shape == want.shape, (got.shape, want.shape)
    g, w = got.view(np.uint32), want.view(np.uint32)
    if not np.array_equal(g, w):
        bad = np.argwhere(g != w)
        i = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} of {g.size} elements differ; first at {i}: "
                             f"got {got[i]!r} (0x{g[i]:08x}) want {want[i]!r} (0x{w[i]:08x})")
