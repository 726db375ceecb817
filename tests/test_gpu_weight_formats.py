"""FP16 and FP32 weights through the CUDA path (C ABI) against the CPU oracle: bit-exact.

The reduction order does not depend on the storage format of W (Eq. 2's up() is exact for every
format); only the bytes streamed from HBM and the widening instruction differ."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import (KERNEL_DECODE, KERNEL_GENERIC, KERNEL_PREFILL, assert_bits_equal, oracle_y,
                            run_gpu)

pytestmark = pytest.mark.gpu

FORMATS = ("fp16", "fp32")
DECODE_SHAPES = [(1, 1024, 512), (2, 77, 1000), (3, 130, 2304), (4, 96, 4096), (8, 257, 1536), (8, 64, 14336),
                 (13, 200, 1000), (16, 96, 2048), (32, 128, 4096), (33, 64, 640), (64, 50, 512), (7, 9, 8),
                 (5, 40, 260)]
RAGGED = [(1, 10, 1), (3, 17, 7), (5, 33, 1001), (8, 50, 1004), (4, 31, 250), (70, 33, 250), (66, 5, 3)]
PREFILL_SHAPES = [(65, 129, 1000), (100, 1000, 1000), (130, 200, 1792), (128, 256, 1024), (200, 72, 4096),
                  (65, 1, 8), (72, 140, 516)]


@pytest.mark.parametrize("wfmt", FORMATS)
def test_plan_reports_format_and_same_order(wfmt):
    plan = B.det_linear_plan_w(8, 4096, 4096, wfmt)
    d = B.det_linear_plan_describe(plan)
    assert d["weight_format"] == wfmt
    p = B.det_linear_plan_get_params(plan)
    assert p.weight_format == B.WEIGHT_FORMATS[wfmt]
    assert p.as_dict() == oracle.order_params(8, 4096, 4096) == B.det_linear_plan_params(8, 4096, 4096).as_dict()
    plan.close()


@pytest.mark.parametrize("wfmt", FORMATS)
@pytest.mark.parametrize("M,N,K", DECODE_SHAPES)
def test_decode_bit_exact_all_tilings(M, N, K, wfmt):
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, "generic")
    n_tilings = 0
    for variant in range(0, 16):               # 0 = automatic, then every compiled tiling for this batch size
        try:
            got = run_gpu(x, W, b, kernel=KERNEL_DECODE, variant=variant)
        except B.DetLinearError:
            break
        assert_bits_equal(got, want, f"variant={variant}")
        n_tilings = variant
    # tilings whose segment groups do not divide S cannot run the shape
    assert n_tilings >= (4 if oracle.order_params(M, N, K)["S"] == 2 else 2)
    assert_bits_equal(run_gpu(x, W, b, max_blocks=3), want, "three blocks")
    assert_bits_equal(run_gpu(x, W, None), oracle_y(x, W, None), "no bias")


@pytest.mark.parametrize("wfmt", FORMATS)
@pytest.mark.parametrize("M,N,K", RAGGED)
def test_ragged_bit_exact(M, N, K, wfmt):
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    assert_bits_equal(run_gpu(x, W, b), oracle_y(x, W, b), "ragged")


@pytest.mark.parametrize("wfmt", FORMATS)
@pytest.mark.parametrize("M,N,K", PREFILL_SHAPES)
def test_prefill_bit_exact(M, N, K, wfmt):
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, "generic")
    assert_bits_equal(run_gpu(x, W, b), want, "automatic")
    assert_bits_equal(run_gpu(x, W, None), oracle_y(x, W, None), "no bias")


def test_fp32_k_multiple_of_4_takes_fast_kernels():
    """FP32 rows have a 16-byte pitch whenever K % 4 == 0 (16-bit rows need K % 8 == 0)."""
    for M, N, K, kernel in ((4, 96, 516, KERNEL_DECODE), (80, 96, 516, KERNEL_PREFILL)):
        plan = B.det_linear_plan_w(M, N, K, "fp32")
        assert B.det_linear_plan_get_params(plan).kernel == kernel
        plan.close()
        x, W, b = inputs.make_case_w(M, N, K, "fp32")
        want = oracle_y(x, W, b)
        assert_bits_equal(run_gpu(x, W, b, kernel=kernel), want, "fast")
        assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, "generic")


def test_fp16_special_values_bit_exact():
    """Every class of binary16 pattern in the weights: subnormals (smallest, largest), signed zeros,
    the largest finite value, and inputs that drive the products into the FP32 subnormal range."""
    M, N, K = 8, 64, 1024
    g = torch.Generator().manual_seed(7)
    x = torch.randn(M, K, generator=g)
    x[1, :] *= 1e-30
    x[2, :] *= 1e-38
    x[3, :] = -0.0
    x[4, :] *= 1e30
    W = (0.02 * torch.randn(N, K, generator=g)).to(torch.float16)
    Wb = inputs.weight_bits(W).copy()
    Wb[0, :] = 0x0001                       # smallest subnormal, 2^-24
    Wb[1, :] = 0x03FF                       # largest subnormal
    Wb[2, :] = 0x8000                       # -0
    Wb[3, :] = 0x7BFF                       # 65504
    Wb[4, ::2] = 0x83FF
    Wb[5, :] = torch.randint(0, 0x0400, (K,), generator=g, dtype=torch.int32).numpy().astype(np.uint16)
    W = torch.from_numpy(Wb.view(np.int16)).view(torch.float16)
    want = oracle_y(x, W, None)
    assert np.isfinite(want).all()
    for kernel in (KERNEL_GENERIC, KERNEL_DECODE):
        assert_bits_equal(run_gpu(x, W, None, kernel=kernel), want, f"kernel={kernel}")
    xp = torch.cat([x] * 9)[:70].contiguous()
    assert_bits_equal(run_gpu(xp, W, None, kernel=KERNEL_PREFILL), oracle_y(xp, W, None), "prefill")


def test_bf16_exact_weights_give_the_same_bits_in_every_format():
    """A BF16-representable weight widens to the same FP32 value from any format that can hold it, so
    the output bits must not depend on the storage format (FP16 only where the value fits)."""
    M, N, K = 8, 200, 2048
    x, W, b = inputs.make_int_case(M, N, K, seed=5)
    x = x + 0.25 * torch.randn(M, K, generator=torch.Generator().manual_seed(1))
    ref = run_gpu(x, W, b)
    assert_bits_equal(ref, oracle_y(x, W, b), "bf16")
    assert_bits_equal(run_gpu(x, W.to(torch.float16), b), ref, "fp16")
    assert_bits_equal(run_gpu(x, W.to(torch.float32), b), ref, "fp32")
    xp = torch.cat([x] * 9)[:70].contiguous()
    refp = run_gpu(xp, W, b)
    assert_bits_equal(run_gpu(xp, W.to(torch.float16), b), refp, "fp16 prefill")
    assert_bits_equal(run_gpu(xp, W.to(torch.float32), b), refp, "fp32 prefill")


@pytest.mark.parametrize("wfmt", FORMATS)
def test_full_size_decode_sampled(wfmt):
    """Llama-3-8B o-projection at M = 8, full size, sampled outputs against the oracle."""
    M, N, K = 8, 4096, 4096
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    got = run_gpu(x, W, b)
    rng = np.random.default_rng(11)
    ms = rng.integers(0, M, 400)
    ns = rng.integers(0, N, 400)
    want = oracle.linear_sampled(x.numpy(), inputs.weight_bits(W), b.numpy(), ms, ns, wfmt=wfmt)
    assert_bits_equal(got[ms, ns], want, "sampled")
    assert not np.isnan(got).any()


@pytest.mark.parametrize("wfmt", FORMATS)
def test_run_rejects_wrong_entry_point_and_run_host_works(wfmt):
    M, N, K = 4, 128, 512
    x, W, b = inputs.make_case_w(M, N, K, wfmt)
    want = oracle_y(x, W, b)
    plan = B.det_linear_plan_w(M, N, K, wfmt)
    xh, yh = x.pin_memory(), torch.empty(M, N).pin_memory()
    B.det_linear_run_host(plan, xh, W.cuda(), b.cuda(), yh)
    assert_bits_equal(yh.numpy(), want, "run_host")
    if wfmt == "fp32":
        y = torch.empty(M, N, device="cuda")
        st = B.lib().det_linear_run(plan.handle, x.cuda().data_ptr(), W.cuda().data_ptr(), None, y.data_ptr(), None)
        assert st == 1 and "det_linear_run_w" in B.det_last_error()
    plan.close()
    with pytest.raises(B.DetLinearError):
        B.det_linear_plan_w(M, N, K, 7)
