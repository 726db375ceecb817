"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact, element by element."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import (KERNEL_DECODE, KERNEL_GENERIC, KERNEL_PREFILL, assert_bits_equal, oracle_y,
                            run_gpu)

pytestmark = pytest.mark.gpu

DECODE_SHAPES = [(1, 1024, 512), (1, 100, 512), (2, 77, 1000), (3, 130, 2304), (4, 96, 4096), (5, 33, 1024),
                 (8, 257, 1536), (8, 64, 14336), (13, 200, 1000), (16, 96, 2048), (17, 40, 768), (32, 128, 4096),
                 (33, 64, 640), (64, 50, 512), (7, 9, 8), (1, 1, 8), (64, 1, 256)]
RAGGED_DECODE = [(1, 10, 1), (3, 17, 7), (5, 33, 1001), (8, 50, 1004), (4, 31, 250)]
PREFILL_SHAPES = [(65, 129, 1000), (100, 1000, 1000), (130, 200, 1792), (128, 256, 1024), (200, 72, 4096),
                  (65, 1, 8), (67, 5, 3)]


def test_plan_params_match_oracle_rule():
    for shp in DECODE_SHAPES + RAGGED_DECODE + PREFILL_SHAPES + [(8, 4096, 14336), (2048, 28672, 4096)]:
        assert B.det_linear_plan_params(*shp).as_dict() == oracle.order_params(*shp), shp
    plan = B.det_linear_plan(1, 1024, 512)
    d = B.det_linear_plan_describe(plan)
    assert (d["bucket"], d["V"], d["L"], d["P"], d["S"], d["seg_len"]) == ("decode", 4, 32, 1, 2, 256)
    assert d["order_version"] == oracle.ORDER_VERSION == B.det_order_version()
    plan.close()


def test_config1_bit_exact():
    """M=1, K=512, N=1024, seed 0, bias present: bit-exact against the oracle on every kernel."""
    x, W, b = inputs.make_case(1, 1024, 512, seed=0)
    want = oracle_y(x, W, b)
    for kernel in (None, KERNEL_GENERIC, KERNEL_DECODE):
        assert_bits_equal(run_gpu(x, W, b, kernel=kernel), want, f"kernel={kernel}")
    assert_bits_equal(run_gpu(x, W, None), oracle_y(x, W, None), "no bias")


@pytest.mark.parametrize("M,N,K", DECODE_SHAPES)
def test_decode_bit_exact_all_tilings(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, "generic")
    n_tilings = 0
    for variant in range(0, 16):               # 0 = automatic choice, then every compiled tiling of this batch class
        try:
            got = run_gpu(x, W, b, kernel=KERNEL_DECODE, variant=variant)
        except B.DetLinearError:
            break
        assert_bits_equal(got, want, f"variant={variant}")
        n_tilings = variant
    # tilings whose segment groups do not divide S cannot run the shape
    assert n_tilings >= (4 if oracle.order_params(M, N, K)["S"] == 2 else 2)
    assert_bits_equal(run_gpu(x, W, b, max_blocks=1), want, "one block")
    assert_bits_equal(run_gpu(x, W, b, max_blocks=3), want, "three blocks")


@pytest.mark.parametrize("M,N,K", RAGGED_DECODE)
def test_decode_ragged_bit_exact(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    assert_bits_equal(run_gpu(x, W, b), oracle_y(x, W, b), "ragged")


@pytest.mark.parametrize("M,N,K", PREFILL_SHAPES)
def test_prefill_bit_exact(M, N, K):
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_GENERIC), want, "generic")
    assert_bits_equal(run_gpu(x, W, b), want, "automatic")
    assert_bits_equal(run_gpu(x, W, None), oracle_y(x, W, None), "no bias")


def test_misaligned_buffers_take_generic_path_same_bits():
    M, N, K = 4, 64, 512
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    xd = torch.empty(M * K + 1, dtype=torch.float32, device="cuda")[1:].view(M, K)
    xd.copy_(x)
    assert xd.data_ptr() % 16 != 0
    y = torch.empty(M, N, dtype=torch.float32, device="cuda")
    plan = B.det_linear_plan(M, N, K)
    B.det_linear_run(plan, xd, W.cuda(), b.cuda(), y)
    B.det_linear_plan_check(plan)
    assert_bits_equal(y.cpu().numpy(), want, "misaligned x")
    plan.close()


def test_special_values_bit_exact():
    """Subnormals, signed zeros, large magnitudes and cancellations: gradual underflow and signed
    zeros must match the oracle exactly (rule R1: IEEE-754 arithmetic, no flush to zero)."""
    M, N, K = 8, 64, 1024
    g = torch.Generator().manual_seed(99)
    x = torch.randn(M, K, generator=g)
    xb = x.view(torch.int32)
    xb[0, :] = torch.randint(1, 1 << 23, (K,), generator=g, dtype=torch.int32)            # subnormals
    xb[1, ::2] = torch.randint(1, 1 << 23, (K // 2,), generator=g, dtype=torch.int32) | (1 << 31)
    x[2, :] = 0.0
    x[3, :] = -0.0
    x[4, :] *= 1e30
    x[5, :] *= 1e-30
    x[6, 1::2] = -x[6, ::2]
    W = (0.02 * torch.randn(N, K, generator=g)).to(torch.bfloat16)
    Wb = inputs.bf16_bits(W).copy()
    Wb[0, :] = 0x0001                       # BF16 subnormal
    Wb[1, :] = 0x8000                       # -0
    Wb[2, :] = 0x7F7F                       # largest finite BF16
    Wb[3, ::2] = Wb[3, 1::2]
    W = inputs.bits_to_bf16(Wb)
    x[4, :] = x[4, :].clamp(-1e30, 1e30)
    want = oracle_y(x, W, None)
    finite = np.isfinite(want)
    for kernel in (KERNEL_GENERIC, KERNEL_DECODE):
        got = run_gpu(x, W, None, kernel=kernel)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        assert_bits_equal(np.where(np.isnan(want), 0, got), np.where(np.isnan(want), 0, want), f"kernel={kernel}")
    assert finite.sum() > want.size // 2


def test_batch_invariance_on_gpu():
    """Rule R4: row m of a batch-M call equals the M = 1 call of that row, for M <= 64."""
    N, K = 96, 2048
    x, W, b = inputs.make_case(64, N, K, seed=3)
    full = run_gpu(x, W, b)
    assert_bits_equal(full, oracle_y(x, W, b), "M=64")
    for M in (1, 2, 5, 8, 16, 31, 32, 33):
        assert_bits_equal(run_gpu(x[:M].contiguous(), W, b), full[:M], f"M={M}")
    assert_bits_equal(run_gpu(x[40:41].contiguous(), W, b), full[40:41], "row 40 alone")


def test_argmax_rows_gpu():
    g = torch.Generator().manual_seed(5)
    y = torch.randn(9, 5000, generator=g)
    y[2, 4000] = y[2, 17] = y[2].max() + 1
    y[3, :] = 1.5
    y[4, 0] = 100.0
    y[5, 4999] = 100.0
    y[6, 300] = float("nan")
    y[7, 10] = 0.0
    y[7, 11] = -0.0
    y[7, :10] = -1
    y[7, 12:] = -1
    want = oracle.argmax_rows(y.numpy())
    idx = torch.empty(9, dtype=torch.int32, device="cuda")
    B.det_argmax_rows(y.cuda(), idx)
    torch.cuda.synchronize()
    assert idx.cpu().tolist() == want.tolist()
    assert want[2] == 17 and want[3] == 0 and want[6] == 300 and want[7] == 10
    # a single-column and a short row
    for n in (1, 31, 1025):
        z = torch.randn(3, n, generator=g)
        idx = torch.empty(3, dtype=torch.int32, device="cuda")
        B.det_argmax_rows(z.cuda(), idx)
        assert idx.cpu().tolist() == oracle.argmax_rows(z.numpy()).tolist()


def test_run_host_matches_device_run():
    M, N, K = 8, 300, 1024
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    plan = B.det_linear_plan(M, N, K)
    xh = x.pin_memory()
    yh = torch.empty(M, N, dtype=torch.float32).pin_memory()
    B.det_linear_run_host(plan, xh, W.cuda(), b.cuda(), yh)
    assert_bits_equal(yh.numpy(), want, "run_host")
    yh.zero_()
    B.det_linear_run_host_async(plan, xh, W.cuda(), b.cuda(), yh)
    torch.cuda.current_stream().synchronize()
    assert_bits_equal(yh.numpy(), want, "run_host_async")
    plan.close()


def test_bad_arguments_are_rejected():
    with pytest.raises(B.DetLinearError):
        B.det_linear_plan(0, 4, 8)
    with pytest.raises(B.DetLinearError):
        B.det_linear_plan_params(1, -1, 8)
    plan = B.det_linear_plan(2, 4, 8)
    rc = B.lib().det_linear_run(plan.handle, None, None, None, None, None)
    assert rc == 1 and "NULL" in B.det_last_error()
    with pytest.raises(B.DetLinearError):
        B.det_test_plan_force_kernel(plan, KERNEL_PREFILL)
    plan.close()


MID_BUCKET = [(65, 130, 520), (72, 256, 1024), (80, 200, 1000), (96, 144, 2048), (100, 1000, 1000), (112, 128, 512),
              (127, 129, 264), (130, 64, 512), (200, 72, 4096), (300, 136, 776)]


@pytest.mark.parametrize("M,N,K", MID_BUCKET)
def test_prefill_tile_heights_bit_exact(M, N, K):
    """The prefill tile height (80, 96, 112 or 128 rows) is schedule only: every height, forced or
    chosen automatically, reproduces the oracle's bits (the mid bucket 65 <= M < 128 and batch
    sizes just above a multiple of 128 get a shorter tile)."""
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    # 5 .. 8: the TMA-fed kernel with that many rows per thread; 15 .. 18: the register-staged kernel
    for variant in (0, 5, 6, 7, 8, 15, 16, 17, 18):
        assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_PREFILL, variant=variant), want, f"rows per thread {variant}")
    # K segments folded by the second launch instead of by the block that completes a tile
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_PREFILL, two_pass_combine=True), want, "two-pass combine")
    # the in-kernel fold leaves its tile counters at zero: a second run of the same plan gives the same bits
    plan = B.det_linear_plan(M, N, K)
    xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
    for rep in range(3):
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        B.det_linear_run(plan, xd, Wd, bd, y)
        torch.cuda.synchronize()
        assert_bits_equal(y.cpu().numpy(), want, f"repeat {rep}")
    plan.close()


def test_prefill_tile_choice():
    for M, bm in ((65, 80), (72, 80), (81, 96), (100, 112), (113, 128), (128, 128), (130, 80), (200, 112), (512, 128),
                  (2048, 128), (257, 96)):
        plan = B.det_linear_plan(M, 256, 512)
        d = B.det_linear_plan_describe(plan)
        plan.close()
        assert d["kernel"] == "prefill" and d["prefill_tile"]["bm"] == bm, (M, d)
        padded = -(-M // bm) * bm
        assert all(padded <= -(-M // h) * h for h in (80, 96, 112, 128)), (M, bm)
    plan = B.det_linear_plan(100, 256, 512)
    with pytest.raises(B.DetLinearError):
        B.det_test_plan_set_variant(plan, 3)
    plan.close()


def test_plan_tune_changes_the_schedule_only():
    """det_linear_plan_tune pins the fastest tiling; the bits before and after are the oracle's."""
    for (M, N, K) in ((2, 6144, 4096), (8, 1000, 1024), (24, 4096, 4096)):
        x, W, b = inputs.make_case(M, N, K)
        xd, Wd, bd = x.cuda(), W.cuda(), b.cuda()
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        plan = B.det_linear_plan(M, N, K)
        B.det_linear_run(plan, xd, Wd, bd, y)
        torch.cuda.synchronize()
        before = y.cpu().numpy()
        variant, us = B.det_linear_plan_tune(plan, xd, Wd, bd, y)
        assert variant >= 1 and us > 0
        d = B.det_linear_plan_describe(plan)
        assert d["variant"] == variant and d["decode_tiling"]["blocks_per_sm"] >= 1
        y.fill_(float("nan"))
        B.det_linear_run(plan, xd, Wd, bd, y)
        B.det_linear_plan_check(plan)
        after = y.cpu().numpy()
        plan.close()
        if N * K <= 4096 * 4096 and M <= 8:
            assert_bits_equal(before, oracle_y(x, W, b), f"before {M},{N},{K}")
        assert_bits_equal(after, before, f"after tuning {M},{N},{K}")
    # nothing to choose in the prefill bucket
    x, W, b = inputs.make_case(100, 256, 512)
    plan = B.det_linear_plan(100, 256, 512)
    y = torch.empty(100, 256, device="cuda")
    assert B.det_linear_plan_tune(plan, x.cuda(), W.cuda(), b.cuda(), y) == (0, -1.0)
    plan.close()


@pytest.mark.parametrize("M,N,K", [(70001, 24, 64), (1048700, 8, 32)])
def test_prefill_very_tall_batches(M, N, K):
    """Batches far taller than a grid dimension: the activation transpose walks the rows in slabs of 2^20 rows,
    the multiply kernel numbers its tiles in one dimension.  Every element against the oracle."""
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    plan = B.det_linear_plan(M, N, K)
    d = B.det_linear_plan_describe(plan)
    assert d["kernel"] == "prefill" and d["prefill_tile"]["feed"] == "tma"
    plan.close()
    assert_bits_equal(run_gpu(x, W, b), want, "automatic")
    assert_bits_equal(run_gpu(x, W, b, variant=18), want, "register-staged")


@pytest.mark.parametrize("M,N,K", [(130, 40, 8), (70, 16, 24), (200, 8, 40), (66, 300, 32), (129, 129, 72)])
def test_prefill_very_short_k(M, N, K):
    """One or two slabs of K, shorter than a slab, not a multiple of it: the TMA-fed kernel against the oracle,
    every element, for BF16 and for FP32 weights (K a multiple of 8 serves both)."""
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b, kernel=KERNEL_PREFILL), want, "bf16")
    W32 = W.float()
    assert_bits_equal(run_gpu(x, W32, b, kernel=KERNEL_PREFILL), oracle_y(x, W32, b), "fp32 weights")
    if K % 8 == 0 and K >= 12:
        W32s = W32[:, : K - 4].contiguous()             # K a multiple of 4 only: the four-element tail
        xs = x[:, : K - 4].contiguous()
        assert_bits_equal(run_gpu(xs, W32s, b, kernel=KERNEL_PREFILL), oracle_y(xs, W32s, b), "fp32 weights, K % 8 == 4")
