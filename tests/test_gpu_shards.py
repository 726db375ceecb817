"""Column shards (N-sharded tensor parallelism) on one GPU: the shards of a layer, computed one after
the other by independent plans, reproduce the bits of the whole-layer plan and of the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from paper_2609_25624_b200.sharded import shard_range
from tests.gpu_util import assert_bits_equal, oracle_y, run_gpu

pytestmark = pytest.mark.gpu


def run_sharded(x, W, b, world, in_place, align=8):
    M, K = x.shape
    N = W.shape[0]
    xd, Wd, bd = x.cuda(), W.cuda(), None if b is None else b.cuda()
    y_full = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for r in range(world):
        n0, cnt = shard_range(N, r, world, align)
        if cnt == 0:
            continue
        Ws = Wd[n0:n0 + cnt]                                   # contiguous rows of the full matrix
        bs = None if bd is None else bd[n0:n0 + cnt]
        if in_place:
            plan = B.det_linear_plan_shard(M, N, K, n0, cnt, N, inputs.weight_format_of(W))
            B.det_linear_run_shard(plan, xd, Ws, bs, y_full[:, n0:n0 + cnt])
        else:
            plan = B.det_linear_plan_shard(M, N, K, n0, cnt, cnt, inputs.weight_format_of(W))
            y_loc = torch.full((M, cnt), float("nan"), dtype=torch.float32, device="cuda")
            B.det_linear_run_shard(plan, xd, Ws, bs, y_loc)
            y_full[:, n0:n0 + cnt] = y_loc
        B.det_linear_plan_check(plan)
        d = B.det_linear_plan_describe(plan)
        assert d["shard"] == {"n_begin": n0, "n_count": cnt, "ldy": N if in_place else cnt}
        assert (d["S"], d["seg_len"]) == (oracle.order_params(M, N, K)["S"], oracle.order_params(M, N, K)["seg_len"])
        plan.close()
    torch.cuda.synchronize()
    return y_full.cpu().numpy()


@pytest.mark.parametrize("M,N,K", [(1, 1024, 512), (4, 2048, 1024), (8, 4096, 1024), (32, 1000, 2048), (3, 250, 520),
                                   (100, 1000, 1000), (130, 512, 1024)])
@pytest.mark.parametrize("world", [2, 3, 8])
def test_shards_reproduce_the_whole_layer(M, N, K, world):
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_gpu(x, W, b), want, "whole layer")
    assert_bits_equal(run_sharded(x, W, b, world, in_place=True), want, "in place")
    assert_bits_equal(run_sharded(x, W, b, world, in_place=False), want, "compact blocks")


def test_shard_uses_the_layers_split_not_its_own():
    """Prefill bucket: the layer (128, 4096, 4096) splits K in 8, a 1024-column shard planned on its own
    would split it in 16 -> different bits.  The shard plan must keep the layer's S.  The same in the
    decode bucket: a layer of 16384 rows is not split, a quarter of it planned on its own would be."""
    M, N, K = 128, 4096, 4096
    assert oracle.order_params(M, N, K)["S"] != oracle.order_params(M, N // 4, K)["S"]
    x, W, b = inputs.make_case(M, N, K)
    ns = np.arange(0, N, 37)
    ms = (np.arange(len(ns)) * 5) % M
    want = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns)
    got = run_sharded(x, W, b, 4, in_place=True)
    assert_bits_equal(got[ms, ns], want, "layer order")
    alone = run_gpu(x, W[:1024].contiguous(), b[:1024].contiguous())
    assert not np.array_equal(alone.view(np.uint32), got[:, :1024].view(np.uint32))
    # decode bucket
    M, N, K = 2, 16384, 1024
    assert oracle.order_params(M, N, K)["S"] != oracle.order_params(M, N // 4, K)["S"]
    x, W, b = inputs.make_case(M, N, K)
    want = oracle_y(x, W, b)
    assert_bits_equal(run_sharded(x, W, b, 4, in_place=True), want, "decode shards")
    alone = run_gpu(x, W[:4096].contiguous(), b[:4096].contiguous())
    assert not np.array_equal(alone.view(np.uint32), want[:, :4096].view(np.uint32))


def test_shard_other_formats_and_no_bias():
    M, N, K = 8, 1536, 1024
    for wfmt in ("fp16", "fp32"):
        x, W, b = inputs.make_case_w(M, N, K, wfmt)
        assert_bits_equal(run_sharded(x, W, None, 4, in_place=True), oracle_y(x, W, None), wfmt)


def test_shard_bad_arguments():
    for args in ((4, 1024, 512, -1, 8, 1024), (4, 1024, 512, 1020, 8, 1024), (4, 1024, 512, 0, 0, 1024),
                 (4, 1024, 512, 0, 16, 8)):
        with pytest.raises(B.DetLinearError):
            B.det_linear_plan_shard(*args)
    plan = B.det_linear_plan_shard(4, 1024, 512, 0, 512, 1024)
    xh, yh = torch.zeros(4, 512).pin_memory(), torch.zeros(4, 1024).pin_memory()
    W = torch.zeros(1024, 512, dtype=torch.bfloat16, device="cuda")
    st = B.lib().det_linear_run_host(plan.handle, xh.data_ptr(), W.data_ptr(), None, yh.data_ptr(), None)
    assert st == 1 and "shard" in B.det_last_error()
    plan.close()
