"""Fixed-order decode attention on the GPU against the oracle: bit-exact on every element, for shapes that
span one and several 128-key chunks and 256-key segments with ragged tails, grouped-query heads, head
dimensions that leave lanes idle, extreme score ranges (weights that underflow), and invariance across
runs, streams, batch size and SM-limited green contexts."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from tests.gpu_util import assert_bits_equal

pytestmark = pytest.mark.gpu


def make_qkv(B_, Hq, Hkv, T, D, seed, spread=1.0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B_, Hq, D, generator=g) * spread
    k = torch.randn(B_, Hkv, T, D, generator=g)
    v = torch.randn(B_, Hkv, T, D, generator=g)
    return q, k, v


def run_gpu_attention(q, k, v, scale, stream=None):
    o = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
    B.det_attention_decode(q.cuda(), k.cuda(), v.cuda(), scale, o, stream=stream)
    torch.cuda.synchronize()
    return o.cpu().numpy()


SHAPES = [(1, 1, 1, 1, 128), (2, 4, 1, 7, 64), (1, 8, 2, 128, 128), (3, 8, 8, 129, 128), (2, 32, 8, 300, 128),
          (1, 4, 2, 513, 96), (2, 16, 2, 1000, 128), (1, 2, 1, 260, 256), (1, 8, 4, 77, 132), (4, 32, 8, 2048, 128),
          (1, 1, 1, 4096, 128), (2, 8, 1, 1500, 128)]


@pytest.mark.parametrize("B_,Hq,Hkv,T,D", SHAPES)
def test_attention_bit_exact(B_, Hq, Hkv, T, D):
    q, k, v = make_qkv(B_, Hq, Hkv, T, D, seed=T * 7 + D)
    scale = float(np.float32(1.0 / math.sqrt(D)))
    want = oracle.attention_decode(q.numpy(), k.numpy(), v.numpy(), scale)
    got = run_gpu_attention(q, k, v, scale)
    assert not np.isnan(got).any()
    assert_bits_equal(got, want, f"attention {B_},{Hq},{Hkv},{T},{D}")


@pytest.mark.parametrize("B_,Hq,Hkv,T,D", [(2, 8, 2, 1000, 128), (1, 32, 8, 2049, 128), (3, 4, 4, 513, 96), (1, 8, 1, 4096, 128),
                                           (2, 2, 1, 260, 256), (1, 8, 2, 255, 128), (1, 4, 1, 16500, 64)])
def test_attention_same_bits_for_every_cluster_size(B_, Hq, Hkv, T, D):
    """The keys of a row are spread over 1, 2, 4, 8 or 16 thread blocks (row maxima, denominators and segment sums meet
    through distributed shared memory): schedule only, every cluster size reproduces the oracle's bits."""
    q, k, v = make_qkv(B_, Hq, Hkv, T, D, seed=T + D)
    scale = float(np.float32(1.0 / math.sqrt(D)))
    want = oracle.attention_decode(q.numpy(), k.numpy(), v.numpy(), scale)
    try:
        for c in (1, 2, 4, 8, 16, 0):
            B.det_test_attention_set_split(c)
            assert_bits_equal(run_gpu_attention(q, k, v, scale), want, f"cluster of {c}")
    finally:
        B.det_test_attention_set_split(0)


def test_attention_extreme_scores_and_zero_query():
    # sharply peaked softmax: most weights underflow to subnormals or zero
    q, k, v = make_qkv(2, 8, 2, 700, 128, seed=3, spread=6.0)
    want = oracle.attention_decode(q.numpy(), k.numpy(), v.numpy(), 1.0)
    assert_bits_equal(run_gpu_attention(q, k, v, 1.0), want, "peaked")
    # q = 0: uniform weights, l = T exactly
    q0 = torch.zeros_like(q)
    want = oracle.attention_decode(q0.numpy(), k.numpy(), v.numpy(), 0.5)
    assert_bits_equal(run_gpu_attention(q0, k, v, 0.5), want, "uniform")


def test_attention_invariance():
    """One result for a row whatever the batch around it, the stream and the number of SMs."""
    B_, Hq, Hkv, T, D = 8, 32, 8, 1024, 128
    q, k, v = make_qkv(B_, Hq, Hkv, T, D, seed=11)
    scale = float(np.float32(1.0 / math.sqrt(D)))
    base = run_gpu_attention(q, k, v, scale)
    assert_bits_equal(base, oracle.attention_decode(q.numpy(), k.numpy(), v.numpy(), scale), "oracle")
    for _ in range(5):
        assert_bits_equal(run_gpu_attention(q, k, v, scale), base, "repeat")
    # batch invariance: batch row 3 on its own
    one = run_gpu_attention(q[3:4], k[3:4], v[3:4], scale)
    assert_bits_equal(one[0], base[3], "batch of one")
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        assert_bits_equal(run_gpu_attention(q, k, v, scale, stream=st), base, "second stream")
    for sms in (8, 64):
        try:
            stream_ptr, handle, granted = B.det_test_green_stream_create(sms)
        except B.DetLinearError:
            continue
        try:
            assert_bits_equal(run_gpu_attention(q, k, v, scale, stream=stream_ptr), base, f"{granted} SMs")
        finally:
            B.det_test_green_stream_destroy(handle)


def test_attention_large_clusters_on_few_sms():
    """A 16-block cluster may not fit the SMs a stream is confined to: the launcher then halves the cluster (schedule
    only) and the bits stay the same."""
    q, k, v = make_qkv(1, 4, 1, 16500, 64, seed=5)
    scale = 0.125
    want = oracle.attention_decode(q.numpy(), k.numpy(), v.numpy(), scale)
    try:
        B.det_test_attention_set_split(16)
        assert_bits_equal(run_gpu_attention(q, k, v, scale), want, "whole device")
        for sms in (8, 16):
            try:
                stream_ptr, handle, granted = B.det_test_green_stream_create(sms)
            except B.DetLinearError:
                continue
            try:
                assert_bits_equal(run_gpu_attention(q, k, v, scale, stream=stream_ptr), want, f"{granted} SMs")
            finally:
                B.det_test_green_stream_destroy(handle)
    finally:
        B.det_test_attention_set_split(0)


def test_attention_argument_checks():
    q, k, v = make_qkv(1, 6, 2, 16, 128, seed=1)              # 3 query heads per KV head: not served
    o = torch.empty(1, 6, 128, device="cuda")
    with pytest.raises(B.DetLinearError) as ei:
        B.det_attention_decode(q.cuda(), k.cuda(), v.cuda(), 1.0, o)
    assert ei.value.status == 2
    q, k, v = make_qkv(1, 4, 1, 200000, 128, seed=1)          # scores do not fit in shared memory, however the row is split
    o = torch.empty(1, 4, 128, device="cuda")
    with pytest.raises(B.DetLinearError) as ei:
        B.det_attention_decode(q.cuda(), k.cuda(), v.cuda(), 1.0, o)
    assert ei.value.status == 2 and "shared memory" in B.det_last_error()
    assert B.lib().det_attention_decode(None, None, None, 1.0, 1, 1, 1, 1, 4, None, None) == 1
