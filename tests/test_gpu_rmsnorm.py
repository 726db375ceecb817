"""Fixed-order RMSNorm on the GPU (through the C ABI) against the CPU oracle: bit-exact."""
import hashlib

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25624_b200 import binding as B
from tests.gpu_util import assert_bits_equal

pytestmark = pytest.mark.gpu


def run(x, g, eps, stream=None):
    xd, gd = x.cuda(), g.cuda()
    y = torch.full(tuple(x.shape), float("nan"), dtype=torch.float32, device="cuda")
    B.det_rmsnorm(xd, gd, eps, y, stream=stream)
    torch.cuda.synchronize()
    return y.cpu().numpy()


def make(M, H, seed, scale=1.0):
    gen = torch.Generator().manual_seed(seed)
    x = scale * torch.randn(M, H, generator=gen)
    g = 1.0 + 0.1 * torch.randn(H, generator=gen)
    return x, g


@pytest.mark.parametrize("M,H", [(1, 4096), (8, 4096), (32, 4096), (64, 14336), (300, 4096), (7, 128), (5, 132), (3, 1),
                                 (9, 127), (4, 129), (2, 1000), (6, 515), (2048, 4096), (11, 8192)])
@pytest.mark.parametrize("eps", [1e-5, 0.0])
def test_bit_exact(M, H, eps):
    x, g = make(M, H, 1000 * M + H)
    assert_bits_equal(run(x, g, eps), oracle.rmsnorm(x.numpy(), g.numpy(), eps), f"{M}x{H} eps={eps}")


def test_hand_examples_and_special_values():
    H = 256
    x = torch.ones(3, H)
    x[1, 0] = 4096.0                          # only lane 0 loses its ones: ss = 2^24 + 248
    x[2] = 0.0
    x[2, 0], x[2, 4], x[2, 8] = 4096.0, 1.0, 1.0
    g = torch.linspace(-2, 2, H)
    want = oracle.rmsnorm(x.numpy(), g.numpy(), 0.0)
    got = run(x, g, 0.0)
    assert_bits_equal(got, want, "hand examples")
    assert np.array_equal(got[0], g.numpy())
    r1 = np.float32(1) / np.sqrt(np.float32(16777464.0) / np.float32(256))
    assert got[1, 1] == np.float32(np.float32(1) * r1) * g.numpy()[1]
    # subnormal and huge rows, signed zeros
    x = torch.randn(4, 1024, generator=torch.Generator().manual_seed(3))
    x[0] *= 1e-22                              # squares are subnormal or zero
    x[1] *= 1e18                               # ss near the top of the range
    x[2, ::2] = -0.0
    x[3] = 0.0
    g = torch.randn(1024, generator=torch.Generator().manual_seed(4))
    for eps in (0.0, 1e-6):
        want = oracle.rmsnorm(x.numpy(), g.numpy(), eps)
        got = run(x, g, eps)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        assert_bits_equal(np.nan_to_num(got, nan=0.0), np.nan_to_num(want, nan=0.0), f"special eps={eps}")


def test_misaligned_and_odd_lengths_same_bits():
    M, H = 6, 1024
    x, g = make(M, H, 77)
    want = oracle.rmsnorm(x.numpy(), g.numpy(), 1e-5)
    buf = torch.empty(M * H + 1, dtype=torch.float32, device="cuda")
    xd = buf[1:].view(M, H)
    xd.copy_(x)
    assert xd.data_ptr() % 16 != 0
    y = torch.empty(M, H, dtype=torch.float32, device="cuda")
    B.det_rmsnorm(xd, g.cuda(), 1e-5, y)
    assert_bits_equal(y.cpu().numpy(), want, "misaligned x (scalar path)")


def test_batch_stream_and_run_invariance():
    H = 4096
    x, g = make(64, H, 5)
    full = run(x, g, 1e-5)
    for M in (1, 3, 8, 33):
        assert_bits_equal(run(x[:M].contiguous(), g, 1e-5), full[:M], f"M={M}")
    s = torch.cuda.Stream()
    digests = set()
    for i in range(20):
        with torch.cuda.stream(s if i % 2 else torch.cuda.current_stream()):
            digests.add(hashlib.sha256(run(x, g, 1e-5, stream=s if i % 2 else None).tobytes()).hexdigest())
    assert len(digests) == 1


def test_bad_arguments():
    x = torch.zeros(2, 8, device="cuda")
    g = torch.ones(8, device="cuda")
    y = torch.empty(2, 8, device="cuda")
    with pytest.raises(B.DetLinearError):
        B.det_rmsnorm(x, g, -1.0, y)
    with pytest.raises(B.DetLinearError):
        B.det_rmsnorm(x, g, float("nan"), y)
    assert B.lib().det_rmsnorm(None, g.data_ptr(), 0.0, 2, 8, y.data_ptr(), None) == 1
