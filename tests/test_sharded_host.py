"""CPU checks of the column-parallel plumbing: shard arithmetic, and a world-size 2 and 3 gloo run in
which every rank computes its column block with the oracle (under the whole layer's order) and the
gathered matrix must equal the oracle's whole-layer result bit for bit."""
import os
import subprocess
import sys

import pytest

from paper_2609_25624_b200.sharded import shard_range

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("N", [1, 7, 8, 9, 250, 1000, 4096, 6144, 28672, 128256])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_shard_ranges_tile_the_columns(N, world):
    edge = 0
    for r in range(world):
        n0, cnt = shard_range(N, r, world)
        assert n0 == edge and cnt >= 0
        if n0 + cnt < N:
            assert cnt % 8 == 0 and n0 % 8 == 0            # every block but the last is a whole number of 8-column units
        edge = n0 + cnt
    assert edge == N
    counts = [shard_range(N, r, world)[1] for r in range(world)]
    assert max(counts) - min(counts) <= 8 + 7               # balanced to within one unit (+ the ragged tail)
    with pytest.raises(ValueError):
        shard_range(N, world, world)


_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from oracle import oracle
from paper_2609_25624_b200 import inputs
from paper_2609_25624_b200.sharded import shard_range, gather_columns
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
for (M, N, K) in ((2, 1024, 4096), (5, 250, 520), (70, 136, 264)):
    x, W, b = inputs.make_case(M, N, K)                      # seeded: every rank draws the same layer
    prm = oracle.order_params(M, N, K)                       # the LAYER's order, not the shard's
    n0, cnt = shard_range(N, rank, world)
    bits = inputs.weight_bits(W)
    y_loc = oracle.linear(x.numpy(), bits[n0:n0 + cnt], b.numpy()[n0:n0 + cnt], params=prm) if cnt else np.zeros((M, 0), np.float32)
    y = gather_columns(torch.from_numpy(np.ascontiguousarray(y_loc)), N)
    want = oracle.linear(x.numpy(), bits, b.numpy())
    assert y.shape == (M, N)
    assert np.array_equal(y.numpy().view(np.uint32), want.view(np.uint32)), (M, N, K)
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


@pytest.mark.parametrize("world,port", [(2, "29541"), (3, "29542")])
def test_gathered_shards_equal_the_whole_layer_gloo(tmp_path, world, port):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=port, WORLD_SIZE=str(world), CUDA_VISIBLE_DEVICES="",
               OMP_NUM_THREADS="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(world)]
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err
        assert "ok" in out
