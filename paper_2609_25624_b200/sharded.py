"""Column-parallel (N-sharded) use of the linear layer across the GPUs of one node.

Each rank keeps a contiguous block of weight rows (= output columns) resident and computes that
block with a shard plan, whose reduction order is the whole layer's: the gathered result is
bit-identical to the single-GPU result for any world size.  The only exchange is one all-gather of
the output blocks (4*M*N bytes in total) through torch.distributed (NCCL on GPUs).  This module is
plumbing: shard arithmetic and the gather; every FLOP runs in the library's kernels.
"""
import torch
import torch.distributed as dist

from . import binding as B


def shard_range(N: int, rank: int, world: int, align: int = 8):
    """Contiguous column block of rank `rank`: (n_begin, n_count).  Blocks are multiples of `align`
    columns (so that every shard's W, b and y slices keep the 16-byte alignment the fast kernels
    want) except the last, which takes the remainder; ranks may get an empty block when N is tiny."""
    if not (0 <= rank < world) or N < 1 or align < 1:
        raise ValueError("bad shard request")
    units = -(-N // align)
    base, rem = divmod(units, world)
    first = rank * base + min(rank, rem)
    count = base + (1 if rank < rem else 0)
    n_begin = min(N, first * align)
    n_end = min(N, (first + count) * align)
    return n_begin, n_end - n_begin


def gather_columns(y_local: torch.Tensor, N: int, group=None, align: int = 8) -> torch.Tensor:
    """All-gather the ranks' column blocks (y_local = [M, n_count] of this rank, in shard_range order)
    into the full [M, N] matrix on every rank.  Blocks are padded to the widest one for the
    collective and cropped afterwards."""
    world = dist.get_world_size(group)
    M = y_local.shape[0]
    counts = [shard_range(N, r, world, align)[1] for r in range(world)]
    widest = max(counts)
    send = y_local if y_local.shape[1] == widest else torch.nn.functional.pad(y_local, (0, widest - y_local.shape[1]))
    send = send.contiguous()
    flat = torch.empty((world * M, widest), dtype=y_local.dtype, device=y_local.device)   # blocks stacked along dim 0
    dist.all_gather_into_tensor(flat, send, group=group)
    recv = flat.view(world, M, widest)
    return torch.cat([recv[r, :, :counts[r]] for r in range(world)], dim=1)


class ColumnParallelLinear:
    """y = x . up(W)^T (+ b) with W's rows split over the ranks of `group`.  `W_shard` / `b_shard` are
    this rank's rows (CUDA tensors); `run(x)` returns the full [M, N] output on every rank."""

    def __init__(self, N: int, K: int, W_shard: torch.Tensor, b_shard=None, group=None, wfmt="bf16", align: int = 8):
        self.N, self.K, self.group, self.wfmt, self.align = int(N), int(K), group, wfmt, align
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.n_begin, self.n_count = shard_range(self.N, self.rank, self.world, align)
        if tuple(W_shard.shape) != (self.n_count, self.K):
            raise ValueError(f"rank {self.rank} owns rows [{self.n_begin}, {self.n_begin + self.n_count}); "
                             f"W_shard has shape {tuple(W_shard.shape)}")
        self.W, self.b = W_shard, b_shard
        self._plans = {}

    def run(self, x: torch.Tensor) -> torch.Tensor:
        M = x.shape[0]
        y_local = torch.empty((M, self.n_count), dtype=torch.float32, device=x.device)
        if self.n_count:
            plan = self._plans.get(M)
            if plan is None:
                plan = self._plans[M] = B.det_linear_plan_shard(M, self.N, self.K, self.n_begin, self.n_count,
                                                                self.n_count, self.wfmt)
            B.det_linear_run_shard(plan, x, self.W, self.b, y_local)
        return gather_columns(y_local, self.N, self.group, self.align)

    def close(self):
        for p in self._plans.values():
            p.close()
        self._plans.clear()
