"""Multi-GPU plumbing.  The path shards by rows of W (N) or by independent matrices with no
exchange step, so the only collective used is the timing reduction (max over ranks) and a
barrier.  Rows are split in multiples of 16 so that every shard keeps the tiled layout."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: str) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def shutdown() -> None:
    """Leave together: a barrier, then the process group is destroyed (a rank that simply exits while another is
    still inside a collective, or still connected to its store, makes that other rank fail at teardown)."""
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()


def shard_rows(N: int, rank: int, world: int, multiple: int = 16) -> tuple[int, int]:
    """[begin, end) of the rows owned by `rank`: contiguous, multiples of `multiple`, sizes differ by
    at most one block, union = [0, N).  N must be a multiple of `multiple`."""
    if N % multiple:
        raise ValueError(f"N={N} is not a multiple of {multiple}")
    blocks = N // multiple
    base, extra = divmod(blocks, world)
    begin = rank * base + min(rank, extra)
    end = begin + base + (1 if rank < extra else 0)
    return begin * multiple, end * multiple


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ---- row-sharded GEMV / GEMM: every rank owns a block of rows of W, the outputs are gathered -------------------------
class RowShard:
    """This rank's rows [begin, end) of one quantized matrix, ready for the tiled kernels.

    The path shards along N: rows of W are independent, so a rank computes its slice of y from its slice of the codes
    and scales and the full activation vector; the only exchange is the all-gather that makes y whole again for the
    next layer.  Shards are multiples of 16 rows (the tiled layout's row block)."""

    def __init__(self, packed_canonical, scales, K: int, bits: int, group: int, rank: int, world: int, repack=None,
                 repack_scales=None):
        N = packed_canonical.shape[0]
        self.N, self.K, self.bits, self.group, self.rank, self.world = N, K, bits, group, rank, world
        self.begin, self.end = shard_rows(N, rank, world)
        self.spans = [shard_rows(N, r, world) for r in range(world)]
        self.even = len({b - a for a, b in self.spans}) == 1
        rows = packed_canonical[self.begin:self.end].contiguous()
        srows = scales[self.begin:self.end].contiguous()
        if repack is None:  # the product path: the library's own repack kernels
            from . import binding
            repack = lambda p: binding.pot_repack(p, K, bits, 0)
            repack_scales = lambda s: binding.pot_repack_scales(s, K, group, 0)
        self.codes = repack(rows) if self.end > self.begin else rows
        self.scales = repack_scales(srows) if self.end > self.begin else srows


def gather_rows(y_local: torch.Tensor, y_full: torch.Tensor, shard: RowShard) -> torch.Tensor:
    """All-gather of the ranks' output slices along the row dimension (last dimension of y): y_full[..., begin:end] of
    every rank.  Equal shards use one all_gather_into_tensor; unequal ones (N / 16 not divisible by the world size) are
    padded to the largest shard.  With one rank it is a copy."""
    if shard.world == 1 or not dist.is_initialized():
        y_full[..., shard.begin:shard.end] = y_local
        return y_full
    lead = y_local.shape[:-1]
    width = max(b - a for a, b in shard.spans)
    send = y_local
    if y_local.shape[-1] != width:
        send = torch.zeros(lead + (width,), dtype=y_local.dtype, device=y_local.device)
        send[..., :y_local.shape[-1]] = y_local
    flat = send.contiguous().reshape(-1)
    recv_flat = torch.empty(shard.world * flat.numel(), dtype=y_local.dtype, device=y_local.device)
    dist.all_gather_into_tensor(recv_flat, flat)
    recv = recv_flat.view((shard.world,) + tuple(lead) + (width,))
    for r, (a, b) in enumerate(shard.spans):
        y_full[..., a:b] = recv[r][..., :b - a]
    return y_full


def sharded_gemv(shard: RowShard, x: torch.Tensor, y_full: torch.Tensor, workspace=None, stream=None, gemv=None) -> torch.Tensor:
    """y_full = W~ x with W row-sharded over the ranks: the local GEMV on this rank's rows, then the all-gather.
    `gemv(codes, scales, K, bits, group, x)` defaults to the library's tiled pot_gemv."""
    if gemv is None:
        from . import binding
        gemv = lambda c, s, K, bits, group, xx: binding.pot_gemv(c, s, K, bits, group, xx, binding.TILED, workspace=workspace,
                                                               stream=stream)
    if shard.end > shard.begin:
        y_local = gemv(shard.codes, shard.scales, shard.K, shard.bits, shard.group, x)
    else:
        y_local = torch.empty(0, dtype=x.dtype, device=x.device)
    return gather_rows(y_local, y_full, shard)
