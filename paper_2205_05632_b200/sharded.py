"""Workers sharded over the ranks of a process group, one process per GPU (Algorithm 2 as the paper
states it: every worker compresses its own corrected gradient and only the compressed gradient travels).

Rank r holds workers r * n_local ... (r + 1) * n_local - 1 of n_total = world * n_local: their
gradients and error accumulators never leave its GPU. One step is compress() on the local rows, an
all-gather of the message buffers - (index, value) pairs for Top-k, sign words and scales for
Block-Sign: n_total * K * 8 bytes or n_total * (d / 8 + 4 M) bytes in total - and apply() on every
rank. Every rank plays the server on its own replica of theta, m, v, v-hat; the update is a
function of the gathered messages alone (the sum over workers is exact, hence order-free, while the
magnitudes met at one coordinate lie within about 2^24 of one another), so the replicas stay bit-identical
and theta is never broadcast. The collective is torch.distributed's (NCCL between GPUs); the gathered rows land in
this rank's own memory and the kernels read them with ordinary loads.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch

from .binding import CompAMS


def shard_rows(n_total: int, world: int, rank: int) -> Tuple[int, int]:
    """(first worker, number of workers) of `rank` when n_total workers are dealt evenly to `world` ranks."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank %d outside a group of %d" % (rank, world))
    if n_total < world or n_total % world:
        raise ValueError("%d workers cannot be dealt evenly to %d ranks" % (n_total, world))
    per = n_total // world
    return rank * per, per


def exchange(buffers: Sequence[torch.Tensor], first_row: int, rows: int, group=None) -> None:
    """Completes every [n_total, width] buffer of which this rank has filled rows first_row ...
    first_row + rows - 1: afterwards each rank holds every rank's rows. Ranks must hold equally many
    rows, in rank order. With a single process (no initialised group) there is nothing to do."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return
    world = dist.get_world_size(group)
    if world == 1:
        return
    on_device = dist.get_backend(group) == "nccl"
    for buf in buffers:
        if buf.shape[0] != world * rows:
            raise ValueError("a buffer of %d rows cannot hold %d rows from each of %d ranks" % (buf.shape[0], rows, world))
        if buf.is_cuda and not on_device:
            # a group whose backend moves host memory only (gloo): this rank's rows go to the host (the copy waits
            # for the work that wrote them, on the current stream), the gathered rows come back from a pinned buffer
            mine = buf[first_row:first_row + rows].cpu()
            whole = torch.empty(buf.shape, dtype=buf.dtype, pin_memory=True)
            dist.all_gather_into_tensor(whole.view(-1), mine.view(-1), group=group)
            buf.copy_(whole, non_blocking=True)
            torch.cuda.current_stream().synchronize()  # `whole` is released on return
            continue
        mine = buf[first_row:first_row + rows].clone()  # the messages are small next to the gradients
        dist.all_gather_into_tensor(buf.view(-1), mine.view(-1), group=group)


class ShardedCompAMS:
    """The COMP-AMS optimizer of one rank in a job of `world` ranks with n_local workers each.

    step(grads_local, theta) takes this rank's [n_local, d] gradients and this rank's replica of theta;
    all ranks must call it together. Use the CUDA stream that was current at construction."""

    def __init__(self, n_local: int, d: int, block_offsets: Sequence[int], compressor: int, k_ratio: float = 1.0,
                 lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 group=None, stream: Optional[torch.cuda.Stream] = None):
        import torch.distributed as dist
        live = dist.is_available() and dist.is_initialized()
        self.group = group
        self.world = dist.get_world_size(group) if live else 1
        self.rank = dist.get_rank(group) if live else 0
        first, per = shard_rows(self.world * int(n_local), self.world, self.rank)
        self.opt = CompAMS(per, d, block_offsets, compressor, k_ratio, lr, beta1, beta2, eps, stream=stream,
                           n_total=self.world * per, first_worker=first)

    def step(self, grads_local: torch.Tensor, theta: torch.Tensor) -> None:
        self.opt.compress(grads_local)
        exchange(self.opt.message_buffers(), self.opt.first_worker, self.opt.n, self.group)
        self.opt.apply(theta)

    def message_bytes_per_step(self) -> int:
        """Bytes this rank receives from the others in one step's exchange."""
        return sum(b[0].numel() * b.element_size() for b in self.opt.message_buffers()) * (self.opt.n_total - self.opt.n)

    def total_message_bytes_per_step(self) -> int:
        """Bytes of all workers' compressed gradients of one step: n_total K 8 for Top-k and Random-k (a 32-bit
        index and a 32-bit value per kept coordinate), n_total (4 W + 4 M) for Block-Sign (W sign words, M scales)."""
        return sum(b[0].numel() * b.element_size() for b in self.opt.message_buffers()) * self.opt.n_total

    def close(self) -> None:
        self.opt.close()
