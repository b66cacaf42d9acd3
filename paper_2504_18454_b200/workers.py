"""Algorithm 1 with the K workers spread over several GPUs (the deployment the paper runs).

Rank r of G holds a context over its own K/G workers (worker indices r*K/G ... in the job) and
runs their inner steps locally: nothing is exchanged between synchronisations, and the branch
decisions come out of the shared (seed, t, k) stream, so every rank draws exactly what one
GPU holding all K workers would draw.  Every H steps the outer synchronisation runs as

    palsgd_outer_partial  ->  all-reduce(sum) of the exchange buffer  ->  palsgd_outer_finish

(Algorithm 1's All-Reduce of the outer gradient, an average by Sec. 2.2; Eq. (3), Eq. (4)); the
initial global model is formed the same way once (`init_global`).
The all-reduce is `torch.distributed`'s (NCCL over NVLink between GPUs); this module is only
the controller: which worker indices a rank owns, when to synchronise, and the three calls.
It holds no arithmetic of the method.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple


def worker_span(K_total: int, rank: int, world: int) -> Tuple[int, int]:
    """[k0, k1): the job's worker indices that `rank` of `world` holds.  K_total must divide evenly."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    if K_total % world != 0:
        raise ValueError(f"{K_total} workers do not divide over {world} ranks")
    per = K_total // world
    return rank * per, (rank + 1) * per


class DistributedPalsgd:
    """One rank's share of a job of K_total workers.

    ctx            a `Palsgd` context over this rank's workers (its K = K_total / world), built with
                   the job's H, p and seed
    exchange       a float32 tensor of ctx.exchange_numel() elements on the context's device, zeroed
    all_reduce_sum callable(tensor) that sums `tensor` in place over all ranks; default:
                   torch.distributed.all_reduce on the default process group
    """

    def __init__(self, ctx, exchange, K_total: int, rank: int, world: int,
                 all_reduce_sum: Optional[Callable] = None):
        self.ctx, self.exchange = ctx, exchange
        self.K_total, self.rank, self.world = int(K_total), int(rank), int(world)
        self.k0, k1 = worker_span(K_total, rank, world)
        if k1 - self.k0 != ctx.K:
            raise ValueError(f"context holds {ctx.K} workers, the rank's share is {k1 - self.k0}")
        if exchange.numel() < ctx.exchange_numel():
            raise ValueError("exchange buffer too small")
        ctx.set_worker_offset(self.k0)
        self.t = 0
        if all_reduce_sum is None:
            import torch.distributed as dist

            def all_reduce_sum(buf):
                if world > 1:
                    dist.all_reduce(buf, op=dist.ReduceOp.SUM)
        self._all_reduce = all_reduce_sum

    def init_global(self, stream: int = 0) -> None:
        """Once after the contexts have been created on every rank: the global model becomes the mean over
        ALL workers of the job (palsgd_init alone gives every rank the mean of its own workers)."""
        self.ctx.outer_partial(self.exchange.data_ptr(), stream)
        self._all_reduce(self.exchange)
        self.ctx.global_from_exchange(self.exchange.data_ptr(), self.K_total, stream)

    def ddp_step(self, lr_t: float, stream: int = 0) -> None:
        """One step of the DDP warm-up phase for the whole job: the gradients of all workers are averaged
        (local sums, all-reduce, division by K_total) and every rank takes the same optimizer step."""
        self.ctx.ddp_partial(self.exchange.data_ptr(), stream)
        self._all_reduce(self.exchange)
        self.ctx.ddp_finish(self.exchange.data_ptr(), self.K_total, lr_t, stream)
        self.t += 1

    def inner_step(self, lr_t: float, eta_t: float, stream: int = 0) -> None:
        self.ctx.inner_step(lr_t, eta_t, stream)
        self.t += 1

    def outer_sync(self, stream: int = 0) -> None:
        """The collective must run on, or be ordered with, `stream` (torch's current stream when the
        default all-reduce is used)."""
        self.ctx.outer_partial(self.exchange.data_ptr(), stream)
        self._all_reduce(self.exchange)
        self.ctx.outer_finish(self.exchange.data_ptr(), self.K_total, stream)

    def step(self, lr_t: float, eta_t: float, stream: int = 0) -> bool:
        """One iteration of Algorithm 1 for this rank's workers; True when it ended with the outer sync."""
        self.inner_step(lr_t, eta_t, stream)
        if self.t % self.ctx.H == 0:
            self.outer_sync(stream)
            return True
        return False
