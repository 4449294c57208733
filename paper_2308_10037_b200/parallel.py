"""Row-sharded data-parallel gradient descent over ``torch.distributed``.

The sums of Algorithm 1 (err.X, sum err, sum loss) split over rows: every rank owns a contiguous block
of rows, forms its local sums, the ranks exchange the ``n+2`` sums (one all-gather per iteration, a few
hundred bytes to 16 KB -- pure latency), and every rank adds the gathered vectors in rank order and
applies the same update, so all ranks hold bit-identical parameters.  X never crosses ranks.

The arithmetic is supplied by two callables so that the orchestration can be exercised on CPU ranks
(gloo) without a GPU; ``fit_sharded_cuda`` plugs in the CUDA entry points.

``fit_sharded_fused`` is the same fit with the exchange inside the persistent kernel (``lr_fit_sharded``): no host loop and
no collective call per iteration; the ranks write their sums straight into each other's exchange buffers, which live in
symmetric memory.  Both give the same bits.
"""
from __future__ import annotations

from typing import Callable

import torch
import torch.distributed as dist


def shard_rows(m: int, rank: int, world: int) -> tuple[int, int]:
    """Row range [r0, r1) of ``rank``: blocks differ by at most one row, earlier ranks take the extra rows."""
    if not (0 <= rank < world) or m < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(m, world)
    r0 = rank * base + min(rank, extra)
    return r0, r0 + base + (1 if rank < extra else 0)


def fit_sharded(local_sums: Callable[[torch.Tensor], None], apply_sums: Callable[[torch.Tensor, int], None],
                sums: torch.Tensor, iters: int, group=None) -> None:
    """Runs ``iters`` synchronous steps.

    ``local_sums(sums)`` fills ``sums`` [n+2] (float64) with this rank's unnormalised sums at the current
    parameters; ``apply_sums(gathered, t)`` consumes the rank-ordered ``gathered`` [world, n+2] and updates
    the parameters for step ``t``.
    """
    world = dist.get_world_size(group)
    gathered = torch.empty((world, sums.numel()), dtype=sums.dtype, device=sums.device)
    rows = [gathered[r] for r in range(world)]          # views: the collective writes straight into `gathered`
    for t in range(int(iters)):
        local_sums(sums)
        dist.all_gather(rows, sums, group=group)        # supported by both NCCL and gloo
        apply_sums(gathered, t)


def fit_sharded_cuda(ctx, X_local, y_local, m_total: int, lr: float, iters: int, w, b, loss_hist=None, group=None):
    """Data-parallel fit on CUDA ranks (NCCL): ``w`` [n], ``b`` [1] are updated in place on every rank."""
    n = int(X_local.shape[1])
    sums = torch.empty(n + 2, dtype=torch.float64, device=X_local.device)

    def local_sums(out):
        ctx.shard_sums(X_local, y_local, w, b, out)

    def apply_sums(gathered, t):
        ctx.apply_sums(gathered, m_total, lr, w, b, None if loss_hist is None else loss_hist[t:t + 1])

    fit_sharded(local_sums, apply_sums, sums, iters, group)


class ExchangeBuffers:
    """This rank's exchange buffer for ``lr_fit_sharded`` in symmetric memory, and every rank's as this rank addresses it.

    The buffer is zeroed once here, with a barrier among the ranks after it; ``epoch`` counts the steps it has carried
    and has to advance in step on every rank (``fit_sharded_fused`` does that).
    """

    def __init__(self, n: int, device, group=None):
        import os
        # the exchange uses plain peer loads and stores only: no multicast object is wanted on the buffer
        os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")
        import torch.distributed._symmetric_memory as symm_mem
        from . import api
        group = dist.group.WORLD if group is None else group
        world = dist.get_world_size(group)
        self.n, self.world, self.rank, self.epoch = int(n), world, dist.get_rank(group), 0
        self.own = symm_mem.empty(api.exchange_bytes(world, n) // 8, dtype=torch.float64, device=device)
        handle = symm_mem.rendezvous(self.own, group)
        self.own.zero_()
        torch.cuda.synchronize(device)
        dist.barrier(group)                        # nobody stores into a buffer that is still being zeroed
        self.ptrs = [int(p) for p in handle.buffer_ptrs]
        self._handle = handle                      # keeps the peer mappings alive


def fit_sharded_fused(ctx, X_local, y_local, m_total: int, lr: float, iters: int, w, b, exchange: ExchangeBuffers,
                      loss_hist=None, wait_ms: int = 10_000):
    """Data-parallel fit with the exchange inside the kernel: one persistent launch per rank for all ``iters`` steps."""
    ctx.fit_sharded(X_local, y_local, m_total, lr, iters, w, b, exchange.rank, exchange.world, exchange.ptrs,
                    epoch=exchange.epoch, wait_ms=wait_ms, loss_hist=loss_hist)
    exchange.epoch += int(iters)
