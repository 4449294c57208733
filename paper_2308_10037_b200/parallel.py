"""Row-sharded data-parallel gradient descent over ``torch.distributed``.

The sums of Algorithm 1 (err.X, sum err, sum loss) split over rows: every rank owns a contiguous block
of rows, forms its local sums, the ranks exchange the ``n+2`` sums (one all-gather per iteration, a few
hundred bytes to 16 KB -- pure latency), and every rank adds the gathered vectors in rank order and
applies the same update, so all ranks hold bit-identical parameters.  X never crosses ranks.

The arithmetic is supplied by two callables so that the orchestration can be exercised on CPU ranks
(gloo) without a GPU; ``fit_sharded_cuda`` plugs in the CUDA entry points.
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
