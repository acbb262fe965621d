"""The N workers of one RegTop-k problem spread over several GPUs, one process per GPU (torch.distributed).

Rank r of G holds a contiguous block of the workers and one library context for them; the residuals, the
accumulate/select/emit steps and the previous masks never leave their GPU.  Per round there is one exchange: an
all-gather of the k (index, value) pairs of every worker (8*N*k bytes in total), the paper's uplink of
Section 2.2 with every GPU acting as the server for itself.  Each rank then adds all N sparse vectors in worker
order (regtopk_aggregate_gathered), so every rank holds the same aggregate g bit for bit, which is also the g^{t-1}
that the next round's distortion needs.  The gathered pairs are in the rank's own memory before any kernel of the
library reads them.

This module holds no arithmetic of the method: it slices the workers, calls the collective and marshals arguments.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def worker_block(n_total: int, rank: int, world: int) -> Tuple[int, int]:
    """[first, first + count): the workers of `rank` when n_total workers are dealt to `world` ranks in contiguous
    blocks whose sizes differ by at most one (the first n_total % world ranks hold one more)."""
    if not (0 <= rank < world) or n_total < world:
        raise ValueError("need 0 <= rank < world <= n_total")
    base, extra = divmod(n_total, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def gather_pairs(idx: torch.Tensor, val: torch.Tensor, n_total: int, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gather of the ranks' [n_local, k] pairs into [n_total, k] tensors in worker order, on every rank.
    Works on the tensors' own device (NCCL for CUDA tensors, gloo for CPU tensors).  Blocks of unequal size are
    padded to the largest for the collective and cut back afterwards."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    counts = [worker_block(n_total, r, world)[1] for r in range(world)]
    if idx.shape[0] != counts[rank] or idx.shape != val.shape:
        raise ValueError("this rank's pairs do not match its block of the workers")
    k = idx.shape[1]
    most = max(counts)

    def run(x: torch.Tensor) -> torch.Tensor:
        if x.shape[0] < most:
            x = torch.cat([x, x.new_zeros((most - x.shape[0], k))], dim=0)
        out = x.new_empty((world * most, k))
        dist.all_gather_into_tensor(out, x.contiguous(), group=group)
        if all(c == most for c in counts):
            return out
        return torch.cat([out[r * most: r * most + counts[r]] for r in range(world)], dim=0)

    return run(idx), run(val)


class ShardedRegTopK:
    """RegTop-k for n_total workers of which this rank runs its block (see worker_block).

    step(grads_local) runs one whole round: worker_step on the local workers, the all-gather, the aggregation over
    all workers.  It returns (idx_all [n_total, k], val_all [n_total, k], g [d]); g is identical on every rank.
    """

    def __init__(self, d: int, n_total: int, k: int, mu: float = 4.0, omega: Optional[Sequence[float]] = None,
                 grad_dtype=torch.float32, flags: int = 0, y: float = 1.0, layers=None, group=None):
        from .binding import RegTopK
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.n_total = int(n_total)
        self.first, self.n_local = worker_block(self.n_total, self.rank, self.world)
        # the weights of all workers; the context needs its own workers' (its default would be 1/n_local)
        self.omega_all: List[float] = ([float(x) for x in omega] if omega is not None
                                       else [float(torch.tensor(1.0, dtype=torch.float32) / self.n_total)] * self.n_total)
        if len(self.omega_all) != self.n_total:
            raise ValueError("omega needs one weight per worker")
        self.lib = RegTopK(d, self.n_local, k, mu=mu, omega=self.omega_all[self.first: self.first + self.n_local],
                           grad_dtype=grad_dtype, flags=flags, y=y, layers=layers)
        self.d, self.k = self.lib.d, self.lib.k

    def step(self, grads_local: torch.Tensor):
        idx, val = self.lib.worker_step(grads_local)
        all_idx, all_val = gather_pairs(idx, val, self.n_total, self.group)
        g = self.lib.aggregate_gathered(all_idx, all_val, self.omega_all)
        return all_idx, all_val, g

    def close(self):
        self.lib.close()
