"""Training-set parallelism over several GPUs (Section 4.3: error and gradient are additive over disjoint
subsets of the patterns, so the patterns are partitioned, the parameters replicated and the per-worker
results summed).  Host-side plumbing only: which slice of the pattern stream a rank evaluates, and the one
exchange per evaluation, a sum of the concatenated gradient and of the loss over the ranks through
torch.distributed (NCCL on GPUs; the same code runs on CPU tensors over gloo in the tests).
"""
from __future__ import annotations


def shard_range(rank: int, world: int, patterns_per_rank: int):
    """[first, last) pattern of `rank` when every rank evaluates `patterns_per_rank` patterns of one stream."""
    if not (0 <= rank < world) or patterns_per_rank < 0:
        raise ValueError("bad shard request")
    first = rank * patterns_per_rank
    return first, first + patterns_per_rank


def split_range(n_patterns: int, world: int, rank: int):
    """[first, last) of `rank` when a fixed set of n_patterns is divided as evenly as possible (the first
    n_patterns % world ranks get one more)."""
    if not (0 <= rank < world) or n_patterns < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_patterns, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


class GradientExchange:
    """Sums per-rank gradients in place.  One flat buffer is kept, so an exchange is one collective for all
    gradient tensors plus one for the loss.

    ordered=False: all-reduce (the library picks the order of the additions).
    ordered=True:  all-gather, then every rank adds the per-rank vectors in rank order: the sum does not depend on
                   the collective's algorithm and is bitwise the same on every rank (the on-device reductions of the
                   library are fixed-order too, so the whole evaluation then repeats bit for bit)."""

    def __init__(self, tensors, dist=None, ordered=False):
        import torch
        self.dist = dist
        self.ordered = ordered
        self.sizes = [int(t.numel()) for t in tensors]
        self.flat = torch.empty(sum(self.sizes), dtype=tensors[0].dtype, device=tensors[0].device)
        self.gathered = None

    def all_reduce(self, tensors, loss):
        """tensors: list of gradient tensors (same shapes as at construction); loss: 1-element tensor."""
        import torch
        if self.dist is None or self.dist.get_world_size() == 1:
            return
        torch.cat([t.reshape(-1) for t in tensors], out=self.flat)
        if self.ordered:
            world = self.dist.get_world_size()
            n = self.flat.numel()
            if self.gathered is None:
                # one row per rank; the loss has its own dtype (double) and travels in its own gather below
                self.gathered = torch.empty(world * n, dtype=self.flat.dtype, device=self.flat.device)
            self.dist.all_gather_into_tensor(self.gathered, self.flat)
            parts = self.gathered.view(world, n)
            self.flat.copy_(parts[0])
            for r in range(1, world):
                self.flat.add_(parts[r])
            losses = torch.empty(world * loss.numel(), dtype=loss.dtype, device=loss.device)
            self.dist.all_gather_into_tensor(losses, loss.reshape(-1))
            lp = losses.view(world, -1)
            acc = lp[0].clone()
            for r in range(1, world):
                acc.add_(lp[r])
            loss.copy_(acc.view_as(loss))
        else:
            self.dist.all_reduce(self.flat)
            self.dist.all_reduce(loss)
        off = 0
        for t, n in zip(tensors, self.sizes):
            t.copy_(self.flat[off:off + n].view_as(t))
            off += n
