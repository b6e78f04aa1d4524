"""Training-set parallelism over several GPUs (Section 4.3: error and gradient are additive over disjoint
subsets of the patterns, so the patterns are partitioned, the parameters replicated and the per-worker
results summed).  Host-side plumbing only: which slice of the pattern stream a rank evaluates, and the
exchange per evaluation, a sum of the gradient tensors and of the loss over the ranks through
torch.distributed (NCCL on GPUs; the same code runs on CPU tensors over gloo in the tests).

The exchange can be cut into groups of tensors that are launched one by one as their gradients become final
(Section 5.2 hides the reduce behind computation; here the top layer's gradient is summed over the ranks while
the products of the layers below still run): `start(group)` launches a group's collective, `finish()` waits for
all of them, copies the sums back and exchanges the loss.  `all_reduce()` is the two in one go.
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


def layer_groups(n_layers: int):
    """Tensor groups of a gradient list [dW_0 .. dW_{L-1}, db_0 .. db_{L-1}] in the order in which the library
    finishes them: the top layer first, the first layer last.  Group g holds (dW_w, db_w) of w = L-1-g."""
    return [[w, n_layers + w] for w in range(n_layers - 1, -1, -1)]


class GradientExchange:
    """Sums per-rank gradients in place.

    tensors: the gradient tensors; groups: lists of indices into `tensors` that travel together (default: one
    group with all of them).  Every group has its own flat buffer, so an exchange is one collective per group plus
    one for the loss.

    ordered=False: all-reduce (the library picks the order of the additions).
    ordered=True:  all-gather, then every rank adds the per-rank vectors in rank order: the sum does not depend on
                   the collective's algorithm and is bitwise the same on every rank (the on-device reductions of the
                   library are fixed-order too, so the whole evaluation then repeats bit for bit)."""

    def __init__(self, tensors, dist=None, ordered=False, groups=None):
        import torch
        self.dist = dist
        self.ordered = ordered
        self.groups = [list(g) for g in groups] if groups is not None else [list(range(len(tensors)))]
        seen = sorted(i for g in self.groups for i in g)
        if seen != list(range(len(tensors))):
            raise ValueError("every tensor must be in exactly one group")
        self.sizes = [[int(tensors[i].numel()) for i in g] for g in self.groups]
        self.flat = [torch.empty(sum(sz), dtype=tensors[g[0]].dtype, device=tensors[g[0]].device)
                     for g, sz in zip(self.groups, self.sizes)]
        self.gathered = [None] * len(self.groups)
        self.pending = [None] * len(self.groups)
        self.started = [False] * len(self.groups)

    def _active(self):
        return self.dist is not None and self.dist.get_world_size() > 1

    def start(self, g, tensors):
        """Launch the exchange of group g (its tensors must be final on the current stream / in memory)."""
        import torch
        if not self._active():
            return
        idx = self.groups[g]
        torch.cat([tensors[i].reshape(-1) for i in idx], out=self.flat[g])
        if self.ordered:
            world = self.dist.get_world_size()
            n = self.flat[g].numel()
            if self.gathered[g] is None:
                self.gathered[g] = torch.empty(world * n, dtype=self.flat[g].dtype, device=self.flat[g].device)
            self.pending[g] = self.dist.all_gather_into_tensor(self.gathered[g], self.flat[g], async_op=True)
        else:
            self.pending[g] = self.dist.all_reduce(self.flat[g], async_op=True)
        self.started[g] = True

    def finish(self, tensors, loss):
        """Wait for every group (starting those not started yet), write the sums back, sum the loss."""
        import torch
        if not self._active():
            return
        for g in range(len(self.groups)):
            if not self.started[g]:
                self.start(g, tensors)
        for g, idx in enumerate(self.groups):
            self.pending[g].wait()
            self.pending[g] = None
            self.started[g] = False
            if self.ordered:
                world = self.dist.get_world_size()
                parts = self.gathered[g].view(world, -1)
                self.flat[g].copy_(parts[0])
                for r in range(1, world):
                    self.flat[g].add_(parts[r])
            off = 0
            for i, n in zip(idx, self.sizes[g]):
                tensors[i].copy_(self.flat[g][off:off + n].view_as(tensors[i]))
                off += n
        if self.ordered:
            world = self.dist.get_world_size()
            losses = torch.empty(world * loss.numel(), dtype=loss.dtype, device=loss.device)
            self.dist.all_gather_into_tensor(losses, loss.reshape(-1))
            lp = losses.view(world, -1)
            acc = lp[0].clone()
            for r in range(1, world):
                acc.add_(lp[r])
            loss.copy_(acc.view_as(loss))
        else:
            self.dist.all_reduce(loss)

    def all_reduce(self, tensors, loss):
        """tensors: list of gradient tensors (same shapes as at construction); loss: 1-element tensor."""
        self.finish(tensors, loss)
