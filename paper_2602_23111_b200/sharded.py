"""A batch whose tokens are spread over the ranks of a process group (data parallel).

Both token sums of the method cross ranks as sums of small matrices: the Gram matrix X^T X of
Algorithm 1's principal fit (d x d fp32, once per refresh) and the middle factor dY^T Z of the
weight gradient (d_out x (k+r) fp32, d / (k+r) times smaller than dW).  Everything else is local:
compression is row-wise, and the random basis is the same on every rank because it is a function
of (seed, draw counter) and U only.  The paper does not say how its multi-GPU runs share the
subspaces; this is one consistent way.

This module is plumbing over a basis object (gram, fit_principal_gram, draw_random, compress,
weight_grad_partial, weight_grad_finish) and torch.distributed; it holds none of the arithmetic.
"""
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_rows(n_rows: int, world: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the contiguous row range of `rank` when n_rows are dealt as evenly as
    possible (the first n_rows % world ranks get one more)."""
    if world <= 0 or not 0 <= rank < world or n_rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def all_reduce_sum(t: torch.Tensor, group=None) -> int:
    """Sum `t` over the group in place; returns the bytes this rank contributed (0 when alone)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return 0
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t.numel() * t.element_size()


class ShardedCompressor:
    """fit / compress / weight_grad for one linear layer's input when each rank holds a slice of
    the tokens.  After fit() every rank holds the same U, Q and c."""

    def __init__(self, basis, group=None):
        self.basis = basis
        self.group = group
        self.bytes_reduced = 0          # what this rank has put through collectives so far

    def fit(self, X_local: torch.Tensor, seed: int = 0, draw_counter: int = 0,
            ws: Optional[torch.Tensor] = None) -> None:
        C = self.basis.gram(X_local, ws=ws)
        self.bytes_reduced += all_reduce_sum(C, self.group)
        self.basis.fit_principal_gram(C, seed=seed, draw_counter=draw_counter, ws=ws)
        self.basis.draw_random(seed=seed, draw_counter=draw_counter, ws=ws)

    def compress(self, X_local: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        return self.basis.compress(X_local, out=out)

    def weight_grad(self, dY_local: torch.Tensor, Z_local: torch.Tensor, out: Optional[torch.Tensor] = None,
                    ws: Optional[torch.Tensor] = None, **finish_args) -> torch.Tensor:
        M = self.basis.weight_grad_partial(dY_local, Z_local, ws=ws)
        self.bytes_reduced += all_reduce_sum(M, self.group)
        return self.basis.weight_grad_finish(M, out=out, **finish_args)
