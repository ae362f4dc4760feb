"""Vocabulary-parallel scoring across ranks: the one exchange step of the path.

Each rank holds rows ``[v0, v1)`` of the LM-head weight, scores every drafted row against its
shard (``specs_score_partials``) and the ranks all-gather the 16-byte per-row partials; every rank
then folds them (``specs_merge_partials``) into the same per-token log-probabilities.  The exchange
is ``rows x 16`` bytes per rank, microseconds over NVLink, so a library all-gather into this GPU's
own memory is the right tool: there is no compute to overlap it with, and no kernel here ever reads
another GPU's memory.  ``torch.distributed`` carries the all-gather (NCCL on GPUs; the CPU tests
drive the same code with gloo and oracle-made partials).
"""
from __future__ import annotations

from typing import Tuple


def shard_bounds(V: int, world: int, rank: int, multiple: int = 256) -> Tuple[int, int]:
    """Rows [v0, v1) of the vocabulary held by ``rank``: contiguous, sizes as equal as whole
    multiples of ``multiple`` (one vocabulary tile) allow, the last rank taking the ragged tail."""
    tiles = -(-V // multiple)
    lo = (tiles * rank) // world * multiple
    hi = (tiles * (rank + 1)) // world * multiple
    return min(lo, V), min(hi, V)


def gather_partials(local, world: int):
    """All-gather the ranks' partials [rows, 4] into [world, rows, 4] (every rank gets all of them)."""
    import torch
    if world == 1:
        return local.unsqueeze(0)
    import torch.distributed as dist
    rows = local.shape[0]
    out = torch.empty((world * rows,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out, local.contiguous())      # rank-major concatenation along the rows
    return out.view((world, rows) + tuple(local.shape[1:]))


class VocabParallelScorer:
    """Scores drafted tokens against a vocabulary sharded over the ranks of the default process group."""

    def __init__(self, ctx, w_shard, V: int, rank: int, world: int):
        self.ctx, self.w_shard, self.V, self.rank, self.world = ctx, w_shard, int(V), int(rank), int(world)
        self.v0, self.v1 = shard_bounds(self.V, world, rank)
        if w_shard.shape[0] != self.v1 - self.v0:
            raise ValueError(f"rank {rank} must hold vocabulary rows [{self.v0}, {self.v1})")

    def token_logprobs(self, hidden, token_ids, tok_logprob, workspace=None):
        import torch
        rows, d = hidden.shape
        if workspace is None:
            workspace = torch.empty(self.ctx.score_workspace_bytes(rows, d, self.v1 - self.v0), dtype=torch.uint8,
                                    device=hidden.device)
        local = torch.empty((rows, 4), dtype=torch.float32, device=hidden.device)
        self.ctx.specs_score_partials(hidden, self.w_shard, token_ids, self.v0, local, workspace)
        allp = gather_partials(local, self.world)
        self.ctx.specs_merge_partials(allp, token_ids, self.V, tok_logprob)
        return tok_logprob
