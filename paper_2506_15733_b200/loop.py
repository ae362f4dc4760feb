"""Algorithm 1 of the paper as a loop around the library: the native controller decides which model drafts
each problem's next candidate blocks, the caller's ``draft_fn`` produces them (it owns the models), the
fused CUDA step scores and selects, the chosen blocks are gathered and appended.

Marshalling only: every decision is taken by the controller (``specs_controller_*``) or by the kernels.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np

from . import binding


@dataclass
class DraftBatch:
    """What ``draft_fn`` returns for the problems that are still running, in the order of ``live``:
    device tensors of one beam step (see ``specs_beam_step``); ``gen_tok_logprob`` may be None when every
    block came from the target itself (pi_gen = pi_target)."""
    hidden: object
    token_ids: object
    block_offsets: object          # int64 [B+1]
    cand_offsets: object           # int32 [len(live)+1]
    reward: object
    uniforms: object
    gen_tok_logprob: Optional[object] = None


@dataclass
class LoopResult:
    traces: List[List[int]]                      # appended token ids per problem
    generators: List[List[int]] = field(default_factory=list)   # who drafted each step, per problem
    stats: dict = field(default_factory=dict)


def run_specs(ctx: "binding.Context", controller: "binding.Controller", draft_fn: Callable[[np.ndarray, np.ndarray], DraftBatch],
              w_vocab, beta: float, tau: float, max_block_len: int, max_iters: int = 1 << 30) -> LoopResult:
    """Runs the loop until every problem reached its target length (or ``max_iters`` steps).

    ``draft_fn(generators, live)`` receives the controller's decision for all problems (GEN_TARGET /
    GEN_DRAFT / GEN_DONE) and the indices of the running ones, and returns their candidate blocks.
    The switch flag is Algorithm 1's (some candidate's reward above ``tau``)."""
    import torch
    P = controller.P
    result = LoopResult(traces=[[] for _ in range(P)], generators=[[] for _ in range(P)])
    for _ in range(max_iters):
        gens = controller.generators()
        live = np.nonzero(gens != binding.GEN_DONE)[0]
        if live.size == 0:
            break
        b = draft_fn(gens, live)
        dev = b.hidden.device
        rows, d = b.hidden.shape
        B, L = b.block_offsets.shape[0] - 1, live.size
        tok = torch.empty(rows, dtype=torch.float32, device=dev)
        blk = torch.empty(B, dtype=torch.float64, device=dev)
        gen = torch.empty(B, dtype=torch.float64, device=dev)
        wts = torch.empty(B, dtype=torch.float32, device=dev)
        chosen = torch.empty(L, dtype=torch.int32, device=dev)
        accept = torch.empty(L, dtype=torch.uint8, device=dev)
        ids_out = torch.empty((L, max_block_len), dtype=torch.int32, device=dev)
        len_out = torch.empty(L, dtype=torch.int32, device=dev)
        ws = torch.empty(ctx.score_workspace_bytes(rows, d, w_vocab.shape[0]), dtype=torch.uint8, device=dev)
        ctx.specs_beam_step(b.hidden, w_vocab, b.token_ids, b.block_offsets, b.cand_offsets, b.gen_tok_logprob,
                            b.reward, b.uniforms, beta, tau, tok, blk, gen, wts, chosen, accept, ws)
        ctx.specs_gather_chosen(b.token_ids, b.block_offsets, b.cand_offsets, chosen, ids_out, len_out)
        torch.cuda.synchronize(dev)
        h_chosen = np.full(P, -1, np.int32)
        h_flag = np.zeros(P, np.uint8)
        h_len = np.zeros(P, np.int64)
        h_chosen[live], h_flag[live], h_len[live] = chosen.cpu().numpy(), accept.cpu().numpy(), len_out.cpu().numpy()
        ids_host = ids_out.cpu().numpy()
        for j, p in enumerate(live):
            result.generators[p].append(int(gens[p]))
            if h_chosen[p] >= 0:
                result.traces[p].extend(ids_host[j, :h_len[p]].tolist())
        controller.advance(h_chosen, h_flag, h_len)
    result.stats = controller.stats()
    return result
