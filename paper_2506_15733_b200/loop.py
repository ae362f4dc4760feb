"""Algorithm 1 of the paper as a loop around the library: the native controller decides which model drafts
each problem's next candidate blocks, the caller's ``draft_fn`` produces them (it owns the models), the
CUDA path scores and selects, the chosen blocks are gathered and appended.

Every policy of the controller gets the selection rule and the switch rule its definition names
(Section 4.1, Baselines; Section 4.3, ablations):

    policy          selection                       flag handed to the controller
    SPECS           SubSample (Algorithm 2)         some reward above tau        (Algorithm 1, Step III)
    ONLY_DRAFT /    SubSample, or the highest       none needed (the generator never changes)
    ONLY_TARGET     reward with ``select_rule``
    RANDOM          SubSample                       none; the caller's uniforms decide the next generator
    DRAFT_START     SubSample                       no reward above tau          ("SPECS (pi_draft start)")
    RSD             highest reward                  picked reward below tau while the draft drafted (RSD++)

Marshalling only: every decision is taken by the controller (``specs_controller_*``) or by the kernels,
and whether a step's block was appended is asked from the controller, not re-derived here.
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


_SWITCH_RULE = {binding.POLICY_SPECS: binding.SWITCH_ANY_ABOVE,
                binding.POLICY_DRAFT_START: binding.SWITCH_NONE_ABOVE,
                binding.POLICY_RSD: binding.SWITCH_CHOSEN_BELOW}


def run_specs(ctx: "binding.Context", controller: "binding.Controller",
              draft_fn: Callable[[np.ndarray, np.ndarray], DraftBatch], w_vocab, beta: float, tau: float,
              max_block_len: int, max_iters: int = 1 << 30,
              select_rule: Optional[int] = None,
              switch_uniforms: Optional[Callable[[int], np.ndarray]] = None) -> LoopResult:
    """Runs the loop until every problem reached its target length (or ``max_iters`` steps).

    ``draft_fn(generators, live)`` receives the controller's decision for all problems (GEN_TARGET /
    GEN_DRAFT / GEN_DONE) and the indices of the running ones, and returns their candidate blocks.
    ``select_rule`` overrides the policy's selection (SELECT_SUBSAMPLE / SELECT_BEST_REWARD); RSD always
    takes the highest reward.  ``switch_uniforms(step)`` supplies the float32 [P] uniforms of POLICY_RANDOM
    (the method's random numbers are the caller's inputs) and is required for that policy."""
    import torch
    P = controller.P
    policy = controller.policy
    if policy == binding.POLICY_RANDOM and switch_uniforms is None:
        raise ValueError("POLICY_RANDOM needs switch_uniforms(step) -> float32 [P]")
    rule = binding.SELECT_BEST_REWARD if policy == binding.POLICY_RSD else \
        (binding.SELECT_SUBSAMPLE if select_rule is None else int(select_rule))
    switch_rule = _SWITCH_RULE.get(policy, binding.SWITCH_ANY_ABOVE)
    fused = policy == binding.POLICY_SPECS and rule == binding.SELECT_SUBSAMPLE
    result = LoopResult(traces=[[] for _ in range(P)], generators=[[] for _ in range(P)])
    for it in range(max_iters):
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
        flag = torch.empty(L, dtype=torch.uint8, device=dev)
        ids_out = torch.empty((L, max_block_len), dtype=torch.int32, device=dev)
        len_out = torch.empty(L, dtype=torch.int32, device=dev)
        ws = torch.empty(ctx.score_workspace_bytes(rows, d, w_vocab.shape[0]), dtype=torch.uint8, device=dev)
        if fused:
            ctx.specs_beam_step(b.hidden, w_vocab, b.token_ids, b.block_offsets, b.cand_offsets, b.gen_tok_logprob,
                                b.reward, b.uniforms, beta, tau, tok, blk, gen, wts, chosen, flag, ws)
        else:
            ctx.specs_score_blocks(b.hidden, w_vocab, b.token_ids, b.block_offsets, tok, None, blk, ws)
            gen_blk = None
            if b.gen_tok_logprob is not None:
                ctx.specs_block_sums(b.gen_tok_logprob, b.block_offsets, None, gen)
                gen_blk = gen
            ctx.specs_select(blk, gen_blk, b.reward, None, b.cand_offsets, beta, b.uniforms, rule, 0, switch_rule,
                             tau, chosen, wts, flag)
        ctx.specs_gather_chosen(b.token_ids, b.block_offsets, b.cand_offsets, chosen, ids_out, len_out)
        torch.cuda.synchronize(dev)
        h_chosen = np.full(P, -1, np.int32)
        h_flag = np.zeros(P, np.uint8)
        h_len = np.zeros(P, np.int64)
        h_chosen[live], h_flag[live], h_len[live] = chosen.cpu().numpy(), flag.cpu().numpy(), len_out.cpu().numpy()
        ids_host = ids_out.cpu().numpy()
        uniforms = None
        if policy == binding.POLICY_RANDOM:
            uniforms = np.ascontiguousarray(switch_uniforms(it), dtype=np.float32)
            if uniforms.shape != (P,):
                raise ValueError("switch_uniforms(step) must return P values")
        controller.advance(h_chosen, h_flag, h_len, uniforms)
        appended = controller.appended()
        for j, p in enumerate(live):
            result.generators[p].append(int(gens[p]))
            if appended[p]:
                result.traces[p].extend(ids_host[j, :h_len[p]].tolist())
    result.stats = controller.stats()
    return result
