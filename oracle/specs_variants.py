"""CPU oracle for the selection variants and the Algorithm-1 controller.  TEST INFRASTRUCTURE ONLY.

Same rules as specs_oracle.py: float64 numpy and plain Python loops, the definitions written out,
nothing imported from the product, never called by it.

What each function follows in the paper:

  select            Algorithm 2 with its candidate set L made explicit (P(i* = i) is proportional to
                    exp(S_i) * 1(i in L)), plus the selection rules of the systems the paper compares
                    with (Section 4.1, Baselines): beam search and RSD++ keep the candidate with the
                    highest PRM score, which is also what Algorithm 2 tends to as beta grows when
                    the log-ratio is dropped; "SPECS (no LL)" (Section 4.3) drops the log-ratio.
  switch_flags      Algorithm 1, Step III (some candidate's reward exceeds tau: the draft generates
                    next); its mirror for "SPECS (pi_draft start)" (Section 4.3: go to the target when
                    no candidate of the draft exceeds tau); and RSD++'s rule (Section 4.1: if the
                    reward of the selected draft candidate falls below the threshold, the step is
                    redone with the target).
  Controller        Algorithm 1 as a per-problem state machine: which model generates the next
                    block, appending the selected block, the switch, the stop at the target length;
                    with the ablation policies of Section 4.3 (only-small generation, random
                    switching, draft start) and the two baselines (beam search with one model, RSD++).

Readings taken where the paper is silent: the switch test looks at every candidate's reward, masked
or not; an empty problem (or one whose candidates are all masked) selects -1 and raises no flag;
ties in the highest reward go to the lowest index; Algorithm 1 only ever assigns pi_gen <- pi_draft,
while Section 2.3 and the reported share of target steps describe a decision taken at every step:
`sticky` chooses between the two.
"""
from __future__ import annotations

import numpy as np

SELECT_SUBSAMPLE, SELECT_BEST_REWARD = 0, 1
SCORE_NO_LL = 0x1
SWITCH_ANY_ABOVE, SWITCH_NONE_ABOVE, SWITCH_CHOSEN_BELOW = 0, 1, 2
GEN_TARGET, GEN_DRAFT, GEN_DONE = 0, 1, -1
POLICY_SPECS, POLICY_ONLY_DRAFT, POLICY_ONLY_TARGET, POLICY_RANDOM, POLICY_DRAFT_START, POLICY_RSD = 0, 1, 2, 3, 4, 5


def select(lp_target, lp_gen, reward, mask, cand_offsets, beta, uniforms, rule=SELECT_SUBSAMPLE, score_flags=0):
    """Per problem: the selected candidate (index local to the problem, -1 if none is eligible), the
    selection weights over the problem's candidates, and the top-two margin of the quantity maximised."""
    r = np.asarray(reward, dtype=np.float64)
    B = r.shape[0]
    beta = float(np.float32(beta))
    if lp_gen is None or (score_flags & SCORE_NO_LL):
        S = beta * r
    else:
        S = (np.asarray(lp_target, dtype=np.float64) - np.asarray(lp_gen, dtype=np.float64)) + beta * r
    in_L = np.ones(B, dtype=bool) if mask is None else (np.asarray(mask) != 0)
    P = len(cand_offsets) - 1
    chosen = np.full(P, -1, dtype=np.int32)
    margin = np.full(P, np.inf)
    w = np.zeros(B)
    for p in range(P):
        a, b = int(cand_offsets[p]), int(cand_offsets[p + 1])
        elig = [i for i in range(a, b) if in_L[i]]
        if not elig:
            continue
        if rule == SELECT_BEST_REWARD:
            key = {i: r[i] for i in elig}
        else:
            u = np.asarray(uniforms, dtype=np.float64)
            if np.any((u[a:b] <= 0.0) | (u[a:b] >= 1.0)):
                raise ValueError("uniforms must lie strictly inside (0, 1)")
            key = {i: S[i] - np.log(-np.log(u[i])) for i in elig}
        best = elig[0]
        for i in elig[1:]:
            if key[i] > key[best]:                    # strict: the lowest index keeps a tie
                best = i
        chosen[p] = best - a
        others = [key[i] for i in elig if i != best]
        if others:
            margin[p] = key[best] - max(others)
        if rule == SELECT_BEST_REWARD:
            w[best] = 1.0
        else:
            m = max(S[i] for i in elig)
            z = sum(np.exp(S[i] - m) for i in elig)
            for i in elig:
                w[i] = np.exp(S[i] - m) / z
    return chosen, w, margin


def switch_flags(reward, cand_offsets, chosen, tau, rule=SWITCH_ANY_ABOVE):
    r = np.asarray(reward, dtype=np.float32)
    tau = np.float32(tau)
    P = len(cand_offsets) - 1
    out = np.zeros(P, dtype=np.uint8)
    for p in range(P):
        a, b = int(cand_offsets[p]), int(cand_offsets[p + 1])
        if b <= a:
            continue
        any_above = bool(np.max(r[a:b]) > tau)
        if rule == SWITCH_ANY_ABOVE:
            out[p] = any_above
        elif rule == SWITCH_NONE_ABOVE:
            out[p] = not any_above
        else:
            out[p] = chosen[p] >= 0 and bool(r[a + int(chosen[p])] < tau)
    return out


class Controller:
    """Algorithm 1 for P problems.  generators() says who drafts the next n blocks of every problem
    (GEN_DONE once its target length is reached); advance() takes the step's selection results."""

    def __init__(self, P, policy=POLICY_SPECS, target_len=1024, sticky=False, p_target=0.5, max_steps=1 << 30):
        self.P, self.policy, self.target_len, self.sticky = P, policy, int(target_len), bool(sticky)
        self.p_target, self.max_steps = float(np.float32(p_target)), int(max_steps)
        start = GEN_DRAFT if policy in (POLICY_ONLY_DRAFT, POLICY_DRAFT_START, POLICY_RSD) else GEN_TARGET
        self.gen = [start] * P
        self.length = [0] * P
        self.steps = [0] * P
        self.target_steps = [0] * P          # blocks appended that the target generated
        self.target_calls = [0] * P          # generation rounds run by the target (RSD++ retries count)

    def generators(self):
        return [GEN_DONE if self._done(p) else self.gen[p] for p in range(self.P)]

    def _done(self, p):
        return self.length[p] >= self.target_len or self.steps[p] >= self.max_steps

    def advance(self, chosen, flag, chosen_len, uniforms=None):
        for p in range(self.P):
            if self._done(p):
                continue
            g = self.gen[p]
            if g == GEN_TARGET:
                self.target_calls[p] += 1
            if self.policy == POLICY_RSD and g == GEN_DRAFT and flag[p]:
                self.gen[p] = GEN_TARGET          # the draft's best candidate is too weak: redo with the target
                continue
            if chosen[p] >= 0:
                self.length[p] += int(chosen_len[p])
                self.steps[p] += 1
                if g == GEN_TARGET:
                    self.target_steps[p] += 1
            if self.policy == POLICY_SPECS:
                if flag[p]:
                    self.gen[p] = GEN_DRAFT
                elif not self.sticky:
                    self.gen[p] = GEN_TARGET
            elif self.policy == POLICY_DRAFT_START:
                if flag[p]:
                    self.gen[p] = GEN_TARGET
                elif not self.sticky:
                    self.gen[p] = GEN_DRAFT
            elif self.policy == POLICY_RANDOM:
                self.gen[p] = GEN_TARGET if float(np.float32(uniforms[p])) < self.p_target else GEN_DRAFT
            elif self.policy == POLICY_RSD:
                self.gen[p] = GEN_DRAFT


# --------------------------------------------------------------------------- both heads, and the append

def beam_step_dual(hidden_target_bits, w_target_bits, hidden_gen_bits, w_gen_bits, token_ids, block_offsets,
                   cand_offsets, reward, beta, uniforms, tau):
    """The step when the generator's log-probabilities are not given but computed: the drafted tokens are
    scored with the generator's own LM head (its hidden states and weights) exactly as with the target's
    (Section 2; the latency breakdown of Appendix E.1 lists scoring with the draft and with the target),
    and Eq. (1) takes the two block log-probabilities."""
    from oracle import specs_oracle as O
    lp_t = O.token_logprobs(hidden_target_bits, w_target_bits, token_ids)
    lp_g = O.token_logprobs(hidden_gen_bits, w_gen_bits, token_ids)
    LP, LQ = O.block_sums(lp_t, block_offsets), O.block_sums(lp_g, block_offsets)
    S = O.scores(LP, LQ, reward, beta)
    chosen, margin = O.gumbel_pick(S, uniforms, cand_offsets)
    return {"tok_logprob": lp_t, "gen_tok_logprob": lp_g, "tok_logratio": lp_t - lp_g, "blk_logprob": LP,
            "blk_logprob_gen": LQ, "score": S, "weights": O.weights(S, cand_offsets), "chosen": chosen,
            "margin": margin, "accept": O.accept_flags(reward, cand_offsets, tau)}


def gather_chosen(token_ids, block_offsets, cand_offsets, chosen, stride):
    """Step II of Algorithm 1 appends the selected block to the trace: the ids of block
    (first block of the problem + chosen) go to row p of an int32 [P, stride] array (-1 beyond the block's
    length, everything -1 when nothing was chosen), its length to chosen_len[p]."""
    P = len(cand_offsets) - 1
    out = np.full((P, stride), -1, dtype=np.int32)
    lens = np.zeros(P, dtype=np.int32)
    for p in range(P):
        if chosen[p] < 0:
            continue
        blk = int(cand_offsets[p]) + int(chosen[p])
        a, b = int(block_offsets[blk]), int(block_offsets[blk + 1])
        if b - a > stride:
            raise ValueError("chosen block longer than the output row")
        for k in range(a, b):
            out[p, k - a] = token_ids[k]
        lens[p] = b - a
    return out, lens


# --------------------------------------------------------------------------- PRM head

def prm_rewards(prm_hidden_bits, block_offsets, w_head_bits, bias):
    """r(Y_i | tr) of every drafted block from the process reward model's final hidden states: the value
    head (one weight vector and a bias) applied to the hidden state of the block's LAST token, squashed
    to (0, 1) by the logistic function.  The paper takes r as given (Section 2: "PRM r") and uses a PRM
    whose scores are thresholded between 0.5 and 0.9, i.e. lie in [0, 1] (Section 4.1, Table 6); which
    position is read and the logistic link are this build's reading.  An empty block has no last token:
    its reward is NaN.  Inputs are bf16 bit patterns; everything is evaluated in float64."""
    from oracle import specs_oracle as O
    H = O.bf16_bits_to_f64(prm_hidden_bits)
    w = O.bf16_bits_to_f64(w_head_bits)
    b = float(np.float32(bias))
    B = len(block_offsets) - 1
    out = np.full(B, np.nan)
    for i in range(B):
        a, e = int(block_offsets[i]), int(block_offsets[i + 1])
        if e <= a:
            continue
        z = b
        for k in range(H.shape[1]):
            z += H[e - 1, k] * w[k]
        out[i] = 1.0 / (1.0 + np.exp(-z))
    return out


# --------------------------------------------------------------------------- vocabulary shards

def shard_partials(hidden_bits, w_bits, token_ids, v0, v1):
    """What one holder of vocabulary rows [v0, v1) can say about every drafted row: the largest logit of its
    shard, the sum of exp(logit - that maximum) over the shard, and the drafted id's logit if the id lies in
    the shard (-inf otherwise).  float64 [rows, 3]."""
    from oracle import specs_oracle as O
    H = O.bf16_bits_to_f64(hidden_bits)
    W = O.bf16_bits_to_f64(w_bits[v0:v1])
    out = np.empty((H.shape[0], 3))
    for t in range(H.shape[0]):
        z = W @ H[t]
        m = np.max(z)
        y = int(token_ids[t])
        out[t] = (m, np.sum(np.exp(z - m)), z[y - v0] if v0 <= y < v1 else -np.inf)
    return out


def merge_partials(partials, token_ids, V):
    """log pi_target(y_t) from the shards' partials: the log-sum-exp of a union is the log-sum-exp of the
    parts' log-sum-exps; the drafted id's logit is held by exactly one shard.  partials float64 [g, rows, 3]."""
    partials = np.asarray(partials, dtype=np.float64)
    g, rows, _ = partials.shape
    out = np.empty(rows)
    for t in range(rows):
        M = np.max(partials[:, t, 0])
        total = 0.0
        for j in range(g):
            total += partials[j, t, 1] * np.exp(partials[j, t, 0] - M)
        y = int(token_ids[t])
        out[t] = np.max(partials[:, t, 2]) - (M + np.log(total)) if 0 <= y < V else np.nan
    return out
