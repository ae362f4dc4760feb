"""CPU oracle for the block-scoring step of SPECS.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
it; the product never does, and this file imports nothing from the product.

Everything is float64 numpy.  Rows of the hidden-state matrix are independent,
so the row loop is taken in chunks purely to bound memory (one chunk of logits
at a time); within a chunk the computation is the definition, with numpy's
matmul as the one library step.  There is no tiling, fusion or online
rescaling here.

What each function follows in the paper:

  token_logprobs   Section 2 ("computing logits of each token" of a drafted
                   block with the target model) and Appendix E.3 (only the
                   newly drafted tokens get log-probabilities): logits are the
                   LM-head product, log pi_target(y_t) is the log-softmax
                   entry of the drafted id.
  block_sums       Eq. (1) is a ratio of *block* probabilities; by the chain
                   rule a block's log-probability is the plain sum of its
                   tokens' log-probabilities (no length normalisation).
  scores           Eq. (1) / Algorithm 2: S_i = log(pi_target/pi_gen) + beta r_i;
                   with pi_gen = pi_target the ratio vanishes and S_i = beta r_i.
  weights          Algorithm 2's sampling law and the SMC definition in
                   Appendix B.2: P(i* = i) = exp(S_i) / sum_j exp(S_j) over the
                   candidates of one problem (the set L is all of them).
  gumbel_pick      An exact sampler of that law driven by caller-supplied
                   uniforms: argmax_i (S_i - log(-log u_i)); lowest index wins
                   exact ties.  Also returns the top-two margin.
  accept_flags     Algorithm 1, Step III: switch to the draft generator when
                   max_i r_i > tau (strict), max over all n candidates.

Parity pins: every function above is pinned by closed forms, brute force or
big-float evaluation in tests/test_oracle_pins.py; none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- decode

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly: bf16 is the top half of an fp32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    as_f32 = (b.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


# --------------------------------------------------------------------------- O1 + O2

def row_logits(h_row: np.ndarray, w: np.ndarray) -> np.ndarray:
    """z_v = sum_k h[k] * W[v, k] for every vocabulary entry v (float64 in, float64 out)."""
    return w @ h_row


def log_softmax_row(z: np.ndarray) -> np.ndarray:
    """log softmax of one row of logits, by the max-shifted definition."""
    m = np.max(z)
    lse = m + np.log(np.sum(np.exp(z - m)))
    return z - lse


def token_logprobs(hidden_bits: np.ndarray, w_bits: np.ndarray, token_ids: np.ndarray,
                   row_chunk: int = 64, w_f64: np.ndarray | None = None) -> np.ndarray:
    """log pi_target(y_t) for every drafted row t.

    hidden_bits uint16 [rows, d], w_bits uint16 [V, d] (bf16 patterns),
    token_ids int [rows].  Returns float64 [rows].  A token id outside [0, V)
    has no probability: its entry is NaN.  ``w_f64`` lets a caller that scores
    several row sets against the same weights pass the decoded matrix once.
    """
    rows = hidden_bits.shape[0]
    W = bf16_bits_to_f64(w_bits) if w_f64 is None else w_f64
    V = W.shape[0]
    out = np.empty(rows, dtype=np.float64)
    for r0 in range(0, rows, row_chunk):
        r1 = min(rows, r0 + row_chunk)
        H = bf16_bits_to_f64(hidden_bits[r0:r1])
        Z = H @ W.T                                   # [chunk, V] logits
        m = Z.max(axis=1)
        lse = m + np.log(np.exp(Z - m[:, None]).sum(axis=1))
        for t in range(r0, r1):
            y = int(token_ids[t])
            out[t] = Z[t - r0, y] - lse[t - r0] if 0 <= y < V else np.nan
    return out


# --------------------------------------------------------------------------- O3

def block_sums(per_token: np.ndarray, block_offsets: np.ndarray) -> np.ndarray:
    """LP_i = sum of per-token values over rows [off[i], off[i+1]); an empty block sums to 0."""
    x = np.asarray(per_token, dtype=np.float64)
    B = len(block_offsets) - 1
    out = np.zeros(B, dtype=np.float64)
    for i in range(B):
        a, b = int(block_offsets[i]), int(block_offsets[i + 1])
        s = 0.0
        for t in range(a, b):
            s += x[t]
        out[i] = s
    return out


# --------------------------------------------------------------------------- O4

def scores(lp_target_blk, lp_gen_blk, reward, beta: float) -> np.ndarray:
    """S_i = (LP_i - LQ_i) + beta * r_i.  ``lp_gen_blk=None`` means pi_gen = pi_target: S_i = beta * r_i."""
    r = np.asarray(reward, dtype=np.float64)
    beta = float(np.float32(beta))          # beta is an fp32 argument of the interface
    if lp_gen_blk is None:
        return beta * r
    lp = np.asarray(lp_target_blk, dtype=np.float64)
    lq = np.asarray(lp_gen_blk, dtype=np.float64)
    return (lp - lq) + beta * r


# --------------------------------------------------------------------------- O5

def weights(S: np.ndarray, cand_offsets: np.ndarray) -> np.ndarray:
    """w_i = exp(S_i) / sum_{j in problem} exp(S_j), per problem."""
    S = np.asarray(S, dtype=np.float64)
    w = np.zeros_like(S)
    for p in range(len(cand_offsets) - 1):
        a, b = int(cand_offsets[p]), int(cand_offsets[p + 1])
        if b <= a:
            continue
        s = S[a:b]
        m = np.max(s)
        lse = m + np.log(np.sum(np.exp(s - m)))
        w[a:b] = np.exp(s - lse)
    return w


# --------------------------------------------------------------------------- O6

def gumbel_pick(S: np.ndarray, uniforms: np.ndarray, cand_offsets: np.ndarray):
    """Per problem: i* = argmax_i (S_i + g_i), g_i = -log(-log u_i); first index on exact ties.

    Returns (chosen int32 [P] with the index local to the problem, -1 for an empty
    problem; margin float64 [P] = best minus second-best perturbed score, +inf when
    there is a single candidate).
    """
    S = np.asarray(S, dtype=np.float64)
    u = np.asarray(uniforms, dtype=np.float64)
    if np.any((u <= 0.0) | (u >= 1.0)):
        raise ValueError("uniforms must lie strictly inside (0, 1)")
    g = -np.log(-np.log(u))
    P = len(cand_offsets) - 1
    chosen = np.full(P, -1, dtype=np.int32)
    margin = np.full(P, np.inf, dtype=np.float64)
    for p in range(P):
        a, b = int(cand_offsets[p]), int(cand_offsets[p + 1])
        if b <= a:
            continue
        pert = S[a:b] + g[a:b]
        best = int(np.argmax(pert))                   # numpy returns the first maximum
        chosen[p] = best
        if b - a > 1:
            rest = np.delete(pert, best)
            margin[p] = pert[best] - np.max(rest)
    return chosen, margin


# --------------------------------------------------------------------------- O7

def accept_flags(reward: np.ndarray, cand_offsets: np.ndarray, tau: float) -> np.ndarray:
    """flag_p = 1 iff max over the problem's candidates of r_i exceeds tau (strictly); 0 for an empty problem."""
    r = np.asarray(reward, dtype=np.float64)
    tau = float(np.float32(tau))            # tau is an fp32 argument of the interface
    P = len(cand_offsets) - 1
    out = np.zeros(P, dtype=np.uint8)
    for p in range(P):
        a, b = int(cand_offsets[p]), int(cand_offsets[p + 1])
        if b > a and np.max(r[a:b]) > tau:
            out[p] = 1
    return out


# --------------------------------------------------------------------------- whole step

def beam_step(hidden_bits, w_bits, token_ids, block_offsets, cand_offsets,
              draft_tok_logprob, reward, beta, uniforms, tau, row_chunk: int = 64):
    """The whole scoring step, in the order the paper takes it.

    ``draft_tok_logprob=None`` means the blocks were generated by the target
    itself (pi_gen = pi_target).  Returns a dict of every intermediate.
    """
    tok_lp = token_logprobs(hidden_bits, w_bits, token_ids, row_chunk=row_chunk)
    LP = block_sums(tok_lp, block_offsets)
    LQ = None if draft_tok_logprob is None else block_sums(draft_tok_logprob, block_offsets)
    S = scores(LP, LQ, reward, beta)
    w = weights(S, cand_offsets)
    chosen, margin = gumbel_pick(S, uniforms, cand_offsets)
    flags = accept_flags(reward, cand_offsets, tau)
    return {"tok_logprob": tok_lp, "blk_logprob": LP, "blk_logprob_gen": LQ, "score": S,
            "weights": w, "chosen": chosen, "margin": margin, "accept": flags}
