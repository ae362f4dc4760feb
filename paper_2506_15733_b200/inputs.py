"""Seeded synthetic inputs for one SPECS beam step (scoring of drafted blocks).

This module only *draws numbers and lays them out*; it holds none of the
method's arithmetic (no logits, no log-softmax, no scores).  The same arrays
are handed, bit for bit, to the CPU oracle and to the CUDA library, so neither
side ever regenerates inputs on its own.

The shapes follow the model pair used in the paper's experiments (Section 4.1:
a 1.5B draft with a 7B target, vocabulary of about 152k entries, beam widths
n in {4, 8, 16}); the value distributions are the ones the benchmark
configurations prescribe.  They stand in for real hidden states, LM-head
weights, drafted tokens, draft log-probabilities and process-reward scores,
none of which are available offline.

Layout conventions (all numpy, host memory):
  * bf16 tensors are carried as ``uint16`` arrays holding the raw bit pattern
    (numpy has no bf16 dtype); rounding from fp32 is round-to-nearest-even.
  * ``hidden``  uint16 ``[rows, d]``  row-major, one row per drafted token.
  * ``w_vocab`` uint16 ``[V, d]``     row-major, one row per vocabulary entry.
  * ``token_ids`` int32 ``[rows]``.
  * ``block_offsets`` int64 ``[B+1]`` CSR offsets of the candidate blocks over rows.
  * ``cand_offsets`` int32 ``[P+1]`` CSR offsets of the problems over blocks.
  * ``draft_tok_logprob`` float32 ``[rows]``, ``reward`` float32 ``[B]``,
    ``uniforms`` float32 ``[B]`` strictly inside (0, 1).
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

# Sub-stream ids: one Philox key per tensor, so that changing how one tensor is
# drawn never shifts another.
_STREAM = {
    "lengths": 1, "hidden": 2, "w_vocab": 3, "token_ids": 4, "draft": 5,
    "reward": 6, "uniforms": 7, "outlier_rows": 8, "zipf_perm": 9,
}


def _rng(seed: int, stream: str, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), _STREAM[stream] + 100 * int(salt)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the uint16 bit pattern."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen a bf16 bit pattern to fp32 (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class StepConfig:
    """Shape and distribution recipe of one beam step."""
    name: str
    seed: int
    problems: int                 # P
    beams: int                    # n candidate blocks per problem
    block_len: Tuple[int, int]    # inclusive range of drafted tokens per block (lo == hi: fixed)
    d: int
    vocab: int
    w_sigma: float
    hidden_scale: float = 1.0
    outlier_frac: float = 0.0     # fraction of rows multiplied by outlier_mult
    outlier_mult: float = 1.0
    token_dist: str = "uniform"   # "uniform" | "zipf" | "zipf_perm"
    zipf_a: float = 1.1
    draft_lo: float = -8.0        # draft per-token log-probs ~ U[draft_lo, 0]
    reward_dist: Tuple[str, float, float] = ("uniform", 0.0, 1.0)   # or ("beta", a, b)
    betas: Tuple[float, ...] = (1.0,)
    taus: Tuple[float, ...] = (0.7,)
    weights_salt: int = 0         # separates the hidden / w_vocab streams of configs sharing a seed

    @property
    def max_rows(self) -> int:
        return self.problems * self.beams * self.block_len[1]


# The five benchmark configurations.  Seeds are 1000 + index.
CONFIGS: Dict[str, StepConfig] = {
    "tiny": StepConfig("tiny", 1000, 1, 4, (16, 16), 256, 1024, 0.05,
                       draft_lo=-6.0, betas=(1.0,)),
    "step7b": StepConfig("step7b", 1001, 1, 16, (64, 64), 3584, 151936, 0.02,
                         reward_dist=("beta", 2.0, 2.0), betas=(0.5, 1.0, 4.0)),
    "batched": StepConfig("batched", 1002, 32, 8, (32, 128), 3584, 151936, 0.02,
                          betas=(2.0,), taus=(0.5, 0.6, 0.7, 0.8, 0.9)),
    "dual_draft": StepConfig("dual_draft", 1003, 8, 32, (256, 256), 1536, 151936, 0.02,
                             token_dist="zipf", betas=(1.0,)),
    "dual_target": StepConfig("dual_target", 1003, 8, 32, (256, 256), 3584, 151936, 0.02,
                              token_dist="zipf", betas=(1.0,), weights_salt=1),
    "stress": StepConfig("stress", 1004, 4, 64, (64, 512), 5120, 152064, 0.02,
                         hidden_scale=5.0, outlier_frac=0.01, outlier_mult=20.0,
                         reward_dist=("beta", 0.5, 0.5), betas=(0.25, 8.0)),
}


def scaled(cfg: StepConfig, **kw) -> StepConfig:
    """A copy of ``cfg`` with some fields replaced (used to shrink a config for CPU-sized tests)."""
    return replace(cfg, **kw)


@dataclass
class StepInputs:
    cfg: StepConfig
    hidden: np.ndarray            # uint16 [rows, d]
    w_vocab: np.ndarray           # uint16 [V, d]
    token_ids: np.ndarray         # int32 [rows]
    block_offsets: np.ndarray     # int64 [B+1]
    cand_offsets: np.ndarray      # int32 [P+1]
    draft_tok_logprob: np.ndarray  # float32 [rows]
    reward: np.ndarray            # float32 [B]
    uniforms: np.ndarray          # float32 [B]
    outlier_rows: np.ndarray      # int64 indices of the rows that were scaled up
    meta: dict = field(default_factory=dict)

    @property
    def rows(self) -> int:
        return int(self.block_offsets[-1])

    @property
    def blocks(self) -> int:
        return int(self.block_offsets.shape[0] - 1)

    def digests(self) -> Dict[str, str]:
        """SHA-256 of every buffer, for result records."""
        out = {}
        for k in ("hidden", "w_vocab", "token_ids", "block_offsets", "cand_offsets",
                  "draft_tok_logprob", "reward", "uniforms"):
            out[k] = hashlib.sha256(np.ascontiguousarray(getattr(self, k)).tobytes()).hexdigest()
        return out


def draw_block_layout(cfg: StepConfig) -> Tuple[np.ndarray, np.ndarray]:
    """Block lengths -> CSR offsets over rows, plus CSR offsets of problems over blocks."""
    B = cfg.problems * cfg.beams
    lo, hi = cfg.block_len
    if lo == hi:
        lens = np.full(B, lo, dtype=np.int64)
    else:
        lens = _rng(cfg.seed, "lengths").integers(lo, hi + 1, size=B).astype(np.int64)
    block_offsets = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(lens, out=block_offsets[1:])
    cand_offsets = (np.arange(cfg.problems + 1, dtype=np.int64) * cfg.beams).astype(np.int32)
    return block_offsets, cand_offsets


def draw_uniforms(seed: int, count: int) -> np.ndarray:
    """Uniforms (k + 1/2) * 2^-23 with k a 23-bit Philox integer.

    2k + 1 < 2^24, so every value is exact in fp32 and lies strictly inside
    (0, 1); a 24-bit k would round (2^25 - 1) * 2^-25 up to exactly 1.0.
    """
    k = _rng(seed, "uniforms").integers(0, 1 << 23, size=count, dtype=np.int64)
    u = ((k.astype(np.float64) + 0.5) * 2.0 ** -23).astype(np.float32)
    assert np.all((u > 0) & (u < 1))
    return u


def _normal_bf16(gen: np.random.Generator, shape: Tuple[int, int], sigma: float,
                 row_scale: Optional[np.ndarray] = None, chunk_rows: int = 8192) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        x = gen.standard_normal((r1 - r0, shape[1]), dtype=np.float32)
        x *= np.float32(sigma)
        if row_scale is not None:
            x *= row_scale[r0:r1, None].astype(np.float32)
        out[r0:r1] = f32_to_bf16_bits(x)
    return out


def draw_token_ids(cfg: StepConfig, rows: int) -> np.ndarray:
    gen = _rng(cfg.seed, "token_ids")
    V = cfg.vocab
    if cfg.token_dist == "uniform":
        return gen.integers(0, V, size=rows, dtype=np.int64).astype(np.int32)
    # Zipf(a) truncated to ranks 1..V, by inverse CDF on fp64 cumulative weights.
    ranks = np.arange(1, V + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-cfg.zipf_a))
    cdf /= cdf[-1]
    u = gen.random(rows)
    rank0 = np.minimum(np.searchsorted(cdf, u, side="right"), V - 1)   # 0-based rank
    if cfg.token_dist == "zipf":
        return rank0.astype(np.int32)          # hot ids all sit in the first vocab tile
    if cfg.token_dist == "zipf_perm":
        perm = _rng(cfg.seed, "zipf_perm").permutation(V)
        return perm[rank0].astype(np.int32)
    raise ValueError(f"unknown token_dist {cfg.token_dist!r}")


def draw_rewards(cfg: StepConfig, B: int) -> np.ndarray:
    gen = _rng(cfg.seed, "reward")
    kind, a, b = cfg.reward_dist
    if kind == "uniform":
        r = gen.uniform(a, b, size=B)
    elif kind == "beta":
        r = gen.beta(a, b, size=B)
    else:
        raise ValueError(f"unknown reward_dist {kind!r}")
    return r.astype(np.float32)


def make_step_inputs(cfg: StepConfig, with_weights: bool = True) -> StepInputs:
    """Draw every tensor of one beam step for ``cfg``.

    ``with_weights=False`` skips ``hidden`` and ``w_vocab`` (zero-size arrays are
    returned) for callers that only need the selection-stage inputs.
    """
    block_offsets, cand_offsets = draw_block_layout(cfg)
    rows = int(block_offsets[-1])
    B = cfg.problems * cfg.beams

    n_out = int(round(cfg.outlier_frac * rows))
    if n_out > 0:
        outlier_rows = np.sort(_rng(cfg.seed, "outlier_rows").choice(rows, size=n_out, replace=False))
    else:
        outlier_rows = np.zeros(0, dtype=np.int64)

    if with_weights:
        row_scale = np.full(rows, cfg.hidden_scale, dtype=np.float32)
        row_scale[outlier_rows] *= np.float32(cfg.outlier_mult)
        hidden = _normal_bf16(_rng(cfg.seed, "hidden", cfg.weights_salt), (rows, cfg.d), 1.0, row_scale)
        w_vocab = _normal_bf16(_rng(cfg.seed, "w_vocab", cfg.weights_salt), (cfg.vocab, cfg.d), cfg.w_sigma)
    else:
        hidden = np.zeros((0, cfg.d), dtype=np.uint16)
        w_vocab = np.zeros((0, cfg.d), dtype=np.uint16)

    token_ids = draw_token_ids(cfg, rows)
    draft = _rng(cfg.seed, "draft").uniform(cfg.draft_lo, 0.0, size=rows).astype(np.float32)
    reward = draw_rewards(cfg, B)
    uniforms = draw_uniforms(cfg.seed, B)
    return StepInputs(cfg, hidden, w_vocab, token_ids, block_offsets, cand_offsets,
                      draft, reward, uniforms, outlier_rows,
                      meta={"rows": rows, "blocks": B, "problems": cfg.problems})
