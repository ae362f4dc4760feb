"""Helpers for the GPU parity tests: run the CUDA path on a StepInputs through the C ABI."""
import numpy as np
import torch

from paper_2506_15733_b200 import binding


class DeviceStep:
    """Device copies of one step's inputs plus output buffers."""

    def __init__(self, ctx, x, rows_slice=None):
        dev = f"cuda:{ctx.device}"
        self.ctx, self.x = ctx, x
        hidden = x.hidden if rows_slice is None else x.hidden[rows_slice]
        self.hidden = binding.bf16_bits_to_device(hidden, dev)
        self.w_vocab = binding.bf16_bits_to_device(x.w_vocab, dev)
        self.token_ids = torch.from_numpy(x.token_ids).to(dev)
        self.block_offsets = torch.from_numpy(x.block_offsets).to(dev)
        self.cand_offsets = torch.from_numpy(x.cand_offsets).to(dev)
        self.draft = torch.from_numpy(x.draft_tok_logprob).to(dev)
        self.reward = torch.from_numpy(x.reward).to(dev)
        self.uniforms = torch.from_numpy(x.uniforms).to(dev)
        rows, B, P = x.rows, x.blocks, len(x.cand_offsets) - 1
        self.tok_lp = torch.full((rows,), float("nan"), dtype=torch.float32, device=dev)
        self.blk_lp = torch.full((B,), float("nan"), dtype=torch.float32, device=dev)
        self.blk_lp64 = torch.full((B,), float("nan"), dtype=torch.float64, device=dev)
        self.gen_blk64 = torch.full((B,), float("nan"), dtype=torch.float64, device=dev)
        self.weights = torch.full((B,), float("nan"), dtype=torch.float32, device=dev)
        self.chosen = torch.full((P,), -7, dtype=torch.int32, device=dev)
        self.accept = torch.full((P,), 9, dtype=torch.uint8, device=dev)
        ws_bytes = ctx.score_workspace_bytes(rows, x.hidden.shape[1], x.w_vocab.shape[0])
        self.workspace = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)

    def score(self):
        self.ctx.specs_score_blocks(self.hidden, self.w_vocab, self.token_ids, self.block_offsets, self.tok_lp,
                                    self.blk_lp, self.blk_lp64, self.workspace)

    def select(self, beta, tau, with_draft=True):
        gen = None
        if with_draft:
            self.ctx.specs_block_sums(self.draft, self.block_offsets, None, self.gen_blk64)
            gen = self.gen_blk64
        self.ctx.specs_subsample(self.blk_lp64, gen, self.reward, self.cand_offsets, beta, self.uniforms,
                                 self.chosen, self.weights, tau, self.accept)

    def step(self, beta, tau, with_draft=True):
        self.score()
        self.select(beta, tau, with_draft)
        torch.cuda.synchronize()
        return self.results()

    def results(self):
        return {"tok_logprob": self.tok_lp.cpu().numpy(), "blk_logprob": self.blk_lp.cpu().numpy(),
                "blk_logprob_f64": self.blk_lp64.cpu().numpy(), "blk_logprob_gen": self.gen_blk64.cpu().numpy(),
                "weights": self.weights.cpu().numpy(), "chosen": self.chosen.cpu().numpy(),
                "accept": self.accept.cpu().numpy()}


# Tolerances of the parity bar: absolute per token log-prob, relative per block log-prob,
# exact picks when the oracle's top-two perturbed-score margin exceeds MARGIN.
TOK_ATOL = 2e-3
BLK_RTOL = 1e-2
MARGIN = 1e-3


def assert_step_matches(got, want, cand_offsets, block_offsets, lp_slack_per_token=0.0):
    """Compare a full step's outputs with the oracle's.

    The pick is compared where the oracle's margin exceeds MARGIN plus the worst-case shift the
    block log-prob error can cause in a perturbed-score difference (two blocks, every token off by
    the per-token tolerance actually observed).
    """
    tok_err = np.abs(got["tok_logprob"] - want["tok_logprob"])
    assert np.all(np.isfinite(got["tok_logprob"])), "non-finite token log-prob"
    assert tok_err.max() <= TOK_ATOL, f"token log-prob off by {tok_err.max():.3e}"
    for key in ("blk_logprob", "blk_logprob_f64"):
        rel = np.abs(got[key] - want["blk_logprob"]) / np.maximum(np.abs(want["blk_logprob"]), 1e-30)
        nz = want["blk_logprob"] != 0
        assert np.all(got[key][~nz] == 0)
        assert rel[nz].max(initial=0.0) <= BLK_RTOL, f"{key} relative error {rel[nz].max():.3e}"
    lens = np.diff(block_offsets)
    P = len(cand_offsets) - 1
    exact = 0
    for p in range(P):
        a, b = cand_offsets[p], cand_offsets[p + 1]
        if b <= a:
            assert got["chosen"][p] == -1
            continue
        blk_err = np.abs(got["blk_logprob_f64"][a:b] - want["blk_logprob"][a:b])
        slack = 2.0 * blk_err.max()
        if want["margin"][p] > MARGIN + slack:
            assert got["chosen"][p] == want["chosen"][p], (p, want["margin"][p], slack)
            exact += 1
        else:
            assert 0 <= got["chosen"][p] < b - a
    assert np.array_equal(got["accept"], want["accept"])
    return {"tok_max_err": float(tok_err.max()), "picks_checked_exactly": exact, "problems": P}
