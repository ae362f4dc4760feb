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


# The end-to-end pick is compared where the oracle's margin exceeds MARGIN plus a slack for the rounding the
# two compared block log-probs carry on the GPU side.  That slack is bounded: a block sum may be off by an
# eighth of the per-token tolerance per token (the error of a token is mostly a bias of one sign, so it adds
# up along a block), and never less than MAX_PICK_SLACK is allowed.
MAX_PICK_SLACK = 1e-2


def pick_slack(got_blk, want_blk, max_block_len=0):
    """Slack on the pick margin of one problem: twice the largest block log-prob error observed in it."""
    slack = 2.0 * float(np.abs(np.asarray(got_blk) - np.asarray(want_blk)).max(initial=0.0))
    bound = max(MAX_PICK_SLACK, 2.0 * max_block_len * TOK_ATOL / 8.0)
    assert slack <= bound, f"block log-prob error widens the pick exemption to {slack:.3e} (bound {bound:.3e})"
    return slack


def assert_step_matches(got, want, cand_offsets, block_offsets, lp_slack_per_token=0.0):
    """Compare a full step's outputs with the oracle's.

    The pick is compared where the oracle's margin exceeds MARGIN plus the worst-case shift the
    block log-prob error can cause in a perturbed-score difference (two blocks, each off by the
    largest block error observed in the problem); that slack is bounded by MAX_PICK_SLACK, and the
    number of problems it exempted (beyond those under the plain MARGIN rule) is returned.
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
    exact, by_slack, max_slack = 0, 0, 0.0
    for p in range(P):
        a, b = cand_offsets[p], cand_offsets[p + 1]
        if b <= a:
            assert got["chosen"][p] == -1
            continue
        slack = pick_slack(got["blk_logprob_f64"][a:b], want["blk_logprob"][a:b], int(lens[a:b].max()))
        max_slack = max(max_slack, slack)
        if want["margin"][p] > MARGIN + slack:
            assert got["chosen"][p] == want["chosen"][p], (p, want["margin"][p], slack)
            exact += 1
        else:
            assert 0 <= got["chosen"][p] < b - a
            if want["margin"][p] > MARGIN:
                by_slack += 1
    assert np.array_equal(got["accept"], want["accept"])
    return {"tok_max_err": float(tok_err.max()), "picks_checked_exactly": exact, "problems": P,
            "picks_exempted_by_slack": by_slack, "max_pick_slack": max_slack}
