"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The CUDA path scores every row; the CPU oracle scores a seeded sample of whole blocks (plus
single rows, e.g. the outlier rows of the stress config) -- rows are independent, so a sample is
exact for parity.  Selection is checked two ways and labelled: end to end on problems whose blocks
were all scored by the oracle, and "selection logic" on all problems by handing the GPU's block
log-probabilities to the oracle's scoring / sampling / switch functions.
"""
import numpy as np
import pytest
import torch

from oracle import specs_oracle as O
from paper_2506_15733_b200 import binding
from paper_2506_15733_b200 import inputs as I
from tests.gpu_util import BLK_RTOL, MARGIN, TOK_ATOL, DeviceStep, pick_slack

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def rows_of_blocks(x, blocks):
    return np.concatenate([np.arange(x.block_offsets[b], x.block_offsets[b + 1]) for b in blocks]).astype(np.int64)


def check_sampled_rows(x, got_tok, rows_idx, w_f64):
    want = O.token_logprobs(x.hidden[rows_idx], x.w_vocab, x.token_ids[rows_idx], w_f64=w_f64)
    err = np.abs(got_tok[rows_idx] - want)
    assert np.all(np.isfinite(got_tok)), "non-finite token log-prob somewhere in the full output"
    assert err.max() <= TOK_ATOL, f"token log-prob off by {err.max():.3e} (row {rows_idx[int(err.argmax())]})"
    return want, float(err.max())


def check_block_sums(x, got, blocks, want_tok_by_row):
    for b in blocks:
        a, e = int(x.block_offsets[b]), int(x.block_offsets[b + 1])
        want = O.block_sums(np.array([want_tok_by_row[t] for t in range(a, e)]), np.array([0, e - a]))[0]
        for key in ("blk_logprob", "blk_logprob_f64"):
            assert abs(got[key][b] - want) <= BLK_RTOL * abs(want), (key, b, got[key][b], want)
    # every block sum on the GPU equals the plain sum of the GPU's own token log-probs (all blocks)
    all_sums = O.block_sums(got["tok_logprob"], x.block_offsets)
    assert np.allclose(got["blk_logprob_f64"], all_sums, rtol=1e-12, atol=1e-9)


def check_selection_logic(x, got, beta, tau, gen_blk):
    """Oracle O4-O7 on the GPU's own block log-probs: picks exact above the margin, weights, flags."""
    S = O.scores(got["blk_logprob_f64"], gen_blk, x.reward, beta)
    want_c, margin = O.gumbel_pick(S, x.uniforms, x.cand_offsets)
    sure = margin > MARGIN
    assert np.array_equal(got["chosen"][sure], want_c[sure])
    assert np.abs(got["weights"] - O.weights(S, x.cand_offsets)).max() < 1e-6
    assert np.array_equal(got["accept"], O.accept_flags(x.reward, x.cand_offsets, tau))
    return int(sure.sum())


@pytest.mark.parametrize("engine", [binding.ENGINE_TCGEN05, binding.ENGINE_TCGEN05_1CTA])
def test_step7b_all_rows_all_betas(ctx, engine):
    # default engine (CTA pairs at this size) and the single-CTA tile shape
    cfg = I.CONFIGS["step7b"]
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    ctx.set_engine(engine)
    try:
        got = s.step(cfg.betas[0], 0.7)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    # the fused two-launch step, which is what bench.py times, gives the same bits as the separate calls
    f = DeviceStep(ctx, x)
    ctx.set_engine(engine)
    try:
        ctx.specs_beam_step(f.hidden, f.w_vocab, f.token_ids, f.block_offsets, f.cand_offsets, f.draft, f.reward,
                            f.uniforms, cfg.betas[0], 0.7, f.tok_lp, f.blk_lp64, f.gen_blk64, f.weights, f.chosen,
                            f.accept, f.workspace)
        torch.cuda.synchronize()
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    fused = f.results()
    for key in ("tok_logprob", "blk_logprob_f64", "blk_logprob_gen", "weights", "chosen", "accept"):
        assert np.array_equal(fused[key], got[key]), key
    del f
    w64 = O.bf16_bits_to_f64(x.w_vocab)
    all_rows = np.arange(x.rows)
    want_tok, err = check_sampled_rows(x, got["tok_logprob"], all_rows, w64)
    check_block_sums(x, got, range(x.blocks), want_tok)
    LP = O.block_sums(want_tok, x.block_offsets)
    LQ = O.block_sums(x.draft_tok_logprob, x.block_offsets)
    assert np.allclose(got["blk_logprob_gen"], LQ, rtol=1e-12)
    for beta in cfg.betas:
        s.select(beta, 0.7)
        torch.cuda.synchronize()
        g = s.results()
        # end to end: oracle block log-probs vs GPU block log-probs
        S = O.scores(LP, LQ, x.reward, beta)
        want_c, margin = O.gumbel_pick(S, x.uniforms, x.cand_offsets)
        slack = pick_slack(g["blk_logprob_f64"], LP, 64)
        if margin[0] > MARGIN + slack:
            assert g["chosen"][0] == want_c[0]
        assert np.abs(g["weights"] - O.weights(S, x.cand_offsets)).max() < 5e-3 + 2 * slack
        check_selection_logic(x, g, beta, 0.7, LQ)


def test_batched_ragged_step(ctx):
    cfg = I.CONFIGS["batched"]
    x = I.make_step_inputs(cfg)
    assert x.rows == 20893
    s = DeviceStep(ctx, x)
    got = s.step(2.0, cfg.taus[0])
    w64 = O.bf16_bits_to_f64(x.w_vocab)
    rng = np.random.Generator(np.random.Philox(key=[7002, 1]))
    blocks = list(range(8)) + sorted(rng.choice(np.arange(8, 256), size=4, replace=False).tolist())   # problem 0 whole
    rows_idx = rows_of_blocks(x, blocks)
    want_tok, err = check_sampled_rows(x, got["tok_logprob"], rows_idx, w64)
    by_row = dict(zip(rows_idx.tolist(), want_tok.tolist()))
    check_block_sums(x, got, blocks, by_row)
    LQ = O.block_sums(x.draft_tok_logprob, x.block_offsets)
    # end to end on problem 0
    LP0 = np.array([sum(by_row[t] for t in range(x.block_offsets[b], x.block_offsets[b + 1])) for b in range(8)])
    S0 = O.scores(LP0, LQ[:8], x.reward[:8], 2.0)
    c0, m0 = O.gumbel_pick(S0, x.uniforms[:8], np.array([0, 8]))
    slack = pick_slack(got["blk_logprob_f64"][:8], LP0, 128)
    if m0[0] > MARGIN + slack:
        assert got["chosen"][0] == c0[0]
    # selection logic on all 32 problems, and the threshold sweep
    for tau in cfg.taus:
        s.select(2.0, tau)
        torch.cuda.synchronize()
        assert check_selection_logic(x, s.results(), 2.0, tau, LQ) >= 24


def check_problem_end_to_end(x, got_chosen, got_blk, p, LP, LQ, beta):
    """Oracle scores, pick and margin of one problem whose blocks the oracle scored in full."""
    a, b = int(x.cand_offsets[p]), int(x.cand_offsets[p + 1])
    S = O.scores(LP, LQ, x.reward[a:b], beta)
    want_c, margin = O.gumbel_pick(S, x.uniforms[a:b], np.array([0, b - a]))
    slack = pick_slack(got_blk[a:b], LP, int(np.diff(x.block_offsets)[a:b].max()))
    if margin[0] > MARGIN + slack:
        assert got_chosen[p] == want_c[0], (p, margin[0], slack)
        return 1
    return 0


@pytest.mark.parametrize("token_dist", ["zipf", "zipf_perm"])
def test_dual_scoring_draft_then_target(ctx, token_dist):
    # the same 65536 drafted tokens scored with a 1.5B-draft-shaped head and a 7B-target-shaped head;
    # the draft pass supplies the generator's block log-probs (Eq. 1's denominator).  For the plain Zipf
    # ids the oracle scores one whole problem (32 blocks of 256 tokens) per pass, which also allows the
    # end-to-end pick of that problem; for the permuted ids three blocks and 128 single rows.
    rng = np.random.Generator(np.random.Philox(key=[7003, 1]))
    if token_dist == "zipf":
        problem = int(rng.integers(8))
        blocks = list(range(32 * problem, 32 * problem + 32))
    else:
        problem = None
        blocks = sorted(rng.choice(256, size=3, replace=False).tolist())
    blk, oracle_blk = {}, {}
    for name in ("dual_draft", "dual_target"):
        cfg = I.scaled(I.CONFIGS[name], token_dist=token_dist)
        x = I.make_step_inputs(cfg)
        s = DeviceStep(ctx, x)
        s.score()
        torch.cuda.synchronize()
        got = s.results()
        w64 = O.bf16_bits_to_f64(x.w_vocab)
        rows_idx = np.unique(np.concatenate([rows_of_blocks(x, blocks), rng.choice(x.rows, 128, replace=False)]))
        want_tok, err = check_sampled_rows(x, got["tok_logprob"], rows_idx, w64)
        by_row = dict(zip(rows_idx.tolist(), want_tok.tolist()))
        check_block_sums(x, got, blocks, by_row)
        oracle_blk[name] = np.array([O.block_sums(np.array([by_row[t] for t in range(x.block_offsets[b],
                                                                                      x.block_offsets[b + 1])]),
                                                  np.array([0, x.block_offsets[b + 1] - x.block_offsets[b]]))[0]
                                     for b in blocks])
        blk[name] = s.blk_lp64.clone()
        keep = s
        del w64
    # selection with LP from the target pass and LQ from the draft pass, on the last pass's buffers
    keep.ctx.specs_subsample(blk["dual_target"], blk["dual_draft"], keep.reward, keep.cand_offsets, 1.0,
                             keep.uniforms, keep.chosen, keep.weights, 0.7, keep.accept)
    torch.cuda.synchronize()
    g = keep.results()
    g["blk_logprob_f64"] = blk["dual_target"].cpu().numpy()
    assert check_selection_logic(x, g, 1.0, 0.7, blk["dual_draft"].cpu().numpy()) >= 6
    if problem is not None:
        # end to end on the whole problem: both block log-probs from the oracle; the slack covers the
        # rounding of the GPU's target AND draft block sums
        a = 32 * problem
        gpu_ratio = g["blk_logprob_f64"] - blk["dual_draft"].cpu().numpy()
        want_ratio = oracle_blk["dual_target"] - oracle_blk["dual_draft"]
        S = O.scores(oracle_blk["dual_target"], oracle_blk["dual_draft"], x.reward[a:a + 32], 1.0)
        want_c, margin = O.gumbel_pick(S, x.uniforms[a:a + 32], np.array([0, 32]))
        slack = pick_slack(gpu_ratio[a:a + 32], want_ratio, 2 * 256)     # two block sums per candidate
        if margin[0] > MARGIN + slack:
            assert g["chosen"][problem] == want_c[0]


def test_dual_head_step_at_full_size(ctx):
    # both heads in one call (generator pass, target pass, finish kernel) on the 65536 drafted tokens
    from oracle import specs_variants as OV
    xg = I.make_step_inputs(I.CONFIGS["dual_draft"])
    xt = I.make_step_inputs(I.CONFIGS["dual_target"])
    assert np.array_equal(xg.token_ids, xt.token_ids) and np.array_equal(xg.block_offsets, xt.block_offsets)
    dev = "cuda:0"
    s = DeviceStep(ctx, xt)
    h_g, w_g = binding.bf16_bits_to_device(xg.hidden, dev), binding.bf16_bits_to_device(xg.w_vocab, dev)
    gen_tok = torch.full((xt.rows,), float("nan"), dtype=torch.float32, device=dev)
    ids_out = torch.full((8, 256), -9, dtype=torch.int32, device=dev)
    len_out = torch.full((8,), -9, dtype=torch.int32, device=dev)
    ws = torch.empty(ctx.beam_step_dual_workspace_bytes(xt.rows, 3584, 1536, 151936), dtype=torch.uint8, device=dev)
    ctx.specs_beam_step_dual(s.hidden, s.w_vocab, h_g, w_g, s.token_ids, s.block_offsets, s.cand_offsets, s.reward,
                             s.uniforms, 1.0, 0.7, s.tok_lp, gen_tok, s.blk_lp64, s.gen_blk64, s.weights, s.chosen,
                             s.accept, ws, ids_out, len_out)
    torch.cuda.synchronize()
    got = s.results()
    g_tok = gen_tok.cpu().numpy()
    rng = np.random.Generator(np.random.Philox(key=[7005, 1]))
    rows_idx = np.unique(np.concatenate([rows_of_blocks(xt, [5]), rng.choice(xt.rows, 96, replace=False)]))
    check_sampled_rows(xt, got["tok_logprob"], rows_idx, O.bf16_bits_to_f64(xt.w_vocab))
    check_sampled_rows(xg, g_tok, rows_idx, O.bf16_bits_to_f64(xg.w_vocab))
    # block sums of both heads are the plain sums of the GPU's own token log-probs; selection logic on all problems
    assert np.allclose(got["blk_logprob_f64"], O.block_sums(got["tok_logprob"], xt.block_offsets), rtol=1e-12)
    assert np.allclose(got["blk_logprob_gen"], O.block_sums(g_tok, xt.block_offsets), rtol=1e-12)
    assert check_selection_logic(xt, got, 1.0, 0.7, got["blk_logprob_gen"]) >= 6
    want_ids, want_len = OV.gather_chosen(xt.token_ids, xt.block_offsets, xt.cand_offsets, got["chosen"], 256)
    assert np.array_equal(ids_out.cpu().numpy(), want_ids) and np.array_equal(len_out.cpu().numpy(), want_len)


@pytest.mark.parametrize("d", [2048, 4096])
def test_llama_shaped_heads(ctx, d):
    # the paper's second model pair (Llama-3.2-1B / Llama-3.1-8B, Section 4.1): d = 2048 / 4096, V = 128256
    cfg = I.StepConfig(f"llama_{d}", 1100 + d, 2, 8, (48, 96), d, 128256, 0.02, reward_dist=("beta", 2.0, 2.0),
                       betas=(1.0,))
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    got = s.step(1.0, 0.7)
    rng = np.random.Generator(np.random.Philox(key=[7006, d]))
    blocks = sorted(rng.choice(x.blocks, size=2, replace=False).tolist())
    rows_idx = np.unique(np.concatenate([rows_of_blocks(x, blocks), rng.choice(x.rows, 64, replace=False)]))
    want_tok, err = check_sampled_rows(x, got["tok_logprob"], rows_idx, O.bf16_bits_to_f64(x.w_vocab))
    check_block_sums(x, got, blocks, dict(zip(rows_idx.tolist(), want_tok.tolist())))
    check_selection_logic(x, got, 1.0, 0.7, O.block_sums(x.draft_tok_logprob, x.block_offsets))


def test_stress_heavy_tailed_logits(ctx):
    cfg = I.CONFIGS["stress"]
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    got = s.step(cfg.betas[0], 0.7)
    # the outlier rows went through the second scoring pass (reported, not an error)
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    w64 = O.bf16_bits_to_f64(x.w_vocab)
    rng = np.random.Generator(np.random.Philox(key=[7004, 1]))
    # one whole problem chosen by seed (64 blocks), the eight blocks of the other problems that hold the
    # most outlier rows, 160 more outlier rows and 64 more ordinary rows
    problem = int(rng.integers(cfg.problems))
    a, b = int(x.cand_offsets[problem]), int(x.cand_offsets[problem + 1])
    assert b - a == 64
    blk_of_row = np.searchsorted(x.block_offsets, x.outlier_rows, side="right") - 1
    per_block = np.bincount(blk_of_row, minlength=x.blocks)
    per_block[a:b] = -1
    heavy = np.argsort(-per_block, kind="stable")[:8].tolist()
    assert all(per_block[h] >= 1 for h in heavy)
    blocks = list(range(a, b)) + sorted(heavy)
    rows_idx = np.unique(np.concatenate([rows_of_blocks(x, blocks),
                                         rng.choice(x.outlier_rows, 160, replace=False),
                                         rng.choice(x.rows, 64, replace=False)]))
    assert np.isin(x.outlier_rows, rows_idx).sum() >= 160
    want_tok, err = check_sampled_rows(x, got["tok_logprob"], rows_idx, w64)
    assert np.abs(want_tok).max() > 100                       # the sample really holds heavy-tailed rows
    by_row = dict(zip(rows_idx.tolist(), want_tok.tolist()))
    check_block_sums(x, got, blocks, by_row)
    LQ = O.block_sums(x.draft_tok_logprob, x.block_offsets)
    LP = np.array([sum(by_row[t] for t in range(x.block_offsets[i], x.block_offsets[i + 1])) for i in range(a, b)])
    for beta in cfg.betas:
        s.select(beta, 0.7)
        torch.cuda.synchronize()
        g = s.results()
        check_selection_logic(x, g, beta, 0.7, LQ)
        check_problem_end_to_end(x, g["chosen"], g["blk_logprob_f64"], problem, LP, LQ[a:b], beta)
