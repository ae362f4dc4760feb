"""GPU parity of the E4M3 variant: the quantiser bit for bit, the scoring within the bf16 path's
tolerances against the quantised definition computed exactly by the oracle."""
import numpy as np
import pytest
import torch

from oracle import specs_fp8 as F
from oracle import specs_oracle as O
from paper_2506_15733_b200 import binding
from paper_2506_15733_b200 import inputs as I
from tests.gpu_util import BLK_RTOL, TOK_ATOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def quantize_on_gpu(ctx, bits):
    x = binding.bf16_bits_to_device(bits, DEV)
    codes = torch.full(x.shape, 0x55, dtype=torch.uint8, device=DEV)
    scale = torch.full((x.shape[0],), -1.0, dtype=torch.float32, device=DEV)
    ctx.specs_quantize_rows_e4m3(x, codes, scale)
    return codes, scale


@pytest.mark.parametrize("n,d,scale", [(37, 16, 1.0), (300, 272, 5.0), (64, 3584, 0.02)])
def test_quantiser_is_bit_exact(ctx, n, d, scale):
    cfg = I.StepConfig("q", 7400 + d, 1, 1, (n, n), d, 16, 0.05, hidden_scale=scale)
    x = I.make_step_inputs(cfg)
    bits = x.hidden.copy()
    bits[3] = 0                                                   # a row of zeros
    bits[5, 1:] = 0                                               # a single non-zero element
    codes, sc = quantize_on_gpu(ctx, bits)
    torch.cuda.synchronize()
    want_c, want_s = F.quantize_rows(bits)
    assert np.array_equal(codes.cpu().numpy(), want_c)
    assert np.array_equal(sc.cpu().numpy(), want_s)


@pytest.mark.parametrize("engine", [binding.ENGINE_TCGEN05_1CTA, binding.ENGINE_TCGEN05_2CTA])
@pytest.mark.parametrize("blk,P,n,d,V", [((1, 1), 1, 1, 16, 8), ((3, 40), 3, 5, 272, 2500), ((129, 129), 1, 1, 128, 1032),
                                         ((250, 250), 4, 10, 256, 2600)])
def test_fp8_scoring_matches_its_definition(ctx, engine, blk, P, n, d, V):
    cfg = I.StepConfig("f8", 7500 + d + V, P, n, blk, d, V, 0.05)
    x = I.make_step_inputs(cfg)
    hq, hs = quantize_on_gpu(ctx, x.hidden)
    wq, ws_ = quantize_on_gpu(ctx, x.w_vocab)
    tok = torch.full((x.rows,), float("nan"), dtype=torch.float32, device=DEV)
    blk64 = torch.full((x.blocks,), float("nan"), dtype=torch.float64, device=DEV)
    work = torch.empty(max(ctx.score_workspace_bytes_fp8(x.rows, d, V), 16), dtype=torch.uint8, device=DEV)
    ctx.set_engine(engine)
    try:
        ctx.specs_score_blocks_fp8(hq, hs, wq, ws_, torch.from_numpy(x.token_ids).to(DEV),
                                   torch.from_numpy(x.block_offsets).to(DEV), tok, None, blk64, work)
        torch.cuda.synchronize()
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    qh, sh = F.quantize_rows(x.hidden)
    qw, sw = F.quantize_rows(x.w_vocab)
    want = F.token_logprobs_fp8(qh, sh, qw, sw, x.token_ids)
    got = tok.cpu().numpy()
    assert np.abs(got - want).max() <= TOK_ATOL
    want_blk = O.block_sums(want, x.block_offsets)
    nz = want_blk != 0
    assert np.all(np.abs(blk64.cpu().numpy()[nz] - want_blk[nz]) <= BLK_RTOL * np.abs(want_blk[nz]))
    # and it is the quantisation, not the kernel, that separates it from the bf16 result
    exact = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    assert np.abs(got - exact).max() < 0.3
    assert ctx.device_status() == 0


def test_fp8_second_pass_rescoring_of_a_large_row(ctx):
    # 8-bit operands with adaptive chunks (d beyond the 1024-element base chunk): one row 128 times larger than
    # the rest is marked and re-scored from the compact buffer, with its gathered scale
    d, V = 2048, 60000                                           # runs of six vocabulary tiles per work unit
    cfg = I.StepConfig("f8fix", 7700, 1, 4, (80, 80), d, V, 1.0 / np.sqrt(d))
    x = I.make_step_inputs(cfg)
    big = x.hidden[123].copy()
    nz = (big & 0x7f80) != 0
    big[nz] += np.uint16(7 << 7)
    x.hidden[123] = big
    hq, hs = quantize_on_gpu(ctx, x.hidden)
    wq, ws_ = quantize_on_gpu(ctx, x.w_vocab)
    tok = torch.full((x.rows,), float("nan"), dtype=torch.float32, device=DEV)
    work = torch.empty(ctx.score_workspace_bytes_fp8(x.rows, d, V), dtype=torch.uint8, device=DEV)
    ctx.specs_score_blocks_fp8(hq, hs, wq, ws_, torch.from_numpy(x.token_ids).to(DEV),
                               torch.from_numpy(x.block_offsets).to(DEV), tok, None, None, work)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    qh, sh = F.quantize_rows(x.hidden)
    qw, sw = F.quantize_rows(x.w_vocab)
    want = F.token_logprobs_fp8(qh, sh, qw, sw, x.token_ids)
    assert abs(want[123]) > 50
    assert np.abs(tok.cpu().numpy() - want).max() <= TOK_ATOL
    # the fused 8-bit step quantises the hidden states itself and takes the second pass's results in its finish kernel
    from tests.gpu_util import DeviceStep
    s = DeviceStep(ctx, x)
    work2 = torch.empty(ctx.beam_step_fp8_workspace_bytes(x.rows, d, V), dtype=torch.uint8, device=DEV)
    ctx.specs_beam_step_fp8(s.hidden, wq, ws_, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.6, s.tok_lp, s.blk_lp64, s.gen_blk64, s.weights, s.chosen, s.accept, work2)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    assert np.array_equal(s.tok_lp.cpu().numpy(), tok.cpu().numpy())


def test_fp8_argument_checks(ctx):
    h = torch.zeros((4, 24), dtype=torch.uint8, device=DEV)       # d % 16 != 0
    s = torch.ones(4, dtype=torch.float32, device=DEV)
    ids = torch.zeros(4, dtype=torch.int32, device=DEV)
    off = torch.tensor([0, 4], dtype=torch.int64, device=DEV)
    tok = torch.zeros(4, dtype=torch.float32, device=DEV)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks_fp8(h, s, h, s, ids, off, tok, None, None, ws)
    assert e.value.status == 2
    h = torch.zeros((4, 32), dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks_fp8(h, None, h, s, ids, off, tok, None, None, ws)
    assert e.value.status == 1


def test_fp8_scoring_at_the_7b_shape(ctx):
    cfg = I.CONFIGS["step7b"]
    x = I.make_step_inputs(cfg)
    hq, hs = quantize_on_gpu(ctx, x.hidden)
    wq, ws_ = quantize_on_gpu(ctx, x.w_vocab)
    tok = torch.full((x.rows,), float("nan"), dtype=torch.float32, device=DEV)
    work = torch.empty(ctx.score_workspace_bytes_fp8(x.rows, cfg.d, cfg.vocab), dtype=torch.uint8, device=DEV)
    ids, off = torch.from_numpy(x.token_ids).to(DEV), torch.from_numpy(x.block_offsets).to(DEV)
    ctx.specs_score_blocks_fp8(hq, hs, wq, ws_, ids, off, tok, None, None, work)
    torch.cuda.synchronize()
    got = tok.cpu().numpy()
    assert np.all(np.isfinite(got))
    # the GPU's codes are the oracle's (checked bit for bit on W, which is the large one)
    qw, sw = F.quantize_rows(x.w_vocab)
    assert np.array_equal(wq.cpu().numpy(), qw) and np.array_equal(ws_.cpu().numpy(), sw)
    rows = np.arange(0, x.rows, 8)                                # every eighth row through the oracle
    qh, sh = F.quantize_rows(x.hidden[rows])
    want = F.token_logprobs_fp8(qh, sh, qw, sw, x.token_ids[rows])
    assert np.abs(got[rows] - want).max() <= TOK_ATOL


def test_fused_fp8_step_equals_the_separate_calls_and_the_oracle(ctx):
    from tests.gpu_util import DeviceStep, assert_step_matches
    cfg = I.StepConfig("f8step", 7600, 3, 5, (3, 60), 272, 2500, 0.05)
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    wq, wsc = quantize_on_gpu(ctx, x.w_vocab)
    work = torch.empty(ctx.beam_step_fp8_workspace_bytes(x.rows, 272, 2500), dtype=torch.uint8, device=DEV)
    ctx.specs_beam_step_fp8(s.hidden, wq, wsc, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.6, s.tok_lp, s.blk_lp64, s.gen_blk64, s.weights, s.chosen, s.accept, work)
    torch.cuda.synchronize()
    got = s.results()
    # separate calls on the same codes
    hq, hs = quantize_on_gpu(ctx, x.hidden)
    tok = torch.empty(x.rows, dtype=torch.float32, device=DEV)
    w2 = torch.empty(ctx.score_workspace_bytes_fp8(x.rows, 272, 2500), dtype=torch.uint8, device=DEV)
    ctx.specs_score_blocks_fp8(hq, hs, wq, wsc, s.token_ids, s.block_offsets, tok, None, None, w2)
    torch.cuda.synchronize()
    assert np.array_equal(tok.cpu().numpy(), got["tok_logprob"])
    # the oracle's step on the quantised definition
    qh, sh = F.quantize_rows(x.hidden)
    qw, sw = F.quantize_rows(x.w_vocab)
    lp = F.token_logprobs_fp8(qh, sh, qw, sw, x.token_ids)
    LP, LQ = O.block_sums(lp, x.block_offsets), O.block_sums(x.draft_tok_logprob, x.block_offsets)
    S = O.scores(LP, LQ, x.reward, 1.0)
    chosen, margin = O.gumbel_pick(S, x.uniforms, x.cand_offsets)
    want = {"tok_logprob": lp, "blk_logprob": LP, "chosen": chosen, "margin": margin,
            "accept": O.accept_flags(x.reward, x.cand_offsets, 0.6)}
    got["blk_logprob"] = got["blk_logprob_f64"].astype(np.float32)
    assert_step_matches(got, want, x.cand_offsets, x.block_offsets)
    assert ctx.device_status() == 0
