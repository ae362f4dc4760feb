"""The allocation-free scoring entry point against the regular one.

specs_score_blocks_noalloc serves hosts that cannot call cudaMalloc (a server whose memory
pool owns the whole device, a step loop that must avoid cudaMalloc's device-wide sync): it
takes no context and no workspace and keeps its scratch in a fixed array inside the library.
This file is collected last on purpose, so that a failure here cannot hide any other test.
It must pass both alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from oracle import specs_oracle as O
from paper_2506_15733_b200 import binding
from paper_2506_15733_b200 import inputs as I
from tests.gpu_util import BLK_RTOL, TOK_ATOL

pytestmark = pytest.mark.gpu


def _device_inputs(cfg):
    x = I.make_step_inputs(cfg)
    dev = "cuda:0"
    return x, dict(hidden=binding.bf16_bits_to_device(x.hidden, dev),
                   w_vocab=binding.bf16_bits_to_device(x.w_vocab, dev),
                   ids=torch.from_numpy(x.token_ids).to(dev),
                   offs=torch.from_numpy(x.block_offsets).to(dev))


def _regular(ctx, t, rows, B):
    tok = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda:0")
    blk = torch.full((B,), float("nan"), dtype=torch.float64, device="cuda:0")
    ws = torch.empty(ctx.score_workspace_bytes(rows, t["hidden"].shape[1], t["w_vocab"].shape[0]),
                     dtype=torch.uint8, device="cuda:0")
    ctx.specs_score_blocks(t["hidden"], t["w_vocab"], t["ids"], t["offs"], tok, None, blk, ws)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), blk.cpu().numpy()


def _noalloc(t, rows, B, status=None):
    tok = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda:0")
    blk = torch.full((B,), float("nan"), dtype=torch.float64, device="cuda:0")
    binding.specs_score_blocks_noalloc(t["hidden"], t["w_vocab"], t["ids"], t["offs"], tok, None, blk, status)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), blk.cpu().numpy()


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    torch.cuda.set_device(0)
    # two different problems back to back: the second call finds the first one's triples in the
    # shared scratch (different plan, different slot count) and must not be affected by them
    cfg_a = I.StepConfig("na_a", 5100, 3, 5, (3, 40), 256, 2500, 0.05)
    cfg_b = I.StepConfig("na_b", 5101, 2, 4, (200, 200), 128, 1000, 0.08)
    # a third one with a long reduction (d = 1024), where the regular entry point would by default lengthen
    # its accumulation chunks; the allocation-free one always uses fixed 512-element chunks
    cfg_c = I.StepConfig("na_d", 5103, 1, 3, (50, 90), 1024, 3000, 0.04)
    ctx = binding.Context(0)
    ctx.set_accum_chunk(512)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    for cfg in (cfg_a, cfg_b, cfg_c, cfg_a):
        x, t = _device_inputs(cfg)
        want_tok, want_blk = _regular(ctx, t, x.rows, x.blocks)
        got_tok, got_blk = _noalloc(t, x.rows, x.blocks, status)
        assert np.all(np.isfinite(got_tok))
        assert np.abs(got_tok - want_tok).max() <= TOK_ATOL
        assert np.all(np.abs(got_blk - want_blk) <= BLK_RTOL * np.abs(want_blk))
        assert np.array_equal(got_tok, want_tok)              # same kernels, same plan: in fact bit-identical
        # and directly against the CPU oracle
        oracle_tok = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
        oracle_blk = O.block_sums(oracle_tok, x.block_offsets)
        assert np.abs(got_tok - oracle_tok).max() <= TOK_ATOL
        assert np.all(np.abs(got_blk - oracle_blk) <= BLK_RTOL * np.abs(oracle_blk))
    assert int(status.item()) == 0
    assert ctx.device_status() == 0
    ctx.close()


def test_noalloc_reports_bad_ids_and_rejects_oversized_problems():
    torch.cuda.set_device(0)
    cfg = I.StepConfig("na_c", 5102, 1, 2, (8, 8), 64, 300, 0.05)
    x, t = _device_inputs(cfg)
    t["ids"][5] = 300
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    tok, _ = _noalloc(t, x.rows, x.blocks, status)
    assert np.isnan(tok[5]) and np.isfinite(np.delete(tok, 5)).all()
    assert int(status.item()) == binding.DEV_TOKEN_RANGE
    _noalloc(t, x.rows, x.blocks, None)                       # NULL status word is allowed

    # a plan that needs more scratch than the fixed array: refused on the host, nothing launched.
    # Only the shapes matter for the refusal, so the tensors below are never read.
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows = 128 * sms * 20                                     # 20 full waves at d = 64 -> 20 * sms * 3072 bytes
    assert binding.score_plan(rows, 64, 300, sms)["workspace_bytes"] > binding.NOALLOC_SCRATCH_BYTES
    big_h = torch.empty((rows, 64), dtype=torch.bfloat16, device="cuda:0")
    big_ids = torch.zeros(rows, dtype=torch.int32, device="cuda:0")
    big_tok = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda:0")
    offs = torch.tensor([0, rows], dtype=torch.int64, device="cuda:0")
    with pytest.raises(binding.SpecsError) as e:
        binding.specs_score_blocks_noalloc(big_h, t["w_vocab"], big_ids, offs, big_tok)
    assert e.value.status == 10
    torch.cuda.synchronize()
    assert torch.isnan(big_tok).all()
