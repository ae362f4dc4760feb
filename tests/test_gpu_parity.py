"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Run with -m gpu on a B200."""
import math

import numpy as np
import pytest
import torch

from oracle import specs_oracle as O
from paper_2506_15733_b200 import binding
from paper_2506_15733_b200 import inputs as I
from tests.gpu_util import BLK_RTOL, MARGIN, TOK_ATOL, DeviceStep, assert_step_matches

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    assert c.device_status() == 0, "device status word not clean at the end of the module"
    c.close()


def oracle_step(x, beta, tau, with_draft=True):
    return O.beam_step(x.hidden, x.w_vocab, x.token_ids, x.block_offsets, x.cand_offsets,
                       x.draft_tok_logprob if with_draft else None, x.reward, beta, x.uniforms, tau)


def small_config(name, rows_per_block, problems, beams, d, V, seed, **kw):
    return I.StepConfig(name, seed, problems, beams, rows_per_block, d, V, kw.pop("w_sigma", 0.05), **kw)


# ------------------------------------------------------------------------------- tiny, both engines

TC_ENGINES = [binding.ENGINE_TCGEN05_1CTA, binding.ENGINE_TCGEN05_2CTA]   # both tile shapes of the tensor-core kernel
# the plain CUDA-core engine exists in the checked build only (SPECS_B200_DEBUG=1, see tests/test_gpu_debug_build.py)
SIMT_ENGINE = [binding.ENGINE_SIMT] if binding.debug_build() else []


@pytest.mark.parametrize("engine", SIMT_ENGINE + [binding.ENGINE_TCGEN05] + TC_ENGINES)
def test_tiny_config_full_step(ctx, engine):
    x = I.make_step_inputs(I.CONFIGS["tiny"])
    ctx.set_engine(engine)
    try:
        got = DeviceStep(ctx, x).step(1.0, 0.7)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    want = oracle_step(x, 1.0, 0.7)
    info = assert_step_matches(got, want, x.cand_offsets, x.block_offsets)
    w_err = np.abs(got["weights"] - want["weights"]).max()
    assert w_err < 5e-3, w_err
    assert abs(got["weights"].sum() - 1.0) < 1e-5
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- tile edges and ragged tails

EDGE_CASES = [
    # rows/block range, problems, beams, d, V
    ((1, 1), 1, 1, 8, 8),            # a single row, a single k-block with a 56-element tail, 8 vocab entries
    ((127, 127), 1, 1, 72, 1000),    # one row short of a tile; d and V with ragged tails
    ((129, 129), 1, 1, 64, 1032),    # one row over a tile; V = 4 tiles + 8
    ((3, 40), 3, 5, 256, 2500),      # ragged blocks, several tiles, vocab tail of 196
    ((16, 16), 2, 4, 520, 257),      # vocab tile with a single valid column in its last tile
    ((50, 50), 1, 6, 1024, 4096),    # exact multiples everywhere
    ((75, 75), 1, 4, 128, 700),      # three row tiles: the last CTA pair has one CTA without rows
]


@pytest.mark.parametrize("engine", TC_ENGINES)
@pytest.mark.parametrize("blk,P,n,d,V", EDGE_CASES)
def test_edge_shapes(ctx, blk, P, n, d, V, engine):
    cfg = small_config("edge", blk, P, n, d, V, seed=4000 + d + V)
    x = I.make_step_inputs(cfg)
    ctx.set_engine(engine)
    try:
        got = DeviceStep(ctx, x).step(1.0, 0.5)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    want = oracle_step(x, 1.0, 0.5)
    assert_step_matches(got, want, x.cand_offsets, x.block_offsets)
    assert ctx.device_status() == 0


def test_empty_blocks_and_empty_problem(ctx):
    cfg = small_config("holes", (5, 9), 3, 3, 64, 300, seed=4100)
    x = I.make_step_inputs(cfg)
    # make block 2 and block 7 empty, and problem 1 empty (its three blocks move to problem 2)
    lens = np.diff(x.block_offsets)
    lens[2] = 0
    lens[7] = 0
    x.block_offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    rows = int(x.block_offsets[-1])
    x.hidden, x.token_ids, x.draft_tok_logprob = x.hidden[:rows], x.token_ids[:rows], x.draft_tok_logprob[:rows]
    x.cand_offsets = np.array([0, 3, 3, 9], dtype=np.int32)
    got = DeviceStep(ctx, x).step(2.0, 0.4)
    want = oracle_step(x, 2.0, 0.4)
    assert_step_matches(got, want, x.cand_offsets, x.block_offsets)
    assert got["blk_logprob"][2] == 0.0 and got["blk_logprob"][7] == 0.0
    assert got["chosen"][1] == -1 and got["accept"][1] == 0


def test_zero_rows_is_a_noop(ctx):
    dev = "cuda:0"
    w = binding.bf16_bits_to_device(np.zeros((16, 8), np.uint16), dev)
    h = torch.empty((0, 8), dtype=torch.bfloat16, device=dev)
    ids = torch.empty((0,), dtype=torch.int32, device=dev)
    offs = torch.zeros(3, dtype=torch.int64, device=dev)
    tok = torch.empty((0,), dtype=torch.float32, device=dev)
    blk = torch.full((2,), 5.0, dtype=torch.float32, device=dev)
    ctx.specs_score_blocks(h, w, ids, offs, tok, blk, None, None)
    torch.cuda.synchronize()
    assert blk.tolist() == [0.0, 0.0]


# ------------------------------------------------------------------------------- several waves of work units

@pytest.mark.parametrize("engine", TC_ENGINES)
@pytest.mark.parametrize("rows_total,d,V", [(20000, 64, 1000), (10000, 1536, 2048), (40000, 128, 520)])
def test_multi_wave_plans(ctx, rows_total, d, V, engine):
    sms = ctx.sm_count()
    plan = binding.score_plan(rows_total, d, V, sms, 1 if engine == binding.ENGINE_TCGEN05_1CTA else 2)
    assert plan["waves"] >= 2, plan
    blocks = 40
    cfg = small_config("waves", (rows_total // blocks, rows_total // blocks), 4, blocks // 4, d, V,
                       seed=4200 + d, w_sigma=0.5 / math.sqrt(d) * 4)
    x = I.make_step_inputs(cfg)
    ctx.set_engine(engine)
    try:
        got = DeviceStep(ctx, x).step(1.0, 0.6)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    want = oracle_step(x, 1.0, 0.6)
    assert_step_matches(got, want, x.cand_offsets, x.block_offsets)
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- device-detected conditions

def test_out_of_range_token_is_nan_and_flagged(ctx):
    cfg = small_config("badid", (8, 8), 1, 2, 64, 300, seed=4300)
    x = I.make_step_inputs(cfg)
    x.token_ids = x.token_ids.copy()
    x.token_ids[3] = 300
    x.token_ids[9] = -2
    for engine in TC_ENGINES + SIMT_ENGINE:
        ctx.set_engine(engine)
        try:
            s = DeviceStep(ctx, x)
            s.score()
            torch.cuda.synchronize()
        finally:
            ctx.set_engine(binding.ENGINE_TCGEN05)
        lp = s.tok_lp.cpu().numpy()
        assert np.isnan(lp[3]) and np.isnan(lp[9])
        ok = np.ones(16, bool)
        ok[[3, 9]] = False
        want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
        assert np.abs(lp[ok] - want[ok]).max() <= TOK_ATOL
        assert ctx.device_status() == binding.DEV_TOKEN_RANGE
        assert ctx.device_status() == 0                       # reading clears it


def test_host_side_argument_errors(ctx):
    cfg = small_config("args", (4, 4), 1, 2, 64, 300, seed=4400)
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.tok_lp, s.blk_lp, None,
                               s.workspace[:64])
    assert e.value.status == 4                                # workspace too small
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks(s.hidden, s.w_vocab, None, s.block_offsets, s.tok_lp, s.blk_lp, None, s.workspace)
    assert e.value.status == 1
    odd = s.hidden.view(torch.int16).reshape(-1)[4:4 + 7 * 64].view(torch.bfloat16).reshape(7, 64)   # 8-byte aligned
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks(odd, s.w_vocab, s.token_ids, s.block_offsets, s.tok_lp, None, None, s.workspace)
    assert e.value.status == 3
    bad_d = torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_score_blocks(bad_d, bad_d, s.token_ids, s.block_offsets, s.tok_lp, None, None, s.workspace)
    assert e.value.status == 2
    torch.cuda.synchronize()
    assert torch.isnan(s.tok_lp).all()                        # nothing was launched, outputs untouched


# ------------------------------------------------------------------------------- selection kernels alone

@pytest.mark.parametrize("beta", [0.0, 1.0, 4.0, 1.0e4])
@pytest.mark.parametrize("f64", [False, True])
def test_subsample_matches_oracle_on_many_problems(ctx, beta, f64):
    rng = np.random.Generator(np.random.Philox(key=[4500, int(beta) + 7 * f64]))
    sizes = rng.integers(0, 70, size=3000)                    # includes empty problems and n > 32
    cand = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    B = int(cand[-1])
    lp_t = rng.uniform(-4000, -5, B)
    lp_g = lp_t + rng.normal(0, 3.0, B)
    if not f64:
        lp_t, lp_g = lp_t.astype(np.float32), lp_g.astype(np.float32)
    r = rng.random(B).astype(np.float32)
    u = I.draw_uniforms(4501, B)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(a).to(dev)
    chosen = torch.empty(len(sizes), dtype=torch.int32, device=dev)
    wts = torch.empty(B, dtype=torch.float32, device=dev)
    acc = torch.empty(len(sizes), dtype=torch.uint8, device=dev)
    ctx.specs_subsample(t(lp_t), t(lp_g), t(r), t(cand), beta, t(u), chosen, wts, 0.97, acc)
    torch.cuda.synchronize()
    S = O.scores(lp_t, lp_g, r, beta)
    want_c, margin = O.gumbel_pick(S, u, cand)
    want_w = O.weights(S, cand)
    got_c = chosen.cpu().numpy()
    sure = margin > MARGIN
    assert sure.sum() > 2000
    assert np.array_equal(got_c[sure], want_c[sure])
    assert np.array_equal(got_c[sizes == 0], np.full((sizes == 0).sum(), -1))
    assert np.all((got_c[sizes > 0] >= 0) & (got_c[sizes > 0] < sizes[sizes > 0]))
    assert np.abs(wts.cpu().numpy() - want_w).max() < 1e-6
    assert np.array_equal(acc.cpu().numpy(), O.accept_flags(r, cand, 0.97))


def test_subsample_same_generator_and_null_outputs(ctx):
    # pi_gen = pi_target: scores collapse to beta * r (text after Eq. 1); weights and accept are optional
    rng = np.random.Generator(np.random.Philox(key=[4600, 1]))
    n, P = 16, 500
    cand = (np.arange(P + 1) * n).astype(np.int32)
    r = rng.beta(2, 2, n * P).astype(np.float32)
    u = I.draw_uniforms(4601, n * P)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(a).to(dev)
    chosen = torch.empty(P, dtype=torch.int32, device=dev)
    wts = torch.empty(n * P, dtype=torch.float32, device=dev)
    ctx.specs_subsample(None, None, t(r), t(cand), 4.0, t(u), chosen, wts)
    chosen2 = torch.empty(P, dtype=torch.int32, device=dev)
    ctx.specs_subsample(None, None, t(r), t(cand), 4.0, t(u), chosen2, None)
    torch.cuda.synchronize()
    S = O.scores(None, None, r, 4.0)
    want_c, margin = O.gumbel_pick(S, u, cand)
    sure = margin > MARGIN
    assert np.array_equal(chosen.cpu().numpy()[sure], want_c[sure])
    assert np.array_equal(chosen.cpu().numpy(), chosen2.cpu().numpy())
    e = np.exp(4.0 * r.astype(np.float64)).reshape(P, n)
    assert np.abs(wts.cpu().numpy().reshape(P, n) - e / e.sum(1, keepdims=True)).max() < 1e-6


@pytest.mark.parametrize("beta", [0.0, 1.0, 4.0])
def test_gpu_sampler_chi_squared(ctx, beta):
    # empirical pick frequencies of the CUDA sampler against the closed-form weights
    from scipy import stats
    LP = np.array([-20.0, -21.0, -19.5, -22.0, -20.5, -23.0, -19.0, -21.5], dtype=np.float32)
    LQ = np.array([-20.5, -20.0, -20.0, -21.0, -21.5, -22.0, -20.0, -21.0], dtype=np.float32)
    r = np.array([0.1, 0.6, 0.3, 0.9, 0.5, 0.7, 0.2, 0.4], dtype=np.float32)
    n, draws = 8, 400_000
    cand = (np.arange(draws + 1) * n).astype(np.int32)
    u = I.draw_uniforms(4700 + int(beta), n * draws)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(a).to(dev)
    chosen = torch.empty(draws, dtype=torch.int32, device=dev)
    ctx.specs_subsample(t(np.tile(LP, draws)), t(np.tile(LQ, draws)), t(np.tile(r, draws)), t(cand), beta, t(u),
                        chosen, None)
    torch.cuda.synchronize()
    counts = np.bincount(chosen.cpu().numpy(), minlength=n)
    expected = draws * O.weights(O.scores(LP, LQ, r, beta), np.array([0, n]))
    assert expected.min() >= 5
    assert stats.chisquare(counts, expected).pvalue > 1e-3, (counts, expected)


def test_accept_threshold_sweep(ctx):
    x = I.make_step_inputs(I.CONFIGS["batched"], with_weights=False)
    dev = "cuda:0"
    r = torch.from_numpy(x.reward).to(dev)
    cand = torch.from_numpy(x.cand_offsets).to(dev)
    acc = torch.empty(32, dtype=torch.uint8, device=dev)
    prev = None
    for tau in (-1.0,) + I.CONFIGS["batched"].taus + (1.0,):
        ctx.specs_accept(r, cand, tau, acc)
        torch.cuda.synchronize()
        got = acc.cpu().numpy()
        assert np.array_equal(got, O.accept_flags(x.reward, x.cand_offsets, tau))
        if prev is not None:
            assert np.all(got <= prev)
        prev = got
    assert prev.sum() == 0                                    # tau = 1: never switches to the draft


def test_block_sums_kernel(ctx):
    rng = np.random.Generator(np.random.Philox(key=[4800, 1]))
    lens = rng.integers(0, 600, 300)
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    v = rng.uniform(-12, 0, int(offs[-1])).astype(np.float32)
    dev = "cuda:0"
    o32 = torch.empty(300, dtype=torch.float32, device=dev)
    o64 = torch.empty(300, dtype=torch.float64, device=dev)
    ctx.specs_block_sums(torch.from_numpy(v).to(dev), torch.from_numpy(offs).to(dev), o32, o64)
    torch.cuda.synchronize()
    want = O.block_sums(v, offs)
    assert np.abs(o64.cpu().numpy() - want).max() < 1e-9
    assert np.array_equal(o32.cpu().numpy(), want.astype(np.float32)) or \
        np.abs(o32.cpu().numpy() - want).max() <= 1e-6 * np.abs(want).max()


# ------------------------------------------------------------------------------- fused device step

def _fused_step(ctx, s, beta, tau, with_draft=True):
    ctx.specs_beam_step(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets,
                        s.draft if with_draft else None, s.reward, s.uniforms, beta, tau, s.tok_lp, s.blk_lp64,
                        s.gen_blk64 if with_draft else None, s.weights, s.chosen, s.accept, s.workspace)
    torch.cuda.synchronize()
    return s.results()


@pytest.mark.parametrize("engine", [binding.ENGINE_TCGEN05] + TC_ENGINES)
@pytest.mark.parametrize("with_draft", [True, False])
def test_fused_beam_step_equals_the_separate_calls(ctx, engine, with_draft):
    cfg = small_config("fused", (3, 90), 7, 5, 256, 2500, seed=4950)
    x = I.make_step_inputs(cfg)
    # holes: an empty block, an empty problem in the middle and one at the end
    lens = np.diff(x.block_offsets)
    lens[4] = 0
    x.block_offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    rows = int(x.block_offsets[-1])
    x.hidden, x.token_ids, x.draft_tok_logprob = x.hidden[:rows], x.token_ids[:rows], x.draft_tok_logprob[:rows]
    x.cand_offsets = np.array([0, 5, 10, 10, 15, 20, 25, 35, 35], dtype=np.int32)
    ctx.set_engine(engine)
    try:
        want = DeviceStep(ctx, x).step(1.5, 0.55, with_draft)
        got = _fused_step(ctx, DeviceStep(ctx, x), 1.5, 0.55, with_draft)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    for key in ("tok_logprob", "blk_logprob_f64", "weights", "chosen", "accept") + (("blk_logprob_gen",) if with_draft else ()):
        assert np.array_equal(got[key], want[key]), key
    assert got["chosen"][2] == -1 and got["chosen"][7] == -1 and got["accept"][2] == 0
    ref = oracle_step(x, 1.5, 0.55, with_draft)
    got["blk_logprob"] = got["blk_logprob_f64"].astype(np.float32)
    assert_step_matches(got, ref, x.cand_offsets, x.block_offsets)
    assert ctx.device_status() == 0


def test_fused_beam_step_flags_bad_ids_and_validates(ctx):
    cfg = small_config("fused_bad", (8, 8), 2, 2, 64, 300, seed=4960)
    x = I.make_step_inputs(cfg)
    x.token_ids = x.token_ids.copy()
    x.token_ids[5] = 999
    s = DeviceStep(ctx, x)
    got = _fused_step(ctx, s, 1.0, 0.5)
    assert np.isnan(got["tok_logprob"][5]) and np.isfinite(np.delete(got["tok_logprob"], 5)).all()
    assert ctx.device_status() == binding.DEV_TOKEN_RANGE
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_beam_step(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.5, s.tok_lp, None, s.gen_blk64, s.weights, s.chosen, s.accept, s.workspace)
    assert e.value.status == 1                                # the block sums are required outputs
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_beam_step(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.5, s.tok_lp, s.blk_lp64, s.gen_blk64, s.weights, s.chosen, s.accept,
                            s.workspace[:64])
    assert e.value.status == 4


# ------------------------------------------------------------------------------- host-buffer entry point

def test_beam_step_host_equals_device_calls(ctx):
    cfg = small_config("host", (3, 40), 3, 5, 256, 2500, seed=4900)
    x = I.make_step_inputs(cfg)
    want_dev = DeviceStep(ctx, x).step(1.5, 0.55)
    rows, B, P = x.rows, x.blocks, 3
    tok = np.empty(rows, np.float32); blk = np.empty(B, np.float64); wts = np.empty(B, np.float32)
    cho = np.empty(P, np.int32); acc = np.empty(P, np.uint8)
    w_dev = binding.bf16_bits_to_device(x.w_vocab, "cuda:0")
    for _ in range(2):                                        # the second call reuses the arena
        ctx.specs_beam_step_host(x.hidden, w_dev, x.token_ids, x.block_offsets, x.cand_offsets,
                                 x.draft_tok_logprob, x.reward, x.uniforms, 1.5, 0.55, tok, blk, wts, cho, acc)
        assert np.array_equal(tok, want_dev["tok_logprob"])
        assert np.array_equal(blk, want_dev["blk_logprob_f64"])
        assert np.array_equal(wts, want_dev["weights"])
        assert np.array_equal(cho, want_dev["chosen"]) and np.array_equal(acc, want_dev["accept"])
    bad = x.block_offsets.copy()
    bad[2] = bad[3] + 1
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_beam_step_host(x.hidden, w_dev, x.token_ids, bad, x.cand_offsets, x.draft_tok_logprob, x.reward,
                                 x.uniforms, 1.5, 0.55, tok, blk, wts, cho, acc)
    assert e.value.status == 5


def test_two_host_steps_in_flight_equal_two_serial_steps(ctx):
    # two different steps submitted back to back (the second one's copies may run under the first one's
    # kernels), waited for in both orders, against the same steps run one after the other
    cfgs = [small_config("inflight_a", (3, 40), 3, 5, 256, 2500, seed=4910),
            small_config("inflight_b", (10, 90), 2, 6, 1024, 3000, seed=4911)]    # the second has adaptive chunks
    xs = [I.make_step_inputs(c) for c in cfgs]
    w_devs = [binding.bf16_bits_to_device(x.w_vocab, "cuda:0") for x in xs]
    pinned = [binding.bf16_bits_to_pinned(x.hidden) for x in xs]

    def outputs(x):
        P = len(x.cand_offsets) - 1
        return [np.empty(x.rows, np.float32), np.empty(x.blocks, np.float64), np.empty(x.blocks, np.float32),
                np.empty(P, np.int32), np.empty(P, np.uint8)]

    serial = []
    for x, w, h in zip(xs, w_devs, pinned):
        o = outputs(x)
        ctx.specs_beam_step_host(h, w, x.token_ids, x.block_offsets, x.cand_offsets, x.draft_tok_logprob, x.reward,
                                 x.uniforms, 1.5, 0.55, *o)
        serial.append(o)
    for order in ((0, 1), (1, 0)):
        outs = [outputs(x) for x in xs]
        for o in outs:
            for a in o:
                a.fill(0)
        tickets = [ctx.specs_beam_step_host_submit(h, w, x.token_ids, x.block_offsets, x.cand_offsets,
                                                   x.draft_tok_logprob, x.reward, x.uniforms, 1.5, 0.55, *o)
                   for x, w, h, o in zip(xs, w_devs, pinned, outs)]
        assert tickets[0] != tickets[1]
        with pytest.raises(binding.SpecsError) as e:          # a third step has no slot
            ctx.specs_beam_step_host_submit(pinned[0], w_devs[0], xs[0].token_ids, xs[0].block_offsets,
                                            xs[0].cand_offsets, xs[0].draft_tok_logprob, xs[0].reward,
                                            xs[0].uniforms, 1.5, 0.55, *outputs(xs[0]))
        assert e.value.status == 10
        for k in order:
            ctx.specs_beam_step_host_wait(tickets[k])
            for got, want in zip(outs[k], serial[k]):
                assert np.array_equal(got, want)
        with pytest.raises(binding.SpecsError) as e:          # waited for already
            ctx.specs_beam_step_host_wait(tickets[0])
        assert e.value.status == 2
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- adaptive accumulation chunks

def _score_only(ctx, x):
    s = DeviceStep(ctx, x)
    s.score()
    torch.cuda.synchronize()
    return s.tok_lp.cpu().numpy()


@pytest.mark.parametrize("sigma_z", [1.5, 3.0, 6.0, 12.0, 24.0, 48.0])
def test_adaptive_chunks_keep_the_tolerance_across_logit_magnitudes(ctx, sigma_z):
    # long reduction (d = 5120), runs of at least three vocabulary tiles per work unit, and logit scales
    # that land in different chunk lengths (unchunked ... 1024 elements ... the 512-element base)
    d, V = 5120, 60000
    cfg = small_config("adapt", (75, 75), 1, 4, d, V, seed=5200 + int(10 * sigma_z), w_sigma=sigma_z / math.sqrt(d))
    x = I.make_step_inputs(cfg)
    p = binding.score_plan(x.rows, d, V, ctx.sm_count())
    runs = [ne - nb for mt, nb, ne in (binding.score_plan_unit(x.rows, d, V, ctx.sm_count(), 0, c)
                                        for c in range(p["grid"])) if mt >= 0]
    assert min(runs) >= 3, "the case must exercise the adaptive path"
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    got = {}
    for mode in (binding.ACCUM_ADAPTIVE, 512):
        ctx.set_accum_chunk(mode)
        try:
            got[mode] = _score_only(ctx, x)
        finally:
            ctx.set_accum_chunk(binding.ACCUM_ADAPTIVE)
        assert ctx.device_status() == 0
        err = np.abs(got[mode] - want).max()
        assert err <= TOK_ATOL, (mode, err)
    # the lengthened chunks stay within a quarter of the tolerance of the fixed short ones
    assert np.abs(got[binding.ACCUM_ADAPTIVE] - got[512]).max() <= TOK_ATOL / 4


def _scale_rows_by_128(bits, rows, log2_factor=7):
    """Exact multiplication by 128 (or 2^log2_factor) of the given rows of a bf16 bit array (exponent + 7),
    zeros left alone."""
    out = bits.copy()
    sel = out[rows]
    nz = (sel & 0x7f80) != 0
    sel[nz] += np.uint16(log2_factor << 7)
    out[rows] = sel
    return out


def _last_tiles_of_runs(ctx, rows, d, V):
    """Vocabulary tiles (of 256 entries) that end some work unit's run in the plan for these sizes."""
    p = binding.score_plan(rows, d, V, ctx.sm_count())
    ends = set()
    for c in range(p["grid"]):
        mt, nb, ne = binding.score_plan_unit(rows, d, V, ctx.sm_count(), 0, c)
        if mt >= 0 and ne - nb >= 3:
            ends.add(ne - 1)
    return sorted(ends)


@pytest.mark.parametrize("case", ["from_second_tile", "last_tile_of_each_run", "one_row", "more_rows_than_gathered"])
def test_adaptive_chunks_rescore_rows_beyond_the_sampled_magnitude(ctx, case):
    # Logits far larger than what the first vocabulary tile of a run showed: the chunk length chosen from
    # that tile is too long for them.  Such rows are marked, re-scored with the base chunks in a second
    # pass, and the per-token tolerance holds wherever in the vocabulary the large logits sit.
    d, V = 5120, 60000
    blocks = 12 if case == "more_rows_than_gathered" else 4
    cfg = small_config("adapt_surprise", (64, 64), 1, blocks, d, V, seed=5300, w_sigma=1.0 / math.sqrt(d))
    x = I.make_step_inputs(cfg)
    if case in ("from_second_tile", "more_rows_than_gathered"):
        x.w_vocab = _scale_rows_by_128(x.w_vocab, np.arange(256, V))
    elif case == "last_tile_of_each_run":
        tiles = _last_tiles_of_runs(ctx, x.rows, d, V)
        assert tiles
        x.w_vocab = _scale_rows_by_128(x.w_vocab, np.concatenate([np.arange(256 * t, min(256 * t + 256, V))
                                                                  for t in tiles]))
    else:
        x.hidden = _scale_rows_by_128(x.hidden, np.array([37]))
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    assert np.abs(want).max() > 50                           # the case really holds large logits
    got = _score_only(ctx, x)
    assert np.all(np.isfinite(got))
    assert np.abs(got - want).max() <= TOK_ATOL
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE    # reported: some rows went through the second pass
    # the fused step takes the second pass's results in its finish kernel: same bits
    f = DeviceStep(ctx, x)
    ctx.specs_beam_step(f.hidden, f.w_vocab, f.token_ids, f.block_offsets, f.cand_offsets, f.draft, f.reward,
                        f.uniforms, 1.0, 0.7, f.tok_lp, f.blk_lp64, f.gen_blk64, f.weights, f.chosen, f.accept,
                        f.workspace)
    torch.cuda.synchronize()
    assert np.array_equal(f.tok_lp.cpu().numpy(), got)
    assert np.allclose(f.blk_lp64.cpu().numpy(), O.block_sums(got, x.block_offsets), rtol=1e-12)
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    # fixed short chunks need no second pass and agree
    ctx.set_accum_chunk(512)
    try:
        fixed = _score_only(ctx, x)
    finally:
        ctx.set_accum_chunk(binding.ACCUM_ADAPTIVE)
    assert ctx.device_status() == 0
    assert np.abs(fixed - want).max() <= TOK_ATOL
    if case == "more_rows_than_gathered":
        assert np.array_equal(fixed, got)                    # every row was re-scored in place, same plan, same chunks
    elif case != "one_row":
        # every row was re-scored with those chunks, under another cut of the vocabulary: rounding only
        assert np.all(np.abs(fixed - got) <= 1e-4 * np.maximum(1.0, np.abs(want)))


@pytest.mark.parametrize("engine", TC_ENGINES)
def test_second_pass_under_both_tile_shapes(ctx, engine):
    # the second pass has its own instantiation per tile shape: one large row, and every row large, under each
    d, V = 2048, 30000
    cfg = small_config("adapt_shapes", (96, 96), 1, 4, d, V, seed=5310, w_sigma=1.0 / math.sqrt(d))
    x = I.make_step_inputs(cfg)
    for rows_scaled in (np.array([200]), np.arange(x.rows)):
        y = I.make_step_inputs(cfg)
        y.hidden = _scale_rows_by_128(x.hidden, rows_scaled)
        want = O.token_logprobs(y.hidden, y.w_vocab, y.token_ids)
        ctx.set_engine(engine)
        try:
            got = _score_only(ctx, y)
        finally:
            ctx.set_engine(binding.ENGINE_TCGEN05)
        # every row large: the first tile already shows it, the base chunks are kept and nothing is re-scored
        expect_bits = binding.DEV_ACCUM_RANGE if len(rows_scaled) == 1 else 0
        assert ctx.device_status() == expect_bits
        assert np.abs(got - want).max() <= TOK_ATOL


@pytest.mark.parametrize("log2_factor", [9, 10])
def test_rows_beyond_the_base_chunks_range_get_shorter_chunks(ctx, log2_factor):
    # |logit| in the thousands: even 512-element chunks would leave a few 1e-3 of truncation there, so such rows
    # are marked whatever chunks the first pass used, and the second pass shortens its chunks to their magnitude
    d, V = 5120, 60000
    cfg = small_config("adapt_huge", (64, 64), 1, 4, d, V, seed=5320, w_sigma=1.0 / math.sqrt(d))
    x = I.make_step_inputs(cfg)
    x.hidden = _scale_rows_by_128(x.hidden, np.array([11, 200]), log2_factor)
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    assert np.abs(want[[11, 200]]).min() > 500
    got = _score_only(ctx, x)
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    assert np.abs(got - want).max() <= TOK_ATOL


def test_second_pass_reaches_the_shard_partials_and_the_two_head_step(ctx):
    # one large row, long reductions: marked and re-scored (a) in a vocabulary shard, whose partials must then
    # be the second pass's, and (b) in both heads of the two-head step, whose finish kernel takes both fix-ups
    from paper_2506_15733_b200 import vocab_parallel as VP
    d, V = 2048, 30000
    cfg = small_config("fix_routes", (96, 96), 2, 4, d, V, seed=5330, w_sigma=1.0 / math.sqrt(d))   # 768 rows
    x = I.make_step_inputs(cfg)
    x.hidden = _scale_rows_by_128(x.hidden, np.array([150]))
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    dev = "cuda:0"
    s = DeviceStep(ctx, x)
    # (a) two shards
    parts = []
    for rank in range(2):
        v0, v1 = VP.shard_bounds(V, 2, rank)
        local = torch.full((x.rows, 4), float("nan"), dtype=torch.float32, device=dev)
        ws = torch.empty(ctx.score_workspace_bytes(x.rows, d, v1 - v0), dtype=torch.uint8, device=dev)
        ctx.specs_score_partials(s.hidden, s.w_vocab[v0:v1], s.token_ids, v0, local, ws)
        parts.append(local)
    out = torch.full((x.rows,), 7.0, dtype=torch.float32, device=dev)
    ctx.specs_merge_partials(torch.stack(parts), s.token_ids, V, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    assert np.abs(out.cpu().numpy() - want).max() <= TOK_ATOL
    # (b) both heads: the generator's head is the target's own here (same hidden states and weights)
    gen_tok = torch.full((x.rows,), float("nan"), dtype=torch.float32, device=dev)
    ws = torch.empty(ctx.beam_step_dual_workspace_bytes(x.rows, d, d, V), dtype=torch.uint8, device=dev)
    ids_out = torch.full((2, 96), -9, dtype=torch.int32, device=dev)
    len_out = torch.full((2,), -9, dtype=torch.int32, device=dev)
    ctx.specs_beam_step_dual(s.hidden, s.w_vocab, s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets,
                             s.reward, s.uniforms, 1.0, 0.6, s.tok_lp, gen_tok, s.blk_lp64, s.gen_blk64, s.weights,
                             s.chosen, s.accept, ws, ids_out, len_out)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    t, g = s.tok_lp.cpu().numpy(), gen_tok.cpu().numpy()
    assert np.abs(t - want).max() <= TOK_ATOL and np.array_equal(t, g)
    assert np.allclose(s.blk_lp64.cpu().numpy(), O.block_sums(t, x.block_offsets), rtol=1e-12)
    # identical heads: the ratio drops out, the weights are softmax(beta r) (text after Eq. 1)
    assert np.abs(s.weights.cpu().numpy() - O.weights(O.scores(None, None, x.reward, 1.0), x.cand_offsets)).max() < 1e-6


def test_one_large_row_does_not_shorten_its_tiles_chunks(ctx):
    # 1 % of the rows 20 times larger (the stress recipe): only those rows are re-scored; the others
    # keep the chunk length their own magnitude allows, and all meet the tolerance
    d, V = 5120, 60000
    cfg = small_config("adapt_outliers", (128, 128), 1, 6, d, V, seed=5301, w_sigma=6.0 / math.sqrt(d),
                       outlier_frac=0.01, outlier_mult=20.0)
    x = I.make_step_inputs(cfg)
    assert 2 <= len(x.outlier_rows) <= 24
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    got = _score_only(ctx, x)
    assert ctx.device_status() == binding.DEV_ACCUM_RANGE
    assert np.abs(got - want).max() <= TOK_ATOL
    ctx.set_accum_chunk(512)
    try:
        fixed = _score_only(ctx, x)
    finally:
        ctx.set_accum_chunk(binding.ACCUM_ADAPTIVE)
    assert ctx.device_status() == 0
    # the outlier rows were re-scored with the base chunks; the ordinary rows were not (different rounding)
    o = x.outlier_rows
    assert np.all(np.abs(got[o] - fixed[o]) <= 1e-4 * np.maximum(1.0, np.abs(want[o])))
    assert not np.array_equal(np.delete(got, o), np.delete(fixed, o))


# ------------------------------------------------------------------------------- selection variants

from oracle import specs_variants as OV   # noqa: E402


@pytest.mark.parametrize("select_rule", [OV.SELECT_SUBSAMPLE, OV.SELECT_BEST_REWARD])
@pytest.mark.parametrize("score_flags", [0, OV.SCORE_NO_LL])
@pytest.mark.parametrize("masked", [False, True])
def test_select_variants_match_the_oracle(ctx, select_rule, score_flags, masked):
    rng = np.random.Generator(np.random.Philox(key=[5400, select_rule * 4 + score_flags * 2 + masked]))
    sizes = rng.integers(0, 70, size=1500)
    cand = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    B, P = int(cand[-1]), len(sizes)
    lp_t = rng.uniform(-4000, -5, B)
    lp_g = lp_t + rng.normal(0, 3.0, B)
    r = rng.random(B).astype(np.float32)
    r[rng.integers(0, B, 200)] = np.float32(0.5)                    # ties in the reward
    u = I.draw_uniforms(5401, B)
    mask = (rng.random(B) < 0.6).astype(np.uint8) if masked else None
    if masked:
        mask[cand[10]:cand[11]] = 0                                 # a problem with nobody in L
    dev = "cuda:0"
    t = lambda a: None if a is None else torch.from_numpy(a).to(dev)
    d_in = [t(lp_t), t(lp_g), t(r), t(mask), t(cand)]
    chosen = torch.full((P,), -7, dtype=torch.int32, device=dev)
    wts = torch.full((B,), float("nan"), dtype=torch.float32, device=dev)
    flag = torch.full((P,), 9, dtype=torch.uint8, device=dev)
    want_c, want_w, margin = OV.select(lp_t, lp_g, r, mask, cand, 2.0, u, select_rule, score_flags)
    for switch_rule in (OV.SWITCH_ANY_ABOVE, OV.SWITCH_NONE_ABOVE, OV.SWITCH_CHOSEN_BELOW):
        ctx.specs_select(*d_in, 2.0, t(u), select_rule, score_flags, switch_rule, 0.8, chosen, wts, flag)
        torch.cuda.synchronize()
        got_c = chosen.cpu().numpy()
        sure = (margin > MARGIN) | (select_rule == OV.SELECT_BEST_REWARD)   # the reward comparison is exact
        assert np.array_equal(got_c[sure], want_c[sure])
        assert np.array_equal(got_c == -1, want_c == -1)
        assert np.abs(wts.cpu().numpy() - want_w).max() < 1e-6
        # flags follow the oracle given the GPU's own pick (they coincide wherever the pick is sure)
        assert np.array_equal(flag.cpu().numpy(), OV.switch_flags(r, cand, got_c, 0.8, switch_rule))
    if masked:
        picked = cand[:-1][got_c >= 0] + got_c[got_c >= 0]
        assert mask[picked].all() and got_c[10] == -1


def test_select_rejects_unknown_rules(ctx):
    dev = "cuda:0"
    r = torch.zeros(4, dtype=torch.float32, device=dev)
    cand = torch.tensor([0, 4], dtype=torch.int32, device=dev)
    chosen = torch.zeros(1, dtype=torch.int32, device=dev)
    for args in ((2, 0, 0), (0, 2, 0), (0, 0, 3)):
        with pytest.raises(binding.SpecsError) as e:
            ctx.specs_select(None, None, r, None, cand, 1.0, r, args[0], args[1], args[2], 0.5, chosen)
        assert e.value.status == 2
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_select(None, None, r, None, cand, 1.0, None, OV.SELECT_SUBSAMPLE, 0, 0, 0.5, chosen)
    assert e.value.status == 1                                      # Algorithm 2 needs its uniforms
    ctx.specs_select(None, None, r, None, cand, 1.0, None, OV.SELECT_BEST_REWARD, 0, 0, 0.5, chosen)
    torch.cuda.synchronize()
    assert chosen.item() == 0                                       # all rewards equal: lowest index


def test_specs_loop_with_stub_generators(ctx):
    # Algorithm 1 end to end for a few steps: the native controller decides who drafts, stub generators
    # (seeded random blocks and hidden states, a higher reward level for the target's blocks) stand in
    # for the models, the CUDA path scores and selects; the oracle runs the same loop on the CPU.
    P, n, d, Vv = 3, 4, 64, 500
    got_ctl = binding.Controller(P, binding.POLICY_SPECS, target_len=60)
    want_ctl = OV.Controller(P, OV.POLICY_SPECS, target_len=60)
    w_cfg = small_config("loop_w", (1, 1), 1, 1, d, Vv, seed=5500)
    w_bits = I.make_step_inputs(w_cfg).w_vocab
    trace_got, trace_want = [], []
    for step in range(8):
        gens = got_ctl.generators()
        assert gens.tolist() == want_ctl.generators()
        live = [p for p in range(P) if gens[p] != binding.GEN_DONE]
        if not live:
            break
        cfg = small_config("loop", (4, 12), len(live), n, d, Vv, seed=5510 + step)
        x = I.make_step_inputs(cfg)
        x.w_vocab = w_bits                                          # the same LM head at every step
        for j, p in enumerate(live):                                # the target's candidates score higher
            if gens[p] == binding.GEN_TARGET:
                x.reward[j * n:(j + 1) * n] = np.float32(0.5) + x.reward[j * n:(j + 1) * n] / 2
            else:
                x.reward[j * n:(j + 1) * n] /= 2
        s = DeviceStep(ctx, x)
        ctx.specs_beam_step(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.8, s.tok_lp, s.blk_lp64, s.gen_blk64, s.weights, s.chosen, s.accept,
                            s.workspace)
        torch.cuda.synchronize()
        g = s.results()
        ref = oracle_step(x, 1.0, 0.8)
        lens = np.diff(x.block_offsets)
        for ctl, res, trace in ((got_ctl, g, trace_got), (want_ctl, ref, trace_want)):
            chosen = np.full(P, -1, np.int32); flag = np.zeros(P, np.uint8); clen = np.zeros(P, np.int64)
            for j, p in enumerate(live):
                chosen[p] = res["chosen"][j]; flag[p] = res["accept"][j]
                clen[p] = lens[j * n + res["chosen"][j]]
            ctl.advance(chosen, flag, clen)
            trace.append((chosen.tolist(), flag.tolist()))
        if np.all(ref["margin"] > MARGIN + 1e-2):
            assert trace_got[-1] == trace_want[-1]
        else:                                                       # an unsure pick: keep both loops on one path
            want_ctl.length, want_ctl.steps = got_ctl.stats()["length"].tolist(), got_ctl.stats()["steps"].tolist()
            want_ctl.target_steps = got_ctl.stats()["target_steps"].tolist()
    st = got_ctl.stats()
    assert st["steps"].sum() >= P and (st["target_steps"] >= 1).all()   # every problem began with the target
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- both LM heads, and the append

def test_dual_head_step_and_gather_match_the_oracle(ctx):
    # the same drafted tokens scored with a small generator-shaped head and a larger target-shaped head
    P, n, V_ = 5, 4, 2500
    cfg_t = small_config("dual_t", (3, 70), P, n, 256, V_, seed=5600)
    cfg_g = small_config("dual_g", (3, 70), P, n, 128, V_, seed=5600, w_sigma=0.07, weights_salt=1)
    xt, xg = I.make_step_inputs(cfg_t), I.make_step_inputs(cfg_g)
    assert np.array_equal(xt.block_offsets, xg.block_offsets) and np.array_equal(xt.token_ids, xg.token_ids)
    xt.cand_offsets = np.array([0, 4, 8, 8, 12, 20], dtype=np.int32)                      # one empty problem
    dev = "cuda:0"
    s = DeviceStep(ctx, xt)
    h_g, w_g = binding.bf16_bits_to_device(xg.hidden, dev), binding.bf16_bits_to_device(xg.w_vocab, dev)
    gen_tok = torch.full((xt.rows,), float("nan"), dtype=torch.float32, device=dev)
    stride = 72
    ids_out = torch.full((P, stride), -9, dtype=torch.int32, device=dev)
    len_out = torch.full((P,), -9, dtype=torch.int32, device=dev)
    ws = torch.empty(ctx.beam_step_dual_workspace_bytes(xt.rows, 256, 128, V_), dtype=torch.uint8, device=dev)
    ctx.specs_beam_step_dual(s.hidden, s.w_vocab, h_g, w_g, s.token_ids, s.block_offsets, s.cand_offsets, s.reward,
                             s.uniforms, 1.0, 0.6, s.tok_lp, gen_tok, s.blk_lp64, s.gen_blk64, s.weights, s.chosen,
                             s.accept, ws, ids_out, len_out)
    torch.cuda.synchronize()
    got = s.results()
    got["blk_logprob"] = got["blk_logprob_f64"].astype(np.float32)
    want = OV.beam_step_dual(xt.hidden, xt.w_vocab, xg.hidden, xg.w_vocab, xt.token_ids, xt.block_offsets,
                             xt.cand_offsets, xt.reward, 1.0, xt.uniforms, 0.6)
    assert_step_matches(got, want, xt.cand_offsets, xt.block_offsets)
    g_tok = gen_tok.cpu().numpy()
    assert np.abs(g_tok - want["gen_tok_logprob"]).max() <= TOK_ATOL
    assert np.abs((got["tok_logprob"] - g_tok) - want["tok_logratio"]).max() <= 2 * TOK_ATOL   # per-token log-ratio
    rel = np.abs(got["blk_logprob_gen"] - want["blk_logprob_gen"]) / np.abs(want["blk_logprob_gen"])
    assert rel.max() <= BLK_RTOL
    # the append: ids and length of the block the GPU selected, bit-exact against the definition
    want_ids, want_len = OV.gather_chosen(xt.token_ids, xt.block_offsets, xt.cand_offsets, got["chosen"], stride)
    assert np.array_equal(ids_out.cpu().numpy(), want_ids) and np.array_equal(len_out.cpu().numpy(), want_len)
    assert got["chosen"][2] == -1 and want_len[2] == 0
    # the stand-alone gather gives the same
    ids2 = torch.full((P, stride), -9, dtype=torch.int32, device=dev)
    len2 = torch.full((P,), -9, dtype=torch.int32, device=dev)
    ctx.specs_gather_chosen(s.token_ids, s.block_offsets, s.cand_offsets, s.chosen, ids2, len2)
    torch.cuda.synchronize()
    assert torch.equal(ids2, ids_out) and torch.equal(len2, len_out)
    # and the two-head step equals the one-head step fed with the generator's log-probs it computed
    s2 = DeviceStep(ctx, xt)
    ctx.specs_beam_step(s2.hidden, s2.w_vocab, s2.token_ids, s2.block_offsets, s2.cand_offsets, gen_tok, s2.reward,
                        s2.uniforms, 1.0, 0.6, s2.tok_lp, s2.blk_lp64, s2.gen_blk64, s2.weights, s2.chosen, s2.accept,
                        s2.workspace)
    torch.cuda.synchronize()
    one = s2.results()
    for key in ("tok_logprob", "blk_logprob_f64", "blk_logprob_gen", "weights", "chosen", "accept"):
        assert np.array_equal(one[key], got[key]), key
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- PRM head

def test_prm_head_matches_the_oracle_and_overlaps_with_scoring(ctx):
    cfg = small_config("prm", (0, 60), 6, 8, 3584, 520, seed=5700)   # blocks of 0..60 tokens, some empty
    x = I.make_step_inputs(cfg)
    assert (np.diff(x.block_offsets) == 0).any()
    rng = np.random.Generator(np.random.Philox(key=[5701, 1]))
    w_head = I.f32_to_bf16_bits((rng.normal(0, 0.03, 3584)).astype(np.float32))
    dev = "cuda:0"
    s = DeviceStep(ctx, x)
    w_dev = binding.bf16_bits_to_device(w_head.reshape(1, -1), dev).reshape(-1)
    reward = torch.full((x.blocks,), -3.0, dtype=torch.float32, device=dev)
    # the paper evaluates the PRM concurrently with the target's log-likelihoods: second stream
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ctx.specs_prm_rewards(s.hidden, s.block_offsets, w_dev, -0.4, reward)
    s.score()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    want = OV.prm_rewards(x.hidden, x.block_offsets, w_head, -0.4)
    got = reward.cpu().numpy()
    empty = np.diff(x.block_offsets) == 0
    assert np.isnan(got[empty]).all() and np.isnan(want[empty]).all()
    assert np.abs(got[~empty] - want[~empty]).max() < 2e-6           # fp32 dot over 3584 terms, fp32 output
    assert want[~empty].min() > 0.01 and want[~empty].max() < 0.99 and np.ptp(want[~empty]) > 0.3
    # scoring on the main stream was not disturbed
    assert np.abs(s.tok_lp.cpu().numpy() - O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)).max() <= TOK_ATOL
    # argument checks
    with pytest.raises(binding.SpecsError) as e:
        ctx.specs_prm_rewards(s.hidden[:, :12], s.block_offsets, w_dev, 0.0, reward)
    assert e.value.status == 2
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- vocabulary shards

@pytest.mark.parametrize("world", [1, 3])
def test_vocab_sharded_scoring_matches_oracle_and_single_gpu_path(ctx, world):
    # the ranks' kernels emulated one after the other on this GPU; the exchange itself is tested under gloo
    from paper_2506_15733_b200 import vocab_parallel as VP
    cfg = small_config("shards", (5, 40), 2, 5, 192, 5000, seed=5800)      # 19.5 vocabulary tiles: ragged last shard
    x = I.make_step_inputs(cfg)
    x.token_ids = x.token_ids.copy()
    x.token_ids[7] = 5000                                                   # not in any shard
    dev = "cuda:0"
    s = DeviceStep(ctx, x)
    parts, bounds = [], []
    for rank in range(world):
        v0, v1 = VP.shard_bounds(5000, world, rank)
        bounds.append((v0, v1))
        w_shard = s.w_vocab[v0:v1]
        local = torch.full((x.rows, 4), float("nan"), dtype=torch.float32, device=dev)
        ws = torch.empty(ctx.score_workspace_bytes(x.rows, 192, v1 - v0), dtype=torch.uint8, device=dev)
        ctx.specs_score_partials(s.hidden, w_shard, s.token_ids, v0, local, ws)
        parts.append(local)
    assert bounds[0][0] == 0 and bounds[-1][1] == 5000 and all(a[1] == b[0] for a, b in zip(bounds, bounds[1:]))
    allp = torch.stack(parts)
    out = torch.full((x.rows,), 7.0, dtype=torch.float32, device=dev)
    ctx.specs_merge_partials(allp, s.token_ids, 5000, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    assert np.isnan(got[7]) and np.isnan(want[7])
    ok = np.arange(x.rows) != 7
    assert np.abs(got[ok] - want[ok]).max() <= TOK_ATOL
    assert ctx.device_status() == binding.DEV_TOKEN_RANGE
    # each shard's partials against the oracle's (natural units there, base-2 units here)
    p_np = allp.cpu().numpy().astype(np.float64)
    for rank, (v0, v1) in enumerate(bounds):
        ref = OV.shard_partials(x.hidden, x.w_vocab, x.token_ids, v0, v1)
        lse_ref = ref[:, 0] + np.log(ref[:, 1])
        lse_got = (p_np[rank, :, 0] + np.log2(p_np[rank, :, 1])) * math.log(2.0)
        assert np.abs(lse_got - lse_ref).max() <= TOK_ATOL
        held = np.isfinite(ref[:, 2])
        assert np.array_equal(np.isfinite(p_np[rank, :, 2]), held)
        assert np.abs(p_np[rank, held, 2] - ref[held, 2]).max() <= TOK_ATOL
    # and the unsharded path
    s.score()
    torch.cuda.synchronize()
    assert np.abs(s.tok_lp.cpu().numpy()[ok] - got[ok]).max() <= 1e-5
    ctx.device_status()


# ------------------------------------------------------------------------------- pacing is advisory

@pytest.mark.parametrize("lead", [0, 1, 3])
def test_pacing_never_changes_results_even_on_a_garbage_workspace(ctx, lead):
    # several waves and several units per vocabulary chunk, so that the pacing path really runs; the workspace
    # starts as random bytes (progress words of "another launch", some looking far ahead): only time may be lost
    cfg = small_config("pace", (250, 250), 4, 10, 128, 2600, seed=5900, w_sigma=0.1)
    x = I.make_step_inputs(cfg)
    plan = binding.score_plan(x.rows, 128, 2600, ctx.sm_count())
    assert plan["waves"] >= 2 and plan["group_m"] > 1
    want = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    s = DeviceStep(ctx, x)
    ctx.set_tile_lead(lead)
    try:
        for fill in ("random", "ones"):
            if fill == "random":
                g = torch.Generator(device="cuda:0"); g.manual_seed(5901)
                s.workspace.copy_(torch.randint(0, 256, s.workspace.shape, generator=g, device="cuda:0",
                                                dtype=torch.uint8))
            else:
                s.workspace.fill_(0xff)
            s.tok_lp.fill_(float("nan"))
            s.score()
            torch.cuda.synchronize()
            assert np.abs(s.tok_lp.cpu().numpy() - want).max() <= TOK_ATOL
    finally:
        ctx.set_tile_lead(1)
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- bounded waits

def test_a_wait_that_nothing_completes_expires_and_is_reported(ctx):
    import time
    t0 = time.perf_counter()
    ctx.probe_wait_expiry(2000)                                   # 2 ms on a barrier nobody arrives at
    with pytest.raises(binding.SpecsError) as e:
        ctx.device_status(raise_on_error=True)                    # synchronises: the kernel did return
    assert e.value.status == 8                                    # SPECS_ERR_DEVICE_TIMEOUT
    assert time.perf_counter() - t0 < 5.0
    assert ctx.device_status() == 0                               # reading cleared the word
    # the context is as usable as before
    x = I.make_step_inputs(I.CONFIGS["tiny"])
    got = DeviceStep(ctx, x).step(1.0, 0.7)
    assert_step_matches(got, oracle_step(x, 1.0, 0.7), x.cand_offsets, x.block_offsets)
    assert ctx.device_status() == 0
    with pytest.raises(binding.SpecsError) as e:
        ctx.probe_wait_expiry(0)
    assert e.value.status == 2


# ------------------------------------------------------------------------------- nothing is written out of bounds

class _Guarded:
    """A device buffer with 4 KB of a known byte pattern on both sides."""
    PAD = 4096

    def __init__(self, nbytes, dtype, dev="cuda:0"):
        self.nbytes = int(nbytes)
        aligned = (self.nbytes + 255) // 256 * 256
        self.raw = torch.full((self.PAD + aligned + self.PAD,), 0xA5, dtype=torch.uint8, device=dev)
        self.view = self.raw[self.PAD:self.PAD + self.nbytes].view(dtype)

    def intact(self):
        tail = self.raw[self.PAD + self.nbytes:]
        return bool((self.raw[:self.PAD] == 0xA5).all()) and bool((tail == 0xA5).all())


@pytest.mark.parametrize("engine", TC_ENGINES)
@pytest.mark.parametrize("blk,P,n,d,V", [((1, 1), 1, 1, 8, 8), ((3, 40), 3, 5, 256, 2500), ((129, 129), 1, 1, 64, 1032),
                                         ((250, 250), 4, 10, 128, 2600)])
def test_outputs_and_workspace_stay_inside_their_buffers(ctx, engine, blk, P, n, d, V):
    cfg = small_config("guard", blk, P, n, d, V, seed=6000 + d + V)
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    rows, B = x.rows, x.blocks
    g = {"tok": _Guarded(rows * 4, torch.float32), "blk": _Guarded(B * 8, torch.float64),
         "gen": _Guarded(B * 8, torch.float64), "wts": _Guarded(B * 4, torch.float32),
         "cho": _Guarded(P * 4, torch.int32), "acc": _Guarded(P, torch.uint8),
         "ws": _Guarded(ctx.score_workspace_bytes(rows, d, V), torch.uint8),
         "ids": _Guarded(P * 130 * 4, torch.int32), "len": _Guarded(P * 4, torch.int32)}
    ctx.set_engine(engine)
    try:
        ctx.specs_beam_step(s.hidden, s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets, s.draft, s.reward,
                            s.uniforms, 1.0, 0.5, g["tok"].view, g["blk"].view, g["gen"].view, g["wts"].view,
                            g["cho"].view, g["acc"].view, g["ws"].view)
        ctx.specs_gather_chosen(s.token_ids, s.block_offsets, s.cand_offsets, g["cho"].view,
                                g["ids"].view.view(P, 130), g["len"].view)
        torch.cuda.synchronize()
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    for name, buf in g.items():
        assert buf.intact(), f"bytes around `{name}` were overwritten"
    want = oracle_step(x, 1.0, 0.5)
    assert np.abs(g["tok"].view.cpu().numpy() - want["tok_logprob"]).max() <= TOK_ATOL
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- seeded random shapes

def _random_shapes(count, seed):
    rng = np.random.Generator(np.random.Philox(key=[seed, 9]))
    out = []
    for _ in range(count):
        d = int(rng.integers(1, 80)) * 8                            # any multiple of 8 up to 632 (k-block tails)
        V = int(rng.integers(1, 3000))
        P = int(rng.integers(1, 6))
        n = int(rng.integers(1, 9))
        hi = int(rng.integers(1, 120))
        lo = int(rng.integers(0, hi + 1))
        out.append((d, V, P, n, lo, hi, int(rng.integers(0, 3))))
    return out


@pytest.mark.parametrize("d,V,P,n,lo,hi,mode", _random_shapes(24, 6100))
def test_random_shapes_against_the_oracle(ctx, d, V, P, n, lo, hi, mode):
    cfg = small_config("fuzz", (lo, hi), P, n, d, V, seed=6100 + d + V, w_sigma=0.6 / math.sqrt(d) * (1 + mode))
    x = I.make_step_inputs(cfg)
    if x.rows == 0:
        pytest.skip("all blocks empty")
    engine = [binding.ENGINE_TCGEN05, binding.ENGINE_TCGEN05_1CTA, binding.ENGINE_TCGEN05_2CTA][mode]
    ctx.set_engine(engine)
    try:
        sep = DeviceStep(ctx, x).step(1.3, 0.6)
        fused = _fused_step(ctx, DeviceStep(ctx, x), 1.3, 0.6)
    finally:
        ctx.set_engine(binding.ENGINE_TCGEN05)
    want = oracle_step(x, 1.3, 0.6)
    assert_step_matches(sep, want, x.cand_offsets, x.block_offsets)
    for key in ("tok_logprob", "blk_logprob_f64", "blk_logprob_gen", "weights", "chosen", "accept"):
        assert np.array_equal(fused[key], sep[key]), key
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------- argument checks of the wider API

def test_argument_checks_of_the_dual_shard_and_gather_calls(ctx):
    cfg = small_config("args2", (4, 4), 1, 2, 64, 300, seed=6200)
    x = I.make_step_inputs(cfg)
    s = DeviceStep(ctx, x)
    dev = "cuda:0"
    gen_tok = torch.empty(x.rows, dtype=torch.float32, device=dev)
    ws = torch.empty(ctx.beam_step_dual_workspace_bytes(x.rows, 64, 64, 300), dtype=torch.uint8, device=dev)

    def status_of(fn):
        with pytest.raises(binding.SpecsError) as e:
            fn()
        return e.value.status

    dual = lambda **kw: ctx.specs_beam_step_dual(
        s.hidden, s.w_vocab, kw.get("h_g", s.hidden), s.w_vocab, s.token_ids, s.block_offsets, s.cand_offsets, s.reward,
        s.uniforms, 1.0, 0.5, s.tok_lp, kw.get("gen_tok", gen_tok), s.blk_lp64, s.gen_blk64, s.weights, s.chosen,
        s.accept, kw.get("ws", ws))
    assert status_of(lambda: dual(gen_tok=None)) == 1             # the generator's log-probs are an output here
    assert status_of(lambda: dual(ws=ws[:64])) == 4
    assert status_of(lambda: dual(h_g=s.hidden[:, :12])) == 2     # d_gen % 8 != 0
    part = torch.empty((x.rows, 4), dtype=torch.float32, device=dev)
    assert status_of(lambda: ctx.specs_score_partials(s.hidden, s.w_vocab, s.token_ids, -1, part, s.workspace)) == 2
    assert status_of(lambda: ctx.specs_score_partials(s.hidden, s.w_vocab, None, 0, part, s.workspace)) == 1
    assert status_of(lambda: ctx.specs_merge_partials(part.view(1, x.rows, 4)[:0], s.token_ids, 300, s.tok_lp)) == 2
    ids_out = torch.empty((1, 8), dtype=torch.int32, device=dev)
    len_out = torch.empty(1, dtype=torch.int32, device=dev)
    assert status_of(lambda: ctx.specs_gather_chosen(s.token_ids, s.block_offsets, s.cand_offsets, s.chosen,
                                                     ids_out[:, :0], len_out)) == 2
    assert status_of(lambda: ctx.specs_gather_chosen(s.token_ids, s.block_offsets, s.cand_offsets, None,
                                                     ids_out, len_out)) == 1
    torch.cuda.synchronize()
    assert torch.isnan(s.tok_lp).all() and ctx.device_status() == 0     # nothing was launched


def test_run_specs_helper_follows_the_controller(ctx):
    # the packaged loop (controller + fused step + gather) with a stub generator that records what it was asked
    from paper_2506_15733_b200 import loop as LP
    P, n, d, Vv = 3, 4, 64, 500
    w_bits = I.make_step_inputs(small_config("loop_w", (1, 1), 1, 1, d, Vv, seed=5500)).w_vocab
    w_dev = binding.bf16_bits_to_device(w_bits, "cuda:0")
    asked, batches = [], []

    def draft_fn(gens, live):
        asked.append(gens.copy())
        x = I.make_step_inputs(small_config("loop", (4, 12), len(live), n, d, Vv, seed=6300 + len(asked)))
        x.w_vocab = w_bits                                 # the same LM head at every step
        for j, p in enumerate(live):                       # the target's candidates earn higher rewards
            sl = slice(j * n, (j + 1) * n)
            x.reward[sl] = np.float32(0.5) + x.reward[sl] / 2 if gens[p] == binding.GEN_TARGET else x.reward[sl] / 2
        s = DeviceStep(ctx, x)
        batches.append((x, live.copy()))
        return LP.DraftBatch(s.hidden, s.token_ids, s.block_offsets, s.cand_offsets, s.reward, s.uniforms, s.draft)

    ctl = binding.Controller(P, binding.POLICY_SPECS, target_len=40)
    res = LP.run_specs(ctx, ctl, draft_fn, w_dev, 1.0, 0.8, max_block_len=16, max_iters=50)
    assert (ctl.generators() == binding.GEN_DONE).all()
    assert all(g[0] == binding.GEN_TARGET for g in res.generators)          # Algorithm 1 begins with the target
    assert [len(t) for t in res.traces] == res.stats["length"].tolist() and min(res.stats["length"]) >= 40
    # every appended token is one of the drafted ids of that step, in block order
    pos = [0] * P
    for (x, live), gens in zip(batches, asked):
        ref = oracle_step(x, 1.0, 0.8)
        for j, p in enumerate(live):
            a = int(x.cand_offsets[j])
            lens = np.diff(x.block_offsets)[a:a + n]
            took = res.traces[p][pos[p]:]
            match = [c for c in range(n) if took[:lens[c]] == x.token_ids[x.block_offsets[a + c]:x.block_offsets[a + c + 1]].tolist()]
            assert match, "the appended tokens are not one of the candidates"
            if ref["margin"][j] > MARGIN + 1e-2:
                assert int(ref["chosen"][j]) in match
            pos[p] += int(lens[match[0]]) if int(ref["chosen"][j]) not in match else int(lens[int(ref["chosen"][j])])
    assert ctx.device_status() == 0


@pytest.mark.parametrize("policy,select_rule", [(binding.POLICY_RSD, None), (binding.POLICY_DRAFT_START, None),
                                                (binding.POLICY_RANDOM, None),
                                                (binding.POLICY_ONLY_DRAFT, binding.SELECT_BEST_REWARD)])
def test_run_specs_dispatches_every_policy_like_the_oracle_loop(ctx, policy, select_rule):
    # The packaged loop under the policies of the baselines and ablations, replayed on the CPU with the
    # oracle's selection, switch rules and controller.  Rewards are spaced by 0.04 and beta is large, so
    # every pick is decided by a wide margin and both loops must agree step by step.
    from paper_2506_15733_b200 import loop as LP
    P, n, d, Vv, beta, tau = 3, 4, 64, 500, 1000.0, 0.6
    w_bits = I.make_step_inputs(small_config("loop_w", (1, 1), 1, 1, d, Vv, seed=5500)).w_vocab
    w_dev = binding.bf16_bits_to_device(w_bits, "cuda:0")
    asked, batches = [], []

    def draft_fn(gens, live):
        step = len(asked)
        asked.append(gens.copy())
        x = I.make_step_inputs(small_config("loop", (4, 12), len(live), n, d, Vv, seed=6400 + 10 * policy + step))
        x.w_vocab = w_bits
        perm = np.random.Generator(np.random.Philox(key=[6450, step])).permutation(n)
        for j, p in enumerate(live):
            lo = 0.62 if gens[p] == binding.GEN_TARGET else (0.40 if (step + p) % 2 else 0.55)
            x.reward[j * n:(j + 1) * n] = (lo + 0.04 * perm).astype(np.float32)
        s = DeviceStep(ctx, x)
        batches.append((x, live.copy()))
        return LP.DraftBatch(s.hidden, s.token_ids, s.block_offsets, s.cand_offsets, s.reward, s.uniforms, s.draft)

    uni = lambda it: I.draw_uniforms(7000 + it, P)
    ctl = binding.Controller(P, policy, target_len=40, p_target=0.5)
    res = LP.run_specs(ctx, ctl, draft_fn, w_dev, beta, tau, max_block_len=16, max_iters=60,
                       select_rule=select_rule, switch_uniforms=uni if policy == binding.POLICY_RANDOM else None)
    assert (ctl.generators() == binding.GEN_DONE).all()

    rule = OV.SELECT_BEST_REWARD if policy == binding.POLICY_RSD or select_rule == binding.SELECT_BEST_REWARD \
        else OV.SELECT_SUBSAMPLE
    switch = {binding.POLICY_DRAFT_START: OV.SWITCH_NONE_ABOVE, binding.POLICY_RSD: OV.SWITCH_CHOSEN_BELOW}.get(
        policy, OV.SWITCH_ANY_ABOVE)
    want_ctl = OV.Controller(P, policy, target_len=40, p_target=0.5)
    want_traces = [[] for _ in range(P)]
    for it, ((x, live), gens) in enumerate(zip(batches, asked)):
        assert gens.tolist() == want_ctl.generators()
        LP_t = O.block_sums(O.token_logprobs(x.hidden, x.w_vocab, x.token_ids), x.block_offsets)
        LQ = O.block_sums(x.draft_tok_logprob, x.block_offsets)
        c, w, margin = OV.select(LP_t, LQ, x.reward, None, x.cand_offsets, beta, x.uniforms, rule)
        assert np.all(margin > (0.03 if rule == OV.SELECT_BEST_REWARD else 1.0))   # rewards 0.04 apart; beta * 0.04 = 40
        f = OV.switch_flags(x.reward, x.cand_offsets, c, tau, switch)
        chosen = np.full(P, -1, np.int32); flag = np.zeros(P, np.uint8); clen = np.zeros(P, np.int64)
        for j, p in enumerate(live):
            a = int(x.cand_offsets[j]) + int(c[j])
            chosen[p], flag[p] = c[j], f[j]
            clen[p] = x.block_offsets[a + 1] - x.block_offsets[a]
        before = list(want_ctl.steps)
        want_ctl.advance(chosen, flag, clen, uni(it))
        for j, p in enumerate(live):
            if want_ctl.steps[p] != before[p]:
                a = int(x.cand_offsets[j]) + int(c[j])
                want_traces[p].extend(x.token_ids[x.block_offsets[a]:x.block_offsets[a + 1]].tolist())
    assert res.traces == want_traces
    st = ctl.stats()
    assert st["length"].tolist() == want_ctl.length == [len(t) for t in res.traces]
    assert st["steps"].tolist() == want_ctl.steps and st["target_calls"].tolist() == want_ctl.target_calls
    if policy == binding.POLICY_RSD:
        assert sum(st["target_calls"]) > 0 and sum(st["target_steps"]) < sum(st["steps"])   # both routes were taken
    assert ctx.device_status() == 0

