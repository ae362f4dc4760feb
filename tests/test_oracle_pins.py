"""Pins for the CPU oracle: closed forms, brute force, big-float evaluation and
statistical laws that the paper and the mathematics fix.  No GPU, no product code.

Each test is chosen so that a plausible slip in the oracle (a transposed operand,
a dropped term, a wrong sign, an off-by-one in an offset) makes it fail.
"""
import itertools
import math
import os
from fractions import Fraction

import mpmath
import numpy as np
import pytest
from scipy import integrate, stats

from oracle import specs_oracle as O
from paper_2506_15733_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_bf16(rng, shape, sigma):
    return bits(rng.standard_normal(shape).astype(np.float32) * sigma)


# ------------------------------------------------------------------ O1/O2: log-softmax of the LM head

def test_bf16_decode_is_exact():
    # a few hand-written patterns: 1.0, -2.0, 0.5, 3.140625 (0x4049), smallest normal, zero
    pat = np.array([0x3F80, 0xC000, 0x3F00, 0x4049, 0x0080, 0x0000], dtype=np.uint16)
    want = [1.0, -2.0, 0.5, 3.140625, 2.0 ** -126, 0.0]
    assert O.bf16_bits_to_f64(pat).tolist() == want


def test_probabilities_of_a_row_sum_to_one():
    rng = np.random.default_rng(1)
    V, d = 37, 24
    H, W = rand_bf16(rng, (3, d), 1.0), rand_bf16(rng, (V, d), 0.3)
    for t in range(3):
        # score the same row V times, once per possible drafted id
        lp = O.token_logprobs(np.repeat(H[t:t + 1], V, axis=0), W, np.arange(V))
        assert abs(np.exp(lp).sum() - 1.0) < 1e-12
        assert np.all(lp < 0)


def test_zero_hidden_row_gives_uniform():
    rng = np.random.default_rng(2)
    for V in (1024, 151936):
        d = 8
        W = rand_bf16(rng, (V, d), 1.0)
        lp = O.token_logprobs(np.zeros((2, d), np.uint16), W, np.array([0, V - 1]))
        assert np.allclose(lp, -math.log(V), atol=1e-12)
    assert abs(-math.log(1024) - (-6.931471805599453)) < 1e-15
    assert abs(-math.log(151936) - (-11.931214)) < 1e-5


def test_identical_vocab_rows_give_uniform():
    rng = np.random.default_rng(3)
    V, d = 50, 16
    w = rand_bf16(rng, (1, d), 1.0)
    lp = O.token_logprobs(rand_bf16(rng, (4, d), 1.0), np.repeat(w, V, axis=0), np.array([0, 7, 20, 49]))
    assert np.allclose(lp, -math.log(V), atol=1e-12)


def test_one_hot_closed_form_catches_transposition():
    # W = alpha * [I 0] (V x d with d >= V), h = c * e_j: logit_j = alpha*c, every other logit 0.
    V, d, alpha, c = 12, 16, 0.5, 3.0           # all exact in bf16
    W = np.zeros((V, d), np.float32)
    W[np.arange(V), np.arange(V)] = alpha
    for j in (0, 5, 11):
        h = np.zeros((1, d), np.float32)
        h[0, j] = c
        denom = math.log(math.exp(alpha * c) + V - 1)
        lp_j = O.token_logprobs(bits(h), bits(W), np.array([j]))[0]
        lp_o = O.token_logprobs(bits(h), bits(W), np.array([(j + 1) % V]))[0]
        assert abs(lp_j - (alpha * c - denom)) < 1e-13
        assert abs(lp_o - (-denom)) < 1e-13
    # a non-symmetric W: row v has a single entry at column (v + 3) % d, so W @ h != W.T @ h
    W2 = np.zeros((V, d), np.float32)
    W2[np.arange(V), (np.arange(V) + 3) % d] = alpha
    h = np.zeros((1, d), np.float32)
    h[0, 7] = c                                   # lights up vocabulary entry v = 4 only
    lp = O.token_logprobs(np.repeat(bits(h), V, axis=0), bits(W2), np.arange(V))
    assert int(np.argmax(lp)) == 4
    assert abs(lp[4] - (alpha * c - math.log(math.exp(alpha * c) + V - 1))) < 1e-13


def test_shift_invariance_constant_column():
    rng = np.random.default_rng(4)
    V, d = 40, 16
    H, W = rand_bf16(rng, (5, d), 1.0), rand_bf16(rng, (V, d), 0.5)
    ids = rng.integers(0, V, 5)
    base = O.token_logprobs(H, W, ids)
    H2 = np.concatenate([H, bits(np.ones((5, 1)))], axis=1)
    W2 = np.concatenate([W, bits(np.full((V, 1), 2.5))], axis=1)
    assert np.allclose(O.token_logprobs(H2, W2, ids), base, atol=1e-12)


def test_large_logits_agree_with_bigfloat():
    # scale hidden by 2^k until logits reach about +-1e3: a naive exp would overflow
    rng = np.random.default_rng(5)
    V, d = 8, 4
    Hf = I.bf16_bits_to_f32(rand_bf16(rng, (4, d), 1.0))
    Wb = rand_bf16(rng, (V, d), 1.0)
    Wf = I.bf16_bits_to_f32(Wb)
    mpmath.mp.dps = 60
    for k in (0, 4, 8, 10):
        Hk = Hf * np.float32(2.0 ** k)
        ids = np.array([0, 3, 5, 7])
        got = O.token_logprobs(bits(Hk), Wb, ids)
        assert np.all(np.isfinite(got))
        for t in range(4):
            z = [sum(mpmath.mpf(float(Hk[t, q])) * mpmath.mpf(float(Wf[v, q])) for q in range(d)) for v in range(V)]
            want = z[int(ids[t])] - mpmath.log(sum(mpmath.exp(x) for x in z))
            assert abs(got[t] - float(want)) <= 1e-12 * max(1.0, abs(float(want)))
    assert np.abs(I.bf16_bits_to_f32(bits(Hf * np.float32(1024.0))) @ Wf.T).max() > 700


def test_against_library_log_softmax():
    # a textbook routine the special case reduces to (scipy's log_softmax in fp64)
    from scipy.special import log_softmax
    x = I.make_step_inputs(I.CONFIGS["tiny"])
    got = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    Z = I.bf16_bits_to_f32(x.hidden).astype(np.float64) @ I.bf16_bits_to_f32(x.w_vocab).astype(np.float64).T
    want = log_softmax(Z, axis=1)[np.arange(x.rows), x.token_ids]
    assert np.allclose(got, want, atol=1e-11)


def test_out_of_range_token_is_nan():
    rng = np.random.default_rng(6)
    H, W = rand_bf16(rng, (3, 8), 1.0), rand_bf16(rng, (5, 8), 1.0)
    lp = O.token_logprobs(H, W, np.array([0, 5, -1]))
    assert np.isfinite(lp[0]) and np.isnan(lp[1]) and np.isnan(lp[2])


def test_row_chunking_does_not_change_results():
    rng = np.random.default_rng(7)
    H, W = rand_bf16(rng, (11, 16), 1.0), rand_bf16(rng, (33, 16), 0.4)
    ids = rng.integers(0, 33, 11)
    a = O.token_logprobs(H, W, ids, row_chunk=1)
    b = O.token_logprobs(H, W, ids, row_chunk=4)
    c = O.token_logprobs(H, W, ids, row_chunk=64)
    assert np.allclose(a, b, atol=1e-13) and np.allclose(a, c, atol=1e-13)


# ------------------------------------------------------------------ whole path by brute force, exact arithmetic

@pytest.mark.parametrize("V,d,rows", [(2, 8, 4), (3, 8, 6), (8, 16, 8)])
def test_brute_force_exact_rational(V, d, rows):
    rng = np.random.default_rng(100 + V)
    Hb, Wb = rand_bf16(rng, (rows, d), 1.0), rand_bf16(rng, (V, d), 0.7)
    ids = rng.integers(0, V, rows)
    offs = np.array([0, 1, rows // 2, rows // 2, rows], dtype=np.int64)    # includes an empty block
    cand = np.array([0, 2, 4], dtype=np.int32)
    draft = rng.uniform(-3, 0, rows).astype(np.float32)
    r = rng.uniform(0, 1, 4).astype(np.float32)
    u = I.draw_uniforms(77 + V, 4)
    beta, tau = 1.5, 0.6
    out = O.beam_step(Hb, Wb, ids, offs, cand, draft, r, beta, u, tau)

    mpmath.mp.dps = 50
    Hq = [[Fraction(float(v)) for v in row] for row in I.bf16_bits_to_f32(Hb)]
    Wq = [[Fraction(float(v)) for v in row] for row in I.bf16_bits_to_f32(Wb)]

    def mp(fr):
        return mpmath.mpf(fr.numerator) / mpmath.mpf(fr.denominator)

    tok = []
    for t in range(rows):
        z = [mp(sum(Hq[t][k] * Wq[v][k] for k in range(d))) for v in range(V)]   # exact rationals
        tok.append(z[int(ids[t])] - mpmath.log(sum(mpmath.exp(x) for x in z)))
    assert max(abs(float(tok[t]) - out["tok_logprob"][t]) for t in range(rows)) < 1e-12
    LP = [sum(tok[offs[i]:offs[i + 1]], mpmath.mpf(0)) for i in range(4)]
    LQ = [sum((mpmath.mpf(float(x)) for x in draft[offs[i]:offs[i + 1]]), mpmath.mpf(0)) for i in range(4)]
    assert LP[2] == 0 and out["blk_logprob"][2] == 0.0
    S = [LP[i] - LQ[i] + mpmath.mpf(float(np.float32(beta))) * mpmath.mpf(float(r[i])) for i in range(4)]
    for p in range(2):
        a, b = cand[p], cand[p + 1]
        Zp = sum(mpmath.exp(S[i]) for i in range(a, b))
        for i in range(a, b):
            assert abs(float(mpmath.exp(S[i]) / Zp) - out["weights"][i]) < 1e-12
        pert = [S[i] - mpmath.log(-mpmath.log(mpmath.mpf(float(u[i])))) for i in range(a, b)]
        assert int(np.argmax([float(x) for x in pert])) == out["chosen"][p]
        assert abs(float(abs(pert[0] - pert[1])) - out["margin"][p]) < 1e-10
        assert out["accept"][p] == (1 if max(float(r[i]) for i in range(a, b)) > float(np.float32(tau)) else 0)


# ------------------------------------------------------------------ O3: block sums

def test_block_sum_properties():
    rng = np.random.default_rng(8)
    x = rng.uniform(-9, 0, 40)
    offs = np.array([0, 5, 5, 6, 40], dtype=np.int64)
    s = O.block_sums(x, offs)
    assert s[1] == 0.0                                       # empty block
    assert s[2] == x[5]                                      # single token
    assert abs(s.sum() - x.sum()) < 1e-12
    split = O.block_sums(x, np.array([0, 5, 5, 6, 20, 40], dtype=np.int64))
    assert abs(split[3] + split[4] - s[3]) < 1e-12           # additivity under splitting
    y = x.copy()
    y[6:40] = rng.permutation(y[6:40])
    assert abs(O.block_sums(y, offs)[3] - s[3]) < 1e-12      # order inside a block is irrelevant
    assert abs(s[3] - math.fsum(x[6:40])) < 1e-12            # offsets are half-open [a, b)
    assert abs(s[0] - math.fsum(x[0:5])) < 1e-13


# ------------------------------------------------------------------ O4/O5: scores and weights

def test_weights_basic_laws():
    rng = np.random.default_rng(9)
    LP, LQ, r = rng.uniform(-50, -5, 12), rng.uniform(-50, -5, 12), rng.uniform(0, 1, 12)
    cand = np.array([0, 5, 5, 12], dtype=np.int32)           # middle problem is empty
    S = O.scores(LP, LQ, r, 2.0)
    w = O.weights(S, cand)
    assert abs(w[0:5].sum() - 1) < 1e-12 and abs(w[5:12].sum() - 1) < 1e-12
    S2 = S.copy()
    S2[0:5] += 123.456
    assert np.allclose(O.weights(S2, cand), w, atol=1e-12)   # constant shift inside a problem
    assert np.allclose(S, LP - LQ + 2.0 * r, atol=1e-12)     # sign of the ratio, place of beta
    # raising only the target log-prob of one candidate raises its weight; raising its draft log-prob lowers it
    LP2 = LP.copy(); LP2[1] += 1.0
    LQ2 = LQ.copy(); LQ2[1] += 1.0
    assert O.weights(O.scores(LP2, LQ, r, 2.0), cand)[1] > w[1]
    assert O.weights(O.scores(LP, LQ2, r, 2.0), cand)[1] < w[1]


def test_two_candidates_is_a_sigmoid():
    S = np.array([0.3, -1.1])
    w = O.weights(S, np.array([0, 2]))
    assert abs(w[1] - 1 / (1 + math.exp(S[0] - S[1]))) < 1e-14


def test_same_generator_collapses_to_reward_softmax():
    # With pi_gen = pi_target the score is beta * r (text after Eq. 1): weights = softmax(beta r).
    r = np.array([0.1, 0.9, 0.5, 0.5], dtype=np.float32)
    for beta in (0.0, 1.0, 4.0):
        w = O.weights(O.scores(None, None, r, beta), np.array([0, 4]))
        e = np.exp(beta * r.astype(np.float64))
        assert np.allclose(w, e / e.sum(), atol=1e-14)
    assert np.allclose(O.weights(O.scores(None, None, r, 0.0), np.array([0, 4])), 0.25)
    # an identical block log-prob on both sides is the same thing
    lp = np.array([-3.0, -7.0, -1.0, -2.0])
    assert np.allclose(O.scores(lp, lp, r, 3.0), 3.0 * r.astype(np.float64), atol=1e-14)


def test_beta_limits_of_the_selection_rule():
    # pi*_beta is proportional to pi_target * exp(beta r) (Eq. 3): beta = 0 with a draft generator gives
    # importance resampling toward pi_target; beta -> infinity gives hard best-of-n on the reward.
    LP = np.array([-10.0, -12.0, -11.0, -30.0])
    LQ = np.array([-11.0, -11.0, -14.0, -12.0])
    r = np.array([0.2, 0.8, 0.5, 0.9], dtype=np.float32)
    cand = np.array([0, 4])
    w0 = O.weights(O.scores(LP, LQ, r, 0.0), cand)
    ratio = np.exp(LP - LQ)
    assert np.allclose(w0, ratio / ratio.sum(), atol=1e-14)
    winf = O.weights(O.scores(LP, LQ, r, 1.0e4), cand)       # beta = 10^4 appears in the paper's Table 6
    assert winf[3] > 1 - 1e-12                               # argmax r wins despite the worst log-ratio
    # ties in the reward are split by the log-ratio alone
    r_tie = np.array([0.9, 0.1, 0.9, 0.0], dtype=np.float32)
    wt = O.weights(O.scores(LP, LQ, r_tie, 1.0e4), cand)
    assert abs(wt[0] / wt[2] - math.exp((LP[0] - LQ[0]) - (LP[2] - LQ[2]))) < 1e-9
    assert wt[1] < 1e-300 and wt[3] < 1e-300


def test_two_response_instance_pick_law():
    # Two responses with r = (0, R) drawn from pi_gen = pi_target: k copies of y1 among n candidates
    # are picked with probability k*theta / (k*theta + n - k), theta = exp(beta R) (Appendix D instance).
    with open(os.path.join(GOLDEN, "two_response_instance.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for beta, R, n, k in [(float(a), float(b), int(c), int(e)) for a, b, c, e in rows]:
        r = np.array([R] * k + [0.0] * (n - k), dtype=np.float64)
        w = O.weights(O.scores(None, None, r, beta), np.array([0, n]))
        theta = math.exp(float(np.float32(beta)) * R)
        assert abs(w[:k].sum() - k * theta / (k * theta + n - k)) < 1e-12


# ------------------------------------------------------------------ O6: the sampler

def _chi2_pvalue(S, draws, seed):
    n = len(S)
    rng = np.random.Generator(np.random.Philox(key=[seed, 42]))
    k = rng.integers(0, 1 << 23, size=(draws, n))
    u = ((k + 0.5) * 2.0 ** -23).astype(np.float32)
    cand = (np.arange(draws + 1) * n).astype(np.int64)
    chosen, _ = O.gumbel_pick(np.tile(S, draws), u.reshape(-1), cand)
    counts = np.bincount(chosen, minlength=n)
    expected = draws * O.weights(S, np.array([0, n]))
    assert expected.min() >= 5
    return stats.chisquare(counts, expected).pvalue, counts, expected


@pytest.mark.parametrize("beta", [0.0, 1.0, 4.0])
def test_sampler_matches_weights_chi_squared(beta):
    # n = 8 candidates whose weights span roughly 0.02 .. 0.4
    LP = np.array([-20.0, -21.0, -19.5, -22.0, -20.5, -23.0, -19.0, -21.5])
    LQ = np.array([-20.5, -20.0, -20.0, -21.0, -21.5, -22.0, -20.0, -21.0])
    r = np.array([0.1, 0.6, 0.3, 0.9, 0.5, 0.7, 0.2, 0.4], dtype=np.float32)
    S = O.scores(LP, LQ, r, beta)
    p, counts, expected = _chi2_pvalue(S, 200_000, seed=11 + int(beta))
    assert p > 1e-3, (p, counts, expected)


def test_sampler_detects_a_wrong_law():
    # the same test must reject a deliberately wrong law (weights proportional to exp(S/2)), so it has power
    S = np.array([0.0, 1.0, 2.0, 3.0])
    n, draws = 4, 100_000
    rng = np.random.Generator(np.random.Philox(key=[5, 42]))
    u = ((rng.integers(0, 1 << 23, size=(draws, n)) + 0.5) * 2.0 ** -23).astype(np.float32)
    chosen, _ = O.gumbel_pick(np.tile(S, draws), u.reshape(-1), (np.arange(draws + 1) * n))
    counts = np.bincount(chosen, minlength=n)
    wrong = np.exp(S / 2) / np.exp(S / 2).sum()
    assert stats.chisquare(counts, draws * wrong).pvalue < 1e-6
    assert stats.chisquare(counts, draws * O.weights(S, np.array([0, n]))).pvalue > 1e-3


def test_pick_ties_margin_and_validation():
    S = np.array([1.0, 1.0, 1.0])
    u = np.array([0.5, 0.5, 0.5], dtype=np.float32)
    chosen, margin = O.gumbel_pick(S, u, np.array([0, 3]))
    assert chosen[0] == 0 and margin[0] == 0.0               # exact tie: lowest index
    chosen, margin = O.gumbel_pick(np.array([2.0]), u[:1], np.array([0, 0, 1]))
    assert chosen.tolist() == [-1, 0] and np.isinf(margin[1])
    # a larger uniform means a larger Gumbel: with equal scores the largest u wins
    chosen, margin = O.gumbel_pick(np.zeros(3), np.array([0.2, 0.9, 0.6], np.float32), np.array([0, 3]))
    g = lambda v: -math.log(-math.log(float(np.float32(v))))
    assert chosen[0] == 1 and abs(margin[0] - (g(0.9) - g(0.6))) < 1e-12
    with pytest.raises(ValueError):
        O.gumbel_pick(np.zeros(2), np.array([0.0, 0.5]), np.array([0, 2]))
    with pytest.raises(ValueError):
        O.gumbel_pick(np.zeros(2), np.array([0.5, 1.0]), np.array([0, 2]))


def _poissonised_pick_probability(theta, n):
    """Closed form for the two-response instance (Lemma integral-0 specialised in Appendix D):
    theta/(1+theta) * n/(1-e^-n) * int_0^1 exp(n((theta t + t^theta)/(1+theta) - 1)) dt."""
    val, _ = integrate.quad(lambda t: math.exp(n * ((theta * t + t ** theta) / (1 + theta) - 1)), 0, 1,
                            epsabs=1e-13, epsrel=1e-13)
    return theta / (1 + theta) * n / (1 - math.exp(-n)) * val


def test_poissonised_smc_closed_form():
    # End-to-end law of the pick: N ~ Poisson(n) conditioned on N > 0 candidates from pi_gen = pi_target
    # on the two-response instance (pi_target(y1) = 1/(1+theta), r = (0, R)); the frequency with which the
    # oracle's scores + sampler return y0 must match the closed form, which is itself >= 1/2.
    beta, R, n = 1.0, 1.5, 4
    theta = math.exp(float(np.float32(beta)) * R)
    want = _poissonised_pick_probability(theta, n)
    assert want >= 0.5
    rng = np.random.Generator(np.random.Philox(key=[2024, 1]))
    trials = 120_000
    N = rng.poisson(n, size=2 * trials)
    N = N[N > 0][:trials]
    cand = np.zeros(trials + 1, dtype=np.int64)
    np.cumsum(N, out=cand[1:])
    total = int(cand[-1])
    is_y1 = rng.random(total) < 1.0 / (1.0 + theta)
    r = np.where(is_y1, R, 0.0)
    u = ((rng.integers(0, 1 << 23, size=total) + 0.5) * 2.0 ** -23).astype(np.float32)
    chosen, _ = O.gumbel_pick(O.scores(None, None, r, beta), u, cand)
    picked_y0 = ~is_y1[cand[:-1] + chosen]
    freq = picked_y0.mean()
    sd = math.sqrt(want * (1 - want) / trials)
    assert abs(freq - want) < 4.5 * sd, (freq, want, sd)


def test_poissonised_law_normalises():
    # sum over y of the Lemma's pick probability is 1 (the sanity check following Lemma integral-0),
    # evaluated for a three-response instance with a draft generator.
    n, beta = 5, 1.0
    p_gen = np.array([0.5, 0.3, 0.2])
    p_tgt = np.array([0.2, 0.3, 0.5])
    r = np.array([0.1, 0.7, 0.4])
    phi = p_tgt / p_gen * np.exp(beta * r)
    Phi = lambda s: float(np.sum(p_gen * np.exp(-s * phi)))
    total = 0.0
    for y in range(3):
        val, _ = integrate.quad(lambda s: math.exp(n * (Phi(s) - 1)) * math.exp(-s * phi[y]), 0, np.inf,
                                epsabs=1e-13, epsrel=1e-12)
        total += n * p_gen[y] * phi[y] / (1 - math.exp(-n)) * val
    assert abs(total - 1.0) < 1e-8
    # the oracle's weights are exp(S) normalised, and exp(S) is exactly phi for these inputs
    w = O.weights(O.scores(np.log(p_tgt), np.log(p_gen), r.astype(np.float32), beta), np.array([0, 3]))
    assert np.allclose(w, phi / phi.sum(), atol=1e-7)


# ------------------------------------------------------------------ O7: the switch test

def test_accept_flag_laws():
    rng = np.random.Generator(np.random.Philox(key=[9, 9]))
    P, n = 20000, 8
    r = rng.random(P * n).astype(np.float32)
    cand = (np.arange(P + 1) * n).astype(np.int32)
    assert O.accept_flags(r, cand, 1.0).sum() == 0            # tau at the top of the range: never switches
    assert O.accept_flags(r, cand, -0.01).sum() == P
    prev = None
    for tau in (0.5, 0.6, 0.7, 0.8, 0.9):
        f = O.accept_flags(r, cand, tau)
        rate = f.mean()
        want = 1 - float(np.float32(tau)) ** n                # P(max of n uniforms > tau)
        assert abs(rate - want) < 5 * math.sqrt(want * (1 - want) / P) + 1e-4
        if prev is not None:
            assert np.all(f <= prev)                          # monotone non-increasing in tau
        prev = f
    # strictness and the all-candidates maximum
    r2 = np.array([0.7, 0.2, 0.1, 0.8], dtype=np.float32)
    c2 = np.array([0, 2, 2, 4], dtype=np.int32)
    assert O.accept_flags(r2, c2, np.float32(0.7)).tolist() == [0, 0, 1]
    assert O.accept_flags(r2, c2, 0.69).tolist() == [1, 0, 1]


def test_oracle_reproduces_its_stored_tiny_step():
    # regression anchor written by tests/golden/make_tiny_step_golden.py (which calls only the oracle)
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_step.txt")
    stored = {}
    for line in open(path):
        if line.startswith("#"):
            continue
        key, *vals = line.split()
        stored[key] = vals
    x = I.make_step_inputs(I.CONFIGS["tiny"])
    r = O.beam_step(x.hidden, x.w_vocab, x.token_ids, x.block_offsets, x.cand_offsets, x.draft_tok_logprob,
                    x.reward, 1.0, x.uniforms, 0.7)
    for key in ("tok_logprob", "blk_logprob", "weights"):
        want = np.array([float.fromhex(v) for v in stored[key]])
        assert np.allclose(r[key], want, rtol=1e-12, atol=1e-13), key     # BLAS summation order may differ between hosts
    assert [int(v) for v in stored["chosen"]] == r["chosen"].tolist()
    assert [int(v) for v in stored["accept"]] == r["accept"].tolist()
