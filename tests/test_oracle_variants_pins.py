"""Pins for oracle/specs_variants.py: the selection variants and the Algorithm-1 controller against
closed forms, brute force, limits the paper states, and the already pinned base oracle."""
import numpy as np
import pytest
from scipy import stats

from oracle import specs_oracle as O
from oracle import specs_variants as V
from paper_2506_15733_b200 import inputs as I


def _problem_set(seed, P=200, nmax=12):
    rng = np.random.Generator(np.random.Philox(key=[seed, 3]))
    sizes = rng.integers(0, nmax, P)
    cand = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    B = int(cand[-1])
    lp_t = rng.uniform(-300, -5, B)
    lp_g = lp_t + rng.normal(0, 2.0, B)
    r = rng.random(B).astype(np.float32)
    u = I.draw_uniforms(seed + 1, B)
    return cand, lp_t, lp_g, r, u


# ------------------------------------------------------------------------------- selection

def test_unmasked_subsample_is_algorithm_2_as_the_base_oracle_has_it():
    cand, lp_t, lp_g, r, u = _problem_set(6000)
    chosen, w, margin = V.select(lp_t, lp_g, r, None, cand, 1.5, u)
    S = O.scores(lp_t, lp_g, r, 1.5)
    c0, m0 = O.gumbel_pick(S, u, cand)
    assert np.array_equal(chosen, c0)
    assert np.allclose(w, O.weights(S, cand), rtol=1e-12, atol=0)
    assert np.allclose(margin, m0, rtol=1e-12)


def test_candidate_set_L_renormalises_the_weights_and_excludes_the_rest():
    # P(i* = i) proportional to exp(S_i) 1(i in L): closed form on three candidates, L = {0, 2}
    lp_t = np.array([-10.0, -9.0, -11.5]); lp_g = np.array([-10.5, -12.0, -11.0]); r = np.array([0.2, 0.9, 0.6], np.float32)
    S = (lp_t - lp_g) + 2.0 * r.astype(np.float64)
    mask = np.array([1, 0, 1], np.uint8)
    _, w, _ = V.select(lp_t, lp_g, r, mask, np.array([0, 3]), 2.0, np.array([0.3, 0.6, 0.9]))
    e = np.exp(S[[0, 2]])
    assert w[1] == 0.0 and np.allclose(w[[0, 2]], e / e.sum(), rtol=1e-13)
    # frequencies of the masked sampler follow those weights (chi-squared), the masked one is never drawn
    draws = 100_000
    u = I.draw_uniforms(6100, 3 * draws).reshape(draws, 3)
    counts = np.zeros(3)
    for k in range(draws):
        c, _, _ = V.select(lp_t, lp_g, r, mask, np.array([0, 3]), 2.0, u[k])
        counts[c[0]] += 1
    assert counts[1] == 0
    assert stats.chisquare(counts[[0, 2]], draws * w[[0, 2]]).pvalue > 1e-3
    # nobody eligible: nothing selected, no weight
    c, w0, _ = V.select(lp_t, lp_g, r, np.zeros(3, np.uint8), np.array([0, 3]), 2.0, u[0])
    assert c[0] == -1 and not w0.any()


def test_best_reward_is_plain_argmax_and_the_large_beta_limit_of_algorithm_2():
    cand, lp_t, lp_g, r, u = _problem_set(6200)
    chosen, w, _ = V.select(lp_t, lp_g, r, None, cand, 1.0, None, rule=V.SELECT_BEST_REWARD)
    for p in range(len(cand) - 1):
        a, b = cand[p], cand[p + 1]
        if b <= a:
            assert chosen[p] == -1
            continue
        assert chosen[p] == max(range(b - a), key=lambda i: (r[a + i], -i))       # brute force, lowest index on ties
        assert w[a + chosen[p]] == 1.0 and w[a:b].sum() == 1.0
    # beta -> infinity with pi_gen = pi_target (hard best-of-n): Algorithm 2's weights pile up on the same candidate
    r_sep = (np.argsort(np.argsort(r)) / len(r)).astype(np.float32)                # distinct rewards, gaps >= 1/B
    hard, _, _ = V.select(None, None, r_sep, None, cand, 1.0, None, rule=V.SELECT_BEST_REWARD)
    soft, w_soft, _ = V.select(None, None, r_sep, None, cand, 1.0e6, u)
    live = np.diff(cand) > 0
    assert np.array_equal(hard[live], soft[live])
    assert all(w_soft[cand[p] + hard[p]] > 1 - 1e-9 for p in np.nonzero(live)[0])
    # ties keep the lowest index
    c, _, _ = V.select(None, None, np.array([0.5, 0.8, 0.8], np.float32), None, np.array([0, 3]), 1.0, None,
                       rule=V.SELECT_BEST_REWARD)
    assert c[0] == 1


def test_no_ll_drops_the_log_ratio():
    cand, lp_t, lp_g, r, u = _problem_set(6300)
    a = V.select(lp_t, lp_g, r, None, cand, 3.0, u, score_flags=V.SCORE_NO_LL)
    b = V.select(None, None, r, None, cand, 3.0, u)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    w_ref = O.weights(O.scores(None, None, r, 3.0), cand)                          # softmax(beta r)
    assert np.allclose(a[1], w_ref, rtol=1e-12)
    c = V.select(lp_t, lp_g, r, None, cand, 3.0, u)
    assert not np.allclose(c[1], a[1])                                             # the ratio does matter


# ------------------------------------------------------------------------------- switch rules

def test_switch_rules_on_a_worked_example():
    r = np.array([0.9, 0.65, 0.2, 0.7, 0.3, 0.1], np.float32)
    cand = np.array([0, 3, 3, 6])
    chosen = np.array([1, -1, 0])
    assert V.switch_flags(r, cand, chosen, 0.7, V.SWITCH_ANY_ABOVE).tolist() == [1, 0, 0]      # 0.7 > 0.7 is false
    assert V.switch_flags(r, cand, chosen, 0.7, V.SWITCH_NONE_ABOVE).tolist() == [0, 0, 1]
    assert V.switch_flags(r, cand, chosen, 0.7, V.SWITCH_CHOSEN_BELOW).tolist() == [1, 0, 0]   # 0.65 < 0.7; 0.7 < 0.7 false
    assert V.switch_flags(r, cand, np.array([0, -1, 1]), 0.7, V.SWITCH_CHOSEN_BELOW).tolist() == [0, 0, 1]


def test_switch_rules_against_the_base_oracle_and_each_other():
    cand, _, _, r, _ = _problem_set(6400)
    live = np.diff(cand) > 0
    for tau in (0.3, 0.7, 0.95, 1.0):
        any_above = V.switch_flags(r, cand, None, tau, V.SWITCH_ANY_ABOVE)
        assert np.array_equal(any_above, O.accept_flags(r, cand, tau))
        none_above = V.switch_flags(r, cand, None, tau, V.SWITCH_NONE_ABOVE)
        assert np.array_equal(none_above[live], 1 - any_above[live]) and not none_above[~live].any()
    assert not V.switch_flags(r, cand, None, 1.0, V.SWITCH_ANY_ABOVE).any()        # tau -> 1: never to the draft
    best, _, _ = V.select(None, None, r, None, cand, 1.0, None, rule=V.SELECT_BEST_REWARD)
    # with the best-reward pick, "chosen below tau" is "none at or above tau"
    below = V.switch_flags(r, cand, best, 0.7, V.SWITCH_CHOSEN_BELOW)
    for p in np.nonzero(live)[0]:
        assert below[p] == (r[cand[p]:cand[p + 1]].max() < np.float32(0.7))


# ------------------------------------------------------------------------------- controller

def _run(ctrl, flags, chosen_len=10, uniforms=None):
    seen = []
    for k, f in enumerate(flags):
        seen.append(ctrl.generators()[0])
        ctrl.advance([0], [f], [chosen_len], None if uniforms is None else [uniforms[k]])
    seen.append(ctrl.generators()[0])
    return seen


def test_controller_follows_algorithm_1():
    T, D, X = V.GEN_TARGET, V.GEN_DRAFT, V.GEN_DONE
    # generation begins with the target; a step with a high reward hands the next step to the draft
    assert _run(V.Controller(1), [0, 1, 0, 1, 1]) == [T, T, D, T, D, D]
    # Algorithm 1 read literally only ever assigns pi_gen <- pi_draft
    assert _run(V.Controller(1, sticky=True), [0, 1, 0, 0, 0]) == [T, T, D, D, D, D]
    # tau -> 1 raises no flag: every block comes from the target (beam search with the large model)
    c = V.Controller(1, target_len=50)
    assert _run(c, [0] * 5) == [T] * 5 + [X]
    assert c.length == [50] and c.steps == [5] and c.target_steps == [5]
    # the loop ends once the target length is reached; later calls change nothing
    c.advance([0], [1], [10])
    assert c.length == [50] and c.generators() == [X]


def test_controller_policies_of_the_ablations_and_baselines():
    T, D = V.GEN_TARGET, V.GEN_DRAFT
    assert _run(V.Controller(1, policy=V.POLICY_ONLY_DRAFT), [0, 1, 0]) == [D, D, D, D]
    assert _run(V.Controller(1, policy=V.POLICY_ONLY_TARGET), [0, 1, 1]) == [T, T, T, T]
    # draft start: the flag (no candidate above tau) sends the next step to the target
    assert _run(V.Controller(1, policy=V.POLICY_DRAFT_START), [0, 1, 0, 1]) == [D, D, T, D, T]
    assert _run(V.Controller(1, policy=V.POLICY_DRAFT_START, sticky=True), [0, 1, 0]) == [D, D, T, T]
    # RSD++: a weak best draft candidate makes the target redo the SAME step; nothing is appended meanwhile
    c = V.Controller(1, policy=V.POLICY_RSD, target_len=40)
    assert _run(c, [0, 1, 0, 0, 1, 1]) == [D, D, T, D, D, T, V.GEN_DONE]
    assert c.steps == [4] and c.length == [40] and c.target_steps == [2] and c.target_calls == [2]
    # an empty problem appends nothing and never finishes by length
    c = V.Controller(1, target_len=20)
    c.advance([-1], [0], [10])
    assert c.length == [0] and c.steps == [0]


def test_random_switching_matches_the_requested_share_of_target_steps():
    steps, p = 20000, 0.35
    u = I.draw_uniforms(6500, steps)
    c = V.Controller(1, policy=V.POLICY_RANDOM, p_target=p, target_len=10 ** 9)
    seen = _run(c, [0] * steps, uniforms=u)
    share = np.mean(np.array(seen[1:]) == V.GEN_TARGET)
    assert abs(share - p) < 4 * np.sqrt(p * (1 - p) / steps)
    assert c.target_steps[0] == sum(g == V.GEN_TARGET for g in seen[:-1])


# ------------------------------------------------------------------------------- both heads, and the append

def test_dual_step_is_eq_1_with_both_block_probabilities_computed():
    # tiny case by brute force: every probability from explicit softmaxes in Python floats
    import math
    rng = np.random.Generator(np.random.Philox(key=[6800, 1]))
    Vv, rows = 5, 6
    def bits(a):
        return (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)       # values exact in bf16
    Ht = bits(rng.integers(-4, 5, (rows, 8)) / 4.0); Wt = bits(rng.integers(-4, 5, (Vv, 8)) / 8.0)
    Hg = bits(rng.integers(-4, 5, (rows, 16)) / 4.0); Wg = bits(rng.integers(-4, 5, (Vv, 16)) / 8.0)
    ids = rng.integers(0, Vv, rows).astype(np.int32)
    boff = np.array([0, 2, 3, 6]); cand = np.array([0, 3])
    r = np.array([0.3, 0.8, 0.5], np.float32); u = np.array([0.2, 0.5, 0.7], np.float32)
    got = V.beam_step_dual(Ht, Wt, Hg, Wg, ids, boff, cand, r, 2.0, u, 0.7)

    def lp(H, W, t):
        h = O.bf16_bits_to_f64(H)[t].tolist(); w = O.bf16_bits_to_f64(W).tolist()
        z = [sum(a * b for a, b in zip(h, wv)) for wv in w]
        return z[ids[t]] - math.log(sum(math.exp(v) for v in z))
    S = []
    for i in range(3):
        ratio = sum(lp(Ht, Wt, t) - lp(Hg, Wg, t) for t in range(boff[i], boff[i + 1]))
        S.append(ratio + 2.0 * float(r[i]))
    assert np.allclose(got["score"], S, rtol=1e-12)
    assert np.allclose(got["tok_logratio"].sum(), sum(S) - 2.0 * float(r.sum()), rtol=1e-12)
    pert = [S[i] - math.log(-math.log(float(u[i]))) for i in range(3)]
    assert got["chosen"][0] == pert.index(max(pert)) and got["accept"][0] == 1
    # identical heads: the ratio vanishes and the score collapses to beta * r (text after Eq. 1)
    same = V.beam_step_dual(Ht, Wt, Ht, Wt, ids, boff, cand, r, 2.0, u, 0.7)
    assert np.allclose(same["score"], 2.0 * r.astype(np.float64), atol=1e-12)


def test_gather_chosen_worked_example():
    ids = np.arange(100, 112, dtype=np.int32)
    boff = np.array([0, 3, 3, 7, 9, 12]); cand = np.array([0, 2, 2, 5])
    out, lens = V.gather_chosen(ids, boff, cand, np.array([0, -1, 2]), 4)
    assert out.tolist() == [[100, 101, 102, -1], [-1, -1, -1, -1], [109, 110, 111, -1]]
    assert lens.tolist() == [3, 0, 3]
    out, lens = V.gather_chosen(ids, boff, cand, np.array([1, -1, 0]), 4)       # an empty block is a valid pick
    assert out[0].tolist() == [-1] * 4 and lens.tolist() == [0, 0, 4] and out[2].tolist() == [103, 104, 105, 106]
    with pytest.raises(ValueError):
        V.gather_chosen(ids, boff, cand, np.array([0, -1, 0]), 3)


# ------------------------------------------------------------------------------- PRM head

def test_prm_head_closed_forms():
    from scipy.special import expit

    def bits(a):
        return (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)
    rng = np.random.Generator(np.random.Philox(key=[6900, 1]))
    d, rows = 24, 9
    H = rng.integers(-8, 9, (rows, d)) / 8.0                     # exact in bf16
    w = rng.integers(-8, 9, d) / 16.0
    boff = np.array([0, 2, 2, 5, 9])
    r = V.prm_rewards(bits(H), boff, bits(w), 0.25)
    last = [1, None, 4, 8]                                        # the block's LAST token is read
    for i, t in enumerate(last):
        if t is None:
            assert np.isnan(r[i])                                 # an empty block has no last token
        else:
            assert abs(r[i] - expit(float(H[t] @ w) + 0.25)) < 1e-15
    assert np.all((r[[0, 2, 3]] > 0) & (r[[0, 2, 3]] < 1))
    # zero hidden state: the logistic of the bias alone; zero weight too: exactly one half
    assert V.prm_rewards(bits(np.zeros((1, d))), np.array([0, 1]), bits(w), 0.25)[0] == expit(0.25)
    assert V.prm_rewards(bits(H[:1]), np.array([0, 1]), bits(np.zeros(d)), 0.0)[0] == 0.5
    # sigma(-z) = 1 - sigma(z): negating the head mirrors the reward
    r_neg = V.prm_rewards(bits(H), boff, bits(-w), -0.25)
    assert np.allclose(r_neg[[0, 2, 3]], 1.0 - r[[0, 2, 3]], rtol=0, atol=1e-15)
    # monotone in the bias
    assert np.all(V.prm_rewards(bits(H), boff, bits(w), 1.0)[[0, 2, 3]] > r[[0, 2, 3]])


# ------------------------------------------------------------------------------- vocabulary shards

@pytest.mark.parametrize("cuts", [(0, 37), (0, 1, 37), (0, 5, 20, 21, 37), (0, 36, 37)])
def test_sharded_log_softmax_equals_the_whole(cuts):
    # the log-sum-exp over a partition of the vocabulary, against the unsharded definition
    cfg = I.StepConfig("shards", 7100, 1, 3, (4, 4), 16, 37, 0.6, hidden_scale=2.0)
    x = I.make_step_inputs(cfg)
    ids = x.token_ids.copy()
    ids[0], ids[1] = 0, 36                                        # first and last vocabulary entry
    whole = O.token_logprobs(x.hidden, x.w_vocab, ids)
    parts = np.stack([V.shard_partials(x.hidden, x.w_vocab, ids, a, b) for a, b in zip(cuts[:-1], cuts[1:])])
    assert np.allclose(V.merge_partials(parts, ids, 37), whole, rtol=0, atol=1e-12)
    assert np.all((parts[:, :, 2] > -np.inf).sum(axis=0) == 1)    # exactly one shard holds the drafted id
    # the order of the shards does not matter
    assert np.allclose(V.merge_partials(parts[::-1], ids, 37), whole, rtol=0, atol=1e-12)
    # an id outside the vocabulary has no probability
    bad = ids.copy(); bad[2] = 37
    parts_bad = np.stack([V.shard_partials(x.hidden, x.w_vocab, bad, a, b) for a, b in zip(cuts[:-1], cuts[1:])])
    assert np.isnan(V.merge_partials(parts_bad, bad, 37)[2])
