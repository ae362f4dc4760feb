"""The native Algorithm-1 controller (host logic in the shared library) against the oracle's state
machine, on seeded random step results; no GPU involved."""
import numpy as np
import pytest

from oracle import specs_variants as V
from paper_2506_15733_b200 import binding
from paper_2506_15733_b200 import inputs as I

POLICIES = [V.POLICY_SPECS, V.POLICY_ONLY_DRAFT, V.POLICY_ONLY_TARGET, V.POLICY_RANDOM, V.POLICY_DRAFT_START,
            V.POLICY_RSD]


def test_constants_agree_with_the_header():
    for name in ("GEN_TARGET", "GEN_DRAFT", "GEN_DONE", "POLICY_SPECS", "POLICY_ONLY_DRAFT", "POLICY_ONLY_TARGET",
                 "POLICY_RANDOM", "POLICY_DRAFT_START", "POLICY_RSD", "SELECT_SUBSAMPLE", "SELECT_BEST_REWARD",
                 "SCORE_NO_LL", "SWITCH_ANY_ABOVE", "SWITCH_NONE_ABOVE", "SWITCH_CHOSEN_BELOW"):
        assert getattr(binding, name) == getattr(V, name), name


@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("sticky", [False, True])
def test_native_controller_tracks_the_oracle(policy, sticky):
    P, steps = 40, 120
    rng = np.random.Generator(np.random.Philox(key=[6600 + policy, int(sticky)]))
    want = V.Controller(P, policy, target_len=900, sticky=sticky, p_target=0.4, max_steps=100)
    got = binding.Controller(P, policy, target_len=900, sticky=sticky, p_target=0.4, max_steps=100)
    for k in range(steps):
        assert got.generators().tolist() == want.generators()
        chosen = rng.integers(-1, 6, P).astype(np.int32)          # -1: nothing eligible this step
        flag = (rng.random(P) < 0.4).astype(np.uint8)
        lens = rng.integers(1, 40, P).astype(np.int64)
        u = I.draw_uniforms(6700 + k, P)
        steps_before = list(want.steps)
        want.advance(chosen, flag, lens, u)
        got.advance(chosen, flag, lens, u)
        # the controller says which problems appended their selected block in this update
        assert got.appended().tolist() == [int(a != b) for a, b in zip(want.steps, steps_before)]
    st = got.stats()
    assert st["length"].tolist() == want.length and st["steps"].tolist() == want.steps
    assert st["target_steps"].tolist() == want.target_steps and st["target_calls"].tolist() == want.target_calls
    assert (np.array(got.generators()) == V.GEN_DONE).sum() > 0   # some problems reached their target length
    got.close()


def test_controller_argument_checks():
    with pytest.raises(binding.SpecsError) as e:
        binding.Controller(4, policy=9)
    assert e.value.status == 2
    with pytest.raises(binding.SpecsError) as e:
        binding.Controller(4, policy=V.POLICY_RANDOM, p_target=1.5)
    assert e.value.status == 2
    c = binding.Controller(2, policy=V.POLICY_RANDOM)
    with pytest.raises(binding.SpecsError) as e:
        c.advance([0, 0], [0, 0], [5, 5])                         # random switching needs its uniforms
    assert e.value.status == 1
    with pytest.raises(binding.SpecsError) as e:
        c.advance([0, 0], [0, 0], [5, -5], [0.5, 0.5])
    assert e.value.status == 2
    assert c.stats()["length"].tolist() == [0, 0]                 # a refused update changes nothing
    empty = binding.Controller(0)
    assert empty.generators().tolist() == []
