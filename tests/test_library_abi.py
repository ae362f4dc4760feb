"""CPU checks of the shared library: it builds, loads, exports every symbol the header
declares, and its host-side work-unit planner tiles the problem exactly once."""
import ctypes
import os
import re

import pytest

from paper_2506_15733_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def header_functions():
    text = open(os.path.join(ROOT, "include", "specs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specs_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = header_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in specs.h but not exported"
    assert sorted(binding.SIGNATURES) == names, "binding.SIGNATURES and specs.h disagree"


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(i) for i in range(0, 11)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert binding.status_string(99) == "unknown status"


def test_host_validation_without_a_device(lib):
    out = (ctypes.c_int32 * 16)()
    assert lib.specs_score_plan(128, 12, 100, 148, 0, out) == 2     # d % 8 != 0
    assert lib.specs_score_plan(-1, 16, 100, 148, 0, out) == 2
    assert lib.specs_score_plan(128, 16, 0, 148, 0, out) == 2
    assert lib.specs_score_plan(128, 16, 100, 148, 3, out) == 2     # no such tile shape
    assert lib.specs_score_plan(128, 16, 100, 148, 0, None) == 1
    # calls that need a context refuse a NULL one instead of crashing
    assert lib.specs_destroy(None) == 0
    assert lib.specs_set_engine(None, 0) == 1
    assert lib.specs_score_workspace_bytes(None, 128, 16, 100) == 0
    assert lib.specs_accept(None, None, None, 1, 0.5, None, None) == 1


PLAN_CASES = [
    (64, 256, 1024, 148), (1024, 3584, 151936, 148), (20893, 3584, 151936, 148),
    (65536, 1536, 151936, 148), (65536, 3584, 151936, 148), (131072, 5120, 152064, 148),
    (1, 8, 8, 148), (129, 72, 1000, 148), (20000, 64, 1000, 148), (10000, 1536, 2048, 148),
    (777, 128, 300, 7), (5000, 4096, 70000, 132), (128 * 148 + 1, 64, 257, 148),
    (636, 5120, 421, 148),           # few vocabulary tiles and wide rows: the units cannot all be used
    (40000, 8192, 300, 148), (129, 5120, 256, 148),
]


@pytest.mark.parametrize("cta_group", [0, 1, 2])
@pytest.mark.parametrize("rows,d,V,sms", PLAN_CASES)
def test_plan_covers_every_tile_exactly_once(lib, rows, d, V, sms, cta_group):
    p = binding.score_plan(rows, d, V, sms, cta_group)
    cg = p["cta_group"]
    assert cg in (1, 2) and (cta_group == 0 or cg == cta_group)
    assert p["row_tiles"] == -(-rows // 128) and p["vocab_tiles"] == -(-V // 256) and p["k_blocks"] == -(-d // 64)
    assert p["super_tiles"] == -(-p["row_tiles"] // cg)
    assert p["units"] == sms // cg and p["grid"] == p["units"] * cg
    assert p["waves"] == p["full_waves"] + (1 if p["rem_m"] else 0)
    assert p["group_m"] * p["split_full"] <= p["units"]
    assert p["full_waves"] * p["group_m"] + p["rem_m"] == p["super_tiles"]
    if p["rem_m"]:
        assert 1 <= p["split_rem"] and p["rem_m"] * p["split_rem"] <= p["units"]
    first = p["waves"] * p["grid"] * 2 * 3 * 128 * 4 + p["units"] * 8        # slots + progress words
    if p["k_blocks"] <= p["chunk_kblocks"] or p["row_tiles"] <= 1:
        assert p["workspace_bytes"] == first                      # one chunk, or one HBM-bound row tile: no second pass
        assert first < 256 * rows + (1 << 20)                     # never anything like rows x V
    else:
        # adaptive chunks: control block, list and gathered hidden states of the rows to re-score (at most
        # an eighth of the super tiles, 32 at most), and the second pass's own slots + progress words
        up = lambda n: -(-n // 256) * 256
        cap_rows = min(max(-(-p["super_tiles"] // 8), 1), 32, p["units"]) * 128 * cg
        gathered = up(cap_rows * d * 2)
        assert p["workspace_bytes"] == up(first) + 256 + up(cap_rows * 4) + gathered + up(first)
        assert p["workspace_bytes"] - gathered < 512 * rows + (2 << 20)
        assert gathered <= rows * d * 2 // 8 + 2 * 256 * d * 2
    covered = {}
    for w in range(p["waves"]):
        for c in range(p["grid"]):
            mt, nb, ne = binding.score_plan_unit(rows, d, V, sms, w, c, cta_group)
            if mt < 0:
                continue
            assert 0 <= mt < p["row_tiles"] and 0 <= nb < ne <= p["vocab_tiles"]
            if cg == 2:
                # both CTAs of a pair work on the same vocabulary tiles, on adjacent row tiles
                mt2, nb2, ne2 = binding.score_plan_unit(rows, d, V, sms, w, c ^ 1, cta_group)
                assert mt2 in (-1, mt ^ 1) and (mt2 < 0 or (nb2, ne2) == (nb, ne))
            for n in range(nb, ne):
                assert (mt, n) not in covered
                covered[(mt, n)] = (w, c)
        assert binding.score_plan_unit(rows, d, V, sms, w, p["grid"], cta_group)[0] == -1
    assert len(covered) == p["row_tiles"] * p["vocab_tiles"]


def test_plan_balance_on_the_benchmark_shapes(lib):
    # makespan in tiles per unit versus the ideal total / units, for both tile shapes
    for rows, d, V in [(1024, 3584, 151936), (65536, 3584, 151936), (131072, 5120, 152064), (65536, 1536, 151936),
                       (20893, 3584, 151936)]:
        for cg in (1, 2):
            p = binding.score_plan(rows, d, V, 148, cg)
            span = 0
            for w in range(p["waves"]):
                span += max(ne - nb for mt, nb, ne in
                            (binding.score_plan_unit(rows, d, V, 148, w, c, cg) for c in range(p["grid"])) if mt >= 0)
            ideal = p["super_tiles"] * p["vocab_tiles"] / p["units"]
            assert span <= 1.06 * ideal + 1, (rows, d, V, cg, span, ideal, p)


def test_planner_prefers_pairs_except_for_a_single_row_tile(lib):
    assert binding.score_plan(1024, 3584, 151936, 148)["cta_group"] == 2
    assert binding.score_plan(65536, 3584, 151936, 148)["cta_group"] == 2
    assert binding.score_plan(100, 3584, 151936, 148)["cta_group"] == 1     # 256-row tiles would be half empty
    assert binding.score_plan(1024, 3584, 151936, 1)["cta_group"] == 1      # no pair fits on one SM


def test_binding_checks_tensor_arguments_before_the_call():
    import numpy as np
    # what the C ABI cannot see from a bare pointer: element type, contiguity, size, device
    import torch
    ok = torch.zeros(8, dtype=torch.int32)
    assert binding.device_arg(None, "i32", 8, 0, "x") is None
    with pytest.raises(TypeError):
        binding.device_arg(ok.to(torch.int64), "i32", 8, 0, "token_ids")          # int64 ids
    with pytest.raises(TypeError):
        binding.device_arg(np.zeros(8, np.int32), "i32", 8, 0, "token_ids")        # not a tensor
    with pytest.raises(ValueError):
        binding.device_arg(torch.zeros((4, 4), dtype=torch.bfloat16)[:, :2], "bf16", 8, 0, "hidden")   # a slice
    with pytest.raises(ValueError):
        binding.device_arg(ok, "i32", 9, 0, "tok_logprob")                        # too short
    with pytest.raises(ValueError):
        binding.device_arg(ok, "i32", 8, 0, "token_ids")                          # a host tensor


def test_checked_build_exports_the_same_symbols_and_says_what_it_is(lib):
    import ctypes
    from paper_2506_15733_b200 import build
    assert lib.specs_debug_build() == (1 if binding.debug_build() else 0)
    if not os.path.exists(build.LIB_PATH_DEBUG):
        pytest.skip("checked library not built")
    dbg = ctypes.CDLL(build.LIB_PATH_DEBUG)
    for name in binding.SIGNATURES:
        assert hasattr(dbg, name), name
    dbg.specs_debug_build.restype = ctypes.c_int
    assert dbg.specs_debug_build() == 1


def test_planner_always_produces_a_covering_plan_on_random_shapes(lib):
    # every (rows, d, V) gets at least one wave, never more units than exist, and waves that add up to all
    # super tiles; wide rows with a vocabulary of a few tiles once came out with no wave at all
    import numpy as np
    rng = np.random.Generator(np.random.Philox(key=[8800, 1]))
    for _ in range(400):
        rows = int(rng.integers(1, 200000))
        d = 8 * int(rng.integers(1, 1100))
        V = int(rng.integers(1, 200000)) if rng.random() < 0.7 else int(rng.integers(1, 2000))
        sms = int(rng.choice([1, 7, 132, 148]))
        for cg in (0, 1, 2):
            p = binding.score_plan(rows, d, V, sms, cg)
            assert p["waves"] >= 1, (rows, d, V, sms, cg, p)
            assert p["full_waves"] * p["group_m"] + p["rem_m"] == p["super_tiles"], (rows, d, V, sms, cg, p)
            if p["full_waves"]:
                assert 1 <= p["group_m"] * p["split_full"] <= p["units"] and p["split_full"] <= p["vocab_tiles"]
            if p["rem_m"]:
                assert 1 <= p["rem_m"] * p["split_rem"] <= p["units"] and 1 <= p["split_rem"] <= p["vocab_tiles"]

