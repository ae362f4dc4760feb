"""Pins for oracle/specs_fp8.py: the E4M3 format against its definition, the rounding rule against
exact rational arithmetic, and the quantised scoring against the unquantised oracle within the bound
the format implies."""
from fractions import Fraction

import numpy as np

from oracle import specs_fp8 as F
from oracle import specs_oracle as O
from paper_2506_15733_b200 import inputs as I


def test_e4m3_values_of_the_format():
    t = F.e4m3_decode_table()
    assert t[0x00] == 0.0 and t[0x38] == 1.0 and t[0x3C] == 1.5 and t[0x40] == 2.0
    assert t[0x7E] == 448.0 and t[0x08] == 2.0 ** -6 and t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF])
    finite = t[:0x7F]
    assert np.all(np.diff(finite) > 0)                            # codes order like their values
    assert np.array_equal(t[0x80:0xFF], -t[0x00:0x7F])
    assert not np.isinf(t[~np.isnan(t)]).any()                    # the format has no infinities


def test_encode_is_round_to_nearest_even_and_saturates():
    t = F.e4m3_decode_table()
    finite = [c for c in range(256) if not np.isnan(t[c])]
    assert np.array_equal(F.e4m3_encode(t[finite].astype(np.float32)) & 0x7F, np.array(finite) & 0x7F)  # fixed points
    # every midpoint between neighbours goes to the even code; a hair to either side goes to that side
    for c in range(0x7E):
        lo, hi = Fraction(t[c]), Fraction(t[c + 1])
        mid = float((lo + hi) / 2)                                # exact in float32 (5 significant bits)
        assert F.e4m3_encode(np.float32(mid)) == (c if c % 2 == 0 else c + 1)
        assert F.e4m3_encode(np.nextafter(np.float32(mid), np.float32(0))) == c
        assert F.e4m3_encode(np.nextafter(np.float32(mid), np.float32(1e9))) == c + 1
    assert F.e4m3_encode(np.float32(1e6)) == 0x7E and F.e4m3_encode(np.float32(-1e6)) == 0xFE
    assert F.e4m3_encode(np.float32(464.0)) == 0x7E               # beyond the last midpoint: still 448
    assert F.e4m3_encode(np.float32(-0.3)) == 0x80 | F.e4m3_encode(np.float32(0.3))
    # brute force against exact nearest search on random inputs
    rng = np.random.Generator(np.random.Philox(key=[7300, 1]))
    y = (rng.normal(0, 100, 4000)).astype(np.float32)
    pos = [Fraction(v) for v in t[:0x7F]]
    for v in y[:400]:
        a = Fraction(float(abs(v)))
        best = min(range(0x7F), key=lambda c: (abs(pos[c] - a), c % 2))
        if a >= 448:
            best = 0x7E
        assert (F.e4m3_encode(v) & 0x7F) == best


def test_row_quantisation_maps_the_largest_magnitude_to_448():
    cfg = I.StepConfig("q", 7310, 1, 2, (5, 5), 64, 40, 0.05, hidden_scale=3.0)
    x = I.make_step_inputs(cfg)
    codes, scale = F.quantize_rows(x.hidden)
    t = F.e4m3_decode_table()
    xf = O.bf16_bits_to_f64(x.hidden)
    assert np.all(np.abs(t[codes]).max(axis=1) == 448.0)
    assert np.allclose(scale, np.abs(xf).max(axis=1) / 448.0, rtol=1e-6)
    rel = np.abs(t[codes] * scale[:, None].astype(np.float64) - xf)
    assert np.all(rel <= np.maximum(np.abs(xf) * 2.0 ** -4, scale[:, None] * 2.0 ** -10) * 1.001)   # half a spacing
    zc, zs = F.quantize_rows(np.zeros((2, 8), np.uint16))
    assert not zc.any() and np.all(zs == 1.0)


def test_quantised_scoring_stays_near_the_exact_one_and_is_exact_on_representable_inputs():
    # inputs whose rows already are 448-scaled E4M3 numbers times a power of two: nothing is lost
    rng = np.random.Generator(np.random.Philox(key=[7320, 1]))
    t = F.e4m3_decode_table()
    def rows_of_codes(n, d):
        c = rng.integers(0, 0x7F, (n, d)).astype(np.uint8) | (rng.integers(0, 2, (n, d)).astype(np.uint8) << 7)
        c[:, 0] = 0x7E                                            # the row maximum is 448
        return c
    hc, wc = rows_of_codes(6, 32), rows_of_codes(24, 32)
    hb = I.f32_to_bf16_bits((t[hc] / 256.0).astype(np.float32)); wb = I.f32_to_bf16_bits((t[wc] / 4096.0).astype(np.float32))
    ids = rng.integers(0, 24, 6).astype(np.int32)
    qh, sh = F.quantize_rows(hb); qw, sw = F.quantize_rows(wb)
    assert np.array_equal(qh, hc) and np.array_equal(qw, wc)
    assert np.allclose(F.token_logprobs_fp8(qh, sh, qw, sw, ids), O.token_logprobs(hb, wb, ids), rtol=0, atol=1e-12)
    # generic inputs: element errors of at most 2^-4 relative give logit errors of a few percent of the logit scale
    cfg = I.StepConfig("q2", 7321, 1, 4, (8, 8), 256, 300, 0.05)
    x = I.make_step_inputs(cfg)
    qh, sh = F.quantize_rows(x.hidden); qw, sw = F.quantize_rows(x.w_vocab)
    lp8 = F.token_logprobs_fp8(qh, sh, qw, sw, x.token_ids)
    lp = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
    assert 1e-4 < np.abs(lp8 - lp).max() < 0.15                   # logit sigma is 0.8 here
    bad = x.token_ids.copy(); bad[0] = 300
    assert np.isnan(F.token_logprobs_fp8(qh, sh, qw, sw, bad)[0])
