"""CPU oracle for the 8-bit (E4M3) variant of block scoring.  TEST INFRASTRUCTURE ONLY.

The paper scores with the models' own weights and states no precision; this variant is an
extension (a "next" item), so what it computes is defined here, step by step:

  1. Every row of the hidden states and every row of the LM-head weight is scaled so that its
     largest magnitude maps to 448, the largest finite E4M3 value, and each element is rounded to
     the nearest E4M3 number (ties to even, saturating).  The scale arithmetic is float32 because
     the codes are integers decided by floating point: inv = 448 / absmax and y = x * inv are
     float32 operations here as on the GPU; scale = absmax / 448 (float32) is what multiplies back.
     A row of zeros gets scale 1 and codes 0.
  2. logit[t, v] = scale_h[t] * scale_w[v] * sum_k q_h[t, k] * q_w[v, k], the sum taken exactly
     (float64 holds it: |q| <= 448 with 4 significant bits).
  3. log-softmax and the drafted id's entry, as in specs_oracle.token_logprobs.

E4M3 is the 8-bit format of the OCP "8-bit floating point" specification: 1 sign, 4 exponent
(bias 7), 3 mantissa bits, subnormals at exponent 0, no infinities, the all-ones pattern is NaN.
Nothing here is imported by the product, and this file imports nothing from it.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def e4m3_decode_table() -> np.ndarray:
    """Value of each of the 256 codes (NaN for 0x7f and 0xff), from the format's definition."""
    out = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            out[code] = np.nan
        elif e == 0:
            out[code] = sign * (m / 8.0) * 2.0 ** (-6)
        else:
            out[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


_TABLE = e4m3_decode_table()
_POS = _TABLE[:0x7F]                      # the 127 non-negative finite values, ascending


def e4m3_encode(y: np.ndarray) -> np.ndarray:
    """Nearest E4M3 code of each float32 in y: round to nearest, ties to the even code, saturate at 448."""
    y = np.asarray(y, dtype=np.float32)
    a = np.abs(y).astype(np.float64)
    hi = np.searchsorted(_POS, a, side="left")           # first value >= a
    hi = np.clip(hi, 0, len(_POS) - 1)
    lo = np.clip(hi - 1, 0, len(_POS) - 1)
    d_hi, d_lo = np.abs(_POS[hi] - a), np.abs(a - _POS[lo])
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(a >= E4M3_MAX, 0x7E, code)           # saturate
    return (code | np.where(np.signbit(y), 0x80, 0)).astype(np.uint8)


def quantize_rows(bits: np.ndarray):
    """bf16 bit patterns [n, d] -> (codes uint8 [n, d], scale float32 [n]) as step 1 describes."""
    x = (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
    absmax = np.max(np.abs(x), axis=1).astype(np.float32)
    live = absmax > 0
    safe = np.where(live, absmax, np.float32(1.0)).astype(np.float32)
    inv = np.where(live, np.float32(E4M3_MAX) / safe, np.float32(1.0)).astype(np.float32)
    scale = np.where(live, safe / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    y = (x * inv[:, None]).astype(np.float32)
    return e4m3_encode(y), scale


def token_logprobs_fp8(h_codes, h_scale, w_codes, w_scale, token_ids, row_chunk: int = 64) -> np.ndarray:
    """log-probability of every drafted id under the quantised head (steps 2 and 3)."""
    Wq = _TABLE[np.asarray(w_codes, dtype=np.uint8)]
    sw = np.asarray(w_scale, dtype=np.float64)
    V = Wq.shape[0]
    rows = h_codes.shape[0]
    out = np.empty(rows)
    for r0 in range(0, rows, row_chunk):
        r1 = min(rows, r0 + row_chunk)
        Hq = _TABLE[np.asarray(h_codes[r0:r1], dtype=np.uint8)]
        Z = (Hq @ Wq.T) * np.asarray(h_scale[r0:r1], dtype=np.float64)[:, None] * sw[None, :]
        m = Z.max(axis=1)
        lse = m + np.log(np.exp(Z - m[:, None]).sum(axis=1))
        for t in range(r0, r1):
            y = int(token_ids[t])
            out[t] = Z[t - r0, y] - lse[t - r0] if 0 <= y < V else np.nan
    return out
