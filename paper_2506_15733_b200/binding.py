"""Thin ctypes binding over the C ABI declared in ``include/specs.h``.

Argument marshalling only: every step of the method runs in the CUDA kernels of
the shared library.  Device buffers are torch tensors (torch is used for device
memory and streams, nothing else); functions take ``tensor.data_ptr()`` and the
current torch stream.  If the shared library is missing the first call raises --
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

# SPECS_B200_DEBUG=1 in the environment selects the checked build (index checks inside the kernels, the plain
# CUDA-core engine): see specs_debug_build in specs.h.
_DEBUG = os.environ.get("SPECS_B200_DEBUG", "0") not in ("", "0")
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libspecs_b200_debug.so" if _DEBUG else "libspecs_b200.so")
_lib = None

OK = 0
ENGINE_TCGEN05 = 0
ENGINE_SIMT = 1
ENGINE_TCGEN05_1CTA = 2
ENGINE_TCGEN05_2CTA = 3
DEV_TIMEOUT = 0x1
DEV_TOKEN_RANGE = 0x2
DEV_ACCUM_RANGE = 0x4
DEV_BOUNDS = 0x8
ACCUM_ADAPTIVE = -1
SELECT_SUBSAMPLE, SELECT_BEST_REWARD = 0, 1
SCORE_NO_LL = 0x1
SWITCH_ANY_ABOVE, SWITCH_NONE_ABOVE, SWITCH_CHOSEN_BELOW = 0, 1, 2
GEN_TARGET, GEN_DRAFT, GEN_DONE = 0, 1, -1
POLICY_SPECS, POLICY_ONLY_DRAFT, POLICY_ONLY_TARGET, POLICY_RANDOM, POLICY_DRAFT_START, POLICY_RSD = range(6)

_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float

# name -> (restype, argtypes); mirrors include/specs.h one to one
SIGNATURES = {
    "specs_debug_build": (C.c_int, []),
    "specs_status_string": (C.c_char_p, [C.c_int]),
    "specs_create": (C.c_int, [C.POINTER(_vp), C.c_int]),
    "specs_destroy": (C.c_int, [_vp]),
    "specs_set_engine": (C.c_int, [_vp, C.c_int]),
    "specs_set_accum_chunk": (C.c_int, [_vp, _i32]),
    "specs_set_tile_lead": (C.c_int, [_vp, _i32]),
    "specs_sm_count": (C.c_int, [_vp]),
    "specs_score_workspace_bytes": (C.c_size_t, [_vp, _i64, _i32, _i32]),
    "specs_score_blocks": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp,
                                     C.c_size_t, _vp]),
    "specs_score_partials": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i32, _i32, _vp, _vp, C.c_size_t, _vp]),
    "specs_merge_partials": (C.c_int, [_vp, _vp, _i32, _i64, _vp, _i32, _vp, _vp]),
    "specs_quantize_rows_e4m3": (C.c_int, [_vp, _vp, _i64, _i32, _vp, _vp, _vp]),
    "specs_score_workspace_bytes_fp8": (C.c_size_t, [_vp, _i64, _i32, _i32]),
    "specs_score_blocks_fp8": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp,
                                         C.c_size_t, _vp]),
    "specs_beam_step_fp8_workspace_bytes": (C.c_size_t, [_vp, _i64, _i32, _i32]),
    "specs_beam_step_fp8": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32,
                                      _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, _vp]),
    "specs_block_sums": (C.c_int, [_vp, _vp, _vp, _i32, _vp, _vp, _vp]),
    "specs_subsample": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _f32, _vp, _vp, _vp, _f32, _vp, _vp]),
    "specs_subsample_f64": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _f32, _vp, _vp, _vp, _f32, _vp, _vp]),
    "specs_accept": (C.c_int, [_vp, _vp, _vp, _i32, _f32, _vp, _vp]),
    "specs_prm_rewards": (C.c_int, [_vp, _vp, _vp, _i32, _i32, _vp, _f32, _vp, _vp]),
    "specs_select": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _f32, _vp, C.c_int, C.c_int, C.c_int, _f32,
                               _vp, _vp, _vp, _vp]),
    "specs_controller_create": (C.c_int, [C.POINTER(_vp), _i32, _vp]),
    "specs_controller_destroy": (C.c_int, [_vp]),
    "specs_controller_generators": (C.c_int, [_vp, _vp]),
    "specs_controller_advance": (C.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "specs_controller_appended": (C.c_int, [_vp, _vp]),
    "specs_controller_stats": (C.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "specs_beam_step": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32, _f32, _f32,
                                  _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, _vp]),
    "specs_beam_step_dual_workspace_bytes": (C.c_size_t, [_vp, _i64, _i32, _i32, _i32]),
    "specs_beam_step_dual": (C.c_int, [_vp, _vp, _vp, _i32, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32,
                                       _i32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp,
                                       C.c_size_t, _vp]),
    "specs_gather_chosen": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _i32, _vp]),
    "specs_device_status": (C.c_int, [_vp, C.POINTER(C.c_uint32), _vp]),
    "specs_beam_step_host": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32,
                                       _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "specs_beam_step_host_submit": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32,
                                              _i32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, C.POINTER(_i32)]),
    "specs_beam_step_host_wait": (C.c_int, [_vp, _i32]),
    "specs_probe_wait_expiry": (C.c_int, [_vp, _i64, _vp]),
    "specs_set_timing": (C.c_int, [_vp, C.c_int]),
    "specs_score_kernel_ms": (C.c_float, [_vp, C.POINTER(_i32)]),
    "specs_score_blocks_noalloc": (C.c_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "specs_score_plan": (C.c_int, [_i64, _i32, _i32, _i32, _i32, C.POINTER(_i32)]),
    "specs_score_plan_unit": (C.c_int, [_i64, _i32, _i32, _i32, _i32, _i32, _i32, C.POINTER(_i32)]),
}


class SpecsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


def load_library():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2506_15733_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(_LIB_PATH)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def debug_build() -> bool:
    """True when the loaded library is the checked build."""
    return bool(load_library().specs_debug_build())


def status_string(status: int) -> str:
    return load_library().specs_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise SpecsError(status, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array, None for None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(device=None) -> Optional[int]:
    """torch's current stream on ``device`` (default: the current device) as an integer handle."""
    import torch
    return torch.cuda.current_stream(device).cuda_stream or None


_TORCH_DTYPES = {"bf16": "bfloat16", "f32": "float32", "f64": "float64", "i32": "int32", "i64": "int64",
                 "u8": "uint8"}


def device_arg(t, dtype: str, count: int, device: int, name: str) -> Optional[int]:
    """Address of a device tensor after checking what the C ABI cannot see: the element type, that the
    elements are contiguous, that there are at least ``count`` of them, and that they live on CUDA device
    ``device``.  None passes through (the library decides whether the argument is optional).
    Raises TypeError (wrong type) or ValueError (layout, size, device)."""
    if t is None:
        return None
    import torch
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name}: expected a torch tensor on cuda:{device}, got {type(t).__name__}")
    want = getattr(torch, _TORCH_DTYPES[dtype])
    if t.dtype != want:
        raise TypeError(f"{name}: expected dtype {want}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: tensor is not contiguous")
    if t.numel() < count:
        raise ValueError(f"{name}: {t.numel()} elements, at least {count} needed")
    if not t.is_cuda or t.device.index != device:
        raise ValueError(f"{name}: tensor is on {t.device}, the context is on cuda:{device}")
    return t.data_ptr()


def score_plan(rows: int, d: int, V: int, num_sms: int, cta_group: int = 0) -> dict:
    out = (_i32 * 16)()
    _check(load_library().specs_score_plan(rows, d, V, num_sms, cta_group, out), "specs_score_plan")
    keys = ["row_tiles", "vocab_tiles", "k_blocks", "grid", "group_m", "split_full", "full_waves", "rem_m",
            "split_rem", "waves"]
    plan = {k: int(out[i]) for i, k in enumerate(keys)}
    plan["workspace_bytes"] = int(out[10]) + (int(out[11]) << 31)
    plan.update(cta_group=int(out[12]), units=int(out[13]), super_tiles=int(out[14]), chunk_kblocks=int(out[15]))
    return plan


def score_plan_unit(rows: int, d: int, V: int, num_sms: int, wave: int, cta: int, cta_group: int = 0):
    out = (_i32 * 3)()
    _check(load_library().specs_score_plan_unit(rows, d, V, num_sms, cta_group, wave, cta, out),
           "specs_score_plan_unit")
    return int(out[0]), int(out[1]), int(out[2])


class Context:
    """Owns a ``specs_ctx`` on one CUDA device."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        h = _vp()
        _check(self._lib.specs_create(C.byref(h), int(device)), "specs_create")
        self._h = h
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.specs_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- small accessors
    def set_engine(self, engine: int):
        _check(self._lib.specs_set_engine(self._h, int(engine)), "specs_set_engine")

    def set_accum_chunk(self, k_elements: int):
        _check(self._lib.specs_set_accum_chunk(self._h, int(k_elements)), "specs_set_accum_chunk")

    def set_tile_lead(self, tiles: int):
        _check(self._lib.specs_set_tile_lead(self._h, int(tiles)), "specs_set_tile_lead")

    def sm_count(self) -> int:
        return int(self._lib.specs_sm_count(self._h))

    def score_workspace_bytes(self, rows: int, d: int, V: int) -> int:
        return int(self._lib.specs_score_workspace_bytes(self._h, rows, d, V))

    def probe_wait_expiry(self, limit_us: int):
        _check(self._lib.specs_probe_wait_expiry(self._h, int(limit_us), self._s()), "specs_probe_wait_expiry")

    def set_timing(self, enabled: bool):
        _check(self._lib.specs_set_timing(self._h, 1 if enabled else 0), "specs_set_timing")

    def pause_timing(self):
        _check(self._lib.specs_set_timing(self._h, 0), "specs_set_timing")

    def resume_timing(self):
        _check(self._lib.specs_set_timing(self._h, 2), "specs_set_timing")

    def score_kernel_ms(self):
        n = _i32(0)
        ms = float(self._lib.specs_score_kernel_ms(self._h, C.byref(n)))
        return ms, int(n.value)

    def device_status(self, raise_on_error: bool = False) -> int:
        bits = C.c_uint32(0)
        st = self._lib.specs_device_status(self._h, C.byref(bits), self._s())
        if raise_on_error:
            _check(st, "specs_device_status")
        return int(bits.value)

    def _a(self, t, dtype, count, name):
        return device_arg(t, dtype, count, self.device, name)

    def _s(self):
        return _stream(self.device)

    # -- the calls of the path (same names as the C ABI)
    def specs_score_blocks(self, hidden, w_vocab, token_ids, block_offsets, tok_logprob,
                           blk_logprob=None, blk_logprob_f64=None, workspace=None):
        rows, d = hidden.shape
        V = w_vocab.shape[0]
        B = block_offsets.shape[0] - 1
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        a = self._a
        _check(self._lib.specs_score_blocks(
            self._h, a(hidden, "bf16", rows * d, "hidden"), a(w_vocab, "bf16", V * w_vocab.shape[1], "w_vocab"),
            a(token_ids, "i32", rows, "token_ids"), a(block_offsets, "i64", B + 1, "block_offsets"), rows, d, V, B,
            a(tok_logprob, "f32", rows, "tok_logprob"), a(blk_logprob, "f32", B, "blk_logprob"),
            a(blk_logprob_f64, "f64", B, "blk_logprob_f64"), a(workspace, "u8", 0, "workspace"), ws_bytes,
            self._s()), "specs_score_blocks")

    def specs_block_sums(self, per_token, block_offsets, out=None, out_f64=None):
        B = block_offsets.shape[0] - 1
        a = self._a
        _check(self._lib.specs_block_sums(self._h, a(per_token, "f32", 0, "per_token"),
                                          a(block_offsets, "i64", B + 1, "block_offsets"), B, a(out, "f32", B, "out"),
                                          a(out_f64, "f64", B, "out_f64"), self._s()), "specs_block_sums")

    def specs_subsample(self, blk_lp_target, blk_lp_gen, reward, cand_offsets, beta, uniforms, chosen,
                        weights=None, tau=float("nan"), accept=None):
        import torch
        P = cand_offsets.shape[0] - 1
        f64 = blk_lp_target is not None and blk_lp_target.dtype == torch.float64
        if blk_lp_gen is not None and (blk_lp_gen.dtype == torch.float64) != f64:
            raise TypeError("target and generator block log-probs must have the same dtype")
        fn = self._lib.specs_subsample_f64 if f64 else self._lib.specs_subsample
        a, lp = self._a, ("f64" if f64 else "f32")
        B = 0 if reward is None else reward.numel()
        _check(fn(self._h, a(blk_lp_target, lp, B, "blk_lp_target"), a(blk_lp_gen, lp, B, "blk_lp_gen"),
                  a(reward, "f32", 0, "reward"), a(cand_offsets, "i32", P + 1, "cand_offsets"), P, float(beta),
                  a(uniforms, "f32", B, "uniforms"), a(chosen, "i32", P, "chosen"), a(weights, "f32", B, "weights"),
                  float(tau), a(accept, "u8", P, "accept"), self._s()), "specs_subsample")

    def specs_accept(self, reward, cand_offsets, tau, accept):
        P = cand_offsets.shape[0] - 1
        a = self._a
        _check(self._lib.specs_accept(self._h, a(reward, "f32", 0, "reward"),
                                      a(cand_offsets, "i32", P + 1, "cand_offsets"), P, float(tau),
                                      a(accept, "u8", P, "accept"), self._s()), "specs_accept")

    def specs_score_partials(self, hidden, w_shard, token_ids, id_offset, partials, workspace):
        """Per-row (max, sum, logit) of one vocabulary shard; partials float32 [rows, 4] out."""
        rows, d = hidden.shape
        _check(self._lib.specs_score_partials(
            self._h, _ptr(hidden), _ptr(w_shard), _ptr(token_ids), int(id_offset), rows, d, w_shard.shape[0],
            _ptr(partials), _ptr(workspace), workspace.numel() * workspace.element_size(), self._s()),
            "specs_score_partials")

    def specs_merge_partials(self, partials, token_ids, V, tok_logprob):
        """Fold the shards' partials float32 [shards, rows, 4] into log pi_target of the drafted ids."""
        shards, rows = partials.shape[0], partials.shape[1]
        _check(self._lib.specs_merge_partials(self._h, _ptr(partials), shards, rows, _ptr(token_ids), int(V),
                                              _ptr(tok_logprob), self._s()), "specs_merge_partials")

    def specs_quantize_rows_e4m3(self, x_bf16, codes, scale):
        """Row-scaled E4M3 quantisation of a bf16 matrix [n, d]: codes uint8 [n, d], scale float32 [n]."""
        n, d = x_bf16.shape
        _check(self._lib.specs_quantize_rows_e4m3(self._h, _ptr(x_bf16), n, d, _ptr(codes), _ptr(scale), self._s()),
               "specs_quantize_rows_e4m3")

    def score_workspace_bytes_fp8(self, rows: int, d: int, V: int) -> int:
        return int(self._lib.specs_score_workspace_bytes_fp8(self._h, rows, d, V))

    def specs_score_blocks_fp8(self, hidden_q, hidden_scale, w_q, w_scale, token_ids, block_offsets, tok_logprob,
                               blk_logprob=None, blk_logprob_f64=None, workspace=None):
        rows, d = hidden_q.shape
        V = w_q.shape[0]
        B = block_offsets.shape[0] - 1
        _check(self._lib.specs_score_blocks_fp8(
            self._h, _ptr(hidden_q), _ptr(hidden_scale), _ptr(w_q), _ptr(w_scale), _ptr(token_ids),
            _ptr(block_offsets), rows, d, V, B, _ptr(tok_logprob), _ptr(blk_logprob), _ptr(blk_logprob_f64),
            _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(), self._s()),
            "specs_score_blocks_fp8")

    def beam_step_fp8_workspace_bytes(self, rows: int, d: int, V: int) -> int:
        return int(self._lib.specs_beam_step_fp8_workspace_bytes(self._h, rows, d, V))

    def specs_beam_step_fp8(self, hidden, w_q, w_scale, token_ids, block_offsets, cand_offsets, gen_tok_logprob, reward,
                            uniforms, beta, tau, tok_logprob, blk_logprob_f64, gen_blk_logprob_f64, weights, chosen,
                            accept, workspace):
        """The whole step with the 8-bit head: quantise the hidden states, score, finish."""
        rows, d = hidden.shape
        V = w_q.shape[0]
        B = block_offsets.shape[0] - 1
        P = cand_offsets.shape[0] - 1
        _check(self._lib.specs_beam_step_fp8(
            self._h, _ptr(hidden), _ptr(w_q), _ptr(w_scale), _ptr(token_ids), _ptr(block_offsets), _ptr(cand_offsets),
            _ptr(gen_tok_logprob), _ptr(reward), _ptr(uniforms), rows, d, V, B, P, float(beta), float(tau),
            _ptr(tok_logprob), _ptr(blk_logprob_f64), _ptr(gen_blk_logprob_f64), _ptr(weights), _ptr(chosen),
            _ptr(accept), _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
            self._s()), "specs_beam_step_fp8")

    def specs_prm_rewards(self, prm_hidden, block_offsets, w_head, bias, reward):
        """Value head of the PRM on each block's last hidden state, logistic link; reward float32 [B] out."""
        B = block_offsets.shape[0] - 1
        _check(self._lib.specs_prm_rewards(self._h, _ptr(prm_hidden), _ptr(block_offsets), B, prm_hidden.shape[1],
                                           _ptr(w_head), float(bias), _ptr(reward), self._s()), "specs_prm_rewards")

    def specs_select(self, blk_lp_target, blk_lp_gen, reward, mask, cand_offsets, beta, uniforms, select_rule,
                     score_flags, switch_rule, tau, chosen, weights=None, flag=None):
        """Selection with the paper's variants; block log-probabilities are float64 tensors."""
        P = cand_offsets.shape[0] - 1
        a = self._a
        B = 0 if reward is None else reward.numel()
        _check(self._lib.specs_select(
            self._h, a(blk_lp_target, "f64", B, "blk_lp_target"), a(blk_lp_gen, "f64", B, "blk_lp_gen"),
            a(reward, "f32", 0, "reward"), a(mask, "u8", B, "mask"), a(cand_offsets, "i32", P + 1, "cand_offsets"),
            P, float(beta), a(uniforms, "f32", B, "uniforms"), int(select_rule), int(score_flags), int(switch_rule),
            float(tau), a(chosen, "i32", P, "chosen"), a(weights, "f32", B, "weights"), a(flag, "u8", P, "flag"),
            self._s()), "specs_select")

    def specs_beam_step(self, hidden, w_vocab, token_ids, block_offsets, cand_offsets, gen_tok_logprob, reward,
                        uniforms, beta, tau, tok_logprob, blk_logprob_f64, gen_blk_logprob_f64, weights, chosen,
                        accept, workspace):
        """The whole step on device tensors as one chain of launches (scoring, merge, second pass, finish)."""
        rows, d = hidden.shape
        V = w_vocab.shape[0]
        B = block_offsets.shape[0] - 1
        P = cand_offsets.shape[0] - 1
        a = self._a
        _check(self._lib.specs_beam_step(
            self._h, a(hidden, "bf16", rows * d, "hidden"), a(w_vocab, "bf16", V * w_vocab.shape[1], "w_vocab"),
            a(token_ids, "i32", rows, "token_ids"), a(block_offsets, "i64", B + 1, "block_offsets"),
            a(cand_offsets, "i32", P + 1, "cand_offsets"), a(gen_tok_logprob, "f32", rows, "gen_tok_logprob"),
            a(reward, "f32", B, "reward"), a(uniforms, "f32", B, "uniforms"), rows, d, V, B, P, float(beta),
            float(tau), a(tok_logprob, "f32", rows, "tok_logprob"), a(blk_logprob_f64, "f64", B, "blk_logprob_f64"),
            a(gen_blk_logprob_f64, "f64", B, "gen_blk_logprob_f64"), a(weights, "f32", B, "weights"),
            a(chosen, "i32", P, "chosen"), a(accept, "u8", P, "accept"), a(workspace, "u8", 0, "workspace"),
            0 if workspace is None else workspace.numel() * workspace.element_size(), self._s()), "specs_beam_step")

    def beam_step_dual_workspace_bytes(self, rows: int, d_target: int, d_gen: int, V: int) -> int:
        return int(self._lib.specs_beam_step_dual_workspace_bytes(self._h, rows, d_target, d_gen, V))

    def specs_beam_step_dual(self, hidden_target, w_target, hidden_gen, w_gen, token_ids, block_offsets, cand_offsets,
                             reward, uniforms, beta, tau, tok_logprob, gen_tok_logprob, blk_logprob_f64,
                             gen_blk_logprob_f64, weights, chosen, accept, workspace, chosen_ids=None,
                             chosen_len=None):
        """The step with both LM heads computed on the device (generator pass, target pass, finish kernel)."""
        rows, d_t = hidden_target.shape
        d_g = hidden_gen.shape[1]
        V = w_target.shape[0]
        B = block_offsets.shape[0] - 1
        P = cand_offsets.shape[0] - 1
        stride = 0 if chosen_ids is None else chosen_ids.shape[1]
        _check(self._lib.specs_beam_step_dual(
            self._h, _ptr(hidden_target), _ptr(w_target), d_t, _ptr(hidden_gen), _ptr(w_gen), d_g, _ptr(token_ids),
            _ptr(block_offsets), _ptr(cand_offsets), _ptr(reward), _ptr(uniforms), rows, V, B, P, float(beta),
            float(tau), _ptr(tok_logprob), _ptr(gen_tok_logprob), _ptr(blk_logprob_f64), _ptr(gen_blk_logprob_f64),
            _ptr(weights), _ptr(chosen), _ptr(accept), _ptr(chosen_ids), _ptr(chosen_len), stride, _ptr(workspace),
            0 if workspace is None else workspace.numel() * workspace.element_size(), self._s()),
            "specs_beam_step_dual")

    def specs_gather_chosen(self, token_ids, block_offsets, cand_offsets, chosen, chosen_ids, chosen_len):
        P = cand_offsets.shape[0] - 1
        _check(self._lib.specs_gather_chosen(self._h, _ptr(token_ids), _ptr(block_offsets), _ptr(cand_offsets),
                                             _ptr(chosen), P, _ptr(chosen_ids), _ptr(chosen_len),
                                             chosen_ids.shape[1], self._s()), "specs_gather_chosen")

    def specs_beam_step_host(self, h_hidden, w_vocab, h_token_ids, h_block_offsets, h_cand_offsets,
                             h_gen_tok_logprob, h_reward, h_uniforms, beta, tau,
                             h_tok_logprob, h_blk_logprob, h_weights, h_chosen, h_accept):
        """Host tensors/arrays in, host tensors/arrays out; ``w_vocab`` is a device tensor."""
        rows, d = h_hidden.shape
        V = w_vocab.shape[0]
        B = h_block_offsets.shape[0] - 1
        P = h_cand_offsets.shape[0] - 1
        _check(self._lib.specs_beam_step_host(
            self._h, _ptr(h_hidden), _ptr(w_vocab), _ptr(h_token_ids), _ptr(h_block_offsets), _ptr(h_cand_offsets),
            _ptr(h_gen_tok_logprob), _ptr(h_reward), _ptr(h_uniforms), rows, d, V, B, P, float(beta), float(tau),
            _ptr(h_tok_logprob), _ptr(h_blk_logprob), _ptr(h_weights), _ptr(h_chosen), _ptr(h_accept), self._s()),
            "specs_beam_step_host")

    def specs_beam_step_host_submit(self, h_hidden, w_vocab, h_token_ids, h_block_offsets, h_cand_offsets,
                                    h_gen_tok_logprob, h_reward, h_uniforms, beta, tau,
                                    h_tok_logprob, h_blk_logprob, h_weights, h_chosen, h_accept) -> int:
        """Enqueue one host-buffer step and return its ticket; the outputs are filled by ``..._wait(ticket)``.
        The host arrays must stay alive and unchanged until then."""
        rows, d = h_hidden.shape
        V = w_vocab.shape[0]
        B = h_block_offsets.shape[0] - 1
        P = h_cand_offsets.shape[0] - 1
        ticket = _i32(0)
        _check(self._lib.specs_beam_step_host_submit(
            self._h, _ptr(h_hidden), _ptr(w_vocab), _ptr(h_token_ids), _ptr(h_block_offsets), _ptr(h_cand_offsets),
            _ptr(h_gen_tok_logprob), _ptr(h_reward), _ptr(h_uniforms), rows, d, V, B, P, float(beta), float(tau),
            _ptr(h_tok_logprob), _ptr(h_blk_logprob), _ptr(h_weights), _ptr(h_chosen), _ptr(h_accept), self._s(),
            C.byref(ticket)), "specs_beam_step_host_submit")
        return int(ticket.value)

    def specs_beam_step_host_wait(self, ticket: int):
        _check(self._lib.specs_beam_step_host_wait(self._h, int(ticket)), "specs_beam_step_host_wait")


class Policy(C.Structure):
    """Mirror of ``specs_policy``."""
    _fields_ = [("policy", _i32), ("sticky", _i32), ("target_len", _i64), ("max_steps", _i64), ("p_target", _f32)]


class Controller:
    """Owns a ``specs_controller`` (host-side Algorithm 1 state for P problems); numpy arrays in and out."""

    def __init__(self, P: int, policy: int = POLICY_SPECS, target_len: int = 1024, sticky: bool = False,
                 p_target: float = 0.5, max_steps: int = 1 << 30):
        self._lib = load_library()
        self.P = int(P)
        self.policy = int(policy)
        pol = Policy(int(policy), int(bool(sticky)), int(target_len), int(max_steps), float(p_target))
        h = _vp()
        _check(self._lib.specs_controller_create(C.byref(h), self.P, C.cast(C.byref(pol), _vp)),
               "specs_controller_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.specs_controller_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def generators(self) -> np.ndarray:
        out = np.empty(self.P, np.int32)
        _check(self._lib.specs_controller_generators(self._h, _ptr(out)), "specs_controller_generators")
        return out

    def advance(self, chosen, flag, chosen_len, uniforms=None):
        chosen = np.ascontiguousarray(chosen, np.int32)
        flag = np.ascontiguousarray(flag, np.uint8)
        chosen_len = np.ascontiguousarray(chosen_len, np.int64)
        uniforms = None if uniforms is None else np.ascontiguousarray(uniforms, np.float32)
        _check(self._lib.specs_controller_advance(self._h, _ptr(chosen), _ptr(flag), _ptr(chosen_len),
                                                  _ptr(uniforms)), "specs_controller_advance")

    def appended(self) -> np.ndarray:
        """Per problem: did the last ``advance`` append the selected block?"""
        out = np.empty(self.P, np.uint8)
        _check(self._lib.specs_controller_appended(self._h, _ptr(out)), "specs_controller_appended")
        return out

    def stats(self) -> dict:
        out = {k: np.empty(self.P, np.int64) for k in ("length", "steps", "target_steps", "target_calls")}
        _check(self._lib.specs_controller_stats(self._h, *[_ptr(v) for v in out.values()]),
               "specs_controller_stats")
        return out


NOALLOC_SCRATCH_BYTES = 8 << 20


def specs_score_blocks_noalloc(hidden, w_vocab, token_ids, block_offsets, tok_logprob,
                               blk_logprob=None, blk_logprob_f64=None, status_word=None):
    """Context-free, allocation-free scoring on the current CUDA device (see specs.h).

    For hosts that cannot call cudaMalloc: the kernel's scratch is a fixed array inside the
    library, shared by all calls on the device, so calls must not overlap on the GPU and
    problems beyond the fixed size raise SpecsError(SPECS_ERR_LIMIT).
    """
    rows, d = hidden.shape
    V = w_vocab.shape[0]
    B = block_offsets.shape[0] - 1
    _check(load_library().specs_score_blocks_noalloc(
        _ptr(hidden), _ptr(w_vocab), _ptr(token_ids), _ptr(block_offsets), rows, d, V, B, _ptr(tok_logprob),
        _ptr(blk_logprob), _ptr(blk_logprob_f64), _ptr(status_word), _stream()), "specs_score_blocks_noalloc")


# ---------------------------------------------------------------------------- torch helpers (marshalling only)

def bf16_bits_to_device(bits: np.ndarray, device="cuda"):
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 tensor on the device, bit for bit."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_bits_to_pinned(bits: np.ndarray):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).pin_memory()
    return t.view(torch.bfloat16)
