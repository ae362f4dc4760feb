#!/usr/bin/env python
"""Benchmark of the block-scoring step: scored draft tokens per second.

One *step* is one pass of the whole hot path over one batch of synthetic input: LM-head scoring of
every drafted token (tcgen05 kernel, with its second pass over re-scored rows), the merge of the
vocabulary splits, and one kernel that sums target and generator log-probabilities per block and
runs SubSample with the switch test (specs_beam_step).
The headline workload is the 7B-target-shaped single step (1 problem, 16 blocks of 64 tokens,
d = 3584, V = 151936); the other configurations are measured after it and reported under
"per_config".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank scores its own replica
of the batch; there is no data-path collective, so scaling is weak.
`--impl reference` times the CPU oracle on the host cores on a bounded sample.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "scored draft tokens/sec (LM-head logprob+SubSample); % of B200 bf16 tensor peak"
UNIT = "tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (read + write) of one launch of the first-pass scoring kernel, by workload, from hardware
# counters of an earlier capture of the same kernel; absent (null in the output) where none was taken
# or the kernel has changed since.
DRAM_TRAFFIC_BYTES = {
    "step7b": 1.0981e9 + 4.2e6,
    "batched": 12.16e9 + 9.1e6,
    "dual_target": 24.485e9 + 16.3e6,
    "stress": 42.67e9 + 19.5e6,
}

PER_CONFIG = ("batched", "dual_draft", "dual_target", "stress", "tiny")
SEVEN_B_SHAPED = ("step7b", "batched", "dual_target")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        out = {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
        # the SM clock the sustained peak was measured at (boards of this machine settle at different clocks under
        # the same power limit, so a sustained figure is also compared per MHz)
        mhz = (p.get("clocks_under_load") or {}).get("sm_mhz_median")
        if mhz:
            out["sustained_sm_mhz"] = float(mhz)
        return out
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clock, throttle reasons and power through NVML every few milliseconds (read-only)."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.002):
        self.t, self.mhz, self.bits, self.watts = [], [], [], []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
        self._period = period_s

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                watts = nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0
                self.t.append(time.perf_counter())
                self.mhz.append(mhz)
                self.bits.append(bits)
                self.watts.append(watts)
            except Exception:
                pass
            self._stop.wait(self._period)

    def start(self):
        if self._nv is not None and self._thread is None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def window(self, t0: float, t1: float) -> dict:
        """Summary of the samples taken while the host was between t0 and t1 (perf_counter seconds)."""
        idx = [i for i, t in enumerate(self.t) if t0 <= t <= t1]
        where = "inside the timed region"
        if not idx and self.t:
            # a region shorter than the sampling period: the sample nearest to its middle
            mid = 0.5 * (t0 + t1)
            idx = [min(range(len(self.t)), key=lambda i: abs(self.t[i] - mid))]
            where = "nearest to the timed region (none fell inside)"
        if not idx:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "where": "no NVML"}
        bits = 0
        for i in idx:
            bits |= self.bits[i]
        capped = sum(1 for i in idx if self.bits[i] & 0x4)
        return {"sm_mhz": float(np.median([self.mhz[i] for i in idx])),
                "sm_mhz_min": int(min(self.mhz[i] for i in idx)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(name for bit, name in self.REASONS.items() if bits & bit),
                "samples": len(idx), "sw_power_cap_samples": capped,
                "power_w_max": max(self.watts[i] for i in idx), "where": where}


def regime_of(clocks: dict) -> str:
    """Which measured peak a timed region is compared with, from what was observed during it: the sustained
    (power-limited) figure when the power cap was active or the SM clock sat well below its maximum, the
    burst figure otherwise."""
    if clocks.get("samples", 0) == 0 or clocks.get("sm_mhz") is None:
        return "burst"
    if clocks.get("sw_power_cap_samples", 0) * 2 >= clocks["samples"]:
        return "sustained"
    if clocks.get("sm_max_mhz") and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"]:
        return "sustained"
    return "burst"


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            pass
    return local_rank


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def time_oracle_sample(x, sample_blocks: int, beta: float, tau: float):
    """Times the CPU oracle, as it stands, on the first `sample_blocks` whole blocks of the batch."""
    from oracle import specs_oracle as O
    nb = min(sample_blocks, x.blocks)
    rows = int(x.block_offsets[nb])
    cand = np.array([0, nb], dtype=np.int32)
    t0 = time.perf_counter()
    O.beam_step(x.hidden[:rows], x.w_vocab, x.token_ids[:rows], x.block_offsets[:nb + 1], cand,
                x.draft_tok_logprob[:rows], x.reward[:nb], beta, x.uniforms[:nb], tau)
    dt = time.perf_counter() - t0
    return rows, dt


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    from paper_2506_15733_b200 import inputs
    x = inputs.make_step_inputs(cfg)
    beta, tau = cfg.betas[0], cfg.taus[0]
    blocks = args.oracle_blocks
    for _ in range(args.warmup):
        time_oracle_sample(x, blocks, beta, tau)
    total_rows, total_t = 0, 0.0
    for _ in range(args.steps):
        rows, dt = time_oracle_sample(x, blocks, beta, tau)
        total_rows += rows
        total_t += dt
    value = total_rows / total_t
    cores = oracle_threads()
    sample = (f"first {blocks} whole blocks ({total_rows // max(args.steps, 1)} rows) of {cfg.name} per step, "
              f"full vocabulary, fp64 numpy oracle incl. bf16->fp64 decode of W")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg, x, beta, tau, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(cfg, x, beta, tau, world):
    """The `config` object of the JSON line (the same keys for both arms)."""
    return {"workload": cfg.name, "rows": x.rows, "blocks": x.blocks, "problems": cfg.problems, "d": cfg.d,
            "V": cfg.vocab, "beta": beta, "tau": tau,
            "l2": f"inputs exceed L2 (W_vocab {cfg.vocab * cfg.d * 2 / 1e9:.2f} GB vs 126 MB); no flush"
                  if cfg.vocab * cfg.d * 2 > 126e6 else "inputs fit L2 (latency case); no flush",
            "parallelism": f"replicas x{world}, no collective"}


class Workload:
    """One configuration resident on the device: inputs, outputs, workspace, and the step that is timed."""

    def __init__(self, ctx, cfg, x, dev, fp8=False):
        import torch
        from paper_2506_15733_b200 import binding
        self.ctx, self.cfg, self.x, self.dev, self.fp8 = ctx, cfg, x, dev, fp8
        rows, B, P, d, V = x.rows, x.blocks, cfg.problems, cfg.d, cfg.vocab
        self.rows, self.B, self.P, self.d, self.V = rows, B, P, d, V
        t = lambda a: torch.from_numpy(a).to(dev)
        self.hidden = binding.bf16_bits_to_device(x.hidden, dev)
        self.w_vocab = binding.bf16_bits_to_device(x.w_vocab, dev)
        self.ids, self.boff, self.coff = t(x.token_ids), t(x.block_offsets), t(x.cand_offsets)
        self.draft, self.reward, self.uni = t(x.draft_tok_logprob), t(x.reward), t(x.uniforms)
        self.tok = torch.empty(rows, dtype=torch.float32, device=dev)
        self.blk64 = torch.empty(B, dtype=torch.float64, device=dev)
        self.gen64 = torch.empty(B, dtype=torch.float64, device=dev)
        self.wts = torch.empty(B, dtype=torch.float32, device=dev)
        self.chosen = torch.empty(P, dtype=torch.int32, device=dev)
        self.accept = torch.empty(P, dtype=torch.uint8, device=dev)
        self.plan = binding.score_plan(rows, d, V, ctx.sm_count())
        two_pass = self.plan["k_blocks"] > self.plan["chunk_kblocks"] and self.plan["row_tiles"] > 1
        # score tiles; merge of the vocabulary splits; second pass (adaptive chunks only); finish (block sums,
        # SubSample + switch)
        # (tiny steps without a second pass merge inside the finish kernel: two launches)
        fused_merge = not two_pass and rows * max(self.plan["split_full"], self.plan["split_rem"]) <= 2048
        self.launches_per_step = 4 if two_pass else (2 if fused_merge else 3)
        if fp8:
            self.w_q = torch.empty((V, d), dtype=torch.uint8, device=dev)
            self.w_s = torch.empty(V, dtype=torch.float32, device=dev)
            ctx.specs_quantize_rows_e4m3(self.w_vocab, self.w_q, self.w_s)   # the weight is quantised once
            self.ws = torch.empty(ctx.beam_step_fp8_workspace_bytes(rows, d, V), dtype=torch.uint8, device=dev)
            self.launches_per_step += 1                       # quantise the hidden states
        else:
            self.ws = torch.empty(ctx.score_workspace_bytes(rows, d, V), dtype=torch.uint8, device=dev)

    def step(self, beta, tau):
        c = self.ctx
        if self.fp8:
            c.specs_beam_step_fp8(self.hidden, self.w_q, self.w_s, self.ids, self.boff, self.coff, self.draft,
                                  self.reward, self.uni, beta, tau, self.tok, self.blk64, self.gen64, self.wts,
                                  self.chosen, self.accept, self.ws)
        else:
            c.specs_beam_step(self.hidden, self.w_vocab, self.ids, self.boff, self.coff, self.draft, self.reward,
                              self.uni, beta, tau, self.tok, self.blk64, self.gen64, self.wts, self.chosen,
                              self.accept, self.ws)

    def flops(self):
        return 2.0 * self.rows * self.d * self.V


def timed_leg(wl, ranks, sampler, steps, beta, tau, time_every=1):
    """`steps` steps bracketed by a barrier + synchronize on both sides, timed with CUDA events on the launching
    stream: one event per step boundary (median and minimum step time) and the library's own events around
    the scoring kernel on every `time_every`-th step."""
    import torch
    ctx = wl.ctx

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ctx.set_timing(time_every == 1)
    barrier()
    t0 = time.perf_counter()
    ev[0].record()
    for k in range(steps):
        timed = time_every > 1 and k % time_every == 0
        if timed:
            ctx.resume_timing()
        wl.step(beta, tau)
        if timed:
            ctx.pause_timing()
        ev[k + 1].record()
    barrier()
    t1 = time.perf_counter()
    total_ms = ev[0].elapsed_time(ev[steps])
    step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(steps)]
    kernel_ms, kernel_calls = ctx.score_kernel_ms()
    ctx.set_timing(False)
    return {"total_ms": total_ms, "step_ms_median": float(np.median(step_ms)), "step_ms_min": float(min(step_ms)),
            "kernel_ms": kernel_ms, "kernel_calls": kernel_calls, "clocks": sampler.window(t0, t1), "steps": steps}


def roofline_fields(flops, kernel_ms, clocks, peaks, nominal, dtype_name):
    """Achieved tensor throughput of the scoring kernel against the measured peak of the regime the clocks
    showed (burst or power-limited), with the other two denominators beside it."""
    achieved = flops / (kernel_ms * 1e-3) / 1e12 if kernel_ms and kernel_ms > 0 else None
    kind = regime_of(clocks)
    peak = peaks["bf16_tflops_sustained"] if kind == "sustained" else peaks["bf16_tflops"]
    frac = lambda p: achieved / p if achieved else None
    at_equal_clock = None
    if achieved and kind == "sustained" and clocks.get("sm_mhz") and peaks.get("sustained_sm_mhz"):
        # time x clock: this kernel's throughput per MHz against the sustained peak's per MHz
        at_equal_clock = (achieved / clocks["sm_mhz"]) / (peaks["bf16_tflops_sustained"] / peaks["sustained_sm_mhz"])
    return {"achieved": achieved, "frac_of_sustained_at_equal_clock": at_equal_clock, "peak": peak, "unit": "TFLOP/s", "frac": frac(peak),
            "peak_kind": f"{dtype_name} {kind}, of {peaks['source']}: chosen from the clocks sampled during the timed "
                         f"region (median {clocks.get('sm_mhz')} MHz of {clocks.get('sm_max_mhz')}, power cap active in "
                         f"{clocks.get('sw_power_cap_samples', 0)} of {clocks.get('samples', 0)} samples)",
            "frac_of_burst": frac(peaks["bf16_tflops"]), "frac_of_sustained": frac(peaks["bf16_tflops_sustained"]),
            "frac_of_nominal": frac(nominal), "kernel_ms": kernel_ms, "flop_per_launch": flops,
            "sm_mhz": clocks.get("sm_mhz")}


def measure(wl, ranks, sampler, steps, warmup, beta, tau, peaks, nominal, dtype_name, world, time_every=1,
            sustain_s=2.0):
    """Warm-up, the timed region of exactly `steps` steps, and a sustained leg of at least `sustain_s` seconds."""
    for _ in range(warmup):
        wl.step(beta, tau)
    main = timed_leg(wl, ranks, sampler, steps, beta, tau, time_every)
    main["total_ms"] = ranks.max_over_ranks(main["total_ms"])
    out = {"value": wl.rows * world * steps / (main["total_ms"] * 1e-3), "ms_per_step": main["total_ms"] / steps,
           "step_ms_median": main["step_ms_median"], "step_ms_min": main["step_ms_min"], "steps": steps,
           "clocks": main["clocks"], "kernel_calls_timed": main["kernel_calls"],
           "roofline": roofline_fields(wl.flops(), main["kernel_ms"], main["clocks"], peaks, nominal, dtype_name),
           "tensor_tflops_whole_step": wl.flops() * steps / (main["total_ms"] * 1e-3) / 1e12}
    if sustain_s > 0:
        add_sustained(out, wl, ranks, sampler, beta, tau, peaks, nominal, dtype_name, sustain_s)
    return out


def add_sustained(out, wl, ranks, sampler, beta, tau, peaks, nominal, dtype_name, sustain_s=2.0):
    """The sustained leg: the same step in a loop of at least `sustain_s` seconds, under out["roofline"]."""
    n = max(5, int(math.ceil(sustain_s * 1e3 / max(out["ms_per_step"], 1e-3))))
    n = min(n, 20000)
    leg = timed_leg(wl, ranks, sampler, n, beta, tau, max(1, n // 200))
    r = roofline_fields(wl.flops(), leg["kernel_ms"], leg["clocks"], peaks, nominal, dtype_name)
    out["roofline"]["sustained"] = {
        "steps": n, "seconds": leg["total_ms"] * 1e-3, "ms_per_step": leg["total_ms"] / n,
        "tokens_per_s": wl.rows * n / (leg["total_ms"] * 1e-3), "kernel_ms": leg["kernel_ms"],
        "achieved": r["achieved"], "peak": peaks["bf16_tflops_sustained"], "frac": r["frac_of_sustained"],
        "frac_at_equal_clock": r["frac_of_sustained_at_equal_clock"],
        "frac_of_burst": r["frac_of_burst"], "frac_of_nominal": r["frac_of_nominal"],
        "sm_mhz": leg["clocks"].get("sm_mhz"), "reasons": leg["clocks"].get("reasons"),
        "regime_observed": regime_of(leg["clocks"]),
        "note": "a loop of at least two seconds, long enough for the board's power limit to set the clocks; "
                "against the measured sustained peak"}


def beta_2l_case(wl, cfg, tau):
    """The paper's heuristic beta = 2 L (Section 4.3; L read as the mean block length) on the same batch:
    not scored against anything, it shows the selection with reward and log-ratio of comparable size."""
    import torch
    L = float(np.diff(wl.x.block_offsets).mean()) if wl.B else 0.0
    beta = 2.0 * L
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wl.step(beta, tau)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        wl.step(beta, tau)
    e1.record()
    torch.cuda.synchronize()
    w = wl.wts.cpu().numpy().astype(np.float64)
    co = wl.x.cand_offsets
    top = [float(w[co[p]:co[p + 1]].max()) for p in range(wl.P) if co[p + 1] > co[p]]
    ess = [float(1.0 / np.square(w[co[p]:co[p + 1]]).sum()) for p in range(wl.P) if co[p + 1] > co[p]]
    return {"beta": beta, "ms_per_step": e0.elapsed_time(e1) / 3.0, "mean_largest_weight": float(np.mean(top)),
            "mean_effective_candidates": float(np.mean(ess)), "scored": False}


def e2e_leg(wl, ranks, steps, beta, tau, world):
    """The same metric through the host-buffer entry points: every step's inputs start in pinned host memory and
    its results end there, with the host<->device copies inside the timed region.  Two steps are kept in
    flight (submit k+1, then wait k), so that one step's copies run under the other's kernels."""
    import torch
    from paper_2506_15733_b200 import binding
    x, ctx = wl.x, wl.ctx
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_hidden = binding.bf16_bits_to_pinned(x.hidden)
    h_ids, h_boff, h_coff = pin(x.token_ids), pin(x.block_offsets), pin(x.cand_offsets)
    h_draft, h_reward, h_uni = pin(x.draft_tok_logprob), pin(x.reward), pin(x.uniforms)
    outs = []
    for _ in range(2):                                       # one set of pinned outputs per step in flight
        outs.append([torch.empty(wl.rows, dtype=torch.float32).pin_memory(),
                     torch.empty(wl.B, dtype=torch.float64).pin_memory(),
                     torch.empty(wl.B, dtype=torch.float32).pin_memory(),
                     torch.empty(wl.P, dtype=torch.int32).pin_memory(),
                     torch.empty(wl.P, dtype=torch.uint8).pin_memory()])
    nbytes = lambda *ts: int(sum(v.numel() * v.element_size() for v in ts))
    h2d = nbytes(h_hidden, h_ids, h_boff, h_coff, h_draft, h_reward, h_uni)
    d2h = nbytes(*outs[0])

    def submit(k):
        return ctx.specs_beam_step_host_submit(h_hidden, wl.w_vocab, h_ids, h_boff, h_coff, h_draft, h_reward,
                                               h_uni, beta, tau, *outs[k & 1])

    def run(n):
        ticket = submit(0)
        for k in range(1, n):
            nxt = submit(k)
            ctx.specs_beam_step_host_wait(ticket)            # step k-1's results are in host memory now
            ticket = nxt
        ctx.specs_beam_step_host_wait(ticket)

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    run(3)
    barrier()
    t0 = time.perf_counter()
    run(steps)
    barrier()
    dt = ranks.max_over_ranks(time.perf_counter() - t0)
    # the serial form of the same call (one step at a time), for comparison
    serial_n = max(3, steps // 4)
    t0 = time.perf_counter()
    for _ in range(serial_n):
        ctx.specs_beam_step_host(h_hidden, wl.w_vocab, h_ids, h_boff, h_coff, h_draft, h_reward, h_uni, beta, tau,
                                 *outs[0])
    barrier()
    dt_serial = time.perf_counter() - t0
    wl.step(beta, tau)
    torch.cuda.synchronize()
    assert torch.equal(outs[0][3].to(wl.dev), wl.chosen) and torch.equal(outs[0][0].to(wl.dev), wl.tok), \
        "host path disagrees with the device-resident step"
    return {"value": wl.rows * world * steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "copies_inside_timed_region": True,
            "api": "specs_beam_step_host_submit / specs_beam_step_host_wait, two steps in flight",
            "serial_value": wl.rows * world * serial_n / dt_serial,
            "note": "W_vocab is the model's weight and stays resident; every step's inputs come from pinned host "
                    "memory and its results return to it"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", default="step7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-blocks", type=int, default=16, help="whole blocks per CPU-oracle sample")
    ap.add_argument("--tile-lead", type=int, default=None,
                    help="pacing of the CTA pairs that stream the same W chunk, in vocabulary tiles (0: off; default: the library's)")
    ap.add_argument("--engine", default="auto", choices=["auto", "1cta", "2cta"],
                    help="tile shape of the scoring kernel: the planner's choice, single CTAs (128-row tiles) or CTA "
                         "pairs (256-row tiles)")
    ap.add_argument("--time-every", type=int, default=4,
                    help="record CUDA events around the scoring kernel on every K-th step of the timed region "
                         "(an event between two kernels of a step keeps the second from being set up early, "
                         "which costs the step about 8 us on the headline workload)")
    ap.add_argument("--fp8", action="store_true",
                    help="time the E4M3 variant instead (reduced precision: not the headline; W quantised once, "
                         "hidden states quantised inside every step)")
    ap.add_argument("--problems", type=int, default=None,
                    help="shrink the workload to this many problems (same recipe; for profiler captures, whose "
                         "size must stay small; the line's config then carries the reduced counts)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="measure the headline workload only")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second sustained legs")
    args = ap.parse_args()

    from paper_2506_15733_b200.replicas import Replicas
    ranks = Replicas.from_env()
    rank, local_rank, world = ranks.rank, ranks.local_rank, ranks.world
    if args.impl == "reference" and rank != 0:
        return                                               # rank 0 alone times the CPU oracle
    from paper_2506_15733_b200 import inputs
    cfg = inputs.CONFIGS[args.config]
    if args.problems is not None:
        cfg = inputs.scaled(cfg, problems=int(args.problems))

    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, cfg, rank)
        return

    args.steps = 1500 if args.steps is None else args.steps
    args.warmup = 50 if args.warmup is None else max(args.warmup, 3)

    import torch
    from paper_2506_15733_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scoring path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    ranks.init("nccl", torch.device(dev))
    sampler = ClockSampler(physical_gpu_index(local_rank)).start()   # runs from before the warm-up to the end

    peaks = load_peaks()
    nominal = NOMINAL_BF16_TFLOPS
    dtype_name = "bf16"
    if args.fp8:                                             # E4M3 runs at twice the bf16 rate
        peaks = {k: (2.0 * v if k.startswith("bf16") else v) for k, v in peaks.items()}   # (the clock is not doubled)
        peaks["source"] = "measured bf16 x 2 (nominal fp8 : bf16 ratio)" if peaks["source"] == "measured" else "fallback x 2"
        nominal, dtype_name = 2.0 * NOMINAL_BF16_TFLOPS, "fp8"
        args.no_e2e = True
    sustain_s = 0.0 if args.no_sustained else 2.0

    # the other configurations' inputs are drawn on a helper thread while the GPU is being timed
    todo = [] if (args.no_per_config or world > 1 or args.fp8) else [n for n in PER_CONFIG if n != cfg.name]
    drawn, draw_err = {}, []

    def draw_all():
        try:
            for name in todo:
                drawn[name] = inputs.make_step_inputs(inputs.CONFIGS[name])
        except Exception as e:                               # reported in the line, never silently dropped
            draw_err.append(repr(e))

    x = inputs.make_step_inputs(cfg)
    drawer = threading.Thread(target=draw_all, daemon=True)
    drawer.start()

    ctx = binding.Context(local_rank)
    if args.tile_lead is not None:
        ctx.set_tile_lead(args.tile_lead)
    if args.engine != "auto":
        ctx.set_engine(binding.ENGINE_TCGEN05_1CTA if args.engine == "1cta" else binding.ENGINE_TCGEN05_2CTA)
    beta, tau = cfg.betas[0], cfg.taus[0]
    wl = Workload(ctx, cfg, x, dev, fp8=args.fp8)
    head = measure(wl, ranks, sampler, args.steps, args.warmup, beta, tau, peaks, nominal, dtype_name, world,
                   args.time_every, 0.0)
    status_bits = ctx.device_status()
    # end to end with the same number of steps, before the sustained leg heats the board
    e2e = None if args.no_e2e else e2e_leg(wl, ranks, max(3, min(args.steps, 2000)), beta, tau, world)
    if sustain_s > 0:
        add_sustained(head, wl, ranks, sampler, beta, tau, peaks, nominal, dtype_name, sustain_s)
    extra_beta = beta_2l_case(wl, cfg, tau) if rank == 0 else None
    status_bits |= ctx.device_status()
    digests = x.digests() if rank == 0 else None

    # the other configurations, one after the other on the same context
    per_config = {}
    if todo:
        del wl
        torch.cuda.empty_cache()
        for name in todo:
            while name not in drawn and drawer.is_alive():
                time.sleep(0.05)                             # its inputs are still being drawn
            if name not in drawn:
                continue
            c2, x2 = inputs.CONFIGS[name], drawn.pop(name)
            b2, t2 = c2.betas[0], c2.taus[0]
            w2 = Workload(ctx, c2, x2, dev)
            est_ms = max(2.0 * x2.rows * c2.d * c2.vocab / 1.3e15 * 1e3, 0.02)
            steps2 = int(min(max(5, math.ceil(1000.0 / est_ms)), 2000))   # at least five steps and about a second
            m = measure(w2, ranks, sampler, steps2, 3, b2, t2, peaks, nominal, dtype_name, world, 1,
                        sustain_s if name != "tiny" else 0.0)
            entry = {"config": workload_config(c2, x2, b2, t2, world), "tokens_per_s": m["value"],
                     "ms_per_step": m["ms_per_step"], "step_ms_median": m["step_ms_median"],
                     "step_ms_min": m["step_ms_min"], "steps": steps2, "clocks": m["clocks"],
                     "gpu_launches_per_step": w2.launches_per_step,
                     "beta_2L": beta_2l_case(w2, c2, t2), "inputs_sha256": x2.digests()}
            entry["device_status"] = ctx.device_status()
            if name == "tiny":
                entry["note"] = "latency case (33 MFLOP, inputs fit L2): no roofline fraction"
            else:
                entry["roofline"] = m["roofline"] | {"bound": "tensor", "traffic": DRAM_TRAFFIC_BYTES.get(name)}
            per_config[name] = entry
            del w2, x2
            torch.cuda.empty_cache()
    sampler.stop()
    drawer.join()

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        # (after the helper thread has finished drawing inputs, so that the oracle has the cores to itself)
        # repeat the sample until about ten seconds of CPU work have been timed
        n_rows, dt = time_oracle_sample(x, args.oracle_blocks, beta, tau)
        reps, total_rows, total_dt = 1, n_rows, dt
        while total_dt < 10.0 and reps < 64:
            n_rows, dt = time_oracle_sample(x, args.oracle_blocks, beta, tau)
            reps, total_rows, total_dt = reps + 1, total_rows + n_rows, total_dt + dt
        cpu = {"value": total_rows / total_dt, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": f"first {args.oracle_blocks} whole blocks ({n_rows} rows) of {cfg.name}, full vocabulary, "
                         f"{reps} times: {total_dt:.1f} s of fp64 numpy incl. bf16->fp64 decode of W"}

    if rank == 0:
        roofline = {"bound": "tensor",
                    "kernel": ("score_tiles_pair" if (args.engine == "2cta" or (args.engine == "auto" and
                                                       wl_plan_pair(binding, x, cfg, ctx))) else "score_tiles") +
                              ("_fp8_kernel" if args.fp8 else "_kernel")} | head["roofline"]
        # the table holds captures of the default launch configuration of the full workloads only
        default_launch = not args.fp8 and args.problems is None and args.engine == "auto" and args.tile_lead is None
        roofline["traffic"] = DRAM_TRAFFIC_BYTES.get(cfg.name) if default_launch else None
        roofline["kernel_calls_timed"] = head["kernel_calls_timed"]
        largest = per_config.get("dual_target")
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "step_ms_median": head["step_ms_median"],
                "step_ms_min": head["step_ms_min"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "e4m3" if args.fp8 else "bf16", "data": "synthetic",
                "config": workload_config(cfg, x, beta, tau, world),
                "clocks": head["clocks"], "e2e": e2e,
                "gpu_launches": launches_of(binding, x, cfg, ctx, args.fp8) * args.steps,
                "roofline": roofline, "cpu_baseline": cpu, "device_status": status_bits,
                "tensor_tflops_whole_step": head["tensor_tflops_whole_step"],
                "inputs": {"seed": cfg.seed, "sha256": digests}, "beta_2L": extra_beta,
                "largest_7b_shaped": None if not largest else
                    {"workload": "dual_target", "tokens_per_s": largest["tokens_per_s"],
                     "achieved_tflops": largest["roofline"]["achieved"], "frac": largest["roofline"]["frac"],
                     "peak_kind": largest["roofline"]["peak_kind"]},
                "per_config": per_config or None}
        if draw_err:
            line["per_config_error"] = draw_err
        print(json.dumps(line))
    ctx.close()
    ranks.shutdown()


def wl_plan_pair(binding, x, cfg, ctx) -> bool:
    return binding.score_plan(x.rows, cfg.d, cfg.vocab, ctx.sm_count())["cta_group"] == 2


def launches_of(binding, x, cfg, ctx, fp8) -> int:
    """Kernels of this library launched per step: score tiles, merge, finish, plus the second scoring pass
    when the plan has adaptive accumulation chunks, plus the quantisation of the hidden states for E4M3."""
    p = binding.score_plan(x.rows, cfg.d, cfg.vocab, ctx.sm_count())
    two_pass = p["k_blocks"] > p["chunk_kblocks"] and p["row_tiles"] > 1
    fused_merge = not two_pass and x.rows * max(p["split_full"], p["split_rem"]) <= 2048
    return (4 if two_pass else (2 if fused_merge else 3)) + (1 if fp8 else 0)


if __name__ == "__main__":
    main()
