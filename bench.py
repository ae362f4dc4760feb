#!/usr/bin/env python
"""Benchmark of the block-scoring step: scored draft tokens per second.

One *step* is one pass of the whole hot path over one batch of synthetic input:
LM-head scoring of every drafted token (tcgen05 kernel), then one kernel that merges
the vocabulary splits, sums target and generator log-probabilities per block and runs
SubSample with the switch test (specs_beam_step).
The default workload is the 7B-target-shaped single step (1 problem, 16 blocks of
64 tokens, d = 3584, V = 151936).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank scores
its own replica of the batch; there is no data-path collective, so scaling is weak.
`--impl reference` times the CPU oracle on the host cores on a bounded sample.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
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

# DRAM bytes (read + write) of one launch of the scoring kernel, from the ncu capture summarised
# under profiles/ (null until a capture for that workload exists).
NCU_TRAFFIC_BYTES = {"step7b": 1.0995e9 + 3.75e6}   # profiles/score_tiles_pair_kernel_step7b.md


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.power = [], set(), []
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
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None}


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
            "data": "synthetic", "config": {"workload": cfg.name, "rows": x.rows, "d": cfg.d, "V": cfg.vocab},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


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
    ap.add_argument("--time-every", type=int, default=1,
                    help="record CUDA events around the scoring kernel on every K-th step of the timed region")
    ap.add_argument("--fp8", action="store_true",
                    help="time the E4M3 variant instead (reduced precision: not the headline; W quantised once, "
                         "hidden states quantised inside every step)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()

    from paper_2506_15733_b200.replicas import Replicas
    ranks = Replicas.from_env()
    rank, local_rank, world = ranks.rank, ranks.local_rank, ranks.world
    if args.impl == "reference" and rank != 0:
        return                                               # rank 0 alone times the CPU oracle
    from paper_2506_15733_b200 import inputs
    cfg = inputs.CONFIGS[args.config]

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

    x = inputs.make_step_inputs(cfg)
    rows, B, P, d, V = x.rows, x.blocks, cfg.problems, cfg.d, cfg.vocab
    beta, tau = cfg.betas[0], cfg.taus[0]
    ctx = binding.Context(local_rank)
    if args.tile_lead is not None:
        ctx.set_tile_lead(args.tile_lead)

    # device-resident copies
    t = lambda a: torch.from_numpy(a).to(dev)
    hidden, w_vocab = binding.bf16_bits_to_device(x.hidden, dev), binding.bf16_bits_to_device(x.w_vocab, dev)
    ids, boff, coff = t(x.token_ids), t(x.block_offsets), t(x.cand_offsets)
    draft, reward, uni = t(x.draft_tok_logprob), t(x.reward), t(x.uniforms)
    tok = torch.empty(rows, dtype=torch.float32, device=dev)
    blk64 = torch.empty(B, dtype=torch.float64, device=dev)
    gen64 = torch.empty(B, dtype=torch.float64, device=dev)
    wts = torch.empty(B, dtype=torch.float32, device=dev)
    chosen = torch.empty(P, dtype=torch.int32, device=dev)
    accept = torch.empty(P, dtype=torch.uint8, device=dev)
    ws = torch.empty(ctx.score_workspace_bytes(rows, d, V), dtype=torch.uint8, device=dev)
    launches_per_step = 2   # score tiles; finish (split merge, target and generator block sums, SubSample + switch)

    def step():
        ctx.specs_beam_step(hidden, w_vocab, ids, boff, coff, draft, reward, uni, beta, tau, tok, blk64, gen64, wts,
                            chosen, accept, ws)

    if args.fp8:
        w_q = torch.empty((V, d), dtype=torch.uint8, device=dev)
        w_s = torch.empty(V, dtype=torch.float32, device=dev)
        ctx.specs_quantize_rows_e4m3(w_vocab, w_q, w_s)          # the weight is quantised once, outside the step
        ws = torch.empty(ctx.beam_step_fp8_workspace_bytes(rows, d, V), dtype=torch.uint8, device=dev)
        launches_per_step = 3   # quantise the hidden states; score tiles; finish
        args.no_e2e = True

        def step():  # noqa: F811
            ctx.specs_beam_step_fp8(hidden, w_q, w_s, ids, boff, coff, draft, reward, uni, beta, tau, tok, blk64, gen64,
                                    wts, chosen, accept, ws)

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    # A short burst first: 100 steps are over before the board's power limit pulls the clocks down, which shows
    # what the kernel does at full clocks; the long loop below is the sustained figure that is reported.
    burst_steps = min(100, args.steps)
    ctx.set_timing(True)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record()
    for _ in range(burst_steps):
        step()
    b1.record()
    barrier()
    burst_ms = b0.elapsed_time(b1) / burst_steps
    burst_kernel_ms, _ = ctx.score_kernel_ms()
    ctx.set_timing(False)
    time.sleep(0.2)

    every = max(1, args.time_every)
    ctx.set_timing(every == 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        barrier()
        e0.record()
        for k in range(args.steps):
            if every > 1 and k % every == 0:
                ctx.resume_timing()
            step()
            if every > 1 and k % every == 0:
                ctx.pause_timing()
        e1.record()
        barrier()
    total_ms = e0.elapsed_time(e1)
    kernel_ms, kernel_launches = ctx.score_kernel_ms()
    ctx.set_timing(False)
    status_bits = ctx.device_status()
    total_ms = ranks.max_over_ranks(total_ms)
    value = rows * world * args.steps / (total_ms * 1e-3)

    # end to end through the host-buffer entry point: pinned host inputs, H2D and D2H inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_hidden = binding.bf16_bits_to_pinned(x.hidden)
        h_ids, h_boff, h_coff = pin(x.token_ids), pin(x.block_offsets), pin(x.cand_offsets)
        h_draft, h_reward, h_uni = pin(x.draft_tok_logprob), pin(x.reward), pin(x.uniforms)
        o_tok = torch.empty(rows, dtype=torch.float32).pin_memory()
        o_blk = torch.empty(B, dtype=torch.float64).pin_memory()
        o_wts = torch.empty(B, dtype=torch.float32).pin_memory()
        o_cho = torch.empty(P, dtype=torch.int32).pin_memory()
        o_acc = torch.empty(P, dtype=torch.uint8).pin_memory()
        nbytes = lambda *ts: int(sum(v.numel() * v.element_size() for v in ts))
        h2d = nbytes(h_hidden, h_ids, h_boff, h_coff, h_draft, h_reward, h_uni)
        d2h = nbytes(o_tok, o_blk, o_wts, o_cho, o_acc)

        def host_step():
            ctx.specs_beam_step_host(h_hidden, w_vocab, h_ids, h_boff, h_coff, h_draft, h_reward, h_uni,
                                     beta, tau, o_tok, o_blk, o_wts, o_cho, o_acc)

        e2e_steps = max(3, min(args.steps, 300))
        for _ in range(3):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            host_step()           # synchronises its stream before returning
        barrier()
        dt = time.perf_counter() - t0
        dt = ranks.max_over_ranks(dt)
        assert torch.equal(o_cho.to(dev), chosen) and torch.equal(o_tok.to(dev), tok), "host path disagrees"
        e2e = {"value": rows * world * e2e_steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "note": "W_vocab is the model's weight and stays resident; the step's inputs come from pinned host memory"}

    if rank == 0:
        peaks = load_peaks()
        flops = 2.0 * rows * d * V
        achieved = flops / (kernel_ms * 1e-3) / 1e12 if kernel_ms > 0 else None
        plan = binding.score_plan(rows, d, V, ctx.sm_count())
        nominal = NOMINAL_BF16_TFLOPS
        if args.fp8:                                             # E4M3 runs at twice the bf16 rate
            peaks = {k: (2.0 * v if k.startswith("bf16") else v) for k, v in peaks.items()}
            peaks["source"] = "measured bf16 x 2 (nominal fp8 : bf16 ratio)" if peaks["source"] == "measured" else "fallback x 2"
            nominal = 2.0 * NOMINAL_BF16_TFLOPS
        peak = peaks["bf16_tflops_sustained"]
        roofline = {"bound": "tensor",
                    "kernel": ("score_tiles_pair" if plan["cta_group"] == 2 else "score_tiles") +
                              ("_fp8_kernel" if args.fp8 else "_kernel"), "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak if achieved else None,
                    "peak_kind": f"{'fp8' if args.fp8 else 'bf16'} sustained, of {peaks['source']} "
                                 "(kernel timed inside a long loop)",
                    "frac_of_burst": achieved / peaks["bf16_tflops"] if achieved else None,
                    "frac_of_nominal": achieved / nominal if achieved else None,
                    "kernel_ms": kernel_ms, "kernel_launches_timed": kernel_launches,
                    "flop_per_launch": flops, "traffic": None if args.fp8 else NCU_TRAFFIC_BYTES.get(cfg.name),
                    "burst": {"steps": burst_steps, "ms_per_step": burst_ms, "kernel_ms": burst_kernel_ms,
                              "achieved": flops / (burst_kernel_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                              "frac": flops / (burst_kernel_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                              "note": "first steps after warm-up, before the power limit lowers the clocks; "
                                      "against the measured burst peak"}}
        cpu = None
        if not args.no_cpu_baseline:
            # repeat the sample until about ten seconds of CPU work have been timed
            n_rows, dt = time_oracle_sample(x, args.oracle_blocks, beta, tau)
            reps, total_rows, total_dt = 1, n_rows, dt
            while total_dt < 10.0 and reps < 64:
                n_rows, dt = time_oracle_sample(x, args.oracle_blocks, beta, tau)
                reps, total_rows, total_dt = reps + 1, total_rows + n_rows, total_dt + dt
            cpu = {"value": total_rows / total_dt, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                   "sample": f"first {args.oracle_blocks} whole blocks ({n_rows} rows) of {cfg.name}, full vocabulary, "
                             f"{reps} times: {total_dt:.1f} s of fp64 numpy incl. bf16->fp64 decode of W"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "e4m3" if args.fp8 else "bf16", "data": "synthetic",
                "config": {"workload": cfg.name, "rows": rows, "blocks": B, "problems": P, "d": d, "V": V,
                           "beta": beta, "tau": tau, "l2": f"inputs exceed L2 (W_vocab {V * d * 2 / 1e9:.2f} GB vs 126 MB); no flush",
                           "parallelism": f"replicas x{world}, no collective"},
                "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "roofline": roofline, "cpu_baseline": cpu, "device_status": status_bits,
                "tensor_tflops_whole_step": flops * args.steps / (total_ms * 1e-3) / 1e12}
        print(json.dumps(line))
    ctx.close()
    ranks.shutdown()


if __name__ == "__main__":
    main()
