#!/usr/bin/env python
"""Benchmark: recursive invocations per second of the tagged-dataflow executor.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input:
lowered graph -> seed tokens -> all forward waves (tag push/pop, matching, batched
cells) -> loss head -> gradient waves -> parameter gradients (workloads 3-5), or
the forward pass alone (workloads 1-2).  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "recursive_invocations_per_sec"
UNIT = "invocations/s"
WORKLOAD_NAMES = {
    1: "config1: fib(n), 1024 calls, n~U[0,18], int64, packed path tags, forward",
    2: "config2: TreeRNN forward, 512 random binary trees, H=64, fp32",
    3: "config3: TreeRNN forward+backward, 8192 trees (lognormal leaves, median 18), H=300, vocab 21000, 5-class loss at every node",
    4: "config4: binary TreeLSTM forward+backward, 8192 trees (same size mix), H=300, vocab 21000, 5-class loss at every node",
    5: "config5: depth stress, TreeRNN H=256 fp32 forward+backward, 64 chains of depth 4096 + 16 perfect trees of 2^16 leaves",
}
# kernels of the library launched per step (memsets and copies not counted):
#   seed, scheduler | + 3 kernels that group the cells by height, operators, root gather | + loss head, loss sum, 4 list kernels, gradient waves, dW, db
#   bf16: + weight packing (TreeLSTM: + table packing); TreeLSTM: + dW_x, db_x, dE
KERNELS_PER_STEP = {"eval_int": 2, "eval_trees": 7, "eval_trees_tc": 8, "grad": 16, "grad_tc": 17, "grad_lstm": 19,
                    "grad_lstm_tc": 21}
CELL = {"treernn": "rnn", "treelstm": "lstm"}


def fib_iter(n):
    a, b = 0, 1
    for _ in range(n):
        a, b = b, a + b
    return a


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(names, p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- workloads
def load(k, seed, fib_batch=None):
    cfg = workloads.config(k, seed=seed, B=fib_batch) if (k == 1 and fib_batch) else workloads.config(k, seed=seed)
    if cfg["kind"] == "fib":
        cfg["N"] = int(sum(2 * fib_iter(int(n) + 1) - 1 for n in cfg["x"]))
    else:
        cfg["N"] = cfg["trees"].N
    return cfg


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu capture of the same kernel
# (profiles/persistent_kernels_config3.md); None where no capture of the current kernel exists
NCU_TRAFFIC_BYTES = {("rdf_backward_kernel", 3, None): 396.0e6, ("rdf_operator_kernel", 3, None): 297.0e6,
                     ("rdf_scheduler_kernel", 3, None): 10.8e6}

# fp32 FMA peak: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_step(cfg, sample):
    """One bounded sample of the workload on the CPU oracle; returns invocations processed."""
    from oracle import direct
    if cfg["kind"] == "fib":
        xs = cfg["x"][:sample]
        n = 0
        for v in xs:
            n += len(direct.fib_invocations(int(v))[1])
        return n
    tb = cfg["trees"]
    trees = list(range(min(sample, tb.B)))
    if cfg["grad"]:
        direct.loss_and_grad(tb, cfg["params"], CELL[cfg["kind"]], trees=trees)
    else:
        direct.forward(tb, cfg["params"], CELL[cfg["kind"]], trees=trees)
    return int(tb.tree_sizes()[trees].sum())


def oracle_sample_size(cfg):
    if cfg["kind"] == "fib":
        return 256
    if cfg["trees"].N > 2_000_000:
        return 1                       # one chain of depth 4096
    return 256 if cfg["grad"] else 512


def time_oracle(cfg, steps, warmup, scale=1, budget_s=None):
    """Times the oracle as it stands on a bounded sample per step.  With budget_s the sample shrinks (never grows) so
    that warm-up and timed steps together stay near that many seconds (a short calibration step decides)."""
    try:
        from threadpoolctl import threadpool_limits
        ctx = threadpool_limits(limits=1)
    except Exception:  # pragma: no cover
        import contextlib
        ctx = contextlib.nullcontext()
    sample = oracle_sample_size(cfg) * scale
    with ctx:
        if budget_s is not None and sample > 8:
            probe = max(1, sample // 16)
            t0 = time.perf_counter()
            oracle_step(cfg, probe)
            per_item = (time.perf_counter() - t0) / probe
            sample = max(min(sample, 8), min(sample, int(budget_s / ((steps + warmup) * per_item))))
        for _ in range(warmup):
            oracle_step(cfg, sample)
        t0 = time.perf_counter()
        n = 0
        for _ in range(steps):
            n += oracle_step(cfg, sample)
        dt = time.perf_counter() - t0
    what = (f"first {sample} instances" if cfg["kind"] == "fib" else f"first {sample} trees") + \
        f" of the workload per step, {steps} step(s), fp64/int Python+numpy oracle, 1 thread"
    return n / dt, dt / steps, what


# --------------------------------------------------------------------------- multi-rank host logic
def rank_seed(seed, rank):
    """Every rank draws a batch of its own: instances never exchange tokens (weak scaling)."""
    return seed + rank


def reduce_job(dist, device, elapsed, units):
    """Whole-job figures from per-rank ones: time = max over ranks, units = sum over ranks."""
    import torch
    if dist is None:
        return float(elapsed), float(units)
    t = torch.tensor([elapsed], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(n)
    return float(t.item()), float(n.item())


def sum_gradients(dist, grads):
    """The one exchange step of data-parallel rdf_grad: parameter gradients are summed over ranks."""
    if dist is not None:
        for t in grads.values():
            dist.all_reduce(t)


# --------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=3, choices=sorted(WORKLOAD_NAMES))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=workloads.DEFAULT_SEED)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fib-batch", type=int, default=None,
                    help="workload 1 only: number of independent fib calls (default 1024, the named configuration)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank != 0:
            return
        cfg = load(args.workload, args.seed, args.fib_batch)
        value, s_per_step, what = time_oracle(cfg, max(1, args.steps), max(0, args.warmup), budget_s=90.0)
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * s_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_NAMES[args.workload]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return

    import torch
    import paper_2410_20225_b200 as rdf

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the recursive-dataflow path has no CPU route")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # every rank processes a batch of its own (instances never exchange tokens): weak scaling
    cfg = load(args.workload, rank_seed(args.seed, rank), args.fib_batch)
    N = cfg["N"]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2

    if cfg["kind"] == "fib":
        fs, r = rdf.fib_program()
        g = rdf.Graph(fs, r, rdf.TAGS_PATH)
        x_host = torch.from_numpy(cfg["x"]).pin_memory()
        x_dev = x_host.cuda()
        y = torch.empty_like(x_dev)
        kind, compute, dtype = "eval_int", None, "int64"

        # the widest wave of fib(18) holds 2048 calls + their continuations per instance: 4096 tokens bound it
        wave_cap = min(N + len(cfg["x"]), 4096 * len(cfg["x"]))

        def step():
            g.eval_int(x_dev, N, check=False, y=y, max_wave_tokens=wave_cap)

        def step_e2e():
            xd = x_host.cuda(non_blocking=True)
            out, _ = g.eval_int(xd, N, check=False, max_wave_tokens=wave_cap)
            return out.cpu()
        h2d, d2h = x_host.numel() * 8, x_host.numel() * 8
        flops_fwd = 0.0
    else:
        tb, p = cfg["trees"], cfg["params"]
        cell = CELL[cfg["kind"]]
        fs, r = rdf.tree_net_program(cell, with_loss=cfg["grad"])
        g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
        compute = rdf.BF16 if cfg["bf16"] else rdf.F32
        # arithmetic type of the contractions: bf16 operands on the tensor cores (fp32 accumulate) for the
        # bf16 workloads, fp32 FMA otherwise
        use_tc = bool(cfg["bf16"])
        dtype = "bf16" if use_tc else "f32"
        host = {k: torch.from_numpy(np.ascontiguousarray(getattr(tb, k), dtype=np.int32)).pin_memory()
                for k in ("tree_root", "left", "right", "tok", "label")}
        dt = {k: v.cuda() for k, v in host.items()}
        dp = rdf.Graph.device_params(p)
        H = cfg["H"]
        h_root = torch.empty(tb.B, H, dtype=torch.float32, device="cuda")
        flops_fwd = tb.n_cells * 2.0 * (2 * H) * H
        if cell == "lstm":
            flops_fwd = tb.n_cells * 2.0 * (2 * H) * (5 * H) + (tb.N - tb.n_cells) * 2.0 * H * (3 * H)
        if cfg["grad"]:
            kind = ("grad_lstm_tc" if use_tc else "grad_lstm") if cell == "lstm" else ("grad_tc" if use_tc else "grad")
            grads = {k: torch.empty_like(v) for k, v in dp.items()}
            loss = torch.zeros(1, dtype=torch.float32, device="cuda")

            def step():
                g.grad_trees(dt, dp, compute, check=False, grads=grads, loss=loss, h_root=h_root)
                sum_gradients(dist, grads)      # data-parallel exchange: one sum of the parameter gradients

            def step_e2e():
                d = {k: v.cuda(non_blocking=True) for k, v in host.items()}
                l, _, _ = g.grad_trees(d, dp, compute, check=False, grads=grads, h_root=h_root)
                sum_gradients(dist, grads)
                return l.item()
            h2d, d2h = sum(v.numel() * 4 for v in host.values()), 4
        else:
            kind = "eval_trees_tc" if use_tc else "eval_trees"

            def step():
                g.eval_trees(dt, dp, compute, check=False, h_root=h_root)

            def step_e2e():
                d = {k: v.cuda(non_blocking=True) for k, v in host.items()}
                out, _ = g.eval_trees(d, dp, compute, check=False)
                return out.cpu()
            h2d, d2h = sum(v.numel() * 4 for v in host.values()), tb.B * H * 4

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    g.set_profiling(True)
    clocks = ClockSampler(local)
    clocks.start()                                   # samples from the warm-up on: short runs still get samples under load
    for _ in range(args.warmup):
        step()
    st = g.stats()                                   # also checks the device status word

    # ---- device-timed region: K steps, L2 flushed between steps, one event pair per step
    barrier()
    times, phases = [], {}
    for _ in range(args.steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
        for k, v in g.phase_ms().items():
            phases.setdefault(k, []).append(v)
    barrier()
    clk = clocks.stop()
    st = g.stats()
    total_ms, N_all = reduce_job(dist, "cuda", sum(times), N)
    value = N_all * args.steps / (total_ms * 1e-3)

    # ---- end to end through the public call, host buffers, copies inside the timed region
    for _ in range(2):
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step_e2e()
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s, _ = reduce_job(dist, "cuda", e2e_s, N)
    e2e_value = N_all * args.steps / e2e_s

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the phase with the largest share of the step)
    pk = peaks()
    mean_phase = {k: sum(v) / len(v) for k, v in phases.items()}
    dominant = max(mean_phase, key=mean_phase.get) if mean_phase else "schedule"
    dom_ms = mean_phase.get(dominant, total_ms / args.steps)
    hbm_roof = lambda kernel, alg_bytes, what: {  # noqa: E731
        "kernel": kernel, "bound": "hbm", "achieved": alg_bytes / (dom_ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
        "unit": "GB/s", "frac": alg_bytes / (dom_ms * 1e-3) / 1e9 / pk["hbm_gbs"], "traffic": None,
        "peak_source": pk["source"], "algorithmic_bytes": alg_bytes, "bytes_are": what}
    if dominant == "schedule" or cfg["kind"] == "fib":
        # 6 token touches x 16 B + one 32 B store slot / frame record per invocation
        roof = hbm_roof("rdf_scheduler_kernel", 128.0 * N, "128 B per invocation (token write+read, return/store slot write+read, frame record)")
    elif dominant == "loss":
        rowbytes = (64 * ((cfg["H"] + 63) // 64)) * 2 if use_tc else cfg["H"] * 4 * (2 if cell == "lstm" else 1)
        roof = hbm_roof("rdf_loss_heads_kernel", float(N) * (rowbytes + 32), "one state row read + 32 B dlog written per invocation")
    else:
        H = cfg["H"]
        C = cfg["trees"].n_cells
        # algorithmic flops of the contraction in each phase: 2 * 2H * (rows of W) per cell
        flops = flops_fwd
        kernel = {"operators": "rdf_operator_kernel", "backward": "rdf_backward_kernel",
                  "dW": "rdf_dw_tc_kernel" if use_tc else "rdf_outer_kernel"}.get(dominant, dominant)
        if use_tc:
            peak = pk["bf16_tflops_sustained"]
            achieved = flops / (dom_ms * 1e-3) / 1e12
            roof = {"kernel": kernel, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak, "traffic": None,
                    "peak_source": pk["source"] + " (bf16 dense, sustained)", "cells": C, "flops_phase": flops,
                    "note": "a persistent kernel: every wave ends at a grid barrier; block0_ms_at_max_clock gives the split"}
            if dominant == "operators" and cell == "rnn":
                Hp = 64 * ((H + 63) // 64)
                # per cell: two bf16 operand rows read, one bf16 state row written; per leaf: an fp32 table row read, a bf16 row written
                alg = C * (3.0 * Hp * 2) + (tb.N - C) * (H * 4.0 + Hp * 2)
                roof["hbm_view"] = {"algorithmic_bytes": alg, "achieved_gbs": alg / (dom_ms * 1e-3) / 1e9,
                                    "frac_of_hbm_peak": alg / (dom_ms * 1e-3) / 1e9 / pk["hbm_gbs"]}
        else:
            achieved = flops / (dom_ms * 1e-3) / 1e12
            roof = {"kernel": kernel, "bound": "alu", "achieved": achieved, "peak": FP32_ALU_PEAK_TFLOPS,
                    "unit": "TFLOP/s", "frac": achieved / FP32_ALU_PEAK_TFLOPS, "traffic": None,
                    "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                    "cells": C, "flops_phase": flops}
    roof["phase"] = dominant
    roof["phase_ms"] = dom_ms

    roof["traffic"] = NCU_TRAFFIC_BYTES.get((roof["kernel"], args.workload, args.fib_batch if args.workload == 1 else None))
    cpu = None
    if not args.no_cpu_baseline:
        v, _, what = time_oracle(cfg, 1, 0, scale=1 if cfg["trees"].N > 2_000_000 else 4) if cfg["kind"] != "fib" else time_oracle(cfg, 1, 0, scale=4)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype, "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload] + (f" [scaled: {args.fib_batch} calls]" if args.fib_batch and args.workload == 1 else ""),
                   "invocations_per_step": N, "instances": cfg.get("B") or cfg["trees"].B,
                   "pass": "forward+backward" if cfg.get("grad") else "forward",
                   "timing": "CUDA events per step; 256 MB L2 flush between steps; inputs and parameters resident"},
        "clocks": clk,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        # (bf16 with padded state rows: db / db_x come out of the dW / dW_x contractions, one / two kernels fewer)
        "gpu_launches": (KERNELS_PER_STEP[kind] - ({"grad_tc": 1, "grad_lstm_tc": 2}.get(kind, 0) if cfg.get("H", 64) % 64 else 0)) * args.steps,
        "roofline": roof,
        "cpu_baseline": cpu,
        "phase_ms": mean_phase,
        "waves": {"forward": st["waves"], "backward": st["waves_backward"], "widest": st["max_wave_tokens"]},
        "block0_ms_at_max_clock": {k[7:]: round(st[k] / 1.965e6, 4) for k in st if k.startswith("cycles_")},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
