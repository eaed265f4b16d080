#!/usr/bin/env python
"""Benchmark: recursive invocations per second of the tagged-dataflow executor.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input:
lowered graph -> seed tokens -> all forward waves (tag push/pop, matching, batched
cells) -> loss head -> gradient waves -> parameter gradients (workloads 3-5), or
the forward pass alone (workloads 1-2).  Prints one JSON line: the headline workload
(default 3) with its roofline, and -- on one GPU -- a table of all five workloads
(forward and forward+backward), a table of every kernel of the headline step with
its algorithmic work against the measured peak, and the CPU oracle's rate.

With --gpus N > 1 and no RANK in the environment the script starts the N ranks
itself (one process per GPU, NCCL); under torchrun it joins the ranks it is given.
"""
from __future__ import annotations

import argparse
import hashlib
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
    6: "extra: top-down recursion shaped by the values (a gate on each node's state decides its expansion), 8192 seeds, H=128, "
       "depth limit 10, fp32, forward",
}
CELL = {"treernn": "rnn", "treelstm": "lstm"}
KERNEL_SOURCES = ["rdf_device.cuh", "rdf_exec.cu", "rdf_exec.h", "rdf_grad.cu", "rdf_internal.h", "rdf_lists.cuh", "rdf_lstm.cuh",
                  "rdf_tc.cuh", "rdf_tc_dw.cuh"]


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
def load(k, seed, fib_batch=None, over=None):
    """Workload k; `over`: generator arguments that replace the named configuration's (reduced cases for profiling)."""
    over = dict(over or {})
    if k == 1 and fib_batch:
        over["B"] = fib_batch
    cfg = workloads.config(k, seed=seed, **over)
    if cfg["kind"] == "fib":
        cfg["N"] = int(sum(2 * fib_iter(int(n) + 1) - 1 for n in cfg["x"]))
    elif cfg["kind"] == "topdown":
        cfg["N"] = 0                   # how many invocations the seeds generate is known after the first run
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


def kernel_source_hash():
    """Fingerprint of the CUDA sources: DRAM traffic taken from a profiler capture is reported only while the
    kernels are the ones that were captured."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2410_20225_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def dram_traffic_table():
    """{(kernel, workload): bytes per launch} from the tracked table of profiler captures; only the rows whose
    source fingerprint is the current one count (a changed kernel has no traffic figure until it is captured again)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    table, cur = {}, kernel_source_hash()
    if not os.path.exists(path):
        return table
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) >= 4 and line[3] == cur:
            table[(line[0], int(line[1]))] = float(line[2])
    return table


# nominal fp32 FMA peak (148 SMs x 128 lanes x 2 flop x 1.965 GHz); the run measures the achieved rate itself
FP32_ALU_NOMINAL_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


# --------------------------------------------------------------------------- CPU oracle arm
def cpu_info():
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except AttributeError:
        usable = os.cpu_count() or 1
    return model, usable


def oracle_step(cfg, sample, grad=None):
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
    if cfg["kind"] == "topdown":
        n = 0
        for t in trees:
            log = {}
            direct.topdown(cfg["params"], int(tb.tok[t]), cfg["D"], log)
            n += 1 + log["expand"] + log["child"]
        return n
    if cfg["grad"] if grad is None else grad:
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


def time_oracle_all_cores(cfg, cores, budget_s=20.0):
    """The oracle over a pool of processes (trees are independent), one per usable core, on a sample sized from the
    one-thread rate for about budget_s of wall time; the wall time includes the start of the worker processes."""
    if cfg["kind"] == "fib" or not cfg["grad"] or cores < 2:
        return None
    from oracle import direct
    tb = cfg["trees"]
    workers = max(1, cores)
    t0 = time.perf_counter()
    probe = list(range(min(8, tb.B)))
    direct.loss_and_grad(tb, cfg["params"], CELL[cfg["kind"]], trees=probe)
    per_node = (time.perf_counter() - t0) / max(1, int(tb.tree_sizes()[probe].sum()))
    want_nodes = budget_s * workers / per_node
    sizes = np.cumsum(tb.tree_sizes())
    n_trees = int(min(tb.B, max(workers, np.searchsorted(sizes, want_nodes) + 1)))
    trees = list(range(n_trees))
    t0 = time.perf_counter()
    direct.loss_and_grad_pool(tb, cfg["params"], CELL[cfg["kind"]], workers=workers, trees=trees)
    dt = time.perf_counter() - t0
    n = int(tb.tree_sizes()[trees].sum())
    return {"value": n / dt, "unit": UNIT, "cores": workers, "kind": "oracle",
            "sample": f"first {n_trees} trees of the workload, one pass, fp64 Python+numpy oracle over {workers} spawned processes "
                      f"(wall time {dt:.1f} s including their start-up)"}


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


def flat_gradients(shapes, device):
    """One buffer for all parameter gradients; returns (flat, {name: view}).  Views start on 256-byte boundaries."""
    import torch
    offs, total = {}, 0
    for k, shp in shapes.items():
        offs[k] = total
        total += (int(np.prod(shp)) + 63) // 64 * 64
    flat = torch.zeros(total, dtype=torch.float32, device=device)
    views = {k: flat[offs[k]: offs[k] + int(np.prod(shp))].view(*shp) for k, shp in shapes.items()}
    return flat, views


def sum_gradients(dist, grads):
    """The one exchange step of data-parallel rdf_grad: parameter gradients are summed over ranks -- one
    all-reduce when the gradients are views of one flat buffer (pass that buffer), else one per tensor."""
    if dist is None:
        return
    import torch
    if isinstance(grads, torch.Tensor):
        dist.all_reduce(grads)
        return
    for t in grads.values():
        dist.all_reduce(t)


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_entry(rank, world, port, target, payload):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    target(payload)


def spawn_ranks(world, target, payload):
    """Starts `world` processes on this node (rank r = local rank r) that each run target(payload) with the
    rendezvous variables set; raises if one of them fails."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_entry, args=(world, _free_port(), target, payload), nprocs=world, join=True)


# --------------------------------------------------------------------------- one workload on the device
class Case:
    """One workload set up on the current device: resident inputs, host copies for the end-to-end path, step functions."""

    def __init__(self, rdf, torch, cfg, grad, dist=None, store="thread", hash_load=None):
        self.rdf, self.torch, self.cfg, self.dist = rdf, torch, cfg, dist
        self.N = cfg["N"]
        self.grad = bool(grad)
        if cfg["kind"] == "fib":
            fs, r = rdf.fib_program()
            self.g = rdf.Graph(fs, r, rdf.TAGS_PATH)
            # token store: probing strategy, and (hash_load) the table sized for that load factor instead of the default
            parked = int(sum(fib_iter(int(n) + 1) - 1 for n in cfg["x"]))
            self.g.set_store(1 if store == "warp" else 0, int(parked / hash_load) if hash_load else 0)
            self.x_host = torch.from_numpy(cfg["x"]).pin_memory()
            self.x_dev = self.x_host.cuda()
            self.y = torch.empty_like(self.x_dev)
            self.y_host = torch.empty_like(self.x_host).pin_memory()
            self.dtype, self.use_tc, self.cell = "int64", False, None
            # the widest wave of fib(18) holds 2048 calls + their continuations per instance: 4096 tokens bound it
            self.wave_cap = min(self.N + len(cfg["x"]), 4096 * len(cfg["x"]))
            self.h2d, self.d2h = self.x_host.numel() * 8, self.x_host.numel() * 8
            self.d2h_full = self.d2h
            return
        tb, p = cfg["trees"], cfg["params"]
        self.tb = tb
        self.topdown = cfg["kind"] == "topdown"
        self.cell = "rnn" if self.topdown else CELL[cfg["kind"]]
        fs, r = rdf.topdown_program(cfg["D"]) if self.topdown else rdf.tree_net_program(self.cell, with_loss=self.grad)
        self.g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
        self.max_inv = cfg.get("max_invocations")
        self.compute = rdf.BF16 if cfg["bf16"] else rdf.F32
        # arithmetic type of the contractions: bf16 operands on the tensor cores (fp32 accumulate) for the
        # bf16 workloads, fp32 FMA otherwise
        self.use_tc = bool(cfg["bf16"])
        self.dtype = "bf16" if self.use_tc else "f32"
        self.host = {k: torch.from_numpy(np.ascontiguousarray(getattr(tb, k), dtype=np.int32)).pin_memory()
                     for k in ("tree_root", "left", "right", "tok", "label")}
        self.dt = {k: v.cuda() for k, v in self.host.items()}
        self.dp = rdf.Graph.device_params(p)
        self.H = cfg["H"]
        self.h_root = torch.empty(tb.B, self.H, dtype=torch.float32, device="cuda")
        self.h_root_host = torch.empty(tb.B, self.H, dtype=torch.float32).pin_memory()
        self.h2d = sum(v.numel() * 4 for v in self.host.values())
        if self.grad:
            self.flat, self.grads = flat_gradients({k: tuple(v.shape) for k, v in self.dp.items()}, "cuda")
            self.flat_host = torch.empty_like(self.flat, device="cpu").pin_memory()
            self.loss = torch.zeros(1, dtype=torch.float32, device="cuda")
            self.d2h = 4
            self.d2h_full = 4 + self.flat.numel() * 4 + tb.B * self.H * 4
        else:
            self.d2h = self.d2h_full = tb.B * self.H * 4
        if self.topdown:               # one run tells how many invocations the seeds generate (the unit of the metric)
            self.step()
            self.N = cfg["N"] = int(self.g.stats()["invocations"])

    # the timed step: inputs and parameters resident
    def step(self):
        if self.cfg["kind"] == "fib":
            self.g.eval_int(self.x_dev, self.N, check=False, y=self.y, max_wave_tokens=self.wave_cap)
        elif self.grad:
            self.g.grad_trees(self.dt, self.dp, self.compute, check=False, grads=self.grads, loss=self.loss, h_root=self.h_root)
            sum_gradients(self.dist, self.flat)      # data-parallel exchange: one sum of the parameter gradients
        else:
            self.g.eval_trees(self.dt, self.dp, self.compute, check=False, h_root=self.h_root, max_invocations=self.max_inv)

    # end to end: host buffers in, result out; full = every output of the call comes back
    def step_e2e(self, full=False):
        if self.cfg["kind"] == "fib":
            xd = self.x_host.cuda(non_blocking=True)
            self.g.eval_int(xd, self.N, check=False, y=self.y, max_wave_tokens=self.wave_cap)
            self.y_host.copy_(self.y, non_blocking=True)
            self.torch.cuda.current_stream().synchronize()
            return self.y_host
        d = {k: v.cuda(non_blocking=True) for k, v in self.host.items()}
        if self.grad:
            self.g.grad_trees(d, self.dp, self.compute, check=False, grads=self.grads, loss=self.loss, h_root=self.h_root)
            sum_gradients(self.dist, self.flat)
            if full:
                self.flat_host.copy_(self.flat, non_blocking=True)
                self.h_root_host.copy_(self.h_root, non_blocking=True)
            return self.loss.item()
        self.g.eval_trees(d, self.dp, self.compute, check=False, h_root=self.h_root, max_invocations=self.max_inv)
        self.h_root_host.copy_(self.h_root, non_blocking=True)
        self.torch.cuda.current_stream().synchronize()
        return self.h_root_host

    def flops_fwd(self):
        if self.cfg["kind"] == "fib":
            return 0.0
        H, tb = self.H, self.tb
        if self.topdown:               # N = B seeds + E expands + (E - B) children, (E - B) / 2 of the expands end in a cell
            E = self.N // 2
            return (E - tb.B) * 2.0 * H * H + (E - tb.B) / 2 * 2.0 * (2 * H) * H
        if self.cell == "lstm":
            return tb.n_cells * 2.0 * (2 * H) * (5 * H) + (tb.N - tb.n_cells) * 2.0 * H * (3 * H)
        return tb.n_cells * 2.0 * (2 * H) * H


def time_case(case, steps, warmup, flush, dist=None, e2e_steps=None, full_e2e=False):
    """W warm-up steps, K device-timed steps (one CUDA event pair per step on the launching stream, L2 flushed
    between steps), then the end-to-end loop.  Returns whole-job figures (max over ranks / sum of units)."""
    torch = case.torch

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    case.g.set_profiling(True)
    for _ in range(warmup):
        case.step()
    case.g.stats()                                   # also checks the device status word
    barrier()
    times, phases = [], {}
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        case.step()
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
        for k, v in case.g.phase_ms().items():
            phases.setdefault(k, []).append(v)
    barrier()
    st = case.g.stats()
    total_ms, N_all = reduce_job(dist, "cuda", sum(times), case.N)
    out = {"ms_per_step": total_ms / steps, "value": N_all * steps / (total_ms * 1e-3), "N_all": N_all,
           "phase_ms": {k: sum(v) / len(v) for k, v in phases.items()}, "stats": st, "min_ms": min(times)}
    # ---- end to end through the public call, host buffers, copies inside the timed region
    ke = e2e_steps or steps
    variants = [("e2e", False)] + ([("e2e_all_outputs", True)] if full_e2e and case.grad else [])
    for name, full in variants:
        for _ in range(2):
            case.step_e2e(full)
        barrier()
        t0 = time.perf_counter()
        for _ in range(ke):
            case.step_e2e(full)
        barrier()
        e2e_s, _ = reduce_job(dist, "cuda", time.perf_counter() - t0, case.N)
        out[name] = {"value": N_all * ke / e2e_s, "unit": UNIT, "h2d_bytes_per_step": case.h2d,
                     "d2h_bytes_per_step": case.d2h_full if full else case.d2h}
        if full:
            out[name]["what_comes_back"] = "loss, every parameter gradient and the root states, to pinned host buffers"
    return out


# --------------------------------------------------------------------------- kernels against their rooflines
def kernel_table(case, phase_ms, pk, fp32_peak, traffic, workload):
    """One row per kernel (group) of the step: CUDA-event time of its phase, algorithmic bytes or flops, the
    measured peak that bounds it and the fraction reached.  Tensor peak: the burst figure for a kernel of under a
    millisecond (it runs alone between two events on an otherwise idle device), the sustained one above that."""
    N = case.N
    rows = []

    def add(kernel, phase, bound, work, what):
        ms = phase_ms.get(phase)
        if ms is None or ms <= 0:
            return
        if bound == "hbm":
            peak, unit, ach, src = pk["hbm_gbs"], "GB/s", work / (ms * 1e-3) / 1e9, pk["source"] + " copy bandwidth"
        elif bound == "tensor":
            burst = ms < 1.0
            peak = pk["bf16_tflops"] if burst else pk["bf16_tflops_sustained"]
            unit, ach = "TFLOP/s", work / (ms * 1e-3) / 1e12
            src = pk["source"] + (" bf16 dense, burst" if burst else " bf16 dense, sustained")
        else:
            peak, unit, ach, src = fp32_peak, "TFLOP/s", work / (ms * 1e-3) / 1e12, "fp32 FMA loop measured in this run"
        rows.append({"kernel": kernel, "phase": phase, "ms": ms, "bound": bound, "algorithmic": work, "work_is": what,
                     "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak if peak else None, "peak_source": src,
                     "traffic": traffic.get((kernel, workload))})

    add("rdf_scheduler_kernel", "schedule", "hbm", 128.0 * N,
        "128 B per invocation: call token write+read, return token / store slot write+read, frame record")
    if case.cfg["kind"] == "fib":
        return rows
    if case.cfg["kind"] == "topdown":
        rows.clear()
        add("rdf_interleaved_kernel", "schedule", "alu", case.flops_fwd(),
            "child operators 2*H*H and cells 2*2H*H per expanded node (token waves and operators share the kernel)")
        return rows
    tb, H = case.tb, case.H
    C, Lf = tb.n_cells, tb.N - tb.n_cells
    Hp = 64 * ((H + 63) // 64)
    lstm = case.cell == "lstm"
    mm = "tensor" if case.use_tc else "alu"
    if case.use_tc:       # tensor-core path: the cells listed by call depth (the same lists serve the gradient pass)
        add("rdf_list_count/scan/fill/ends/compact/zdst_kernel", "group", "hbm", N * 32.0 + C * 24.0,
            "operand ids and frame records read (two passes), cell lists and operand-row destinations written")
    else:
        add("rdf_height_count/scan/scatter_kernel", "group", "hbm", 48.0 * C, "16 B cell record read twice and written once")
    add("rdf_operator_kernel", "operators", mm, case.flops_fwd(),
        "cell contraction 2*2H*H per cell" + (" (x5 gates) + leaf projection 2*D*3H per leaf" if lstm else ""))
    add("rdf_gather_roots_kernel", "roots", "hbm", tb.B * H * (4.0 + (2 if case.use_tc and not lstm else 4)), "root rows read and written")
    if case.grad:
        rowbytes = Hp * 2 if case.use_tc else H * 4 * (2 if lstm else 1)
        add("rdf_loss_heads_kernel", "loss", "hbm", float(N) * (rowbytes + 32), "one state row read + 32 B of dlog written per invocation")
        if not case.use_tc:
            add("rdf_list_count/scan/fill/ends/compact_kernel", "lists", "hbm", N * 28.0 + C * 24.0,
                "operand ids and frame records read (two passes), cell lists written")
        bwd = C * 2.0 * H * (2 * H) * (5 if lstm else 1)
        add("rdf_backward_kernel", "backward", mm, bwd, "operand-gradient contraction W^T dz: 2*H*2H per cell" + (" (x5 gates)" if lstm else ""))
        dw = bwd + (Lf * 2.0 * H * 3 * H if lstm else 0.0)
        add("rdf_dw_tc_kernel" if case.use_tc else "rdf_outer_kernel", "dW", mm, dw,
            "weight-gradient contraction dz (x) [h_l;h_r]: 2*H*2H per cell" + (" (x5 gates) + leaf 2*3H*D" if lstm else ""))
        if not (case.use_tc and H % 64):       # (bf16 with padded rows: db is a column of the dW contraction, no kernel of its own)
            add("rdf_colsum_kernel", "db", "hbm", C * (5 if lstm else 1) * H * (2.0 if case.use_tc else 4.0), "one gradient row read per cell")
        if lstm:
            add("rdf_de_tc_kernel" if case.use_tc else "rdf_de_lstm_kernel", "dE", mm, Lf * 2.0 * H * 3 * H, "W_x^T dg: 2*3H*D per leaf")
    return rows


# --------------------------------------------------------------------------- main
def run(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    import paper_2410_20225_b200 as rdf
    from paper_2410_20225_b200.binding import probe_fp32_fma_tflops

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the recursive-dataflow path has no CPU route")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} wants GPU {local} but this node has {torch.cuda.device_count()}")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # every rank processes a batch of its own (instances never exchange tokens): weak scaling
    cfg = load(args.workload, rank_seed(args.seed, rank), args.fib_batch, args.override)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2
    case = Case(rdf, torch, cfg, cfg.get("grad", False), dist, args.store, args.hash_load)

    clocks = ClockSampler(local)
    clocks.start()                                   # samples from the warm-up on: short runs still get samples under load
    head = time_case(case, args.steps, args.warmup, flush, dist, full_e2e=True)
    clk = clocks.stop()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = peaks()
    fp32_peak = probe_fp32_fma_tflops()
    traffic = dram_traffic_table()
    kernels = kernel_table(case, head["phase_ms"], pk, fp32_peak, traffic, args.workload)
    # ---- roofline of the dominant kernel (the phase with the largest share of the step)
    dom = max(kernels, key=lambda r: r["ms"])
    roof = {"kernel": dom["kernel"], "bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"], "unit": dom["unit"],
            "frac": dom["frac"], "traffic": dom["traffic"], "peak_source": dom["peak_source"], "phase": dom["phase"],
            "phase_ms": dom["ms"], "algorithmic": dom["algorithmic"], "work_is": dom["work_is"],
            "note": "a persistent kernel: every wave ends at a grid barrier; block0_ms_at_max_clock gives the split"}
    st = head["stats"]

    # ---- the other workloads, forward and forward+backward (one GPU only: the table is not part of the scaling run)
    table = None
    if world == 1 and not args.no_table:
        table = []
        for k in sorted(WORKLOAD_NAMES):
            c_k = cfg if k == args.workload and not args.fib_batch and not args.override else load(k, args.seed)
            passes = [False, True] if c_k.get("grad") else [False]
            for grad in passes:
                if k == args.workload and grad == bool(cfg.get("grad", False)) and not args.fib_batch and not args.override:
                    res, cs = head, case
                else:
                    cs = Case(rdf, torch, c_k, grad)
                    n = 5 if c_k["N"] > 2_000_000 else min(args.steps, 20)
                    res = time_case(cs, n, 3, flush, e2e_steps=min(n, 5))
                kt = kernel_table(cs, res["phase_ms"], pk, fp32_peak, traffic, k)
                top = max(kt, key=lambda r: r["ms"])
                table.append({"workload": k, "pass": "forward+backward" if grad else "forward", "dtype": cs.dtype,
                              "invocations_per_step": c_k["N"], "ms_per_step": res["ms_per_step"], "value": res["value"],
                              "e2e": res["e2e"]["value"], "unit": UNIT, "waves": res["stats"]["waves"],
                              "waves_backward": res["stats"]["waves_backward"],
                              "kernels": [{"kernel": r["kernel"], "ms": round(r["ms"], 4), "bound": r["bound"],
                                           "achieved": r["achieved"], "unit": r["unit"], "frac": r["frac"]} for r in kt],
                              "dominant": {"kernel": top["kernel"], "bound": top["bound"], "frac": top["frac"]}})
                del cs
                torch.cuda.empty_cache()
        # the hash token store with warp-cooperative probes, and the scaled run (131072 calls) that takes the store out of L2
        for label, fb, store in (("1 (warp-cooperative probes)", None, "warp"), ("1 scaled: 131072 calls", 131072, "thread"),
                                 ("1 scaled: 131072 calls (warp-cooperative probes)", 131072, "warp")):
            c_k = load(1, args.seed, fb)
            cs = Case(rdf, torch, c_k, False, store=store)
            res = time_case(cs, 5, 3, flush, e2e_steps=3)
            kt = kernel_table(cs, res["phase_ms"], pk, fp32_peak, traffic, 1)
            table.append({"workload": label, "pass": "forward", "dtype": cs.dtype, "invocations_per_step": c_k["N"],
                          "ms_per_step": res["ms_per_step"], "value": res["value"], "e2e": res["e2e"]["value"], "unit": UNIT,
                          "waves": res["stats"]["waves"], "waves_backward": 0,
                          "kernels": [{"kernel": r["kernel"], "ms": round(r["ms"], 4), "bound": r["bound"], "achieved": r["achieved"],
                                       "unit": r["unit"], "frac": r["frac"]} for r in kt],
                          "dominant": {"kernel": kt[0]["kernel"], "bound": kt[0]["bound"], "frac": kt[0]["frac"]}})
            del cs
            torch.cuda.empty_cache()

    # ---- the same step with reproducible sums (tensor-core path only)
    repro = None
    if world == 1 and case.grad and case.use_tc and not args.no_table:
        rep_times = []
        for k in range(3 + min(args.steps, 10)):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            case.g.grad_trees(case.dt, case.dp, case.compute, check=False, grads=case.grads, loss=case.loss, h_root=case.h_root,
                              reproducible=True)
            e1.record()
            e1.synchronize()
            if k >= 3:
                rep_times.append(e0.elapsed_time(e1))
        case.g.stats()
        repro = {"ms_per_step": sum(rep_times) / len(rep_times), "what": "rdf_grad with rdf_params.reproducible = 1: bit-identical gradients and loss on every call"}

    cpu, cpu_all = None, None
    if not args.no_cpu_baseline:
        model, usable = cpu_info()
        v, _, what = time_oracle(cfg, 1, 0, scale=1 if cfg["kind"] != "fib" and cfg["trees"].N > 2_000_000 else 4)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what, "cpu_model": model, "usable_cores": usable}
        cpu_all = time_oracle_all_cores(cfg, usable)
        if cpu_all is not None:
            cpu["all_cores"] = cpu_all

    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": case.dtype, "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload] + (f" [scaled: {args.fib_batch} calls]" if args.fib_batch and args.workload == 1 else "")
                   + (f" [reduced: {args.override}]" if args.override else "")
                   + (f" [store: {args.store} probes" + (f", load {args.hash_load}" if args.hash_load else "") + "]" if args.workload == 1 else ""),
                   "invocations_per_step": case.N, "instances": cfg.get("B") or cfg["trees"].B,
                   "pass": "forward+backward" if cfg.get("grad") else "forward",
                   "timing": "CUDA events per step; 256 MB L2 flush between steps; inputs and parameters resident"},
        "clocks": clk,
        "e2e": head["e2e"],
        "e2e_all_outputs": head.get("e2e_all_outputs"),
        "reproducible_mode": repro,
        "gpu_launches": st["kernel_launches"] * args.steps,          # counted by the library at every launch of the call
        "roofline": roof,
        "kernels": kernels,
        "workloads": table,
        "cpu_baseline": cpu,
        "phase_ms": head["phase_ms"],
        "min_ms_per_step": head["min_ms"],
        "fp32_fma_tflops": {"measured": fp32_peak, "nominal": FP32_ALU_NOMINAL_TFLOPS},
        "waves": {"forward": st["waves"], "backward": st["waves_backward"], "widest": st["max_wave_tokens"]},
        "block0_ms_at_max_clock": {k[7:]: round(st[k] / 1.965e6, 4) for k in st if k.startswith("cycles_")},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def reference(args):
    cfg = load(args.workload, args.seed, args.fib_batch)
    value, s_per_step, what = time_oracle(cfg, max(1, args.steps), max(0, args.warmup), budget_s=90.0)
    model, usable = cpu_info()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * s_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what, "cpu_model": model,
                         "usable_cores": usable},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=3, choices=sorted(WORKLOAD_NAMES))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=workloads.DEFAULT_SEED)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="skip the table of the other workloads")
    ap.add_argument("--store", default="thread", choices=["thread", "warp"],
                    help="workload 1: probing of the hash token store (per thread / warp-cooperative)")
    ap.add_argument("--hash-load", type=float, default=None,
                    help="workload 1: size the hash table for this load factor (parked operands / slots, rounded to a power of two)")
    ap.add_argument("--override", action="append", default=[], metavar="KEY=INT",
                    help="replace an argument of the workload generator (B, V, H, chains, chain_depth, perfect, perfect_height): "
                         "reduced cases for profiler captures; the line says so in config.workload")
    ap.add_argument("--fib-batch", type=int, default=None,
                    help="workload 1 only: number of independent fib calls (default 1024, the named configuration)")
    args = ap.parse_args()
    args.override = {kv.split("=")[0]: int(kv.split("=")[1]) for kv in args.override}
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            reference(args)
        return
    in_ranks = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if args.gpus > 1 and not in_ranks:
        # no launcher gave us ranks: start them here, one process per GPU
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: this node has {have} CUDA device(s); refusing to report fewer GPUs than asked")
        spawn_ranks(args.gpus, run, args)
        return
    if in_ranks and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} but the launcher started {os.environ['WORLD_SIZE']} rank(s)")
    run(args)


if __name__ == "__main__":
    main()
