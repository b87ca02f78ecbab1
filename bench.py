#!/usr/bin/env python
"""Benchmark of the fused CP-head log-likelihood on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path of the workload over one batch of seeded
synthetic inputs: forward for `train_fwd`, forward + backward for the `*_fwd_bwd`
workloads, draft scoring for `decode_*`.  Prints ONE JSON line.

Without --workload the line's headline is the large forward+backward step
(`train_fwd_bwd`) and its `workloads` list carries the other regimes of the metric
(training-shape forward, draft scoring at 1 / 8 / 64 positions, the big-vocabulary
step), each timed in the same process with its own clock record, roofline and
host-buffer leg.  With --workload NAME only that workload runs.  With N > 1 ranks
(torchrun) every rank runs the same per-GPU batch (positions are independent, no
collective on the data path) and the reported value is the whole-job rate.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "cp_head_positions_per_second"
UNIT = "positions/s"

WORKLOADS = {
    # name: (synth config, kind, extra make_inputs kwargs, aux coefficient)
    "train_fwd": ("train_fwd", "fwd", {}, None),
    "train_fwd_bwd": ("train_fwd_bwd", "fwd_bwd", {}, None),
    "bigvocab_fwd_bwd": ("bigvocab_fwd_bwd", "fwd_bwd", {"targets": "zipf"}, 1.0),
    # head-only fine-tuning as in the paper: shared unembedding and trunk frozen (no dE, no dh)
    "finetune_fwd_bwd": ("train_fwd_bwd", "fwd_bwd", {}, None),
    # the paper's fine-tuning objective (Eq. 14): KL to the frozen head's logits + discounted CE, head only
    "distill_fwd_bwd": ("train_fwd_bwd", "distill", {}, None),
    "distill_fwd_bwd_small": ("train_fwd_bwd_small", "distill", {}, None),
    "decode_1": ("decode_1", "score", {}, None),
    "decode_8": ("decode_8", "score", {}, None),
    "decode_64": ("decode_64", "score", {}, None),
    "draft_8": ("decode_8", "sample", {}, None),
    "full_head_fwd_bwd": ("full_head_train", "full_fwd_bwd", {}, None),
    "train_fwd_bwd_small": ("train_fwd_bwd_small", "fwd_bwd", {}, None),
    "bigvocab_fwd_small": ("bigvocab_fwd_small", "fwd", {"targets": "zipf"}, 1.0),
    "tiny": ("tiny", "fwd_bwd", {}, None),
}

HEADLINE = "train_fwd_bwd"
# The other regimes of the metric, run after the headline when no --workload is given, with the number of
# timed steps each gets (enough for the clock sampler to see the timed region; few for the 1.8 s step).
ALSO = [("train_fwd", 50), ("decode_1", 500), ("decode_8", 500), ("decode_64", 200), ("bigvocab_fwd_bwd", 4)]


def ncu_traffic_bytes(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the workload's dominant kernel, from the
    tracked table of ncu captures; None when there is no capture of the current kernel."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            entry = json.load(f).get(workload)
    except (OSError, ValueError):
        return None
    return None if entry is None else entry.get("bytes_per_launch")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], burst=p["bf16_tflops"], sustained=p["bf16_tflops_sustained"], src="measured")
    return dict(hbm_gbs=6650.0, burst=1590.0, sustained=1400.0, src="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples.  One query loop runs for the whole process (it needs a
    moment to come up) and every sample is stamped on arrival; summary(t0, t1) covers only the samples that
    arrived in that window, i.e. while one timed region ran."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        import threading

        self.proc = None
        self.samples = []
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.perf_counter(), line))

    def summary(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)   # let the reader thread take in what was printed up to t1
        snapshot = list(self.samples)
        inside = [ln for t, ln in snapshot if t0 <= t <= t1]
        window = "timed region"
        if not inside:   # region shorter than the query interval: the samples closest to its end
            inside = [ln for t, ln in snapshot if t <= t1 + 0.05][-3:]
            window = "last samples before the end of the timed region"
        sm, mx, reasons = [], [], set()
        for line in inside:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}

    def stop(self) -> None:
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)


def flops_per_position(s, kind, skip=()):
    K = s.n * s.r
    fwd = 2 * K * (s.d * s.d + s.V * s.d) + 2 * s.r * s.d
    if kind == "full_fwd_bwd":
        return 3 * (2 * K * s.V * s.d + 2 * s.r * s.d)
    if kind == "distill":
        # projection, two vocabulary sweeps forward (log-sum-exp, KL), logits recompute + dz backward, dW_head
        return 4 * K * s.d * s.d + 4 * 2 * K * s.V * s.d + 2 * s.r * s.d
    if kind == "fwd_bwd" and skip:
        # forward + dz always; dE, dW_head, dh only when asked for
        total = fwd + 2 * K * s.V * s.d
        total += 0 if "dE" in skip else 2 * K * s.V * s.d
        total += 0 if "dW_head" in skip else 2 * K * s.d * s.d
        total += 0 if "dh" in skip else 2 * K * s.d * s.d
        return total
    return fwd if kind != "fwd_bwd" else 3 * fwd


def oracle_seconds_per_position(inp, kind, aux, sample: int):
    """Time the fp64 oracle, as it stands, on the first `sample` positions."""
    import torch
    from oracle import cp_head
    from paper_2410_17765_b200 import synth

    s = inp.shape
    sample = min(sample, s.N)
    sub = synth.subsample_positions(inp, torch.arange(sample))
    t0 = time.perf_counter()
    if kind == "distill":
        from oracle import distill

        T = synth.make_teacher_logits(sub.shape, sub.x, seed=0)
        t0 = time.perf_counter()
        distill.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, T, s.n, s.r, beta=0.9, gamma=0.8)
    elif kind == "full_fwd_bwd":
        cp_head.backward_full(sub.h, synth.make_full_head(s, seed=0), sub.W_g, sub.x, s.n, s.r, aux_coef=aux or 0.0)
    elif kind == "fwd_bwd":
        cp_head.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, aux_coef=aux or 0.0)
    else:
        cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, aux_coef=aux or 0.0)
    return (time.perf_counter() - t0) / sample, sample


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        counts = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if counts:
            return max(counts)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_sample_size(s, kind) -> int:
    # about 10-15 s of fp64 numpy work: assume ~40 GFLOP/s on the host cores
    per_pos = flops_per_position(s, kind) * (1.4 if kind in ("fwd_bwd", "distill") else 1.0)
    return max(1, min(s.N, int(40e9 * 15 / per_pos)))


def config_of(workload: str) -> dict:
    """The `config` object of a JSON line: the same for the library's arm and for the oracle's arm."""
    from paper_2410_17765_b200 import synth

    cfg, kind, extra, aux = WORKLOADS[workload]
    shape = synth.CONFIGS[cfg]
    return {"workload": workload, "kind": kind, **shape.__dict__, "aux_coef": aux,
            "targets": extra.get("targets", "uniform"), "l2": "inputs larger than L2 (no flush)",
            "per_gpu_positions": shape.N}


def run_reference(args, rank: int):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only).  Every step runs the
    oracle on the same bounded sample of positions that the library arm's `cpu_baseline` leg times once
    (the oracle's matrix products only use all cores when the sample is not a handful of rows)."""
    if rank != 0:
        return
    from paper_2410_17765_b200 import synth

    workload = args.workload or HEADLINE
    cfg, kind, extra, aux = WORKLOADS[workload]
    shape = synth.CONFIGS[cfg]
    inp = synth.make_inputs(shape, seed=0, **extra)
    per_step = oracle_sample_size(shape, kind)
    for _ in range(args.warmup):
        oracle_seconds_per_position(inp, kind, aux, per_step)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_seconds_per_position(inp, kind, aux, per_step)
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    cores = blas_threads()
    sample = f"first {per_step} of {shape.N} positions per step at full d, V, n, r (fp64 numpy)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(workload),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def roofline_of(shape, kind, workload, avg_ms, long_run, peaks) -> dict:
    """Roofline of the dominant kernel (the fused unembedding; the KL sweep for the distillation workload):
    algorithmic flops or bytes of one launch over its mean CUDA-event duration.  Draft scoring sits below,
    at or above the ridge depending on the number of logit rows N*n*r (flop per byte of E streamed), so for
    it both fractions are given: the binding one as the roofline itself, the other under "also"."""
    K = shape.n * shape.r
    rows = shape.N * K
    sec = max(avg_ms, 1e-9) * 1e-3
    t_alg = 2.0 * rows * shape.V * shape.d
    b_alg = 2.0 * shape.V * shape.d
    tensor_peak = peaks["sustained"] if long_run else peaks["burst"]
    tensor = {"bound": "tensor", "achieved": t_alg / sec / 1e12, "peak": tensor_peak, "unit": "TFLOP/s",
              "peak_kind": "sustained" if long_run else "burst", "algorithmic_per_launch": t_alg}
    hbm = {"bound": "hbm", "achieved": b_alg / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
           "algorithmic_per_launch": b_alg}
    for r in (tensor, hbm):
        r["frac"] = r["achieved"] / r["peak"]
    if kind in ("score", "sample"):
        ridge = peaks["burst"] * 1e12 / (peaks["hbm_gbs"] * 1e9)   # flop per byte where the two bounds meet
        roof, other = (hbm, tensor) if rows < ridge else (tensor, hbm)
        roof["also"] = {k: other[k] for k in ("bound", "achieved", "peak", "unit", "frac")}
        roof["flop_per_byte"] = float(rows)
        roof["ridge_flop_per_byte"] = ridge
    else:
        roof = tensor
    roof["traffic"] = ncu_traffic_bytes(workload)
    roof["kernel"] = "tc_gemm_kernel<EpiLse> (unembedding + logsumexp_V)"
    if kind == "distill":
        roof["kernel"] = "tc_gemm_kernel<EpiKl> (unembedding + expert mixture + KL to the teacher, grouped rows)"
    if kind == "full_fwd_bwd":
        roof["kernel"] = "tc_gemm_kernel<EpiLseFull> (all heads' unembeddings + logsumexp_V in one GEMM)"
    roof["peak_source"] = peaks["src"]
    roof["avg_launch_ms"] = avg_ms
    return roof


def bench_workload(env, workload: str, steps: int, warmup: int, with_graph: bool):
    """Time one workload: `warmup` untimed steps, `steps` timed ones (device time, max over ranks), the same
    through host buffers, and for draft scoring a CUDA-graph replay.  Returns (entry, inputs)."""
    import torch

    binding, dist_util, synth = env["binding"], env["dist_util"], env["synth"]
    rank, world, device, sampler, peaks = env["rank"], env["world"], env["device"], env["sampler"], env["peaks"]
    cfg, kind, extra, aux = WORKLOADS[workload]
    shape = synth.CONFIGS[cfg]
    inp = synth.make_inputs(shape, seed=dist_util.shard_seed(0, rank), **extra)
    h, W_head, E, W_g, x = [t.cuda() for t in (inp.h, inp.W_head, inp.E, inp.W_g, inp.x)]
    cs = binding.make_shape(shape.N, shape.d, shape.V, shape.n, shape.r, aux)
    ws_fwd = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_FORWARD) +
                                     binding.host_staging_bytes(cs) + 512)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    saved = binding.Saved.alloc(cs) if kind in ("fwd_bwd", "distill") else None
    W_full = ws_ff = ws_fb = None
    teacher = dsaved = ws_df = ws_db = None
    if kind == "distill":
        teacher = synth.make_teacher_logits(shape, inp.x, seed=dist_util.shard_seed(0, rank)).cuda()
        dsaved = binding.DistillSaved.alloc(cs)
        ws_df = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_DISTILL_FORWARD))
        ws_db = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_DISTILL_BACKWARD))
    if kind == "full_fwd_bwd":
        W_full = synth.make_full_head(shape, seed=dist_util.shard_seed(0, rank)).cuda()
        saved = binding.Saved.alloc_full(cs)
        ws_ff = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_FORWARD_FULL))
        ws_fb = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_BACKWARD_FULL))
    ws_bwd = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_BACKWARD)) if kind == "fwd_bwd" else None
    ws_smp = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_SAMPLE)) if kind == "sample" else None
    out_f, out_b, out_s = {}, {}, {}
    skip = ("dE", "dh") if workload == "finetune_fwd_bwd" or kind == "distill" else ()

    def step():
        if kind == "fwd":
            binding.forward(h, W_head, E, W_g, x, aux_coef=aux, workspace=ws_fwd, dev_status=status, out=out_f)
        elif kind == "fwd_bwd":
            binding.forward(h, W_head, E, W_g, x, aux_coef=aux, saved=saved, workspace=ws_fwd, dev_status=status,
                            out=out_f)
            binding.backward(h, W_head, E, W_g, x, saved, aux_coef=aux, workspace=ws_bwd, dev_status=status,
                             out=out_b, skip=skip)
        elif kind == "distill":
            binding.distill_forward(h, W_head, E, W_g, x, teacher, saved, dsaved, beta=0.9, gamma=0.8,
                                    workspace=ws_df, dev_status=status, out=out_f)
            binding.distill_backward(h, W_head, E, W_g, x, teacher, saved, dsaved, beta=0.9, gamma=0.8,
                                     workspace=ws_db, dev_status=status, out=out_b, skip=skip)
        elif kind == "sample":
            binding.sample_draft(h, W_head, E, W_g, shape.n, topk=5, workspace=ws_smp, dev_status=status, out=out_s)
        elif kind == "full_fwd_bwd":
            binding.forward_full(h, W_full, W_g, x, saved=saved, workspace=ws_ff, dev_status=status, out=out_f)
            binding.backward_full(h, W_full, W_g, x, saved, workspace=ws_fb, dev_status=status, out=out_b)
        else:
            binding.score_draft(h, W_head, E, W_g, x, workspace=ws_fwd, dev_status=status, out=out_s)

    h_pin, x_pin = inp.h.pin_memory(), inp.x.pin_memory()
    logp_pin = torch.empty(shape.N, dtype=torch.float32).pin_memory()
    prefix_pin = torch.empty((shape.N, shape.n), dtype=torch.float32).pin_memory()
    loss_pin = torch.empty(1, dtype=torch.float32).pin_memory()
    draft_pin = torch.empty((shape.N, shape.n), dtype=torch.int32).pin_memory()

    def step_e2e():
        """The same step with the per-step operands in pinned host memory and the result read on the host."""
        if kind == "sample":
            h.copy_(h_pin, non_blocking=True)
            binding.sample_draft(h, W_head, E, W_g, shape.n, topk=5, workspace=ws_smp, dev_status=status, out=out_s)
            draft_pin.copy_(out_s["draft"], non_blocking=True)
        elif kind == "score":
            h.copy_(h_pin, non_blocking=True)
            x.copy_(x_pin, non_blocking=True)
            step()
            logp_pin.copy_(out_s["logp_joint"], non_blocking=True)
            prefix_pin.copy_(out_s["logp_prefix"], non_blocking=True)
        elif kind in ("full_fwd_bwd", "distill"):
            h.copy_(h_pin, non_blocking=True)
            x.copy_(x_pin, non_blocking=True)
            step()
            loss_pin.copy_(out_f["loss"], non_blocking=True)
        else:
            binding.forward_host(h_pin, W_head, E, W_g, x_pin, logp_pin, loss_pin, aux_coef=aux, saved=saved,
                                 workspace=ws_fwd, dev_status=status)
            if kind == "fwd_bwd":
                binding.backward(h, W_head, E, W_g, x, saved, aux_coef=aux, workspace=ws_bwd, dev_status=status,
                                 out=out_b, skip=skip)
        torch.cuda.current_stream().synchronize()   # the step's result is read on the host

    if kind == "sample":
        h2d, d2h = shape.N * shape.d * 2, shape.N * shape.n * 4
    elif kind == "score":
        h2d, d2h = shape.N * shape.d * 2 + shape.N * shape.n * 4, shape.N * 4 + shape.N * shape.n * 4
    elif kind in ("full_fwd_bwd", "distill"):
        h2d, d2h = shape.N * shape.d * 2 + shape.N * shape.n * 4, 4
    else:
        h2d, d2h = shape.N * shape.d * 2 + shape.N * shape.n * 4, shape.N * 4 + 4

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()
        torch.cuda.synchronize()

    def timed(fn, count, profile):
        barrier()
        if profile:
            binding.profile_begin()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        for _ in range(count):
            fn()
        e1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        stages = binding.profile_end() if profile else {}
        ms = e0.elapsed_time(e1)
        barrier()
        return dist_util.max_over_ranks(ms, device), stages, (t0, t1)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    t_probe = time.perf_counter()
    step()
    torch.cuda.synchronize()
    est_ms = dist_util.max_over_ranks(1e3 * (time.perf_counter() - t_probe), device)   # one decision for all ranks
    if est_ms >= 2.0:
        # long steps: a pair of CUDA events around every launch costs nothing measurable, so the per-stage times
        # (and the dominant kernel's mean duration for the roofline) come from the timed region itself
        ms_total, stages, window = timed(step, steps, True)
        prof_steps, ms_prof = steps, ms_total
    else:
        # launch-bound steps (draft scoring): the timed region holds nothing but the library's own launches, and
        # the per-stage times come from the same steps run once more with events around every launch (which keep
        # consecutive launches from overlapping, so that pass is a little slower and `value` does not use it)
        ms_total, _, window = timed(step, steps, False)
        prof_steps = steps
        ms_prof, stages, _ = timed(step, prof_steps, True)
    clocks = sampler.summary(*window) if sampler is not None else None
    graph_ms = None
    if kind in ("score", "sample") and with_graph:   # launch-bound regime: the same step replayed from a CUDA graph
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        for _ in range(3):
            graph.replay()
        graph_ms, _, _ = timed(graph.replay, steps, False)
        del graph
    for _ in range(min(warmup, 3)):
        step_e2e()
    ms_e2e, _, window_e2e = timed(step_e2e, steps, False)
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item())} raised during the benchmark of {workload}")

    positions = shape.N * world
    dominant = "kl" if kind == "distill" else "lse"
    dom_ms, dom_launches = stages.get(dominant, (0.0, 0))
    avg_ms = dom_ms / max(1, dom_launches)
    roof = roofline_of(shape, kind, workload, avg_ms, ms_total > 2000.0, peaks)
    total_flops = flops_per_position(shape, kind, skip) * positions * steps
    entry = {
        "value": dist_util.whole_job_rate(shape.N, steps, world, ms_total), "unit": UNIT, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_total / steps, "config": config_of(workload), "clocks": clocks,
        "e2e": {"value": dist_util.whole_job_rate(shape.N, steps, world, ms_e2e), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps,
                "clocks": sampler.summary(*window_e2e) if sampler is not None else None},
        "gpu_launches": int(round(sum(c for _, c in stages.values()) * steps / prof_steps)),
        "roofline": roof,
        "model_flops_tflops": total_flops / (ms_total * 1e-3) / 1e12,
        "stages_ms_per_step": {k: v[0] / prof_steps for k, v in stages.items()},
        "profiled_pass": {"steps": prof_steps, "ms_per_step": ms_prof / prof_steps},
    }
    if graph_ms is not None:
        entry["cuda_graph_ms_per_step"] = graph_ms / steps
    return entry, inp


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch

    from paper_2410_17765_b200 import binding, dist_util, synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist_util.init("nccl", device)
    env = {"binding": binding, "dist_util": dist_util, "synth": synth, "rank": rank, "world": world,
           "device": device, "sampler": ClockSampler(local_rank) if rank == 0 else None, "peaks": measured_peaks()}
    headline = args.workload or HEADLINE
    entry, inp = bench_workload(env, headline, args.steps, args.warmup, not args.no_graph)
    cfg, kind, extra, aux = WORKLOADS[headline]
    shape = synth.CONFIGS[cfg]
    sec_per_pos = n_sub = None
    if rank == 0:   # the oracle, as it stands, on a bounded sample of the headline's positions (host cores)
        sec_per_pos, n_sub = oracle_seconds_per_position(inp, kind, aux, oracle_sample_size(shape, kind))
    del inp
    others = []
    if args.workload is None and world == 1:   # the scaling runs (N > 1) time the headline only
        for name, count in ALSO:
            gc.collect()
            torch.cuda.empty_cache()
            other, other_inp = bench_workload(env, name, count, max(3, min(args.warmup, 5)), not args.no_graph)
            del other_inp
            others.append(other)
    if env["sampler"] is not None:
        env["sampler"].stop()
    if rank != 0:
        dist_util.finalize()
        return
    line = {
        "metric": METRIC, "value": entry["value"], "unit": UNIT, "n_gpus": world, "steps": entry["steps"],
        "warmup": entry["warmup"], "ms_per_step": entry["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
    }
    for key in ("config", "clocks", "e2e", "gpu_launches", "roofline"):
        line[key] = entry[key]
    line["cpu_baseline"] = {"value": 1.0 / sec_per_pos, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                            "sample": f"first {n_sub} of {shape.N} positions at full d, V, n, r (fp64 numpy)"}
    for key in ("model_flops_tflops", "stages_ms_per_step", "cuda_graph_ms_per_step"):
        if key in entry:
            line[key] = entry[key]
    if others:
        line["workloads"] = others
    print(json.dumps(line))
    dist_util.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(WORKLOADS),
                    help="time this workload alone (default: the large forward+backward step as the headline, "
                         "then the other regimes of the metric in a `workloads` list)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay leg of the decode workloads")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
