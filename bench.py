#!/usr/bin/env python
"""Benchmark of the fused CP-head log-likelihood on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path of the workload over one batch of seeded
synthetic inputs: forward for `train_fwd`, forward + backward for the `*_fwd_bwd`
workloads, draft scoring for `decode_*`.  Prints ONE JSON line.  With N > 1 ranks
(torchrun) every rank runs the same per-GPU batch (positions are independent, no
collective on the data path) and the reported value is the whole-job rate.
"""
from __future__ import annotations

import argparse
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None until captured, or once the kernel has changed since).
NCU_TRAFFIC_BYTES = {
    "train_fwd": 1.211966e9 + 5.231616e6,   # profiles/lse_train_fwd.md
    "decode_1": 1.051677e9 + 3.764992e6,    # profiles/decode_1.md
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], burst=p["bf16_tflops"], sustained=p["bf16_tflops_sustained"], src="measured")
    return dict(hbm_gbs=6650.0, burst=1590.0, sustained=1400.0, src="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples.  The query loop is started early (it needs a moment to come
    up) and every sample is stamped on arrival; only those that arrived between begin() and end(), i.e. while
    the timed region ran, are summarised."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        import threading

        self.proc = None
        self.samples = []
        self.t0 = self.t1 = None
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

    def begin(self):
        self.t0 = time.perf_counter()

    def end(self):
        self.t1 = time.perf_counter()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)
        inside = [ln for t, ln in self.samples if self.t0 is not None and self.t0 <= t <= self.t1]
        window = "timed region"
        if not inside:   # region shorter than the query interval: the samples closest to it
            inside = [ln for _, ln in self.samples[-3:]]
            window = "last samples before the end of the timed region"
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in inside:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}


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
    # about 10-30 s of fp64 numpy work: assume ~40 GFLOP/s on the host cores
    per_pos = flops_per_position(s, kind) * (1.4 if kind in ("fwd_bwd", "distill") else 1.0)
    return max(1, min(s.N, int(40e9 * 15 / per_pos)))


def run_reference(args, rank: int):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from paper_2410_17765_b200 import synth

    cfg, kind, extra, aux = WORKLOADS[args.workload]
    shape = synth.CONFIGS[cfg]
    inp = synth.make_inputs(shape, seed=0, **extra)
    # bounded sample per step so that the whole run ends within a few minutes
    per_step = max(1, oracle_sample_size(shape, kind) // max(1, 2 * (args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_seconds_per_position(inp, kind, aux, per_step)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_seconds_per_position(inp, kind, aux, per_step)
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    cores = blas_threads()
    sample = f"first {per_step} of {shape.N} positions per step at full d, V, n, r"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "kind": kind, **shape.__dict__},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch

    from paper_2410_17765_b200 import binding, dist_util, synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist_util.init("nccl", device)

    cfg, kind, extra, aux = WORKLOADS[args.workload]
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
    skip = ("dE", "dh") if args.workload == "finetune_fwd_bwd" or kind == "distill" else ()

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
    loss_pin = torch.empty(1, dtype=torch.float32).pin_memory()

    draft_pin = torch.empty((shape.N, shape.n), dtype=torch.int32).pin_memory()

    def step_e2e():
        if kind == "sample":
            h.copy_(h_pin, non_blocking=True)
            binding.sample_draft(h, W_head, E, W_g, shape.n, topk=5, workspace=ws_smp, dev_status=status, out=out_s)
            draft_pin.copy_(out_s["draft"], non_blocking=True)
            torch.cuda.current_stream().synchronize()
            return
        if kind in ("full_fwd_bwd", "distill"):
            h.copy_(h_pin, non_blocking=True)
            x.copy_(x_pin, non_blocking=True)
            step()
            loss_pin.copy_(out_f["loss"], non_blocking=True)
            torch.cuda.current_stream().synchronize()
            return
        binding.forward_host(h_pin, W_head, E, W_g, x_pin, logp_pin, loss_pin, aux_coef=aux, saved=saved,
                             workspace=ws_fwd, dev_status=status)
        if kind == "fwd_bwd":
            binding.backward(h, W_head, E, W_g, x, saved, aux_coef=aux, workspace=ws_bwd, dev_status=status,
                             out=out_b, skip=skip)
        torch.cuda.current_stream().synchronize()   # the step's result is read on the host

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, profile, clock_sampler=None):
        barrier()
        if profile:
            binding.profile_begin()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if clock_sampler is not None:
            clock_sampler.begin()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        if clock_sampler is not None:
            clock_sampler.end()
        stages = binding.profile_end() if profile else {}
        ms = e0.elapsed_time(e1)
        barrier()
        return dist_util.max_over_ranks(ms, device), stages

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    ms_total, stages = timed(step, args.steps, True, sampler)
    clocks = sampler.stop() if sampler is not None else None
    graph_ms = None
    if kind in ("score", "sample") and not args.no_graph:   # launch-bound regime: the same step replayed from a CUDA graph
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        for _ in range(3):
            graph.replay()
        graph_ms, _ = timed(graph.replay, args.steps, False)
    for _ in range(min(args.warmup, 3)):
        step_e2e()
    ms_e2e, _ = timed(step_e2e, args.steps, False)
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item())} raised during the benchmark")

    if rank != 0:
        dist_util.finalize()
        return
    peaks = measured_peaks()
    positions = shape.N * world
    value = dist_util.whole_job_rate(shape.N, args.steps, world, ms_total)
    e2e_value = dist_util.whole_job_rate(shape.N, args.steps, world, ms_e2e)
    K = shape.n * shape.r
    dominant = "kl" if kind == "distill" else "lse"
    dom_ms, dom_launches = stages.get(dominant, (0.0, 0))
    avg_ms = dom_ms / max(1, dom_launches)
    if kind in ("score", "sample") and shape.N * K * 2 < 250:   # below the ridge: HBM-bound streaming of E
        alg = 2.0 * shape.V * shape.d
        roof = {"bound": "hbm", "achieved": alg / (avg_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        alg = 2.0 * shape.N * K * shape.V * shape.d
        long_run = ms_total > 2000.0
        roof = {"bound": "tensor", "achieved": alg / (avg_ms * 1e-3) / 1e12,
                "peak": peaks["sustained"] if long_run else peaks["burst"], "unit": "TFLOP/s",
                "peak_kind": "sustained" if long_run else "burst"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(args.workload)
    roof["kernel"] = "tc_gemm_kernel<EpiLse> (unembedding + logsumexp_V)"
    if kind == "distill":
        roof["kernel"] = "tc_gemm_kernel<EpiKl> (unembedding + expert mixture + KL to the teacher, grouped rows)"
    if kind == "full_fwd_bwd":
        roof["kernel"] = "tc_gemm_kernel<EpiLseFull> (all heads' unembeddings + logsumexp_V in one GEMM)"
    roof["peak_source"] = peaks["src"]
    roof["avg_launch_ms"] = avg_ms
    roof["algorithmic_per_launch"] = alg
    total_flops = flops_per_position(shape, kind, skip) * positions * args.steps
    n_sub = oracle_sample_size(shape, kind)
    sec_per_pos, n_sub = oracle_seconds_per_position(inp, kind, aux, n_sub)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "kind": kind, **shape.__dict__, "aux_coef": aux,
                   "targets": extra.get("targets", "uniform"), "l2": "inputs larger than L2 (no flush)",
                   "per_gpu_positions": shape.N},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": shape.N * shape.d * 2 + (0 if kind == "sample" else shape.N * shape.n * 4),
                "d2h_bytes_per_step": shape.N * shape.n * 4 if kind == "sample" else shape.N * 4 + 4,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(sum(c for _, c in stages.values())),
        "roofline": roof,
        "cpu_baseline": {"value": 1.0 / sec_per_pos, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"first {n_sub} of {shape.N} positions at full d, V, n, r (fp64 numpy)"},
        "model_flops_tflops": total_flops / (ms_total * 1e-3) / 1e12,
        "stages_ms_per_step": {k: v[0] / args.steps for k, v in stages.items()},
    }
    if graph_ms is not None:
        line["cuda_graph_ms_per_step"] = graph_ms / args.steps
    print(json.dumps(line))
    dist_util.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="train_fwd", choices=sorted(WORKLOADS))
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
