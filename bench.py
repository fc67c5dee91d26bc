#!/usr/bin/env python
"""Benchmark of the restructured-FFN MoE forward on B200.

    python bench.py --gpus N --steps K --warmup W [--workload NAME --tokens T]
    python bench.py --impl reference ...        # the CPU oracle, as it stands, on host cores

A step is one pass of the whole forward (router, histogram/permute, shared and
routed SwiGLU expert GEMMs, combine) over one batch of T synthetic tokens.  The
path shards by tokens with no exchange, so N GPUs run N independent replicas
("replicas only"): value = N*T*K / max-over-ranks device time.  Prints ONE JSON
line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2502_04416_b200 import workloads as wl  # noqa: E402

METRIC = "moe_ffn_layer_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# ------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index
        self.begin = self.end = None

    def wait_first(self, timeout: float = 5.0):
        t0 = time.time()
        while not self.rows and time.time() - t0 < timeout and self.proc is not None:
            time.sleep(0.02)

    def mark_begin(self):
        self.begin = len(self.rows)

    def mark_end(self):
        self.end = len(self.rows)

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows, window = self.rows, "all samples while the process ran"
        if self.begin is not None and self.end is not None and self.end > self.begin:
            rows, window = self.rows[self.begin:self.end + 1], "timed region"
        elif self.begin is not None:
            rows, window = self.rows[max(self.begin - 1, 0):], "timed region shorter than one sample: nearest samples"
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm), "window": window}


# ------------------------------------------------------------- CPU oracle arm
def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_step(inputs: wl.WorkloadInputs, x: np.ndarray):
    """One oracle forward on x (the oracle as it stands: fp64 numpy)."""
    from oracle import cmoe_oracle as oracle
    w = inputs.workload
    s = w.shape

    def kw(lay):
        return dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down,
                    neuron_perm=lay.neuron_perm, rep_idx=lay.rep_idx, n_experts=s.n_experts,
                    n_shared=s.n_shared, top_k=s.top_k, gate_scale_u=lay.gate_scale_u,
                    select_bias_b=lay.select_bias_b)
    if w.n_outer:
        return oracle.hier_forward(x, inputs.w_router, w.outer_top_k, [kw(l) for l in inputs.layers])[0]
    return oracle.cmoe_layer_forward(x, **kw(inputs.layers[0]))[0]


def time_oracle(inputs, x, sample_tokens: int, repeats: int = 1):
    xs = x[:sample_tokens]
    oracle_step(inputs, xs[:min(8, len(xs))])              # import + BLAS warm-up
    t0 = time.perf_counter()
    for _ in range(repeats):
        oracle_step(inputs, xs)
    dt = (time.perf_counter() - t0) / repeats
    return len(xs) / dt, dt


def load_select_bias(name: str):
    path = os.path.join(ROOT, "tests", "golden", f"{name}_select_bias.txt")
    if not os.path.exists(path):
        return None
    return np.array([float(l) for l in open(path) if l.strip() and not l.startswith("#")],
                    dtype=np.float32)


def prepare_inputs(name: str):
    w = wl.WORKLOADS[name]
    inputs = wl.make_inputs(w)
    if w.zipf_s:
        b = load_select_bias(name)
        if b is not None:
            inputs.layers[0].select_bias_b = b
    return inputs


# DRAM bytes (read + write) per forward of the dominant kernels (the two expert GEMMs), from the ncu
# captures summarised under profiles/; an entry is only valid for the kernel version it was taken on,
# so the table is emptied whenever those kernels change and refilled from a new capture.
NCU_TRAFFIC = {
    ("c5_skew_13b", 16384): {"bytes": (1586.5 + 162.8 + 363.8 + 795.8) * 1e6,
                             "source": "profiles/umma2_pair_gemm_c5_skew_13b.md"},
    ("c2_llama2_7b", 4096): {"bytes": (282.2 + 34.5 + 138.5 + 68.2) * 1e6,
                             "source": "profiles/launch_lists_c2_c3_c4_prefill_and_mid_size.md"},
    ("c3_llama3_8b", 8192): {"bytes": (517.0 + 52.0 + 182.0 + 281.5) * 1e6,
                             "source": "profiles/launch_lists_c2_c3_c4_prefill_and_mid_size.md"},
    ("c4_hier_8x7b", 4096): {"bytes": (2038.5 + 111.7 + 1064.4 + 184.3) * 1e6,
                             "source": "profiles/launch_lists_c2_c3_c4_prefill_and_mid_size.md"},
}

# Every (workload, T) point the metric is quoted on; the last one (the largest single-GPU
# configuration) is the headline.
SWEEP_POINTS = [("c2_llama2_7b", 1), ("c2_llama2_7b", 16), ("c2_llama2_7b", 64), ("c2_llama2_7b", 512),
                ("c2_llama2_7b", 4096), ("c3_llama3_8b", 32), ("c3_llama3_8b", 8192), ("c4_hier_8x7b", 4096),
                ("c5_skew_13b", 16384)]
HEADLINE = SWEEP_POINTS[-1]
SWEEP_POINTS_FP8 = [("c2_llama2_7b", 1), ("c2_llama2_7b", 16), ("c2_llama2_7b", 64), ("c3_llama3_8b", 32)]
# between the decode and the prefill regime (not points of the metric: reported beside the sweep)
MID_POINTS = [("c2_llama2_7b", 128), ("c2_llama2_7b", 256), ("c2_llama2_7b", 1024),
              ("c3_llama3_8b", 128), ("c3_llama3_8b", 256), ("c3_llama3_8b", 512), ("c3_llama3_8b", 1024)]


def traffic_note(name, tokens, use_graph):
    rec = NCU_TRAFFIC.get((name, tokens))
    if rec is None or use_graph:
        return None
    return rec["bytes"]


def max_over_ranks(ms_local: float, device: str) -> float:
    """Slowest rank's device time: the job's time when every rank runs its own replica."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(world: int, tokens_per_step: int, steps: int, ms_max: float) -> float:
    """Whole-job tokens/s of `world` independent replicas (tokens shard with no exchange)."""
    return world * tokens_per_step * steps / (ms_max * 1e-3)


def replica_launch_command(n_gpus: int, argv, port: int):
    """The command that starts one process per GPU for `bench.py --gpus N` run without a launcher."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


# ------------------------------------------------------------------ GPU arm
class Rig:
    """Process-wide state of one benchmark run: rank layout, stream, timing helpers."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        self.torch, self.dist, self.args = torch, dist, args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if self.world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
        torch.cuda.set_device(self.local)
        self.stream = torch.cuda.current_stream()

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def timed(self, fn, steps):
        """Exactly `steps` calls between CUDA events on the launching stream, a barrier and a
        synchronize on both sides; the max over ranks, in milliseconds."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record(self.stream)
        for _ in range(steps):
            fn()
        e1.record(self.stream)
        self.barrier()
        return max_over_ranks(e0.elapsed_time(e1), "cuda")

    def timed_blocks(self, fn, steps, min_region_s, max_blocks):
        """Repeats the K-step block until the timed region reaches min_region_s (or max_blocks);
        returns the per-block times in ms.  Every rank runs the same number of blocks: the
        decision uses the max-over-ranks times."""
        blocks = []
        while True:
            blocks.append(self.timed(fn, steps))
            if sum(blocks) >= min_region_s * 1e3 or len(blocks) >= max_blocks:
                return blocks

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def dense_comparison(rig, inputs, x, steps, min_region_s=0.2):
    """The comparison run, never the product path: the dense FFN of the same d and d_ff through
    torch (cuBLAS); for the hierarchical workload the layer it replaces, a plain top-2 MoE whose
    selected experts run as dense per-expert cuBLAS GEMMs on their tokens."""
    torch = rig.torch
    from paper_2502_04416_b200 import torch_io
    F = torch.nn.functional
    w, s = inputs.workload, inputs.workload.shape
    T = x.shape[0]
    ws = [tuple(torch_io.to_device(a, s.dtype) for a in (l.w_gate, l.w_up, l.w_down)) for l in inputs.layers]
    if w.n_outer:
        w_r = torch_io.to_device(inputs.w_router, s.dtype)
        kind = ("plain top-%d MoE over the %d dense outer experts: torch router + per-expert F.linear x3 + "
                "silu*mul on the expert's tokens (cuBLAS) + index_add" % (w.outer_top_k, w.n_outer))

        def step():
            logits = F.linear(x, w_r).float()
            top, idx = logits.topk(w.outer_top_k, dim=1)
            wt = torch.softmax(top, dim=1).to(x.dtype)
            out = torch.zeros_like(x)
            for i, (wg, wu, wd) in enumerate(ws):
                tok, slot = (idx == i).nonzero(as_tuple=True)
                if tok.numel():
                    xi = x[tok]
                    y = F.linear(F.silu(F.linear(xi, wg)) * F.linear(xi, wu), wd)
                    out.index_add_(0, tok, y * wt[tok, slot].unsqueeze(1))
            return out
    else:
        wg, wu, wd = ws[0]
        kind = "torch F.linear x3 + silu*mul (cuBLAS), same d and d_ff"

        def step():
            return F.linear(F.silu(F.linear(x, wg)) * F.linear(x, wu), wd)
    for _ in range(3):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    while sum(times) < min_region_s * 1e3 and len(times) < 50:
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    dms = statistics.median(times) / steps
    del ws
    return {"kind": kind, "ms_per_step": dms, "value": T / (dms * 1e-3), "unit": UNIT}


def roofline_record(peaks, w, T, touched, step_ms, first_ms, gemm_ms, stage_ms, use_graph, weight_bytes=None):
    """Algorithmic work of one forward against the measured peaks (flops 6 d m (N_s+N_k) per
    token; bytes = every touched expert's weights once + x read + out write)."""
    s = w.shape
    mult = w.outer_top_k if w.n_outer else 1
    flops = mult * T * 6 * s.d_model * s.m * (s.n_shared + s.top_k)
    w_bytes = (w.n_outer if w.n_outer else 1) * (s.n_shared + touched) * s.expert_weight_bytes()
    if weight_bytes is not None:               # quantised weights: bytes per weight instead of the storage type's
        w_bytes = w_bytes // s.elem_bytes * weight_bytes
    alg_bytes = w_bytes + 2 * T * s.d_model * s.elem_bytes
    t_tensor = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        ach = flops / (gemm_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops"], "frac_of_sustained": ach / peaks["bf16_tflops_sustained"]}
        t_roof, t_sus = t_tensor, flops / (peaks["bf16_tflops_sustained"] * 1e12)
    else:
        ach = alg_bytes / (gemm_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"]}
        t_roof, t_sus = t_hbm, t_hbm
    roof.update({
        "kernel": ("expert GEMMs (gate/up + SwiGLU, down), timed by per-stage events in a separate short loop"
                   if not use_graph else "whole forward, all kernels (CUDA graph replay; no per-stage events)"),
        "kernel_ms": gemm_ms, "peak_source": peaks["source"], "traffic": traffic_note(w.name, T, use_graph),
        "algorithmic_flops": flops, "algorithmic_bytes": alg_bytes,
        "whole_step_frac": t_roof / (step_ms * 1e-3),                    # median block, against the burst peak
        "whole_step_frac_first_block": t_roof / (first_ms * 1e-3),
        "whole_step_frac_of_sustained": t_sus / (step_ms * 1e-3),
        "other_bound_frac": (t_hbm if t_tensor >= t_hbm else t_tensor) / (step_ms * 1e-3),
        "stage_ms": stage_ms})
    return roof, w_bytes


def measure_point(rig, inputs, layer, T, min_region_s, max_blocks, with_dense, fp8=False):
    """Times the forward of `layer` on the first T tokens of the workload, device-resident.
    Returns the sweep record plus what the headline line needs."""
    torch, args = rig.torch, rig.args
    from paper_2502_04416_b200 import binding, torch_io
    w, s = inputs.workload, inputs.workload.shape
    x = torch_io.to_device(inputs.x[:T], s.dtype)
    out = torch.empty_like(x)
    use_graph = args.graph == "on" or (args.graph == "auto" and T <= 512)
    layer.set_launch_chaining(args.chain != "off")
    if args.gemm_path:
        layer.set_gemm_path(args.gemm_path)
    layer.enable_stage_timing(0)
    if use_graph:     # launch-bound sizes: the same C-ABI call captured once and replayed
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                layer.forward(x, out)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            layer.forward(x, out)
        step = graph.replay
    else:
        step = lambda: layer.forward(x, out)
    sampler = ClockSampler(rig.local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    sampler.wait_first()
    sampler.mark_begin()
    blocks = rig.timed_blocks(step, args.steps, min_region_s, max_blocks)
    sampler.mark_end()
    time.sleep(0.12)                                          # let the sample that covers the end arrive
    clocks = sampler.stop()
    launches_per_step = layer.launch_count()
    assert layer.status() == 0, "device-side wait timed out"
    step_ms = statistics.median(blocks) / args.steps
    first_ms = blocks[0] / args.steps
    # per-stage split: a second, short loop with the library's stage events (ordinary launches)
    stage_ms, gemm_ms = None, step_ms
    if not use_graph:
        n_st = max(3, min(args.steps, 50))
        layer.enable_stage_timing(n_st)
        for _ in range(n_st):
            layer.forward(x, out)
        ms, n_cov = layer.stage_times()
        layer.enable_stage_timing(0)
        stage_ms = {n: v / max(n_cov, 1) for n, v in zip(binding.STAGE_NAMES, ms)}
        gemm_ms = stage_ms["gemm1_swiglu"] + stage_ms["gemm2_down"]
    touched = s.n_routed
    if not w.n_outer and T * s.top_k < 64 * s.n_routed:
        layer.forward(x, out)
        touched = int((layer.routing(T, s.n_routed)["counts"] > 0).sum())
    peaks = load_peaks()
    roof, w_bytes = roofline_record(peaks, w, T, touched, step_ms, first_ms, gemm_ms, stage_ms, use_graph,
                                    weight_bytes=1 if (fp8 and T <= 64) else None)
    dense = dense_comparison(rig, inputs, x, args.steps) if (with_dense and rig.rank == 0) else None
    rec = {"workload": w.name, "tokens": T, "expert_weights": "fp8 e4m3 + per-channel 2^k scale" if fp8 else s.dtype,
           "ms_per_step": step_ms, "first_block_ms_per_step": first_ms,
           "blocks": len(blocks), "timed_region_s": sum(blocks) * 1e-3,
           "value": replica_throughput(rig.world, T, 1, step_ms), "unit": UNIT,
           "launch": "CUDA graph replay" if use_graph else "direct launches, chained",
           "launches_per_step": launches_per_step, "routed_experts_touched": touched,
           "roofline": {k: roof[k] for k in ("bound", "frac", "achieved", "peak", "unit", "kernel_ms", "traffic", "whole_step_frac",
                                             "whole_step_frac_first_block", "whole_step_frac_of_sustained",
                                             "other_bound_frac", "stage_ms")},
           "dense_cublas": dense, "clocks": clocks}
    if dense:
        rec["speedup_vs_dense"] = dense["ms_per_step"] / step_ms
    return rec, roof, (x, out, step, w_bytes)


def run_gpu(args):
    import torch
    from paper_2502_04416_b200 import binding
    from paper_2502_04416_b200 import torch_io

    rig = Rig(args)
    binding.load()
    world, rank = rig.world, rig.rank
    name = args.workload or HEADLINE[0]
    inputs = prepare_inputs(name)
    w = inputs.workload
    s = w.shape
    T = args.tokens or w.t_max
    layer = torch_io.layer_from_workload(inputs, w.t_max if T <= w.t_max else T)
    if args.fp8:
        layer.quantise_fp8()

    if args.forward_only:                     # profiling runs: nothing but the forward passes
        x = torch_io.to_device(inputs.x[:T], s.dtype)
        out = torch.empty_like(x)
        if args.chain == "off":
            layer.set_launch_chaining(False)
        for _ in range(args.warmup):
            layer.forward(x, out)
        ms = rig.timed(lambda: layer.forward(x, out), args.steps)
        assert layer.status() == 0
        if rank == 0:
            print(json.dumps({"forward_only": True, "workload": f"{w.name} T={T}", "ms_per_step": ms / args.steps}))
        rig.close()
        return None

    # ---- headline: device-resident, K-step blocks repeated over at least a second
    head, roof, (x, out, step, w_bytes) = measure_point(rig, inputs, layer, T, args.min_region_s, 400,
                                                        with_dense=True, fp8=args.fp8)
    launches = head["launches_per_step"] * args.steps

    # ---- end to end through the public host-buffer call: H2D and D2H copies inside the timed region
    x_pin = torch.empty(x.shape, dtype=x.dtype).pin_memory()
    x_pin.copy_(x.cpu())
    out_pin = torch.empty(x.shape, dtype=x.dtype).pin_memory()

    def e2e_step():
        layer.forward_host(x_pin, out_pin, args.e2e_chunk)
    for _ in range(max(min(args.warmup, 5), 3)):
        e2e_step()
    e2e_blocks = rig.timed_blocks(e2e_step, args.steps, min(args.min_region_s, 0.5), 100)
    e2e_ms = statistics.median(e2e_blocks) / args.steps
    io_bytes = T * s.d_model * s.elem_bytes
    torch.cuda.synchronize()
    same = bool(torch.equal(out_pin.view(torch.int16), out.cpu().view(torch.int16))) if s.dtype == "bf16" else None

    # ---- CPU baseline: the oracle on a bounded sample, on this machine's host cores (rank 0)
    cpu = None
    if rank == 0:
        sample = min(args.cpu_sample_tokens, T)
        cpu_v, cpu_dt = time_oracle(inputs, inputs.x[:T], sample)
        cpu = {"value": cpu_v, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
               "sample": f"first {sample} tokens of the same workload, one pass, {cpu_dt:.2f} s"}

    # ---- the other (workload, T) points
    sweep = None
    mid = []
    do_sweep = args.sweep == "on" or (args.sweep == "auto" and world == 1 and (name, T) == HEADLINE)
    if do_sweep:
        found = {(head["workload"], head["tokens"]): head}
        del x, out, step
        order = [name] + [n_ for n_ in dict.fromkeys(p_[0] for p_ in SWEEP_POINTS) if n_ != name]
        for n_ in order:
            ts = [t_ for m_, t_ in SWEEP_POINTS if m_ == n_ and (m_, t_) not in found]
            ts_mid = [t_ for m_, t_ in MID_POINTS if m_ == n_]
            if not ts and not ts_mid:
                continue
            if n_ != name:
                layer.destroy()
                del inputs, layer
                torch.cuda.empty_cache()
                inputs = prepare_inputs(n_)
                layer = torch_io.layer_from_workload(inputs, inputs.workload.t_max)
                name = n_
            for t_ in ts:
                found[(n_, t_)], _, _ = measure_point(rig, inputs, layer, t_, args.sweep_region_s, 200, with_dense=True)
            for t_ in ts_mid:
                rec, _, _ = measure_point(rig, inputs, layer, t_, args.sweep_region_s / 2, 200, with_dense=True)
                mid.append(rec)
        sweep = [found[p_] for p_ in SWEEP_POINTS if p_ in found]
        # decode points again with FP8 expert weights (quantising a layer is permanent, so these come last)
        for n_ in dict.fromkeys(p_[0] for p_ in SWEEP_POINTS_FP8):
            if n_ != name:
                layer.destroy()
                del inputs, layer
                torch.cuda.empty_cache()
                inputs = prepare_inputs(n_)
                layer = torch_io.layer_from_workload(inputs, 64)
                name = n_
            layer.quantise_fp8()
            for m_, t_ in SWEEP_POINTS_FP8:
                if m_ == n_:
                    rec, _, _ = measure_point(rig, inputs, layer, t_, args.sweep_region_s, 200, with_dense=False, fp8=True)
                    sweep.append(rec)

    if rank != 0:
        rig.close()
        return None

    line = {
        "metric": METRIC, "value": replica_throughput(world, T, 1, head["ms_per_step"]), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": s.dtype, "data": "synthetic",
        "config": {"workload": f"{w.name} T={T}", "note": w.note, "d_model": s.d_model,
                   "d_ff": s.d_ff, "experts": f"S{s.n_shared}A{s.top_k}E{s.n_experts}",
                   "tokens_per_step": T, "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "weights (%.0f MB) exceed the 126 MB L2" % (w_bytes / 1e6),
                   "launch": head["launch"],
                   "timing": "the K-step block is repeated until the timed region reaches %.1f s; ms_per_step is "
                             "the median block / K, first_block_ms_per_step the first" % args.min_region_s},
        "first_block_ms_per_step": head["first_block_ms_per_step"], "blocks": head["blocks"],
        "timed_region_s": head["timed_region_s"],
        "e2e": {"value": world * T / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": io_bytes, "d2h_bytes_per_step": io_bytes,
                "call": "cmoe_ffn_forward_host: pinned host x and out, chunks double-buffered on two copy streams",
                "chunk_tokens": args.e2e_chunk or "auto", "ms_per_step": e2e_ms,
                "bit_identical_to_device_call": same},
        "gpu_launches": launches, "clocks": head["clocks"], "roofline": roof, "cpu_baseline": cpu,
        "dense_cublas": head["dense_cublas"], "speedup_vs_dense": head.get("speedup_vs_dense"),
    }
    if sweep is not None:
        line["sweep"] = sweep
        line["mid_size"] = mid
    rig.close()
    return line


def run_ranks(args):
    """Launch-path self-check that needs no GPU: every rank joins a gloo group, reports a
    rank-dependent stand-in time, and rank 0 prints the replica arithmetic of the real run."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = max_over_ranks(10.0 + 5.0 * rank, "cpu")
    line = {"stage": "ranks", "n_gpus": world, "ms_max": ms,
            "value": replica_throughput(world, 4096, args.steps, ms)}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return line if rank == 0 else None


# ------------------------------------------------------------ reference arm
# ------------------------------------------------- activation profiling stage
def run_profile(args):
    """Steps 1-4 of the paper's activation-profiling pipeline on a synthetic calibration set of the
    paper's size (8 x 2048 tokens, K_a = 10) for the workload's FFN: a step is one pass over the set
    in chunks of 4096 rows plus the shared-neuron selection."""
    import dataclasses
    import numpy as np
    import torch
    from paper_2502_04416_b200 import binding, torch_io

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    binding.load()
    w = wl.WORKLOADS[args.workload]
    shape = dataclasses.replace(w.shape, n_shared=w.shape.n_experts, top_k=0)
    inputs = wl.make_inputs(dataclasses.replace(w, shape=shape, tokens=(8,), n_outer=0))
    lay = inputs.layers[0]
    lay.neuron_perm = np.arange(shape.d_ff, dtype=np.int32)
    lay.rep_idx = np.zeros(0, dtype=np.int32)
    q, chunk, k_a = args.tokens or 16384, 4096, 10
    n_select = 2 * (shape.d_ff // shape.n_experts)
    rng = np.random.Generator(np.random.PCG64(1234))
    x_host = wl.round_to_storage(rng.standard_normal((q, shape.d_model), dtype=np.float32), shape.dtype)
    layer = torch_io.layer_from_inputs(lay, min(chunk, q))
    x = torch_io.to_device(x_host, shape.dtype)
    bits = torch.zeros((shape.d_ff, (q + 31) // 32), dtype=torch.int32, device="cuda")
    count = torch.zeros(shape.d_ff, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        bits.zero_()
        count.zero_()
        for t0 in range(0, q, chunk):
            layer.profile_activations(x[t0:t0 + chunk], k_a, bits, count, token0=t0)
        return binding.select_shared(count, n_select)

    steps = min(args.steps, 200)
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler.wait_first()
    sampler.mark_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    sampler.mark_end()
    time.sleep(0.12)
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), "cuda")
    assert layer.status() == 0
    value = world * q * steps / (ms_total * 1e-3)
    peaks = load_peaks()
    flops = 4.0 * shape.d_model * shape.d_ff * q
    ach = flops / (ms_total / steps * 1e-3) / 1e12
    line = {
        "metric": "activation_profile_tokens_per_s", "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": shape.dtype, "data": "synthetic",
        "config": {"workload": f"{w.name} profiling q={q} K_a={k_a}", "d_model": shape.d_model, "d_ff": shape.d_ff,
                   "chunk": chunk, "l2": "weights and H exceed the 126 MB L2"},
        "gpu_launches": (3 * ((q + chunk - 1) // chunk) + 1) * steps, "clocks": clocks,
        "roofline": {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": ach / peaks["bf16_tflops"], "traffic": None,
                     "kernel": "whole profiling pass (gate/up GEMM + ATopK + selection)",
                     "peak_source": peaks["source"]},
    }
    if rank == 0:
        from oracle import cmoe_oracle as oracle
        sample = min(args.cpu_sample_tokens, q)
        t0 = time.perf_counter()
        oracle.profile_activations(x_host[:sample], lay.w_gate, lay.w_up, k_a, n_select)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": sample / dt, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                                "sample": f"first {sample} calibration rows, one pass, {dt:.2f} s"}
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return line if rank == 0 else None


# ----------------------------------------------------- clustering-round stage
def run_cluster(args):
    """One round of the data-parallel clustering pieces (centroid update, distance matrix,
    representatives) at the paper's scale: 16384 calibration tokens, K_a = 10, the workload's d_h,
    N_r clusters of m neurons.  The activation matrix and the balanced assignment are synthetic
    inputs (the assignment solver is a sequential CPU algorithm and not part of the step)."""
    import numpy as np
    import torch
    from paper_2502_04416_b200 import binding

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if int(os.environ.get("RANK", "0")) != 0:
        return None
    torch.cuda.set_device(local)
    binding.load()
    w = wl.WORKLOADS[args.workload]
    s = w.shape
    q, k_a, m, n_r = args.tokens or 16384, 10, s.d_ff // s.n_experts, s.n_routed
    rng = np.random.Generator(np.random.PCG64(4321))
    # K_a active neurons per token, popularity skewed as in the paper's rate histogram
    pop = np.exp(rng.normal(scale=1.0, size=s.d_ff))
    picks = np.stack([rng.choice(s.d_ff, size=k_a, replace=False, p=pop / pop.sum()) for _ in range(q)])
    words = (q + 31) // 32
    bits_host = np.zeros((s.d_ff, words), dtype=np.uint32)
    t = np.repeat(np.arange(q), k_a)
    np.bitwise_or.at(bits_host, (picks.ravel(), t // 32), (np.uint32(1) << (t % 32).astype(np.uint32)))
    counts = np.bincount(picks.ravel(), minlength=s.d_ff)
    order = np.argsort(-counts, kind="stable")
    rest = np.sort(order[s.n_shared * m:]).astype(np.int32)          # the N_r * m neurons to cluster
    assign_host = rng.permutation(np.repeat(np.arange(n_r), m)).astype(np.int32)
    bits = torch.from_numpy(bits_host.view(np.int32)).cuda()
    rest_d, assign_d = torch.from_numpy(rest).cuda(), torch.from_numpy(assign_host).cuda()
    count = torch.zeros((n_r, q), dtype=torch.int32, device="cuda")
    size = torch.ones(n_r, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        binding.cluster_update(bits, q, rest_d, assign_d, count, size)
        sd = binding.cluster_distances(bits, q, rest_d, count, size)
        return binding.cluster_representatives(sd, rest_d, assign_d)

    steps = min(args.steps, 200)
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler.wait_first()
    sampler.mark_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    sampler.mark_end()
    time.sleep(0.12)
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    n = len(rest)
    peaks = load_peaks()
    alg_bytes = 2.0 * n * words * 4 + 3.0 * n_r * q * 4 + n * n_r * 8     # bit rows twice, counts written/read, D written
    line = {
        "metric": "cluster_round_neurons_per_s", "value": n / (ms * 1e-3), "unit": "neurons/s", "n_gpus": 1,
        "steps": steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": f"{w.name} clustering round q={q} K_a={k_a}", "neurons": n, "clusters": n_r,
                   "l2": "inputs (19 MB) fit the 126 MB L2: a latency-bound step"},
        "gpu_launches": 5 * steps, "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": alg_bytes / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": alg_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "kernel": "centroid update + distance matrix + representatives", "peak_source": peaks["source"]},
    }
    from oracle import cmoe_oracle as oracle
    sample_q, sample_n = min(q, 512), min(n, 1024)
    a = ((bits_host[rest[:sample_n]][:, np.arange(sample_q) // 32] >> (np.arange(sample_q) % 32).astype(np.uint32)) & 1).T
    sub = np.minimum(assign_host[:sample_n], n_r - 1)
    t0 = time.perf_counter()
    cent = oracle.cluster_update(a, sub, np.zeros((sample_q, n_r)))
    oracle.representatives(a, sub, cent)
    dt = time.perf_counter() - t0
    line["cpu_baseline"] = {"value": sample_n / dt, "unit": "neurons/s", "cores": host_threads(), "kind": "oracle",
                            "sample": f"{sample_n} neurons x {sample_q} tokens, one round, {dt:.2f} s"}
    return line


def run_reference(args):
    """The CPU oracle, unmodified, timed on the host cores on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    inputs = prepare_inputs(args.workload)
    w = inputs.workload
    T = args.tokens or w.t_max
    sample = min(args.cpu_sample_tokens, T)
    # The oracle streams every active expert's fp64 weights on each call, so a step costs a fixed
    # fraction of a second however few tokens it carries.  The run is held to a few minutes: the sample
    # per step is sized from a two-point calibration (never below 64 tokens), and where K such steps do
    # not fit, the timed loop stops at the time budget and reports the steps it took ("steps_requested" keeps K).
    budget_s = 240.0
    oracle_step(inputs, inputs.x[:1])                          # import + BLAS warm-up
    t0 = time.perf_counter()
    oracle_step(inputs, inputs.x[:1])
    t_one = time.perf_counter() - t0
    cal = min(32, sample)
    t0 = time.perf_counter()
    oracle_step(inputs, inputs.x[:cal])
    t_cal = time.perf_counter() - t0
    per_tok = max((t_cal - t_one) / max(cal - 1, 1), 1e-7)
    room = budget_s / max(args.steps, 1) - t_one               # seconds a step may spend on tokens
    sample = max(min(64, sample), min(sample, int(room / per_tok) if room > 0 else 1))   # at least 64 tokens: fewer steps instead
    xs = inputs.x[:sample]
    for _ in range(min(args.warmup, 2)):
        oracle_step(inputs, xs)
    steps_done = 0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(inputs, xs)
        steps_done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    v = sample * steps_done / dt
    s = w.shape
    desc = f"first {sample} tokens of the workload per step"
    return {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps_done, "steps_requested": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / steps_done * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name} T={T}", "sample": desc, "d_model": s.d_model, "d_ff": s.d_ff,
                   "experts": f"S{s.n_shared}A{s.top_k}E{s.n_experts}"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=None, choices=sorted(wl.WORKLOADS),
                    help="default: the largest single-GPU configuration, c5_skew_13b")
    ap.add_argument("--tokens", type=int, default=0, help="tokens per step (default: the workload's largest T)")
    ap.add_argument("--cpu-sample-tokens", type=int, default=256)
    ap.add_argument("--graph", choices=["auto", "on", "off"], default="auto",
                    help="replay the forward from a CUDA graph (auto: batches of at most 512 tokens)")
    ap.add_argument("--chain", choices=["on", "off"], default="on",
                    help="programmatic dependent launches between the kernels of a forward (library default: on)")
    ap.add_argument("--gemm-path", type=int, default=0, choices=[0, 1, 2, 3],
                    help="expert-GEMM implementation (cmoe_layer_set_gemm_path); 0 = the library's choice")
    ap.add_argument("--fp8", action="store_true", help="quantise the expert weights to FP8 (cmoe_layer_quantise_fp8) first")
    ap.add_argument("--sweep", choices=["auto", "on", "off"], default="auto",
                    help="add one record per (workload, T) point of the metric to the JSON line "
                         "(auto: on for the default single-GPU headline run)")
    ap.add_argument("--min-region-s", type=float, default=1.0,
                    help="the K-step block is repeated until the timed region is at least this long")
    ap.add_argument("--sweep-region-s", type=float, default=0.4)
    ap.add_argument("--e2e-chunk", type=int, default=0, help="tokens per chunk of the host-buffer call (0: automatic)")
    ap.add_argument("--stage", choices=["forward", "profile", "cluster", "ranks"], default="forward",
                    help="forward: the MoE forward pass (the headline metric); profile: the activation-profiling "
                         "pass; cluster: one round of the GPU clustering pieces")
    ap.add_argument("--forward-only", action="store_true",
                    help="run only the timed forward passes (for profiler captures)")
    args = ap.parse_args()
    world_env = os.environ.get("WORLD_SIZE")
    if args.gpus > 1 and world_env is None:
        # run directly with --gpus N: start one replica process per GPU (the launcher's job otherwise)
        sys.exit(subprocess.call(replica_launch_command(args.gpus, sys.argv[1:], free_port())))
    if world_env is not None and int(world_env) != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}", file=sys.stderr)
        sys.exit(2)
    if args.impl == "reference":
        args.workload = args.workload or HEADLINE[0]
        line = run_reference(args)
    elif args.stage == "ranks":
        line = run_ranks(args)
    else:
        args.warmup = max(args.warmup, 3)
        if args.stage != "forward":
            args.workload = args.workload or "c2_llama2_7b"
        line = (run_profile(args) if args.stage == "profile" else
                run_cluster(args) if args.stage == "cluster" else run_gpu(args))
    if line is not None:
        print(json.dumps(line))


if __name__ == "__main__":
    main()
