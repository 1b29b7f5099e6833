#!/usr/bin/env python
"""Benchmark of the joint compute-memory fusion path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl comfuse|reference]

A step is one pass of the whole hot path over one batch of synthetic input: for the default workload (c3, the largest
of the five configurations: GEMM + bias + GELU + residual + RMSNorm + row max / arg max over 4096-wide rows) that is one
launch of the fused kernel.  `value` is GEMM TFLOP/s over the K timed steps with every input already resident in HBM;
`e2e` repeats the measurement with the step's activations copied from pinned host memory and the result copied back
inside the timed region.  Where the working set of one step fits the L2 cache, the steps rotate over several distinct
buffer sets whose total exceeds L2 (see config.l2).  `per_workload` carries the same kernel-level measurement (time,
roofline fraction, the in-library unfused path) for each of c2, c3, c4 and c5, taken in the same process under the same
clock sampler.  `--impl reference` times the fp64 CPU oracle on host cores instead.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank processes its own batch of rows with
replicated weights -- the path has no exchange step, so there is no collective in the data path -- and `value`
is the sum over ranks divided by the slowest rank's time (weak scaling).
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
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "fused-kernel TFLOP/s (GEMM flops / time of the fused kernel)"
# a1 (target attention), a2 (self-attention 512 x 512) and p1 (an epilogue given as data, on-chip interpreter) lie beyond
# the five named configurations
WORKLOADS = {"c1": 0, "c2": 1, "c3": 2, "c4": 3, "c5": 4, "a1": 5, "p1": 6, "a2": 7, "d1": 8}
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, in bytes, and the ncu
# summary under profiles/ it was read from; None = not captured.
NCU_TRAFFIC = {
    "c1": (None, None),
    "c2": (68_911_872, "profiles/fused_layernorm_c2_bert_ffn_out.md"),
    # two-kernel form: the GEMM kernel with the fused element-wise part (the dominant launch, 87.5 % of the step) moves
    # 227.6 MB in its window, the finish kernel another 77.1 MB
    "c3": (227_593_984, "profiles/fused_rmsnorm_max_c3_complex_subgraph.md"),
    "c4": (512_291_328, "profiles/softmax_rows_c4_scaled_causal_softmax.md"),
    "c5": (8_711_936, "profiles/b2b_mlp_c5.md"),
    "a1": (38_943_488, "profiles/b2b_attention_a1_target_attention.md"),
    "a2": (112_186_112, "profiles/b2b_attention_a2_self_attention_512.md"),
    "d1": (69_688_832, "profiles/b2b_stream_d1_dlrm_bottom_mlp.md"),
    "p1": (18_941_184, "profiles/fused_program_p1_range_normalise.md"),
}
PER_WORKLOAD = ("c2", "c3", "c4", "c5")   # the full-size configurations whose kernels carry a roofline target
BEYOND_CONFIGS = ("a1", "a2", "d1", "p1")  # the shapes beyond the named configurations, measured the same way after them


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz, self.reason_log = [], set(), None, []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                active = [name for bit, name in names.items() if r & bit]
                if active:
                    self.reasons.update(active)
                    self.reason_log.append((len(self.samples) - 1, active))
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def mark(self):
        """Position in the sample list; `since(mark)` summarises what was sampled from there on."""
        return len(self.samples)

    def _summary(self, samples, reasons):
        med = float(np.median(samples)) if samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(reasons), "samples": len(samples)}

    def since(self, n0):
        return self._summary(self.samples[n0:], {name for i, names in self.reason_log if i >= n0 for name in names})

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        return self._summary(self.samples, self.reasons)


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_call(w, rows):
    """One evaluation of the fp64 oracle on `rows` of workload `w` (inputs already widened to fp64)."""
    from oracle import comfuse_oracle as orc
    t = w._f64
    if w.kind == wl.KIND_GEMM_PROGRAM:
        from oracle import fusion_spec_oracle as spo
        pr = w.program
        params = [t[f"p{k}"] if kd == "rowvec" else t[f"p{k}"][rows] for k, kd in enumerate(pr.param_kinds)]
        return spo.gemm_spec(t["A"][rows], t["B"], pr.nodes, pr.terminal, params, pr.row_outputs)
    if w.kind == wl.KIND_B2B_SOFTMAX_ATTENTION:
        return orc.b2b_softmax_attention(t["X"][0][rows], t["W1"][0], t["W2"][0], w.scalars["alpha"])
    if w.kind == wl.KIND_B2B_MLP_RELU:
        return orc.b2b_mlp_relu(t["X"][rows], t["W1"], t["b1"], t["W2"], t["b2"])
    if w.kind == wl.KIND_B2B_MLP_LAYERNORM:
        return orc.b2b_mlp_layernorm(t["X"][rows], t["W1"], t["b1"], t["W2"], t["b2"], t.get("gamma"), t.get("beta"), w.scalars["eps"])
    if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
        return orc.bias_res_layernorm(t["A"][rows], t["B"], t["bias"], t["residual"][rows], t.get("gamma"), t.get("beta"),
                                      w.scalars["alpha"], w.scalars["eps"])
    if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
        return orc.bias_gelu_res_rmsnorm_max(t["A"][rows], t["B"], t["bias"], t["residual"][rows], t["gamma"],
                                             w.scalars["alpha"], w.scalars["eps"])
    mask = orc.causal_mask(w.dims["M"], w.dims["N"], rows=rows) if w.scalars.get("causal") else None
    return orc.scale_mask_softmax(t["A"][0][rows], t["B"][0], w.scalars["alpha"], mask)


def widen_for_oracle(w, softmax_batches=1):
    w._f64 = {}
    for k, v in w.tensors.items():
        if w.kind in (wl.KIND_SCALE_MASK_SOFTMAX, wl.KIND_B2B_SOFTMAX_ATTENTION):
            v = v[:softmax_batches]
        w._f64[k] = wl.bf16_to_f64(v)


def sample_flops(w, nrows):
    d = w.dims
    if w.kind in (wl.KIND_B2B_MLP_LAYERNORM, wl.KIND_B2B_SOFTMAX_ATTENTION, wl.KIND_B2B_MLP_RELU):
        return 2.0 * nrows * (d["K"] * d["N1"] + d["N1"] * d["N2"])
    return 2.0 * nrows * d["N"] * d["K"]


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return int(max(n)) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(w, nrows, steps, warmup):
    rows = np.arange(min(nrows, w.dims["M"]))
    for _ in range(warmup):
        oracle_call(w, rows)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_call(w, rows)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    return dt, sample_flops(w, len(rows))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    w = wl.config(WORKLOADS[name])
    widen_for_oracle(w)
    # size the per-step sample so that steps + warmup stay within a couple of minutes
    probe_rows = 64
    dt, fl = time_oracle(w, probe_rows, 1, 1)
    budget_s = 120.0 / max(args.steps + args.warmup, 1)
    nrows = int(min(w.dims["M"], max(probe_rows, probe_rows * min(budget_s, 2.0) / max(dt, 1e-6))))
    nrows = max(64, (nrows // 64) * 64)
    dt, fl = time_oracle(w, nrows, args.steps, args.warmup)
    tflops = fl / dt / 1e12
    cores = blas_threads()
    sample = f"rows 0..{nrows - 1} of {w.name} per step, fp64 numpy oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": w.name, **w.dims, "sample_rows_per_step": nrows},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ multi-process helpers
def max_over_ranks(ms: float, device=None) -> float:
    """The slowest rank's time (every rank gets it).  Works on any initialised process group (nccl or gloo)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Weak scaling: every rank processes `units_per_rank` per step; the job's rate is all ranks' units over the
    slowest rank's time."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------------------ CUDA arm
WARM_MS = 12.0   # the step graph is replayed untimed for about this long right in front of the timed region


def measure(name, args, env, full):
    """Kernel-level measurement of one workload (and, with `full`, the end-to-end, eager and CPU legs).  Returns the JSON
    fields of that workload.  `env` = (torch, dist, cf, dev, world, rank, peaks, sampler)."""
    torch, dist, cf, dev, world, rank, peaks, sampler = env
    w = wl.config(WORKLOADS[name])
    fused = not args.unfused

    def to_dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)

    # ---- buffer sets: per-step activations (inputs read once per step and the outputs) are replicated until the
    # rotation exceeds 3x the L2 capacity; weights and row vectors are shared (they are meant to be L2 resident)
    attention = w.kind == wl.KIND_B2B_SOFTMAX_ATTENTION
    relu_mlp = w.kind == wl.KIND_B2B_MLP_RELU
    b2b = w.kind in (wl.KIND_B2B_MLP_LAYERNORM, wl.KIND_B2B_SOFTMAX_ATTENTION, wl.KIND_B2B_MLP_RELU)
    program = w.kind == wl.KIND_GEMM_PROGRAM
    if program:
        spec = cf.make_spec(w.program.nodes, w.program.terminal, len(w.program.param_kinds), w.program.row_outputs)
        pshape = cf.make_gemm_shape(1, w.dims["M"], w.dims["N"], w.dims["K"])
        plan = cf.spec_plan(spec, pshape)
        # the fused path of a program: the kernel generated for it (compiled at run time, ahead of the timed region and of
        # any graph capture), else the on-chip interpreter of the same lowering
        generated = (args.program_path == "generated" and plan.program_path == cf.SPEC_PATH_FUSED_PROGRAM
                     and plan.path != cf.SPEC_PATH_FUSED_KERNEL and cf.program_compiler_status()[0] == cf.OK)
        if generated:
            cf.gemm_spec_prepare(spec, pshape, cf.GENERATED)
        interpreted = 2 if plan.path == cf.SPEC_PATH_FUSED_PROGRAM else 1
        pmode = lambda use_fused: (cf.GENERATED if generated else interpreted) if use_fused else 0
    act_names = {"A", "B"} if w.kind == wl.KIND_SCALE_MASK_SOFTMAX else ({"X", "W1", "W2"} if attention else {"A", "residual", "X"})
    base = {k: to_dev(v) for k, v in w.tensors.items()}
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    d = w.dims
    out_shape = (d["batch"], d["M"], d.get("N", d.get("N2"))) if "batch" in d else (d["M"], d.get("N", d.get("N2")))
    per_set = sum(base[k].numel() * 2 for k in base if k in act_names) + int(np.prod(out_shape)) * 2
    nsets = int(max(2, min(16, -(-3 * l2_bytes // per_set))))
    sets = []
    for i in range(nsets):
        s = {k: (v.clone() if (k in act_names and i > 0) else v) for k, v in base.items()}
        s["Y"] = torch.zeros(out_shape, dtype=torch.bfloat16, device=dev)
        if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
            s["row_max"] = torch.zeros(out_shape[:-1], dtype=torch.float32, device=dev)
            s["row_argmax"] = torch.zeros(out_shape[:-1], dtype=torch.int32, device=dev)
        if program:
            s["row_out"] = [torch.zeros(d["M"], dtype=torch.int32 if w.program.nodes[r][0] == "argmax" else torch.float32, device=dev)
                            for r in w.program.row_outputs]
        sets.append(s)

    # workspace (unfused path only)
    def b2b_desc(use_fused):
        if attention:
            return cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], 0.0, use_fused, cf.B2B_SOFTMAX_ATTENTION, d["batch"], w.scalars["alpha"])
        if relu_mlp:
            return cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], 0.0, use_fused, cf.B2B_MLP_RELU)
        return cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], w.scalars["eps"], use_fused)

    if b2b:
        ws_bytes = cf.b2b_workspace_size(b2b_desc(fused))
    elif program:
        ws_bytes = cf.gemm_spec_workspace_size(spec, pshape, pmode(fused))
    else:
        kind = {wl.KIND_BIAS_RES_LAYERNORM: cf.EPI_BIAS_RES_LAYERNORM,
                wl.KIND_BIAS_GELU_RES_RMSNORM_MAX: cf.EPI_BIAS_GELU_RES_RMSNORM_MAX,
                wl.KIND_SCALE_MASK_SOFTMAX: cf.EPI_SCALE_MASK_SOFTMAX}[w.kind]
        mask = cf.MASK_CAUSAL if w.scalars.get("causal") else cf.MASK_NONE
        desc = cf.make_gemm_desc(base["A"], base["B"], sets[0]["Y"], kind, residual=base.get("residual"), mask=mask, fused=fused)
        ws_bytes = cf.workspace_size(desc)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)

    def step(s, use_fused=fused, workspace=ws):
        if program:
            cf.gemm_spec(s["A"], s["B"], s["Y"], spec, params=[s[f"p{k}"] for k in range(len(w.program.param_kinds))],
                         row_out=s["row_out"], fused=pmode(use_fused), workspace=workspace)
        elif attention:
            cf.b2b_attention(s["X"], s["W1"], s["W2"], s["Y"], alpha=w.scalars["alpha"], fused=use_fused, workspace=workspace)
        elif relu_mlp:
            cf.b2b_mlp_relu(s["X"], s["W1"], s["b1"], s["W2"], s["b2"], s["Y"], fused=use_fused, workspace=workspace)
        elif w.kind == wl.KIND_B2B_MLP_LAYERNORM:
            cf.b2b_gemm(s["X"], s["W1"], s["b1"], s["W2"], s["b2"], s["Y"], gamma=s.get("gamma"), beta=s.get("beta"),
                        eps=w.scalars["eps"], fused=use_fused, workspace=workspace)
        elif w.kind == wl.KIND_BIAS_RES_LAYERNORM:
            cf.gemm_epilogue(s["A"], s["B"], s["Y"], cf.EPI_BIAS_RES_LAYERNORM, bias=s.get("bias"), residual=s.get("residual"),
                             gamma=s.get("gamma"), beta=s.get("beta"), alpha=w.scalars["alpha"], eps=w.scalars["eps"],
                             fused=use_fused, workspace=workspace)
        elif w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
            cf.gemm_epilogue(s["A"], s["B"], s["Y"], cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, bias=s.get("bias"),
                             residual=s.get("residual"), gamma=s.get("gamma"), alpha=w.scalars["alpha"], eps=w.scalars["eps"],
                             row_max=s["row_max"], row_argmax=s["row_argmax"], fused=use_fused, workspace=workspace)
        else:
            cf.gemm_epilogue(s["A"], s["B"], s["Y"], cf.EPI_SCALE_MASK_SOFTMAX, alpha=w.scalars["alpha"],
                             mask=cf.MASK_CAUSAL if w.scalars.get("causal") else cf.MASK_NONE, fused=use_fused,
                             workspace=workspace)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(nsteps, fn):
        """K direct launches bracketed by barrier + synchronize; device time from CUDA events on the launching stream."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda._sleep(400_000)  # the host enqueues the launches while this busy-wait kernel runs
        e0.record()
        for i in range(nsteps):
            fn(i)
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dev)

    # ---- warm-up, then the timed region.  The K steps are replayed from a CUDA graph that holds one launch per
    # buffer set (the paper's protocol, Sec. 6 Setup: capture and replay to take host launch cost out of the device
    # time); steps that do not fill a whole graph are replayed from a second, shorter graph.
    for i in range(max(args.warmup, 3)):
        step(sets[i % nsets])
    torch.cuda.synchronize()
    graph = rest_graph = None
    graph_launches = 0
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        c0 = cf.launch_count()
        with torch.cuda.graph(graph):
            for s in sets:
                step(s)
        graph_launches = cf.launch_count() - c0
        graph.replay()
        if args.steps % nsets:
            rest_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(rest_graph):
                for s in sets[:args.steps % nsets]:
                    step(s)
            rest_graph.replay()
        torch.cuda.synchronize()

    def run_steps(n):
        full_graphs, rest = (n // nsets, n % nsets) if graph is not None else (0, n)
        for _ in range(full_graphs):
            graph.replay()
        if rest and rest_graph is not None:
            rest_graph.replay()
        else:
            for i in range(rest):
                step(sets[i % nsets])

    # a first estimate of the step time sizes the untimed run-in
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    run_steps(nsets)
    e1.record()
    torch.cuda.synchronize()
    est_ms = max(e0.elapsed_time(e1) / nsets, 1e-3)
    warm_replays = int(max(2, min(400, WARM_MS / (est_ms * nsets)))) if graph is not None else 0

    # ---- the timed region: exactly K steps between two events.  Right in front of it, on the same stream and without a
    # gap, the same graph is replayed untimed for about WARM_MS: clocks, caches and the launch pipeline are in their steady
    # state when the first timed step starts (without the run-in, 20 timed steps read 4-5 % slower than 200), and the clock
    # sampler, which polls once per millisecond over run-in and timed region, sees the load the timed steps run under.
    # A busy-wait kernel in front of everything lets the host enqueue the whole sequence before the device starts on it.
    launches0 = cf.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    mark = sampler.mark()
    torch.cuda._sleep(2_000_000)
    for _ in range(warm_replays):
        graph.replay()
    e0.record()
    run_steps(args.steps)
    e1.record()
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dev)
    clocks = sampler.since(mark)
    launches = cf.launch_count() - launches0
    if graph is not None:   # replayed launches do not pass through the library's host code: count them from the graph
        launches += (args.steps // nsets) * graph_launches
        if rest_graph is not None:
            launches += (args.steps % nsets) * (graph_launches // nsets)
    status = cf.last_device_status()
    if status != cf.OK:
        raise SystemExit(f"device status {status} after the timed region of {name}")
    ms_step = ms_total / args.steps
    flops = w.gemm_flops()
    bytes_min = w.min_hbm_bytes()
    value = whole_job_value(flops, world, ms_step) / 1e12

    # ---- roofline of the dominant kernel (the fused kernel; one launch per step)
    t_tensor = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = bytes_min / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        roof = {"bound": "tensor", "achieved": flops / (ms_step * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": bytes_min / (ms_step * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"], roof["traffic_source"] = NCU_TRAFFIC.get(name, (None, None))
    roof["peak_source"] = f"of {peaks['source']} (burst figure, kernel timed alone)"
    if program:
        roof["kernel"] = {cf.SPEC_PATH_FUSED_KERNEL: "fused_pair_kernel (compiled kind)", cf.SPEC_PATH_FUSED_PROGRAM: "fused_pair_kernel<EPI_PROGRAM> (generated for the program)" if generated else "fused_pair_kernel<EPI_PROGRAM> (on-chip interpreter)",
                          cf.SPEC_PATH_ROW_PROGRAM: "fused_pair_kernel<EPI_NONE> + row_program_kernel"}[plan.path if fused else cf.SPEC_PATH_ROW_PROGRAM]
    elif b2b:
        roof["kernel"] = "b2b_stream_kernel" if relu_mlp else ("b2b_pair_kernel" if attention else "b2b_mlp_kernel")
    elif w.kind == wl.KIND_SCALE_MASK_SOFTMAX and d["K"] <= 256:
        roof["kernel"] = "softmax_rows_kernel"      # short K: score chunks computed twice, no cluster exchange
    elif fused and ws_bytes > 0:
        # rows behind a long contraction: element-wise part fused into 256-column tiles on all SMs, the row leaves the chip
        # once as fp16, a second kernel normalises; `achieved` divides by the whole step (both launches)
        roof["kernel"] = "fused_pair_kernel (256-column tiles, fp16 row out) + wide_row_finish_kernel"
        roof["traffic_finish_kernel"] = 77_068_032 if name == "c3" else None
    else:
        roof["kernel"] = "fused_pair_kernel"
    roof["algorithmic_flops_per_launch"] = flops
    roof["algorithmic_bytes_per_launch"] = bytes_min
    roof["roofline_us"] = max(t_tensor, t_hbm) * 1e6
    # the same fraction against the nominal figures (2250 TFLOP/s dense bf16, 8 TB/s), for context
    nominal = 2250.0 if roof["bound"] == "tensor" else 8000.0
    roof["frac_of_nominal"] = roof["achieved"] / nominal
    roof["nominal_peak"] = nominal
    if w.kind == wl.KIND_SCALE_MASK_SOFTMAX and w.scalars.get("causal"):
        # GEMM flops of the 128 x 128 score tiles the causal mask leaves (value counts all tiles, as a dense GEMM would)
        t = -(-d["M"] // 128)
        roof["flops_causal_tiles_only"] = flops * (t * (t + 1) / 2) / (t * t)

    config = {"workload": w.name, **w.dims, "path": "fused" if fused else "unfused",
              "launch": "direct" if graph is None else f"CUDA graph replay, {nsets} steps per graph; {warm_replays} untimed replays run in front of the timed steps",
              "parallelism": f"replicas x{world}, rows sharded, no collective",
              "l2": f"rotating {nsets} buffer sets of {per_set / 1e6:.1f} MB activations+outputs "
                    f"({nsets * per_set / 1e6:.0f} MB > L2 {l2_bytes / 1e6:.0f} MB), weights shared"}
    res = {"value": value, "ms_per_step": ms_step, "config": config, "roofline": roof, "gpu_launches": int(launches), "clocks": clocks}
    if args.kernel_only:
        return res

    extra = {}
    # ---- the paper reports mean and minimum over its timed replays (Sec. 6 Setup): the minimum over eight single replays
    # of the step graph, each between its own pair of events, all enqueued behind one busy-wait kernel and a run-in
    if graph is not None and world == 1:
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(9)]
        torch.cuda._sleep(1_000_000)
        for _ in range(max(2, warm_replays // 4)):
            graph.replay()
        evs[0].record()
        for k in range(8):
            graph.replay()
            evs[k + 1].record()
        torch.cuda.synchronize()
        extra["min_ms_per_step"] = min(evs[k].elapsed_time(evs[k + 1]) for k in range(8)) / nsets
        extra["min_over"] = f"8 consecutive graph replays ({nsets} steps each), each between its own events"
    # ---- the in-library unfused path on the same buffers (context: speedup of fusion)
    try:
        other = not fused
        if b2b:
            ob = cf.b2b_workspace_size(b2b_desc(other))
        elif program:
            ob = cf.gemm_spec_workspace_size(spec, pshape, pmode(other))
        else:
            desc.fused = int(other)
            ob = cf.workspace_size(desc)
        ws2 = torch.empty(max(ob, 16), dtype=torch.uint8, device=dev)
        for i in range(3):
            step(sets[i % nsets], other, ws2)
        n2 = max(3, min(args.steps, 50))
        ms_other = timed(n2, lambda i: step(sets[i % nsets], other, ws2)) / n2
        key = "unfused_ms_per_step" if fused else "fused_ms_per_step"
        extra[key] = ms_other
        extra["speedup_vs_unfused"] = (ms_other / ms_step) if fused else (ms_step / ms_other)
        del ws2
    except cf.ComfuseError as e:
        extra["unfused_error"] = str(e)
    if program and fused and generated:
        # context: the same lowering run as data by the on-chip interpreter (what the generated kernel replaces)
        def interp(i):
            s = sets[i % nsets]
            cf.gemm_spec(s["A"], s["B"], s["Y"], spec, params=[s[f"p{k}"] for k in range(len(w.program.param_kinds))],
                         row_out=s["row_out"], fused=2, workspace=ws)
        for i in range(3):
            interp(i)
        n2 = max(3, min(args.steps, 50))
        extra["interpreter_ms_per_step"] = timed(n2, interp) / n2
    res.update(extra)
    if not full:
        return res

    extra = {}
    # ---- context: the same step with its inputs and outputs resident in L2 (one buffer set, back to back), and the
    # GEMM(s) alone through the vendor library, so that "residual" = what the subgraph costs on top of the GEMM
    # (Sec. 6.1 reports fusion benefit this way: residual time)
    n3 = max(3, min(args.steps, 50))
    for i in range(3):
        step(sets[0])
    extra["warm_l2_ms_per_step"] = timed(n3, lambda i: step(sets[0])) / n3

    def gemm_only(sx):
        if b2b:
            return torch.matmul(torch.matmul(sx["X"], sx["W1"]), sx["W2"])
        return torch.matmul(sx["A"], sx["B"])
    for i in range(3):
        gemm_only(sets[i % nsets])
    ms_gemm = timed(n3, lambda i: gemm_only(sets[i % nsets])) / n3
    extra["gemm_only_ms_per_step"] = ms_gemm
    extra["gemm_only_impl"] = "torch.matmul (vendor library), bf16 output"
    # ---- context: the same subgraph as framework library calls on the same buffers (vendor GEMM, vendor / framework
    # element-wise, normalisation, softmax and attention kernels), each op its own launch(es)
    import torch.nn.functional as F

    def eager(sx):
        if program:
            return None
        if attention:   # keys in the layout the library call wants ([S, d], made once, outside the timed region)
            if "K_rows" not in sx:
                sx["K_rows"] = sx["W1"].transpose(1, 2).contiguous()
            return F.scaled_dot_product_attention(sx["X"].unsqueeze(0), sx["K_rows"].unsqueeze(0), sx["W2"].unsqueeze(0), scale=w.scalars["alpha"])
        if relu_mlp:
            return torch.relu(torch.addmm(sx["b2"], torch.relu(torch.addmm(sx["b1"], sx["X"], sx["W1"])), sx["W2"]))
        if w.kind == wl.KIND_B2B_MLP_LAYERNORM:
            hid = F.gelu(torch.addmm(sx["b1"], sx["X"], sx["W1"]), approximate="tanh")
            return F.layer_norm(torch.addmm(sx["b2"], hid, sx["W2"]) + sx["X"], (d["N2"],), sx.get("gamma"), sx.get("beta"), w.scalars["eps"])
        if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
            return F.layer_norm(torch.addmm(sx["bias"], sx["A"], sx["B"]) + sx["residual"], (d["N"],), sx.get("gamma"), sx.get("beta"), w.scalars["eps"])
        if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
            y = F.rms_norm(F.gelu(torch.addmm(sx["bias"], sx["A"], sx["B"]), approximate="tanh") + sx["residual"], (d["N"],), sx["gamma"], w.scalars["eps"])
            return y.max(dim=-1)
        t = torch.bmm(sx["A"], sx["B"]) * w.scalars["alpha"]
        if w.scalars.get("causal"):
            t = t.masked_fill(causal_mask, float("-inf"))
        return torch.softmax(t, dim=-1)
    if not program:
        causal_mask = torch.ones(d["M"], d.get("N", 1), dtype=torch.bool, device=dev).triu(1) if w.scalars.get("causal") else None
        try:
            for i in range(max(3, nsets)):
                eager(sets[i % nsets])
            extra["torch_eager_ms_per_step"] = timed(n3, lambda i: eager(sets[i % nsets])) / n3
            extra["torch_eager_impl"] = ("F.scaled_dot_product_attention" if attention else
                                         "torch.addmm / bmm + framework element-wise, normalisation and softmax kernels") + ", bf16"
        except Exception as ex:  # an op missing from this torch build is no reason to lose the bench line
            extra["torch_eager_error"] = repr(ex)[:200]
    fused_ms = ms_step if fused else res.get("fused_ms_per_step")
    unfused_ms = res.get("unfused_ms_per_step") if fused else ms_step
    extra["residual_ms"] = {"fused": None if fused_ms is None else fused_ms - ms_gemm,
                            "unfused": None if unfused_ms is None else unfused_ms - ms_gemm}

    # ---- end to end: activations from pinned host memory, result back to pinned host memory, every step.
    # One call of the library's host-buffer entry point per step: it copies the step's activations from pinned host
    # memory into a device staging buffer, runs the same kernels, and copies the result back to pinned host memory.
    host_in = {k: torch.from_numpy(np.ascontiguousarray(w.tensors[k]).view(np.int16)).view(torch.bfloat16).pin_memory()
               for k in w.tensors if k in act_names}
    host_out = torch.empty(out_shape, dtype=torch.bfloat16).pin_memory()
    h2d = sum(t.numel() * 2 for t in host_in.values())
    d2h = host_out.numel() * 2
    s0 = sets[0]
    if program:
        # no host-buffer form of the program entry point: the step's activations are copied from pinned memory with
        # stream copies around the same call, all inside the timed region
        dA = torch.empty_like(s0["A"])

        def e2e_step(i):
            dA.copy_(host_in["A"], non_blocking=True)
            cf.gemm_spec(dA, s0["B"], s0["Y"], spec, params=[s0[f"p{k}"] for k in range(len(w.program.param_kinds))],
                         row_out=s0["row_out"], fused=pmode(fused), workspace=ws)
            host_out.copy_(s0["Y"], non_blocking=True)
    elif b2b:
        bdesc = b2b_desc(fused)
        staging = torch.empty(cf.b2b_host_staging_size(bdesc), dtype=torch.uint8, device=dev)

        def e2e_step(i):
            if attention:
                cf.b2b_attention_host(host_in["X"], host_in["W1"], host_in["W2"], host_out, staging=staging,
                                      alpha=w.scalars["alpha"], fused=fused, workspace=ws)
            elif relu_mlp:
                cf.b2b_mlp_relu_host(host_in["X"], s0["W1"], s0["b1"], s0["W2"], s0["b2"], host_out, staging=staging, fused=fused,
                                     workspace=ws)
            else:
                cf.b2b_gemm_host(host_in["X"], s0["W1"], s0["b1"], s0["W2"], s0["b2"], host_out, staging=staging,
                                 gamma=s0.get("gamma"), beta=s0.get("beta"), eps=w.scalars["eps"], fused=fused, workspace=ws)
    else:
        hmask = cf.HOST_A | cf.HOST_Y | (cf.HOST_B if "B" in host_in else 0) | (cf.HOST_RESIDUAL if "residual" in host_in else 0)
        hB = host_in.get("B", s0["B"])
        desc.fused = int(fused)
        hdesc = cf.make_gemm_desc(host_in["A"], hB, host_out, kind, residual=host_in.get("residual"), mask=mask, fused=fused)
        staging = torch.empty(cf.host_staging_size(hdesc, hmask), dtype=torch.uint8, device=dev)
        ekw = dict(alpha=w.scalars["alpha"], mask=mask, fused=fused, workspace=ws, staging=staging, host_mask=hmask)
        if w.kind != wl.KIND_SCALE_MASK_SOFTMAX:
            ekw.update(bias=s0.get("bias"), residual=host_in.get("residual"), gamma=s0.get("gamma"), eps=w.scalars["eps"])
        if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
            ekw.update(beta=s0.get("beta"))
        if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
            ekw.update(row_max=s0["row_max"], row_argmax=s0["row_argmax"])

        def e2e_step(i):
            cf.gemm_epilogue_host(host_in["A"], hB, host_out, kind, **ekw)

    n_e2e = max(3, min(args.steps, 20))
    for i in range(2):
        e2e_step(i)
    ms_e2e = timed(n_e2e, e2e_step) / n_e2e
    extra["e2e"] = {"value": whole_job_value(flops, world, ms_e2e) / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": n_e2e,
                    "call": "comfuse_gemm_spec between stream copies from / to pinned memory" if program
                            else ("comfuse_b2b_gemm_host" if b2b else "comfuse_gemm_epilogue_host")}

    # ---- CPU baseline: the oracle as it stands, on rank 0 at N = 1 only, on a bounded sample
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        widen_for_oracle(w)
        dt, fl = time_oracle(w, 64, 1, 1)
        nrows = int(min(w.dims["M"], max(64, 64 * 10.0 / max(dt, 1e-6))))   # aim at ~10 s of CPU work
        nrows = max(64, (nrows // 64) * 64)
        dt, fl = time_oracle(w, nrows, 1, 0)
        if dt < 5.0 and nrows < w.dims["M"]:   # the 64-row probe underrates BLAS on large blocks: size once more from this pass
            nrows = int(min(w.dims["M"], nrows * 10.0 / max(dt, 1e-6)))
            nrows = max(64, (nrows // 64) * 64)
            dt, fl = time_oracle(w, nrows, 1, 0)
        cpu = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle",
               "sample": f"rows 0..{nrows - 1} of {w.name}, one pass of the fp64 numpy oracle (BLAS threads), {dt:.2f} s", "seconds": dt}
    extra["cpu_baseline"] = cpu
    res.update(extra)
    return res


def run_comfuse(args):
    import torch
    import torch.distributed as dist
    import paper_2608_03537_b200 as cf

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    cf.lib()  # fail loudly if the CUDA library is missing
    peaks = load_peaks()
    sampler = ClockSampler(local)
    sampler.start()
    env = (torch, dist, cf, dev, world, rank, peaks, sampler)

    head = measure(args.workload, args, env, full=not args.kernel_only)
    per = []
    if world == 1 and not args.kernel_only and not args.no_per_workload:
        # the kernel-level figures of every full-size configuration, in this process, under the same clock sampler
        for name in PER_WORKLOAD + (() if args.no_beyond_configs else BEYOND_CONFIGS):
            if name == args.workload:
                r = head
            else:
                torch.cuda.empty_cache()
                r = measure(name, args, env, full=False)
            per.append({"workload": name, "ms_per_step": r["ms_per_step"], "value": r["value"], "unit": "TFLOP/s",
                        "roofline": r["roofline"], "min_ms_per_step": r.get("min_ms_per_step"),
                        "unfused_ms_per_step": r.get("unfused_ms_per_step"), "speedup_vs_unfused": r.get("speedup_vs_unfused"),
                        "gpu_launches": r["gpu_launches"], "clocks": r["clocks"], "named_config": name in PER_WORKLOAD})
            if "interpreter_ms_per_step" in r:
                per[-1]["interpreter_ms_per_step"] = r["interpreter_ms_per_step"]
    all_clocks = sampler.stop()

    if rank == 0:
        line = {"metric": METRIC, "value": head.pop("value"), "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": head.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
        if args.kernel_only:
            line["kernel_only"] = True
        line.update(head)
        if per:
            line["per_workload"] = per
            line["clocks_whole_run"] = all_clocks
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="comfuse", choices=["comfuse", "reference"])
    ap.add_argument("--unfused", action="store_true", help="time the in-library unfused path as the main number")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--kernel-only", action="store_true", help="skip the unfused, end-to-end and CPU legs (for profiler runs)")
    ap.add_argument("--program-path", default="generated", choices=["generated", "interpreter"],
                    help="workload p1: the kernel generated for the program (default where the run-time compiler is there) or the on-chip interpreter")
    ap.add_argument("--no-beyond-configs", action="store_true", help="per_workload: c2-c5 only, not a1, a2, d1, p1")
    ap.add_argument("--no-per-workload", action="store_true", help="only the headline workload, not the c2-c5 list")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_comfuse(args)


if __name__ == "__main__":
    main()
