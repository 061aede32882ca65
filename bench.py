#!/usr/bin/env python
"""Benchmark of the CASCADE tree-verification step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload lumina+janus|janus|lumina|mini]
                    [--mode layer|pieces|loop|sweep] [--impl ours|reference]

One "step" is one pass of the whole verification hot path over one synthetic batch: the tree tokens go
through one decoder layer (embedding, q/k/v, rotary, tree attention over the prefix cache, output
projection, SwiGLU MLP), the final norm, the LM head with guidance, relaxed acceptance and path selection
(`--mode pieces` runs the four named pieces on stand-alone inputs without the layer's projections).  Prints ONE JSON
line: verify-steps/s (device-timed with CUDA events, inputs resident in HBM), the same through the
host-buffer C-ABI entry (`e2e`), the roofline of the dominant kernel measured live with CUDA events, the
CPU checker timed on the host cores (`cpu_baseline`), and the SM clocks seen under load.

The default run measures both model shapes: the headline keys are the Lumina-mGPT-7B-768-shaped step (the
largest single-GPU verification step), and the Janus-Pro-7B-shaped step is reported in the same line under
"janus" with its own value / ms_per_step / roofline / e2e / cpu_baseline.  The K-step timed region is run
`--repeats` times and the median is reported with the spread.

With N > 1 every rank runs an independent replica on its own GPU (the step has no exchange between
prompts, so there is nothing to shard or reduce); the time is the max over ranks.
`--impl reference` times the CPU checker alone (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
# (step_kernels_layer_*_full.txt: default step, one launch of each kernel), and the first 16 hex digits of
# the SHA-256 of the kernel sources (the .cu file, ptx.cuh, operand.cuh) they were taken on.  A kernel whose source has changed since reports
# "traffic": null.
NCU_TRAFFIC = {
    "janus": {"gemm_qkv": 108145664, "tree_attn": 15632384, "gemm_o": 35681792, "gemm_gate_up": 190507264, "gemm_down": 100555520, "gemm_head": 139249664},
    "lumina": {"gemm_qkv": 107926272, "tree_attn": 86904320, "gemm_o": 35683072, "gemm_gate_up": 190346752, "gemm_down": 100851456, "gemm_head": 544933632},
}
NCU_TRAFFIC_SOURCES = {"gemm_tc.cu": "3bbc44bff5fc1692", "attn_bf16.cu": "729009871e987da3"}

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "tree_verify_steps_per_s"
UNIT = "steps/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(x: float, device=None) -> float:
    """The slowest rank's time: N replicas have finished a step when the last of them has."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(steps_per_rank: int, world: int, seconds: float) -> float:
    """Steps per second of the whole job: every rank ran `steps_per_rank` steps of its own replica."""
    return world * steps_per_rank / seconds


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed regions run."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
        self.period = period_s

    def _run(self):
        nv = self.nv
        names = {
            nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_step(w, parent, host, mode):
    """One whole verification step on the CPU checker (same inputs as the device step)."""
    from oracle import cascade_oracle as O
    scale = 1.0 / np.sqrt(w.head_dim)
    if mode == "layer":
        out = O.verify_step(host["embed"], host["layers"], host["gamma_final"], host["w_head"], host["tok"], parent,
                            host["k_prefix"], host["v_prefix"], host["prefix_len"], host["draft_p"], host["uniforms"],
                            w.n_heads, w.head_dim, w.eps, w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq,
                            w.tvd_budget, kv_bf16=w.dtype == "bf16")
        return out["accept"]
    O.tree_attention(host["q"], host["k_prefix"], host["v_prefix"], host["prefix_len"], host["k_tree"],
                     host["v_tree"], parent, scale)
    head, res = O.verify_tail(host["hidden"], host["gamma_final"], w.eps, host["w_head"], w.cfg_scale, 1.0,
                              host["tok"], parent, host["draft_p"], host["uniforms"], w.tau_pos, w.tau_seq,
                              w.tvd_budget)
    return res


def time_oracle(w, parent, host, mode, budget_s=25.0, max_steps=3):
    t0 = time.perf_counter()
    n = 0
    while n < max_steps and (n == 0 or (time.perf_counter() - t0) * (n + 1) / n < budget_s):
        oracle_step(w, parent, host, mode)
        n += 1
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return n / dt, n, cores


def host_inputs(w, mode):
    from paper_2605_07230_b200 import synth
    parent = w.parent()
    rng = np.random.default_rng(w.seed)
    if mode == "layer":
        return parent, synth.layer_step_inputs(w, rng, parent, 1)
    host = {}
    host.update(synth.attention_inputs(w, rng, len(parent)))
    host.update(synth.tail_inputs(w, rng, parent))
    return parent, host


def run_reference(args, w):
    """The CPU checker as the reference arm: a bounded number of whole steps on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    parent, host = host_inputs(w, args.mode)
    for _ in range(min(args.warmup, 1)):
        oracle_step(w, parent, host, args.mode)
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(w, parent, host, args.mode)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    v = steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * dt / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "tree_rows": len(parent), "prefix_len": w.prefix_len, "V": w.V,
                   "h": w.h, "mode": args.mode, "note": "CPU checker (numpy fp64), whole step; steps capped at 3"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{steps} whole step(s) of the {w.name} workload"},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def oracle_cores():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count()


def source_digest(src):
    """First 16 hex digits of the SHA-256 of a kernel's sources (its .cu file and the headers its device code uses)."""
    csrc = os.path.join(ROOT, "paper_2605_07230_b200", "csrc")
    digest = hashlib.sha256()
    for name in (src, "ptx.cuh", "operand.cuh"):
        with open(os.path.join(csrc, name), "rb") as f:
            digest.update(f.read())
    return digest.hexdigest()[:16]


def kernel_rooflines(w, T, timing, n_timed_steps, peaks, mode, traffic_key):
    """Per streaming kernel: algorithmic bytes (its weight matrix or K/V once + operands) / event-timed launch
    duration against the measured copy bandwidth; for the GEMMs also the algorithmic tensor rate."""
    hd = w.n_heads * w.head_dim
    e = 2 if w.dtype == "bf16" else 4
    R = 2 * w.B
    act = R * T * e
    alg_b = {
        "tree_attn": R * (w.prefix_len + T) * hd * 2 * e + 2 * R * T * hd * e,
        "gemm_head": w.V * w.h * e + R * T * w.h * e,
        "gemm_qkv": 3 * hd * w.h * e + act * w.h,
        "gemm_o": w.h * hd * e + act * hd,
        "gemm_gate_up": 2 * w.ffn * w.h * e + act * w.h,
        "gemm_down": w.h * w.ffn * e + act * w.ffn,
    }
    # algorithmic flops: the head's guidance mix is taken before the product (half of two heads); the layer
    # projections work on both rows of every prompt
    M2 = R * T
    alg_f = {"gemm_head": 2.0 * w.B * T * w.h * w.V, "gemm_qkv": 2.0 * M2 * w.h * 3 * hd, "gemm_o": 2.0 * M2 * hd * w.h,
             "gemm_gate_up": 2.0 * M2 * w.h * 2 * w.ffn, "gemm_down": 2.0 * M2 * w.ffn * w.h}
    per_kernel = {k: {"us": 1e3 * v[0] / v[1], "launches_per_step": v[1] / n_timed_steps} for k, v in timing.items()}

    def traffic(k):
        # dram bytes per launch from the ncu capture summarised under profiles/: only for the step they were taken
        # on (layer mode) and only while the kernel's source is what it was then
        if mode != "layer" or k not in NCU_TRAFFIC.get(traffic_key, {}):
            return None
        src = "attn_bf16.cu" if k == "tree_attn" else "gemm_tc.cu"
        if source_digest(src) != NCU_TRAFFIC_SOURCES[src]:
            return None
        return NCU_TRAFFIC[traffic_key][k]

    def roof(k):
        us = per_kernel[k]["us"]
        ach = alg_b[k] / (us * 1e-6) / 1e9
        d = {"kernel": k, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
             "frac": ach / peaks["hbm_gbs"], "traffic": traffic(k), "peak_source": peaks["source"], "us_per_launch": us,
             "algorithmic_bytes": alg_b[k]}
        if k in alg_f:
            d["tensor_tflops"] = alg_f[k] / (us * 1e-6) / 1e12
            d["tensor_frac_of_bf16_peak"] = d["tensor_tflops"] / peaks["bf16_tflops"]
            d["tensor_frac_of_bf16_sustained"] = d["tensor_tflops"] / peaks["bf16_tflops_sustained"]
            # the operand is a bf16 pair (value + remainder): twice the algorithmic tensor work is executed
            d["executed_tflops"] = 2 * d["tensor_tflops"]
            if alg_f[k] / (peaks["bf16_tflops"] * 1e12) > alg_b[k] / (peaks["hbm_gbs"] * 1e9):
                # more rows than the ridge: the tensor cores bound this launch, not the weight stream
                d.update({"bound": "tensor", "achieved": d["tensor_tflops"], "peak": peaks["bf16_tflops"],
                          "unit": "TFLOP/s", "frac": d["tensor_frac_of_bf16_peak"],
                          "hbm_gbs": ach, "hbm_frac": ach / peaks["hbm_gbs"]})
        return d

    roofs = {k: roof(k) for k in per_kernel if k in alg_b}
    step_bytes = sum(alg_b[k] for k in roofs)
    return per_kernel, roofs, step_bytes


def measure_step(name, args, dev, peaks, world, local, over=None, light=False):
    """Everything measured for one workload: device-timed steps/s (median of `--repeats` runs of exactly K steps),
    per-kernel event times and rooflines, the host-buffer entry end to end, the truncation kernel, the checker.
    `light`: only the device-timed rate and the kernel times (sweep cells)."""
    import torch
    import torch.distributed as dist
    from paper_2605_07230_b200 import binding as cb
    from paper_2605_07230_b200 import synth
    from paper_2605_07230_b200.workload import LayerWorkload, PiecesWorkload

    over = dict(over or {})
    host_given = over.pop("_host", None)
    w = synth.workload(name, **over)
    parent = w.parent()
    T = len(parent)
    hd = w.n_heads * w.head_dim
    # enough rotating copies of the inputs that a step never finds its operands in the 126 MB L2
    layer_bytes = (4 * hd * w.h + 3 * w.ffn * w.h) * 2 if args.mode != "pieces" else 0
    per_set = (w.V * w.h + 2 * 2 * w.B * (w.prefix_len + T) * hd) * 2 + layer_bytes
    n_sets = args.sets or max(2, int(np.ceil(3 * 126e6 / per_set)))
    if args.mode != "pieces":
        wl = LayerWorkload(w, n_layers=1, device=dev, n_sets=n_sets, want_hidden=False, keep_logits=args.truncate,
                           host=host_given)
    else:
        wl = PiecesWorkload(w, device=dev, n_sets=n_sets, keep_logits=args.truncate)
    if args.truncate:
        for st_ in wl.sets:
            st_.step.top_k = args.top_k
    K, W = max(args.steps, 1), max(args.warmup, 3)
    reps = max(1, args.repeats)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.Stream()
    graph = None
    res = {}
    with torch.cuda.stream(stream):
        for i in range(W):
            wl.run(i)
        stream.synchronize()
        wl.ctx.check()
        launches_per_step = wl.ctx.last_launch_count
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(n_sets):
                    wl.run(i)
            graph.replay()
            stream.synchronize()

        def run_steps(n):
            # exactly n steps: whole replays of the n_sets-step graph, the remainder enqueued step by step
            if graph is not None:
                for _ in range(n // n_sets):
                    graph.replay()
                for i in range(n % n_sets):
                    wl.run(i)
                return n
            for i in range(n):
                wl.run(i)
            return n

        sampler = ClockSampler(local)
        run_steps(W)
        barrier()
        sampler.start()
        times = []
        for _ in range(reps):
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            done = run_steps(K)
            e1.record(stream)
            barrier()
            times.append(max_over_ranks(e0.elapsed_time(e1), dev))
        ms = float(np.median(times))
        res.update(value=whole_job_rate(done, world, ms * 1e-3), ms_per_step=ms / done, steps=done, warmup=W,
                   timed_region={"repeats": reps, "ms_median": ms, "ms_min": min(times), "ms_max": max(times),
                                 "steps_per_s_min": whole_job_rate(done, world, max(times) * 1e-3),
                                 "steps_per_s_max": whole_job_rate(done, world, min(times) * 1e-3)})

        # per-kernel durations, measured live with CUDA events on the launching stream (no graph)
        wl.ctx.timing_enable(True)
        kt_steps = max(min(K, 300), 20)
        for i in range(kt_steps):
            wl.run(i)
        stream.synchronize()
        timing = wl.ctx.timing_read()
        wl.ctx.timing_enable(False)

        per_kernel, roofs, step_bytes = kernel_rooflines(w, T, timing, kt_steps, peaks, args.mode, name)
        dom = max(roofs, key=lambda k: timing[k][0])
        res.update(
            launches_per_step=launches_per_step, gpu_launches=launches_per_step * done,
            kernels_us={k: round(v["us"], 3) for k, v in sorted(per_kernel.items())},
            kernel_time_per_step_us=sum(1e3 * v[0] for v in timing.values()) / kt_steps, dominant_kernel=dom,
            roofline=roofs[dom], roofline_other={k: v for k, v in roofs.items() if k != dom},
            tree_attn_frac_of_hbm=roofs["tree_attn"]["frac"] if "tree_attn" in roofs else None,
            tree_attn_us=roofs["tree_attn"]["us_per_launch"] if "tree_attn" in roofs else None,
            lm_head_frac_of_hbm=roofs["gemm_head"].get("hbm_frac", roofs["gemm_head"]["frac"]) if "gemm_head" in roofs else None,
            lm_head_tensor_frac_of_bf16_peak=roofs["gemm_head"]["tensor_frac_of_bf16_peak"] if "gemm_head" in roofs else None,
            lm_head_us=roofs["gemm_head"]["us_per_launch"] if "gemm_head" in roofs else None,
            step_roofline={"algorithmic_bytes": step_bytes, "floor_us": step_bytes / peaks["hbm_gbs"] / 1e3,
                           "frac_of_hbm_floor": step_bytes / peaks["hbm_gbs"] / 1e3 / (1e3 * ms / done)},
            config={"workload": w.name, "B": w.B, "tree_rows": T, "prefix_len": w.prefix_len, "V": w.V, "h": w.h,
                    "heads": w.n_heads, "head_dim": w.head_dim, "ffn": w.ffn, "cfg_scale": w.cfg_scale, "sigma": w.sigma,
                    "mode": args.mode, "top_k_in_step": args.top_k if args.truncate else 0,
                    "step": ("embedding + one decoder layer (q/k/v, rotary, tree attention, output projection, SwiGLU MLP) + "
                             if args.mode != "pieces" else "tree attention + ") +
                            "final norm + LM head/CFG + relaxed acceptance + path selection",
                    "l2": f"inputs rotate over {n_sets} sets of {per_set / 1e6:.0f} MB (> 126 MB L2 between reuses)",
                    "cuda_graph": graph is not None, "parallelism": "replicas" if world > 1 else "single"})
        if light:
            res["clocks"] = sampler.stop()
            acc = [int(s_.out["path_len"].sum()) for s_ in wl.sets]
            res["accepted_tokens_per_step"] = float(np.mean(acc)) / w.B
            wl.close()
            return res, None, None

        # top-k truncation of the target distribution (the paper's sampling setting; not part of the timed step)
        filter_info = None
        if args.top_k > 0:
            gen = torch.Generator(device=dev).manual_seed(w.seed)
            centres = torch.randn(256, generator=gen, device=dev)
            rows_f = w.B * T
            base = centres[torch.arange(w.V, device=dev) % 256][None, :] * (8.0 / 3.0) + \
                0.3 * torch.randn((rows_f, w.V), generator=gen, device=dev)
            copies = [base.clone() for _ in range(22)]
            cb.cascade_filter_logits(wl.ctx, copies[0], args.top_k, 1.0)
            cb.cascade_filter_logits(wl.ctx, copies[1], args.top_k, 1.0)
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            for c in copies[2:]:
                cb.cascade_filter_logits(wl.ctx, c, args.top_k, 1.0)
            f1.record(stream)
            stream.synchronize()
            wl.ctx.check()
            filter_info = {"top_k": args.top_k, "top_p": 1.0, "rows": rows_f, "V": w.V,
                           "us_per_call": 1e3 * f0.elapsed_time(f1) / 20, "logits_bytes": rows_f * w.V * 4,
                           "kept_per_row": int((~torch.isinf(copies[2][0])).sum()), "bound": "latency",
                           "note": "stand-alone call on [B*T, V] fp32 logits resident in the L2"}
            del copies, base
        res["filter_logits"] = filter_info

        # end to end through the host-buffer entry: pinned host inputs in, results out, every step
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_tok = [pin(s.host["tok"]) for s in wl.sets]
        h_p = [pin(s.host["draft_p"]) for s in wl.sets]
        h_u = [pin(s.host["uniforms"]) for s in wl.sets]
        h_acc = torch.zeros((w.B, T), dtype=torch.uint8).pin_memory()
        h_nodes = torch.zeros((w.B, wl.tree.depth + 1), dtype=torch.int32).pin_memory()
        h_len = torch.zeros(w.B, dtype=torch.int32).pin_memory()
        e2e_steps = min(K, 500)

        def host_step(i):
            j = i % n_sets
            cb.cascade_verify_step_host(wl.ctx, wl.tree, wl.sets[j].step, h_tok[j], h_p[j], h_u[j], h_acc, h_nodes, h_len)
            return int(h_len.sum())

        # every input set at least three times before the clock starts: the library records a set's step at its
        # second call and replays it from the third on
        for i in range(max(3 * n_sets, W)):
            host_step(i)
        e2e_times, alpha_sum = [], 0
        for _ in range(reps):
            barrier()
            t0 = time.perf_counter()
            for i in range(e2e_steps):
                alpha_sum += host_step(i)
            e2e_times.append(max_over_ranks(time.perf_counter() - t0, dev))
        e2e_s = float(np.median(e2e_times))
        wl.ctx.check()
        res["clocks"] = sampler.stop()
    res["accepted_tokens_per_step"] = alpha_sum / (reps * e2e_steps * w.B)
    res["e2e"] = {"value": whole_job_rate(e2e_steps, world, e2e_s), "unit": UNIT, "h2d_bytes_per_step": 3 * w.B * T * 4,
                  "d2h_bytes_per_step": w.B * T + w.B * (wl.tree.depth + 1) * 4 + w.B * 4, "steps": e2e_steps,
                  "repeats": reps, "steps_per_s_min": whole_job_rate(e2e_steps, world, max(e2e_times)),
                  "steps_per_s_max": whole_job_rate(e2e_steps, world, min(e2e_times))}
    return res, wl, parent


def attention_back_to_back(w, dev, peaks, launches_per_graph=8, replays=10):
    """The tree-attention kernel alone, launched back to back: a CUDA graph of `launches_per_graph` calls of
    cascade_tree_attn over rotating stand-alone inputs (q, K, V ~ N(0,1), more bytes than the L2 between reuses), timed
    with CUDA events around `replays` replays.  An event pair around a single launch inside the step also times the
    launch and drain of the stream (about 5 us); this figure is the kernel's average duration when launches follow
    each other."""
    import torch
    from paper_2605_07230_b200 import binding as cb
    parent = w.parent()
    T = len(parent)
    R, H, D, P = 2 * w.B, w.n_heads, w.head_dim, w.prefix_len
    ctx = cb.Context(cb.BF16, w.B, T, max(P, 1), w.h, H, H, D, w.V, 0)
    tree = cb.Tree(ctx, parent)
    per_set = R * (P + T) * H * D * 4
    n_sets = max(2, int(np.ceil(3 * 126e6 / per_set)))
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    mk = lambda *shape: torch.randn(shape, generator=gen, device=dev).to(torch.bfloat16)
    sets = [dict(q=mk(R, T, H, D), kp=mk(R, P, H, D), vp=mk(R, P, H, D), kt=mk(R, T, H, D), vt=mk(R, T, H, D),
                 out=torch.zeros((R, T, H, D), dtype=torch.bfloat16, device=dev)) for _ in range(n_sets)]
    plen = torch.full((R,), P, dtype=torch.int32, device=dev)

    def run(i):
        x = sets[i % n_sets]
        cb.cascade_tree_attn(ctx, tree, x["q"], x["kp"], x["vp"], P, plen, x["kt"], x["vt"], x["out"], 1.0 / np.sqrt(D))

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(4):
            run(i)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(launches_per_graph):
                run(i)
        for _ in range(3):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(replays):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    ctx.check()
    us = 1e3 * e0.elapsed_time(e1) / (replays * launches_per_graph)
    nbytes = per_set + 2 * R * T * H * D * 2
    tree.close()
    ctx.close()
    return {"us_per_launch": us, "launches": replays * launches_per_graph, "algorithmic_bytes": nbytes,
            "achieved_gbs": nbytes / us / 1e3, "frac_of_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
            "peak_source": peaks["source"], "inputs": f"{n_sets} rotating sets of {per_set / 1e6:.0f} MB, stand-alone q/K/V"}


def accepted_length_table(dev, steps=8):
    """What the acceptance rule does on the Janus-shaped step: mean accepted drafts per step for three cluster
    tightnesses of the codebook, with the relaxation on (Eq. 1 + Eq. 2 sets) and off (plain Algorithm 1 test)."""
    import torch
    from paper_2605_07230_b200 import binding as cb
    from paper_2605_07230_b200 import synth
    from paper_2605_07230_b200.workload import LayerWorkload
    out = {}
    for sigma in (0.05, 0.1, 0.3):
        w = synth.workload("janus", sigma=sigma)
        wl = LayerWorkload(w, n_layers=1, device=dev, n_sets=1, want_hidden=False)
        row = {}
        for label, flags in (("relaxed", cb.USE_I | cb.USE_C), ("plain", 0)):
            s = wl.sets[0]
            s.step.params = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, flags)
            tot = 0
            for i in range(steps):
                fresh = wl._fresh_step(100 + i)
                for k in ("tok", "draft_p", "uniforms"):
                    s.dev[k].copy_(torch.from_numpy(fresh[k]))
                wl.run(0)
                tot += int(s.out["path_len"].sum())
            row[label] = tot / (steps * w.B)
        out[f"sigma_{sigma}"] = row
        wl.close()
    return {"workload": "janus", "steps_per_entry": steps, "tau": [0.85, 0.5], "tvd_budget": 0.5,
            "accepted_drafts_per_step": out}


def run_loop(args, dev, peaks, rank, world):
    """The last workload of the set: a speculative decode loop through `--layers` decoder layers at the
    Janus-shaped widths, prompt cache 64 rows growing by the accepted tokens until `--tokens` image tokens per
    prompt have been emitted (576 = a 24 x 24 grid).  A step = cascade_verify_step (all layers, head, acceptance,
    path) + cascade_bonus_token + cascade_kv_append; the stand-in drafter and the read-back of path and token run
    on the host between steps and are outside the device time.  Every layer has its own weights and caches on the
    device (12 GB at 30 layers); the values of the layers' weights are those of one seeded layer (see DecodeLoop)."""
    import torch
    import torch.distributed as dist
    from paper_2605_07230_b200 import synth
    from paper_2605_07230_b200.workload import DecodeLoop

    W = 4
    w = synth.workload("janus", prefix_len=64)
    depth = int(synth.tree_depth(w.parent()).max())
    max_steps = args.steps if args.steps > 0 else args.tokens        # at least one token per step
    cap_rows = 64 + args.tokens + (W + 2) * (depth + 1)
    loop = DecodeLoop(w, n_layers=args.layers, max_steps=max_steps + W, device=dev, seed=5, tile_layers=True,
                      cap=cap_rows)
    for _ in range(W):
        loop.step()
    warm_tokens = min(len(e) for e in loop.emitted)
    if not args.no_graph:
        loop.capture()      # note: capturing runs nothing; the caches do not advance
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(int(dev.split(":")[1]))
    sampler.start()
    ev = []
    accepted = 0
    t0 = time.perf_counter()
    K = 0
    while K < max_steps and min(len(e) for e in loop.emitted) < args.tokens:
        drafted = loop.draft()
        ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
        ev[-1][0].record()
        out = loop.step(drafted, events_after=ev[-1][1])
        accepted += int(out["path_len"].sum())
        K += 1
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    clocks = sampler.stop()
    dev_ms = sum(a.elapsed_time(b) for a, b in ev)
    launches = loop.launches_last_step * K
    dev_ms = max_over_ranks(dev_ms, dev)
    wall = max_over_ranks(wall, dev)
    emitted = min(len(e) for e in loop.emitted)
    final_prefix = int(loop.prefix_len_host[0])
    host = loop.host
    parent = loop.parent
    T = loop.T
    loop.close()
    if rank != 0:
        return
    hd = w.n_heads * w.head_dim
    layer_bytes = (4 * hd * w.h + 3 * w.ffn * w.h) * 2
    step_bytes = args.layers * layer_bytes + w.V * w.h * 2
    value = whole_job_rate(K, world, dev_ms * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": dev_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": "loop", "layers": args.layers, "B": w.B, "tree_rows": T, "prefix_len": "64 -> %d" % final_prefix,
                   "tokens_emitted_per_prompt": emitted, "tokens_emitted_in_warmup": warm_tokens,
                   "V": w.V, "h": w.h, "ffn": w.ffn, "heads": w.n_heads, "head_dim": w.head_dim,
                   "step": "verify step through all layers + bonus token + cache append; drafter and read-back on the host, outside the device time",
                   "l2": "each layer streams its own 405 MB of weights (> 126 MB L2)", "cuda_graph": not args.no_graph,
                   "parallelism": "replicas" if world > 1 else "single"},
        "accepted_tokens_per_step": accepted / (K * w.B), "tokens_per_step_with_bonus": accepted / (K * w.B) + 1,
        "tokens_per_s": value * (accepted / (K * w.B) + 1),
        "e2e": {"value": whole_job_rate(K, world, wall), "unit": UNIT, "h2d_bytes_per_step": 3 * w.B * T * 4 + 4 * w.B,
                "d2h_bytes_per_step": w.B * (depth + 1) * 4 + 8 * w.B,
                "note": "wall clock per step including the host drafter, the copies of its output and the read-back of path and token"},
        "gpu_launches": launches,
        "step_roofline": {"algorithmic_bytes": step_bytes, "floor_us": step_bytes / peaks["hbm_gbs"] / 1e3,
                          "frac_of_hbm_floor": step_bytes / peaks["hbm_gbs"] / 1e3 / (1e3 * dev_ms / K)},
        # no kernel is timed alone inside the replayed graph: the whole step against the weight stream it must read
        "roofline": {"kernel": "whole step (every kernel of %d layers + head + acceptance)" % args.layers, "bound": "hbm",
                     "achieved": step_bytes / (1e6 * dev_ms / K), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": step_bytes / (1e6 * dev_ms / K) / peaks["hbm_gbs"], "traffic": None,
                     "peak_source": peaks["source"]},
        "cpu_baseline": None, "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        # the checker on ONE step of the same loop (all layers, the 64-row prompt cache the loop starts from)
        from oracle import cascade_oracle as O
        kp = [k[:, :64] for k in host["k_prefix"]]
        vp = [v[:, :64] for v in host["v_prefix"]]
        t0 = time.perf_counter()
        O.verify_step(host["embed"], host["layers"], host["gamma_final"], host["w_head"], host["tok"], parent, kp, vp,
                      np.full(2 * w.B, 64), host["draft_p"], host["uniforms"], w.n_heads, w.head_dim, w.eps, w.rope_base,
                      w.cfg_scale, 1.0, w.tau_pos, w.tau_seq, w.tvd_budget)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 1.0 / dt, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle",
                                "sample": f"1 verification step through all {args.layers} layers at the loop's first cache length (64 rows); bonus token and cache append not included"}
    print(json.dumps(line))


def run_sweep(args, dev, peaks, rank, world):
    """Every cell of the batched sweep (8 prompts x CFG pair, Janus-shaped widths): draft trees of 16 / 32 / 64 /
    128 nodes x prefix 256 / 1024 / 2048 / 2880 x codebook tightness 0.05 / 0.1 / 0.3.  Per cell: steps/s (device
    time, CUDA-graph replay), accepted drafts per step, the tree attention against the HBM copy rate and the LM
    head against the bf16 tensor peak (burst and sustained).  One JSON line with the table."""
    from paper_2605_07230_b200 import synth
    cells = []
    nodes_list = [int(x) for x in args.sweep_nodes.split(",")]
    prefix_list = [int(x) for x in args.sweep_prefix.split(",")]
    sigma_list = [float(x) for x in args.sweep_sigma.split(",")]
    base = synth.workload("sweep")
    # the seeded pieces that do not depend on the cell are made once: layer weights, the longest cache (shorter
    # prefixes use its first rows), one codebook per tightness
    rng = np.random.default_rng(base.seed)
    R, H, D = 2 * base.B, base.n_heads, base.head_dim
    lw = synth.layer_weights(rng, base.h, H, D, base.ffn)
    lw.wo = lw.wo * np.float32(0.05)
    lw.w_down = lw.w_down * np.float32(0.005)
    for nm in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
        setattr(lw, nm, synth.quantize(getattr(lw, nm), "bf16"))
    Pmax = max(prefix_list)
    kfull = synth.quantize(rng.standard_normal((R, Pmax, H, D), dtype=np.float32), "bf16")
    vfull = synth.quantize(rng.standard_normal((R, Pmax, H, D), dtype=np.float32), "bf16")
    gamma = (1.0 + 0.1 * rng.standard_normal(base.h, dtype=np.float32)).astype(np.float32)
    for sigma in sigma_list:
        E = synth.quantize(synth.clustered_codebook(np.random.default_rng(base.seed + int(1000 * sigma)), base.V, base.h,
                                                    base.n_clusters, sigma), "bf16")
        for nodes in nodes_list:
            for P in prefix_list:
                w = synth.workload("sweep", tree=f"topk{nodes}", prefix_len=P, sigma=sigma)
                parent = w.parent()
                T = len(parent)
                r2 = np.random.default_rng(nodes * 10007 + P)
                tok, p = synth.cluster_drafter(r2, parent, w.B, w.V, w.n_clusters)
                host = dict(embed=E, w_head=E, layers=[lw], k_prefix=[kfull[:, :P]], v_prefix=[vfull[:, :P]],
                            gamma_final=gamma, tok=tok, draft_p=p, uniforms=synth.uniforms(r2, w.B, T),
                            prefix_len=np.full(R, P, np.int32))
                res, _, _ = measure_step("sweep", args, dev, peaks, world, 0,
                                         over=dict(tree=f"topk{nodes}", prefix_len=P, sigma=sigma, _host=host), light=True)
                ro = dict(res["roofline_other"])
                ro[res["dominant_kernel"]] = res["roofline"]
                head, att = ro["gemm_head"], ro["tree_attn"]
                cells.append({"draft_nodes": nodes, "prefix_len": P, "sigma": sigma, "steps_per_s": res["value"],
                              "us_per_step": 1e3 * res["ms_per_step"], "accepted_drafts_per_step": res["accepted_tokens_per_step"],
                              "tree_attn_us": att["us_per_launch"], "tree_attn_frac_of_hbm": att["frac"],
                              "lm_head_us": head["us_per_launch"], "lm_head_rows": w.B * T,
                              "lm_head_tensor_frac_of_bf16_peak": head["tensor_frac_of_bf16_peak"],
                              "lm_head_tensor_frac_of_bf16_sustained": head["tensor_frac_of_bf16_sustained"],
                              "lm_head_frac_of_hbm": head.get("hbm_frac", head["frac"]),
                              "projection_tensor_frac_of_bf16_peak": {k: ro[k]["tensor_frac_of_bf16_peak"] for k in
                                                                      ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down")},
                              "sm_mhz": res["clocks"]["sm_mhz"], "reasons": res["clocks"]["reasons"]})
                print(json.dumps(cells[-1]), file=sys.stderr, flush=True)
    if rank != 0:
        return
    best = max(cells, key=lambda c: c["steps_per_s"])
    line = {"metric": METRIC, "value": best["steps_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": best["us_per_step"] / 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "sweep", "B": base.B, "V": base.V, "h": base.h, "mode": "layer",
                       "note": "value = the fastest cell; every cell is in `cells`", "peaks": peaks},
            "cells": cells}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps per repeat (default 2000; loop mode: until --tokens are emitted)")
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--repeats", type=int, default=5, help="how many times the K-step region is timed (median reported)")
    ap.add_argument("--workload", default="lumina+janus",
                    help="lumina+janus: headline on the Lumina-shaped step, the Janus-shaped step under its own key")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="layer", choices=["layer", "pieces", "loop", "sweep"],
                    help="layer: the step runs through one decoder layer; pieces: the four named pieces alone; "
                         "loop: a 30-layer speculative decode loop (verify, bonus token, cache append each step); "
                         "sweep: every cell of the batched sweep, layer mode")
    ap.add_argument("--layers", type=int, default=30, help="decoder layers in --mode loop")
    ap.add_argument("--tokens", type=int, default=576, help="image tokens per prompt to generate in --mode loop")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every step from Python instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-accept-table", action="store_true")
    ap.add_argument("--top-k", type=int, default=2000,
                    help="also time cascade_filter_logits (top-k truncation of the target logits, outside the step); 0 = skip")
    ap.add_argument("--truncate", action="store_true",
                    help="the timed step itself truncates the target distribution to --top-k (logits are then stored)")
    ap.add_argument("--sets", type=int, default=0, help="rotating input sets (0 = enough to exceed the L2 per step)")
    ap.add_argument("--sweep-nodes", default="16,32,64,128")
    ap.add_argument("--sweep-prefix", default="256,1024,2048,2880")
    ap.add_argument("--sweep-sigma", default="0.05,0.1,0.3")
    args = ap.parse_args()

    from paper_2605_07230_b200 import synth
    names = args.workload.split("+")
    if args.impl == "reference":
        if args.steps <= 0:
            args.steps = 3
        run_reference(args, synth.workload(names[0]))
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = f"cuda:{local}"
    peaks = load_peaks()
    if args.mode == "loop":
        run_loop(args, dev, peaks, rank, world)
    elif args.mode == "sweep":
        if args.steps <= 0:
            args.steps = 200
        run_sweep(args, dev, peaks, rank, world)
    else:
        if args.steps <= 0:
            args.steps = 2000
        line = None
        for i, name in enumerate(names):
            res, wl, parent = measure_step(name, args, dev, peaks, world, local)
            if not args.no_cpu_baseline and world == 1 and rank == 0:
                v, n, cores = time_oracle(wl.w, parent, wl.sets[0].host, "layer" if args.mode == "layer" else "pieces",
                                          max_steps=1 if args.mode == "layer" else 3)
                res["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                       "sample": f"{n} whole step(s) of the {name} workload"}
            wl.close()
            del wl
            torch.cuda.empty_cache()
            if args.mode == "layer" and rank == 0 and synth.workload(name).dtype == "bf16":
                res["tree_attn_back_to_back"] = attention_back_to_back(synth.workload(name), dev, peaks)
            if i == 0:
                line = {"metric": METRIC, "value": res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": res.pop("steps"),
                        "warmup": res.pop("warmup"), "ms_per_step": res.pop("ms_per_step"), "higher_is_better": True,
                        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if name != "toy" else "f32",
                        "data": "synthetic"}
                line.update(res)
            else:
                res.update(metric=METRIC, unit=UNIT)
                line[name] = res
        if not args.no_accept_table and world == 1 and rank == 0 and "janus" in names:
            line["acceptance"] = accepted_length_table(dev)
        if rank == 0:
            print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
