#!/usr/bin/env python
"""Benchmark of the attention-layer training step (forward + backward) on B200.

One step = fbl_layer_fwd + fbl_layer_bwd over one batch of synthetic input.  Without --config the five
workloads are timed one after the other in the same process; the JSON line's top-level figures are those of the
largest one (workload 5, the Llama-7B-shaped long-sequence layer) and `per_config` carries all five.  Reported:
algorithmic TFLOP/s (multiply-add = 2, causal pairs counted once, no recompute), tokens/s, the end-to-end figure
with host buffers, a roofline object for the dominant kernel, the layer's memory efficiency and the float64
oracle timed on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config i] [--impl reference]

With --gpus N > 1 the step runs as N independent replicas, one process per GPU (started by torchrun, or by this
script itself when it is not under a launcher); no tensor of the data path crosses ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from fbl_inputs import get_config, make_inputs, scaled_config  # noqa: E402

NOMINAL_TFLOPS, NOMINAL_GBS = 2250.0, 8000.0
FALLBACK_TFLOPS, FALLBACK_GBS = 1590.0, 6650.0
HEADLINE = 5                      # the largest single-GPU workload
ORDER = (5, 1, 2, 3, 4)           # the headline first: a run cut short still has it


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return dict(tflops_burst=m["bf16_tflops"], tflops_sustained=m["bf16_tflops_sustained"], gbs=m["hbm_gbs"],
                    source="measured")
    return dict(tflops_burst=FALLBACK_TFLOPS, tflops_sustained=1400.0, gbs=FALLBACK_GBS, source="fallback")


def workload_name(cfg):
    return (f"{cfg.name}: B={cfg.batch} T={cfg.seq} D={cfg.d_model} Hq={cfg.n_q_heads} Hkv={cfg.n_kv_heads} "
            f"hd={cfg.head_dim} {cfg.norm} {'causal' if cfg.causal else 'full'} {cfg.dtype}")


def step_flops(cfg):
    """Algorithmic flops of each named step (for the roofline of the dominant one)."""
    n = cfg.n_tokens
    pairs = cfg.seq * (cfg.seq + 1) / 2 if cfg.causal else float(cfg.seq) * cfg.seq
    att = 2.0 * cfg.batch * cfg.n_q_heads * pairs * cfg.head_dim
    pq, pk, po = 2.0 * n * cfg.d_model * cfg.d_q, 2.0 * n * cfg.d_model * cfg.d_kv, 2.0 * n * cfg.d_q * cfg.d_model
    return {"proj_q": pq, "proj_k": pk, "proj_v": pk, "proj_qkv": pq + 2 * pk, "attn_fwd": 2 * att, "proj_o": po,
            "dA": po, "dWo": po, "dWo+dA": 2 * po, "attn_bwd": 4 * att, "dXn": pq + 2 * pk, "dWq": pq, "dWk": pk,
            "dWv": pk, "dWqkv": pq + 2 * pk, "dWqkv+dXn": 2 * (pq + 2 * pk)}


def step_bytes(cfg):
    """Algorithmic HBM bytes of the bandwidth-bound steps."""
    e = 2 if cfg.dtype == "bf16" else 4
    nd = cfg.n_tokens * cfg.d_model * e
    nb = (4 if cfg.residual else 3) * nd
    db = (cfg.n_tokens * (cfg.d_model + cfg.d_q + 2 * cfg.d_kv) * e) if cfg.has_bias else 0
    return {"norm_fwd": 2 * nd, "norm_bwd": nb, "db+norm_bwd": nb + db, "db": db}


def min_bytes(cfg):
    """Once-only minimum HBM traffic of a step: every distinct tensor crosses HBM once per pass that needs it
    (forward: read X and the weights, write Q, K, V, A, LSE, the norm statistics and Y; backward: read dY, X, the
    weights and the saved tensors, write dX and the weight gradients).  The numerator of the memory efficiency."""
    e = 2 if cfg.dtype == "bf16" else 4
    n = cfg.n_tokens
    nd = n * cfg.d_model * e
    w = (cfg.d_model * (cfg.d_q + 2 * cfg.d_kv) + cfg.d_q * cfg.d_model) * e
    qkva = n * (2 * cfg.d_q + 2 * cfg.d_kv) * e
    small = cfg.batch * cfg.n_q_heads * cfg.seq * 4 + n * 8            # LSE, statistics
    return 5 * nd + 3 * w + 2 * qkva + 2 * small


# DRAM bytes per step kernel (dram__bytes_read.sum + dram__bytes_write.sum, MB in the table, bytes in the dict) from the
# ncu capture of one step of every workload summarised in profiles/ncu_step_kernels_all_workloads.md.  ncu flushes the
# caches before each captured launch, so reads are cold; a kernel's own output mostly stays in L2 and is not counted.
# Workload 5 is captured at sequence 2048 (the full 8192-token step holds 2.5 GB and its kernels run for milliseconds:
# too large for a multi-pass capture).  For the kernels whose traffic grows with the tokens (attention, norms) the
# full workload's entries are that capture's figures times 4, the ratio of the token counts; the GEMMs' traffic has
# a weight share that does not grow, so they get no scaled entry.
_MB = 1e6
_NCU_MB = {
    "cfg1-tiny-fp32": {"norm_fwd": 0.03, "proj_q": 0.10, "proj_k": 0.10, "proj_v": 0.10, "attn_fwd": 0.07, "proj_o": 0.10,
                       "dA": 0.10, "dWo": 0.11, "attn_bwd": 0.04 + 0.11 + 0.02, "dXn": 0.16, "dWq": 0.11, "dWk": 0.11,
                       "dWv": 0.11, "norm_bwd": 0.05},
    "cfg2-gpt2-small": {"norm_fwd": 3.46, "proj_qkv": 6.76, "attn_fwd": 9.47, "proj_o": 4.39, "dWo+dA": 7.53,
                        "attn_bwd": 19.12 + 6.30, "dWqkv+dXn": 16.18, "db+norm_bwd": 18.92 + 1.69},
    "cfg3-vit-base": {"norm_fwd": 10.16, "proj_qkv": 13.43, "attn_fwd": 29.53, "proj_o": 11.07, "dWo+dA": 23.26,
                      "attn_bwd": 59.97 + 19.67, "dWqkv+dXn": 50.12, "dW round": 11.06, "norm_bwd": 19.75 + 1.83},
    "cfg4-llama1b-gqa": {"norm_fwd": 16.81, "proj_qkv": 29.42, "attn_fwd": 25.22, "proj_o": 25.23, "dWo+dA": 45.53,
                         "attn_bwd": 77.46 + 33.56, "dWqkv+dXn": 62.33, "norm_bwd": 33.72 + 2.44},
    "cfg5-llama7b-long-scaled": {"norm_fwd": 16.82, "proj_qkv": 147.11, "attn_fwd": 50.56, "proj_o": 50.49, "dWo+dA": 110.03,
                                 "attn_bwd": 118.07 + 33.56, "dWqkv+dXn": 383.49, "norm_bwd": 33.91 + 4.87},
}
_NCU_MB["cfg5-llama7b-long"] = {k: 4.0 * v for k, v in _NCU_MB["cfg5-llama7b-long-scaled"].items()
                                if k in ("norm_fwd", "attn_fwd", "attn_bwd", "norm_bwd")}     # the token-proportional kernels
NCU_TRAFFIC_BYTES = {(w, k): v * _MB for w, steps in _NCU_MB.items() for k, v in steps.items()}
NCU_TRAFFIC_NOTE = {"cfg5-llama7b-long": "seq-2048 capture x 4 (token ratio)"}
# the layer's memory efficiency of workload 5 is the one of its captured seq-2048 instance
MEM_EFF_PROXY = {"cfg5-llama7b-long": ("cfg5-llama7b-long-scaled", dict(seq=2048))}


class ClockSampler:
    """Samples the SM clock and the throttle reasons of one GPU while the timed region runs.

    Uses NVML from a background thread (every 5 ms); falls back to an `nvidia-smi -lms 100` child process.
    Only reads: no clock, power or persistence setting is touched."""

    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"), (0x4, "sw_power_cap"))
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        import threading
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self.stop_flag = threading.Event()
        self.thread = self.proc = self.f = None
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(visible.split(",")[gpu_index]) if visible and visible.split(",")[gpu_index].isdigit() else gpu_index
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def poll():
                while not self.stop_flag.is_set():
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        mask = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                        for bit, name in self.REASONS:
                            if mask & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    time.sleep(0.005)

            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
        except Exception:
            self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                              "-lms", "100", "-i", str(gpu_index)], stdout=self.f,
                                             stderr=subprocess.DEVNULL)
            except OSError:
                self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
        elif self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.f.flush()
            self.f.seek(0)
            for line in self.f.read().splitlines():
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    self.sm.append(float(parts[1]))
                    self.max_mhz = float(parts[2])
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                    if val.lower().startswith("active"):
                        self.reasons.add(name)
            os.unlink(self.f.name)
        if self.sm:
            sm = sorted(self.sm)
            out.update(sm_mhz=sm[len(sm) // 2], sm_mhz_min=sm[0], sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons),
                       samples=len(sm))
        return out


# ---- the float64 oracle on the host cores (the cpu_baseline leg and the reference arm) ---------------------------
def time_oracle(cfg, inp, repeats):
    from oracle import layer as orc
    t = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.layer_fwd_bwd(cfg, inp)
        t.append(time.perf_counter() - t0)
    return t


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_sample(cfg, flop_budget=1.0e12):
    """A bounded sample of the workload for the oracle (about ten seconds of float64 work on the host): fewer
    batch elements first, then, for a single long sequence, its first tokens (a causal layer's prefix is a
    smaller instance of the same layer)."""
    batch = max(1, min(cfg.batch, int(flop_budget // max(cfg.flops() / cfg.batch, 1.0))))
    scfg = scaled_config(cfg, batch=batch)
    seq, what = cfg.seq, f"batch {batch} of {cfg.batch}, full sequence"
    while scfg.flops() > flop_budget and seq > 256:
        seq //= 2
        scfg = scaled_config(cfg, batch=batch, seq=seq)
        what = f"batch {batch} of {cfg.batch}, the first {seq} of {cfg.seq} tokens of each sequence"
    return scfg, what


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    import numpy as np  # noqa: F401  (loads the BLAS threadpool before it is inspected)
    scfg, what = oracle_sample(cfg)
    inp = make_inputs(scfg)
    passes = max(1, min(args.steps, 3))                   # a few passes, not --steps of them: each takes seconds
    time_oracle(scfg, inp, min(args.warmup, 1))
    t = time_oracle(scfg, inp, passes)
    sec = sum(t) / len(t)
    tfl = scfg.flops() / sec / 1e12
    sample = f"{what}; one fwd+bwd per step, {passes} timed steps (--steps {args.steps} capped at 3)"
    line = {"impl": "reference", "metric": "fwd+bwd layer TFLOP/s", "value": tfl, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "tokens_per_s": scfg.n_tokens / sec,
            "config": {"workload": workload_name(cfg)},
            "cpu_baseline": {"value": tfl, "unit": "TFLOP/s", "cores": host_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": tfl, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---- one workload on this rank's GPU ---------------------------------------------------------------------------
def lora_flops(cfg, r):
    """Algorithmic flops of a step with rank-r adapters on Q, K, V and frozen base weights: the base step without its
    four weight-gradient products, plus the adapters' six thin products (and their term in dXn)."""
    n, d, dqkv = cfg.n_tokens, cfg.d_model, cfg.d_q + 2 * cfg.d_kv
    frozen = 2.0 * n * d * dqkv + 2.0 * n * cfg.d_q * d
    return cfg.flops() - frozen + 3 * 2.0 * n * d * 3 * r + 3 * 2.0 * n * r * dqkv


def measure(cfg, args, rep, local_rank, flush_l2, want_cpu, lora_rank=0):
    import torch
    from paper_2607_21624_b200 import TENSOR, LayerRunner, LoraRunner

    if lora_rank:
        from fbl_inputs import make_lora_inputs
        inp = make_lora_inputs(cfg, lora_rank)
        run = LoraRunner(cfg, lora_rank, device=f"cuda:{local_rank}")
    else:
        inp = make_inputs(cfg)
        run = LayerRunner(cfg, device=f"cuda:{local_rank}")
    run.plan.set_kernel_path(args.path)
    run.load_inputs(inp)
    stream = torch.cuda.Stream()
    steps, warmup = args.steps, args.warmup

    graph = g_fwd = g_bwd = None
    with torch.cuda.stream(stream):
        run.step()                      # first call sets kernel attributes; keep it outside any capture
        stream.synchronize()
        assert run.status() == 0
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                run.step()
            g_fwd = torch.cuda.CUDAGraph()      # the two halves on their own: timed separately, and used by the
            with torch.cuda.graph(g_fwd, stream=stream):      # end-to-end leg (host copies overlap the other half)
                run.forward()
            g_bwd = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_bwd, stream=stream):
                run.backward()

    one_step = graph.replay if graph is not None else run.step
    fwd_only = g_fwd.replay if g_fwd is not None else run.forward
    bwd_only = g_bwd.replay if g_bwd is not None else run.backward

    def barrier():
        torch.cuda.synchronize()
        rep.barrier()
        torch.cuda.synchronize()

    launches0 = run.plan.launch_count()
    with torch.cuda.stream(stream):
        run.step()
    launches_per_step = run.plan.launch_count() - launches0
    torch.cuda.synchronize()

    def timed(fn, n, cold=True, pre=None):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                if pre:
                    pre()
                if cold:
                    flush_l2()
                fn()
        barrier()
        with torch.cuda.stream(stream):
            for a, b in ev:
                if pre:
                    pre()
                if cold:
                    flush_l2()
                a.record(stream)
                fn()
                b.record(stream)
        barrier()
        t = [a.elapsed_time(b) for a, b in ev]
        return sum(t) / len(t), min(t)

    # ---- device-resident timing: L2 flushed before every step, events around each step ----------
    sampler = ClockSampler(local_rank)
    t_wall0 = time.perf_counter()
    ms, ms_min = timed(one_step, steps, cold=True)
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    assert run.status() == 0
    n_aux = max(3, min(steps, 30))
    ms_warm, _ = timed(one_step, n_aux, cold=False)                      # operands left in L2 by the step before
    ms_fwd, _ = timed(fwd_only, n_aux, cold=True)
    ms_bwd, _ = timed(bwd_only, n_aux, cold=True, pre=fwd_only)          # `saved` from a forward, then flush, then time

    # ---- end to end with host buffers: H2D of X and dY, pack, step, unpack, D2H of Y and dX --------
    tdt = run.tdtype
    shape = (cfg.batch, cfg.seq, cfg.d_model)
    hX = run.to_device_rowmajor(inp["X"]).cpu().pin_memory()
    hdY = run.to_device_rowmajor(inp["dY"]).cpu().pin_memory()
    hY = torch.empty(shape, dtype=tdt).pin_memory()
    hdX = torch.empty(shape, dtype=tdt).pin_memory()
    dX_rm = torch.empty(shape, dtype=tdt, device="cuda")
    dY_rm = torch.empty(shape, dtype=tdt, device="cuda")
    oY_rm = torch.empty(shape, dtype=tdt, device="cuda")
    odX_rm = torch.empty(shape, dtype=tdt, device="cuda")

    # A second stream carries what the other half of the step does not wait for: dY comes in while the forward runs,
    # Y goes out while the backward runs.  The timed region (events on the main stream) ends after both have joined.
    side = torch.cuda.Stream()
    ev_start, ev_dy, ev_fwd, ev_y = (torch.cuda.Event() for _ in range(4))

    def e2e_step():
        s = stream.cuda_stream
        ev_start.record(stream)
        dX_rm.copy_(hX, non_blocking=True)
        with torch.cuda.stream(side):
            side.wait_event(ev_start)
            dY_rm.copy_(hdY, non_blocking=True)
            ev_dy.record(side)
        run.plan.pack(TENSOR["X"], dX_rm.data_ptr(), run.buf["X"].data_ptr(), s)
        fwd_only()
        ev_fwd.record(stream)
        with torch.cuda.stream(side):
            side.wait_event(ev_fwd)
            run.plan.unpack(TENSOR["Y"], run.buf["Y"].data_ptr(), oY_rm.data_ptr(), side.cuda_stream)
            hY.copy_(oY_rm, non_blocking=True)
            ev_y.record(side)
        stream.wait_event(ev_dy)
        run.plan.pack(TENSOR["DY"], dY_rm.data_ptr(), run.buf["dY"].data_ptr(), s)
        bwd_only()
        run.plan.unpack(TENSOR["DX"], run.buf["dX"].data_ptr(), odX_rm.data_ptr(), s)
        hdX.copy_(odX_rm, non_blocking=True)
        stream.wait_event(ev_y)

    ms_e2e, _ = timed(e2e_step, max(3, min(steps, 50)), cold=True)
    assert run.status() == 0
    assert torch.equal(hY, oY_rm.cpu()) and torch.equal(hdX, odX_rm.cpu())     # both streams had joined
    io_bytes = 2 * cfg.n_tokens * cfg.d_model * (2 if cfg.dtype == "bf16" else 4)

    # ---- per-kernel event timing: a separate pass of direct launches with an event after every kernel group.  The
    # event between two kernels keeps the second from starting its set-up under the first one's tail (programmatic
    # dependent launch), so each figure is a kernel's stand-alone duration and their sum exceeds the step time. ----
    run.plan.profile_enable(True)
    acc = {}
    with torch.cuda.stream(stream):
        for _ in range(max(3, min(steps, 10))):
            flush_l2()
            run.forward()
            stream.synchronize()
            for name, t in run.plan.profile_read():
                acc.setdefault(name, []).append(t)
            run.backward()
            stream.synchronize()
            for name, t in run.plan.profile_read():
                acc.setdefault(name, []).append(t)
    run.plan.profile_enable(False)
    kernel_ms = {k: sum(v) / len(v) for k, v in acc.items()}

    ms, ms_warm, ms_fwd, ms_bwd, ms_e2e = rep.max_over_ranks([ms, ms_warm, ms_fwd, ms_bwd, ms_e2e])   # the slowest replica counts
    sizes = dict(run.sizes)
    del run, graph, g_fwd, g_bwd, hX, hdY, hY, hdX, dX_rm, dY_rm, oY_rm, odX_rm
    torch.cuda.empty_cache()
    if rep.rank != 0:
        return None

    peaks = measured_peaks()
    flops = lora_flops(cfg, lora_rank) if lora_rank else cfg.flops()
    tfl = rep.whole_job_rate(flops, ms) / 1e12
    sf, sbytes = step_flops(cfg), step_bytes(cfg)
    if lora_rank:
        thin = 2.0 * cfg.n_tokens * lora_rank
        sf.update({"lora_T": thin * 3 * cfg.d_model, "lora_dA": thin * 3 * cfg.d_model, "lora_dT": thin * (cfg.d_q + 2 * cfg.d_kv),
                   "proj_qkv": sf["proj_qkv"] + thin * (cfg.d_q + 2 * cfg.d_kv),
                   "dB+dXn": sf["dXn"] + thin * (cfg.d_q + 2 * cfg.d_kv) + thin * 3 * cfg.d_model})
    dom = max(kernel_ms, key=kernel_ms.get)
    total_k = sum(kernel_ms.values())
    if dom in sf:
        ach = sf[dom] / (kernel_ms[dom] * 1e-3) / 1e12
        if cfg.dtype == "bf16" and args.path == 0:
            roof = {"bound": "tensor", "kernel": dom, "achieved": ach, "peak": peaks["tflops_burst"], "unit": "TFLOP/s",
                    "frac": ach / peaks["tflops_burst"], "traffic": None, "peak_source": peaks["source"] + " (burst)"}
        else:
            # FFMA path: SMs x 128 lanes x 2 flop x 1.965 GHz
            sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
            alu = sms * 128 * 2 * 1.965e9 / 1e12
            roof = {"bound": "alu", "kernel": dom, "achieved": ach, "peak": alu, "unit": "TFLOP/s", "frac": ach / alu,
                    "traffic": None, "peak_source": f"{sms} SM x 128 FFMA/clk x 1.965 GHz"}
    else:
        ach = sbytes.get(dom, 0.0) / (kernel_ms[dom] * 1e-3) / 1e9
        roof = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peaks["gbs"], "unit": "GB/s",
                "frac": ach / peaks["gbs"], "traffic": None, "peak_source": peaks["source"]}
    roof["traffic"] = NCU_TRAFFIC_BYTES.get((cfg.name, dom))
    if cfg.name in NCU_TRAFFIC_NOTE:
        roof["traffic_note"] = NCU_TRAFFIC_NOTE[cfg.name]
    roof["kernel_share"] = kernel_ms[dom] / total_k
    roof["kernel_ms"] = {k: round(v, 5) for k, v in sorted(kernel_ms.items(), key=lambda kv: -kv[1])}
    roof["kernel_ms_sum_over_step_ms"] = total_k / ms      # > 1: what programmatic launch overlap hides in a real step
    roof["timing"] = "stand-alone kernel durations (an event after every kernel group; no launch overlap)"
    # the bandwidth-bound kernels of the step against the measured HBM copy rate
    roof["hbm_kernels"] = {k: {"GBps": sbytes[k] / (kernel_ms[k] * 1e-3) / 1e9,
                               "frac": sbytes[k] / (kernel_ms[k] * 1e-3) / 1e9 / peaks["gbs"]}
                           for k in kernel_ms if sbytes.get(k)}
    # per-kernel fraction of the tensor peak for the tensor-bound ones
    roof["tensor_kernels"] = {k: {"TFLOPs": sf[k] / (kernel_ms[k] * 1e-3) / 1e12,
                                  "frac": sf[k] / (kernel_ms[k] * 1e-3) / 1e12 / peaks["tflops_burst"]}
                              for k in kernel_ms if k in sf} if cfg.dtype == "bf16" and args.path == 0 else {}

    # memory efficiency of the layer (the paper's Eq. 2 factor): once-only minimum bytes over the DRAM bytes ncu saw
    proxy_name, proxy_cfg = cfg.name, cfg
    if cfg.name in MEM_EFF_PROXY:
        proxy_name = MEM_EFF_PROXY[cfg.name][0]
        proxy_cfg = scaled_config(cfg, **MEM_EFF_PROXY[cfg.name][1])
    steps_with_traffic = {k: NCU_TRAFFIC_BYTES.get((proxy_name, k)) for k in kernel_ms}
    if all(v is not None for v in steps_with_traffic.values()):
        dram = sum(steps_with_traffic.values())
        mem_eff = {"min_bytes": min_bytes(proxy_cfg), "ncu_dram_bytes": dram, "value": min_bytes(proxy_cfg) / dram,
                   "source": "profiles/ncu_step_kernels_all_workloads.md (cold-cache captures, one per kernel)"
                             + ("; measured on this workload's 2048-token instance" if proxy_name != cfg.name else "")}
    else:
        mem_eff = {"min_bytes": min_bytes(cfg), "ncu_dram_bytes": None, "value": None,
                   "source": "no ncu capture of every kernel of this workload under profiles/"}

    cpu = None
    if want_cpu:
        scfg, what = oracle_sample(cfg)
        sinp = make_inputs(scfg)
        t = time_oracle(scfg, sinp, 2)
        sec = min(t)
        cpu = {"value": scfg.flops() / sec / 1e12, "unit": "TFLOP/s", "cores": host_threads(), "kind": "oracle",
               "sample": f"{what}; best of 2 fwd+bwd passes", "seconds": sec}

    t_tensor = flops / (peaks["tflops_burst"] * 1e12)
    return {
        "workload": workload_name(cfg) + (f" + rank-{lora_rank} adapters on Q, K, V, base weights frozen" if lora_rank else ""),
        "ms_per_step": ms, "ms_per_step_min": ms_min, "ms_per_step_warm_l2": ms_warm,
        "ms_fwd": ms_fwd, "ms_bwd": ms_bwd,
        "tflops": tfl, "tokens_per_s": rep.whole_job_rate(cfg.n_tokens, ms), "flops_per_step": flops,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
        "layer_roofline": {"binds": "tensor" if cfg.dtype == "bf16" else "launch latency",
                           "t_tensor_us_at_measured_burst": t_tensor * 1e6,
                           "frac_of_measured_burst": t_tensor / (ms * 1e-3),
                           "frac_of_measured_sustained": flops / (peaks["tflops_sustained"] * 1e12) / (ms * 1e-3),
                           "frac_of_nominal_2250": flops / (NOMINAL_TFLOPS * 1e12) / (ms * 1e-3),
                           "t_hbm_us_min_bytes_at_measured": min_bytes(cfg) / (peaks["gbs"] * 1e9) * 1e6},
        "mem_efficiency": mem_eff,
        "activation_bytes": {"saved": sizes["saved"], "scratch": sizes["scratch_fwd"] + sizes["scratch_bwd"]},
        "e2e": {"value": rep.whole_job_rate(flops, ms_e2e) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": io_bytes, "d2h_bytes_per_step": io_bytes},
        "launches_per_step": launches_per_step, "clocks": clocks, "roofline": roof, "cpu_baseline": cpu,
        "wall_s_timed_region": t_wall,
    }


def measure_mlp(key, args, rep, local_rank, flush_l2):
    """The feed-forward block `key` of fbl_inputs.MLP_CONFIGS on this rank's GPU: forward + backward, cold L2, graph replay."""
    import torch
    from fbl_inputs import MLP_CONFIGS, make_mlp_inputs
    from paper_2607_21624_b200 import MlpRunner
    cfg = MLP_CONFIGS[key]
    run = MlpRunner(cfg, device=f"cuda:{local_rank}")
    run.plan.set_kernel_path(args.path)
    run.load_inputs(make_mlp_inputs(cfg))
    return time_runner(run, cfg, f"{cfg.name}: B={cfg.batch} T={cfg.seq} D={cfg.d_model} F={cfg.d_ff} {cfg.act} {cfg.norm} {cfg.dtype}",
                       args, rep, flush_l2)


def measure_xattn(key, args, rep, local_rank, flush_l2):
    """The cross-attention layer `key` of fbl_inputs.XATTN_CONFIGS, timed like the feed-forward blocks."""
    from fbl_inputs import XATTN_CONFIGS, make_xattn_inputs
    from paper_2607_21624_b200 import XattnRunner
    cfg = XATTN_CONFIGS[key]
    run = XattnRunner(cfg, device=f"cuda:{local_rank}")
    run.plan.set_kernel_path(args.path)
    run.load_inputs(make_xattn_inputs(cfg))
    return time_runner(run, cfg, f"{cfg.name}: B={cfg.batch} Tq={cfg.seq} Tkv={cfg.seq_kv} D={cfg.d_model} Dmem={cfg.d_mem} "
                       f"Hq={cfg.n_q_heads} Hkv={cfg.n_kv_heads} hd={cfg.head_dim} {cfg.norm} {cfg.dtype}", args, rep, flush_l2)


def time_runner(run, cfg, workload, args, rep, flush_l2):
    """Forward + backward of a loaded runner: cold L2 before every step, graph replay, max over ranks."""
    import torch
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run.step()
        stream.synchronize()
        assert run.status() == 0
        l0 = run.plan.launch_count()
        run.step()
        launches = run.plan.launch_count() - l0
        graph = g_fwd = None
        if not args.no_graph:
            graph, g_fwd = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                run.step()
            with torch.cuda.graph(g_fwd, stream=stream):
                run.forward()
    step = graph.replay if graph is not None else run.step
    fwd = g_fwd.replay if g_fwd is not None else run.forward

    def timed(fn, n):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        with torch.cuda.stream(stream):
            for _ in range(args.warmup):
                flush_l2()
                fn()
            for a, b in ev:
                flush_l2()
                a.record(stream)
                fn()
                b.record(stream)
        torch.cuda.synchronize()
        rep.barrier()
        t = [a.elapsed_time(b) for a, b in ev]
        return sum(t) / len(t)

    ms = timed(step, args.steps)
    ms_fwd = timed(fwd, max(3, min(args.steps, 30)))
    assert run.status() == 0
    ms, ms_fwd = rep.max_over_ranks([ms, ms_fwd])
    sizes = dict(run.sizes)
    del run, graph, g_fwd
    torch.cuda.empty_cache()
    if rep.rank != 0:
        return None
    peaks = measured_peaks()
    flops = cfg.flops()
    return {"workload": workload,
            "ms_per_step": ms, "ms_fwd": ms_fwd, "tflops": rep.whole_job_rate(flops, ms) / 1e12,
            "tokens_per_s": rep.whole_job_rate(cfg.n_tokens, ms), "flops_per_step": flops, "dtype": "bf16",
            "layer_roofline": {"binds": "tensor", "frac_of_measured_burst": flops / (peaks["tflops_burst"] * 1e12) / (ms * 1e-3),
                               "frac_of_nominal_2250": flops / (NOMINAL_TFLOPS * 1e12) / (ms * 1e-3)},
            "activation_bytes": {"saved": sizes["saved"], "scratch": sizes["scratch_fwd"] + sizes["scratch_bwd"]},
            "launches_per_step": launches}


def run_rank(args):
    """Body of one rank (the only one at N = 1)."""
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    def pick(i):
        cfg = get_config(i)
        if args.seq or args.batch:
            cfg = scaled_config(cfg, name=cfg.name + "-scaled", seq=args.seq or cfg.seq, batch=args.batch or cfg.batch)
        return cfg

    if args.impl == "reference":
        run_reference(args, pick(args.config or HEADLINE), rank)
        return

    import torch
    from paper_2607_21624_b200.build import build
    build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local_rank)
    from paper_2607_21624_b200.replicas import Replicas
    rep = Replicas(backend="nccl", device=torch.device("cuda", local_rank))

    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # 256 MiB > 126 MB L2
    flush_rd = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device="cuda")  # 256 MiB, only ever read
    flush_sink = torch.zeros(1, dtype=torch.int32, device="cuda")

    def flush_l2():
        # Write a buffer larger than L2, then read another one: the write evicts the step's data, the read evicts
        # the write's dirty lines, whose write-back would otherwise run inside the timed step and take DRAM bandwidth
        # from it (an artefact of the flush, not of the workload).
        flush.zero_()
        if not args.flush_write_only:
            torch.sum(flush_rd, dim=0, keepdim=True, dtype=torch.int32, out=flush_sink)

    head = args.config or HEADLINE
    todo = [args.config] if args.config else list(ORDER)
    results = {}
    for i in todo:
        cfg = pick(i)
        results[i] = measure(cfg, args, rep, local_rank, flush_l2, want_cpu=(i == head and not args.no_cpu_baseline))
    mlp = {}
    if not args.config and not args.no_mlp:          # the feed-forward blocks behind these attention layers
        for key in ("matmul-512x2048x8192", "gpt2", "llama1b"):
            mlp[key] = measure_mlp(key, args, rep, local_rank, flush_l2)
    lora = {}
    xattn = {}
    if not args.config and not args.no_mlp:          # the paper's fine-tuning setting on two of the workloads
        for i in (2, 4):
            lora[i] = measure(pick(i), args, rep, local_rank, flush_l2, want_cpu=False, lora_rank=16)
        xattn["whisper-large"] = measure_xattn("whisper-large", args, rep, local_rank, flush_l2)
    if rank != 0:
        rep.close()
        return

    h = results[head]
    peaks = measured_peaks()
    line = {
        "metric": "fwd+bwd layer TFLOP/s", "value": h["tflops"], "unit": "TFLOP/s", "n_gpus": rep.world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": h["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": h["dtype"], "data": "synthetic",
        "config": {"workload": h["workload"],
                   "l2": "256 MiB written" + ("" if args.flush_write_only else ", then 256 MiB read (so that the write-back of the flush is over)") + " before every timed step",
                   "launch": "direct launches" if args.no_graph else "cuda graph replay",
                   "kernel_path": "default" if args.path == 0 else "ffma", "parallelism": "replicas only",
                   "also_timed": "per_config holds all five workloads, each timed the same way in this process"},
        "tokens_per_s": h["tokens_per_s"], "layer_roofline": h["layer_roofline"], "mem_efficiency": h["mem_efficiency"],
        "activation_bytes": h["activation_bytes"], "e2e": h["e2e"],
        "gpu_launches": (sum(r["launches_per_step"] for r in results.values())
                         + sum(r["launches_per_step"] for r in mlp.values())
                         + sum(r["launches_per_step"] for r in lora.values())
                         + sum(r["launches_per_step"] for r in xattn.values())) * args.steps,
        "clocks": h["clocks"], "roofline": h["roofline"], "cpu_baseline": h["cpu_baseline"],
        "peaks": peaks,
        "per_config": {**{f"workload{i}": results[i] for i in sorted(results)}, **{f"mlp_{k}": v for k, v in mlp.items()},
                       **{f"lora16_workload{i}": v for i, v in lora.items()},
                       **{f"xattn_{k}": v for k, v in xattn.items()}},
    }
    print(json.dumps(line))
    rep.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=0, help="1-based index of one workload (default: all five, headline = the fifth)")
    ap.add_argument("--impl", default="fblayout", choices=["fblayout", "reference"])
    ap.add_argument("--path", type=int, default=0, help="0 default kernels, 1 FFMA kernels only")
    ap.add_argument("--no-graph", action="store_true", help="enqueue kernels directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-mlp", action="store_true", help="skip the feed-forward and adapter entries of per_config")
    ap.add_argument("--flush-write-only", action="store_true", help="flush L2 by the 256 MiB write alone (its write-back then overlaps the step)")
    ap.add_argument("--seq", type=int, default=0, help="override the workload's sequence length (profiling captures)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "fblayout" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "fblayout":
        # not under a launcher: start the replicas ourselves, one process per GPU
        from paper_2607_21624_b200.replicas import spawn_replicas
        spawn_replicas(args.gpus, run_rank, args)
        return
    run_rank(args)


if __name__ == "__main__":
    main()
