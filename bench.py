#!/usr/bin/env python
"""Benchmark of the DDTS hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1|cfg2|cfg4|cfg3]
                    [--impl ours|reference]

One "step" is one pass of the whole path over one batch of seeded synthetic input:
for the prefill workloads one ``rodimus_ddts_fwd`` call (gates, in-chunk cumulative decay,
intra-chunk scores and outputs, inter-chunk readout, state update, output and final-state
stores); for ``cfg3`` one ``rodimus_ddts_step`` call over all sequences.  Prints ONE JSON line.

With N > 1 (launched by ``torch.distributed.run``) every rank runs its own replica of the
workload on its own GPU (independent batches: no collective on the data path) and the value
is all ranks' tokens over the slowest rank's device time.

``--impl reference`` times the fp64 CPU oracle, as it stands, on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
WORKLOADS = {"cfg1": 1, "cfg2": 2, "cfg3": 3, "cfg4": 4}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"])}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu summary, if one covers this kernel/workload."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        d = json.load(f)
    ent = d.get(f"{kernel}:{workload}")
    return None if ent is None else ent.get("bytes_per_launch")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only queries) while the timed region
    runs; falls back to ``nvidia-smi`` if the NVML binding is unavailable."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.samples = []          # (sm_mhz, max_mhz, [active reason names])
        self.stop = threading.Event()
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            # NVML numbers devices in PCI order; honour CUDA_VISIBLE_DEVICES when it holds indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [t for t in vis.split(",") if t.strip().isdigit()]
            phys = int(ids[gpu_index]) if gpu_index < len(ids) else gpu_index
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.masks = {
                "hw_slowdown": pynvml.nvmlClocksEventReasonHwSlowdown,
                "hw_thermal_slowdown": pynvml.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": pynvml.nvmlClocksEventReasonSwThermalSlowdown,
                "sw_power_cap": pynvml.nvmlClocksEventReasonSwPowerCap,
            }
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _once(self):
        try:
            if self.nvml is not None:
                mhz = float(self.nvml.nvmlDeviceGetClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
                bits = int(self.nvml.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                self.samples.append((mhz, self.max_mhz, [n for n, m in self.masks.items() if bits & m]))
                return
            out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                  "-i", str(self.idx)], capture_output=True, text=True, timeout=10).stdout
            f = [t.strip() for t in out.strip().split(",")]
            if len(f) >= 6:
                act = [n for n, v in zip(self.NAMES, f[2:6]) if v.lower().startswith("active")]
                self.samples.append((float(f[0]), float(f[1]), act))
        except Exception:
            pass

    def _run(self):
        while not self.stop.is_set():
            self._once()
            self.stop.wait(0.002 if self.nvml is not None else 0.05)

    def __enter__(self):
        self.thread.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        self.thread.join(timeout=15)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        reasons = sorted({n for s in self.samples for n in s[2]})
        return {"sm_mhz": float(np.median([s[0] for s in self.samples])),
                "sm_max_mhz": float(self.samples[0][1]), "reasons": reasons,
                "samples": len(self.samples), "source": "nvml" if self.nvml is not None else "nvidia-smi"}


# ----------------------------------------------------------------------------------------------
# workload description shared by both arms
# ----------------------------------------------------------------------------------------------

def describe(workload: str, p, n_gpus: int):
    if workload == "cfg3":
        Nseq, H, dk, dv = p.state.shape
        return {"workload": "cfg3_decode: 256 sequences x 16 heads, one token each, fp32 state in place",
                "Nseq_per_gpu": Nseq, "H": H, "dk": dk, "dv": dv, "ingate": "g^tau",
                "replicas": n_gpus, "l2": "state (1.07 GB) larger than L2"}
    B, H, T, dk, dv = p.shape
    names = {"cfg1": "cfg1_layer_prefill: B=4 H=16 T=2048 dk=128 dv=256 bf16, zero initial state",
             "cfg2": "cfg2_long_context: B=1 H=16 T=32768 dk=128 dv=256 bf16, nonzero initial state",
             "cfg4": "cfg4_varlen: 64 packed sequences, lengths U[128,4096], H=16 dk=128 dv=256 bf16"}
    return {"workload": names[workload], "B_per_gpu": B, "H": H, "T": T, "dk": dk, "dv": dv,
            "tokens_per_gpu": p.tokens, "ingate": "g^tau", "replicas": n_gpus,
            "l2": "inputs larger than L2, no flush"}


def prefill_bytes(p) -> int:
    """Algorithmic HBM bytes of one prefill call: q,k,x,y,v read, o written, states read/written."""
    B, H, T, dk, dv = p.shape
    el = 2 if p.dtype == "bf16" else 4
    nseq = B if p.cu_seqlens is None else len(p.cu_seqlens) - 1
    tok = B * H * T * (4 * dk + 2 * dv) * el
    st = nseq * H * dk * dv * 4
    return tok + st * (2 if p.s0 is not None else 1)


def decode_bytes(p) -> int:
    Nseq, H, dk, dv = p.state.shape
    return Nseq * H * (2 * dk * dv * 4 + (4 * dk + 2 * dv) * 2)


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle
# ----------------------------------------------------------------------------------------------

def oracle_sample_run(workload: str, p, budget_s: float = 10.0):
    """Times the oracle on a bounded sample of the workload; returns (units, seconds, what)."""
    from oracle import ddts_oracle as orc
    if workload == "cfg3":
        Nseq = min(p.state.shape[0], 64)
        st = np.ascontiguousarray(p.state[:Nseq]).astype(np.float64)
        sl = lambda a: np.ascontiguousarray(a[0][:Nseq])
        args = [sl(a) for a in (p.q, p.k, p.x, p.y, p.v)]
        t0 = time.perf_counter()
        steps = 0
        while steps < 64 and (time.perf_counter() - t0 < budget_s or steps < 2):
            orc.ref_step(*args, st)
            steps += 1
        dt = time.perf_counter() - t0
        per_seq = decode_bytes(p) / p.state.shape[0]
        return per_seq * Nseq * steps, dt, f"{steps} steps over the first {Nseq} of {p.state.shape[0]} sequences"
    B, H, T, dk, dv = p.shape
    if p.cu_seqlens is not None:
        heads = min(H, 2)
        sl = lambda a: np.ascontiguousarray(a[:, :heads])
        t0 = time.perf_counter()
        orc.ref_fwd(sl(p.q), sl(p.k), sl(p.x), sl(p.y), sl(p.v), cu_seqlens=p.cu_seqlens, want_o=True)
        dt = time.perf_counter() - t0
        return p.tokens * heads / H, dt, f"{heads} of {H} heads of all {len(p.cu_seqlens) - 1} sequences"
    heads = H if B * H * T <= 4 * 16 * 2048 else max(1, (4 * 16 * 2048) // (B * T))
    sl = lambda a: np.ascontiguousarray(a[:, :heads])
    s0 = None if p.s0 is None else sl(p.s0).astype(np.float64)
    args = [sl(a) for a in (p.q, p.k, p.x, p.y, p.v)]
    t0 = time.perf_counter()
    reps = 0
    while reps < 8 and (time.perf_counter() - t0 < budget_s or reps < 1):
        orc.ref_fwd(*args, s0=s0)
        reps += 1
    dt = time.perf_counter() - t0
    return p.tokens * heads / H * reps, dt, f"{reps} pass(es) over {heads} of {H} heads, all {B * T} tokens"


def run_reference(args, workload, p):
    from oracle import ddts_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = orc.num_threads()
    for _ in range(args.warmup):
        oracle_sample_run(workload, p, budget_s=0.0)
    units = secs = 0.0
    what = ""
    for _ in range(args.steps):
        u, s, what = oracle_sample_run(workload, p, budget_s=max(2.0, 60.0 / max(args.steps, 1)))
        units += u
        secs += s
    decode = workload == "cfg3"
    val = units / secs / (1e9 if decode else 1.0)
    unit = "GB/s" if decode else "tokens/s"
    line = {
        "impl": "reference",
        "metric": "DDTS decode state GB/s" if decode else "DDTS prefill tokens/s",
        "value": val, "unit": unit, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": describe(workload, p, args.gpus),
        "cpu_baseline": {"value": val, "unit": unit, "cores": cores, "kind": "oracle",
                         "sample": f"each step: {what}"},
        "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------

# Work per token-head behind the three bound times printed beside every prefill roofline
# (dk = 128, dv = 256): tensor flops of the chunkwise form at chunk length 64 (state update and
# readout 2*dk*dv each, causal intra-chunk (C+1)(dk+dv)) and special-function approximations of
# the gate math (6 per key channel with the paper's input gate: softplus 2, sigmoid 1, log g 1,
# the two operand exponentials 2).
DATASHEET = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
DATASHEET_TF32_RATIO = 1100.0 / 2250.0   # nominal dense tf32 : bf16


def work_per_token_head(dk: int, dv: int, chunk: int = 64):
    return {"tensor_flops": 4 * dk * dv + (chunk + 1) * (dk + dv), "sfu_ops": 6 * dk}


def measure_sfu_rate(rd, torch, device):
    """Special-function approximations per second of the whole device (CUDA events around the
    library's probe launch, best of 5 after a warm-up)."""
    sink = torch.zeros(1, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream()
    best = None
    for it in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ops = rd.sfu_probe(4096, sink)
        e1.record(stream)
        torch.cuda.synchronize()
        if it:
            rate = ops / (e0.elapsed_time(e1) / 1e3)
            best = rate if best is None else max(best, rate)
    return best


def measure(workload, p, steps, warmup, world, rank, local, peaks, peak_kind, sfu_rate,
            min_region_ms=60.0, with_e2e=True, variant=None):
    """Times `steps` calls of the workload (regions of exactly `steps` calls, repeated back to
    back until the clock sampler has had at least `min_region_ms` to look at; the median region
    is reported) and returns the record with value, roofline, clocks, e2e and launch count."""
    import torch
    import paper_2410_06577_b200 as rd
    from paper_2410_06577_b200 import dist as rdist

    device = torch.device("cuda", local)
    decode = workload == "cfg3"
    tdt = torch.bfloat16 if p.dtype == "bf16" else torch.float32
    stream = torch.cuda.current_stream()

    def barrier():
        rdist.barrier()
        torch.cuda.synchronize()

    host = {n: torch.from_numpy(getattr(p, n)).to(tdt).pin_memory() for n in ("q", "k", "x", "y", "v")}
    devt = {n: host[n].to(device) for n in host}
    if decode:
        ring = p.q.shape[0]
        state = torch.from_numpy(p.state).to(device)
        Nseq, H, dk, dv = p.state.shape
        o = torch.empty((Nseq, H, dv), dtype=tdt, device=device)
        units_per_step = decode_bytes(p) / 1e9          # GB moved per step
        alg_bytes = decode_bytes(p)
        kernel = "ddts_step_kernel"
        token_heads = Nseq * H
        ws = None

        def step(i):
            s = i % ring
            rd.ddts_step(devt["q"][s], devt["k"][s], devt["x"][s], devt["y"][s], devt["v"][s], state, out=o)

        o_host = torch.empty(o.shape, dtype=tdt).pin_memory()
        h2d = sum(host[n][0].numel() * host[n].element_size() for n in host)
        d2h = o_host.numel() * o_host.element_size()
        stage = {n: torch.empty_like(devt[n][0]) for n in host}

        def step_e2e(i):
            s = i % ring
            for n in host:
                stage[n].copy_(host[n][s], non_blocking=True)
            rd.ddts_step(stage["q"], stage["k"], stage["x"], stage["y"], stage["v"], state, out=o)
            o_host.copy_(o, non_blocking=True)
    else:
        s0 = None if p.s0 is None else torch.from_numpy(p.s0).to(device)
        cu = None if p.cu_seqlens is None else torch.from_numpy(p.cu_seqlens).to(device)
        cu_host = None if p.cu_seqlens is None else torch.from_numpy(p.cu_seqlens)
        B, H, T, dk, dv = p.shape
        nseq = B if cu is None else cu.numel() - 1
        o = torch.empty((B, H, T, dv), dtype=tdt, device=device)
        sT = torch.empty((nseq, H, dk, dv), dtype=torch.float32, device=device)
        # variants of the same workload: "block" adds the value
        # gate and the feed-through (seeded, +2 tensors of v's shape read per call); "shared" keeps
        # one q,k,x,y per token for all heads (head 0's), the layout the paper writes the block in
        kw = {}
        alg_bytes = prefill_bytes(p)
        el = 2 if p.dtype == "bf16" else 4
        if variant == "block":
            g = torch.Generator(device="cpu").manual_seed(1234)
            kw = {"beta_hat": torch.rand(p.v.shape, generator=g).to(tdt).to(device),
                  "feed_x": torch.randn(p.v.shape, generator=g).to(tdt).to(device),
                  "feed_d": torch.randn((H, dv), generator=g).to(device)}
            alg_bytes += 2 * B * H * T * dv * el
        elif variant == "vdecay":
            from paper_2410_06577_b200 import workloads as wl_
            kw = {"value_decay": torch.from_numpy(wl_.make_value_decay(77, p.v.shape, p.dtype)).to(tdt).to(device)}
            alg_bytes += B * H * T * dv * el
        elif variant == "shared":
            for n in ("q", "k", "x", "y"):
                devt[n] = devt[n][:, :1].contiguous()
            alg_bytes -= (H - 1) * B * T * 4 * dk * el
        units_per_step = p.tokens
        token_heads = B * H * T
        if variant == "backward":
            # the backward pass of the same workload: seeded dL/do and dL/dS_T in, all six
            # gradients out; bytes = every input and every output once
            from paper_2410_06577_b200 import workloads as wl_
            g_o, g_s = wl_.make_grads(4321, p, True)
            g_o = torch.from_numpy(g_o).to(tdt).to(device)
            g_s = torch.from_numpy(g_s).to(device)
            grads = [torch.empty_like(devt["q"]) for _ in range(4)] + [torch.empty_like(devt["v"])]
            d_s0 = torch.empty_like(sT)
            bprm = rd.bwd_params(devt["q"], devt["k"], devt["x"], devt["y"], devt["v"], g_o, *grads,
                                 s0=s0, d_sT=g_s, d_s0=d_s0, cu_seqlens=cu, cu_seqlens_host=cu_host)
            ws = torch.empty(rd.bwd_workspace_bytes(bprm), dtype=torch.uint8, device=device)
            bprm.workspace, bprm.workspace_bytes = ws.data_ptr(), ws.numel()
            kernel = "ddts_bwd_sweep_kernel"
            alg_bytes = token_heads * (8 * dk + 3 * dv) * el + nseq * H * dk * dv * 4 * (2 + (s0 is not None))

            def step(i):
                rc = rd.bwd_raw(bprm)
                if rc != rd.OK:
                    raise SystemExit(f"rodimus_ddts_bwd: {rd.status_str(rc)}")
        else:
            prm = rd.fwd_params(devt["q"], devt["k"], devt["x"], devt["y"], devt["v"], o, s0, sT, cu, cu_host, **kw)
            ws = rd.new_workspace(prm, device)
            kernel = "ddts_fwd_" + rd.fwd_kernel_name(prm)

            def step(i):
                rd.ddts_fwd(devt["q"], devt["k"], devt["x"], devt["y"], devt["v"], s0, cu, cu_host,
                            out=o, final_state=sT, workspace=ws, **kw)

        o_host = torch.empty(o.shape, dtype=tdt).pin_memory()
        sT_host = torch.empty(sT.shape, dtype=torch.float32).pin_memory()
        h2d = sum(host[n].numel() * host[n].element_size() for n in host)
        d2h = o_host.numel() * o_host.element_size() + sT_host.numel() * 4

        def step_e2e(i):
            # the stage buffers ARE the resident inputs: every step overwrites them from the host
            for n in host:
                devt[n].copy_(host[n], non_blocking=True)
            rd.ddts_fwd(devt["q"], devt["k"], devt["x"], devt["y"], devt["v"], s0, cu, cu_host,
                        out=o, final_state=sT, workspace=ws)
            o_host.copy_(o, non_blocking=True)
            sT_host.copy_(sT, non_blocking=True)

    def timed_regions(fn, steps, warmup, min_ms):
        """Regions of exactly `steps` calls, event-bracketed, back to back; returns their times
        (ms, max over ranks each)."""
        for i in range(warmup):
            fn(i)
        barrier()
        times = []
        n = warmup
        total = 0.0
        while True:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for i in range(steps):
                fn(n + i)
            ev1.record(stream)
            barrier()
            t = rdist.max_over_ranks(ev0.elapsed_time(ev1), device)
            times.append(t)
            total += t
            n += steps
            if total >= min_ms or len(times) >= 200:
                return times

    step(0)
    torch.cuda.synchronize()
    launches_per_step = rd.last_launch_count()
    with ClockSampler(local) as clk:
        regions = timed_regions(step, steps, warmup, min_region_ms)
    clocks = clk.summary()
    if ws is not None:
        st = rd.device_status(ws)
        if st != rd.OK:
            raise SystemExit(f"device status after the timed region: {st} ({rd.status_str(st)})")
    ms = float(np.median(regions))
    sec = ms / 1e3
    value = units_per_step * world * steps / sec
    kern_s = sec / steps
    achieved = alg_bytes / kern_s / 1e9
    rec = {
        "metric": "DDTS decode state GB/s" if decode else "DDTS prefill tokens/s",
        "value": value, "unit": "GB/s" if decode else "tokens/s",
        "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32" if decode else ("bf16" if p.dtype == "bf16" else "f32"),
        "data": "synthetic (seeded)", "config": describe(workload, p, world),
        "timed_regions": {"count": len(regions), "steps_each": steps, "reported": "median",
                          "ms_min": float(min(regions)), "ms_median": ms, "ms_max": float(max(regions))},
        "clocks": clocks,
        "gpu_launches": int(launches_per_step * steps),
    }
    wk = work_per_token_head(128, 256)
    bounds = {"hbm_us": alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6}
    if variant == "backward":
        # five [chunk x dk x dv] contractions per chunk (two in the forward sweep, three in the two
        # reverse sweeps) on tf32 operands: measured bf16 peak x the nominal tf32/bf16 ratio
        tf32_peak = peaks["bf16_tflops"] * DATASHEET_TF32_RATIO
        bounds["tensor_us"] = token_heads * 10 * 128 * 256 / (tf32_peak * 1e12) * 1e6
        bounds["tensor_peak_tflops"] = tf32_peak
    elif not decode:
        bounds["tensor_us"] = token_heads * wk["tensor_flops"] / (peaks["bf16_tflops"] * 1e12) * 1e6
        bounds["sfu_us"] = (token_heads * wk["sfu_ops"] / sfu_rate * 1e6) if sfu_rate else "unmeasured"
        bounds["sfu_rate_gops"] = (sfu_rate / 1e9) if sfu_rate else "unmeasured"
    rec["roofline"] = {"bound": "hbm", "kernel": kernel, "achieved": achieved,
                       "peak": peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                       "frac": achieved / peaks["hbm_gbs"],
                       "frac_of_datasheet_peak": achieved / DATASHEET["hbm_gbs"],
                       "datasheet_peak": DATASHEET["hbm_gbs"],
                       "algorithmic_bytes_per_launch": int(alg_bytes),
                       "bound_times": bounds,
                       "traffic": load_traffic(kernel, f"{workload}_{variant}" if variant else workload)}
    if variant:
        rec["config"] = dict(rec["config"], variant={
            "block": "value gate beta_hat and feed-through d*x' fused (Eq. beta_def, Eq. rodimus_recurrent_form)",
            "shared": "one q,k,x,y per token for all 16 heads ([B,1,T,dk])",
            "backward": "backward pass (dq, dk, dx, dy, dv, ds0 from dL/do and dL/dS_T), two launches",
            "vdecay": "value-side decay beta_t of the general transition (the paper's ablation arm), fp32 CUDA-core kernel"}[variant])
        if variant == "backward":
            rec["metric"] = "DDTS prefill backward tokens/s"
    if with_e2e:
        e2e_steps = max(1, min(steps, 200 if decode else 5))
        e2e_regions = timed_regions(step_e2e, e2e_steps, 1, 0.0)
        rec["e2e"] = {"value": units_per_step * world * e2e_steps / (e2e_regions[0] / 1e3),
                      "unit": "GB/s" if decode else "tokens/s",
                      "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps}
    return rec


def measure_swska(steps, warmup, local, peaks, peak_kind, B=4, H=16, T=2048, d=128, window=1024):
    """Sub-record for the sliding-window shared-key attention on the layer shape (window = half the
    context, as the paper sets it): CUDA events around `steps` calls, tensor roofline against the
    measured bf16 rate.  Flops counted from the definition: 4 d per (query, visible key)."""
    import torch
    import paper_2410_06577_b200 as rd
    from paper_2410_06577_b200 import workloads as wl
    device = torch.device("cuda", local)
    # Three sets of inputs and outputs used in rotation: a call's 105 MB would otherwise still be
    # in L2 (126 MB) from the call before; with 315 MB in rotation every call reads from DRAM.
    n_sets = 3
    sets, prms = [], []
    for s_ in range(n_sets):
        q, k, v = (torch.from_numpy(a).to(torch.bfloat16).to(device) for a in wl.make_swska(31 + s_, B, H, T, d))
        o = torch.empty_like(q)
        sets.append((q, k, v, o))
        prms.append(rd.swska_params(q, k, v, o, window, d ** -0.5))
    stream = torch.cuda.current_stream()

    def region(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(n):
            rc = rd.swska_raw(prms[i % n_sets])
            if rc != rd.OK:
                raise SystemExit(f"rodimus_swska_fwd: {rd.status_str(rc)}")
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    region(warmup)
    with ClockSampler(local) as clk:
        times = [region(steps) for _ in range(5)]
    ms = float(np.median(times)) / steps
    pairs = sum(min(t + 1, window) for t in range(T))          # visible (query, key) pairs per head
    flops = 4.0 * d * pairs * B * H
    alg_bytes = (3 * B * H * T * d + B * T * d) * 2
    achieved = flops / (ms / 1e3) / 1e12
    return {
        "metric": "SW-SKA tokens/s", "value": B * T / (ms / 1e3), "unit": "tokens/s", "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "dtype": "bf16",
        "config": {"workload": f"SW-SKA B={B} H={H} T={T} d={d} window={window} bf16, one key per token for all heads",
                   "l2": "three input/output sets of 105 MB in rotation (315 MB > L2), no flush"},
        "timed_regions": {"count": len(times), "steps_each": steps, "reported": "median",
                          "ms_min": float(min(times)), "ms_median": float(np.median(times)),
                          "ms_max": float(max(times))},
        "clocks": clk.summary(), "gpu_launches": steps,
        "roofline": {"bound": "tensor", "kernel": "swska_fwd_tc_kernel", "achieved": achieved,
                     "peak": peaks["bf16_tflops"], "peak_kind": f"of {peak_kind} (burst)", "unit": "TFLOP/s",
                     "frac": achieved / peaks["bf16_tflops"], "algorithmic_flops_per_launch": flops,
                     "bound_times": {"tensor_us": flops / (peaks["bf16_tflops"] * 1e12) * 1e6,
                                     "hbm_us": alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6},
                     "traffic": load_traffic("swska_fwd_tc_kernel", "layer")},
    }


SUB_DEFAULTS = {"cfg1": (500, 5), "cfg2": (100, 5), "cfg4": (40, 5), "cfg3": (1000, 10)}


def run_ours(args, workload, p):
    import torch
    import torch.distributed as dist
    import paper_2410_06577_b200 as rd
    from paper_2410_06577_b200 import dist as rdist
    from paper_2410_06577_b200 import workloads as wl

    rank, world, local = rdist.env_rank()
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    rdist.init("nccl", device)
    peaks, peak_kind = load_peaks()
    sfu_rate = measure_sfu_rate(rd, torch, device)

    line = measure(workload, p, args.steps, args.warmup, world, rank, local, peaks, peak_kind, sfu_rate,
                   with_e2e=args.variant is None, variant=args.variant)
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.variant is None:
        from oracle import ddts_oracle as orc
        decode = workload == "cfg3"
        u, s, what = oracle_sample_run(workload, p, budget_s=10.0)
        line["cpu_baseline"] = {"value": u / s / (1e9 if decode else 1.0),
                                "unit": "GB/s" if decode else "tokens/s",
                                "cores": orc.num_threads(), "kind": "oracle", "sample": what}
    # The metric has a prefill half and a decode half, and the prefill bar holds on the long and
    # the packed workloads too: at one GPU the other named workloads ride along as sub-records,
    # each timed with its own step count (the top-level fields stay those of `workload`).
    if world == 1 and not args.no_extra:
        del p
        extra = {}
        for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
            if name == workload and args.steps >= SUB_DEFAULTS[name][0]:
                continue
            torch.cuda.empty_cache()
            pw = wl.config(WORKLOADS[name])
            k, w = SUB_DEFAULTS[name]
            r = measure(name, pw, k, w, world, rank, local, peaks, peak_kind, sfu_rate, with_e2e=False)
            extra[name] = {key: r[key] for key in ("metric", "value", "unit", "steps", "warmup", "ms_per_step",
                                                   "dtype", "config", "timed_regions", "clocks",
                                                   "gpu_launches", "roofline")}
            del pw
        for name, variant in (("cfg1_block_terms", "block"), ("cfg1_shared_gates", "shared"),
                              ("cfg1_backward", "backward"), ("cfg1_value_decay", "vdecay")):
            torch.cuda.empty_cache()
            pw = wl.config(1)
            r = measure("cfg1", pw, {"backward": 40, "vdecay": 10}.get(variant, 500), 5, world, rank, local, peaks,
                        peak_kind, sfu_rate, with_e2e=False, variant=variant)
            extra[name] = {key: r[key] for key in ("metric", "value", "unit", "steps", "warmup", "ms_per_step",
                                                   "dtype", "config", "timed_regions", "clocks",
                                                   "gpu_launches", "roofline")}
            del pw
        torch.cuda.empty_cache()
        extra["swska_layer"] = measure_swska(50, 5, local, peaks, peak_kind)
        line["workloads"] = extra
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="cfg1")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--swska", action="store_true",
                    help="time the sliding-window shared-key attention alone (for profiling)")
    ap.add_argument("--variant", choices=["block", "shared", "backward", "vdecay"], default=None,
                    help="time a variant of the config-1 workload instead (for profiling; no e2e)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="only the workload named by --workload, no sub-records for the others")
    args = ap.parse_args()
    decode = args.workload == "cfg3"
    if args.steps is None:
        args.steps = SUB_DEFAULTS[args.workload][0] if args.impl == "ours" else 3
    if args.warmup is None:
        args.warmup = (10 if decode else 20) if args.impl == "ours" else 1
    if args.impl == "ours" and args.warmup < 3:
        args.warmup = 3

    from paper_2410_06577_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if args.impl == "reference" and rank != 0:
        return
    if args.swska and args.impl == "ours":
        import torch
        torch.cuda.set_device(0)
        peaks, peak_kind = load_peaks()
        print(json.dumps(measure_swska(args.steps, args.warmup, 0, peaks, peak_kind)), flush=True)
        return
    p = wl.config(WORKLOADS[args.workload])
    if args.impl == "reference":
        run_reference(args, args.workload, p)
    else:
        run_ours(args, args.workload, p)


if __name__ == "__main__":
    main()
