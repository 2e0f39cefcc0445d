#!/usr/bin/env python
"""Benchmark of S2-Attn forward+backward on B200.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (this repository)
    python bench.py --impl reference --steps K --warmup W    # the CPU fp64 oracle, as it stands

A step is one forward + backward pass of the whole operator over one synthetic batch of the
workload (default: Llama2-7B attention shape, N=32768, G=8192, H=Hkv=32, d=128, bf16).  The metric
is TFLOP/s counting only the causal in-group FLOPs: 14 * d per attended (query, key) pair.
With more than one GPU every rank runs an independent replica (the operator has no exchange
step); the value is the sum over ranks divided by the slowest rank's time.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "S2-Attn fwd+bwd TFLOP/s (causal in-group FLOPs)"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "llama2_7b_32k"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}
# DRAM bytes (read + write) per launch, from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum) of each kernel on llama2_7b_8k.  The tensors q, k, v, o, dO, dq, dk, dv are
# each touched once, so that part scales with B*N*(H+Hkv)*d; the spilled dS (written by the dK/dV
# kernel, read by the dQ product kernel) is 2 bytes per entry of every 128 x 64 block and scales with
# the number of blocks.  An entry is None where the kernel has changed since its capture.
#   name: (bytes that scale with the tensors, bytes that scale with the spill) at 8k
NCU_TRAFFIC_8K = {
    "fwd": (249.6e6, 0.0),
    "bwd_preprocess": (137.9e6, 0.0),
    "bwd_dkdv": (373.3e6, 0.0),                     # 270.7 MB read + 102.6 MB written
    "bwd_dq": (322.8e6, 0.0),
    "bwd_dkdv_spill": (920.2e6 - 570.4e6, 570.4e6),  # 270.9 MB read + 649.3 MB written, 570.4 MB of it the spill
    "bwd_dq_spill": (695.9e6 - 570.4e6, 570.4e6),    # 637.6 MB read + 58.3 MB written
}
NCU_TRAFFIC_8K_SIZE = 1 * 8192 * (32 + 32) * 128
NCU_SPILL_8K_BLOCKS = 32 * 4 * 16 * 17             # units x T (T + 1) blocks of 16 KiB, T = 2048 / 128


def spill_blocks(w):
    T = w.G // 128 if w.G % 256 == 0 else (w.G + 127) // 128 + 1
    return w.B * w.H * (w.N // w.G) * T * (T + 1)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# clocks: sample nvidia-smi while the timed region runs
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None
        self.skip_bytes = 0

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="s2a_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
            return
        # nvidia-smi needs a moment before its first sample: wait for it (bounded), then forget
        # what was sampled while idle
        t0 = time.time()
        while time.time() - t0 < 5.0 and os.path.getsize(self.path) == 0:
            time.sleep(0.05)
        self.skip_bytes = os.path.getsize(self.path)

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            f.seek(self.skip_bytes)
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 8:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for n, val in zip(names, parts[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(power))
        return res


# ------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands (never tuned for this)
# ------------------------------------------------------------------------------------------------
# A sample is the tail of one (batch, KV head, group) unit: the query rows (of every query head of
# the KV head) and the key rows at in-group positions [G - n, G); n = G is the whole unit.
# FLOPs credited to a sample, so that a whole unit gets exactly 14 d per attended pair:
#   an o row: 4 d per pair it attends; a dq row: 10 d / 3 per pair; a (dk, dv) row: 20 d / 3 per
#   pair that attends it  (the 10 d of the backward split evenly over its three outputs).
def oracle_sample_rows(w, which: int, n: int):
    """Step 0 takes the shifted, wrapped last group of the last head, step 1 the first group of
    head 0, and so on alternating through heads."""
    H, G, N = w.H, w.G, w.N
    if which % 2 == 0:
        h = H - 1 - (which // 2) % (H // 2)
        g, s = N // G - 1, G // 2
    else:
        h = (which // 2) % (H // 2)
        g, s = 0, 0
    toks = [(g * G + p + s) % N for p in range(G - n, G)]
    rep = H // w.Hkv
    hk = h // rep
    q_rows = [(0, hq, t) for hq in range(hk * rep, (hk + 1) * rep) for t in toks]
    kv_rows = [(0, hk, t) for t in toks]
    return q_rows, kv_rows


def oracle_sample_flops(w, n: int) -> float:
    rep = w.H // w.Hkv
    pairs_q = n * w.G - n * (n - 1) // 2      # sum over positions p in [G-n, G) of (p + 1)
    pairs_kv = n * (n + 1) // 2               # sum over positions p' in [G-n, G) of (G - p')
    return rep * w.d * (4.0 * pairs_q + 10.0 / 3.0 * pairs_q + 20.0 / 3.0 * pairs_kv)


def oracle_run_sample(w, inputs, which: int, n: int, keep=None) -> float:
    """Times the oracle on one sample; with `keep` (a list) also hands back the rows it computed."""
    from oracle import s2a_oracle as orc

    q, k, v, dO = inputs
    q_rows, kv_rows = oracle_sample_rows(w, which, n)
    t0 = time.perf_counter()
    o_ref, lse_ref = orc.fwd(q, k, v, w.G, rows=q_rows)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, w.G, q_rows=q_rows, kv_rows=kv_rows)
    dt = time.perf_counter() - t0
    if keep is not None:
        keep.append((q_rows, kv_rows, o_ref, lse_ref, dq_ref, dk_ref, dv_ref))
    return dt


def time_oracle_steps(w, inputs, steps: int, warmup: int, n: int, keep=None):
    from oracle import s2a_oracle as orc

    times = []
    for it in range(warmup + steps):
        dt = oracle_run_sample(w, inputs, it, n, keep if it >= warmup else None)
        if it >= warmup:
            times.append(dt)
    total = sum(times)
    return oracle_sample_flops(w, n) * steps / total / 1e12, total / steps, orc.num_threads()


def parity_against_oracle(kept, gpu_out):
    """Element-by-element comparison of the units the oracle just computed with what the GPU holds.

    kept: [(q_rows, kv_rows, o, lse, dq, dk, dv)] from the oracle; gpu_out: the device tensors
    (o, lse, dq, dk, dv) of the last step.  Returns max abs errors of o and lse, and for each gradient
    the relative L2 error pooled over all compared rows and that of the worst single row (its norm
    floored at 5 % of the rms row norm of its unit)."""
    import numpy as np
    import torch

    o, lse, dq, dk, dv = gpu_out
    res = {"o_max_abs": 0.0, "lse_max_abs": 0.0, "rows_q": 0, "rows_kv": 0}
    pooled = {n: [0.0, 0.0] for n in ("dq", "dk", "dv")}
    worst = {n: 0.0 for n in ("dq", "dk", "dv")}
    for q_rows, kv_rows, o_ref, lse_ref, dq_ref, dk_ref, dv_ref in kept:
        qi = torch.tensor(q_rows, device=o.device)
        ki = torch.tensor(kv_rows, device=o.device)
        got = {
            "o": o[qi[:, 0], qi[:, 2], qi[:, 1]], "lse": lse[qi[:, 0], qi[:, 1], qi[:, 2]],
            "dq": dq[qi[:, 0], qi[:, 2], qi[:, 1]], "dk": dk[ki[:, 0], ki[:, 2], ki[:, 1]],
            "dv": dv[ki[:, 0], ki[:, 2], ki[:, 1]],
        }
        got = {n: x.double().cpu().numpy() for n, x in got.items()}
        res["o_max_abs"] = max(res["o_max_abs"], float(np.abs(got["o"] - o_ref).max()))
        res["lse_max_abs"] = max(res["lse_max_abs"], float(np.abs(got["lse"] - lse_ref).max()))
        res["rows_q"] += len(q_rows)
        res["rows_kv"] += len(kv_rows)
        for n, ref in (("dq", dq_ref), ("dk", dk_ref), ("dv", dv_ref)):
            diff2 = ((got[n] - ref) ** 2).sum(axis=-1)
            ref2 = (ref ** 2).sum(axis=-1)
            pooled[n][0] += float(diff2.sum())
            pooled[n][1] += float(ref2.sum())
            # a row's own norm, floored at 5 % of the rms row norm (the first row of a group has dq = 0 exactly)
            floor2 = 0.0025 * float(ref2.mean())
            worst[n] = max(worst[n], float(np.sqrt(diff2 / np.maximum(ref2, max(floor2, 1e-300))).max()))
    for n in ("dq", "dk", "dv"):
        res[f"{n}_rel_l2"] = (pooled[n][0] / max(pooled[n][1], 1e-300)) ** 0.5
        res[f"{n}_rel_l2_worst_row"] = worst[n]
    res["tolerance"] = {"o_max_abs": 2e-2, "grad_rel_l2": 1e-2}
    res["ok"] = bool(res["o_max_abs"] <= 2e-2 and max(res["dq_rel_l2"], res["dk_rel_l2"], res["dv_rel_l2"]) <= 1e-2)
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2309_12307_b200.inputs import WORKLOADS, make_workload_inputs

    w = WORKLOADS[args.workload]
    inputs = make_workload_inputs(w, seed=0)
    # size the per-step sample so that all warm-up and timed steps fit in about two minutes
    n_cal = min(64, w.G)
    t_cal = oracle_run_sample(w, inputs, 1, n_cal)
    rate = oracle_sample_flops(w, n_cal) / max(t_cal, 1e-6)           # credited FLOP/s, roughly constant
    budget = 120.0 / max(args.steps + args.warmup, 1)
    n = w.G
    while n > 64 and oracle_sample_flops(w, n) / rate > budget:
        n //= 2
    tflops, sec_per_step, cores = time_oracle_steps(w, inputs, args.steps, args.warmup, n)
    sample = (f"each step = oracle forward+backward of the query rows and key rows at the last {n} of {w.G} "
              f"in-group positions of one (batch, head, group) unit of {w.name}, fp64, OpenMP; FLOPs credited: "
              f"4d per pair of an o row, 10d/3 of a dq row, 20d/3 of a dk/dv row")
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "G": w.G, "H": w.H, "Hkv": w.Hkv, "d": w.d},
        "cpu_baseline": {"value": tflops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------------
# the CUDA library
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2309_12307_b200 import binding as s2a
    from paper_2309_12307_b200.inputs import WORKLOADS, make_workload_inputs
    from paper_2309_12307_b200.replicas import slowest_rank_ms, whole_job_rate

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the operator has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    s2a.load()

    w = WORKLOADS[args.workload]
    B, N, H, Hkv, d, G = w.B, w.N, w.H, w.Hkv, w.d, w.G
    host_in = make_workload_inputs(w, seed=0)                       # same bits on every rank (replicas)
    q, k, v, dO = (x.to(dev) for x in host_in)
    o = torch.empty_like(q)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    # Backward workspace: with room for the spilled dS of every KV head (--bwd-workspace fast, the
    # library's fastest path: dq is a plain product) or the minimum (dq recomputes the scores).
    ws_min = s2a.bwd_workspace_bytes(B, N, H, Hkv, d, G)
    ws_bytes = ws_min
    if args.bwd_workspace == "fast":
        ws_bytes = s2a.bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, int(args.workspace_budget_gib * 2**30))
    spilling = ws_bytes >= s2a.bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, 1 << 50) > ws_min
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step_plain():
        s2a.s2a_fwd(q, k, v, G, o=o, lse=lse, stream=stream)
        s2a.s2a_bwd(q, k, v, o, lse, dO, G, dq=dq, dk=dk, dv=dv, workspace=ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)   # the timing rules want at least three; the line reports what was run
    if warmup != args.warmup and rank == 0:
        print(f"bench.py: --warmup {args.warmup} raised to {warmup}", file=sys.stderr)
    for _ in range(warmup):
        step_plain()
    barrier()
    # host side of a step: time spent in the entry points (argument checks, tensor maps, launches),
    # nothing on the device waited for
    t0 = time.perf_counter()
    for _ in range(5):
        step_plain()
    host_us = (time.perf_counter() - t0) / 5 * 1e6
    barrier()
    rc, where = s2a.device_status()
    if rc != 0:
        raise RuntimeError(f"device status {rc} (wait code {where}) after warm-up")

    # ---- timed region: exactly K steps; the same four launches per step as s2a_fwd + s2a_bwd, with
    # events between them so that every kernel's duration is measured inside the region
    names = ["fwd", "bwd_preprocess", "bwd_dkdv", "bwd_dq"]
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K)]
    try:
        smi_index = int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank])
    except (KeyError, ValueError, IndexError):
        smi_index = local_rank
    sampler = ClockSampler(smi_index)
    barrier()
    if rank == 0:
        sampler.start()
    barrier()
    for i in range(K):
        ev[i][0].record(stream)
        s2a.s2a_fwd(q, k, v, G, o=o, lse=lse, stream=stream)
        ev[i][1].record(stream)
        for stage in range(3):
            s2a.s2a_bwd_stage(q, k, v, o, lse, dO, G, dq, dk, dv, ws, stage, stream=stream)
            ev[i][2 + stage].record(stream)
    end = torch.cuda.Event(enable_timing=True)
    end.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = ev[0][0].elapsed_time(end)
    step_ms = [ev[i][0].elapsed_time(ev[i + 1][0] if i + 1 < K else end) for i in range(K)]
    kernel_ms = {n: sum(ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(K)) for j, n in enumerate(names)}
    rc, where = s2a.device_status()
    if rc != 0:
        raise RuntimeError(f"device status {rc} (wait code {where}) in the timed region")

    total_ms_max = slowest_rank_ms(total_ms, dev)
    flops_step = w.flops_fwd_bwd
    value = world * flops_step * K / (total_ms_max * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point: pinned host inputs copied in, all outputs
    # copied back, every step
    pin = [x.pin_memory() for x in host_in]
    host_out = [torch.empty(o.shape, dtype=torch.bfloat16).pin_memory(),
                torch.empty(lse.shape, dtype=torch.float32).pin_memory(),
                torch.empty(dq.shape, dtype=torch.bfloat16).pin_memory(),
                torch.empty(dk.shape, dtype=torch.bfloat16).pin_memory(),
                torch.empty(dv.shape, dtype=torch.bfloat16).pin_memory()]
    dev_bufs = (q, k, v, dO, o, lse, dq, dk, dv)
    h2d = sum(x.numel() * x.element_size() for x in pin)
    d2h = sum(x.numel() * x.element_size() for x in host_out)
    Ke = max(3, min(K, 10))
    for _ in range(2):
        s2a.s2a_fwd_bwd_host(pin, host_out, dev_bufs, G, ws, stream=stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(Ke):
        s2a.s2a_fwd_bwd_host(pin, host_out, dev_bufs, G, ws, stream=stream)
    e1.record(stream)
    barrier()
    e2e_value = whole_job_rate(flops_step * Ke, e0.elapsed_time(e1), dev) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel (tensor-core bound: a dense contraction).  Algorithmic
    # FLOPs per launch: forward 4 d per pair; dK/dV kernel 8 d per pair (S, dP, dV, dK); dQ kernel
    # 2 d per pair (its recomputed S and dP are not counted); preprocess: none counted.
    peaks, peak_src = load_peaks()
    pairs = w.pairs
    alg_flops = {"fwd": 4 * d * pairs, "bwd_preprocess": 0, "bwd_dkdv": 8 * d * pairs, "bwd_dq": 2 * d * pairs}
    exe_flops = {"fwd": 4 * d * pairs, "bwd_preprocess": 0, "bwd_dkdv": 8 * d * pairs,
                 "bwd_dq": (2 if spilling else 6) * d * pairs}
    kernels = {}
    for n in names:
        ms = kernel_ms[n] / K
        kernels[n] = {"launches": K, "ms_per_launch": ms, "share": kernel_ms[n] / sum(kernel_ms.values()),
                      "algorithmic_tflops": alg_flops[n] / (ms * 1e-3) / 1e12 if ms > 0 else None,
                      "executed_tflops": exe_flops[n] / (ms * 1e-3) / 1e12 if ms > 0 else None}
    dom = max(names, key=lambda n: kernel_ms[n])
    peak_sustained = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    peak_burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    # Which measured peak this run is comparable with: the sustained one when the run itself was held
    # back by the power cap (the reason was active, or the SM clock sat well below its maximum),
    # the burst one when it ran at full clock throughout.
    regime = "sustained"
    if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        capped = "sw_power_cap" in clocks.get("reasons", []) or clocks["sm_mhz"] < 0.97 * clocks["sm_max_mhz"]
        regime = "sustained" if capped else "burst"
    peak = peak_sustained if regime == "sustained" else peak_burst
    achieved = kernels[dom]["algorithmic_tflops"]
    traffic = NCU_TRAFFIC_8K.get(dom + "_spill" if spilling and dom in ("bwd_dkdv", "bwd_dq") else dom)
    if traffic is not None:
        traffic = (traffic[0] * (B * N * (H + Hkv) * d) / NCU_TRAFFIC_8K_SIZE
                   + traffic[1] * spill_blocks(w) / NCU_SPILL_8K_BLOCKS)
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic, "traffic_unit": "bytes per launch (ncu on 8k, scaled)",
                "peak_source": f"{peak_src} bf16 {regime} (chosen from this run's clock record)",
                "frac_of_burst": achieved / peak_burst, "frac_of_sustained": achieved / peak_sustained,
                "peaks": {"burst": peak_burst, "sustained": peak_sustained},
                "whole_step_frac": value / world / peak,
                "whole_step_frac_of_burst": value / world / peak_burst,
                "whole_step_frac_of_sustained": value / world / peak_sustained}

    cpu_baseline = None
    parity = None
    if world == 1 and not args.no_cpu_baseline:
        kept = []
        tf, sec, cores = time_oracle_steps(w, host_in, steps=2, warmup=0, n=w.G, keep=kept)
        cpu_baseline = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"2 whole (batch, head, group) units of {w.name} (the shifted wrapped last group "
                                  f"of head {H - 1}, the first group of head 0), forward+backward, {sec:.1f} s each"}
        # the same two units, every row of them, against the device path (the host-buffer entry point
        # above used the device tensors, inputs included, as staging space: restore the inputs and run
        # one more plain step)
        for dst, src in zip((q, k, v, dO), host_in):
            dst.copy_(src)
        step_plain()
        torch.cuda.synchronize()
        parity = parity_against_oracle(kept, (o, lse, dq, dk, dv))
        parity["sample"] = "every query row and key row of the two units of cpu_baseline"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": warmup,
        "ms_per_step": total_ms_max / K, "ms_per_step_median": statistics.median(step_ms), "ms_per_step_best": min(step_ms),
        "host_enqueue_us_per_step": host_us, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": B, "N": N, "G": G, "H": H, "Hkv": Hkv, "d": d,
                   "l2": "inputs (5 x %.0f MB) larger than L2" % (q.numel() * 2 / 1e6),
                   "bwd_workspace_bytes": ws_bytes,
                   "bwd_dq": "product with spilled dS" if spilling else "recomputes S and dP",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "tokens_per_s": world * B * N * K / (total_ms_max * 1e-3),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke},
        "gpu_launches": 4 * K,
        "roofline": roofline,
        "kernels": kernels,
        "cpu_baseline": cpu_baseline,
        "parity": parity,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--bwd-workspace", choices=["fast", "min"], default="fast",
                    help="backward workspace: room for the spilled dS of all KV heads (fast) or the minimum")
    ap.add_argument("--workspace-budget-gib", type=float, default=24.0)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args)
    return run_ours(args)


def launch_ranks(args):
    """`python bench.py --gpus N` without a launcher around it: start N ranks, one GPU each, under
    torch.distributed.run on this node and let rank 0's JSON line through."""
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


if __name__ == "__main__":
    sys.exit(main())
