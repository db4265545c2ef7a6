#!/usr/bin/env python
"""Benchmark of the multi-scale linear attention module forward on B200.

A step is one whole-module forward (QKV projection, 5x5 aggregation, KV-state
reduction, apply, output projection; the last two as one kernel where the
library fuses them) on one seeded synthetic feature map.
Prints one JSON line (rank 0): `value` is tokens/s of the whole job from CUDA
events around the timed steps, `stages` the per-step times and algorithmic
HBM rates from events recorded between the steps, `roofline` the slowest
step against the measured HBM copy rate, `attention_core` the stand-alone
core entry point at the workload's head and token counts, `e2e` the same
metric with pinned host buffers and the copies inside the timed region,
`cpu_baseline` the fp64 oracle on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2205_14756_b200 import inputs  # noqa: E402

METRIC = "msla_fwd_tokens_per_s"
UNIT = "tokens/s"
STAGES = ("project_in", "aggregate", "kv_state", "apply", "project_out")
# when the library runs steps 4 and 5 as one kernel (msla_forward_fuses_apply), they are one stage
STAGES_FUSED = ("project_in", "aggregate", "kv_state", "apply_project")
FALLBACK_HBM_GBS = 6650.0


def workload_by_name(name: str) -> inputs.ModuleShape:
    table = {s.name: s for s in (inputs.CONFIG1, inputs.CONFIG3, inputs.CONFIG4) + inputs.CONFIG5}
    return table[name]


def stage_bytes_per_token(s: inputs.ModuleShape) -> dict:
    """Algorithmic HBM bytes per token of each step (materialised intermediates)."""
    e = 4 if s.dtype == "f32" else 2
    C, Cp, Co = s.C, s.Cp, s.C_out
    return {
        "project_in": (C + 3 * Cp) * e,
        "aggregate": (3 * Cp + 3 * Cp) * e,
        "kv_state": 2 * 2 * Cp * e,              # K and V of both scales
        "apply": (2 * Cp + 2 * Cp) * e,          # Q of both scales in, attention out
        "project_out": (2 * Cp + Co) * e,
        "apply_project": (2 * Cp + Co) * e,      # fused: Q of both scales in, y out; the head concat stays on chip
    }


def stage_flops_per_token(s: inputs.ModuleShape) -> dict:
    C, Cp, Co, d = s.C, s.Cp, s.C_out, s.d
    return {
        "project_in": 2 * 3 * Cp * C,
        "aggregate": 2 * (25 * 3 * Cp + 3 * Cp * d),
        "kv_state": 2 * 2 * Cp * (d + 1),
        "apply": 2 * 2 * Cp * (d + 1),
        "project_out": 2 * 2 * Cp * Co,
        "apply_project": 2 * 2 * Cp * (d + 1) + 2 * 2 * Cp * Co,
    }


def measured_peaks() -> tuple:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2205_14756_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(stage: str, workload: str):
    """DRAM bytes per launch from the committed ncu capture, or None when the
    kernels changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None
    try:
        rec = json.load(open(p))
        if rec.get("csrc_hash") != kernel_source_hash():
            return None
        return rec.get("bytes_per_launch", {}).get(workload, {}).get(stage)
    except Exception:
        return None


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, smax, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def rank_shape(s: inputs.ModuleShape, rank: int) -> inputs.ModuleShape:
    """Weak scaling: every rank runs the same-shaped module on its own image (own seed)."""
    return inputs.ModuleShape(s.name, s.dtype, s.B, s.C, s.H, s.W, s.heads, s.d, seed=s.seed + 1000 * rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of per-rank timings over the process group (identity on one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    buf = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(buf, op=dist.ReduceOp.MAX)
    return buf.tolist()


def whole_job_value(tokens_per_rank_step: int, world: int, ms_total_max: float, steps: int) -> float:
    """Tokens per second of the whole job: all ranks' tokens over the slowest rank's time."""
    return tokens_per_rank_step * world / (ms_total_max * 1e-3 / steps)


def oracle_sample_shape(s: inputs.ModuleShape, side: int) -> inputs.ModuleShape:
    return inputs.ModuleShape(f"{s.name}_sample{side}", s.dtype, 1, s.C, min(side, s.H), min(side, s.W), s.heads, s.d,
                              seed=s.seed)


def time_oracle(s: inputs.ModuleShape, side: int, repeats: int = 1) -> tuple:
    """Oracle as it stands on a bounded sample of the workload: a crop of the
    token grid with the same channels, heads and weights shapes."""
    import oracle
    ss = oracle_sample_shape(s, side)
    t = inputs.module_inputs(ss)
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=ss.heads, d=ss.d, eps=ss.eps)
        best = min(best, time.perf_counter() - t0)
    return ss.B * ss.N / best, best, ss, oracle.num_threads()


def run_reference(args, s: inputs.ModuleShape, rank: int) -> None:
    if rank != 0:
        return
    import oracle
    # size the per-step sample so that the whole run stays within a few minutes
    _, t32, _, cores = time_oracle(s, 32)
    side = 32
    for cand in (64, 128, 256):
        if t32 * (cand / 32) ** 2 * (args.steps + args.warmup) <= 150.0 and cand <= max(s.H, s.W):
            side = cand
    ss = oracle_sample_shape(s, side)
    t = inputs.module_inputs(ss)
    call = lambda: oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=ss.heads, d=ss.d, eps=ss.eps)
    for _ in range(args.warmup):
        call()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        call()
    dt = (time.perf_counter() - t0) / args.steps
    value = ss.B * ss.N / dt
    sample = f"{ss.H}x{ss.W} crop of the token grid per step (same C, heads, d), fp64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": s.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=inputs.CONFIG5[-1].name)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    s = workload_by_name(args.workload)

    if args.impl == "reference":
        run_reference(args, s, rank)
        return

    import torch
    import torch.distributed as dist
    import __graft_entry__  # noqa: F401  builds libmsla.so if needed
    from paper_2205_14756_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # every rank runs the same-shaped module on its own image (weak scaling, no collective on the data path)
    shape = rank_shape(s, rank)
    t = inputs.module_inputs(shape)
    tdt = torch.float32 if s.dtype == "f32" else torch.bfloat16
    code = binding.MSLA_F32 if s.dtype == "f32" else binding.MSLA_BF16
    host_x = torch.from_numpy(t["x"]).to(tdt).contiguous().pin_memory()
    x = host_x.to("cuda")
    wt = [torch.from_numpy(t[n]).to("cuda").to(tdt).contiguous() for n in ("w_qkv", "w_dw", "w_pw", "w_proj")]
    weights = binding.make_weights(*wt)
    out = torch.empty(s.B, s.C_out, s.H, s.W, dtype=tdt, device="cuda")
    host_out = torch.empty(s.B, s.C_out, s.H, s.W, dtype=tdt).pin_memory()
    d0 = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, code, s.eps)
    ws = torch.empty(binding.msla_forward_host_workspace_bytes(d0), dtype=torch.uint8, device="cuda")
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, code, s.eps, workspace=ws)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K, W = args.steps, args.warmup
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(K)]
    for row in evs:
        for e in row:
            e.record(stream)        # creates the underlying cudaEvent_t
    for _ in range(W):
        binding.msla_forward_profiled(desc, x, weights, out, stream, evs[0])
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    launches0 = binding.msla_kernel_launches()
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev_a.record(stream)
    for i in range(K):
        binding.msla_forward_profiled(desc, x, weights, out, stream, evs[i])
    ev_b.record(stream)
    barrier()
    launches = binding.msla_kernel_launches() - launches0
    ms_total = ev_a.elapsed_time(ev_b)

    # The same K steps through msla_forward, i.e. without the event records between the steps,
    # which lets each kernel's set-up overlap its predecessor's tail.  Reported beside the
    # headline, not as the headline: the per-step durations above come from the profiled loop.
    p_a, p_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p_a.record(stream)
    for _ in range(K):
        binding.msla_forward(desc, x, weights, out, stream)
    p_b.record(stream)
    barrier()
    ms_plain = p_a.elapsed_time(p_b)

    # end to end: pinned host input -> device -> five steps -> host result, every step.
    # (a) one stream: the latency of a single call; (b) three calls in flight on three
    # streams, each with its own workspace and pinned buffers, so that the PCIe copies of
    # one step overlap the kernels of another (the throughput a serving loop would see).
    for _ in range(2):
        binding.msla_forward_host(desc, host_x, weights, host_out, stream)
    barrier()
    e_a, e_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_a.record(stream)
    for _ in range(K):
        binding.msla_forward_host(desc, host_x, weights, host_out, stream)
    e_b.record(stream)
    barrier()
    ms_e2e_serial = e_a.elapsed_time(e_b)

    PIPE = 3
    lanes = []
    for i in range(PIPE):
        st_i = torch.cuda.Stream()
        ws_i = ws if i == 0 else torch.empty_like(ws)
        hx_i = host_x if i == 0 else host_x.clone().pin_memory()
        ho_i = host_out if i == 0 else torch.empty_like(host_out).pin_memory()
        d_i = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, code, s.eps, workspace=ws_i)
        lanes.append((st_i, d_i, hx_i, ho_i, ws_i))
    for st_i, d_i, hx_i, ho_i, _ in lanes:          # warm-up of every lane
        binding.msla_forward_host(d_i, hx_i, weights, ho_i, st_i)
    barrier()
    e_a, e_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_a.record(stream)
    for st_i, *_ in lanes:
        st_i.wait_event(e_a)
    for k in range(K):
        st_i, d_i, hx_i, ho_i, _ = lanes[k % PIPE]
        binding.msla_forward_host(d_i, hx_i, weights, ho_i, st_i)
    for st_i, *_ in lanes:
        done = torch.cuda.Event()
        done.record(st_i)
        stream.wait_event(done)
    e_b.record(stream)
    barrier()
    ms_e2e = e_a.elapsed_time(e_b)
    clocks = sampler.stop() if rank == 0 else None
    del lanes

    # The attention core (steps 3 + 4) on its own entry point, at this workload's head and token counts:
    # in the fused module the apply step has no kernel of its own to time.
    core = None
    if s.dtype == "bf16" and rank == 0:
        cB, cH, cN, cd = s.B, 2 * s.heads, s.N, s.d
        q, k, v = (torch.randn(cB, cH, cN, cd, device="cuda").to(tdt) for _ in range(3))
        o = torch.empty_like(q)
        nb = binding.msla_linattn_relu_workspace_bytes(cB, cH, cN, cd)
        cws = torch.empty(nb, dtype=torch.uint8, device="cuda")
        for _ in range(3):
            binding.msla_linattn_relu_ws(code, q, k, v, o, cB, cH, cN, cd, s.eps, cws, nb)
        c_a, c_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c_a.record(stream)
        for _ in range(K):
            binding.msla_linattn_relu_ws(code, q, k, v, o, cB, cH, cN, cd, s.eps, cws, nb)
        c_b.record(stream)
        torch.cuda.synchronize()
        core = (c_a.elapsed_time(c_b) / K, 4 * cB * cH * cN * cd * 2)
        del q, k, v, o, cws

    ms_total, ms_e2e, ms_e2e_serial, ms_plain = max_over_ranks([ms_total, ms_e2e, ms_e2e_serial, ms_plain], device="cuda")

    if rank == 0:
        fused = binding.msla_forward_fuses_apply(desc) == 1
        stage_names = STAGES_FUSED if fused else STAGES
        stage_ms = {}
        for j, name in enumerate(STAGES):
            stage_ms[name] = statistics.mean(evs[i][j].elapsed_time(evs[i][j + 1]) for i in range(K))
        if fused:  # the event between steps 4 and 5 falls directly after the one that ends step 3
            stage_ms["apply_project"] = stage_ms.pop("apply") + stage_ms.pop("project_out")
        bpt, fpt = stage_bytes_per_token(s), stage_flops_per_token(s)
        peak, peak_kind = measured_peaks()
        stages = {}
        for name in stage_names:
            sec = stage_ms[name] * 1e-3
            stages[name] = {"ms": round(stage_ms[name], 5),
                            "GBps": round(bpt[name] * s.B * s.N / sec / 1e9, 1),
                            "frac_of_%s_hbm" % peak_kind: round(bpt[name] * s.B * s.N / sec / 1e9 / peak, 4),
                            "frac_of_8TBps": round(bpt[name] * s.B * s.N / sec / 8e12, 4),
                            "TFLOPps": round(fpt[name] * s.B * s.N / sec / 1e12, 2)}
        dom = max(stage_names, key=lambda n: stage_ms[n])
        achieved = bpt[dom] * s.B * s.N / (stage_ms[dom] * 1e-3) / 1e9
        if core is not None:
            core_ms, core_how = core[0], "stand-alone core entry (msla_linattn_relu_ws) on [B, 2*heads, N, d] of this workload"
            core_gbps = core[1] / (core_ms * 1e-3) / 1e9
        else:
            core_ms, core_how = stage_ms["kv_state"] + stage_ms["apply"], "steps 3 + 4 inside the module"
            core_gbps = (bpt["kv_state"] + bpt["apply"]) * s.B * s.N / (core_ms * 1e-3) / 1e9
        module_bytes = sum(bpt[n] for n in stage_names) * s.B * s.N
        e = 4 if s.dtype == "f32" else 2
        roofline = {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                    "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}",
                    "traffic": recorded_traffic(dom, s.name),
                    "algorithmic_bytes_per_launch": bpt[dom] * s.B * s.N}
        if dom == "aggregate":
            # HBM is the roof this step is judged against.  What limits the kernel as built is the shared-memory
            # pipe (the staged tile is turned to channel-planar there, then read as MMA operands: about 65 % busy)
            # together with the issue rate of mma.sync (112 warp-level MMAs per 8x8 pixel block).
            roofline["limiter"] = "shared-memory pipe (tile transposition + ldmatrix operand loads) and mma.sync issue rate"
        result = {
            "metric": METRIC, "value": whole_job_value(s.B * s.N, world, ms_total, K), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": s.name, "B": s.B, "C": s.C, "H": s.H, "W": s.W, "heads_per_scale": s.heads, "d": s.d,
                       "tokens_per_step_per_gpu": s.B * s.N, "accumulate": "f32",
                       "l2": "inputs and intermediates of one step exceed the 126 MB L2" if
                       module_bytes > 4 * 126e6 else "working set fits L2: numbers are L2-resident",
                       "steps_4_5_fused": fused,
                       "parallelism": f"replicas x{world}, one image per GPU, no collective"},
            "e2e": {"value": whole_job_value(s.B * s.N, world, ms_e2e, K), "unit": UNIT,
                    "h2d_bytes_per_step": s.B * s.C * s.N * e, "d2h_bytes_per_step": s.B * s.C_out * s.N * e,
                    "ms_per_step": ms_e2e / K, "calls_in_flight": 3,
                    "single_stream_ms_per_step": ms_e2e_serial / K},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "attention_core": {"how": core_how, "ms": round(core_ms, 5), "GBps": round(core_gbps, 1),
                               "frac_of_%s_hbm" % peak_kind: round(core_gbps / peak, 4),
                               "frac_of_8TBps": round(core_gbps / 8000.0, 4)},
            "stages": stages,
            "ms_per_step_without_stage_events": round(ms_plain / K, 5),
            "module_GBps": round(module_bytes / (ms_total * 1e-3 / K) / 1e9, 1),
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            side = 512 if max(s.H, s.W) >= 512 else max(s.H, s.W)
            v, sec, ss, cores = time_oracle(s, side)
            result["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                      "sample": f"{ss.H}x{ss.W} crop of the token grid (same C, heads, d), one pass, "
                                                f"{sec:.1f} s, fp64 oracle as it stands"}
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
