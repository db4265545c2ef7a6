#!/usr/bin/env python
"""Benchmark of the multi-scale linear attention module forward on B200.

A step is one whole-module forward (QKV projection, 5x5 aggregation, KV-state
reduction, apply, output projection; the last two as one kernel where the
library fuses them) on one seeded synthetic feature map.
Prints one JSON line (rank 0).  The timed region is BLOCKS blocks of `--steps`
forwards, each block bracketed by CUDA events: `ms_per_step` is the median
block (`ms_per_step_min/max` the fastest and slowest), `value` tokens/s of the
whole job from it; `stages` the per-step times and algorithmic HBM rates from
events recorded between the steps, `roofline` the slowest step against the
measured HBM copy rate, `attention_core` the stand-alone core entry point at
the workload's head and token counts, `e2e` the same metric with pinned host
buffers and the copies inside the timed region, `configs` the other
configurations (attention core alone, the two feature-map shapes, the
resolution sweep with its linear fit), `cpu_baseline` the oracle's source
instantiated in fp32 at -O3 on the host cores.

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
BLOCKS = 7           # timed blocks of --steps forwards; the median block is reported


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


# Sources that decide each stage's kernels: the recorded DRAM traffic of a stage stays valid while these are unchanged.
STAGE_SOURCES = {
    "project_in": ["gemm_tcgen05.cu", "tcgen05_util.cuh", "tma_host.h", "msla_common.cuh"],
    "aggregate": ["agg_bf16.cu", "tma_host.h", "msla_common.cuh"],
    "kv_state": ["core_bf16.cu", "msla_common.cuh"],
    "apply_project": ["fused_out.cu", "tcgen05_util.cuh", "tma_host.h", "msla_common.cuh"],
}


def kernel_source_hash(stage: str) -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2205_14756_b200", "csrc")
    for f in STAGE_SOURCES[stage]:
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(stage: str, workload: str):
    """DRAM bytes per launch of the stage's kernels from the committed ncu capture, or None when the
    stage's sources changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None
    try:
        rec = json.load(open(p)).get("bytes_per_launch", {}).get(workload, {}).get(stage)
        if not rec or rec.get("source_hash") != kernel_source_hash(stage):
            return None
        return rec.get("bytes")
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


def _oracle_f32_lib():
    """The oracle's own source file, unchanged, compiled a second time with every `double` read as `float` at
    -O3 -march=native: the fp32 instantiation the CPU baseline is quoted on.  A three-line wrapper includes the
    system headers first (their `long double` declarations must not see the macro), defines it, and includes the
    source."""
    import ctypes
    import tempfile
    src = os.path.join(ROOT, "oracle", "msla_oracle.c")
    tag = f"{os.getuid()}_{int(os.path.getmtime(src))}"
    out = os.path.join(tempfile.gettempdir(), f"libmsla_oracle_f32_{tag}.so")
    if not os.path.exists(out):
        wrap = os.path.join(tempfile.gettempdir(), f"msla_oracle_f32_{tag}_{os.getpid()}.c")
        with open(wrap, "w") as f:
            f.write('#include <stddef.h>\n#include <stdlib.h>\n#include <string.h>\n#if defined(_OPENMP)\n#include <omp.h>\n#endif\n'
                    f'#define double float\n#include "{src}"\n')
        tmp = out + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O3", "-march=native", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, wrap, "-lm"], check=True)
        os.replace(tmp, out)
        os.remove(wrap)
    lib = ctypes.CDLL(out)
    fp = ctypes.POINTER(ctypes.c_float)
    lib.oracle_msla_forward.argtypes = [fp] * 7 + [ctypes.c_int] * 8 + [ctypes.c_float]
    lib.oracle_msla_forward.restype = ctypes.c_int
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
    return lib, fp


def time_oracle_f32(s: inputs.ModuleShape, side: int, threads: int, repeats: int = 3) -> tuple:
    """Best of `repeats` runs of the fp32 instantiation on a side x side crop of the token grid with `threads`
    threads (0 = all).  Returns (tokens/s, seconds, threads used)."""
    lib, fp = _oracle_f32_lib()
    ss = oracle_sample_shape(s, side)
    t = inputs.module_inputs(ss)
    a = {k: np.ascontiguousarray(v, dtype=np.float32) for k, v in t.items()}
    out = np.empty((ss.B, ss.C_out, ss.H, ss.W), dtype=np.float32)
    all_threads = lib.oracle_num_threads()
    lib.oracle_set_num_threads(threads if threads > 0 else all_threads)
    used = lib.oracle_num_threads()
    best = float("inf")
    p = lambda v: v.ctypes.data_as(fp)
    for _ in range(repeats):
        t0 = time.perf_counter()
        rc = lib.oracle_msla_forward(p(a["x"]), p(a["w_qkv"]), p(a["w_dw"]), p(a["w_pw"]), p(a["w_proj"]), None, p(out),
                                     ss.B, ss.C, ss.H, ss.W, ss.heads, ss.d, 5, ss.C_out, ss.eps)
        best = min(best, time.perf_counter() - t0)
        assert rc == 0
    lib.oracle_set_num_threads(all_threads)
    return ss.B * ss.N / best, best, used


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


def time_token_sharded(s: inputs.ModuleShape, rank: int, world: int, steps: int, warmup: int, blocks: int = BLOCKS):
    """ms per forward (each block's, max over ranks) of ONE image of shape `s` cut into `world` bands of rows:
    halo exchange, steps 1-3 on the band, all-gather of the states, steps 4-5 on the band."""
    import torch
    import torch.distributed as dist
    from paper_2205_14756_b200 import sharded
    t = inputs.module_inputs(s)                       # the same image on every rank; each keeps its own rows
    tdt = torch.float32 if s.dtype == "f32" else torch.bfloat16
    r0, r1 = sharded.band_rows(s.H, world, rank)
    x_band = torch.from_numpy(np.ascontiguousarray(t["x"][:, :, r0:r1])).to("cuda").to(tdt)
    wt = [torch.from_numpy(t[n]).to("cuda").to(tdt).contiguous() for n in ("w_qkv", "w_dw", "w_pw", "w_proj")]
    comp = sharded.CudaBandCompute(*wt, heads=s.heads, d=s.d, eps=s.eps)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(warmup, 3)):
        sharded.sharded_forward(comp, x_band, rank, world)
    barrier()
    res = []
    for _ in range(blocks):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record(stream)
        for _ in range(steps):
            sharded.sharded_forward(comp, x_band, rank, world)
        b.record(stream)
        barrier()
        res.append(a.elapsed_time(b) / steps)
    return max_over_ranks(res, device="cuda")


def run_token_sharded(args, s: inputs.ModuleShape, rank: int, world: int) -> None:
    """`--shard tokens`: strong scaling of one image over the ranks."""
    import torch
    from paper_2205_14756_b200 import binding
    sampler = ClockSampler(torch.cuda.current_device())
    if rank == 0:
        sampler.start()
    ms = time_token_sharded(s, rank, world, args.steps, args.warmup)
    clocks = sampler.stop() if rank == 0 else None
    timeouts = binding.msla_debug_wait_timeouts()
    if timeouts != 0:
        raise SystemExit(f"a bounded wait inside a kernel ran out on rank {rank} (flag {timeouts})")
    if rank != 0:
        return
    m = statistics.median(ms)
    print(json.dumps({
        "metric": METRIC, "value": s.B * s.N / (m * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": m, "ms_per_step_min": min(ms), "ms_per_step_max": max(ms), "timed_blocks": len(ms), "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": s.name, "B": s.B, "C": s.C, "H": s.H, "W": s.W, "heads_per_scale": s.heads, "d": s.d,
                   "tokens_per_step": s.B * s.N,
                   "parallelism": f"one image in {world} bands of rows; per forward: halo rows of x by send/recv, one all-gather of "
                                  f"{s.B * 2 * s.heads * s.d * (s.d + 1) * 4} bytes of partial states per rank, summed in band order"},
        "clocks": clocks}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=inputs.CONFIG5[-1].name)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the other configurations (the `configs` key)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "tokens"],
                    help="N > 1: one image per GPU (weak scaling, the default), or ONE image cut into bands of rows over the GPUs "
                         "(strong scaling: halo rows by send/recv, one all-gather of the partial states)")
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

    if args.shard == "tokens":
        run_token_sharded(args, s, rank, world)
        return

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

    def timed_blocks(call, blocks=BLOCKS, steps=K):
        """ms of each of `blocks` blocks of `steps` calls (CUDA events on the launching stream around each block)."""
        res = []
        for _ in range(blocks):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(steps):
                call(i)
            b.record(stream)
            barrier()
            res.append(a.elapsed_time(b))
        return res

    # Headline: BLOCKS blocks of K forwards with the events between the steps.
    launches0 = binding.msla_kernel_launches()
    stage_acc = {name: [] for name in STAGES}

    def profiled(i):
        binding.msla_forward_profiled(desc, x, weights, out, stream, evs[i])

    ms_blocks = []
    for _ in range(BLOCKS):
        ms_blocks += timed_blocks(profiled, blocks=1)
        for j, name in enumerate(STAGES):
            stage_acc[name] += [evs[i][j].elapsed_time(evs[i][j + 1]) for i in range(K)]
    launches = (binding.msla_kernel_launches() - launches0) // BLOCKS   # per block of K steps

    # The same through msla_forward, i.e. without the event records between the steps, which lets each
    # kernel's set-up overlap its predecessor's tail.  Reported beside the headline, not as the headline.
    ms_plain_blocks = timed_blocks(lambda i: binding.msla_forward(desc, x, weights, out, stream))

    # end to end: pinned host input -> device -> five steps -> host result, every step.
    # (a) one stream: the latency of a single call; (b) three calls in flight on three
    # streams, each with its own workspace and pinned buffers, so that the PCIe copies of
    # one step overlap the kernels of another (the throughput a serving loop would see).
    for _ in range(2):
        binding.msla_forward_host(desc, host_x, weights, host_out, stream)
    barrier()
    ms_e2e_serial_blocks = timed_blocks(lambda i: binding.msla_forward_host(desc, host_x, weights, host_out, stream), blocks=3)

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
    ms_e2e_blocks = []
    for _ in range(3):
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
        ms_e2e_blocks.append(e_a.elapsed_time(e_b))
    clocks = sampler.stop() if rank == 0 else None
    del lanes

    med = statistics.median

    def time_core(cs: inputs.CoreShape, blocks=BLOCKS, steps=K):
        """Stand-alone attention core (steps 3 + 4) on seeded q, k, v: (median ms per call, min, max, bytes)."""
        ct = inputs.core_inputs(cs)
        cdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[cs.dtype]
        ccode = {"f32": binding.MSLA_F32, "bf16": binding.MSLA_BF16, "f16": binding.MSLA_F16}[cs.dtype]
        q, k, v = (torch.from_numpy(ct[n]).to("cuda").to(cdt).contiguous() for n in ("q", "k", "v"))
        o = torch.empty_like(q)
        nb = binding.msla_linattn_relu_workspace_bytes(cs.B, cs.heads, cs.N, cs.d)
        cws = torch.empty(nb, dtype=torch.uint8, device="cuda")
        call = lambda i: binding.msla_linattn_relu_ws(ccode, q, k, v, o, cs.B, cs.heads, cs.N, cs.d, cs.eps, cws, nb)
        for i in range(3):
            call(i)
        ms = [m / steps for m in timed_blocks(call, blocks=blocks, steps=steps)]
        return med(ms), min(ms), max(ms), 4 * q.numel() * q.element_size()

    # The attention core on its own entry point, at this workload's head and token counts:
    # in the fused module the apply step has no kernel of its own to time.
    core = None
    if s.dtype == "bf16" and rank == 0:
        core = time_core(inputs.CoreShape("core_of_workload", "bf16", s.B, 2 * s.heads, s.N, s.d, seed=s.seed))

    def time_module(ms_shape: inputs.ModuleShape, blocks=5, steps=10):
        """Plain msla_forward on another configuration: dict with ms per step, tokens/s and module GB/s."""
        mt = inputs.module_inputs(ms_shape)
        mdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[ms_shape.dtype]
        mcode = {"f32": binding.MSLA_F32, "bf16": binding.MSLA_BF16, "f16": binding.MSLA_F16}[ms_shape.dtype]
        mx = torch.from_numpy(mt["x"]).to("cuda").to(mdt).contiguous()
        mw = [torch.from_numpy(mt[n]).to("cuda").to(mdt).contiguous() for n in ("w_qkv", "w_dw", "w_pw", "w_proj")]
        mweights = binding.make_weights(*mw)
        mo = torch.empty(ms_shape.B, ms_shape.C_out, ms_shape.H, ms_shape.W, dtype=mdt, device="cuda")
        md0 = binding.make_desc(ms_shape.B, ms_shape.C, ms_shape.H, ms_shape.W, ms_shape.heads, ms_shape.d, ms_shape.C_out, mcode, ms_shape.eps)
        mws = torch.empty(binding.msla_forward_workspace_bytes(md0), dtype=torch.uint8, device="cuda")
        mdesc = binding.make_desc(ms_shape.B, ms_shape.C, ms_shape.H, ms_shape.W, ms_shape.heads, ms_shape.d, ms_shape.C_out, mcode,
                                  ms_shape.eps, workspace=mws)
        call = lambda i: binding.msla_forward(mdesc, mx, mweights, mo, stream)
        for i in range(3):
            call(i)
        ms = [m / steps for m in timed_blocks(call, blocks=blocks, steps=steps)]
        fused_m = binding.msla_forward_fuses_apply(mdesc) == 1
        bpt_m = stage_bytes_per_token(ms_shape)
        names = STAGES_FUSED if fused_m else STAGES
        mbytes = sum(bpt_m[n] for n in names) * ms_shape.B * ms_shape.N
        return {"workload": ms_shape.name, "tokens": ms_shape.B * ms_shape.N, "ms": round(med(ms), 5), "ms_min": round(min(ms), 5),
                "ms_max": round(max(ms), 5), "tokens_per_s": ms_shape.B * ms_shape.N / (med(ms) * 1e-3),
                "module_GBps": round(mbytes / (med(ms) * 1e-3) / 1e9, 1),
                "l2": "exceeds L2" if mbytes > 4 * 126e6 else "L2-resident", "steps_4_5_fused": fused_m}

    def time_ffn_block(ms_shape: inputs.ModuleShape, c_hidden: int, blocks=5, steps=5):
        """The other half of the building block at this workload's shape: FFN+DWConv alone (hard-swish, biases,
        residual) and the whole block (attention module + FFN, both residual connections)."""
        fs = inputs.FfnShape(f"ffn_{ms_shape.name}", ms_shape.dtype, ms_shape.B, ms_shape.C, ms_shape.H, ms_shape.W, c_hidden, ms_shape.C,
                             seed=ms_shape.seed)
        ft = inputs.ffn_inputs(fs)
        mt = inputs.module_inputs(ms_shape)
        mdt = torch.float32 if ms_shape.dtype == "f32" else torch.bfloat16
        mcode = binding.MSLA_F32 if ms_shape.dtype == "f32" else binding.MSLA_BF16
        fd = {k: torch.from_numpy(v).to("cuda").to(mdt).contiguous() for k, v in ft.items()}
        md = {k: torch.from_numpy(v).to("cuda").to(mdt).contiguous() for k, v in mt.items()}
        B, C, H, W = ms_shape.B, ms_shape.C, ms_shape.H, ms_shape.W
        f0 = binding.make_ffn_desc(B, C, H, W, c_hidden, C, mcode, binding.MSLA_ACT_HARDSWISH, True)
        fws = torch.empty(binding.msla_ffn_workspace_bytes(f0), dtype=torch.uint8, device="cuda")
        fdesc = binding.make_ffn_desc(B, C, H, W, c_hidden, C, mcode, binding.MSLA_ACT_HARDSWISH, True, workspace=fws)
        fw = binding.make_ffn_weights(fd["w1"], fd["w_dw"], fd["w2"], fd["b1"], fd["b_dw"], fd["b2"])
        a0 = binding.make_desc(B, C, H, W, ms_shape.heads, ms_shape.d, C, mcode, ms_shape.eps)
        aws = torch.empty(binding.msla_forward_workspace_bytes(a0), dtype=torch.uint8, device="cuda")
        adesc = binding.make_desc(B, C, H, W, ms_shape.heads, ms_shape.d, C, mcode, ms_shape.eps, workspace=aws)
        aw = binding.make_weights(md["w_qkv"], md["w_dw"], md["w_pw"], md["w_proj"])
        y, o = torch.empty_like(md["x"]), torch.empty_like(md["x"])
        res = {}
        e = 2 if ms_shape.dtype == "bf16" else 4
        tokens = B * ms_shape.N
        # bytes with materialised intermediates: first layer C + Ch, depthwise 2 Ch, second layer Ch + 2 C (residual read, output)
        ffn_bytes = (4 * c_hidden + 4 * C) * e * tokens
        for name, call in (("ffn_dwconv", lambda i: binding.msla_ffn_dwconv(fdesc, md["x"], fw, o, stream)),
                           ("evit_block", lambda i: binding.msla_evit_block(adesc, aw, fdesc, fw, md["x"], y, o, stream))):
            for i in range(3):
                call(i)
            ms = [m / steps for m in timed_blocks(call, blocks=blocks, steps=steps)]
            res[name] = {"workload": f"{ms_shape.name}_hidden{c_hidden}", "tokens": tokens, "ms": round(med(ms), 5),
                         "ms_min": round(min(ms), 5), "ms_max": round(max(ms), 5), "tokens_per_s": tokens / (med(ms) * 1e-3)}
        res["ffn_dwconv"]["GBps_of_materialised_plan"] = round(ffn_bytes / (res["ffn_dwconv"]["ms"] * 1e-3) / 1e9, 1)
        return res

    other = None
    if rank == 0 and world == 1 and not args.no_configs:
        other = {}
        c2 = inputs.CONFIG2
        m2, lo2, hi2, b2 = time_core(c2, blocks=5, steps=10)
        other["cfg2_core"] = {"workload": c2.name, "ms": round(m2, 5), "ms_min": round(lo2, 5), "ms_max": round(hi2, 5),
                              "token_heads_per_s": c2.B * c2.heads * c2.N / (m2 * 1e-3), "GBps": round(b2 / (m2 * 1e-3) / 1e9, 1),
                              "l2": "L2-resident (134 MB in and out)"}
        m2h, lo2h, hi2h, b2h = time_core(inputs.CoreShape(c2.name.replace("bf16", "f16"), "f16", c2.B, c2.heads, c2.N, c2.d, c2.seed), blocks=5, steps=10)
        other["cfg2_core_f16"] = {"workload": c2.name.replace("bf16", "f16"), "ms": round(m2h, 5), "ms_min": round(lo2h, 5), "ms_max": round(hi2h, 5),
                                  "token_heads_per_s": c2.B * c2.heads * c2.N / (m2h * 1e-3), "GBps": round(b2h / (m2h * 1e-3) / 1e9, 1),
                                  "l2": "L2-resident (134 MB in and out)"}
        other["cfg3"] = time_module(inputs.CONFIG3)
        other["cfg4"] = time_module(inputs.CONFIG4)
        # a bf16, d = 16 sibling of config 1's width at 256 x 256 tokens, 384 channels
        other["d16_256x256_c384"] = time_module(inputs.ModuleShape("bf16_d16_256x256_c384", "bf16", 1, 384, 256, 256, 24, 16, seed=7))
        # fp16 storage at the bench workload's shape: the same tensor-core kernels instantiated for binary16
        other["cfg5_512x512_f16"] = time_module(inputs.ModuleShape(s.name.replace("bf16", "f16"), "f16", s.B, s.C, s.H, s.W, s.heads, s.d, seed=s.seed))
        # the token-sharded path's two band calls on one rank (no halo, one state): what the split itself costs
        band1 = time_token_sharded(s, 0, 1, steps=10, warmup=3, blocks=5)
        other["band_calls_one_rank"] = {"workload": s.name, "ms": round(med(band1), 5), "ms_min": round(min(band1), 5),
                                        "ms_max": round(max(band1), 5)}
        # the rest of the building block (FFN with a depthwise convolution, expansion 4) at the bench workload's shape
        other.update(time_ffn_block(s, 4 * s.C))
        sweep = [time_module(c) for c in inputs.CONFIG5]
        ns = np.array([c["tokens"] for c in sweep], dtype=np.float64)
        ts = np.array([c["ms"] for c in sweep], dtype=np.float64) * 1e3
        slope, icpt = np.polyfit(ns, ts, 1)     # least squares: t [us] = a + b * N
        other["cfg5_sweep"] = {"points": sweep, "fit_us": {"a_us": round(float(icpt), 2), "b_ns_per_token": round(float(slope) * 1e3, 4),
                                                           "max_rel_residual": round(float(np.max(np.abs(icpt + slope * ns - ts) / ts)), 3)}}

    ms_total, ms_lo, ms_hi = med(ms_blocks), min(ms_blocks), max(ms_blocks)
    ms_total, ms_lo, ms_hi, ms_e2e, ms_e2e_serial, ms_plain = max_over_ranks(
        [ms_total, ms_lo, ms_hi, med(ms_e2e_blocks), med(ms_e2e_serial_blocks), med(ms_plain_blocks)], device="cuda")

    if rank == 0:
        fused = binding.msla_forward_fuses_apply(desc) == 1
        stage_names = STAGES_FUSED if fused else STAGES
        stage_ms = {name: statistics.mean(v) for name, v in stage_acc.items()}
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
            core_ms, core_how = core[0], "stand-alone core entry (msla_linattn_relu_ws) on seeded [B, 2*heads, N, d] tensors of this workload"
            core_gbps = core[3] / (core_ms * 1e-3) / 1e9
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
            "warmup": W, "ms_per_step": ms_total / K, "ms_per_step_min": ms_lo / K, "ms_per_step_max": ms_hi / K,
            "timed_blocks": BLOCKS, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": s.name, "B": s.B, "C": s.C, "H": s.H, "W": s.W, "heads_per_scale": s.heads, "d": s.d,
                       "tokens_per_step_per_gpu": s.B * s.N, "accumulate": "f32",
                       "l2": "inputs and intermediates of one step exceed the 126 MB L2" if
                       module_bytes > 4 * 126e6 else "working set fits L2: numbers are L2-resident",
                       "steps_4_5_fused": fused,
                       "timing": f"median of {BLOCKS} blocks of {K} steps, CUDA events around each block",
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
            "module_GBps_of_the_unfused_21Ce_plan": round(sum(bpt[n] for n in STAGES) * s.B * s.N / (ms_total * 1e-3 / K) / 1e9, 1),
            "clocks": clocks,
        }
        if core is not None:
            result["attention_core"]["ms_min"], result["attention_core"]["ms_max"] = round(core[1], 5), round(core[2], 5)
        if other is not None:
            result["configs"] = other
        if world == 1 and not args.no_cpu_baseline:
            side = 512 if max(s.H, s.W) >= 512 else max(s.H, s.W)
            v_all, sec_all, cores = time_oracle_f32(s, side, 0)
            v_one, sec_one, _ = time_oracle_f32(s, min(side, 128), 1)
            result["cpu_baseline"] = {"value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
                                      "sample": f"the oracle's source instantiated in fp32 (-Ddouble=float, gcc -O3 -march=native), best of 3: "
                                                f"{min(side, s.H)}x{min(side, s.W)} crop of the token grid on {cores} threads ({sec_all:.1f} s per pass); "
                                                f"one thread on a {min(side, 128, s.H)}x{min(side, 128, s.W)} crop: {v_one:.0f} tokens/s ({sec_one:.1f} s per pass)",
                                      "single_thread_value": v_one}
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
