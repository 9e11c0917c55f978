#!/usr/bin/env python
"""Benchmark of the bounded-cache decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch: one bct_decode_step (one token
per sequence: K stream, softmax statistics, V stream with the in-place update rule).
The default workload is the batched 7B-MHA-shaped configuration (batch 64, 32 heads,
head_dim 128, capacity 2048, bfloat16 cache) with seeded Gaussian inputs.  Prints ONE
JSON line.  With N > 1 (torchrun) every rank runs the same per-GPU batch on its own GPU
(units are independent: no collective on the data path) and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2411_15785_b200 import workloads as W  # noqa: E402

METRIC = "bounded-cache decode tokens/s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        mhz.sort()
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def max_over_ranks(values, device):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (the job is as slow as its slowest rank).  Works on any backend; a single process returns its own."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def rank_workload(w, rank):
    """The workload of one rank: the same per-GPU batch (weak scaling; units never interact, so there
    is no data-path collective), drawn from a rank-specific seed."""
    return w.scaled(seed=w.seed + 1000 * rank)


def algorithmic_bytes_per_step(w: W.Workload) -> int:
    """Bytes the method must move per step: MK once + MV once per unit, plus the step vectors.
    The write-back of the few rows the update rule changes is left out (a conservative count)."""
    s = w.elem_bytes
    per_unit = 2 * w.capacity * w.head_dim * s + (2 * w.group + 2) * w.head_dim * s
    return w.units * per_unit


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the committed ncu capture of
# decode_tc_kernel (profiles/decode_tc_kernel_ncu_full.txt), taken at batch 37 and scaled by units:
# 1.0949 MB per (sequence, kv-head) unit of the mha7b shape.  None for any other kernel / shape.
TRAFFIC_PER_UNIT = {("mha7b", True): 1.2942e9 / 1184}


def measured_traffic(w, tensor_path):
    per_unit = TRAFFIC_PER_UNIT.get((w.name.split("_")[0], bool(tensor_path)))
    return None if per_unit is None else per_unit * w.units


def stream_roofline(w, tok_per_step, ms_step, precise=False, write_only=False):
    """Tensor-core roofline of stream_tc_kernel: the dense flops its MMAs execute per step (operand rows padded
    to M = 128 included) against the measured bf16 matmul peak."""
    Tc = {1: 64, 2: 40, 3: 32, 4: 24}.get(w.group, 16)
    Tcp = (Tc + 15) // 16 * 16                    # the products run on the chunk padded to 16 tokens
    C, d = w.capacity, w.head_dim
    if write_only:                                 # bct_update_kv: chunks of 128 write rows, no outputs
        Tc = 128
        per_chunk = 2 * (2 * 128 * C * d) + 2 * (2 * C * Tc * d)
    else:
        per_chunk = 2 * (2 * 128 * C * d)          # scores of the 128 operand rows, two passes over MK
        per_chunk += (3 if precise else 1) * (2 * 128 * C * d)   # outputs: P MV_hi (+ P_lo MV_hi + P MV_lo with PRECISE_READ)
        per_chunk += 2 * 128 * C * Tcp             # A = P WW^T
        per_chunk += 2 * (2 * C * Tcp * d)         # MV increment with value + residual weights
        per_chunk += 2 * 128 * Tcp * d             # strict_tril(A) Vc
    flops = per_chunk * (tok_per_step // Tc) * w.units
    peak = FALLBACK_BF16_TFLOPS
    kind = "fallback"
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            peak, kind = float(json.load(open(path))["bf16_tflops_sustained"]), "measured"
        except Exception:
            pass
    ach = flops / (ms_step * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
            "peak_kind": "of " + kind, "kernel": "stream_tc_kernel", "flops_per_launch": flops}


def cpu_oracle_sample(w: W.Workload, budget_s: float = 25.0):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: a few
    (sequence, kv-head) units per core, for as many tokens as fit the time budget."""
    from oracle import bct_oracle as O
    import numpy as np
    cores = os.cpu_count() or 1
    n_units = min(w.units, 2 * cores)
    rng = np.random.default_rng(w.seed)

    def fresh():
        mk = rng.standard_normal((n_units, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
        mv = rng.standard_normal((n_units, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
        return O.OracleCache(n_units, w.group, 1, w.head_dim, w.capacity, read_scale=w.read_scale,
                             write_scale=w.write_scale, init_len=w.init_len, mk_init=mk, mv_init=mv)

    def draw(T):
        return (rng.standard_normal((n_units, T, w.group, w.head_dim)) * w.q_std,
                rng.standard_normal((n_units, T, 1, w.head_dim)) * w.kv_std,
                rng.standard_normal((n_units, T, 1, w.head_dim)) * w.kv_std)

    ora = fresh()
    ora.prefill_stream(*draw(2))                      # loads the library, warms the caches
    x = draw(8)
    t0 = time.perf_counter()
    ora.prefill_stream(*x)
    per_token = max((time.perf_counter() - t0) / 8, 1e-6)
    T = int(max(8, min(20000, budget_s / per_token)))
    x = draw(T)
    t0 = time.perf_counter()
    ora.prefill_stream(*x)
    dt = time.perf_counter() - t0
    unit_tokens_per_s = n_units * T / dt
    return {"value": unit_tokens_per_s / w.n_kv_heads, "unit": UNIT, "cores": int(ora.threads_used), "kind": "oracle",
            "sample": "%d of %d (sequence, kv-head) units x %d tokens in %.1f s of wall time, scaled by %d units per sequence"
                      % (n_units, w.units, T, dt, w.n_kv_heads), "seconds": dt, "tokens": T}


def run_reference(args, w):
    """The reference arm: the double-precision CPU oracle, as it stands, on the host cores.
    Each step is a bounded sample of the workload (a few units per core for a few tokens),
    sized so that the whole run ends within about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import bct_oracle as O
    import numpy as np
    cores = os.cpu_count() or 1
    n_units = min(w.units, 2 * cores)
    rng = np.random.default_rng(w.seed)
    mk = rng.standard_normal((n_units, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
    mv = rng.standard_normal((n_units, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
    ora = O.OracleCache(n_units, w.group, 1, w.head_dim, w.capacity, read_scale=w.read_scale,
                        write_scale=w.write_scale, init_len=w.init_len, mk_init=mk, mv_init=mv)

    def draw(T):
        return (rng.standard_normal((n_units, T, w.group, w.head_dim)) * w.q_std,
                rng.standard_normal((n_units, T, 1, w.head_dim)) * w.kv_std,
                rng.standard_normal((n_units, T, 1, w.head_dim)) * w.kv_std)

    ora.prefill_stream(*draw(2))
    x = draw(8)
    t0 = time.perf_counter()
    ora.prefill_stream(*x)
    per_token = max((time.perf_counter() - t0) / 8, 1e-6)
    total = args.steps + args.warmup
    T = int(max(1, min(4096, (100.0 / total) / per_token)))
    elapsed = 0.0
    for i in range(total):
        x = draw(T)
        t0 = time.perf_counter()
        ora.prefill_stream(*x)
        if i >= args.warmup:
            elapsed += time.perf_counter() - t0
    val = n_units * T * args.steps / elapsed / w.n_kv_heads
    sample = ("each step: %d of %d (sequence, kv-head) units x %d tokens; value scaled by %d units per sequence"
              % (n_units, w.units, T, w.n_kv_heads))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch / val, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "n_q_heads": w.n_q_heads,
                       "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "capacity": w.capacity,
                       "write_scale": w.write_scale, "read_scale": w.read_scale},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": int(ora.threads_used), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def secondary_regime(B, w, wr, dev, pool, outs, peak, steps=200):
    """The diffuse write regime (write_scale = 1/sqrt(d): every row of the value memory is rewritten each
    token) on a second cache of the same shape: ms per step and the bytes it must move, five planes
    (K and MV value read, MV residual read, MV value and residual written), against the copy peak."""
    ws = w.head_dim ** -0.5
    mk, mv = W.initial_cache(wr, dev)
    cache = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, read_scale=w.read_scale,
                    write_scale=ws, init_len=w.init_len, mk_init=mk, mv_init=mv, device=dev)
    del mk, mv
    for i in range(5):
        cache.decode_step(*pool[i % len(pool)], out=outs[i & 1])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        cache.decode_step(*pool[i % len(pool)], out=outs[i & 1])
    e1.record()
    torch.cuda.synchronize()
    cache.check_status()
    ms = e0.elapsed_time(e1) / steps
    eb = 4 if w.dtype == "f32" else 2
    planes = 3 if w.dtype == "f32" else 5
    nbytes = planes * w.units * w.capacity * w.head_dim * eb
    ach = nbytes / (ms * 1e-3) / 1e9
    cache.destroy()
    return {"write_scale": ws, "steps": steps, "ms_per_step": ms, "value": w.batch / (ms * 1e-3), "unit": UNIT,
            "bytes_per_step": nbytes, "achieved": ach, "peak": peak, "frac": ach / peak,
            "note": "every row rewritten: K, MV value and residual read, MV value and residual written"}


def run_project(args, w):
    """Times bct_project_qkv alone (the projections in front of the layer) for --project-tokens rows of
    x with the workload's head counts: one step = one launch.  Two weight sets are used alternately so
    that the weights of a step (100 MB at d_model 4096) do not come from L2."""
    from paper_2411_15785_b200 import binding as B
    from paper_2411_15785_b200 import build as bld
    bld.build()
    B.load()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    M, K = args.project_tokens, args.d_model
    n_q, n_kv = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    g = torch.Generator(device=dev).manual_seed(w.seed)
    sets = [tuple((torch.randn((n, K), generator=g, device=dev) * K ** -0.5).to(torch.bfloat16) for n in (n_q, n_kv, n_kv))
            for _ in range(2)]
    xs = [torch.randn((M, K), generator=g, device=dev).to(torch.bfloat16) for _ in range(4)]
    warm = max(args.warmup, 3)
    outs = (torch.empty((M, n_q), dtype=torch.bfloat16, device=dev), torch.empty((M, n_kv), dtype=torch.bfloat16, device=dev),
            torch.empty((M, n_kv), dtype=torch.bfloat16, device=dev))
    for i in range(warm):
        B.project_qkv(xs[i % 4], *sets[i & 1], out=outs)
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        B.project_qkv(xs[i % 4], *sets[i & 1], out=outs)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_step = e0.elapsed_time(e1) / args.steps
    n_out = n_q + 2 * n_kv
    flops = 2.0 * M * n_out * K
    nbytes = 2.0 * (n_out * K + M * K + M * n_out)
    hbm_peak, kind = _peaks()
    tf_peak = FALLBACK_BF16_TFLOPS
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            tf_peak = float(json.load(open(path))["bf16_tflops_sustained"])
        except Exception:
            pass
    t_hbm, t_tensor = nbytes / (hbm_peak * 1e9), flops / (tf_peak * 1e12)
    if t_hbm >= t_tensor:
        ach = nbytes / (ms_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak,
                "algorithmic_bytes_per_launch": nbytes}
    else:
        ach = flops / (ms_step * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": tf_peak, "unit": "TFLOP/s", "frac": ach / tf_peak,
                "flops_per_launch": flops}
    roof.update({"traffic": None, "peak_kind": "of " + kind, "kernel": "project_kernel"})
    print(json.dumps({
        "metric": "projection tokens/s", "value": M / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16, f32 accumulate", "data": "synthetic",
        "config": {"workload": "project_qkv", "tokens": M, "d_model": K, "n_q": n_q, "n_kv": n_kv,
                   "l2": "two weight sets used alternately (%.0f MB each)" % (2e-6 * n_out * K)},
        "clocks": clocks, "gpu_launches": args.steps, "roofline": roof}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="mha7b_b64_c2048", choices=sorted(W.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--write-scale", type=float, default=None, help="override the write score scale")
    ap.add_argument("--stream-tokens", type=int, default=256,
                    help="tokens per sequence pushed by one step of a stream workload")
    ap.add_argument("--write-eps", type=float, default=0.0, help="override write_eps (0 = library default 2^-24)")
    ap.add_argument("--flags", type=int, default=0, help="BCT_FLAG_* bits for the cache")
    ap.add_argument("--batch", type=int, default=None, help="override the batch (profiling on a smaller case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short run of the diffuse write regime")
    ap.add_argument("--update-kv", action="store_true",
                    help="stream workloads: time bct_update_kv (Algorithm 1's UpdateKV, state only) instead of bct_prefill_stream")
    ap.add_argument("--project-tokens", type=int, default=0,
                    help="time bct_project_qkv alone on this many tokens (the workload gives the head counts)")
    ap.add_argument("--d-model", type=int, default=4096, help="model width of the projections")
    args = ap.parse_args()
    w = W.CONFIGS[args.workload]
    if args.write_scale is not None:
        w = w.scaled(write_scale=args.write_scale)
    if args.batch is not None:
        w = w.scaled(batch=args.batch, name="%s@batch%d" % (w.name, args.batch))
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.project_tokens > 0:
        run_project(args, w)
        return
    if args.warmup < 3:
        args.warmup = 3

    from paper_2411_15785_b200 import binding as B
    from paper_2411_15785_b200 import build as bld

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        bld.build()
    if world > 1:
        dist.barrier()
    B.load()

    # per-rank workload: the same per-GPU batch on every rank (weak scaling), a different seed per rank
    wr = rank_workload(w, rank)
    mk, mv = W.initial_cache(wr, dev)
    cache = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype,
                    read_scale=w.read_scale, write_scale=w.write_scale, init_len=w.init_len, mk_init=mk, mv_init=mv,
                    write_eps=args.write_eps, flags=args.flags, max_stream=(args.stream_tokens if w.api == "stream" else 1),
                    device=dev)
    torch.cuda.synchronize()
    del mk, mv
    stream = (w.api == "stream")
    tok_per_step = args.stream_tokens if stream else 1   # tokens per sequence in one step
    if stream:
        # fill the cache (untimed), then every step pushes one block of tokens through bct_prefill_stream
        t_fill = 0
        while cache.len < w.capacity:
            n = min(256, w.capacity - cache.len)
            cache.prefill_stream(*W.stream_inputs(wr, t_fill, n, dev), want_out=False)
            t_fill += n
        pool = [W.stream_inputs(wr, w.capacity + i * tok_per_step, tok_per_step, dev) for i in range(8)]
    else:
        pool = [W.step_inputs(wr, t, dev) for t in range(min(args.steps + args.warmup, 64))]
    outs = [torch.empty_like(pool[0][0], dtype=cache.out_dtype) for _ in range(2)]

    update_only = stream and args.update_kv

    def step_dev(i):
        if update_only:
            cache.update_kv(pool[i % len(pool)][1], pool[i % len(pool)][2])
        elif stream:
            cache.prefill_stream(*pool[i % len(pool)], out=outs[i & 1])
        else:
            cache.decode_step(*pool[i % len(pool)], out=outs[i & 1])

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---------- device-resident timing ----------
    for i in range(args.warmup):
        step_dev(i)
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = cache.launches
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step_dev(args.warmup + i)
    e1.record()
    sync_all()
    ms_total = e0.elapsed_time(e1)
    launches = cache.launches - launches0
    clocks = sampler.stop() if rank == 0 else None
    cache.check_status()

    # ---------- end to end through the host-buffer entry point ----------
    hpool = [tuple(x.cpu().pin_memory() for x in pool[i]) for i in range(min(len(pool), 16))]
    hout = [torch.empty_like(hpool[0][0], dtype=cache.out_dtype).pin_memory() for _ in range(2)]

    def step_host(i):
        if update_only:   # no host-buffer form of UpdateKV: the stream call without outputs
            cache.prefill_stream_host(*hpool[i % len(hpool)], None)
        elif stream:
            cache.prefill_stream_host(*hpool[i % len(hpool)], hout[i & 1])
        else:
            cache.decode_step_host(*hpool[i % len(hpool)], hout[i & 1])

    for i in range(3):
        step_host(i)
    sync_all()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for i in range(args.steps):
        step_host(i)
    e3.record()
    sync_all()
    ms_e2e = e2.elapsed_time(e3)
    cache.check_status()
    h2d = sum(x.numel() * x.element_size() for x in hpool[0])
    d2h = 0 if update_only else hout[0].numel() * hout[0].element_size()

    if world > 1:
        ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dev)

    if rank == 0:
        peak, peak_kind = _peaks()
        ms_step = ms_total / args.steps
        tokens = w.batch * world * args.steps * tok_per_step
        alg = algorithmic_bytes_per_step(w)
        achieved = alg / (ms_step * 1e-3) / 1e9
        if stream:
            roof = stream_roofline(w, tok_per_step, ms_step, precise=bool(args.flags & 16), write_only=update_only)
        else:
            roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": measured_traffic(w, cache.tensor_path), "peak_kind": "of " + peak_kind,
                    "kernel": "decode_tc_kernel" if cache.tensor_path else "decode_kernel",
                    "algorithmic_bytes_per_launch": alg, "frac_of_8TBps_nominal": achieved / 8000.0}
        line = {
            "metric": METRIC, "value": tokens / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if w.dtype == "f32" else "bf16 cache, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "n_q_heads": w.n_q_heads,
                       "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "capacity": w.capacity,
                       "write_scale": w.write_scale, "read_scale": w.read_scale,
                       "tokens_per_step": tok_per_step, "call": "bct_update_kv" if update_only else (
                           "bct_prefill_stream" if stream else "bct_decode_step"),
                       "l2": ("cache planes of all units (%.2f GB) exceed L2" % (1.5 * alg / 1e9)) if stream else
                             ("cache planes streamed per step (%.2f GB) exceed L2" % (alg / 1e9)),
                       "parallelism": "independent units; replicas per GPU" if world > 1 else "1 GPU"},
            "clocks": clocks,
            "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches,
            "roofline": roof,
        }
        if world == 1 and not stream and args.write_scale is None and not args.no_secondary:
            line["secondary_write_regime"] = secondary_regime(B, w, wr, dev, pool, outs, peak)
        if world == 1 and not args.no_cpu_baseline:
            cb = cpu_oracle_sample(w)
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
        print(json.dumps(line))
    cache.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
