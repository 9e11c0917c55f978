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
    """Roofline denominators: this machine's measured copy bandwidth and sustained bf16 matmul rate
    (MEASURED_PEAKS.json, written by the run's driver), else the fallback figures."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {"hbm": float(d["hbm_gbs"]), "tf": float(d["bf16_tflops_sustained"]), "kind": "measured"}
        except Exception:
            pass
    return {"hbm": FALLBACK_HBM_GBS, "tf": FALLBACK_BF16_TFLOPS, "kind": "fallback"}


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


def algorithmic_bytes_per_step(w: W.Workload, w_frac: float = 0.0) -> int:
    """Bytes the method must move per decode step and unit: MK once + MV's value plane once, the rows the
    update rule rewrites (fraction w_frac of the C slots, counted by the kernels: residual read, value and
    residual written; their value read is already in the MV stream), and the step vectors."""
    s = w.elem_bytes
    planes_rw = 3 if w.dtype == "bf16" else 1     # float caches have no residual plane: the row is written once
    per_unit = 2 * w.capacity * w.head_dim * s + w_frac * w.capacity * w.head_dim * planes_rw * s \
        + (2 * w.group + 2) * w.head_dim * s
    return int(w.units * per_unit)


# DRAM bytes per launch and unit (dram__bytes_read.sum + dram__bytes_write.sum) from the committed ncu capture of
# decode_tc_kernel on the mha7b shape (profiles/decode_tc_kernel_ncu_full.txt: 1.2630 GB read + 0.0318 GB written at
# batch 37 = 1184 units; the traffic grows in proportion to the units).  None for any other kernel / shape.
NCU_TRAFFIC_PER_UNIT = {("mha7b", True): 1.2948e9 / 1184}


def measured_traffic(w, tensor_path):
    per_unit = NCU_TRAFFIC_PER_UNIT.get((w.name.split("_")[0], bool(tensor_path)))
    return None if per_unit is None else per_unit * w.units


def stream_chunk_tokens(group: int) -> int:
    return {1: 64, 2: 40, 3: 32, 4: 24}.get(group, 16)


def backward_flops(w, tok_per_step):
    """(executed, algorithmic) flops of one bct_update_kv_backward step: five contractions of 2 T C d per unit
    (scores, R = WW G, A = Wv G^T, dWq = dS MK, dMK = dS^T Wq); the kernel forms the scores three times and pads
    the tokens to blocks of 128."""
    C, d = w.capacity, w.head_dim
    Tp = (tok_per_step + 127) // 128 * 128
    return 7 * 2 * Tp * C * d * w.units, 5 * 2 * tok_per_step * C * d * w.units


def stream_flops(w, tok_per_step, precise=False, write_only=False):
    """(executed, algorithmic) dense flops of one stream step.  Executed: what stream_tc_kernel's MMAs run
    (operand rows padded to M = 128, two score passes, value + residual products).  Algorithmic: the method's
    own contractions per chunk (one score pass of the G*Tc read and Tc write rows, G*Tc output rows, one
    increment, A = Pr WW^T and strict_tril(A) Vc)."""
    Tc = stream_chunk_tokens(w.group)
    Tcp = (Tc + 15) // 16 * 16                    # the products run on the chunk padded to 16 tokens
    C, d, G = w.capacity, w.head_dim, w.group
    if write_only:                                 # bct_update_kv: chunks of 128 write rows, no outputs
        Tc = 128
        executed = 2 * (2 * 128 * C * d) + 2 * (2 * C * Tc * d)
        algorithmic = 2 * Tc * C * d + 2 * C * Tc * d
    else:
        executed = 2 * (2 * 128 * C * d)          # scores of the 128 operand rows, two passes over MK
        executed += (2 if precise else 1) * (2 * 128 * C * d)   # outputs: P MV_hi (+ P MV_lo with PRECISE_READ)
        executed += 2 * 128 * C * Tcp             # A = P WW^T
        executed += 2 * (2 * C * Tcp * d)         # MV increment with value + residual weights
        executed += 2 * 128 * Tcp * d             # strict_tril(A) Vc
        algorithmic = 2 * (G + 1) * Tc * C * d + 2 * G * Tc * C * d + 2 * Tc * C * d + 2 * G * Tc * C * Tc \
            + G * Tc * Tc * d
    n = (tok_per_step // Tc) * w.units
    return executed * n, algorithmic * n


def stream_roofline(w, tok_per_step, ms_step, precise=False, write_only=False, backward=False):
    """Tensor-core roofline of stream_tc_kernel (update_bwd_kernel for the backward) against the measured
    sustained bf16 matmul rate: `frac` on the method's own flops, `frac_executed` on the flops the kernel's MMAs run."""
    executed, algorithmic = backward_flops(w, tok_per_step) if backward else stream_flops(w, tok_per_step, precise, write_only)
    pk = _peaks()
    ach = algorithmic / (ms_step * 1e-3) / 1e12
    ach_x = executed / (ms_step * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": ach, "peak": pk["tf"], "unit": "TFLOP/s", "frac": ach / pk["tf"],
            "traffic": None, "peak_kind": "of " + pk["kind"], "kernel": "update_bwd_kernel" if backward else "stream_tc_kernel",
            "flops_per_launch": algorithmic, "executed_flops_per_launch": executed, "achieved_executed": ach_x,
            "frac_executed": ach_x / pk["tf"]}


class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of a workload: a few (sequence, kv-head) units per
    core with inputs of the workload's shapes and value scales (the one place besides the parity check where
    the benchmark runs anything under oracle/)."""

    def __init__(self, w: W.Workload):
        from oracle import bct_oracle as O
        import numpy as np
        self.w = w
        self.n_units = min(w.units, 2 * (os.cpu_count() or 1))
        self.rng = np.random.default_rng(w.seed)
        n, r = self.n_units, self.rng
        mk = r.standard_normal((n, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
        mv = r.standard_normal((n, 1, w.init_len, w.head_dim)) * w.init_std if w.init_len else None
        self.ora = O.OracleCache(n, w.group, 1, w.head_dim, w.capacity, read_scale=w.read_scale,
                                 write_scale=w.write_scale, init_len=w.init_len, mk_init=mk, mv_init=mv)
        self.run(2)                                   # loads the library, warms the caches
        self.per_token = max(self.run(8) / 8, 1e-6)   # seconds per token of the sample

    def run(self, T: int) -> float:
        """Push T tokens through the sampled units; returns the wall time of the oracle call alone."""
        w, n, r = self.w, self.n_units, self.rng
        x = (r.standard_normal((n, T, w.group, w.head_dim)) * w.q_std,
             r.standard_normal((n, T, 1, w.head_dim)) * w.kv_std,
             r.standard_normal((n, T, 1, w.head_dim)) * w.kv_std)
        t0 = time.perf_counter()
        self.ora.prefill_stream(*x)
        return time.perf_counter() - t0

    def tokens_per_s(self, T: int, seconds: float) -> float:
        """Whole-sequence tokens/s: unit-tokens per second scaled by the units one sequence holds."""
        return self.n_units * T / seconds / self.w.n_kv_heads

    @property
    def cores(self) -> int:
        return int(self.ora.threads_used)


def cpu_oracle_sample(w: W.Workload, budget_s: float = 15.0):
    """cpu_baseline: the oracle on the sample for as many tokens as fit the time budget."""
    smp = OracleSample(w)
    T = int(max(8, min(20000, budget_s / smp.per_token)))
    dt = smp.run(T)
    return {"value": smp.tokens_per_s(T, dt), "unit": UNIT, "cores": smp.cores, "kind": "oracle",
            "sample": "%d of %d (sequence, kv-head) units x %d tokens in %.1f s of wall time, scaled by %d units per sequence"
                      % (smp.n_units, w.units, T, dt, w.n_kv_heads)}


def run_reference(args, w):
    """The reference arm: the double-precision CPU oracle, as it stands, on the host cores.  Each step is a
    bounded sample of the workload (a few units per core for a few tokens), sized so that the whole run
    ends within about two minutes.  Rank 0 alone runs and prints it."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    smp = OracleSample(w)
    total = args.steps + args.warmup
    T = int(max(1, min(4096, (args.ref_seconds / total) / smp.per_token)))
    elapsed = 0.0
    for i in range(total):
        dt = smp.run(T)
        if i >= args.warmup:
            elapsed += dt
    val = smp.tokens_per_s(T * args.steps, elapsed)
    sample = ("each step: %d of %d (sequence, kv-head) units x %d tokens; value scaled by %d units per sequence"
              % (smp.n_units, w.units, T, w.n_kv_heads))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch / val, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, args.stream_tokens if w.api == "stream" else 1),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def config_of(w: W.Workload, tok_per_step: int):
    """The workload's description, the same keys and values on both arms (`l2` says why no L2 flush is needed
    between the GPU arm's timed steps)."""
    planes = (3 if w.dtype == "bf16" else 2) * w.units * w.capacity * w.head_dim * w.elem_bytes
    if w.api == "stream":
        l2 = "cache planes of all units (%.2f GB) exceed L2" % (planes / 1e9)
    else:
        l2 = "cache planes streamed per step (%.2f GB of %.2f GB resident) exceed L2" % (
            2 * w.units * w.capacity * w.head_dim * w.elem_bytes / 1e9, planes / 1e9)
    return {"workload": w.name, "batch_per_gpu": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "capacity": w.capacity, "write_scale": w.write_scale, "read_scale": w.read_scale,
            "tokens_per_step": tok_per_step, "l2": l2}


def make_cache(B, w, wr, dev, flags=0, write_eps=0.0, max_stream=1, write_scale=None):
    """A cache of the workload's shape with its seeded initial state."""
    mk, mv = W.initial_cache(wr, dev)
    cache = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, read_scale=w.read_scale,
                    write_scale=w.write_scale if write_scale is None else write_scale, init_len=w.init_len,
                    mk_init=mk if w.init_len else None, mv_init=mv if w.init_len else None, write_eps=write_eps,
                    flags=flags, max_stream=max_stream, device=dev)
    torch.cuda.synchronize()
    del mk, mv
    return cache


def fill_stream_cache(cache, wr, dev):
    """Push the first `capacity` tokens of the stream (the fill phase, untimed)."""
    t = 0
    while cache.len < cache.C:
        n = min(256, cache.C - cache.len)
        cache.prefill_stream(*W.stream_inputs(wr, t, n, dev), want_out=False)
        t += n
    return t


def timed(fn, steps, warmup):
    """warmup untimed calls of fn(i), then `steps` timed ones between CUDA events on the current stream
    (the stream every launch of the binding goes to); returns the milliseconds of the timed calls."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def decode_roofline(w, cache, ms_step, rows0, steps_counted):
    """HBM roofline of a decode step: algorithmic bytes, with the share of MV rows the kernels rewrote per token
    (their own counter) in them, over the mean launch duration."""
    pk = _peaks()
    rows = cache.rows_rewritten() - rows0
    w_frac = rows / float(max(1, w.units * steps_counted * w.capacity))
    alg = algorithmic_bytes_per_step(w, w_frac)
    ach = alg / (ms_step * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s", "frac": ach / pk["hbm"],
            "traffic": measured_traffic(w, cache.tensor_path), "peak_kind": "of " + pk["kind"],
            "kernel": "decode_tc_kernel" if cache.tensor_path else "decode_kernel",
            "algorithmic_bytes_per_launch": alg, "rows_rewritten_fraction": w_frac,
            "frac_of_8TBps_nominal": ach / 8000.0}


def secondary_regime(B, w, wr, dev, pool, outs, steps=200):
    """The diffuse write regime (write_scale = 1/sqrt(d): every row of the value memory is rewritten each
    token) on a second cache of the same shape: ms per step and the bytes it must move (K and MV value read,
    MV residual read, MV value and residual written), against the copy peak."""
    ws = w.head_dim ** -0.5
    # BCT_FLAG_DENSE_WRITE states what this regime does anyway (no weight is below the threshold at this scale) and
    # lets the tensor-core kernel rebuild whole tiles in its ring instead of listing and staging single rows
    cache = make_cache(B, w, wr, dev, write_scale=ws, flags=4)
    rows0 = cache.rows_rewritten()
    ms = timed(lambda i: cache.decode_step(*pool[i % len(pool)], out=outs[i & 1]), steps, 5) / steps
    cache.check_status()
    roof = decode_roofline(w, cache, ms, rows0, steps + 5)
    cache.destroy()
    return {"write_scale": ws, "steps": steps, "ms_per_step": ms, "value": w.batch / (ms * 1e-3), "unit": UNIT,
            "bytes_per_step": roof["algorithmic_bytes_per_launch"], "achieved": roof["achieved"], "peak": roof["peak"],
            "frac": roof["frac"], "rows_rewritten_fraction": roof["rows_rewritten_fraction"], "kernel": roof["kernel"],
            "flags": 4, "note": "every row rewritten: K, MV value and residual read, MV value and residual written"}


def parity_check(B, w, wr, dev, flags, n_steps, n_units=8, stream_tokens=0):
    """Replay the workload from its initial state on a fresh cache in the launch configuration that was timed
    and follow n_units sampled (sequence, kv-head) units with the CPU oracle (units never interact, so the
    sample is exact for those units): worst max-abs error of `out` over the steps, and of the exported MV
    after the last one.  Outside every timed region; the oracle is the checker here, as in the tests."""
    import numpy as np
    from oracle import bct_oracle as O
    tol = 1e-5 if w.dtype == "f32" else 2e-2
    U, G = w.units, w.group
    rng = np.random.default_rng(w.seed)
    ids = sorted(set([0, U - 1] + rng.choice(U, size=max(0, min(U, n_units) - 2), replace=False).tolist()))
    units = [(u // w.n_kv_heads, u % w.n_kv_heads) for u in ids]
    f64 = lambda t: t.double().cpu().numpy()
    mk, mv = W.initial_cache(wr, dev)
    ok = f64(torch.stack([mk[b, h] for b, h in units])[:, None]) if w.init_len else None
    ov = f64(torch.stack([mv[b, h] for b, h in units])[:, None]) if w.init_len else None
    del mk, mv
    ora = O.OracleCache(len(units), G, 1, w.head_dim, w.capacity, read_scale=w.read_scale, write_scale=w.write_scale,
                        init_len=w.init_len, mk_init=ok, mv_init=ov)
    cache = make_cache(B, w, wr, dev, flags=flags)

    def sl(x, heads):  # [B, T, H, d] -> the sampled units' [n, T, heads, d]
        return f64(torch.stack([x[b, :, h * heads:(h + 1) * heads] for b, h in units]))

    worst, t = 0.0, 0
    while t < n_steps:
        if stream_tokens:
            n = min(stream_tokens, n_steps - t)
            q, k, v = W.stream_inputs(wr, t, n, dev)
            out = cache.prefill_stream(q, k, v)
        else:
            n = 1
            q, k, v = (x[:, None] for x in W.step_inputs(wr, t, dev))
            out = cache.decode_step(q[:, 0], k[:, 0], v[:, 0])[:, None]
        ref = ora.prefill_stream(sl(q, G), sl(k, 1), sl(v, 1))
        worst = max(worst, float(np.abs(sl(out, G) - ref).max()))
        t += n
    cache.check_status()
    vals = cache.export(torch.float32)[1]
    state = max(float(np.abs(f64(vals[b, h]) - ora.MV[i]).max()) for i, (b, h) in enumerate(units))
    del vals
    cache.destroy()
    return {"max_abs_out_per_step": worst, "max_abs_state_final": state, "tol": tol, "steps": n_steps,
            "units_checked": len(units), "of_units": U, "flags": flags, "pass": bool(worst <= tol and state <= tol),
            "against": "double-precision CPU oracle on the same seeded inputs"}


def run_config(B, name, dev, steps=60, warmup=5, flags=0, stream_tokens=256, with_parity=True):
    """One short run of another configuration for the per_config block: ms per step, tokens/s, the roofline
    fraction of its kernel, its own clock samples and a short parity check."""
    w = W.CONFIGS[name]
    sampler = ClockSampler(dev.index)
    if w.api == "stream":
        cache = make_cache(B, w, w, dev, flags=flags, max_stream=stream_tokens)
        t0 = fill_stream_cache(cache, w, dev)
        pool = [W.stream_inputs(w, t0 + i * stream_tokens, stream_tokens, dev) for i in range(4)]
        outs = [torch.empty_like(pool[0][0], dtype=cache.out_dtype) for _ in range(2)]
        sampler.start()
        ms = timed(lambda i: cache.prefill_stream(*pool[i % 4], out=outs[i & 1]), steps, warmup) / steps
        clocks = sampler.stop()
        roof = stream_roofline(w, stream_tokens, ms, precise=bool(flags & 16))
        tok = stream_tokens
    else:
        cache = make_cache(B, w, w, dev, flags=flags)
        pool = [W.step_inputs(w, t, dev) for t in range(16)]
        outs = [torch.empty_like(pool[0][0], dtype=cache.out_dtype) for _ in range(2)]
        for t in range(w.capacity - w.init_len):   # a cache that starts empty is filled first (untimed): the update rule is timed
            cache.decode_step(*pool[t % 16], out=outs[t & 1])
        rows0 = cache.rows_rewritten()
        sampler.start()
        ms = timed(lambda i: cache.decode_step(*pool[i % 16], out=outs[i & 1]), steps, warmup) / steps
        clocks = sampler.stop()
        roof = decode_roofline(w, cache, ms, rows0, steps + warmup)
        tok = 1
    cache.check_status()
    cache.destroy()
    del pool, outs
    torch.cuda.empty_cache()
    res = {"workload": name, "flags": flags, "steps": steps, "ms_per_step": ms, "value": w.batch * tok / (ms * 1e-3),
           "unit": UNIT, "tokens_per_step": tok, "capacity": w.capacity,
           "roofline": {k: roof[k] for k in roof if k in ("bound", "achieved", "peak", "unit", "frac", "kernel", "frac_executed",
                                                          "rows_rewritten_fraction", "frac_of_8TBps_nominal")},
           "clocks": clocks}
    if with_parity:
        if w.api == "stream":   # the fill phase and the first chunks of the full phase
            p = parity_check(B, w, w, dev, flags, w.capacity + 256, n_units=8, stream_tokens=256)
        else:
            p = parity_check(B, w, w, dev, flags, 8 if w.init_len == w.capacity else w.capacity - w.init_len + 32, n_units=8)
        res["parity"] = {k: p[k] for k in ("max_abs_out_per_step", "max_abs_state_final", "tol", "steps", "units_checked", "pass")}
        torch.cuda.empty_cache()
    return res


def stream_constancy(B, w, dev, flags, block=1024, n_late=3):
    """The paper's Results state that the time per input vector stays about constant once the inference
    length exceeds the cache capacity.  Here: the whole stream of the long-stream configuration goes
    through bct_prefill_stream in blocks of `block` tokens per sequence; every block is timed by CUDA events,
    and the per-token time of the first block after the fill (tokens C .. C + block) is set beside the last
    blocks of the stream.  (Inputs cycle through eight seeded blocks: the time does not depend on the values.  The
    stream runs once untimed first, so that every timed block sees the sustained clock.)"""
    cache = make_cache(B, w, w, dev, flags=flags, max_stream=1)
    pool = [W.stream_block(w, i, dev) for i in range(8)]
    out = torch.empty_like(pool[0][0], dtype=cache.out_dtype)
    n_blocks = w.steps // block
    # The same stream once untimed, on a cache of its own: the whole stream is 0.2 s, within which the SM clock settles
    # from its maximum to what the power cap allows; timed from a cold start, the early blocks would be faster for that alone.
    warm = make_cache(B, w, w, dev, flags=flags, max_stream=1)
    for i in range(n_blocks):
        warm.prefill_stream(*pool[i % 8], out=out)
    torch.cuda.synchronize()
    warm.destroy()
    del warm
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
    ev[0].record()
    for i in range(n_blocks):
        cache.prefill_stream(*pool[i % 8], out=out)
        ev[i + 1].record()
    torch.cuda.synchronize()
    cache.check_status()
    ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(n_blocks)]
    cache.destroy()
    del pool, out
    torch.cuda.empty_cache()
    first_full = (w.capacity + block - 1) // block          # first block that runs entirely against a full cache
    us_tok = lambda m: 1e3 * m / block                      # microseconds per token of every sequence
    late = ms[-n_late:]
    mid = ms[n_blocks // 2]
    return {"workload": w.name, "flags": flags, "tokens": n_blocks * block, "block_tokens": block,
            "fill_us_per_token": us_tok(sum(ms[:first_full]) / max(1, first_full)),
            "early_us_per_token": us_tok(ms[first_full]), "early_tokens": [first_full * block, (first_full + 1) * block],
            "middle_us_per_token": us_tok(mid), "late_us_per_token": us_tok(sum(late) / len(late)),
            "late_over_early": (sum(late) / len(late)) / ms[first_full],
            "max_over_min_after_fill": max(ms[first_full:]) / min(ms[first_full:]),
            "whole_stream_s": sum(ms) * 1e-3}


PAPER_CONTEXT = {
    "source": "arxiv 2411.15785, Experiments / Results",
    "hardware": "not stated", "precision": "not stated",
    "setup": "1B-parameter Transformer, cache capacity M = 2048",
    "reported": ["memory use constant once the context exceeds 2048 tokens (a conventional cache grows linearly)",
                 "time per input vector about constant once the inference length exceeds 2048",
                 "generation quality close to the conventional cache (the figure is cut off in the source)"],
    "numbers": "the paper prints no throughput, bandwidth or latency figure: vs_baseline is null",
}


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
    pk = _peaks()
    hbm_peak, tf_peak, kind = pk["hbm"], pk["tf"], pk["kind"]
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
    ap.add_argument("--ref-seconds", type=float, default=100.0,
                    help="--impl reference: CPU seconds the whole run (warm-up and timed steps) is sized for")
    ap.add_argument("--write-scale", type=float, default=None, help="override the write score scale")
    ap.add_argument("--stream-tokens", type=int, default=256,
                    help="tokens per sequence pushed by one step of a stream workload")
    ap.add_argument("--write-eps", type=float, default=0.0, help="override write_eps (0 = library default 2^-24)")
    ap.add_argument("--flags", type=int, default=None,
                    help="BCT_FLAG_* bits for the cache (default: 0 for decode workloads; PRECISE_READ | OUT_F32 = 24 for "
                         "stream workloads, the setting at which the full 131072-token stream stays within 2e-2)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch (profiling on a smaller case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short run of the diffuse write regime")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle replay of the timed launch configuration")
    ap.add_argument("--repeats", type=int, default=5, help="timed blocks of --steps steps (median and spread are reported)")
    ap.add_argument("--update-kv", action="store_true",
                    help="stream workloads: time bct_update_kv (Algorithm 1's UpdateKV, state only) instead of bct_prefill_stream")
    ap.add_argument("--update-kv-backward", action="store_true",
                    help="stream workloads: time bct_update_kv_backward (gradients of UpdateKV's token-parallel form)")
    ap.add_argument("--project-tokens", type=int, default=0,
                    help="time bct_project_qkv alone on this many tokens (the workload gives the head counts)")
    ap.add_argument("--d-model", type=int, default=4096, help="model width of the projections")
    args = ap.parse_args()
    w = W.CONFIGS[args.workload]
    default_run = (args.workload == "mha7b_b64_c2048" and args.write_scale is None and args.batch is None and
                   args.flags is None and args.write_eps == 0.0)
    if args.flags is None:
        args.flags = 24 if (w.api == "stream" and not args.update_kv and not args.update_kv_backward) else 0
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
    stream = (w.api == "stream")
    tok_per_step = args.stream_tokens if stream else 1   # tokens per sequence in one step
    cache = make_cache(B, w, wr, dev, flags=args.flags, write_eps=args.write_eps,
                       max_stream=(args.stream_tokens if stream else 1))
    if stream:
        # fill the cache (untimed), then every step pushes one block of tokens through bct_prefill_stream
        t_fill = fill_stream_cache(cache, wr, dev)
        pool = [W.stream_inputs(wr, t_fill + i * tok_per_step, tok_per_step, dev) for i in range(8)]
    else:
        pool = [W.step_inputs(wr, t, dev) for t in range(min(args.steps + args.warmup, 64))]
    outs = [torch.empty_like(pool[0][0], dtype=cache.out_dtype) for _ in range(2)]

    update_only = stream and (args.update_kv or args.update_kv_backward)
    backward = stream and args.update_kv_backward
    if backward:   # G = dL/dMV_N and the gradient tensors, allocated once
        gen = torch.Generator(device=dev).manual_seed(wr.seed + 77)
        d_mv = torch.randn((w.batch, w.n_kv_heads, w.capacity, w.head_dim), generator=gen, device=dev).to(torch.bfloat16)
        f32 = dict(dtype=torch.float32, device=dev)
        grads = (torch.empty(tuple(pool[0][1].shape), **f32), torch.empty(tuple(pool[0][2].shape), **f32),
                 torch.empty(tuple(d_mv.shape), **f32), torch.empty((w.batch, tok_per_step, w.n_kv_heads), **f32))

    def step_dev(i):
        if backward:
            cache.update_kv_backward(pool[i % len(pool)][1], pool[i % len(pool)][2], d_mv, out=grads)
        elif update_only:
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

    # ---------- device-resident timing: W warm-up steps, then exactly K timed steps ----------
    for i in range(args.warmup):
        step_dev(i)
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = cache.launches
    rows0 = cache.rows_rewritten()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step_dev(args.warmup + i)
    e1.record()
    sync_all()
    ms_total = e0.elapsed_time(e1)
    launches = cache.launches - launches0
    rows1 = cache.rows_rewritten()
    # further blocks of K steps: the spread tells how far a single short block can be trusted
    rep_ms = [ms_total / args.steps]
    for r in range(max(0, args.repeats - 1)):
        sync_all()
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ea.record()
        for i in range(args.steps):
            step_dev(args.warmup + (r + 1) * args.steps + i)
        eb.record()
        sync_all()
        rep_ms.append(ea.elapsed_time(eb) / args.steps)
    clocks = sampler.stop() if rank == 0 else None
    cache.check_status()

    # ---------- end to end through the host-buffer entry point ----------
    hpool = [tuple(x.cpu().pin_memory() for x in pool[i]) for i in range(min(len(pool), 16))]
    hout = [torch.empty_like(hpool[0][0], dtype=cache.out_dtype).pin_memory() for _ in range(2)]
    hgrad = torch.empty(tuple(grads[0].shape), dtype=torch.float32).pin_memory() if backward else None

    def step_host(i):
        if backward:      # no host-buffer form: inputs up, the call, one gradient tensor down
            xs = [x.to(dev, non_blocking=True) for x in hpool[i % len(hpool)][1:]]
            cache.update_kv_backward(xs[0], xs[1], d_mv, out=grads)
            hgrad.copy_(grads[0], non_blocking=True)
        elif update_only:   # no host-buffer form of UpdateKV: the stream call without outputs
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
    d2h = hgrad.numel() * 4 if backward else (0 if update_only else hout[0].numel() * hout[0].element_size())

    if world > 1:
        ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dev)
        rep_ms = max_over_ranks(rep_ms, dev)

    line = None
    if rank == 0:
        ms_step = ms_total / args.steps
        tokens = w.batch * world * args.steps * tok_per_step
        if stream:
            roof = stream_roofline(w, tok_per_step, ms_step, precise=bool(args.flags & 16), write_only=update_only,
                                   backward=backward)
        else:
            rows = max(0, rows1 - rows0)
            w_frac = rows / float(max(1, w.units * args.steps * w.capacity))
            alg = algorithmic_bytes_per_step(w, w_frac)
            pk = _peaks()
            achieved = alg / (ms_step * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": achieved, "peak": pk["hbm"], "unit": "GB/s", "frac": achieved / pk["hbm"],
                    "traffic": measured_traffic(w, cache.tensor_path), "peak_kind": "of " + pk["kind"],
                    "kernel": "decode_tc_kernel" if cache.tensor_path else "decode_kernel",
                    "algorithmic_bytes_per_launch": alg, "rows_rewritten_fraction": w_frac,
                    "rows_rewritten_per_unit_step": rows / float(max(1, w.units * args.steps)),
                    "frac_of_8TBps_nominal": achieved / 8000.0}
        srt = sorted(rep_ms)
        cfg = config_of(w, tok_per_step)
        run = {"call": "bct_update_kv_backward" if backward else "bct_update_kv" if update_only else (
                   "bct_prefill_stream" if stream else "bct_decode_step"),
               "flags": args.flags, "parallelism": "independent units; replicas per GPU" if world > 1 else "1 GPU"}
        line = {
            "metric": METRIC, "value": tokens / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if w.dtype == "f32" else "bf16 cache, f32 accumulate",
            "data": "synthetic", "config": cfg, "run": run, "clocks": clocks,
            "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches,
            "roofline": roof,
            "repeats": {"blocks": len(rep_ms), "steps_per_block": args.steps, "ms_per_step": rep_ms,
                        "median_ms_per_step": srt[len(srt) // 2], "min_ms_per_step": srt[0], "max_ms_per_step": srt[-1],
                        "median_value": w.batch * world * tok_per_step / (srt[len(srt) // 2] * 1e-3)},
            "paper_context": PAPER_CONTEXT,
        }
        if world == 1 and not stream and args.write_scale is None and not args.no_secondary:
            line["secondary_write_regime"] = secondary_regime(B, w, wr, dev, pool, outs)
    cache.destroy()
    del cache, pool, outs
    torch.cuda.empty_cache()
    if rank == 0 and world == 1:
        if not args.no_parity and not update_only:
            # the launch configuration that was timed, replayed from the initial state beside the oracle
            n_par = (w.capacity + 2 * tok_per_step) if stream else min(args.warmup + args.steps, 48)
            line["parity"] = parity_check(B, w, wr, dev, args.flags, n_par, n_units=8,
                                          stream_tokens=tok_per_step if stream else 0)
        if default_run and not args.no_per_config:
            per = []
            # the single-sequence float configuration: one unit of 64 KiB, a latency measurement (its roofline fraction
            # says how far a lone unit is from streaming, not how good the kernel is)
            per.append(run_config(B, "single_fp32_c128", dev, steps=200))
            for name in ("gqa8b_b128_c4096", "sweep_b256_c256", "sweep_b256_c1024", "sweep_b256_c4096",
                         "sweep_b256_c16384"):
                per.append(run_config(B, name, dev))
            # the long-stream configuration at the flags its full-length parity test needs, and at the default
            # flags, whose bfloat16 output and value-plane read leave 2e-2 late in the stream
            per.append(run_config(B, "stream_b8_c1024", dev, steps=50, flags=24))
            dflt = run_config(B, "stream_b8_c1024", dev, steps=50, flags=0, with_parity=False)
            dflt["note"] = "default flags: outside 2e-2 over the full 131072-token stream (0.04 max-abs); within it early on"
            per.append(dflt)
            line["per_config"] = per
            line["stream_constancy"] = stream_constancy(B, W.CONFIGS["stream_b8_c1024"], dev, 24)
        if not args.no_cpu_baseline:
            cb = cpu_oracle_sample(w)
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    if rank == 0:
        print(json.dumps(line))
        if line.get("parity") is not None and not line["parity"]["pass"]:
            sys.stderr.write("bench: parity against the oracle is out of tolerance\n")
            sys.exit(3)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
