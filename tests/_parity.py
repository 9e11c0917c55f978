"""Shared harness of the GPU parity tests: run a workload through the C-ABI library on the
device and through the CPU oracle on a subset of (sequence, kv-head) units, on the same
seeded, dtype-rounded inputs, and compare element by element.  Units are independent, so
a subset is exact for those units."""
from __future__ import annotations

import numpy as np
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import workloads as W

TOL = {"f32": 1e-5, "bf16": 2e-2}  # max-abs bars of the benchmark contract


def pick_units(w: W.Workload, n: int, seed: int = 0):
    """First, last and a seeded sample of units, as (b, h) pairs."""
    U = w.units
    if U <= n:
        ids = list(range(U))
    else:
        rng = np.random.default_rng(seed)
        ids = sorted(set([0, U - 1] + rng.choice(U, size=n - 2, replace=False).tolist()))
    return [(u // w.n_kv_heads, u % w.n_kv_heads) for u in ids]


def _unit_slices(w, units, q, k, v):
    """q [B,(T,)Hq,d], k/v [B,(T,)Hkv,d] on device -> float64 numpy [n,T,G,d], [n,T,1,d]."""
    G = w.group
    if q.dim() == 3:
        q, k, v = q[:, None], k[:, None], v[:, None]
    qs = torch.stack([q[b, :, h * G:(h + 1) * G] for b, h in units]).double().cpu().numpy()
    ks = torch.stack([k[b, :, h:h + 1] for b, h in units]).double().cpu().numpy()
    vs = torch.stack([v[b, :, h:h + 1] for b, h in units]).double().cpu().numpy()
    return qs, ks, vs


def make_pair(w: W.Workload, units, device="cuda", flags=0, oracle_flags=0, write_eps=0.0, max_stream=1,
              oracle_write_eps=0.0):
    """(gpu cache, oracle cache over `units`) from the workload's seeded initial state.  write_eps = 0 leaves
    the library at its default threshold of 2^-24, which the oracle's exact rule (oracle_write_eps = 0) is
    compared with; a test of the threshold itself passes the same value to both."""
    mk = mv = None
    ok = ov = None
    if w.init_len:
        mk, mv = W.initial_cache(w, device)
        ok = torch.stack([mk[b, h] for b, h in units])[:, None].double().cpu().numpy()
        ov = torch.stack([mv[b, h] for b, h in units])[:, None].double().cpu().numpy()
    gpu = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype,
                  read_scale=w.read_scale, write_scale=w.write_scale, init_len=w.init_len, flags=flags,
                  write_eps=write_eps, max_stream=max_stream, mk_init=mk, mv_init=mv, device=device, guard_bytes=4096)
    torch.cuda.synchronize()
    del mk, mv
    ora = O.OracleCache(len(units), w.group, 1, w.head_dim, w.capacity, read_scale=w.read_scale,
                        write_scale=w.write_scale, init_len=w.init_len, mk_init=ok, mv_init=ov,
                        flags=oracle_flags, write_eps=oracle_write_eps)
    return gpu, ora


def compare_out(w, units, out_gpu, out_ref):
    """out_gpu device [B,(T,)Hq,d]; out_ref numpy [n,T,G,d].  Returns max-abs error."""
    G = w.group
    if out_gpu.dim() == 3:
        out_gpu = out_gpu[:, None]
    got = torch.stack([out_gpu[b, :, h * G:(h + 1) * G] for b, h in units]).double().cpu().numpy()
    assert np.isfinite(got).all()
    return float(np.abs(got - out_ref).max())


def compare_state(w, units, gpu, ora):
    """Max-abs error of the exported MV (and exact equality of MK) on the checked units."""
    k, v = gpu.export(torch.float32)
    torch.cuda.synchronize()
    gpu.check_guards()   # nothing wrote outside the workspace (0xA5 bands on either side of it)
    n = ora.len
    assert gpu.len == n
    err = 0.0
    for i, (b, h) in enumerate(units):
        kk = k[b, h].double().cpu().numpy()
        vv = v[b, h].double().cpu().numpy()
        assert np.array_equal(kk[:n], ora.MK[i, :n]), "MK must be bit-identical (never rewritten)"
        assert not kk[n:].any() and not vv[n:].any()
        err = max(err, float(np.abs(vv[:n] - ora.MV[i, :n]).max()))
    del k, v
    return err


def run_decode_parity(w: W.Workload, units, steps=None, device="cuda", expect_tensor_path=None, **kw):
    """Step both sides token by token; return (max out error, state error)."""
    steps = w.steps if steps is None else steps
    gpu, ora = make_pair(w, units, device, **kw)
    if expect_tensor_path is not None:
        assert gpu.tensor_path == expect_tensor_path
    worst = 0.0
    for t in range(steps):
        q, k, v = W.step_inputs(w, t, device)
        out = gpu.decode_step(q, k, v)
        qs, ks, vs = _unit_slices(w, units, q, k, v)
        ref = ora.prefill_stream(qs, ks, vs)
        worst = max(worst, compare_out(w, units, out, ref))
    gpu.check_status()
    state = compare_state(w, units, gpu, ora)
    gpu.destroy()
    return worst, state
