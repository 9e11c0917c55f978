"""GPU parity of the per-token step size (bct_decode_step_eta / bct_prefill_stream_eta:
MV_t = MV_{t-1} + eta_t ww_t^T wv_t) against the CPU oracle, on all three kernels."""
import numpy as np
import pytest
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

from _parity import TOL, compare_out, compare_state, make_pair, pick_units, _unit_slices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    bld.build()
    B.load()


def _eta(w, T, seed, lo=-0.5, hi=2.0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.rand((w.batch, T, w.n_kv_heads), generator=g) * (hi - lo) + lo).cuda()


def _eta_units(w, units, eta):
    return torch.stack([eta[b, :, h] for b, h in units])[:, :, None].double().cpu().numpy()


@pytest.mark.parametrize("dtype,d,G,C,init_len,T,flags,oflags,tc", [
    ("bf16", 128, 1, 512, 512, 12, 0, 0, True),                      # tensor-core decode kernel
    ("bf16", 128, 4, 4224, 4224, 6, 0, 0, True),                     # cluster of 2, ragged slice
    ("bf16", 128, 2, 384, 380, 10, B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ, True),   # 4 fill tokens ignore eta
    ("bf16", 128, 1, 256, 256, 8, B.FLAG_CUDA_CORES, 0, False),      # CUDA-core kernel, bfloat16
    ("f32", 64, 2, 200, 200, 16, B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ, False),    # float cache
    ("f32", 64, 1, 3000, 3000, 5, 0, 0, False),                      # float cache over a cluster
])
def test_decode_step_eta_matches_oracle(dtype, d, G, C, init_len, T, flags, oflags, tc):
    w = W.Workload("t", 3, 2 * G, 2, d, C, dtype, init_len, T, 71, d ** -0.5, 1.0, 1.0, "decode", 1.0, 0.5)
    units = pick_units(w, 6)
    gpu, ora = make_pair(w, units, flags=flags, oracle_flags=oflags)
    assert gpu.tensor_path == tc
    eta = _eta(w, T, 5)
    worst = 0.0
    for t in range(T):
        q, k, v = W.step_inputs(w, t, "cuda")
        out = gpu.decode_step(q, k, v, eta=eta[:, t].contiguous())
        uq, uk, uv = _unit_slices(w, units, q[:, None], k[:, None], v[:, None])
        ref = ora.prefill_stream(uq, uk, uv, eta=_eta_units(w, units, eta[:, t:t + 1]))
        worst = max(worst, compare_out(w, units, out, ref))
    gpu.check_status()
    assert worst <= TOL[dtype], worst
    assert compare_state(w, units, gpu, ora) <= TOL[dtype]
    gpu.destroy()


@pytest.mark.parametrize("G,C,init_len,T,flags,oflags", [
    (1, 512, 512, 200, 0, 0),                       # chunks of 64 + 8 single tokens
    (2, 384, 300, 150, B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),   # fill chunks, fill tokens, then full chunks
    (5, 1024, 1024, 40, B.FLAG_OUT_F32, 0),         # chunks of 16
])
def test_prefill_stream_eta_matches_oracle(G, C, init_len, T, flags, oflags):
    d = 128
    w = W.Workload("t", 2, 2 * G, 2, d, C, "bf16", init_len, T, 73, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    units = pick_units(w, 4)
    gpu, ora = make_pair(w, units, flags=flags, oracle_flags=oflags)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    eta = _eta(w, T, 7)
    out = gpu.prefill_stream(q, k, v, eta=eta)
    gpu.check_status()
    uq, uk, uv = _unit_slices(w, units, q, k, v)
    ref = ora.prefill_stream(uq, uk, uv, eta=_eta_units(w, units, eta))
    assert compare_out(w, units, out, ref) <= TOL["bf16"]
    assert compare_state(w, units, gpu, ora) <= TOL["bf16"]
    gpu.destroy()


def test_eta_of_ones_is_the_plain_call_bit_for_bit_and_zero_freezes_the_state():
    d, C, T = 128, 512, 96
    w = W.Workload("t", 2, 2, 2, d, C, "bf16", C, T, 79, d ** -0.5, 1.0, 1.0, "stream")
    units = pick_units(w, 4)
    a, _ = make_pair(w, units)
    b, _ = make_pair(w, units)
    z, _ = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    oa = a.prefill_stream(q, k, v)
    ob = b.prefill_stream(q, k, v, eta=torch.ones((2, T, 2), device="cuda"))
    assert torch.equal(oa, ob)
    assert all(torch.equal(x, y) for x, y in zip(a.export(v_dtype=torch.int32), b.export(v_dtype=torch.int32)))
    before = z.export(v_dtype=torch.int32)
    z.prefill_stream(q, k, v, eta=torch.zeros((2, T, 2), device="cuda"), want_out=False)
    for t in range(4):
        z.decode_step(q[:, t].contiguous(), k[:, t].contiguous(), v[:, t].contiguous(),
                      eta=torch.zeros((2, 2), device="cuda"))
    after = z.export(v_dtype=torch.int32)
    assert torch.equal(before[0], after[0])
    # value + residual of every row is unchanged (a rewritten row may re-split the same sum)
    def total(x):
        hi = (x & -65536).view(torch.float32)
        lo = (x << 16).view(torch.float32)
        return hi.double() + lo.double()
    assert torch.equal(total(before[1]), total(after[1]))
    for c in (a, b, z):
        c.destroy()


def test_eta_argument_checks():
    w = W.Workload("t", 2, 2, 2, 128, 256, "bf16", 256, 4, 83, 128 ** -0.5, 1.0, 1.0, "decode")
    gpu, _ = make_pair(w, pick_units(w, 2))
    q, k, v = W.step_inputs(w, 0, "cuda")
    with pytest.raises(ValueError):
        gpu.decode_step(q, k, v, eta=torch.ones((2, 3), device="cuda"))
    with pytest.raises(ValueError):
        gpu.decode_step(q, k, v, eta=torch.ones((2, 2), device="cuda", dtype=torch.float64))
    gpu.destroy()
