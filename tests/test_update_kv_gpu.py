"""GPU parity of bct_update_kv (Algorithm 1's procedure UpdateKV: state only, chunks of up to 128
tokens on the tensor path) against the CPU oracle and against the stream call without outputs."""
import numpy as np
import pytest
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

from _parity import TOL, compare_state, make_pair, pick_units, _unit_slices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    bld.build()
    B.load()


@pytest.mark.parametrize("G,C,T,with_eta,write_scale", [
    (1, 512, 256, False, 1.0),      # two whole chunks of 128
    (1, 1024, 300, True, 1.0),      # two whole chunks and a ragged one (44 tokens in a chunk of 48)
    (4, 333, 100, False, 1.0),      # ragged capacity; one short chunk only (100 tokens in 112)
    (2, 2048, 129, True, 1.0),      # 16 tiles; one whole chunk and a single token in a chunk of 16
    (1, 256, 384, False, 128 ** -0.5),   # diffuse write weights: every row gains from every token
])
def test_update_kv_matches_oracle(G, C, T, with_eta, write_scale):
    d = 128
    w = W.Workload("t", 2, 2 * G, 2, d, C, "bf16", C, T, 97, d ** -0.5, 1.0, 1.0, "stream", 1.0, write_scale)
    units = pick_units(w, 4)
    gpu, ora = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    eta = None
    if with_eta:
        g = torch.Generator(device="cpu").manual_seed(19)
        eta = (torch.rand((w.batch, T, w.n_kv_heads), generator=g) * 2.0 - 0.25).cuda()
    gpu.update_kv(k, v, eta=eta)
    gpu.check_status()
    _, uk, uv = _unit_slices(w, units, q, k, v)
    ueta = None if eta is None else torch.stack([eta[b, :, h] for b, h in units])[:, :, None].double().cpu().numpy()
    ora.update_kv(uk, uv, eta=ueta)
    tol = 1e-3 if write_scale < 1.0 else TOL["bf16"]
    assert compare_state(w, units, gpu, ora) <= tol
    assert gpu.len == C
    gpu.destroy()


def test_update_kv_with_more_units_than_ctas_deals_the_chunks_round_the_ctas():
    # 160 units, three chunks of 128 tokens: the (unit, chunk) pairs go chunk-major (4 turns on 148 CTAs instead of 6),
    # so a unit's state is handed from CTA to CTA between its chunks
    d, C, T = 128, 256, 384
    w = W.Workload("t", 80, 2, 2, d, C, "bf16", C, T, 103, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    units = pick_units(w, 16)
    gpu, ora = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    gpu.update_kv(k, v)
    gpu.check_status()
    _, uk, uv = _unit_slices(w, units, q, k, v)
    ora.update_kv(uk, uv)
    assert compare_state(w, units, gpu, ora) <= TOL["bf16"]
    gpu.destroy()


def test_update_kv_tracks_the_stream_call_and_continues_it():
    d, C, T = 128, 512, 200
    w = W.Workload("t", 2, 2, 2, d, C, "bf16", C, 2 * T, 101, d ** -0.5, 1.0, 1.0, "stream")
    units = pick_units(w, 4)
    a, ora = make_pair(w, units)
    b, _ = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, 2 * T, "cuda")
    # a: UpdateKV on the first half, the stream call (with outputs) on the second; b: the stream call on both
    a.update_kv(k[:, :T].contiguous(), v[:, :T].contiguous())
    oa = a.prefill_stream(q[:, T:].contiguous(), k[:, T:].contiguous(), v[:, T:].contiguous())
    b.prefill_stream(q[:, :T].contiguous(), k[:, :T].contiguous(), v[:, :T].contiguous(), want_out=False)
    ob = b.prefill_stream(q[:, T:].contiguous(), k[:, T:].contiguous(), v[:, T:].contiguous())
    va, vb = a.export()[1].double(), b.export()[1].double()
    assert float((va - vb).abs().max()) <= 2e-3
    assert float((oa.double() - ob.double()).abs().max()) <= TOL["bf16"]
    uq, uk, uv = _unit_slices(w, units, q, k, v)
    ora.prefill_stream(uq, uk, uv, want_out=False)
    assert compare_state(w, units, a, ora) <= TOL["bf16"]
    a.destroy()
    b.destroy()


def test_update_kv_refuses_what_it_does_not_serve():
    d = 128
    w = W.Workload("t", 2, 2, 2, d, 256, "bf16", 200, 8, 103, d ** -0.5, 1.0, 1.0, "stream")
    gpu, _ = make_pair(w, pick_units(w, 2))
    q, k, v = W.stream_inputs(w, 0, 8, "cuda")
    with pytest.raises(B.BctError) as e:
        gpu.update_kv(k, v)              # the cache is still filling
    assert e.value.status == B.BCT_ERR_STATE
    gpu.destroy()
    w = W.Workload("t", 1, 2, 1, 64, 128, "f32", 128, 8, 105, 0.125, 0.125, 1.0, "stream")
    gpu, _ = make_pair(w, pick_units(w, 1))
    q, k, v = W.stream_inputs(w, 0, 8, "cuda")
    with pytest.raises(B.BctError) as e:
        gpu.update_kv(k, v)              # float cache: not on the tensor path
    assert e.value.status == B.BCT_ERR_UNSUPPORTED
    gpu.destroy()
