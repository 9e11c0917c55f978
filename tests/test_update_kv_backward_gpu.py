"""GPU parity of bct_update_kv_backward (backward of Algorithm 1's UpdateKV in its token-parallel form) against
the double-precision CPU oracle, through the C ABI, and of bct_stack_forward against the oracle layer by layer."""
import numpy as np
import pytest
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

pytestmark = pytest.mark.gpu

# bfloat16 operands (the write weights and dS are rounded once, relative 2^-9) with fp32 accumulation: every
# gradient is compared on the scale of its tensor, with the bar the forward's bfloat16 parity uses
REL_TOL = 2e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    bld.build()
    B.load()


def _f64(t):
    return t.double().cpu().numpy()


def _case(Bt, Hkv, C, T, seed, write_scale=1.0, with_eta=False, write_eps=0.0, flags=0):
    d = 128
    w = W.Workload("t", Bt, Hkv, Hkv, d, C, "bf16", C, T, seed, d ** -0.5, 1.0, 1.0, "stream", 1.0, write_scale)
    mk, mv = W.initial_cache(w, "cuda")
    gpu = B.Cache(Bt, Hkv, Hkv, d, C, torch.bfloat16, read_scale=1.0, write_scale=write_scale, init_len=C, mk_init=mk,
                  mv_init=mv, write_eps=write_eps, flags=flags)
    _, k, v = W.stream_inputs(w, 0, T, "cuda")
    g = torch.Generator(device="cpu").manual_seed(seed + 1)
    G = torch.randn((Bt, Hkv, C, d), generator=g).to(torch.bfloat16).cuda()
    eta = (torch.rand((Bt, T, Hkv), generator=g) * 1.5 + 0.1).cuda() if with_eta else None
    return gpu, mk, k, v, G, eta


def _check(gpu, mk, k, v, G, eta, write_scale, write_eps=0.0):
    d_wq, d_wv, d_mk, d_eta = gpu.update_kv_backward(k, v, G, eta=eta)
    gpu.check_status()
    ref = O.update_kv_backward(_f64(mk), _f64(k), _f64(v), _f64(G), eta=None if eta is None else _f64(eta),
                               write_scale=write_scale, write_eps=write_eps)
    errs = []
    for name, got, want in zip(("d_wq", "d_wv", "d_mk", "d_eta"), (d_wq, d_wv, d_mk, d_eta), ref):
        got = _f64(got)
        assert np.isfinite(got).all(), name
        scale = float(np.abs(want).max())
        err = float(np.abs(got - want).max())
        errs.append((name, err, scale))
        assert err <= REL_TOL * scale + 1e-6, (name, err, scale)
    return errs


@pytest.mark.parametrize("Bt,Hkv,C,T,write_scale,with_eta", [
    (2, 2, 512, 256, 1.0, False),          # four tiles, two token blocks: dMK sums over the blocks
    (1, 3, 333, 100, 1.0, True),           # ragged capacity and a ragged token block
    (2, 2, 1024, 300, 1.0, True),          # the long-stream capacity; three token blocks, the last one ragged
    (1, 2, 128, 5, 1.0, False),            # one tile, five tokens
    (2, 1, 2048, 128, 128 ** -0.5, True),  # diffuse write weights over 16 tiles
    (1, 2, 640, 200, 0.3, False),          # in between
])
def test_update_kv_backward_matches_oracle(Bt, Hkv, C, T, write_scale, with_eta):
    gpu, mk, k, v, G, eta = _case(Bt, Hkv, C, T, 201, write_scale, with_eta)
    n0 = gpu.launches
    _check(gpu, mk, k, v, G, eta, write_scale)
    assert gpu.launches == n0 + 1 and gpu.len == C
    # the cache itself is only read
    k_after, _ = gpu.export()
    assert torch.equal(k_after, mk)
    gpu.destroy()


def test_update_kv_backward_with_a_write_threshold_and_without_optional_outputs():
    Bt, Hkv, C, T, ws, eps = 1, 2, 384, 130, 0.35, 1e-3
    gpu, mk, k, v, G, eta = _case(Bt, Hkv, C, T, 211, ws, True, write_eps=eps)
    _check(gpu, mk, k, v, G, eta, ws, write_eps=eps)
    # the threshold matters here: the exact rule's gradient is measurably different
    exact = O.update_kv_backward(_f64(mk), _f64(k), _f64(v), _f64(G), eta=_f64(eta), write_scale=ws)
    thr = O.update_kv_backward(_f64(mk), _f64(k), _f64(v), _f64(G), eta=_f64(eta), write_scale=ws, write_eps=eps)
    assert float(np.abs(exact[1] - thr[1]).max()) > 1e-2
    a = gpu.update_kv_backward(k, v, G, eta=eta, want_d_mk=False, want_d_eta=False)
    b = gpu.update_kv_backward(k, v, G, eta=eta)
    assert a[2] is None and a[3] is None
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])      # d_wq and d_wv do not go through atomics
    gpu.destroy()


def test_update_kv_backward_is_consistent_with_the_forward_kernel():
    # directional derivative: <G, MV_N(v + h dv) - MV_N(v - h dv)> / 2h against <d_wv, dv>, both on the GPU
    # (the forward is linear in wv, so the difference quotient is exact up to the state's rounding)
    Bt, Hkv, C, T = 2, 2, 256, 128
    gpu, mk, k, v, G, _ = _case(Bt, Hkv, C, T, 221)
    _, d_wv, _, _ = gpu.update_kv_backward(k, v, G)
    g = torch.Generator(device="cpu").manual_seed(5)
    dv = torch.randn(v.shape, generator=g).to(torch.bfloat16).cuda()
    vals = []
    for sgn in (+1.0, -1.0):
        c = B.Cache(Bt, Hkv, Hkv, 128, C, torch.bfloat16, read_scale=1.0, write_scale=1.0, init_len=C, mk_init=mk)
        c.update_kv(k, (sgn * dv).to(torch.bfloat16))          # MV_0 = 0: the state is the increment of dv alone
        vals.append(float((c.export(torch.float32)[1].double() * G.double()).sum()))
        c.destroy()
    lhs = (vals[0] - vals[1]) / 2.0
    rhs = float((d_wv.double() * dv.double()).sum())
    assert abs(lhs - rhs) <= 1e-2 * max(1.0, abs(rhs)), (lhs, rhs)
    gpu.destroy()


def test_update_kv_backward_refuses_what_it_does_not_serve():
    d = 128
    w = W.Workload("t", 1, 2, 2, d, 256, "bf16", 200, 8, 103, d ** -0.5, 1.0, 1.0, "stream")
    mk, mv = W.initial_cache(w, "cuda")
    gpu = B.Cache(1, 2, 2, d, 256, torch.bfloat16, init_len=200, mk_init=mk, mv_init=mv)
    _, k, v = W.stream_inputs(w, 0, 8, "cuda")
    G = torch.zeros((1, 2, 256, d), dtype=torch.bfloat16, device="cuda")
    n0 = gpu.launches
    with pytest.raises(B.BctError) as e:
        gpu.update_kv_backward(k, v, G)            # the cache is still filling
    assert e.value.status == B.BCT_ERR_STATE and gpu.launches == n0
    gpu.destroy()
    c = B.Cache(1, 1, 1, 64, 128, torch.float32)
    z = torch.zeros(1, 4, 1, 64, device="cuda")
    p = z.data_ptr()
    assert c.lib.bct_update_kv_backward(c._h, p, p, None, p, 4, p, p, None, None, None) in (B.BCT_ERR_STATE, B.BCT_ERR_UNSUPPORTED)
    assert c.lib.bct_update_kv_backward(c._h, p, p, None, None, 4, p, p, None, None, None) == B.BCT_ERR_INVALID_ARG
    c.destroy()


def test_stack_of_two_layers_matches_the_oracle_layer_by_layer():
    # layer 0: 4 query heads over 2 kv-heads on tokens of width 256; layer 1 reads layer 0's outputs (width 4 * 128)
    # with other head counts and another capacity; both start empty, so the call runs fill chunks, then soft writes
    Bt, T, d = 2, 200, 128
    shapes = [(4, 2, 128, 256), (2, 2, 256, 4 * 128)]          # (Hq, Hkv, C, d_model) per layer
    g = torch.Generator(device="cpu").manual_seed(31)
    x = torch.randn((Bt, T, 256), generator=g).to(torch.bfloat16).cuda()
    caches, oracles, wq, wwq, wwv = [], [], [], [], []
    h1_dev = None
    for l, (Hq, Hkv, C, dm) in enumerate(shapes):
        # layer 1's tokens are layer 0's attention outputs: its weights are scaled by their measured size, so that
        # its write queries and values are of unit scale like the benchmark's (and the 2e-2 bar means the same)
        s_in = 1.0 if l == 0 else 1.0 / float(h1_dev.float().pow(2).mean().sqrt())
        mkw = lambda n, s: (torch.randn((n, dm), generator=g) * s).to(torch.bfloat16).cuda()
        wq.append(mkw(Hq * d, s_in * dm ** -0.5 * d ** -0.5))
        wwq.append(mkw(Hkv * d, s_in * dm ** -0.5))
        wwv.append(mkw(Hkv * d, s_in * dm ** -0.5))
        caches.append(B.Cache(Bt, Hq, Hkv, d, C, torch.bfloat16, read_scale=1.0, write_scale=1.0))
        oracles.append(O.OracleCache(Bt, Hq, Hkv, d, C, read_scale=1.0, write_scale=1.0))
        if l == 0:
            # Layer 0 alone on a twin cache gives the tokens layer 1 reads, bit for bit (the stack is the composition
            # of bct_layer_forward calls).  Each layer is held to the 2e-2 bar on ITS inputs: the oracle's layer 1
            # reads the device's layer-0 outputs, so that one layer's rounding is not counted against the next.
            twin = B.Cache(Bt, Hq, Hkv, d, C, torch.bfloat16, read_scale=1.0, write_scale=1.0)
            h1_dev = twin.layer_forward(x, wq[0], wwq[0], wwv[0])
            twin.destroy()
    out = B.stack_forward(caches, x, wq, wwq, wwv)
    for c in caches:
        c.check_status()
    h = _f64(x)
    for l, (Hq, Hkv, C, dm) in enumerate(shapes):
        q, k, v = O.layer_step_inputs(h, _f64(wq[l]), _f64(wwq[l]), _f64(wwv[l]), Hq, Hkv, d)
        o = oracles[l].prefill_stream(q, k, v)
        # The projections round to bfloat16 from an fp32 sum on the device and from a double sum in the oracle: an
        # element that sits near a rounding boundary lands one bfloat16 step apart, and a token that attends mostly
        # to itself hands that step of its write value straight to the output.  The bar allows for one such step.
        ulp = 2.0 ** (np.floor(np.log2(np.abs(v).max())) - 7)
        assert caches[l].len == min(T, C) == oracles[l].len
        state = float(np.abs(_f64(caches[l].export(torch.float32)[1]) - oracles[l].values()).max())
        assert state <= 2e-2 + ulp, (l, state)
        if l == 0:
            assert float(np.abs(_f64(h1_dev) - o).max()) <= 2e-2 + ulp
            h = _f64(h1_dev).reshape(Bt, T, Hq * d)
    err = float(np.abs(_f64(out) - o).max())
    assert err <= 2e-2 + ulp, (err, ulp)
    # one layer through the stack call is bct_layer_forward itself
    one = B.Cache(Bt, 4, 2, d, 128, torch.bfloat16, read_scale=1.0, write_scale=1.0)
    two = B.Cache(Bt, 4, 2, d, 128, torch.bfloat16, read_scale=1.0, write_scale=1.0)
    a = B.stack_forward([one], x, wq[:1], wwq[:1], wwv[:1])
    b = two.layer_forward(x, wq[0], wwq[0], wwv[0])
    assert torch.equal(a, b)
    # refused before anything is enqueued: the same cache twice, a float-output layer
    n0 = one.launches
    with pytest.raises(B.BctError):
        B.stack_forward([one, one], x, wq, wwq, wwv)
    f32out = B.Cache(Bt, 2, 2, d, 256, torch.bfloat16, flags=B.FLAG_OUT_F32)
    with pytest.raises(B.BctError):
        B.stack_forward([one, f32out], x, wq, wwq, wwv)
    assert one.launches == n0
    for c in caches + [one, two, f32out]:
        c.destroy()
