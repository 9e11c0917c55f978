"""GPU parity of the projections in front of the layer (bct_project_qkv: wq_t = W_wq x_t,
wv_t = W_wv x_t, read query) and of the fused layer call against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

from _parity import TOL, compare_out, compare_state, make_pair, pick_units

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    bld.build()
    B.load()


def _weights(n_q, n_kv, d_model, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    s = d_model ** -0.5
    mk = lambda n: (torch.randn((n, d_model), generator=g) * s).to(torch.bfloat16).cuda()
    return mk(n_q), mk(n_kv), mk(n_kv)


def _tokens(shape, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).cuda()


# fp32 accumulation of bfloat16 products, then one rounding to bfloat16: |y| is O(1), so the error is
# half a bfloat16 ulp of the result (2^-9 |y|) plus the accumulation error (<< 1e-3 at these depths)
def _proj_tol(ref):
    return 2.0 ** -8 * np.abs(ref) + 2e-3


@pytest.mark.parametrize("M,d_model,n_q,n_kv", [
    (64, 512, 256, 128),        # a decode step: 32-feature tiles, one row tile with rows past the last token
    (1, 64, 32, 32),            # a single token, one stage of depth
    (77, 1032, 96, 32),         # ragged tokens, d_model not a multiple of 64 (zero-filled columns)
    (300, 256, 256, 128),       # 128-feature tiles, three row tiles, ragged last one
    (1024, 2048, 512, 256),     # many tiles per CTA ring wrap (32 k-blocks)
    (257, 128, 160, 64),        # more than 256 tokens but features not multiples of 128: 32-feature tiles
])
def test_project_qkv_matches_oracle(M, d_model, n_q, n_kv):
    w_q, w_wq, w_wv = _weights(n_q, n_kv, d_model, 3)
    x = _tokens((M, d_model), 5)
    q, k, v = B.project_qkv(x, w_q, w_wq, w_wv)
    torch.cuda.synchronize()
    xd = x.double().cpu().numpy()
    for got, w in ((q, w_q), (k, w_wq), (v, w_wv)):
        ref = O.project(xd, w.double().cpu().numpy())
        g = got.double().cpu().numpy()
        assert g.shape == ref.shape
        assert np.isfinite(g).all()
        assert (np.abs(g - ref) <= _proj_tol(ref)).all(), float(np.abs(g - ref).max())


def test_project_qkv_rejects_bad_shapes():
    w_q, w_wq, w_wv = _weights(64, 32, 64, 7)
    x = _tokens((4, 64), 9)
    lib = B.load()
    q = torch.empty((4, 64), dtype=torch.bfloat16, device="cuda")
    k = torch.empty((4, 32), dtype=torch.bfloat16, device="cuda")
    args = (x.data_ptr(), w_q.data_ptr(), w_wq.data_ptr(), w_wv.data_ptr(), q.data_ptr(), k.data_ptr(), k.data_ptr(), None)
    assert lib.bct_project_qkv(0, 64, 64, 32, *args) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_project_qkv(4, 60, 64, 32, *args) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_project_qkv(4, 64, 48, 32, *args) == B.BCT_ERR_UNSUPPORTED
    assert lib.bct_project_qkv(4, 64, 64, 32, x.data_ptr() + 2, *args[1:]) == B.BCT_ERR_INVALID_ARG
    assert "aligned" in B.last_error()


@pytest.mark.parametrize("G,C,init_len,T,d_model,with_eta", [
    (1, 512, 512, 96, 256, False),      # full cache: one chunk of 64 and 32 single tokens behind the projections
    (4, 640, 600, 80, 512, True),       # fill chunks, then soft writes, with step sizes
])
def test_layer_forward_matches_oracle(G, C, init_len, T, d_model, with_eta):
    d, Hkv, Bt = 128, 2, 2
    w = W.Workload("t", Bt, Hkv * G, Hkv, d, C, "bf16", init_len, T, 91, d ** -0.5, 1.0, 1.0, "stream")
    units = pick_units(w, 4)
    gpu, ora_units = make_pair(w, units)
    # the oracle runs every unit here: the projections mix all heads of a token
    mk, mv = W.initial_cache(w, "cuda")
    ora = O.OracleCache(Bt, Hkv * G, Hkv, d, C, read_scale=w.read_scale, write_scale=w.write_scale, init_len=init_len,
                        mk_init=mk.double().cpu().numpy(), mv_init=mv.double().cpu().numpy())
    w_q, w_wq, w_wv = _weights(Hkv * G * d, Hkv * d, d_model, 11)
    # tokens scaled so that the read scores stay O(1) and the write scores as peaked as the benchmark's
    x = _tokens((Bt, T, d_model), 13)
    w_q = (w_q.float() * d ** -0.5).to(torch.bfloat16)
    eta = None
    if with_eta:
        g = torch.Generator(device="cpu").manual_seed(17)
        eta = (torch.rand((Bt, T, Hkv), generator=g) * 1.5).cuda()
    out = gpu.layer_forward(x, w_q, w_wq, w_wv, eta=eta)
    gpu.check_status()
    q, k, v = O.layer_step_inputs(x.double().cpu().numpy(), w_q.double().cpu().numpy(), w_wq.double().cpu().numpy(),
                                  w_wv.double().cpu().numpy(), Hkv * G, Hkv, d)
    ref = ora.prefill_stream(q, k, v, eta=None if eta is None else eta.double().cpu().numpy())
    got = out.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert float(np.abs(got - ref).max()) <= TOL["bf16"]
    k_gpu, v_gpu = gpu.export()
    assert float(np.abs(v_gpu.double().cpu().numpy() - ora.values()).max()) <= TOL["bf16"]
    # keys appended during the fill phase are the projected write queries, up to one bfloat16 rounding
    assert float(np.abs(k_gpu.double().cpu().numpy() - ora.keys()).max()) <= 2.0 ** -7 * float(np.abs(ora.keys()).max())
    gpu.destroy()
