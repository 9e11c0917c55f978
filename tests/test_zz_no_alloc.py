"""bct_prefill_stream_host_static: the stream call for callers that cannot allocate device memory.

Some users of this library can never call cudaMalloc once they are running: a serving loop whose
memory pool was frozen at start-up, a plug-in that only owns the arena its host gave it, a process
in which other libraries hold the rest of the device.  They cannot enlarge the staging area that
bct_prefill_stream_host keeps in the workspace (sized by max_stream at create).  The static entry
point stages the step vectors in a device array built into the library instead.  This test calls
it through the C ABI twice in a row and compares each result with the ordinary entry point's, and
checks that a request beyond the built-in array's size is refused with a message.

The file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import pytest
import torch

from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2  # the max-abs bar the other bfloat16 parity tests use


def _pinned(t):
    return t.cpu().pin_memory()


def test_static_staging_matches_workspace_staging_on_two_calls_in_a_row():
    bld.build()
    B.load()
    T = 6
    w = W.Workload("t", 3, 8, 2, 128, 600, "bf16", 596, 2 * T, 31, 128 ** -0.5, 1.0, 1.0, "stream")
    mk, mv = W.initial_cache(w, "cuda")
    kw = dict(read_scale=1.0, write_scale=1.0, init_len=w.init_len, mk_init=mk, mv_init=mv)
    ref = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, max_stream=T, **kw)
    # max_stream = 1: this cache's own staging area could not hold T tokens
    sta = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, max_stream=1, **kw)
    assert sta.lib.bct_prefill_stream_host(sta._h, 4096, 4096, 4096, 4096, T, None) == B.BCT_ERR_INVALID_ARG
    q, k, v = W.stream_inputs(w, 0, 2 * T, "cuda")
    for call in range(2):  # the second call reuses the array with the first call's bytes still in it
        sl = slice(call * T, (call + 1) * T)
        hq, hk, hv = (_pinned(x[:, sl].contiguous()) for x in (q, k, v))
        out_ref = torch.empty_like(hq).pin_memory()
        out_sta = torch.full_like(hq, float("nan")).pin_memory()
        ref.prefill_stream_host(hq, hk, hv, out_ref)
        sta.prefill_stream_host_static(hq, hk, hv, out_sta)
        torch.cuda.synchronize()
        assert torch.isfinite(out_sta.float()).all()
        err = (out_sta.float() - out_ref.float()).abs().max().item()
        assert err <= TOL_BF16, (call, err)
        # the same kernels on the same inputs, only staged elsewhere: the results agree bit for bit
        assert torch.equal(out_sta, out_ref), call
    ref.check_status()
    sta.check_status()
    assert ref.len == sta.len == w.capacity
    for a, b in zip(ref.export(torch.float32), sta.export(torch.float32)):
        assert (a.float() - b.float()).abs().max().item() <= TOL_BF16
        assert torch.equal(a, b)

    # a request that cannot fit the built-in array is refused before anything is enqueued
    n0 = sta.launches
    too_many = B.STATIC_STAGE_BYTES // (w.batch * w.n_q_heads * w.head_dim * 2) + 1
    st = sta.lib.bct_prefill_stream_host_static(sta._h, hq.data_ptr(), hk.data_ptr(), hv.data_ptr(),
                                                out_sta.data_ptr(), too_many, None)
    assert st == B.BCT_ERR_INVALID_ARG and "static staging area" in B.last_error()
    assert sta.launches == n0 and sta.len == w.capacity
    # a token count so large that its byte sizes would wrap is refused the same way
    st = sta.lib.bct_prefill_stream_host_static(sta._h, hq.data_ptr(), hk.data_ptr(), hv.data_ptr(),
                                                out_sta.data_ptr(), 1 << 56, None)
    assert st == B.BCT_ERR_INVALID_ARG and sta.launches == n0
    ref.destroy()
    sta.destroy()
