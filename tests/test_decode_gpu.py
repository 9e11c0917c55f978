"""GPU parity of bct_decode_step / bct_prefill_stream against the CPU oracle (through the C ABI)."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import bct_oracle as O
from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld
from paper_2411_15785_b200 import workloads as W

from _parity import TOL, compare_out, compare_state, make_pair, pick_units, run_decode_parity, _unit_slices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    bld.build()
    B.load()


def _small(name, **kw):
    return W.CONFIGS[name].scaled(**kw)


# ---- small shapes spanning several tiles, ragged tails, every dtype / head_dim / group -------------
@pytest.mark.parametrize("dtype,d,G,C,init_len,steps", [
    ("f32", 64, 1, 128, 0, 160),        # fills, then updates
    ("f32", 64, 2, 197, 197, 6),        # ragged: not a multiple of the 64-row tile
    ("f32", 128, 1, 75, 70, 12),        # fill finishes mid-run, 32-row tiles
    ("f32", 128, 3, 300, 300, 4),
    ("bf16", 128, 1, 333, 333, 8),
    ("bf16", 128, 4, 520, 500, 30),
    ("bf16", 64, 2, 1000, 1000, 5),     # 128-row tiles
    ("bf16", 64, 8, 130, 0, 140),
    ("bf16", 128, 8, 257, 257, 5),
    ("bf16", 128, 5, 64, 64, 5),
    ("f32", 64, 7, 3, 0, 9),            # tiny capacity
    ("bf16", 128, 1, 1, 1, 4),          # C = 1: running sum
])
def test_small_shapes_match_oracle(dtype, d, G, C, init_len, steps):
    w = W.Workload("t", 2, 2 * G, 2, d, C, dtype, init_len, steps, 11, d ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 4)
    out_err, state_err = run_decode_parity(w, units)
    assert out_err <= TOL[dtype], out_err
    assert state_err <= TOL[dtype], state_err


# ---- the tensor-core kernel (bfloat16, head_dim 128, G <= 15, C >= 128) and the CUDA-core kernel
# ---- on the same shapes: both must match the oracle ----------------------------------------------------
@pytest.mark.parametrize("cores", [False, True])
@pytest.mark.parametrize("B_,G,C,init_len,steps", [
    (2, 1, 333, 333, 8),       # ragged last tile
    (2, 4, 520, 500, 30),      # fill finishes mid-run
    (5, 7, 128, 0, 140),       # fills from empty, one tile
    (5, 2, 2048, 2048, 6),     # 16 tiles: a full slice
    (2, 3, 2500, 2500, 5),     # cluster of 2, ragged
    (40, 4, 300, 290, 14),     # more units than one pass of the persistent grid
    (1, 1, 16384, 16384, 3),   # cluster of 8, full slices
    (2, 2, 2500, 2490, 14),    # cluster of 2, fill finishes inside the second CTA's slice
    (1, 1, 4200, 2040, 12),    # cluster of 4, the appended slot crosses from one CTA's slice to the next
    (20, 2, 5000, 5000, 4),    # cluster of 2, each CTA's 2560-slot slice in two sub-slices
    (20, 1, 16384, 16384, 3),  # cluster of 2, 8192-slot slices in four sub-slices
    (20, 3, 5000, 4993, 12),   # sub-slices while the cache is still filling
    (80, 1, 128, 0, 5),        # starts empty with more units than SMs: several tile-less units per CTA
    (3, 8, 600, 590, 24),      # 8 read heads: the 16-row query / weight operands; fill finishes mid-run
    (2, 12, 2048, 2048, 5),    # 12 read heads, a full 16-tile slice
    (2, 15, 2500, 2500, 5),    # 15 read heads + the write query = all 16 rows; cluster of 2
    (6, 8, 5000, 5000, 4),     # 8 read heads, sub-slices
])
def test_tensor_core_and_cuda_core_kernels_match_oracle(cores, B_, G, C, init_len, steps):
    d = 128
    if cores and G > 8:
        pytest.skip("the CUDA-core kernel serves at most 8 query heads per kv-head")
    w = W.Workload("t", B_, 2 * G, 2, d, C, "bf16", init_len, steps, 13, d ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 6)
    out_err, state_err = run_decode_parity(w, units, flags=B.FLAG_CUDA_CORES if cores else 0,
                                           expect_tensor_path=not cores)
    assert out_err <= TOL["bf16"], out_err
    assert state_err <= TOL["bf16"], state_err


@pytest.mark.parametrize("flag,oflag", [(B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ), (B.FLAG_DENSE_WRITE, 0),
                                        (B.FLAG_OUT_F32, 0)])
@pytest.mark.parametrize("C,B_,G", [(400, 2, 3), (5000, 2, 3), (6000, 20, 3), (700, 2, 9)])
def test_tensor_core_kernel_flags(flag, oflag, C, B_, G):
    d = 128
    w = W.Workload("t", B_, 2 * G, 2, d, C, "bf16", C, 6, 17, d ** -0.5, 1.0, 1.0, "decode", 1.0, 0.3)
    out_err, state_err = run_decode_parity(w, pick_units(w, 4), flags=flag, oracle_flags=oflag,
                                           expect_tensor_path=True)
    assert out_err <= TOL["bf16"] and state_err <= TOL["bf16"], (out_err, state_err)


def test_diffuse_writes_rewrite_every_row():
    d = 128
    w = W.Workload("t", 2, 4, 2, d, 700, "bf16", 700, 12, 5, d ** -0.5, 1.0, 1.0, "decode", 1.0, d ** -0.5)
    out_err, state_err = run_decode_parity(w, pick_units(w, 4))
    assert out_err <= TOL["bf16"] and state_err <= 1e-3, (out_err, state_err)


def test_cluster_split_path_small_batch_large_capacity():
    # one unit, C = 8192: the planner spreads the slots over an 8-CTA cluster
    d = 128
    w = W.Workload("t", 1, 4, 1, d, 8192, "bf16", 8192, 6, 6, d ** -0.5, 1.0, 1.0, "decode")
    out_err, state_err = run_decode_parity(w, pick_units(w, 1))
    assert out_err <= TOL["bf16"] and state_err <= TOL["bf16"], (out_err, state_err)
    w2 = W.Workload("t", 1, 1, 1, 64, 5000, "f32", 4990, 20, 7, 0.125, 1.0, 1.0, "decode")
    out_err, state_err = run_decode_parity(w2, pick_units(w2, 1))
    assert out_err <= TOL["f32"] and state_err <= TOL["f32"], (out_err, state_err)


@pytest.mark.parametrize("flag,oflag", [(B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),
                                        (B.FLAG_SKIP_FIRST_WRITE, O.SKIP_FIRST_WRITE),
                                        (B.FLAG_DENSE_WRITE, 0)])
def test_flags_match_oracle(flag, oflag):
    w = W.Workload("t", 2, 4, 2, 64, 150, "f32", 150, 5, 8, 0.125, 0.5, 1.0, "decode")
    out_err, state_err = run_decode_parity(w, pick_units(w, 4), flags=flag, oracle_flags=oflag)
    assert out_err <= TOL["f32"] and state_err <= TOL["f32"], (out_err, state_err)


@pytest.mark.parametrize("C,G,init_len", [(333, 1, 333), (520, 4, 500), (8192, 2, 8192)])
def test_precise_read_and_float_out_on_large_magnitude_state(C, G, init_len):
    # MV_0 ~ N(0, 100^2): a bfloat16 ulp of the state is ~0.5, so the default value-plane-only read
    # cannot meet an absolute 2e-2; value + residual with float out does.
    d = 128
    B_ = 1 if C > 4096 else 2
    w = W.Workload("t", B_, 2 * G, 2, d, C, "bf16", init_len, 25, 21, d ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 4)
    gpu, ora = make_pair(w, units, flags=B.FLAG_PRECISE_READ | B.FLAG_OUT_F32)
    scale = torch.tensor(100.0, device="cuda")
    k0, v0 = gpu.export(torch.float32)
    v0 = (v0 * scale).to(torch.bfloat16).float() + 0.001953125 * torch.sign(v0)  # value + a residual part
    gpu.import_state(k0[:, :, :init_len].contiguous(), v0[:, :, :init_len].contiguous(), init_len)
    for i, (b, h) in enumerate(units):
        ora.MV[i, :init_len] = v0[b, h, :init_len].double().cpu().numpy()
    worst = 0.0
    for t in range(w.steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        out = gpu.decode_step(q, k, v)
        assert out.dtype == torch.float32
        ref = ora.prefill_stream(*_unit_slices(w, units, q, k, v))
        worst = max(worst, compare_out(w, units, out, ref))
    gpu.check_status()
    state = compare_state(w, units, gpu, ora)
    assert worst <= 2e-3 and state <= TOL["bf16"], (worst, state)


def test_prefill_stream_equals_decode_steps_and_state_only_mode():
    w = W.CONFIGS["stream_b8_c1024"].scaled(batch=2, n_q_heads=4, n_kv_heads=4, capacity=96, steps=160)
    units = pick_units(w, 8)
    q, k, v = W.stream_inputs(w, 0, w.steps, "cuda")
    gpu, ora = make_pair(w, units)
    out = gpu.prefill_stream(q[:, :100].contiguous(), k[:, :100].contiguous(), v[:, :100].contiguous())
    out2 = gpu.prefill_stream(q[:, 100:].contiguous(), k[:, 100:].contiguous(), v[:, 100:].contiguous())
    ref = ora.prefill_stream(*_unit_slices(w, units, q, k, v))
    err = compare_out(w, units, torch.cat([out, out2], dim=1), ref)
    assert err <= TOL["bf16"], err
    assert compare_state(w, units, gpu, ora) <= TOL["bf16"]
    # the same tokens one decode step at a time give the same bits
    gpu2, _ = make_pair(w, units)
    outs = [gpu2.decode_step(q[:, t].contiguous(), k[:, t].contiguous(), v[:, t].contiguous()) for t in range(w.steps)]
    assert torch.equal(torch.stack(outs, dim=1), torch.cat([out, out2], dim=1))
    # state-only (UpdateKV): out = NULL
    gpu3, _ = make_pair(w, units)
    assert gpu3.prefill_stream(q, k, v, want_out=False) is None
    k1, v1 = gpu.export()
    k3, v3 = gpu3.export()
    assert torch.equal(k1, k3) and torch.equal(v1, v3)


def test_export_import_resume_is_bitwise():
    w = W.Workload("t", 2, 4, 2, 128, 200, "bf16", 200, 10, 9, 128 ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 4)
    a, _ = make_pair(w, units)
    b, _ = make_pair(w, units)
    for t in range(5):
        x = W.step_inputs(w, t, "cuda")
        a.decode_step(*x)
        b.decode_step(*x)
    k, v = b.export(torch.int32)  # lossless checkpoint words
    c = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype,
                read_scale=w.read_scale, write_scale=w.write_scale)
    c.import_state(k, v, b.len)
    for t in range(5, 10):
        x = W.step_inputs(w, t, "cuda")
        oa, oc = a.decode_step(*x), c.decode_step(*x)
        assert torch.equal(oa, oc)
    ka, va = a.export()
    kc, vc = c.export()
    assert torch.equal(ka, kc) and torch.equal(va, vc)
    # a float checkpoint carries the same values (value + residual), exactly
    d = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype)
    d.import_state(ka, va, a.len)
    assert torch.equal(d.export()[1], va)


def test_run_twice_is_deterministic_and_host_entry_matches_device_entry():
    w = W.Workload("t", 3, 8, 2, 128, 600, "bf16", 590, 24, 10, 128 ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 6)
    a, _ = make_pair(w, units)
    b, _ = make_pair(w, units)
    for t in range(w.steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        oa = a.decode_step(q, k, v)
        hq, hk, hv = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
        ho = torch.empty_like(hq).pin_memory()
        b.decode_step_host(hq, hk, hv, ho)
        torch.cuda.synchronize()
        assert torch.equal(oa.cpu(), ho)
    assert all(torch.equal(x, y) for x, y in zip(a.export(), b.export()))


def test_bad_arguments_on_device_launch_nothing():
    import ctypes
    c = B.Cache(1, 1, 1, 64, 16, torch.float32)
    n0 = c.launches
    q = torch.zeros(1, 1, 64, device="cuda")
    p = q.data_ptr()
    assert c.lib.bct_decode_step(c._h, p + 4, p, p, p, None) == B.BCT_ERR_INVALID_ARG          # misaligned
    assert c.lib.bct_decode_step(c._h, p, p, p, None, None) == B.BCT_ERR_INVALID_ARG           # out missing
    assert c.lib.bct_prefill_stream(c._h, p, p, p, None, 0, None) == B.BCT_ERR_INVALID_ARG     # T = 0
    assert c.lib.bct_prefill_stream_host(c._h, 4096, 4096, 4096, 4096, 5, None) == B.BCT_ERR_INVALID_ARG  # > max_stream
    assert c.lib.bct_cache_export(c._h, p, p, B.BCT_BF16_PAIR, None) == B.BCT_ERR_UNSUPPORTED  # float cache
    assert c.launches == n0 and c.len == 0
    assert c.status() == B.BCT_OK
    with pytest.raises(B.BctError):
        B.Cache(1, 1, 1, 64, 16, torch.float32, init_len=4)  # mk_init missing
    # capacity too large for the score array of an 8-CTA cluster: refused before any device work
    prm = B.make_params(1, 8, 1, 128, 1 << 20, torch.bfloat16)
    h = ctypes.c_void_p(None)
    need, align = B.cache_bytes(prm)                       # the size is defined even where no kernel serves the shape
    ws = torch.empty(need + align, dtype=torch.uint8, device="cuda")   # an honest workspace (about 0.8 GB): if the
    base = (ws.data_ptr() + align - 1) // align * align                  # refusal ever regressed, nothing would be overrun
    st = c.lib.bct_cache_create(ctypes.byref(prm), base, need, None, None, None, ctypes.byref(h))
    assert st == B.BCT_ERR_UNSUPPORTED and not h.value
    del ws
    c.destroy()
    assert c.lib.bct_cache_destroy(None) == B.BCT_OK


def test_groups_above_eight_need_the_tensor_core_path():
    # 9..15 query heads per kv-head exist on the tensor-core kernel only: a float cache of that shape is refused
    prm = B.make_params(2, 24, 2, 128, 256, torch.float32)
    lib = B.load()
    n, al = ctypes.c_size_t(0), ctypes.c_size_t(0)
    assert lib.bct_cache_bytes(ctypes.byref(prm), ctypes.byref(n), ctypes.byref(al)) == B.BCT_OK
    ws = torch.empty(n.value, dtype=torch.uint8, device="cuda")
    h = ctypes.c_void_p(None)
    st = lib.bct_cache_create(ctypes.byref(prm), ws.data_ptr(), n.value, None, None, None, ctypes.byref(h))
    assert st == B.BCT_ERR_UNSUPPORTED and "tensor-core" in B.last_error()
    prm = B.make_params(2, 34, 2, 128, 256, torch.bfloat16)      # 17 per kv-head: nowhere
    assert lib.bct_cache_bytes(ctypes.byref(prm), ctypes.byref(n), ctypes.byref(al)) == B.BCT_ERR_UNSUPPORTED


def test_destroyed_handle_is_refused_without_being_read():
    c = B.Cache(1, 1, 1, 64, 16, torch.float32)
    h = ctypes.c_void_p(c._h.value)
    c.destroy()
    n = ctypes.c_int32(0)
    assert c.lib.bct_cache_len(h, ctypes.byref(n)) == B.BCT_ERR_STATE
    assert c.lib.bct_cache_destroy(h) == B.BCT_ERR_STATE          # a second destroy
    assert c.lib.bct_cache_status(h, None) == B.BCT_ERR_STATE
    assert "destroyed" in B.last_error()


def test_rows_rewritten_counter_counts_the_slots_the_rule_touches():
    # DENSE_WRITE rewrites every slot: units * tokens * C rows exactly, on both decode kernels; the default
    # threshold rewrites fewer, and the fill phase none
    w = W.Workload("t", 2, 4, 2, 128, 384, "bf16", 384, 5, 13, 128 ** -0.5, 1.0, 1.0, "decode")
    for flags in (B.FLAG_DENSE_WRITE, B.FLAG_DENSE_WRITE | B.FLAG_CUDA_CORES):
        gpu, _ = make_pair(w, pick_units(w, 2), flags=flags)
        for t in range(w.steps):
            gpu.decode_step(*W.step_inputs(w, t, "cuda"))
        assert gpu.rows_rewritten() == w.units * w.steps * w.capacity
        gpu.destroy()
    counts = []
    for flags in (0, B.FLAG_CUDA_CORES):
        gpu, _ = make_pair(w, pick_units(w, 2), flags=flags)
        for t in range(w.steps):
            gpu.decode_step(*W.step_inputs(w, t, "cuda"))
        counts.append(gpu.rows_rewritten())
        gpu.destroy()
    assert 0 < counts[0] < w.units * w.steps * w.capacity // 4
    assert abs(counts[0] - counts[1]) <= max(4, counts[0] // 50)   # weights at the threshold may fall either way
    wf = w.scaled(init_len=0)
    gpu, _ = make_pair(wf, pick_units(wf, 2))
    for t in range(w.steps):
        gpu.decode_step(*W.step_inputs(wf, t, "cuda"))
    assert gpu.rows_rewritten() == 0 and gpu.len == w.steps
    gpu.destroy()


def test_bounded_wait_runs_out_and_the_cache_stays_usable():
    # the self-test block waits on a barrier nothing arrives on; its wait gives up after a thousand polls and
    # reports through the status words.  No fault, no hang: the next steps on the same cache match the oracle.
    w = W.Workload("t", 2, 4, 2, 128, 300, "bf16", 300, 6, 17, 128 ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 4)
    gpu, ora = make_pair(w, units)
    assert gpu.status() == B.BCT_OK
    gpu.selftest_timeout()
    assert gpu.status() == B.BCT_ERR_TIMEOUT
    assert "site 99" in B.last_error()
    assert gpu.status() == B.BCT_ERR_TIMEOUT          # sticky until cleared
    gpu.status_clear()
    assert gpu.status() == B.BCT_OK
    worst = 0.0
    for t in range(w.steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        out = gpu.decode_step(q, k, v)
        worst = max(worst, compare_out(w, units, out, ora.prefill_stream(*_unit_slices(w, units, q, k, v))))
    gpu.check_status()
    assert worst <= TOL["bf16"] and compare_state(w, units, gpu, ora) <= TOL["bf16"]
    gpu.destroy()


@pytest.mark.parametrize("name,steps", [("mha7b_b64_c2048", 12), ("gqa8b_b128_c4096", 6), ("sweep_b256_c256", 12),
                                        ("sweep_b256_c1024", 8)])
def test_every_unit_tensor_core_kernel_against_cuda_core_kernel(name, steps):
    # A net beside the oracle sample, not instead of it: at the full batch, ALL units of the tensor-core kernel
    # (persistent CTAs, deferred row rewrite, last-unit flush) against the CUDA-core kernel (one cluster per unit).
    w = W.CONFIGS[name]
    mk, mv = W.initial_cache(w, "cuda")
    kw = dict(read_scale=w.read_scale, write_scale=w.write_scale, init_len=w.init_len, mk_init=mk, mv_init=mv)
    a = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, **kw)
    b = B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.torch_dtype, flags=B.FLAG_CUDA_CORES, **kw)
    del mk, mv
    assert a.tensor_path and not b.tensor_path
    for t in range(steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        oa, ob = a.decode_step(q, k, v), b.decode_step(q, k, v)
        err = (oa.float() - ob.float()).abs().amax(dim=(1, 2))       # per sequence
        assert err.max().item() <= TOL["bf16"], (t, int(err.argmax()), err.max().item())
    a.check_status()
    b.check_status()
    va, vb = a.export(torch.float32)[1], b.export(torch.float32)[1]
    per_unit = (va - vb).abs().amax(dim=(2, 3))
    assert per_unit.max().item() <= TOL["bf16"], (int(per_unit.argmax()), per_unit.max().item())
    del va, vb
    a.destroy()
    b.destroy()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("B_,G,C,steps,write_scale,flags,oflags", [
    (3, 1, 333, 6, 1.0, 0, 0),                                   # ragged last tile: its rows past C are clipped by the store
    (5, 2, 2048, 5, 128 ** -0.5, 0, 0),                         # 16 tiles: a full slice, diffuse weights
    (2, 3, 2500, 5, 128 ** -0.5, 0, 0),                         # cluster of 2, ragged
    (40, 4, 384, 8, 0.3, 0, 0),                                  # more units than one pass of the persistent grid
    (2, 4, 640, 6, 128 ** -0.5, B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),
    (2, 1, 4096, 4, 128 ** -0.5, 0, 0),                          # two CTAs of 2048 slots each
    (1, 2, 8192, 3, 128 ** -0.5, 0, 0),                          # slices beyond one sub-slice: the staged path serves them
])
def test_dense_write_rebuilds_whole_tiles(B_, G, C, steps, write_scale, flags, oflags):
    # BCT_FLAG_DENSE_WRITE on the tensor-core kernel: value and residual tiles are rebuilt in their ring stages and
    # stored whole; against the oracle's exact rule (every slot updated), with step sizes
    w = W.Workload("t", B_, 2 * G, 2, 128, C, "bf16", C, steps, 83, 128 ** -0.5, 1.0, 1.0, "decode", 1.0, write_scale)
    units = pick_units(w, 6)
    gpu, ora = make_pair(w, units, flags=flags | B.FLAG_DENSE_WRITE, oracle_flags=oflags)
    assert gpu.tensor_path
    g = torch.Generator(device="cpu").manual_seed(3)
    worst = 0.0
    for t in range(steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        eta = (torch.rand((w.batch, w.n_kv_heads), generator=g) * 1.5 + 0.25).cuda()
        out = gpu.decode_step(q, k, v, eta=eta)
        qs, ks, vs = _unit_slices(w, units, q, k, v)
        es = torch.stack([eta[b, h] for b, h in units])[:, None, None].double().cpu().numpy()
        worst = max(worst, compare_out(w, units, out, ora.prefill_stream(qs, ks, vs, eta=es)))
    gpu.check_status()
    assert gpu.rows_rewritten() == w.units * steps * C
    state = compare_state(w, units, gpu, ora)
    assert worst <= TOL["bf16"] and state <= TOL["bf16"], (worst, state)
    gpu.destroy()


@pytest.mark.parametrize("B_,G,C,init_len,steps,write_scale,flags,oflags", [
    (160, 4, 256, 256, 10, 1.0, 0, 0),                # two tiles per unit, 320 units: more than two per SM
    (170, 1, 300, 290, 16, 1.0, 0, 0),                # ragged capacity; the fill finishes mid-run
    (150, 7, 512, 512, 6, 0.3, 0, 0),                 # four tiles, 7 read heads, many rows rewritten (several staging rounds)
    (150, 2, 128, 0, 133, 1.0, 0, 0),                 # starts empty: tile-less units first, then one tile, then soft writes
    (160, 3, 384, 384, 6, 0.5, B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),
    (160, 2, 384, 384, 6, 1.0, B.FLAG_SKIP_FIRST_WRITE, O.SKIP_FIRST_WRITE),
])
def test_units_of_a_few_tiles_two_ctas_per_sm(B_, G, C, init_len, steps, write_scale, flags, oflags):
    # bfloat16 units of up to 512 slots with more than two units per SM run as two CTAs per SM (half the tensor
    # memory and a two-stage ring each); same step, same oracle, with step sizes
    w = W.Workload("t", B_, 2 * G, 2, 128, C, "bf16", init_len, steps, 89, 128 ** -0.5, 1.0, 1.0, "decode", 1.0, write_scale)
    assert w.units > 2 * 148
    units = pick_units(w, 8, seed=5)
    gpu, ora = make_pair(w, units, flags=flags, oracle_flags=oflags)
    assert gpu.tensor_path
    g = torch.Generator(device="cpu").manual_seed(7)
    worst = 0.0
    for t in range(steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        eta = (torch.rand((w.batch, w.n_kv_heads), generator=g) * 1.5 + 0.25).cuda()
        out = gpu.decode_step(q, k, v, eta=eta)
        qs, ks, vs = _unit_slices(w, units, q, k, v)
        es = torch.stack([eta[b, h] for b, h in units])[:, None, None].double().cpu().numpy()
        worst = max(worst, compare_out(w, units, out, ora.prefill_stream(qs, ks, vs, eta=es)))
    gpu.check_status()
    state = compare_state(w, units, gpu, ora)
    assert worst <= TOL["bf16"] and state <= TOL["bf16"], (worst, state)
    gpu.destroy()


def test_largest_capacity_the_tensor_core_kernel_takes():
    # 65536 slots: a cluster of 8 CTAs with 8192 slots each, four sub-slices per CTA; beyond it the CUDA-core kernel's limits
    # apply and the create call refuses the shape
    w = W.Workload("t", 1, 2, 1, 128, 65536, "bf16", 65536, 3, 97, 128 ** -0.5, 1.0, 1.0, "decode")
    out_err, state_err = run_decode_parity(w, [(0, 0)], expect_tensor_path=True)
    assert out_err <= TOL["bf16"] and state_err <= TOL["bf16"], (out_err, state_err)
    prm = B.make_params(1, 2, 1, 128, 65537, torch.bfloat16)
    need, align = B.cache_bytes(prm)
    ws = torch.empty(need + align, dtype=torch.uint8, device="cuda")
    h = ctypes.c_void_p(None)
    base = (ws.data_ptr() + align - 1) // align * align
    st = B.load().bct_cache_create(ctypes.byref(prm), base, need, None, None, None, ctypes.byref(h))
    if st == B.BCT_OK:       # served by the CUDA-core kernel when its score array still fits: then it must be usable
        assert h.value
        B.load().bct_cache_destroy(h)
    else:
        assert st == B.BCT_ERR_UNSUPPORTED and not h.value


def test_two_handles_on_two_streams_are_independent():
    # different handles share nothing but read-only tables: steps enqueued alternately on two streams give each cache
    # the results it gives alone
    w = W.Workload("t", 4, 8, 2, 128, 640, "bf16", 640, 12, 101, 128 ** -0.5, 1.0, 1.0, "decode")
    units = pick_units(w, 4)
    solo, _ = make_pair(w, units)
    a, _ = make_pair(w, units)
    b, _ = make_pair(w.scaled(seed=202), units)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs_solo, outs_a = [], []
    for t in range(w.steps):
        q, k, v = W.step_inputs(w, t, "cuda")
        q2, k2, v2 = W.step_inputs(w.scaled(seed=202), t, "cuda")
        torch.cuda.synchronize()
        outs_solo.append(solo.decode_step(q, k, v))
        with torch.cuda.stream(sa):
            outs_a.append(a.decode_step(q, k, v, stream=sa))
        with torch.cuda.stream(sb):
            b.decode_step(q2, k2, v2, stream=sb)
    torch.cuda.synchronize()
    for x, y in zip(outs_solo, outs_a):
        assert torch.equal(x, y)
    assert all(torch.equal(x, y) for x, y in zip(solo.export(v_dtype=torch.int32), a.export(v_dtype=torch.int32)))
    for c in (solo, a, b):
        c.check_status()
        c.destroy()
