"""GPU parity of the chunked tensor-core stream kernel (bct_prefill_stream on a full bfloat16 cache,
head_dim 128) against the CPU oracle, through the C ABI."""
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


def _stream_parity(w, T, pieces, flags=0, oracle_flags=0, want_out=True, write_eps=0.0, n_units=8):
    units = pick_units(w, n_units)
    gpu, ora = make_pair(w, units, flags=flags, oracle_flags=oracle_flags, write_eps=write_eps, oracle_write_eps=write_eps)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    launches0 = gpu.launches
    outs, t = [], 0
    for n in pieces:
        sl = slice(t, t + n)
        outs.append(gpu.prefill_stream(q[:, sl].contiguous(), k[:, sl].contiguous(), v[:, sl].contiguous(),
                                       want_out=want_out))
        t += n
    assert t == T
    gpu.check_status()
    ref = ora.prefill_stream(*_unit_slices(w, units, q, k, v))
    err = compare_out(w, units, torch.cat(outs, dim=1), ref) if want_out else 0.0
    state = compare_state(w, units, gpu, ora)
    n_launch = gpu.launches - launches0
    gpu.destroy()
    return err, state, n_launch


@pytest.mark.parametrize("G,C,init_len,T,pieces", [
    (1, 256, 256, 200, [200]),            # 3 chunks of 64 + 8 single tokens
    (1, 1024, 1024, 256, [128, 128]),     # the long-stream shape, two calls
    (1, 333, 300, 170, [170]),            # ragged capacity; 33 fill tokens first, then chunks
    (2, 512, 512, 100, [64, 36]),         # chunks of 32
    (3, 640, 640, 64, [64]),
    (4, 520, 520, 50, [50]),              # chunks of 16
    (7, 2048, 2048, 32, [32]),            # 16 tiles
    (4, 4096, 4096, 40, [40]),            # 32 tiles per unit: beyond one decode CTA's slice
    (1, 3000, 3000, 130, [130]),          # ragged capacity above 2048
])
def test_chunked_stream_matches_oracle(G, C, init_len, T, pieces):
    d = 128
    w = W.Workload("t", 2, 2 * G, 2, d, C, "bf16", init_len, T, 41, d ** -0.5, 1.0, 1.0, "stream")
    w = w.scaled(batch=3 if C <= 512 else 2)
    err, state, n_launch = _stream_parity(w, T, pieces)
    assert err <= TOL["bf16"] and state <= TOL["bf16"], (err, state)
    assert n_launch < T  # whole chunks went through the chunked kernel, not one launch per token


@pytest.mark.parametrize("flags,oflags", [(B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ), (B.FLAG_OUT_F32, 0),
                                          (B.FLAG_SKIP_FIRST_WRITE, O.SKIP_FIRST_WRITE)])
def test_chunked_stream_flags(flags, oflags):
    d = 128
    w = W.Workload("t", 3, 4, 2, d, 384, "bf16", 384, 150, 43, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.4)
    err, state, _ = _stream_parity(w, 150, [150], flags=flags, oracle_flags=oflags)
    assert err <= TOL["bf16"] and state <= TOL["bf16"], (err, state)


def test_chunked_stream_state_only_and_diffuse_writes():
    d = 128
    w = W.Workload("t", 2, 2, 2, d, 256, "bf16", 256, 192, 47, d ** -0.5, 1.0, 1.0, "stream", 1.0, d ** -0.5)
    err, state, _ = _stream_parity(w, 192, [192], want_out=False)
    assert state <= 1e-3, state
    err, state, _ = _stream_parity(w, 192, [192])
    assert err <= TOL["bf16"] and state <= 1e-3, (err, state)


def test_chunked_stream_tracks_decode_steps_on_a_long_run():
    # the per-token path (tensor-core decode kernel) and the chunked path on the same 2048 tokens
    d = 128
    w = W.Workload("t", 1, 4, 4, d, 512, "bf16", 512, 2048, 53, d ** -0.5, 1.0, 1.0, "stream")
    units = pick_units(w, 4)
    a, ora = make_pair(w, units, flags=B.FLAG_OUT_F32)
    b, _ = make_pair(w, units, flags=B.FLAG_OUT_F32)
    q, k, v = W.stream_inputs(w, 0, w.steps, "cuda")
    oa = a.prefill_stream(q, k, v)
    ob = torch.stack([b.decode_step(q[:, t].contiguous(), k[:, t].contiguous(), v[:, t].contiguous())
                      for t in range(w.steps)], dim=1)
    ref = ora.prefill_stream(*_unit_slices(w, units, q, k, v))
    ea, eb = compare_out(w, units, oa, ref), compare_out(w, units, ob, ref)
    assert ea <= TOL["bf16"] and eb <= TOL["bf16"], (ea, eb)
    assert compare_state(w, units, a, ora) <= TOL["bf16"]


@pytest.mark.parametrize("G,C,init_len,T,pieces,flags", [
    (1, 1024, 0, 1200, [1200], 0),                 # from empty: 16 fill chunks of 64, then the full phase
    (1, 333, 0, 400, [100, 300], 0),               # ragged capacity: 5 fill chunks, 13 single tokens, full phase
    (2, 512, 100, 300, [300], 0),                  # starts inside tile 0; chunks of 32 cross tile borders
    (3, 640, 37, 200, [70, 130], B.FLAG_OUT_F32),  # odd start, second call resumes the fill phase
    (7, 2048, 1900, 140, [140], 0),                # chunks of 16 over 15 resident tiles
    (2, 2500, 2400, 160, [160], 0),                # fill chunks above 2048 slots, then soft writes
    (1, 256, 192, 64, [64], B.FLAG_PRECISE_READ | B.FLAG_OUT_F32),  # exactly fills the cache
])
def test_fill_phase_chunks_match_oracle(G, C, init_len, T, pieces, flags):
    d = 128
    w = W.Workload("t", 2, 2 * G, 2, d, C, "bf16", init_len, T, 59, d ** -0.5, 1.0, 1.0, "stream")
    w = w.scaled(batch=3 if C <= 512 else 2)
    err, state, n_launch = _stream_parity(w, T, pieces, flags=flags)
    tol = 5e-3 if flags & B.FLAG_PRECISE_READ else TOL["bf16"]   # float out; the numerators are bfloat16 (2^-9 relative)
    assert err <= tol and state <= TOL["bf16"], (err, state)
    Tc = 64 if G == 1 else (32 if G <= 3 else 16)
    assert n_launch <= len(pieces) * (2 + 2 * Tc)  # the fill phase went in chunks, not one launch per token


def test_fill_phase_chunks_equal_single_tokens_in_the_cache():
    # keys and values appended by the chunked kernel are the bits the per-token path appends
    d = 128
    w = W.Workload("t", 2, 2, 2, d, 512, "bf16", 0, 256, 61, d ** -0.5, 1.0, 1.0, "stream")
    units = pick_units(w, 4)
    a, _ = make_pair(w, units)
    b, _ = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, 256, "cuda")
    a.prefill_stream(q, k, v, want_out=False)
    for t in range(256):
        b.decode_step(q[:, t].contiguous(), k[:, t].contiguous(), v[:, t].contiguous())
    assert a.len == b.len == 256
    ka, va = a.export(v_dtype=torch.int32)
    kb, vb = b.export(v_dtype=torch.int32)
    assert torch.equal(ka, kb) and torch.equal(va, vb)
    a.destroy()
    b.destroy()


@pytest.mark.parametrize("G,C,init_len,T,max_launches", [
    (1, 256, 256, 100, 2),       # one chunk of 64, one of 40 tokens of which 36 exist
    (1, 512, 512, 5, 1),         # fewer tokens than the smallest chunk: 8 rows, 5 of them real
    (1, 512, 512, 3, 3),         # below 4 tokens the decode kernel is the cheaper one
    (4, 384, 384, 61, 3),        # chunks of 24: two whole ones and 13 tokens in a chunk of 16
    (2, 300, 130, 250, 12),      # fill: 4 chunks of 40, one of 8, 2 single tokens; then 40 + 40 of the full phase
    (1, 256, 251, 30, 7),        # 5 free slots: single tokens, then one ragged chunk of the full phase
])
def test_ragged_ends_go_in_short_chunks(G, C, init_len, T, max_launches):
    d = 128
    w = W.Workload("t", 3, 2 * G, 2, d, C, "bf16", init_len, T, 67, d ** -0.5, 1.0, 1.0, "stream")
    err, state, n_launch = _stream_parity(w, T, [T])
    assert err <= TOL["bf16"] and state <= TOL["bf16"], (err, state)
    assert n_launch <= max_launches + 1, n_launch   # + the export launch of the state comparison


@pytest.mark.parametrize("flags,oflags", [(0, 0), (B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ)])
def test_write_threshold_is_the_same_in_chunks_and_in_decode_steps(flags, oflags):
    # a caller-chosen write_eps drops the same slots whether the tokens go through the chunked kernel, the
    # write-only chunks or one decode step each; all three against the oracle with the same threshold
    d, eps, T = 128, 1e-3, 150
    w = W.Workload("t", 3, 4, 2, d, 384, "bf16", 384, T, 71, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.35)
    err, state, _ = _stream_parity(w, T, [T], flags=flags, oracle_flags=oflags, write_eps=eps)
    assert err <= TOL["bf16"] and state <= TOL["bf16"], (err, state)
    units = pick_units(w, 8)
    chunks, ora = make_pair(w, units, flags=flags, oracle_flags=oflags, write_eps=eps, oracle_write_eps=eps)
    steps, exact = make_pair(w, units, flags=flags, oracle_flags=oflags, write_eps=eps, oracle_write_eps=0.0)
    wonly, _ = make_pair(w, units, flags=flags, write_eps=eps)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    chunks.prefill_stream(q, k, v)
    for t in range(T):
        steps.decode_step(q[:, t].contiguous(), k[:, t].contiguous(), v[:, t].contiguous())
    wonly.update_kv(k, v)
    qs, ks, vs = _unit_slices(w, units, q, k, v)
    ora.prefill_stream(qs, ks, vs)
    exact.prefill_stream(qs, ks, vs)
    # the threshold matters at this write scale: the exact rule's state is measurably different
    assert float(np.abs(ora.MV - exact.MV).max()) > 8e-3
    for gpu in (chunks, steps, wonly):
        gpu.check_status()
        # (a weight within rounding of the threshold may fall either way in fp32: one such slot moves an element by
        # about eps * |v|, so the bar sits between that and the distance to the exact rule)
        assert compare_state(w, units, gpu, ora) <= 6e-3
        gpu.destroy()


@pytest.mark.parametrize("B_,G,T,pieces,flags,oflags", [
    (4, 1, 256, [256], 0, 0),                                         # four chunks of 64 on a resident tile
    (80, 1, 200, [200], 0, 0),                                        # 160 units on 148 CTAs: a CTA takes a second unit after a resident one
    (4, 2, 250, [120, 130], B.FLAG_PRECISE_READ | B.FLAG_OUT_F32, 0),  # two calls, chunks of 40, value + residual read
    (4, 4, 100, [100], B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),
])
def test_single_tile_cache_stays_resident_across_chunks(B_, G, T, pieces, flags, oflags):
    # C = 128: the unit's one tile of MK and of MV (value + residual) stays in shared memory for all chunks of a call;
    # only the first chunk loads it and only the last one stores it
    d = 128
    w = W.Workload("t", B_, 2 * G, 2, d, 128, "bf16", 128, T, 73, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    err, state, n_launch = _stream_parity(w, T, pieces, flags=flags, oracle_flags=oflags)
    tol = 5e-3 if flags & B.FLAG_PRECISE_READ else TOL["bf16"]   # float out; the numerators are bfloat16 (2^-9 relative)
    assert err <= tol and state <= TOL["bf16"], (err, state)
    assert n_launch <= 3 * len(pieces) + 1


def test_single_tile_cache_resident_in_update_kv_and_counts_its_stores():
    d, T = 128, 384
    w = W.Workload("t", 8, 2, 2, d, 128, "bf16", 128, T, 79, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    units = pick_units(w, 6)
    gpu, ora = make_pair(w, units)
    q, k, v = W.stream_inputs(w, 0, T, "cuda")
    gpu.update_kv(k, v)            # three chunks of 128 write rows
    gpu.check_status()
    _, ks, vs = _unit_slices(w, units, q, k, v)
    ora.update_kv(ks, vs)
    assert compare_state(w, units, gpu, ora) <= TOL["bf16"]
    assert gpu.rows_rewritten() == w.units * 128      # one store of the tile per unit, after the last chunk
    gpu.destroy()


@pytest.mark.parametrize("G,C,init_len,T,pieces,flags,oflags", [
    (1, 256, 256, 192, [192], 0, 0),               # 160 units x 3 chunks on 148 CTAs: 4 turns instead of 6
    (1, 384, 0, 512, [512], 0, 0),                 # from empty: 6 fill chunks dealt round the CTAs (appended keys handed over), then 2
    (2, 256, 256, 200, [120, 80], B.FLAG_WRITE_THEN_READ, O.WRITE_THEN_READ),   # chunks of 40, two calls (two launch numbers)
    (1, 512, 512, 256, [256], B.FLAG_PRECISE_READ | B.FLAG_OUT_F32, 0),
])
def test_chunks_of_a_unit_go_round_the_ctas(G, C, init_len, T, pieces, flags, oflags):
    # more units than CTAs and several chunks per call: the (unit, chunk) pairs are dealt chunk-major, so a unit's
    # consecutive chunks run on different CTAs and are handed over through global memory and the unit's progress word
    d = 128
    w = W.Workload("t", 80, 2 * G, 2, d, C, "bf16", init_len, T, 57, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    err, state, n_launch = _stream_parity(w, T, pieces, flags=flags, oracle_flags=oflags, n_units=16)
    tol = 5e-3 if flags & B.FLAG_PRECISE_READ else TOL["bf16"]
    assert err <= tol and state <= TOL["bf16"], (err, state)


@pytest.mark.parametrize("init_len,flags", [(256, 0), (0, 0), (256, B.FLAG_PRECISE_READ | B.FLAG_OUT_F32)])
def test_chunk_major_launch_is_bit_equal_to_chunk_by_chunk_calls(init_len, flags):
    # One call of 12 chunks on 170 units (chunks dealt round the CTAs, units handed from CTA to CTA) against the
    # same tokens fed one chunk per call (every launch a single chunk: no hand-over).  The arithmetic of a chunk
    # is the same in both, so outputs and the exported state agree bit for bit on every unit; three rounds.
    d, C, G, Tc = 128, 256, 1, 64
    T = 12 * Tc
    w = W.Workload("t", 85, 2 * G, 2, d, C, "bf16", init_len, T, 61, d ** -0.5, 1.0, 1.0, "stream", 1.0, 0.5)
    mk = mv = None
    if init_len:
        mk, mv = W.initial_cache(w, "cuda")
    mk_cache = lambda: B.Cache(w.batch, w.n_q_heads, w.n_kv_heads, d, C, torch.bfloat16, read_scale=w.read_scale,
                               write_scale=w.write_scale, init_len=init_len, flags=flags, mk_init=mk, mv_init=mv,
                               guard_bytes=4096)
    one, many = mk_cache(), mk_cache()
    for rnd in range(3):
        q, k, v = W.stream_inputs(w, rnd * T, T, "cuda")
        o1 = one.prefill_stream(q, k, v)
        parts = [many.prefill_stream(q[:, i:i + Tc].contiguous(), k[:, i:i + Tc].contiguous(), v[:, i:i + Tc].contiguous())
                 for i in range(0, T, Tc)]
        o2 = torch.cat(parts, dim=1)
        one.check_status()
        many.check_status()
        assert torch.equal(o1, o2)
        (k1, v1), (k2, v2) = one.export(), many.export()
        assert torch.equal(k1, k2) and torch.equal(v1, v2)
    one.check_guards()
    many.check_guards()
    one.destroy()
    many.destroy()
