"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test states which passage or identity it uses.  None of them re-types the
oracle's loops: they use textbook routines (causal softmax attention), closed
forms that follow from the update rule, invariances, hand-worked fixtures and a
long-hand brute force on tiny inputs.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import bct_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(20241016)


def _rand(*shape, scale=1.0):
    return RNG.normal(size=shape) * scale


def _np_softmax(x, axis=-1):
    x = x - x.max(axis=axis, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=axis, keepdims=True)


# ---------------------------------------------------------------------------------------
# Hand-worked fixtures (tests/golden): Algorithm 1 + Method step 4 evaluated by hand
# ---------------------------------------------------------------------------------------
def _parse_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, rest = line.split(None, 1)
            rows = []
            for row in rest.split(";"):
                r = []
                for tok in row.split():
                    if tok == "L3":
                        r.append(math.log(3.0))
                    else:
                        r.append(float(Fraction(tok)))
                rows.append(r)
            vals[key] = np.array(rows if len(rows) > 1 else rows[0], dtype=np.float64)
    return vals


def test_golden_full_phase_hand_worked():
    g = _parse_golden("hand_worked_full_c2_d2.txt")
    c = O.OracleCache(1, 1, 1, 2, 2, read_scale=1.0, write_scale=1.0, init_len=2,
                      mk_init=g["MK"][None, None], mv_init=g["MV0"][None, None])
    o1 = c.decode_step(g["q1"][None, None], g["k1"][None, None], g["v1"][None, None])
    np.testing.assert_allclose(o1[0, 0], g["o1"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(c.values()[0, 0], g["MV1"], rtol=0, atol=1e-14)
    o2 = c.decode_step(g["q2"][None, None], g["k2"][None, None], g["v2"][None, None])
    np.testing.assert_allclose(o2[0, 0], g["o2"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(c.values()[0, 0], g["MV2"], rtol=0, atol=1e-13)
    np.testing.assert_array_equal(c.keys()[0, 0], g["MK"])  # MK is never assigned by Algorithm 1


def test_golden_fill_phase_hand_worked():
    g = _parse_golden("hand_worked_fill_c2_d2.txt")
    c = O.OracleCache(1, 1, 1, 2, 2, read_scale=1.0, write_scale=1.0)
    for t in (1, 2, 3):
        o = c.decode_step(g["q%d" % t][None, None], g["k%d" % t][None, None], g["v%d" % t][None, None])
        np.testing.assert_allclose(o[0, 0], g["o%d" % t], rtol=0, atol=1e-14)
        assert c.len == min(t, 2)
    np.testing.assert_allclose(c.keys()[0, 0], g["MK3"], rtol=0, atol=0)
    np.testing.assert_allclose(c.values()[0, 0], g["MV3"], rtol=0, atol=1e-14)


# ---------------------------------------------------------------------------------------
# Capacity >= sequence length, cache starting empty  ==>  full causal softmax attention
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,Hq,Hkv,d,T,C", [(2, 4, 2, 8, 13, 13), (1, 3, 1, 5, 9, 32), (2, 2, 2, 16, 20, 21)])
def test_capacity_ge_length_is_full_causal_attention(B, Hq, Hkv, d, T, C):
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    scale = 0.37
    c = O.OracleCache(B, Hq, Hkv, d, C, read_scale=scale)
    out = c.prefill_stream(q, k, v)
    assert c.len == T and c.n_written == 0
    G = Hq // Hkv
    tq = torch.from_numpy(q).permute(0, 2, 1, 3)                                   # [B,Hq,T,d]
    tk = torch.from_numpy(k).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)       # kv head h serves q heads h*G..
    tv = torch.from_numpy(v).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    ref = ref.permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    # and with a plain numpy causal attention, head by head
    for b in range(B):
        for h in range(Hq):
            s = scale * q[b, :, h] @ k[b, :, h // G].T
            s[np.triu_indices(T, 1)] = -np.inf
            np.testing.assert_allclose(out[b, :, h], _np_softmax(s) @ v[b, :, h // G], rtol=0, atol=1e-12)


def test_len_never_exceeds_capacity_and_keys_freeze():
    B, H, d, C, T = 1, 2, 4, 5, 17
    q, k, v = _rand(B, T, H, d), _rand(B, T, H, d), _rand(B, T, H, d)
    c = O.OracleCache(B, H, H, d, C)
    lens = []
    for t in range(T):
        c.decode_step(q[:, t], k[:, t], v[:, t])
        lens.append(c.len)
        assert c.MK.shape == (B * H, C, d) and c.MV.shape == (B * H, C, d)  # allocation fixed
    assert lens == [min(t + 1, C) for t in range(T)]
    # keys resident after the fill are exactly the first C write queries, untouched afterwards
    np.testing.assert_array_equal(c.keys()[0], np.transpose(k[0, :C], (1, 0, 2)))
    assert c.n_written == T - C


# ---------------------------------------------------------------------------------------
# Softmax rows sum to one
# ---------------------------------------------------------------------------------------
def test_weight_rows_sum_to_one():
    C, d = 257, 16
    MK = _rand(C, d)
    for scale in (1.0, 0.05, 7.0):
        ww = O.write_weights(MK, _rand(d), scale)
        assert abs(ww.sum() - 1.0) < 1e-14 and (ww >= 0).all()
        p = O.read_weights(MK[:100], _rand(d), scale)
        assert abs(p.sum() - 1.0) < 1e-14 and (p >= 0).all()
    big = O.write_weights(MK * 100.0, _rand(d) * 100.0, 1.0)  # scores ~1e4: max-subtraction needed
    assert np.isfinite(big).all() and abs(big.sum() - 1.0) < 1e-14


# ---------------------------------------------------------------------------------------
# Mass conservation: sum_j MV_t[j] - sum_j MV_{t-1}[j] = wv_t   (ww sums to one)
# ---------------------------------------------------------------------------------------
def test_mass_conservation_per_step_and_total():
    B, Hq, Hkv, d, C, T = 2, 4, 2, 8, 11, 9
    mk, mv = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    c = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, write_scale=0.8)
    prev = c.values().sum(axis=2).copy()
    for t in range(T):
        c.decode_step(q[:, t], k[:, t], v[:, t])
        cur = c.values().sum(axis=2)
        np.testing.assert_allclose(cur - prev, v[:, t], rtol=0, atol=1e-12)
        prev = cur.copy()
    np.testing.assert_allclose(c.values().sum(axis=2), mv.sum(axis=2) + v.sum(axis=1), rtol=0, atol=1e-11)
    np.testing.assert_array_equal(c.keys(), mk)


# ---------------------------------------------------------------------------------------
# Dense restatement (token-level parallelism, "Optimized for Parallelism"): with MK frozen
#   MV_N = MV_0 + softmax(Kc MK^T)^T Vc ,  O = Pr MV_0 + strict_tril(Pr WW^T) Vc
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("G", [1, 3])
def test_dense_two_matmul_restatement(G):
    d, C, T = 8, 10, 14
    rs, ws = 0.3, 0.9
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, T, G, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    c = O.OracleCache(1, G, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, read_scale=rs, write_scale=ws)
    out = c.prefill_stream(q, k, v)
    MK, MV0, Kc, Vc = mk[0, 0], mv0[0, 0], k[0, :, 0], v[0, :, 0]
    WW = _np_softmax(ws * Kc @ MK.T)                      # [T, C]
    np.testing.assert_allclose(c.values()[0, 0], MV0 + WW.T @ Vc, rtol=0, atol=1e-12)
    for g in range(G):
        Pr = _np_softmax(rs * q[0, :, g] @ MK.T)          # [T, C]
        A = np.tril(Pr @ WW.T, -1)                        # token t sees writes of tokens < t
        np.testing.assert_allclose(out[0, :, g], Pr @ MV0 + A @ Vc, rtol=0, atol=1e-12)


def test_write_then_read_differs_by_closed_form_term():
    d, C, T = 6, 7, 5
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, T, 1, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    a = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, read_scale=0.5)
    b = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, read_scale=0.5,
                      flags=O.WRITE_THEN_READ)
    oa, ob = a.prefill_stream(q, k, v), b.prefill_stream(q, k, v)
    np.testing.assert_allclose(a.values(), b.values(), rtol=0, atol=1e-13)
    for t in range(T):
        p = O.read_weights(mk[0, 0], q[0, t, 0], 0.5)
        ww = O.write_weights(mk[0, 0], k[0, t, 0], 1.0)
        np.testing.assert_allclose(ob[0, t, 0] - oa[0, t, 0], (p @ ww) * v[0, t, 0], rtol=0, atol=1e-12)


def test_skip_first_write_is_algorithm_1_literal():
    d, C, T = 4, 6, 5
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, T, 1, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    lit = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, flags=O.SKIP_FIRST_WRITE)
    lit.prefill_stream(q, k, v)
    WW = _np_softmax(k[0, :, 0] @ mk[0, 0].T)
    # Algorithm 1: MV_1 = MV_0, then MV_t = MV_{t-1} + ww_t^T wv_t for t = 2..N
    np.testing.assert_allclose(lit.values()[0, 0], mv0[0, 0] + WW[1:].T @ v[0, 1:, 0], rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------------------
# Closed forms of special cases
# ---------------------------------------------------------------------------------------
def test_zero_write_query_gives_uniform_write():
    d, C, T = 5, 8, 6
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, v = _rand(1, T, 1, d), _rand(1, T, 1, d)
    k = np.zeros((1, T, 1, d))
    c = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0)
    c.prefill_stream(q, k, v)
    expect = mv0[0, 0] + np.ones((C, 1)) / C * v[0, :, 0].sum(axis=0)[None, :]
    np.testing.assert_allclose(c.values()[0, 0], expect, rtol=0, atol=1e-13)
    # identical keys give the same uniform weights whatever the write query
    mk_same = np.repeat(_rand(1, 1, 1, d), C, axis=2)
    c2 = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk_same, mv_init=mv0)
    c2.prefill_stream(q, _rand(1, T, 1, d), v)
    np.testing.assert_allclose(c2.values()[0, 0], expect, rtol=0, atol=1e-12)


def test_capacity_one_is_running_sum():
    d, T = 4, 7
    mk, mv0 = _rand(1, 1, 1, d), _rand(1, 1, 1, d)
    q, k, v = _rand(1, T, 2, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    c = O.OracleCache(1, 2, 1, d, 1, init_len=1, mk_init=mk, mv_init=mv0)
    out = c.prefill_stream(q, k, v)
    run = mv0[0, 0, 0] + np.concatenate([np.zeros((1, d)), np.cumsum(v[0, :, 0], axis=0)])
    for t in range(T):  # o_t = MV_{t-1}: the fixed-size-state (RNN-like) corner of Table 1
        np.testing.assert_allclose(out[0, t, 0], run[t], rtol=0, atol=1e-13)
        np.testing.assert_allclose(out[0, t, 1], run[t], rtol=0, atol=1e-13)
    np.testing.assert_allclose(c.values()[0, 0, 0], run[T], rtol=0, atol=1e-13)


def test_hard_addressing_limit():
    d, C = 8, 8
    mk = np.eye(C, d)[None, None] * 1.0
    mv0 = _rand(1, 1, C, d)
    i, beta = 5, 200.0
    k = (beta * mk[0, 0, i])[None, None, None]
    v = _rand(1, 1, 1, d)
    c = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0)
    c.prefill_stream(_rand(1, 1, 1, d), k, v, want_out=False)
    expect = mv0[0, 0].copy()
    expect[i] += v[0, 0, 0]
    np.testing.assert_allclose(c.values()[0, 0], expect, rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------------------
# Invariances
# ---------------------------------------------------------------------------------------
def test_slot_permutation_equivariance():
    B, Hq, Hkv, d, C, T = 1, 2, 1, 6, 9, 7
    mk, mv0 = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    perm = RNG.permutation(C)
    a = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv0)
    b = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk[:, :, perm], mv_init=mv0[:, :, perm])
    oa, ob = a.prefill_stream(q, k, v), b.prefill_stream(q, k, v)
    np.testing.assert_allclose(oa, ob, rtol=0, atol=1e-12)
    np.testing.assert_allclose(a.values()[:, :, perm], b.values(), rtol=0, atol=1e-12)


def test_score_shift_invariance_and_value_linearity():
    d, C, T = 6, 8, 5
    mk, q, k, v = _rand(1, 1, C, d), _rand(1, T, 1, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    # make every q_t and k_t orthogonal to u up to a fixed component, so MK + c*u shifts all
    # scores of a token by the same constant
    u = np.zeros(d)
    u[0] = 1.0
    q[..., 0] = 0.7
    k[..., 0] = -1.3
    a = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk)  # MV_0 = 0
    b = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk + 50.0 * u)
    oa, ob = a.prefill_stream(q, k, v), b.prefill_stream(q, k, v)
    np.testing.assert_allclose(oa, ob, rtol=0, atol=1e-11)
    np.testing.assert_allclose(a.values(), b.values(), rtol=0, atol=1e-11)
    s = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk)
    os_ = s.prefill_stream(q, k, -2.5 * v)
    np.testing.assert_allclose(os_, -2.5 * oa, rtol=0, atol=1e-12)
    np.testing.assert_allclose(s.values(), -2.5 * a.values(), rtol=0, atol=1e-12)


def test_units_are_independent_and_gqa_head_mapping():
    B, Hq, Hkv, d, C, T = 2, 6, 3, 4, 5, 8
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    full = O.OracleCache(B, Hq, Hkv, d, C)
    out = full.prefill_stream(q, k, v)
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hkv):
            one = O.OracleCache(1, G, 1, d, C)
            o1 = one.prefill_stream(q[b:b + 1, :, h * G:(h + 1) * G], k[b:b + 1, :, h:h + 1], v[b:b + 1, :, h:h + 1])
            np.testing.assert_array_equal(o1[0], out[b, :, h * G:(h + 1) * G])
            np.testing.assert_array_equal(one.values()[0, 0], full.values()[b, h])


# ---------------------------------------------------------------------------------------
# Consistency: chunked streams concatenate; stream == repeated decode steps
# ---------------------------------------------------------------------------------------
def test_split_stream_equals_one_stream_and_decode_steps():
    B, Hq, Hkv, d, C, T = 2, 2, 1, 4, 6, 15
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    a = O.OracleCache(B, Hq, Hkv, d, C)
    oa = a.prefill_stream(q, k, v)
    b = O.OracleCache(B, Hq, Hkv, d, C)
    ob = np.concatenate([b.prefill_stream(q[:, :4], k[:, :4], v[:, :4]),
                         b.prefill_stream(q[:, 4:9], k[:, 4:9], v[:, 4:9]),
                         b.prefill_stream(q[:, 9:], k[:, 9:], v[:, 9:])], axis=1)
    np.testing.assert_array_equal(oa, ob)
    np.testing.assert_array_equal(a.values(), b.values())
    c = O.OracleCache(B, Hq, Hkv, d, C)
    oc = np.stack([c.decode_step(q[:, t], k[:, t], v[:, t]) for t in range(T)], axis=1)
    np.testing.assert_array_equal(oa, oc)
    # resume from an exported state
    r = O.OracleCache(B, Hq, Hkv, d, C, init_len=b.len, mk_init=b.keys(), mv_init=b.values())
    x = _rand(B, 3, Hq, d), _rand(B, 3, Hkv, d), _rand(B, 3, Hkv, d)
    np.testing.assert_array_equal(r.prefill_stream(*x), b.prefill_stream(*x))


# ---------------------------------------------------------------------------------------
# Brute force on tiny inputs, long-hand in pure Python (no numpy, no oracle code)
# ---------------------------------------------------------------------------------------
def _longhand(C, d, G, T, MK0, MV0, init_len, q, k, v, rs, ws):
    """Evaluate the method token by token with Python scalars and math.exp only."""
    MK = [[MK0[j][e] for e in range(d)] for j in range(init_len)]
    MV = [[MV0[j][e] for e in range(d)] for j in range(init_len)]
    outs = []
    for t in range(T):
        full = len(MK) == C
        if not full:
            MK.append(list(k[t]))
            MV.append(list(v[t]))
        n = len(MK)
        row = []
        for g in range(G):
            sc = [rs * sum(q[t][g][e] * MK[j][e] for e in range(d)) for j in range(n)]
            z = sum(math.exp(x) for x in sc)              # no max-subtraction: tiny scores
            row.append([sum(math.exp(sc[j]) / z * MV[j][e] for j in range(n)) for e in range(d)])
        outs.append(row)
        if full:
            sc = [ws * sum(k[t][e] * MK[j][e] for e in range(d)) for j in range(C)]
            z = sum(math.exp(x) for x in sc)
            MV = [[MV[j][e] + math.exp(sc[j]) / z * v[t][e] for e in range(d)] for j in range(C)]
    return outs, MV


@pytest.mark.parametrize("C,d,G,T,init_len", [(1, 1, 1, 3, 0), (2, 2, 1, 4, 0), (3, 2, 2, 4, 3), (3, 1, 1, 4, 1),
                                              (2, 2, 2, 3, 2)])
def test_brute_force_tiny(C, d, G, T, init_len):
    MK0, MV0 = _rand(C, d), _rand(C, d)
    q, k, v = _rand(T, G, d), _rand(T, d), _rand(T, d)
    rs, ws = 0.6, 1.1
    outs, MV = _longhand(C, d, G, T, MK0.tolist(), MV0.tolist(), init_len, q.tolist(), k.tolist(), v.tolist(), rs, ws)
    c = O.OracleCache(1, G, 1, d, C, read_scale=rs, write_scale=ws, init_len=init_len,
                      mk_init=MK0[None, None, :init_len] if init_len else None,
                      mv_init=MV0[None, None, :init_len] if init_len else None)
    out = c.prefill_stream(q[None], k[None, :, None], v[None, :, None])
    np.testing.assert_allclose(out[0], np.array(outs), rtol=0, atol=1e-12)
    np.testing.assert_allclose(c.values()[0, 0, :len(MV)], np.array(MV), rtol=0, atol=1e-12)


def test_default_scales():
    d, C = 16, 4
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, 1, 1, d), _rand(1, 1, 1, d), _rand(1, 1, 1, d)
    c = O.OracleCache(1, 1, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0)
    o = c.prefill_stream(q, k, v)
    p = _np_softmax((q[0, 0, 0] @ mk[0, 0].T) / math.sqrt(d))  # textbook 1/sqrt(d) read scale
    ww = _np_softmax(k[0, 0, 0] @ mk[0, 0].T)                  # Algorithm 1 prints no write scale
    np.testing.assert_allclose(o[0, 0, 0], p @ mv0[0, 0], rtol=0, atol=1e-13)
    np.testing.assert_allclose(c.values()[0, 0], mv0[0, 0] + np.outer(ww, v[0, 0, 0]), rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------------------
# Step size of each token's write (Features, "Learning Rate Adaptation"), read as
#   MV_t = MV_{t-1} + eta_t * ww_t^T wv_t
# ---------------------------------------------------------------------------------------
def test_step_size_one_is_the_printed_rule_bit_for_bit():
    B, Hq, Hkv, d, C, T = 2, 4, 2, 6, 5, 9
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    a = O.OracleCache(B, Hq, Hkv, d, C)
    b = O.OracleCache(B, Hq, Hkv, d, C)
    np.testing.assert_array_equal(a.prefill_stream(q, k, v), b.prefill_stream(q, k, v, eta=np.ones((B, T, Hkv))))
    np.testing.assert_array_equal(a.values(), b.values())


def test_step_size_scales_the_mass_each_token_adds():
    B, Hq, Hkv, d, C, T = 2, 2, 2, 8, 7, 6
    mk, mv = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    eta = RNG.uniform(-0.5, 2.0, size=(B, T, Hkv))
    c = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv)
    prev = c.values().sum(axis=2).copy()
    for t in range(T):
        c.decode_step(q[:, t], k[:, t], v[:, t], eta=eta[:, t])
        cur = c.values().sum(axis=2)
        np.testing.assert_allclose(cur - prev, eta[:, t, :, None] * v[:, t], rtol=0, atol=1e-12)
        prev = cur.copy()
    np.testing.assert_array_equal(c.keys(), mk)


@pytest.mark.parametrize("flags", [0, O.WRITE_THEN_READ])
def test_step_size_dense_restatement(flags):
    # MV_N = MV_0 + WW^T diag(eta) Vc ;  O = Pr MV_0 + tril(Pr WW^T) diag(eta) Vc
    d, C, T, G = 8, 9, 12, 2
    rs, ws = 0.4, 0.7
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, T, G, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    eta = RNG.uniform(0.0, 1.5, size=(1, T, 1))
    c = O.OracleCache(1, G, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, read_scale=rs, write_scale=ws, flags=flags)
    out = c.prefill_stream(q, k, v, eta=eta)
    MK, MV0, Kc, Vc = mk[0, 0], mv0[0, 0], k[0, :, 0], v[0, :, 0]
    EV = eta[0, :, 0, None] * Vc
    WW = _np_softmax(ws * Kc @ MK.T)
    np.testing.assert_allclose(c.values()[0, 0], MV0 + WW.T @ EV, rtol=0, atol=1e-12)
    for g in range(G):
        Pr = _np_softmax(rs * q[0, :, g] @ MK.T)
        A = np.tril(Pr @ WW.T, 0 if flags else -1)
        np.testing.assert_allclose(out[0, :, g], Pr @ MV0 + A @ EV, rtol=0, atol=1e-12)


def test_step_size_zero_freezes_the_state_and_fill_phase_ignores_it():
    B, Hq, Hkv, d, C, T = 1, 2, 1, 4, 6, 10
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    eta = np.zeros((B, T, Hkv))
    a = O.OracleCache(B, Hq, Hkv, d, C)
    oa = a.prefill_stream(q, k, v, eta=eta)
    # the six fill tokens are appended as they are; afterwards nothing changes
    np.testing.assert_array_equal(a.keys()[0, 0], k[0, :C, 0])
    np.testing.assert_array_equal(a.values()[0, 0], v[0, :C, 0])
    for t in range(C, T):  # a frozen cache: plain attention over the six appended slots
        for g in range(Hq):
            p = _np_softmax(q[0, t, g] @ k[0, :C, 0].T / math.sqrt(d))
            np.testing.assert_allclose(oa[0, t, g], p @ v[0, :C, 0], rtol=0, atol=1e-13)
    b = O.OracleCache(B, Hq, Hkv, d, C)
    ob = b.prefill_stream(q[:, :C], k[:, :C], v[:, :C])            # fill phase with and without eta
    np.testing.assert_array_equal(oa[:, :C], ob)


def test_step_size_equals_a_scaled_write_value_in_the_full_phase():
    B, Hq, Hkv, d, C, T = 2, 4, 2, 5, 4, 7
    mk, mv = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    q, k, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    eta = RNG.uniform(0.1, 3.0, size=(B, T, Hkv))
    for flags in (0, O.WRITE_THEN_READ):
        a = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, flags=flags)
        b = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, flags=flags)
        oa = a.prefill_stream(q, k, v, eta=eta)
        ob = b.prefill_stream(q, k, eta[..., None] * v)
        np.testing.assert_allclose(oa, ob, rtol=0, atol=1e-12)
        np.testing.assert_allclose(a.values(), b.values(), rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------------------
# Projections in front of the layer (Algorithm 1: wq_t = W_wq x_t, wv_t = W_wv x_t)
# ---------------------------------------------------------------------------------------
def test_projection_brute_force_and_operand_roles():
    M, K, N = 3, 4, 5                               # all different: a transposed operand cannot pass
    x, W = _rand(M, K), _rand(N, K)
    y = O.project(x, W)
    assert y.shape == (M, N)
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(x[m, k]) * float(W[n, k])
            assert abs(y[m, n] - acc) <= 1e-14
    # one-hot token picks a column of W; identity weights return the token
    e = np.zeros((1, K)); e[0, 2] = 1.0
    np.testing.assert_array_equal(O.project(e, W)[0], W[:, 2])
    np.testing.assert_array_equal(O.project(x, np.eye(K)), x)
    # linear in both arguments, leading dimensions kept
    x3 = _rand(2, 3, K)
    np.testing.assert_allclose(O.project(2.0 * x3 + 1.0, W), 2.0 * O.project(x3, W) + W.sum(axis=1), rtol=0, atol=1e-13)
    assert O.project(x3, W).shape == (2, 3, N)


def test_round_bf16_is_nearest_even_on_the_bfloat16_grid():
    vals = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -0.3, 1e-3, 255.5, 0.0])
    got = O.round_bf16(vals)
    # ties go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3 * 2^-8 -> 1 + 2^-6
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.0 + 2.0 ** -7 and got[3] == 1.0 + 2.0 ** -6
    ref = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(got, ref)
    assert np.all(np.abs(got - vals) <= np.abs(vals) * 2.0 ** -8)


def test_layer_step_inputs_feed_the_layer():
    # a layer with identity-like projections is the plain layer on the tokens themselves
    B, T, Hq, Hkv, d, C = 1, 5, 1, 1, 4, 3
    x = _rand(B, T, d)
    I = np.eye(d)
    q, k, v = O.layer_step_inputs(x, I, 2.0 * I, -I, Hq, Hkv, d, bf16=False)
    f32 = x.astype(np.float32).astype(np.float64)
    np.testing.assert_array_equal(q[:, :, 0], f32)
    np.testing.assert_allclose(k[:, :, 0], 2.0 * f32, rtol=1e-7)
    np.testing.assert_allclose(v[:, :, 0], -f32, rtol=1e-7)
    a = O.OracleCache(B, Hq, Hkv, d, C)
    b = O.OracleCache(B, Hq, Hkv, d, C)
    np.testing.assert_array_equal(a.prefill_stream(q, k, v), b.prefill_stream(f32[:, :, None], 2 * f32[:, :, None], -f32[:, :, None]))


def test_layer_step_inputs_head_split_with_several_heads():
    # Weights stacked from per-head scaled identities: head h of q must be (h + 1) x, head h of the write query
    # -(h + 1) x and of the write value 10 (h + 1) x, token by token and sequence by sequence.  Hq != Hkv, B > 1 and
    # T != H != d, so that a split along the wrong axis, a transposed (T, H) order or a swapped k / v cannot pass.
    B, T, Hq, Hkv, d = 2, 5, 6, 3, 4
    x = _rand(B, T, d)
    I = np.eye(d)
    Wq = np.concatenate([(h + 1.0) * I for h in range(Hq)], axis=0)            # [Hq * d, d]
    Wwq = np.concatenate([-(h + 1.0) * I for h in range(Hkv)], axis=0)         # [Hkv * d, d]
    Wwv = np.concatenate([10.0 * (h + 1.0) * I for h in range(Hkv)], axis=0)
    q, k, v = O.layer_step_inputs(x, Wq, Wwq, Wwv, Hq, Hkv, d, bf16=False)
    assert q.shape == (B, T, Hq, d) and k.shape == (B, T, Hkv, d) and v.shape == (B, T, Hkv, d)
    f32 = lambda z: np.asarray(z, dtype=np.float32).astype(np.float64)
    for b in range(B):
        for t in range(T):
            for h in range(Hq):
                np.testing.assert_array_equal(q[b, t, h], f32((h + 1.0) * x[b, t]))
            for h in range(Hkv):
                np.testing.assert_array_equal(k[b, t, h], f32(-(h + 1.0) * x[b, t]))
                np.testing.assert_array_equal(v[b, t, h], f32(10.0 * (h + 1.0) * x[b, t]))
    # with bfloat16 storage every element is the nearest bfloat16 of the same product
    qb, kb, vb = O.layer_step_inputs(x, Wq, Wwq, Wwv, Hq, Hkv, d, bf16=True)
    ref = torch.tensor(3.0 * x[1, 2], dtype=torch.float32).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(qb[1, 2, 2], ref)
    # and the layer on those vectors is the layer fed head by head: kv-head h serves query heads h*G .. h*G+G-1
    C, G = 3, Hq // Hkv
    whole = O.OracleCache(B, Hq, Hkv, d, C)
    out = whole.prefill_stream(q, k, v)
    for h in range(Hkv):
        one = O.OracleCache(B, G, 1, d, C)
        qs = np.stack([f32((h * G + g + 1.0) * x) for g in range(G)], axis=2)
        o1 = one.prefill_stream(qs, f32(-(h + 1.0) * x)[:, :, None], f32(10.0 * (h + 1.0) * x)[:, :, None])
        np.testing.assert_array_equal(out[:, :, h * G:(h + 1) * G], o1)


def test_update_kv_is_algorithm_1():
    # UpdateKV(x_1..x_N, MV_0, MK, ...) returns MV_N = MV_0 + sum_t ww_t^T wv_t, reads nothing, leaves MK alone
    B, Hq, Hkv, d, C, T = 2, 4, 2, 6, 5, 11
    mk, mv = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    k, v = _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    c = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, write_scale=0.7)
    c.update_kv(k, v)
    for b in range(B):
        for h in range(Hkv):
            WW = _np_softmax(0.7 * k[b, :, h] @ mk[b, h].T)
            np.testing.assert_allclose(c.values()[b, h], mv[b, h] + WW.T @ v[b, :, h], rtol=0, atol=1e-12)
    np.testing.assert_array_equal(c.keys(), mk)
    assert c.len == C and c.n_written == T


# ---------------------------------------------------------------------------------------
# Write threshold (a reading of the library, not of the paper): slots with ww_j < write_eps keep their row
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, O.WRITE_THEN_READ])
def test_write_threshold_masked_two_matmul_restatement(flags):
    # MV_N = MV_0 + (WW * [WW >= eps])^T Vc ;  O = Pr MV_0 + tril(Pr (WW * mask)^T) Vc: the read of a token that
    # follows its own write sees the rows actually rewritten.  eps = 0 is the printed rule, bit for bit.
    d, C, T, G, eps = 6, 11, 9, 2, 0.08
    mk, mv0 = _rand(1, 1, C, d), _rand(1, 1, C, d)
    q, k, v = _rand(1, T, G, d), _rand(1, T, 1, d), _rand(1, T, 1, d)
    eta = RNG.uniform(0.2, 1.5, size=(1, T, 1))
    c = O.OracleCache(1, G, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, read_scale=0.5, write_scale=0.9, flags=flags,
                      write_eps=eps)
    out = c.prefill_stream(q, k, v, eta=eta)
    MK, MV0, Kc, Vc = mk[0, 0], mv0[0, 0], k[0, :, 0], v[0, :, 0]
    WW = _np_softmax(0.9 * Kc @ MK.T)
    assert (WW < eps).any() and (WW >= eps).any()                      # the threshold bites, but not everywhere
    WM = np.where(WW >= eps, WW, 0.0)
    EV = eta[0, :, 0, None] * Vc
    np.testing.assert_allclose(c.values()[0, 0], MV0 + WM.T @ EV, rtol=0, atol=1e-12)
    for g in range(G):
        Pr = _np_softmax(0.5 * q[0, :, g] @ MK.T)
        A = np.tril(Pr @ WM.T, 0 if flags else -1)
        np.testing.assert_allclose(out[0, :, g], Pr @ MV0 + A @ EV, rtol=0, atol=1e-12)
    # mass added per token = (sum of the weights that pass) * eta_t * v_t
    np.testing.assert_allclose(c.values()[0, 0].sum(axis=0) - MV0.sum(axis=0), (WM.sum(axis=1)[:, None] * EV).sum(axis=0),
                               rtol=0, atol=1e-12)
    a = O.OracleCache(1, G, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, flags=flags, write_eps=0.0)
    b = O.OracleCache(1, G, 1, d, C, init_len=C, mk_init=mk, mv_init=mv0, flags=flags)
    np.testing.assert_array_equal(a.prefill_stream(q, k, v), b.prefill_stream(q, k, v))
    np.testing.assert_array_equal(a.values(), b.values())


def test_write_threshold_against_uniform_weights():
    # a zero write query gives ww_j = 1/C exactly: a threshold just above 1/C freezes the state, one at 1/C does not
    B, Hq, Hkv, d, C, T = 1, 1, 1, 3, 8, 4
    mk, mv = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    q, v = _rand(B, T, Hq, d), _rand(B, T, Hkv, d)
    k = np.zeros((B, T, Hkv, d))
    frozen = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, write_eps=0.126)
    frozen.prefill_stream(q, k, v)
    np.testing.assert_array_equal(frozen.values(), mv)
    live = O.OracleCache(B, Hq, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv, write_eps=0.125)
    live.prefill_stream(q, k, v)
    np.testing.assert_allclose(live.values()[0, 0], mv[0, 0] + v[0, :, 0].sum(axis=0)[None, :] / C, rtol=0, atol=1e-13)
    # the fill phase appends whatever the threshold
    f = O.OracleCache(B, Hq, Hkv, d, C, write_eps=0.9)
    f.prefill_stream(q, _rand(B, T, Hkv, d), v)
    np.testing.assert_array_equal(f.values()[0, 0, :T], v[0, :, 0])


# ---------------------------------------------------------------------------------------
# Backward of UpdateKV in its token-parallel form ("Optimized for Parallelism"): pinned by central
# finite differences of the forward oracle, by automatic differentiation of the two-matmul form,
# and by closed forms
# ---------------------------------------------------------------------------------------
def _loss_through_forward(mk, mv0, k, v, eta, G, ws, eps=0.0):
    """L = <G, MV_N> with MV_N from the forward oracle's sequential loop."""
    B, Hkv, C, d = mk.shape
    c = O.OracleCache(B, Hkv, Hkv, d, C, init_len=C, mk_init=mk, mv_init=mv0, write_scale=ws, write_eps=eps)
    c.update_kv(k, v, eta=eta)
    return float((G * c.values()).sum())


def test_update_kv_backward_against_finite_differences_of_the_forward_oracle():
    B, Hkv, C, d, T, ws = 2, 2, 5, 3, 4, 0.8
    mk, mv0 = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    k, v = _rand(B, T, Hkv, d), _rand(B, T, Hkv, d)
    eta = RNG.uniform(0.3, 1.7, size=(B, T, Hkv))
    G = _rand(B, Hkv, C, d)
    dk, dv, dmk, deta = O.update_kv_backward(mk, k, v, G, eta=eta, write_scale=ws)
    h = 1e-6

    def fd(arr, idx, which):
        out = []
        for sgn in (+1, -1):
            a = arr.copy()
            a[idx] += sgn * h
            args = dict(mk=mk, mv0=mv0, k=k, v=v, eta=eta)
            args[which] = a
            out.append(_loss_through_forward(args["mk"], args["mv0"], args["k"], args["v"], args["eta"], G, ws))
        return (out[0] - out[1]) / (2 * h)

    for which, arr, grad in (("k", k, dk), ("v", v, dv), ("mk", mk, dmk), ("eta", eta, deta), ("mv0", mv0, G)):
        for _ in range(12):
            idx = tuple(int(RNG.integers(0, n)) for n in arr.shape)
            assert abs(fd(arr, idx, which) - grad[idx]) <= 2e-8 * (1 + abs(grad[idx])), (which, idx)


def test_update_kv_backward_against_autograd_of_the_two_matmul_form():
    B, Hkv, C, d, T, ws = 1, 3, 7, 4, 6, 1.3
    mk, k, v, G = _rand(B, Hkv, C, d), _rand(B, T, Hkv, d), _rand(B, T, Hkv, d), _rand(B, Hkv, C, d)
    eta = RNG.uniform(0.0, 2.0, size=(B, T, Hkv))
    dk, dv, dmk, deta = O.update_kv_backward(mk, k, v, G, eta=eta, write_scale=ws)
    tmk, tk, tv, te = (torch.tensor(a, requires_grad=True) for a in (mk, k, v, eta))
    loss = 0.0
    for h in range(Hkv):   # MV_N - MV_0 = softmax(ws Kc MK^T)^T diag(eta) Vc, head by head
        WW = torch.softmax(ws * tk[0, :, h] @ tmk[0, h].T, dim=-1)
        loss = loss + (torch.tensor(G[0, h]) * (WW.T @ (te[0, :, h, None] * tv[0, :, h]))).sum()
    loss.backward()
    for got, ref in ((dk, tk.grad), (dv, tv.grad), (dmk, tmk.grad), (deta, te.grad)):
        np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=1e-12)


def test_update_kv_backward_closed_forms():
    B, Hkv, C, d, T = 1, 1, 6, 3, 5
    mk, v, G = _rand(B, Hkv, C, d), _rand(B, T, Hkv, d), _rand(B, Hkv, C, d)
    eta = RNG.uniform(0.5, 1.5, size=(B, T, Hkv))
    # a zero write query writes uniformly: dwv_t = eta_t * mean_j G_j, and dwq_t is the covariance, under the
    # uniform weights, of <wv_t, G_j> with MK_j
    k0 = np.zeros((B, T, Hkv, d))
    dk, dv, dmk, deta = O.update_kv_backward(mk, k0, v, G, eta=eta, write_scale=0.7)
    gbar = G[0, 0].mean(axis=0)
    np.testing.assert_allclose(dv[0, :, 0], eta[0, :, 0, None] * gbar[None, :], rtol=0, atol=1e-13)
    np.testing.assert_allclose(deta[0, :, 0], v[0, :, 0] @ gbar, rtol=0, atol=1e-13)
    a = v[0, :, 0] @ G[0, 0].T                                  # [T, C]: <wv_t, G_j>
    cov = ((a - a.mean(axis=1, keepdims=True))[:, :, None] * mk[0, 0][None]).mean(axis=1)
    np.testing.assert_allclose(dk[0, :, 0], 0.7 * eta[0, :, 0, None] * cov, rtol=0, atol=1e-13)
    np.testing.assert_allclose(dmk, 0.0, atol=1e-13)           # dMK_j is proportional to the write queries: zero here
    # a G whose rows are all equal tells the softmax nothing: dwq = 0, dMK = 0, dwv_t = eta_t * that row
    k = _rand(B, T, Hkv, d)
    Gc = np.broadcast_to(_rand(d), (B, Hkv, C, d)).copy()
    dk, dv, dmk, deta = O.update_kv_backward(mk, k, v, Gc, eta=eta, write_scale=1.0)
    np.testing.assert_allclose(dk, 0.0, atol=1e-13)
    np.testing.assert_allclose(dmk, 0.0, atol=1e-13)
    np.testing.assert_allclose(dv[0, :, 0], eta[0, :, 0, None] * Gc[0, 0, 0][None, :], rtol=0, atol=1e-13)
    # eta = 0 leaves the state alone: only deta survives
    dk, dv, dmk, deta = O.update_kv_backward(mk, k, v, G, eta=np.zeros((B, T, Hkv)))
    assert not dk.any() and not dv.any() and not dmk.any() and np.abs(deta).max() > 0
    # units do not mix, and the gradient is linear in G
    mk2, k2, v2, G2 = _rand(2, 2, C, d), _rand(2, T, 2, d), _rand(2, T, 2, d), _rand(2, 2, C, d)
    full = O.update_kv_backward(mk2, k2, v2, G2)
    one = O.update_kv_backward(mk2[1:, 1:], k2[1:, :, 1:], v2[1:, :, 1:], G2[1:, 1:])
    np.testing.assert_array_equal(full[0][1:, :, 1:], one[0])
    np.testing.assert_array_equal(full[2][1:, 1:], one[2])
    twice = O.update_kv_backward(mk2, k2, v2, 2.0 * G2)
    for a, b in zip(full, twice):
        np.testing.assert_allclose(2.0 * a, b, rtol=0, atol=1e-13)


def test_update_kv_backward_with_the_write_threshold():
    # the mask of dropped slots is piecewise constant: away from the threshold the gradient is that of the masked sum
    B, Hkv, C, d, T, ws, eps = 1, 1, 8, 3, 3, 1.1, 0.07
    mk, mv0 = _rand(B, Hkv, C, d), _rand(B, Hkv, C, d)
    k, v, G = _rand(B, T, Hkv, d), _rand(B, T, Hkv, d), _rand(B, Hkv, C, d)
    WW = _np_softmax(ws * k[0, :, 0] @ mk[0, 0].T)
    assert (WW < eps).any() and (WW >= eps).any() and np.abs(WW - eps).min() > 1e-3
    dk, dv, dmk, deta = O.update_kv_backward(mk, k, v, G, write_scale=ws, write_eps=eps)
    h = 1e-6
    for which, arr, grad in (("k", k, dk), ("v", v, dv), ("mk", mk, dmk)):
        for _ in range(10):
            idx = tuple(int(RNG.integers(0, n)) for n in arr.shape)
            vals = []
            for sgn in (+1, -1):
                a = arr.copy()
                a[idx] += sgn * h
                args = dict(mk=mk, k=k, v=v)
                args[which] = a
                vals.append(_loss_through_forward(args["mk"], mv0, args["k"], args["v"], None, G, ws, eps))
            assert abs((vals[0] - vals[1]) / (2 * h) - grad[idx]) <= 2e-8 * (1 + abs(grad[idx])), (which, idx)
