"""The seeded input recipes: shapes, dtypes, determinism, statelessness, value scales."""
import torch

from paper_2411_15785_b200 import workloads as W


def test_configs_present_and_shapes():
    names = set(W.CONFIGS)
    assert {"single_fp32_c128", "mha7b_b64_c2048", "gqa8b_b128_c4096", "stream_b8_c1024",
            "sweep_b256_c256", "sweep_b256_c1024", "sweep_b256_c4096", "sweep_b256_c16384"} <= names
    w = W.CONFIGS["gqa8b_b128_c4096"]
    assert (w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.group, w.units) == (128, 32, 8, 128, 4096, 4, 1024)
    assert W.CONFIGS["single_fp32_c128"].init_len == 0 and W.CONFIGS["mha7b_b64_c2048"].init_len == 2048


def test_step_inputs_deterministic_and_stateless():
    w = W.CONFIGS["mha7b_b64_c2048"].scaled(batch=2)
    a = W.step_inputs(w, 7)
    W.step_inputs(w, 3)
    b = W.step_inputs(w, 7)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    q, k, v = a
    assert q.shape == (2, 32, 128) and k.shape == (2, 32, 128) and v.dtype == torch.bfloat16
    assert not torch.equal(W.step_inputs(w, 8)[0], q)
    assert abs(q.float().std().item() - 128 ** -0.5) < 0.01 and abs(k.float().std().item() - 1.0) < 0.05


def test_initial_cache_per_sequence_matches_batch():
    w = W.CONFIGS["mha7b_b64_c2048"].scaled(batch=3, n_q_heads=2, n_kv_heads=2, capacity=16, init_len=16)
    mk, mv = W.initial_cache(w)
    assert mk.shape == (3, 2, 16, 128) and mk.dtype == torch.bfloat16
    k1, v1 = W.initial_cache_seq(w, 1)
    assert torch.equal(mk[1], k1) and torch.equal(mv[1], v1)
    assert not torch.equal(mk, mv)


def test_stream_inputs_assemble_from_blocks():
    w = W.CONFIGS["stream_b8_c1024"].scaled(batch=1, n_q_heads=2, n_kv_heads=2, head_dim=8)
    q, k, v = W.stream_inputs(w, W.STREAM_BLOCK - 3, 10)
    b0, b1 = W.stream_block(w, 0), W.stream_block(w, 1)
    assert q.shape == (1, 10, 2, 8)
    assert torch.equal(q[:, :3], b0[0][:, -3:]) and torch.equal(v[:, 3:], b1[2][:, :7])
