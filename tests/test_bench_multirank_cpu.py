"""Host logic of the multi-GPU benchmark path on CPU: two gloo ranks shard nothing but seeds
(units never interact) and agree on the slowest rank's time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent('''
    import os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    from paper_2411_15785_b200 import workloads as W
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    w = W.CONFIGS["mha7b_b64_c2048"].scaled(batch=2, n_q_heads=2, n_kv_heads=2, capacity=8, init_len=8)
    wr = bench.rank_workload(w, rank)
    assert wr.batch == w.batch and wr.seed == w.seed + 1000 * rank
    q0 = W.step_inputs(wr, 0)[0]
    gathered = [torch.empty_like(q0) for _ in range(world)]
    dist.all_gather(gathered, q0)
    assert not torch.equal(gathered[0], gathered[1])          # different data per rank
    ms = bench.max_over_ranks([10.0 + rank, 5.0 - rank], "cpu")
    assert ms == [10.0 + world - 1, 5.0], ms                  # slowest rank wins, on every rank
    dist.barrier()
    dist.destroy_process_group()
    print("ok", rank)
''') % ROOT


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert r.stdout.count("ok") == 2
