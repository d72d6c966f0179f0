"""The multi-GPU path of bench.py is N independent replicas (one request per rank, no exchange step): what the
ranks share is the barrier, the max-over-ranks timing and the whole-job arithmetic. Its other mode deals the layers of
one request out over the ranks. Two CPU processes over gloo."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    from paper_2604_06694_b200 import workloads as wl
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    # every rank times its own replica; the job's step time is the slowest rank's
    local_ms = 1.0 + 0.5 * rank
    ms = bench.max_over_ranks(local_ms, world)
    assert ms == 1.5, ms
    dist.barrier()
    # weak scaling: world x the layers in the same time
    assert bench.whole_job_us_per_layer(ms, 28, world) == 1.5e3 / 56
    # the ranks draw different requests of the same shape
    spec = wl.config(0)
    w = wl.generate(spec, seed=bench.rank_seed(rank))
    digest = float(w.k.astype("float64").sum())
    out = [None] * world
    dist.all_gather_object(out, digest)
    assert out[0] != out[1]
    # the layer-sharded mode: one request, its layers dealt out over the ranks; the shards are disjoint, cover the
    # stack, hold exactly the full draw's layers, and every rank holds the whole head-score table and total budget
    import dataclasses, numpy as np
    spec3 = dataclasses.replace(spec, n_layers=3)
    full = wl.generate(spec3, seed=0)
    l0, l1 = wl.layer_shard(3, world, rank)
    mine = wl.generate(spec3, seed=0, layer_range=(l0, l1))
    assert np.array_equal(mine.k, full.k[l0:l1]) and np.array_equal(mine.q, full.q[:, l0:l1])
    assert np.array_equal(mine.head_scores, full.head_scores) and np.array_equal(mine.total_budget, full.total_budget)
    assert mine.layer_begin == l0 and mine.full_layers == 3 and mine.spec.n_layers == l1 - l0
    heads = wl.shard_heads(len(spec3.seq_lens), 3, spec3.n_kv_heads, l0, l1).tolist()
    parts = [None] * world
    dist.all_gather_object(parts, (l0, l1, heads))
    assert [p[:2] for p in parts] == [(0, 2), (2, 3)]
    assert sorted(h for p in parts for h in p[2]) == list(range(len(spec3.seq_lens) * 3 * spec3.n_kv_heads))
    dist.destroy_process_group()
    print("rank", rank, "ok")
""") % ROOT


def test_two_ranks_over_gloo(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=300)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
