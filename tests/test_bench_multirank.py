"""The multi-GPU path of bench.py is N independent replicas (one request per rank, no exchange step): what the
ranks share is the barrier, the max-over-ranks timing and the whole-job arithmetic. Two CPU processes over gloo."""
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
