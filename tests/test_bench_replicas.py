"""The multi-GPU plumbing of bench.py is "N independent replicas": no data-path collective, a
barrier, and the MAX over ranks of the timed duration.  Checked here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    bench.barrier(world)
    ms = bench.reduce_max_ms(10.0 * (rank + 1), world, backend_device="cpu")   # rank 1 is the slow replica
    steps = 5
    value = world * steps / (ms * 1e-3)                                         # whole-job tokens/s
    with open(os.path.join({out!r}, f"rank{{rank}}.json"), "w") as f:           # one file per rank: stdout interleaves
        json.dump({{"rank": rank, "ms": ms, "value": value}}, f)
    dist.destroy_process_group()
""")


def test_two_gloo_ranks_take_the_max_duration(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, out=str(tmp_path)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29631", str(script)],
                         capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.load(open(tmp_path / f"rank{r}.json")) for r in (0, 1)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["ms"] == 20.0                      # the slower replica's time on every rank
        assert abs(r["value"] - 2 * 5 / 0.020) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=120, env=env, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""
