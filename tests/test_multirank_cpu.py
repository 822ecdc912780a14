"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): the path shards by sequence with no
data-path collective, so what N > 1 adds is per-rank seeding, the max-over-ranks timing reduction and
rank 0 alone printing the result line."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, port, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_and_seeding_gloo(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys
        sys.path.insert(0, {ROOT!r})
        import torch, torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        slowest = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu", world)
        seeds = [None] * world
        dist.all_gather_object(seeds, bench.rank_seed(2, rank))
        print(f"RESULT rank={{rank}} world={{world}} slowest={{slowest}} seeds={{seeds}}", flush=True)
        dist.destroy_process_group()
    """))
    res = _torchrun([str(script)], 29731)
    assert res.returncode == 0, res.stdout + res.stderr
    import re
    # both ranks agree on the slowest rank's time; inputs are seeded per rank (the two ranks' lines can share a line)
    ranks = re.findall(r"RESULT rank=(\d) world=2 slowest=15\.0 seeds=\[2000, 2001\]", res.stdout)
    assert sorted(ranks) == ["0", "1"], res.stdout


def test_reference_arm_prints_one_line_from_rank_zero():
    res = _torchrun(["bench.py", "--impl", "reference", "--config", "tiny", "--gpus", "2", "--steps", "1",
                     "--warmup", "0"], 29732)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = [json.loads(ln) for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
