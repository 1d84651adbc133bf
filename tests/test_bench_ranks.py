"""Host-side logic of the multi-process benchmark path, on CPU with gloo (world size 2):
replicas only -- every rank reports its own time, the slowest one counts -- and the
reference arm prints one line from rank 0 while the other ranks exit quietly."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["GAR_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
got = bench.max_over_ranks(10.0 + 5.0 * rank, world)
assert got == 10.0 + 5.0 * (world - 1), got
dist.barrier()
sys.stdout.write("rank %d ok %.1f\n" % (rank, got)); sys.stdout.flush()
dist.destroy_process_group()
"""


def _torchrun(args, port):
    env = dict(os.environ, GAR_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    return subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=600)


def test_max_over_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    res = _torchrun([str(script)], 29731)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok 15.0") == 2


def test_reference_arm_under_torchrun_prints_one_line():
    res = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                     "--warmup", "0", "--ref-sample", "4096"], 29733)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0


def test_paper_protocol_statistic_drops_the_two_farthest_from_the_median():
    """Section 5.1: seven runs, the two farthest from the median removed, mean and deviation of five."""
    from paper_1905_04374_b200.paper_sweep import robust_mean_std
    runs = [10.0, 10.2, 9.9, 10.1, 50.0, 10.0, 0.5]          # median 10.0; 50.0 and 0.5 are the outliers
    mean, std = robust_mean_std(runs)
    kept = [10.0, 10.2, 9.9, 10.1, 10.0]
    assert abs(mean - sum(kept) / 5) < 1e-12
    assert abs(std - (sum((k - mean) ** 2 for k in kept) / 5) ** 0.5) < 1e-12
    # both outliers on one side are dropped as well
    mean2, _ = robust_mean_std([1.0, 1.0, 1.0, 1.0, 1.0, 9.0, 8.0])
    assert mean2 == 1.0
    # with five runs nothing is dropped
    assert robust_mean_std([1.0, 2.0, 3.0, 4.0, 5.0])[0] == 3.0
