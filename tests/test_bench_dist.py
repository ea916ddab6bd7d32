"""The multi-rank plumbing of bench.py on CPU: two gloo ranks agree on the max-over-ranks time."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, os.environ["M2_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group(backend="gloo", init_method="env://")
r = dist.get_rank()
bench.barrier()
m = bench.reduce_max(10.0 + 5.0 * r)
assert m == 15.0, m
# weak scaling: every rank processes the same number of units; aggregate = world * units / max time
units = 1000
agg = dist.get_world_size() * units / m
assert abs(agg - 2000 / 15.0) < 1e-12
bench.barrier()
dist.destroy_process_group()
print("rank", r, "ok")
"""


def test_two_gloo_ranks_reduce_max(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    env = dict(os.environ, M2_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29531", str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.count("ok") == 2


def test_reference_arm_prints_one_json_line():
    import json
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["value"] > 0 and d["unit"] == "tokens*ch/s"


def test_gpus_flag_without_launcher_never_reports_one_gpu():
    """`bench.py --gpus 2` started without a launcher must start two ranks itself or refuse; on a box with fewer GPUs it
    refuses with a non-zero exit code and prints no result line."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=300, env={k: v for k, v in os.environ.items() if k != "WORLD_SIZE"})
    import torch
    if torch.cuda.device_count() < 2:
        assert r.returncode != 0 and "n_gpus" not in r.stdout
    else:
        assert r.returncode == 0 and '"n_gpus": 2' in r.stdout
