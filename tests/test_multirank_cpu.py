"""The multi-rank logic of bench.py on CPU: two gloo ranks, whole-job time = max over ranks,
whole-job units = sum over ranks (replicas only, no data-path collective), and the reference arm
running on rank 0 alone."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
t, u = bench.reduce_job(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
assert t == 15.0 and u == 300.0, (t, u)
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_reduce_job_two_gloo_ranks(tmp_path):
    port = 29500 + os.getpid() % 2000
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True) for r in range(2)]
    for r, p in enumerate(procs):
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        assert f"ok {r}" in out


def test_reduce_job_single_process():
    import bench
    assert bench.reduce_job(3.5, 7.0, None) == (3.5, 7.0)


def test_reference_arm_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_algorithmic_bytes_formula():
    import bench
    sizes = dict(stream_bytes=1000, offset_index_bytes=100, ri_bytes=50, cb_bytes=20, k_eff=8, n=10, m=5)
    assert bench.algorithmic_bytes_gemv(sizes, 3) == 1000 + 100 + (16 + 32 + 544) + 50 + 20 + 40 + 20
