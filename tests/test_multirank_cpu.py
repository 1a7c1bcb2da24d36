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


# ---------------------------------------------------------------- column sharding (one product over several GPUs)
SHARD_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch
import torch.distributed as dist
from paper_2108_12704_b200 import sharded
import synth_inputs as si
rank = int(sys.argv[1])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=2)
wl = si.scaled(si.CFG3_FC_SHAC, 300, 37)                      # 37 columns: shards of 18 and 19
W = si.weights(wl)
quant = dict(sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters, seed=wl.seed)
Wq = sharded.quantized_matrix("shac", W, **quant)
sh = sharded.ColumnSharded("shac", W, rank, 2, **quant)
lo, hi = sh.bounds[rank]
assert sh.bounds == [(0, 18), (18, 37)]
# the shard stands for exactly its columns of the quantized matrix
assert np.array_equal(sh.format.decode_host().view(np.uint32), np.ascontiguousarray(Wq[:, lo:hi]).view(np.uint32))
# the exchange: a stand-in for the device product (no GPU here) on this rank's columns, gathered on both ranks
X = si.inputs(wl, 3)
for x in (X[0], X.T):
    y_local = torch.from_numpy(np.ascontiguousarray((x.T.astype(np.float64) @ Wq[:, lo:hi].astype(np.float64)).T))
    y = sharded.gather_columns(y_local, sh.bounds, rank).numpy()
    assert np.array_equal(y, (x.T.astype(np.float64) @ Wq.astype(np.float64)).T), rank
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_column_sharding_two_gloo_ranks(tmp_path):
    port = 31500 + os.getpid() % 2000
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True) for r in range(2)]
    for r, p in enumerate(procs):
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err
        assert f"ok {r}" in out


def test_column_bounds():
    from paper_2108_12704_b200.sharded import column_bounds
    for m, g in ((4096, 8), (10, 4), (37, 2), (5, 5)):
        b = column_bounds(m, g)
        assert b[0][0] == 0 and b[-1][1] == m and all(b[i][1] == b[i + 1][0] for i in range(g - 1))
        sizes = [hi - lo for lo, hi in b]
        assert max(sizes) - min(sizes) <= 1
