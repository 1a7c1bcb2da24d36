#!/usr/bin/env python
"""Benchmark of the HAC compressed-domain product on one B200 (per rank).

One step = one pass of the whole hot path over the dense-HAC workload (4096 x 4096, uniform
quantization to k = 256 levels, Huffman-coded column segments): the matrix-vector product for
one input (GEMV) followed by the matrix-matrix product for a batch of 64 inputs (GEMM), both
computed directly on the compressed stream.  Throughput is in dense-equivalent weights per
second (n*m*B per product), and the GEMV kernel is also rated against the HBM roofline on the
compressed bytes it has to read.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (torchrun, one rank per GPU) every rank runs the same workload on its own replica of
the format; there is no data-path collective (weak scaling, replicas only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "compressed-format GEMV/GEMM Gweights/s and HBM GB/s vs ~8 TB/s peak"
UNIT = "Gweights/s"
L2_BYTES = 126 * 1024 * 1024
GEMM_BATCH = 64
FALLBACK_HBM_GBS = 6650.0


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the GEMV kernel from one ncu capture
# (profiles/hac_vec_kernel_config2_gemv.md), valid only for the device code it was taken on.
NCU_GEMV_TRAFFIC = {"bytes": 14614272, "kernel_source_sha256": "ee838ebffb4d5b73d2c37ed2f9a5797a446af2612ad2873648db3d6d7a6ef1cc"}


def device_code(text: bytes) -> bytes:
    """The part of hac_kernels.cu that holds device code (everything before the host section)."""
    cut = text.find(b"// Host side")
    return text if cut < 0 else text[:cut]


def gemv_traffic():
    import hashlib
    src = os.path.join(ROOT, "paper_2108_12704_b200", "csrc", "hac_kernels.cu")
    try:
        with open(src, "rb") as f:
            same = hashlib.sha256(device_code(f.read())).hexdigest() == NCU_GEMV_TRAFFIC["kernel_source_sha256"]
    except OSError:
        same = False
    return NCU_GEMV_TRAFFIC["bytes"] if same else None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


# --------------------------------------------------------------------------------------------
# clocks during the timed region (NVML, read only)
# --------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        self.handle = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.handle is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons - {"gpu_idle"}), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
# helpers shared with the CPU tests of the multi-rank logic
# --------------------------------------------------------------------------------------------
def reduce_job(elapsed_ms: float, units: float, dist=None):
    """Whole-job figures from per-rank ones: time = max over ranks, units = sum over ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def algorithmic_bytes_gemv(sizes: dict, lut_bits: int) -> int:
    """Bytes one single-input product has to move: the stream, the offset index, the decoding
    tables (primary table, values, per-length tables), the row indices and column bounds of sHAC,
    the input vector and the output vector."""
    tables = (2 << lut_bits) + 4 * sizes["k_eff"] + 34 * 16
    return (sizes["stream_bytes"] + sizes["offset_index_bytes"] + tables + sizes["ri_bytes"] + sizes["cb_bytes"]
            + 4 * sizes["n"] + 4 * sizes["m"])


# --------------------------------------------------------------------------------------------
# reference arm: the CPU oracle (Algorithms 1 and 3 as they stand) on the host cores
# --------------------------------------------------------------------------------------------
def oracle_format(wl):
    from oracle import hac_oracle as orc
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    return orc.hac_encode(Wq)


def oracle_sample_rate(fmt, wl, rows: int, cols: int, threads: int, repeats: int = 1, X=None):
    """Time Algorithm 3 (threads over input rows, Algorithm 1 per row) on `rows` inputs and the first
    `cols` columns of W.  Returns (seconds per call, weights per call)."""
    from oracle import hac_oracle as orc
    part = dict(fmt)
    part["m"] = cols
    if X is None:
        X = si.inputs(wl, rows, salt=1)
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.pardot(part, X, threads)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best, float(wl.n) * cols * rows


def plan_oracle_sample(fmt, wl, cores: int, seconds_per_step: float):
    """Rows and columns of a per-step sample that should take about `seconds_per_step`."""
    t, w = oracle_sample_rate(fmt, wl, cores, max(1, wl.m // 64), cores)
    rate = w / t                                           # weights per second, all cores
    budget = rate * seconds_per_step
    full = float(wl.n) * wl.m
    if budget >= cores * full:
        return int(min(1 + GEMM_BATCH, budget // full)), wl.m
    return cores, int(max(1, min(wl.m, budget // (cores * wl.n))))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = si.CFG2_DENSE_HAC
    cores = os.cpu_count() or 1
    fmt = oracle_format(wl)
    total_budget = 150.0
    per_step = max(0.002, min(10.0, total_budget / (args.steps + args.warmup)))
    rows, cols = plan_oracle_sample(fmt, wl, cores, per_step)
    X = si.inputs(wl, rows, salt=1)
    for _ in range(args.warmup):
        oracle_sample_rate(fmt, wl, rows, cols, cores, X=X)
    t0 = time.perf_counter()
    weights = 0.0
    for _ in range(args.steps):
        _, w = oracle_sample_rate(fmt, wl, rows, cols, cores, X=X)
        weights += w
    elapsed = time.perf_counter() - t0
    value = weights / elapsed / 1e9
    sample = (f"each step: Algorithm 3 with {min(cores, rows)} threads over {rows} input rows x the first {cols} of "
              f"{wl.m} columns of the {wl.n}x{wl.m} HAC stream")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "n": wl.n, "m": wl.m, "k": wl.k, "batches": [1, GEMM_BATCH]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, rows), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def make_replicas(fmt, torch, count):
    """`count` byte-identical copies of the uploaded device image, 256-byte aligned."""
    image = fmt.image()
    nbytes = image.numel()
    reps = []
    for _ in range(count):
        buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=image.device)
        off = (-buf.data_ptr()) % 256
        view = buf[off:off + nbytes]
        view.copy_(image)
        reps.append(view)
    return reps


def capture(torch, fn):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            fn()
    torch.cuda.current_stream().wait_stream(s)
    return g


def run_ours(args):
    import torch
    import paper_2108_12704_b200 as hb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)

    wl = si.CFG2_DENSE_HAC
    S = int(os.environ.get("HAC_BENCH_SEG_SYMBOLS", "0"))
    W = si.weights(wl)
    fmt = hb.Format("hac", W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                    seed=wl.seed, seg_symbols=S).upload(dev)
    sizes = fmt.sizes()
    n, m = wl.n, wl.m
    lut_bits = min(12, sizes["max_code_len"])
    image_bytes = fmt.device_bytes()
    R = max(2, math.ceil(3 * L2_BYTES / image_bytes))
    reps = make_replicas(fmt, torch, R)

    # inputs resident in HBM: one x and one X per replica slot, [n] and [n, B]
    x1 = [torch.from_numpy(si.inputs(wl, 1, salt=r)[0]).to(dev) for r in range(R)]
    xb_host = si.inputs(wl, GEMM_BATCH)
    xB = [torch.from_numpy(np.ascontiguousarray(xb_host.T)).to(dev) for _ in range(R)]
    y1 = [torch.empty(m, dtype=torch.float32, device=dev) for _ in range(R)]
    yB = [torch.empty((m, GEMM_BATCH), dtype=torch.float32, device=dev) for _ in range(R)]
    ws_bytes = max(fmt.workspace_bytes(1), fmt.workspace_bytes(GEMM_BATCH), 16)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)

    launches = {"gemv": 0, "gemm": 0}

    def gemv(r):
        fmt.attach(reps[r])
        fmt.dot(x1[r], y1[r], ws)
        return fmt.last_launch_count()

    def gemm(r):
        fmt.attach(reps[r])
        fmt.dot(xB[r], yB[r], ws, layout="nb")
        return fmt.last_launch_count()

    # parity spot check in this process before timing (one output column set against numpy fp64)
    launches["gemv"] = gemv(0)
    launches["gemm"] = gemm(0)
    torch.cuda.synchronize()
    Wq = fmt.decode_host().astype(np.float64)
    ref1 = x1[0].cpu().numpy().astype(np.float64) @ Wq
    tol1 = 1e-5 * (np.abs(x1[0].cpu().numpy().astype(np.float64)) @ np.abs(Wq)) + 1e-7
    if not np.all(np.abs(y1[0].cpu().numpy() - ref1) <= tol1):
        raise RuntimeError("GEMV result outside tolerance; refusing to time it")
    refB = (xb_host.astype(np.float64) @ Wq).T
    tolB = 1e-5 * (np.abs(xb_host.astype(np.float64)) @ np.abs(Wq)).T + 1e-7
    if not np.all(np.abs(yB[0].cpu().numpy() - refB) <= tolB):
        raise RuntimeError("GEMM result outside tolerance; refusing to time it")
    del Wq

    K, Wm = args.steps, args.warmup
    chunk = R                                    # one graph = one rotation over the replicas

    def graph_of(fn, count, start=0):
        return capture(torch, lambda: [fn((start + i) % R) for i in range(count)])

    for i in range(max(Wm, 3)):                  # warm-up steps, direct launches
        gemv(i % R)
        gemm(i % R)
    torch.cuda.synchronize()
    full, rem = divmod(K, chunk)
    g_gemv = graph_of(gemv, chunk) if full else None
    g_gemm = graph_of(gemm, chunk) if full else None
    g_gemv_rem = graph_of(gemv, rem) if rem else None
    g_gemm_rem = graph_of(gemm, rem) if rem else None
    for g in (g_gemv, g_gemm, g_gemv_rem, g_gemm_rem):     # graph warm-up (upload of the executable graph)
        if g is not None:
            g.replay()
    torch.cuda.synchronize()

    e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local_rank) as clocks:
        e[0].record()
        for _ in range(full):
            g_gemv.replay()
        if g_gemv_rem is not None:
            g_gemv_rem.replay()
        e[1].record()
        for _ in range(full):
            g_gemm.replay()
        if g_gemm_rem is not None:
            g_gemm_rem.replay()
        e[2].record()
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t_gemv_ms = e[0].elapsed_time(e[1])
    t_gemm_ms = e[1].elapsed_time(e[2])
    t_total_ms = e[0].elapsed_time(e[2])

    weights_per_step = float(n) * m * (1 + GEMM_BATCH)
    job_ms, job_units = reduce_job(t_total_ms, weights_per_step * K, dist)
    value = job_units / (job_ms * 1e-3) / 1e9

    # end to end through the host entry point: pinned host X / Y, copies inside the timed region
    Ke = min(K, 2000)
    xh1 = torch.from_numpy(si.inputs(wl, 1)).pin_memory()
    yh1 = torch.empty((1, m), dtype=torch.float32).pin_memory()
    xhB = torch.from_numpy(xb_host).pin_memory()
    yhB = torch.empty((GEMM_BATCH, m), dtype=torch.float32).pin_memory()
    scratch = torch.empty(max(fmt.dot_host_scratch_bytes(1), fmt.dot_host_scratch_bytes(GEMM_BATCH)),
                          dtype=torch.uint8, device=dev)
    for i in range(3):
        fmt.attach(reps[i % R]); fmt.dot_host(xh1, yh1, scratch); fmt.dot_host(xhB, yhB, scratch)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        fmt.attach(reps[i % R])
        fmt.dot_host(xh1, yh1, scratch)
        fmt.dot_host(xhB, yhB, scratch)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_job_ms, e2e_units = reduce_job(e2e_ms, weights_per_step * Ke, dist)
    e2e_value = e2e_units / (e2e_job_ms * 1e-3) / 1e9

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    gemv_s = t_gemv_ms * 1e-3 / K
    gemm_s = t_gemm_ms * 1e-3 / K
    alg_bytes = algorithmic_bytes_gemv(sizes, lut_bits)
    achieved = alg_bytes / gemv_s / 1e9
    roofline = {"kernel": "hac_vec_kernel (GEMV, batch 1)", "bound": "hbm", "achieved": achieved,
                "peak": peaks["hbm_gbs"], "peak_source": f"of {peak_kind}", "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "frac_of_nominal_8TBs": achieved / 8000.0,
                "traffic": gemv_traffic(), "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_us": gemv_s * 1e6,
                "symbols_per_s": sizes["symbols"] / gemv_s,
                "note": "the metric's HBM figure is defined on the single-input product, so this object rates that kernel; "
                        "the batch-64 product, which takes the larger share of a step, is rated in roofline_gemm"}
    gemm_flops = 2.0 * n * m * GEMM_BATCH
    tf32_peak = peaks.get("bf16_tflops", 1590.0) * 0.5        # measured bf16 x nominal tf32/bf16 ratio
    roofline_gemm = {"kernel": "hac_gemm_tc_kernel (GEMM, batch 64, tcgen05 TF32 x3 split)", "bound": "tensor",
                     "achieved": gemm_flops / gemm_s / 1e12, "peak": tf32_peak, "unit": "TFLOP/s",
                     "peak_source": f"measured bf16 GEMM ({peak_kind}) x 0.5 (nominal tf32 : bf16)",
                     "frac": gemm_flops / gemm_s / 1e12 / tf32_peak, "avg_launch_us": gemm_s * 1e6,
                     "note": "algorithmic flops 2*n*m*B; the kernel is bound by the Huffman decode, not by the MMAs"}

    # the oracle as it stands on the host cores, bounded sample (about 10-30 s of CPU work)
    cores = os.cpu_count() or 1
    ofmt = oracle_format(wl)
    rows, cols = plan_oracle_sample(ofmt, wl, cores, 4.0)
    t_cpu, w_cpu = oracle_sample_rate(ofmt, wl, rows, cols, cores, repeats=3)
    cpu_baseline = {"value": w_cpu / t_cpu / 1e9, "unit": UNIT, "cores": min(cores, rows), "kind": "oracle",
                    "sample": f"Algorithm 3, {min(cores, rows)} threads, {rows} input rows x first {cols} of {m} "
                              f"columns of the same HAC stream, best of 3 ({t_cpu:.2f} s per run)"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(Wm, 3),
        "ms_per_step": job_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "n": n, "m": m, "k": wl.k, "k_eff": sizes["k_eff"],
                   "quantizer": "uniform over [min,max]", "step": f"one GEMV (batch 1) + one GEMM (batch {GEMM_BATCH})",
                   "batches": [1, GEMM_BATCH], "seg_symbols": sizes["seg_symbols"],
                   "format_bytes": sizes["total_bytes"], "stream_bytes": sizes["stream_bytes"],
                   "avg_code_len_bits": sizes["avg_code_len"],
                   "l2_defeat": f"{R} replicas of the {image_bytes}-byte device image rotated per launch (> 3 x L2)",
                   "timing": "CUDA graphs of one replica rotation each, K GEMV launches then K GEMM launches, "
                             "CUDA events on the launching stream"},
        "gemv": {"value": float(n) * m / gemv_s / 1e9, "unit": UNIT, "us": gemv_s * 1e6},
        "gemm": {"value": float(n) * m * GEMM_BATCH / gemm_s / 1e9, "unit": UNIT, "us": gemm_s * 1e6},
        "roofline": roofline, "roofline_gemm": roofline_gemm, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": Ke,
                "h2d_bytes_per_step": 4 * n * (1 + GEMM_BATCH), "d2h_bytes_per_step": 4 * m * (1 + GEMM_BATCH)},
        "gpu_launches": K * (launches["gemv"] + launches["gemm"]),
        "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
