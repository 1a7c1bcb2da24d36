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
MIN_TIMED_SECONDS = 0.5     # the K-step region is repeated until this much device time has been measured
MAX_REPEATS = 4000


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the single-input kernels from ncu captures (profiles/), valid
# only for the device code they were taken on (hash of the device part of hac_kernels.cu).
NCU_TRAFFIC = {"kernel_source_sha256": "bb43a934e583e3f20d5b87507b66635643ec829888d74bdbd318e48ee54aafb2",
               "hac_gemv": 14642688, "shac_gemv": 11704320}


def device_code(text: bytes) -> bytes:
    """The part of hac_kernels.cu that holds device code (everything before the host section)."""
    cut = text.find(b"// Host side")
    return text if cut < 0 else text[:cut]


def ncu_traffic(which):
    import hashlib
    src = os.path.join(ROOT, "paper_2108_12704_b200", "csrc", "hac_kernels.cu")
    try:
        with open(src, "rb") as f:
            same = hashlib.sha256(device_code(f.read())).hexdigest() == NCU_TRAFFIC["kernel_source_sha256"]
    except OSError:
        same = False
    return NCU_TRAFFIC[which] if same else None


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


def median(v):
    return float(np.median(np.asarray(v, dtype=np.float64)))


class Leg:
    """One product (a format at a batch size) timed as CUDA graphs of K launches that rotate over the replicas of
    the device image, so that every launch reads cold HBM."""

    def __init__(self, torch, fmt, reps, xs, ys, ws, layout, K):
        self.torch, self.fmt, self.reps, self.xs, self.ys, self.ws, self.layout = torch, fmt, reps, xs, ys, ws, layout
        self.R, self.K = len(reps), K
        self.launches_per_product = self.launch(0)
        for i in range(3):
            self.launch(i % self.R)
        torch.cuda.synchronize()
        full, rem = divmod(K, self.R)
        self.full = full
        self.g_full = capture(torch, lambda: [self.launch(r) for r in range(self.R)]) if full else None
        self.g_rem = capture(torch, lambda: [self.launch(r) for r in range(rem)]) if rem else None
        for g in (self.g_full, self.g_rem):
            if g is not None:
                g.replay()
        torch.cuda.synchronize()

    def launch(self, r):
        self.fmt.attach(self.reps[r])
        if self.layout is None:
            self.fmt.dot(self.xs[r % len(self.xs)], self.ys[r % len(self.ys)], self.ws)
        else:
            self.fmt.dot(self.xs[r % len(self.xs)], self.ys[r % len(self.ys)], self.ws, layout=self.layout)
        return self.fmt.last_launch_count()

    def replay(self):
        """Enqueues exactly K launches."""
        for _ in range(self.full):
            self.g_full.replay()
        if self.g_rem is not None:
            self.g_rem.replay()


def time_regions(torch, legs, min_seconds, max_repeats, dist=None):
    """Repeats the timed region (every leg's K launches, one leg after the other, CUDA events between the
    legs on the launching stream, a synchronize on both sides) until `min_seconds` of device time have been
    measured.  Returns per-leg lists of milliseconds per region and the list of whole-region milliseconds."""
    per_leg = [[] for _ in legs]
    whole = []
    total = 0.0
    while len(whole) < max_repeats and (total < min_seconds * 1e3 or len(whole) < 3):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(legs) + 1)]
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        ev[0].record()
        for i, leg in enumerate(legs):
            leg.replay()
            ev[i + 1].record()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        for i in range(len(legs)):
            per_leg[i].append(ev[i].elapsed_time(ev[i + 1]))
        whole.append(ev[0].elapsed_time(ev[-1]))
        total += whole[-1]
    return per_leg, whole


def build_format(hb, kind, wl, dev, seg_symbols=0):
    W = si.weights(wl)
    fmt = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                    seed=wl.seed, seg_symbols=seg_symbols).upload(dev)
    del W
    return fmt


def check_against_host_decode(fmt, X, Y, what):
    """Guard before timing (not the parity test, which compares with the oracle under tests/): the product must
    agree with a float64 product on the format's own host decode."""
    Wq = fmt.decode_host().astype(np.float64)
    X64 = X.astype(np.float64)
    ref = X64 @ Wq
    tol = 1e-5 * (np.abs(X64) @ np.abs(Wq)) + 1e-7
    if not np.all(np.abs(Y.astype(np.float64) - ref) <= tol):
        raise RuntimeError(f"{what}: result outside tolerance; refusing to time it")


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
    K, Wm = args.steps, max(args.warmup, 3)

    # ---- workload of the metric: dense HAC, one input and a batch of 64 ---------------------------------------
    wl = si.CFG2_DENSE_HAC
    fmt = build_format(hb, "hac", wl, dev, int(os.environ.get("HAC_BENCH_SEG_SYMBOLS", "0")))
    sizes = fmt.sizes()
    n, m = wl.n, wl.m
    lut_bits = min(12, sizes["max_code_len"])
    image_bytes = fmt.device_bytes()
    R = max(2, math.ceil(3 * L2_BYTES / image_bytes))
    reps = make_replicas(fmt, torch, R)
    x1_host = [si.inputs(wl, 1, salt=r)[0] for r in range(R)]
    x1 = [torch.from_numpy(v).to(dev) for v in x1_host]
    xb_host = si.inputs(wl, GEMM_BATCH)
    xB = [torch.from_numpy(np.ascontiguousarray(xb_host.T)).to(dev) for _ in range(R)]
    y1 = [torch.empty(m, dtype=torch.float32, device=dev) for _ in range(R)]
    yB = [torch.empty((m, GEMM_BATCH), dtype=torch.float32, device=dev) for _ in range(R)]
    ws = torch.empty(max(fmt.workspace_bytes(1), fmt.workspace_bytes(GEMM_BATCH), 16), dtype=torch.uint8, device=dev)
    leg_gemv = Leg(torch, fmt, reps, x1, y1, ws, None, K)
    leg_gemm = Leg(torch, fmt, reps, xB, yB, ws, "nb", K)
    check_against_host_decode(fmt, x1_host[0][None], y1[0].cpu().numpy()[None], "HAC GEMV")
    check_against_host_decode(fmt, xb_host, yB[0].cpu().numpy().T, "HAC GEMM")
    for i in range(Wm):                          # warm-up steps
        leg_gemv.launch(i % R)
        leg_gemm.launch(i % R)
    torch.cuda.synchronize()

    with ClockSampler(local_rank) as clocks:
        (t_gemv, t_gemm), t_whole = time_regions(torch, [leg_gemv, leg_gemm], MIN_TIMED_SECONDS, MAX_REPEATS, dist)
    repeats = len(t_whole)
    step_ms = median(t_whole) / K
    weights_per_step = float(n) * m * (1 + GEMM_BATCH)
    job_ms, job_units = reduce_job(step_ms, weights_per_step, dist)
    value = job_units / (job_ms * 1e-3) / 1e9
    gemv_s = median(t_gemv) * 1e-3 / K
    gemm_s = median(t_gemm) * 1e-3 / K

    # ---- end to end through the host entry point: pinned host X / Y, copies inside the timed region ----------
    # Two streams, each with its own pinned buffers and device staging area, take the steps in turn through the
    # asynchronous host entry point, so that the copies of one step overlap the kernels of the other.
    lanes = []
    for _ in range(2):
        lanes.append(dict(
            stream=torch.cuda.Stream(device=dev),
            xh1=torch.from_numpy(si.inputs(wl, 1)).pin_memory(), yh1=torch.empty((1, m), dtype=torch.float32).pin_memory(),
            xhB=torch.from_numpy(xb_host).pin_memory(), yhB=torch.empty((GEMM_BATCH, m), dtype=torch.float32).pin_memory(),
            scratch=torch.empty(max(fmt.dot_host_scratch_bytes(1), fmt.dot_host_scratch_bytes(GEMM_BATCH)),
                                dtype=torch.uint8, device=dev)))

    def e2e_step(i):
        ln = lanes[i % 2]
        with torch.cuda.stream(ln["stream"]):
            fmt.attach(reps[i % R])
            fmt.dot_host(ln["xh1"], ln["yh1"], ln["scratch"], wait=False)
            fmt.dot_host(ln["xhB"], ln["yhB"], ln["scratch"], wait=False)

    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    check_against_host_decode(fmt, xb_host, lanes[0]["yhB"].numpy(), "HAC GEMM through the host entry point")
    if dist is not None:
        dist.barrier()
    Ke = 0
    t0 = time.perf_counter()
    while Ke < K or time.perf_counter() - t0 < 0.3:
        e2e_step(Ke)
        Ke += 1
        if Ke >= 20000:
            break
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_job_ms, e2e_units = reduce_job(e2e_ms, weights_per_step * Ke, dist)
    e2e_value = e2e_units / (e2e_job_ms * 1e-3) / 1e9
    hac_launches = leg_gemv.launches_per_product + leg_gemm.launches_per_product
    del leg_gemv, leg_gemm, reps, x1, xB, y1, yB, lanes
    torch.cuda.empty_cache()

    # ---- the sHAC workload (large pruned fully connected layer), timed the same way, reported beside ----------
    swl = si.CFG3_FC_SHAC
    sfmt = build_format(hb, "shac", swl, dev)
    ssizes = sfmt.sizes()
    sR = max(2, math.ceil(3 * L2_BYTES / sfmt.device_bytes()))
    sreps = make_replicas(sfmt, torch, sR)
    sx1_host = [si.inputs(swl, 1, salt=r)[0] for r in range(sR)]
    sx1 = [torch.from_numpy(v).to(dev) for v in sx1_host]
    sy1 = [torch.empty(swl.m, dtype=torch.float32, device=dev) for _ in range(sR)]
    sbatches = [b for b in swl.batches if b > 1]
    sX_host = {b: si.inputs(swl, b) for b in sbatches}
    sX = {b: [torch.from_numpy(np.ascontiguousarray(sX_host[b].T)).to(dev) for _ in range(min(sR, 8))] for b in sbatches}
    sY = {b: [torch.empty((swl.m, b), dtype=torch.float32, device=dev) for _ in range(min(sR, 8))] for b in sbatches}
    sws = torch.empty(max([sfmt.workspace_bytes(b) for b in [1] + sbatches] + [16]), dtype=torch.uint8, device=dev)
    Ks = max(1, min(K, 2000))
    sleg1 = Leg(torch, sfmt, sreps, sx1, sy1, sws, None, Ks)
    slegB = [Leg(torch, sfmt, sreps, sX[b], sY[b], sws, "nb", max(1, Ks // b)) for b in sbatches]
    check_against_host_decode(sfmt, sx1_host[0][None], sy1[0].cpu().numpy()[None], "sHAC GEMV")
    for b, leg in zip(sbatches, slegB):
        if b <= 16:
            check_against_host_decode(sfmt, sX_host[b], sY[b][0].cpu().numpy().T, f"sHAC GEMM B={b}")
    st_legs, st_whole = time_regions(torch, [sleg1] + slegB, MIN_TIMED_SECONDS, MAX_REPEATS, dist)
    shac_gemv_s = median(st_legs[0]) * 1e-3 / Ks
    shac_gemm_s = {b: median(t) * 1e-3 / leg.K for b, leg, t in zip(sbatches, slegB, st_legs[1:])}
    shac_launches = sleg1.launches_per_product * Ks + sum(leg.launches_per_product * leg.K for leg in slegB)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    alg_bytes = algorithmic_bytes_gemv(sizes, lut_bits)
    achieved = alg_bytes / gemv_s / 1e9
    roofline = {"kernel": "single-input HAC product (GEMV, batch 1)", "bound": "hbm", "achieved": achieved,
                "peak": peaks["hbm_gbs"], "peak_source": f"of {peak_kind}", "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "frac_of_nominal_8TBs": achieved / 8000.0,
                "traffic": ncu_traffic("hac_gemv"), "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_us": gemv_s * 1e6,
                "symbols_per_s": sizes["symbols"] / gemv_s,
                "note": "the metric's HBM figure is defined on the single-input product, so this object rates that kernel; "
                        "the batch-64 product, which takes the larger share of a step, is rated in roofline_gemm"}
    gemm_flops = 2.0 * n * m * GEMM_BATCH
    tf32_peak = peaks.get("bf16_tflops", 1590.0) * 0.5        # measured bf16 x nominal tf32/bf16 ratio
    roofline_gemm = {"kernel": "batched HAC product (GEMM, batch 64, tcgen05 TF32 x3 split)", "bound": "tensor",
                     "achieved": gemm_flops / gemm_s / 1e12, "peak": tf32_peak, "unit": "TFLOP/s",
                     "peak_source": f"measured bf16 GEMM ({peak_kind}) x 0.5 (nominal tf32 : bf16)",
                     "frac": gemm_flops / gemm_s / 1e12 / tf32_peak, "avg_launch_us": gemm_s * 1e6,
                     "note": "algorithmic flops 2*n*m*B; the kernel is bound by the Huffman decode, not by the MMAs"}
    s_alg = algorithmic_bytes_gemv(ssizes, min(12, ssizes["max_code_len"]))
    s_ach = s_alg / shac_gemv_s / 1e9
    roofline_shac = {"kernel": "single-input sHAC product (GEMV, batch 1)", "workload": swl.name, "bound": "hbm",
                     "achieved": s_ach, "peak": peaks["hbm_gbs"], "peak_source": f"of {peak_kind}", "unit": "GB/s",
                     "frac": s_ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": s_ach / 8000.0,
                     "traffic": ncu_traffic("shac_gemv"), "algorithmic_bytes_per_launch": s_alg,
                     "avg_launch_us": shac_gemv_s * 1e6, "stored_entries_per_s": ssizes["nnz"] / shac_gemv_s}

    # the oracle as it stands on the host cores, bounded sample (about 10-30 s of CPU work)
    cores = os.cpu_count() or 1
    ofmt = oracle_format(wl)
    rows, cols = plan_oracle_sample(ofmt, wl, cores, 4.0)
    t_cpu, w_cpu = oracle_sample_rate(ofmt, wl, rows, cols, cores, repeats=3)
    cpu_baseline = {"value": w_cpu / t_cpu / 1e9, "unit": UNIT, "cores": min(cores, rows), "kind": "oracle",
                    "sample": f"Algorithm 3, {min(cores, rows)} threads, {rows} input rows x first {cols} of {m} "
                              f"columns of the same HAC stream, best of 3 ({t_cpu:.2f} s per run)"}

    def spread(ts, per):
        v = np.asarray(ts, dtype=np.float64) / per * 1e3
        return {"us": float(np.median(v)), "min_us": float(v.min()), "max_us": float(v.max())}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": job_ms, "ms_per_step_min": min(t_whole) / K, "ms_per_step_max": max(t_whole) / K,
        "repeats": repeats, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "n": n, "m": m, "k": wl.k, "k_eff": sizes["k_eff"],
                   "quantizer": "uniform over [min,max]", "step": f"one GEMV (batch 1) + one GEMM (batch {GEMM_BATCH})",
                   "batches": [1, GEMM_BATCH], "seg_symbols": sizes["seg_symbols"],
                   "format_bytes": sizes["total_bytes"], "stream_bytes": sizes["stream_bytes"],
                   "avg_code_len_bits": sizes["avg_code_len"],
                   "l2_defeat": f"{R} replicas of the {image_bytes}-byte device image rotated per launch (> 3 x L2)",
                   "timing": f"a timed region is K GEMV launches then K GEMM launches (CUDA graphs of one replica rotation "
                             f"each), CUDA events on the launching stream, synchronize on both sides; the region was "
                             f"repeated {repeats} times and ms_per_step is the median region / K"},
        "gemv": dict(spread(t_gemv, K), value=float(n) * m / gemv_s / 1e9, unit=UNIT),
        "gemm": dict(spread(t_gemm, K), value=float(n) * m * GEMM_BATCH / gemm_s / 1e9, unit=UNIT),
        "shac_gemv": dict(spread(st_legs[0], Ks), workload=swl.name, value=float(swl.n) * swl.m / shac_gemv_s / 1e9,
                          unit=UNIT, launches=Ks),
        "shac_gemm": {str(b): dict(spread(t, leg.K), value=float(swl.n) * swl.m * b / shac_gemm_s[b] / 1e9, unit=UNIT,
                                   launches=leg.K)
                      for b, leg, t in zip(sbatches, slegB, st_legs[1:])},
        "roofline": roofline, "roofline_gemm": roofline_gemm, "roofline_shac": roofline_shac,
        "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": Ke, "how": "hac_dot_host_async on two alternating streams, pinned host X and Y, one synchronize at the end",
                "h2d_bytes_per_step": 4 * n * (1 + GEMM_BATCH), "d2h_bytes_per_step": 4 * m * (1 + GEMM_BATCH)},
        "gpu_launches": repeats * K * hac_launches,
        "gpu_launches_shac": len(st_whole) * shac_launches,
        "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
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
