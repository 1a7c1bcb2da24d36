"""Per-configuration report: format sizes against the paper's bounds (Corollaries 1 and 2) and
kernel times against the HBM roofline on the compressed bytes, for the benchmark configurations
and the sparsity x k sweep.  One JSON line per (configuration, format, batch).

    python -m paper_2108_12704_b200.report [--configs 1,2,3,4] [--sweep] [--paper-shapes] [--chain] [--compare] [--out FILE]

Timing protocol as in bench.py: device images replicated to more than three times the L2 size and
rotated per launch, launches captured in CUDA graphs, CUDA events on the launching stream, best of
five replays.  Results are checked in-process against the format's own host decode (fp64 product).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

L2_BYTES = 126 * 1024 * 1024


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _capture(torch, fn):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            fn()
    torch.cuda.current_stream().wait_stream(s)
    return g


def algorithmic_bytes(sizes: dict) -> int:
    """Bytes a single-input product has to move (stream, offset index, tables, ri, cb, x, y)."""
    lut_bits = min(12, sizes["max_code_len"])
    tables = (2 << lut_bits) + 4 * sizes["k_eff"] + 34 * 16
    return (sizes["stream_bytes"] + sizes["offset_index_bytes"] + tables + sizes["ri_bytes"] + sizes["cb_bytes"]
            + 4 * sizes["n"] + 4 * sizes["m"])


def measure(wl, kind, batches, W=None, seg_symbols=0, max_check_batch=128, replays=5):
    import torch
    import paper_2108_12704_b200 as hb
    W = si.weights(wl) if W is None else W
    fmt = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                    seed=wl.seed, seg_symbols=seg_symbols).upload()
    sizes = fmt.sizes()
    peak, peak_kind = _peaks()
    nbytes = fmt.device_bytes()
    R = min(64, max(2, math.ceil(3 * L2_BYTES / nbytes)))
    reps = []
    for _ in range(R):
        buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        off = (-buf.data_ptr()) % 256
        view = buf[off:off + nbytes]
        view.copy_(fmt.image())
        reps.append(view)
    Wq = fmt.decode_host().astype(np.float64)
    dense_bytes = 4 * wl.n * wl.m
    common = dict(config=wl.config, workload=wl.name, format=kind, n=wl.n, m=wl.m, sparsity=wl.sparsity, k=wl.k,
                  k_eff=sizes["k_eff"], nnz=sizes["nnz"], seg_symbols=sizes["seg_symbols"],
                  avg_code_len=round(sizes["avg_code_len"], 4), entropy=round(sizes["entropy"], 4),
                  max_code_len=sizes["max_code_len"], stream_bytes=sizes["stream_bytes"],
                  offset_index_bytes=sizes["offset_index_bytes"], ri_bytes=sizes["ri_bytes"],
                  total_bytes=sizes["total_bytes"], psi=round(sizes["total_bytes"] / dense_bytes, 5),
                  paper_bits=sizes["paper_bits"], bound_bits=sizes["bound_bits"],
                  bound_over_size=round(sizes["bound_bits"] / max(1, sizes["paper_bits"]), 3))
    rows = []
    for B in batches:
        Xh = si.inputs(wl, B)
        nx = R if B == 1 else min(R, max(1, (1 << 28) // max(1, 4 * wl.n * B)))
        if B == 1:
            xs = [torch.from_numpy(Xh[0]).cuda() for _ in range(nx)]
            ys = [torch.empty(wl.m, device="cuda") for _ in range(nx)]
        else:
            xt = torch.from_numpy(np.ascontiguousarray(Xh.T)).cuda()
            xs = [xt.clone() for _ in range(nx)]
            ys = [torch.empty((wl.m, B), device="cuda") for _ in range(nx)]
        ws = torch.empty(max(16, fmt.workspace_bytes(B)), dtype=torch.uint8, device="cuda")

        def step(r):
            fmt.attach(reps[r])
            fmt.dot(xs[r % nx], ys[r % nx], ws)

        step(0)
        torch.cuda.synchronize()
        ok = None
        if B <= max_check_batch:
            got = ys[0].cpu().numpy().astype(np.float64)
            got = got[None] if B == 1 else got.T
            ref = Xh.astype(np.float64) @ Wq
            tol = 1e-5 * (np.abs(Xh.astype(np.float64)) @ np.abs(Wq)) + 1e-7
            ok = bool(np.all(np.abs(got - ref) <= tol))
        for i in range(3):
            step(i % R)
        g = _capture(torch, lambda: [step(r) for r in range(R)])
        g.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / R * 1e3)
        # the same product with the format resident in L2: every launch of the graph on replica 0
        gw = _capture(torch, lambda: [step(0) for _ in range(R)])
        gw.replay()
        torch.cuda.synchronize()
        warm = float("inf")
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            gw.replay()
            e1.record()
            torch.cuda.synchronize()
            warm = min(warm, e0.elapsed_time(e1) / R * 1e3)
        row = dict(common, batch=B, us=round(best, 2), us_l2_warm=round(warm, 2), within_tolerance=ok,
                   launches=fmt.last_launch_count(),
                   gweights_per_s=round(wl.n * wl.m * B / best / 1e3, 1),
                   symbols_per_s=round(sizes["symbols"] / best * 1e6, 0))
        if B > 1:                              # flops on the stored non-null weights only
            row.update(effective_gflops=round(2.0 * sizes["nnz"] * B / best / 1e3, 1))
        if B == 1:
            ab = algorithmic_bytes(sizes)
            row.update(algorithmic_bytes=ab, gb_per_s=round(ab / best / 1e3, 1),
                       frac_of_hbm=round(ab / best / 1e3 / peak, 4), hbm_peak=f"{peak} GB/s ({peak_kind})",
                       frac_of_8tb=round(ab / best / 1e3 / 8000.0, 4))
        rows.append(row)
        del xs, ys
    return rows


def measure_chain(batches=(1, 64), replays=200):
    """The fully connected stack of the paper's VGG19 (512 -> 4096 -> 4096 -> 10, Sect. V) evaluated on the
    compressed formats with bias and ReLU applied in the product kernels: time of the three layers submitted as
    one chain (hac_chain in one CUDA graph) against the three layers each submitted and waited for on its own."""
    import torch
    import paper_2108_12704_b200 as hb
    specs = [(dataclasses.replace(si.CFG3_FC_SHAC, n=512, m=4096, sparsity=0.9, k=32, item=11), "shac", True),
             (dataclasses.replace(si.CFG2_DENSE_HAC, n=4096, m=4096, k=64, item=12), "hac", True),
             (dataclasses.replace(si.CFG2_DENSE_HAC, n=4096, m=10, k=32, quantizer=si.QUANT_KMEANS, item=13), "hac", False)]
    layers = []
    rng = np.random.default_rng(99)
    for wl, kind, relu in specs:
        fmt = hb.Format(kind, si.weights(wl), sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer,
                        kmeans_iters=wl.kmeans_iters, seed=wl.seed).upload()
        bias = torch.from_numpy((rng.standard_normal(wl.m) * 0.1).astype(np.float32)).cuda()
        layers.append((fmt, bias, relu))
    rows = []
    for B in batches:
        X = np.maximum(np.random.default_rng(B).standard_normal((B, 512)), 0).astype(np.float32)
        x = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
        ws = torch.empty(max(16, max(f.workspace_bytes(B) for f, _, _ in layers)), dtype=torch.uint8, device="cuda")
        shape = lambda mm: (mm,) if B == 1 else (mm, B)
        acts = [torch.empty(shape(f.m), device="cuda") for f, _, _ in layers]
        ins = [x] + acts[:-1]
        y_chain, launches = hb.hac_chain(layers, x, workspace=ws)
        for (f, b, r), i, o in zip(layers, ins, acts):
            f.dot(i, o, ws, bias=b, relu=r)
        torch.cuda.synchronize()
        same = bool(torch.equal(acts[-1], y_chain))
        g_chain = _capture(torch, lambda: hb.hac_chain(layers, x, y_chain, ws))
        g_layer = [_capture(torch, (lambda f=f, b=b, r=r, i=i, o=o: f.dot(i, o, ws, bias=b, relu=r)))
                   for (f, b, r), i, o in zip(layers, ins, acts)]

        def timed(graphs, wait_each):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(replays):
                for g in graphs:
                    g.replay()
                    if wait_each:
                        torch.cuda.synchronize()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / replays * 1e3

        timed([g_chain], False)
        t_chain = min(timed([g_chain], False) for _ in range(3))
        t_alone = [min(timed([g], True) for _ in range(3)) for g in g_layer]
        rows.append(dict(report="layer_chain", stack="512-4096-4096-10 (sHAC 90 % pruned k=32, HAC k=64, HAC k=32), bias + ReLU",
                         batch=B, launches_per_chain=launches, chain_us=round(t_chain, 2),
                         per_layer_in_chain_us=round(t_chain / len(layers), 2),
                         layers_alone_us=[round(t, 2) for t in t_alone], sum_alone_us=round(sum(t_alone), 2),
                         chain_equals_layers=same,
                         note="chain: one graph of the chained submission replayed back to back; alone: each layer's graph "
                              "replayed and waited for by the host before the next (launch and wait latency included); "
                              "the format stays in L2 here (no replica rotation)"))
    return rows


def measure_compare(wl, replays=5):
    """One-input product of the same quantized matrix in the formats the paper compares (Sect. V): dense fp32
    (the library's matrix-vector product, for context), index map, CSC, and HAC / sHAC; psi as the paper counts it."""
    import torch
    import paper_2108_12704_b200 as hb
    from paper_2108_12704_b200.binding import Csc, IndexMap
    W = si.weights(wl)
    peak, peak_kind = _peaks()
    ours = {kind: hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                            seed=wl.seed) for kind in ("hac", "shac")}
    Wq = ours["hac"].decode_host()
    Xh = si.inputs(wl, 1)
    ref = Xh.astype(np.float64) @ Wq.astype(np.float64)
    tol = 1e-5 * (np.abs(Xh.astype(np.float64)) @ np.abs(Wq.astype(np.float64))) + 1e-7
    x = torch.from_numpy(Xh[0]).cuda()
    rows = []

    def timed(name, psi, nbytes, make_step, R):
        steps = [make_step(r) for r in range(R)]
        y = steps[0]()
        torch.cuda.synchronize()
        ok = bool(np.all(np.abs(y.cpu().numpy().astype(np.float64)[None] - ref) <= (tol if name != "dense_fp32" else 10 * tol)))
        for st in steps[:3]:
            st()
        g = _capture(torch, lambda: [st() for st in steps])
        g.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g.replay(); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / R * 1e3)
        rows.append(dict(report="format_comparison", workload=wl.name, n=wl.n, m=wl.m, sparsity=wl.sparsity, k=wl.k,
                         format=name, psi=round(psi, 5), bytes=int(nbytes), us=round(best, 2), within_tolerance=ok,
                         gb_per_s=round(nbytes / best / 1e3, 1), frac_of_hbm=round(nbytes / best / 1e3 / peak, 4),
                         hbm_peak=f"{peak} GB/s ({peak_kind})"))

    def replicas(nbytes):
        return min(64, max(2, math.ceil(3 * L2_BYTES / max(1, nbytes))))

    # dense fp32, [m, n] row-major so that the library reads every column of W contiguously
    dense_bytes = 4 * wl.n * wl.m
    R = replicas(dense_bytes)
    Wd = [torch.from_numpy(np.ascontiguousarray(Wq.T)).cuda() for _ in range(R)]
    yd = torch.empty(wl.m, device="cuda")
    timed("dense_fp32", 1.0, dense_bytes, lambda r: (lambda: torch.mv(Wd[r], x, out=yd)), R)
    del Wd
    im = IndexMap(Wq, 8 if len(np.unique(Wq)) <= 256 else 16)
    nbytes = im.index.nbytes + 4 * im.k
    R = replicas(nbytes)
    ims = [IndexMap.__new__(IndexMap) for _ in range(R)]
    for o in ims:
        o.__dict__.update(im.__dict__)
        o.upload()
    yi = torch.empty(wl.m, device="cuda")
    timed(f"index_map{im.index_bits}", im.psi(), nbytes, lambda r: (lambda: ims[r].dot(x, yi)), R)
    del ims
    c = Csc(Wq)
    nbytes = 8 * c.q + 4 * (wl.m + 1)
    R = replicas(nbytes)
    cs = [Csc.__new__(Csc) for _ in range(R)]
    for o in cs:
        o.__dict__.update(c.__dict__)
        o.upload()
    yc = torch.empty(wl.m, device="cuda")
    timed("csc", c.psi(), nbytes, lambda r: (lambda: cs[r].dot(x, yc)), R)
    del cs
    for kind, fmt in ours.items():
        fmt.upload()
        sizes = fmt.sizes()
        nbytes = fmt.device_bytes()
        R = replicas(nbytes)
        reps = []
        for _ in range(R):
            buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
            off = (-buf.data_ptr()) % 256
            view = buf[off:off + nbytes]
            view.copy_(fmt.image())
            reps.append(view)
        yo = torch.empty(wl.m, device="cuda")
        ws = torch.empty(max(16, fmt.workspace_bytes(1)), dtype=torch.uint8, device="cuda")

        def make(r, fmt=fmt, reps=reps, yo=yo, ws=ws):
            def step():
                fmt.attach(reps[r])
                return fmt.dot(x, yo, ws)
            return step
        timed(kind, sizes["paper_bits"] / (32.0 * wl.n * wl.m), algorithmic_bytes(sizes), make, R)
        del reps
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4")
    ap.add_argument("--sweep", action="store_true", help="configuration 5: sparsity x k grid, HAC and sHAC")
    ap.add_argument("--paper-shapes", action="store_true", help="the fully connected shapes of the paper's Sect. V-C")
    ap.add_argument("--chain", action="store_true", help="the fully connected stack as a chain of layers")
    ap.add_argument("--compare", action="store_true", help="dense, index map, CSC, HAC and sHAC on configurations 2 and 3")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    out = open(args.out, "w") if args.out else None

    def emit(rows):
        for r in rows:
            line = json.dumps(r)
            print(line, flush=True)
            if out:
                out.write(line + "\n")
                out.flush()

    wanted = {int(c) for c in args.configs.split(",") if c}
    table = {1: si.CFG1_TINY_SHAC, 2: si.CFG2_DENSE_HAC, 3: si.CFG3_FC_SHAC, 4: si.CFG4_CONV}
    for c in sorted(wanted):
        wl = table[c]
        W = si.weights(wl)
        for kind in wl.formats:
            emit(measure(wl, kind, wl.batches if c != 4 else (1,) + tuple(wl.batches), W=W))
    if args.sweep:
        cells = si.sweep_cells()
        W = si.weights(cells[0])
        for wl in cells:
            for kind in wl.formats:
                emit(measure(wl, kind, wl.batches, W=W))
    if args.chain:
        emit(measure_chain())
    if args.compare:
        for wl in (si.CFG2_DENSE_HAC, si.CFG3_FC_SHAC):
            emit(measure_compare(wl))
    if args.paper_shapes:
        for wl in si.paper_shaped_cells():
            for kind in wl.formats:
                emit(measure(wl, kind, (1, 8)))


if __name__ == "__main__":
    main()
