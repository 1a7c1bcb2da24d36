"""Parity of the CUDA path with the oracle, through the C ABI, on the same seeded inputs:
decoded weights bit for bit, outputs within |y - y_ref| <= 1e-5 * sum_i |w_ij x_i| + 1e-7."""
import dataclasses

import numpy as np
import pytest

import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

RTOL_A, ATOL = 1e-5, 1e-7


def build_both(wl, kind, S=0, W=None, ri_bits=0):
    W = si.weights(wl) if W is None else W
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    lf = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                   seed=wl.seed, seg_symbols=S, ri_bits=ri_bits).upload()
    return lf, Wq, mask


def check_decode(lf, Wq, mask):
    got = lf.debug_decode().cpu().numpy()
    if lf.kind == "hac":
        assert np.array_equal(got.view(np.uint32), np.ascontiguousarray(Wq.T).view(np.uint32))
    else:
        nz = Wq.T[mask.T]
        assert np.array_equal(got.view(np.uint32), nz.view(np.uint32))


def check_outputs(y, y_ref, a):
    err = np.abs(y.astype(np.float64) - y_ref)
    bound = RTOL_A * a + ATOL
    worst = float((err / bound).max()) if err.size else 0.0
    assert np.all(err <= bound), f"worst error / bound = {worst}"
    return worst


def run_dot(lf, X, layout="nb"):
    """X: numpy [B, n].  Returns numpy [B, m]."""
    B = X.shape[0]
    if B == 1:
        y = lf.dot(torch.from_numpy(X[0]).cuda())
        torch.cuda.synchronize()
        return y.cpu().numpy()[None, :]
    if layout == "nb":
        y = lf.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda(), layout="nb")
        torch.cuda.synchronize()
        return y.cpu().numpy().T
    y = lf.dot(torch.from_numpy(X).cuda(), layout="bn")
    torch.cuda.synchronize()
    return y.cpu().numpy()


SMALL = [
    # workload, kind, S, batches
    (si.CFG1_TINY_SHAC, "shac", 0, (1, 5)),
    (si.CFG1_TINY_SHAC, "hac", 0, (1, 33)),
    (si.scaled(si.CFG2_DENSE_HAC, 2100, 70), "hac", 64, (1, 64)),        # 2 segments per column, ragged
    (si.scaled(si.CFG2_DENSE_HAC, 1000, 130), "hac", 0, (1, 3)),
    (si.scaled(si.CFG2_DENSE_HAC, 777, 45), "hac", 7, (1, 40)),          # odd S, 4 segments per column
    (si.scaled(si.CFG3_FC_SHAC, 6000, 200), "shac", 0, (1, 16, 128)),
    (si.scaled(si.CFG3_FC_SHAC, 6000, 90), "shac", 3, (1, 16)),          # several segments per column
    (si.scaled(si.CFG4_CONV, 1152, 128), "shac", 0, (1, 200)),
    (si.scaled(si.CFG4_CONV, 1152, 128), "hac", 0, (1, 200)),
    (dataclasses.replace(si.scaled(si.CFG4_CONV, 1152, 128), quantizer=si.QUANT_GRID, k=33), "shac", 0, (1, 12)),
    (dataclasses.replace(si.scaled(si.CFG2_DENSE_HAC, 900, 140), quantizer=si.QUANT_GRID, k=200), "hac", 0, (1, 70)),    (dataclasses.replace(si.scaled(si.CFG3_FC_SHAC, 5000, 150), quantizer=si.QUANT_PWS, k=32), "shac", 0, (1, 7)),
    (si.scaled(si.CFG2_DENSE_HAC, 3000, 40), "hac", 1024, (1, 3)),       # largest S: the batch runs input by input
    (si.scaled(si.CFG2_DENSE_HAC, 40000, 12), "hac", 512, (1, 2)),       # and with several segments per column
]


@pytest.mark.parametrize("wl,kind,S,batches", SMALL, ids=[f"{c[0].name}-{c[1]}-S{c[2]}" for c in SMALL])
def test_small_cases_element_by_element(wl, kind, S, batches):
    lf, Wq, mask = build_both(wl, kind, S)
    check_decode(lf, Wq, mask)
    for B in batches:
        X = si.inputs(wl, B)
        y_ref, a = orc.dot_definition(Wq, X)
        for layout in (("nb", "bn") if B > 1 else ("nb",)):
            check_outputs(run_dot(lf, X, layout), y_ref, a)
    # Algorithm 1 / 2 run literally give the same reference
    x = si.inputs(wl, 1)[0]
    ofmt = orc.hac_encode(Wq) if kind == "hac" else orc.shac_encode(Wq, mask)
    y_alg = (orc.dot_hac if kind == "hac" else orc.dot_shac)(ofmt, x)
    assert np.array_equal(y_alg, orc.dot_definition(Wq, x)[0][0])


def test_host_entry_point():
    wl = si.scaled(si.CFG3_FC_SHAC, 3000, 150)
    for kind in ("shac", "hac"):
        lf, Wq, mask = build_both(wl, kind)
        for B in (1, 20):
            X = si.inputs(wl, B)
            y_ref, a = orc.dot_definition(Wq, X)
            Xh = torch.from_numpy(X).pin_memory()
            Yh = torch.empty((B, wl.m), dtype=torch.float32).pin_memory()
            scratch = torch.empty(lf.dot_host_scratch_bytes(B), dtype=torch.uint8, device="cuda")
            lf.dot_host(Xh, Yh, scratch)
            check_outputs(Yh.numpy(), y_ref, a)


def test_edge_cases():
    rng = np.random.default_rng(77)
    # empty columns (first, middle, last), an all-zero matrix, a single shared value
    W = (rng.standard_normal((300, 40)) * 0.1).astype(np.float32)
    W[:, 0] = 0; W[:, 17] = 0; W[:, 39] = 0
    wl = dataclasses.replace(si.CFG1_TINY_SHAC, n=300, m=40, sparsity=0.5, k=8)
    for kind in ("shac", "hac"):
        lf, Wq, mask = build_both(wl, kind, W=W)
        check_decode(lf, Wq, mask)
        for B in (1, 9):
            X = si.inputs(wl, B)
            y_ref, a = orc.dot_definition(Wq, X)
            y = run_dot(lf, X)
            check_outputs(y, y_ref, a)
            assert np.all(y[:, [0, 17, 39]] == 0)
    Z = np.zeros((50, 6), dtype=np.float32)
    wz = dataclasses.replace(wl, n=50, m=6, sparsity=0.0, quantizer=si.QUANT_NONE)
    for kind in ("shac", "hac"):
        lf, Wq, mask = build_both(wz, kind, W=Z)
        for B in (1, 4):
            assert np.all(run_dot(lf, si.inputs(wz, B)) == 0)
    C1 = np.full((70, 9), 0.375, dtype=np.float32)
    for kind in ("shac", "hac"):
        lf, Wq, mask = build_both(wz, kind, W=C1)
        check_decode(lf, Wq, mask)
        X = si.inputs(dataclasses.replace(wz, n=70), 3)
        y_ref, a = orc.dot_definition(Wq, X)
        check_outputs(run_dot(lf, X), y_ref, a)


def test_long_code_words_take_the_slow_path():
    # geometric symbol frequencies: code lengths up to ~20 bits, beyond the primary table
    rng = np.random.default_rng(5)
    k = 22
    p = 0.5 ** np.arange(1, k + 1)
    p /= p.sum()
    values = np.sort(rng.standard_normal(k).astype(np.float32))
    W = values[rng.choice(k, size=(4096, 300), p=p)].astype(np.float32)
    W[:k, 0] = values                                     # every value occurs
    wl = dataclasses.replace(si.CFG1_TINY_SHAC, n=4096, m=300, sparsity=0.0, quantizer=si.QUANT_NONE)
    for kind in ("hac", "shac"):
        lf, Wq, mask = build_both(wl, kind, W=W)
        assert lf.sizes()["max_code_len"] > 12
        check_decode(lf, Wq, mask)
        X = si.inputs(wl, 2)
        y_ref, a = orc.dot_definition(Wq, X)
        check_outputs(run_dot(lf, X), y_ref, a)
        check_outputs(run_dot(lf, X[:1]), y_ref[:1], a[:1])


def test_wide_row_index_and_large_n():
    wl = si.scaled(si.CFG3_FC_SHAC, 70000, 24)            # n > 65536: 32-bit ri, x too large for shared memory
    lf, Wq, mask = build_both(wl, "shac")
    assert lf.sizes()["ri_bits"] == 32
    check_decode(lf, Wq, mask)
    for B in (1, 8):
        X = si.inputs(wl, B)
        y_ref, a = orc.dot_definition(Wq, X)
        check_outputs(run_dot(lf, X), y_ref, a)
    lf, Wq, mask = build_both(dataclasses.replace(wl, sparsity=0.5, k=16), "hac")
    X = si.inputs(wl, 1)
    y_ref, a = orc.dot_definition(Wq, X)
    check_outputs(run_dot(lf, X), y_ref, a)


def _structured_sample(rng, m, B, ncols):
    """Columns: `ncols` random ones plus one from every block of 128 columns (the unit a block of the batched
    kernels owns; every column carries all row splits).  Inputs: all when there are at most 8, else 8 random
    ones plus one from every tile of 64 inputs."""
    cols = set(rng.choice(m, size=min(ncols, m), replace=False).tolist())
    for c0 in range(0, m, 128):
        cols.add(int(c0 + rng.integers(0, min(128, m - c0))))
    if B <= 8:
        rows = set(range(B))
    else:
        rows = set(rng.choice(B, size=8, replace=False).tolist())
        for b0 in range(0, B, 64):
            rows.add(int(b0 + rng.integers(0, min(64, B - b0))))
    return np.array(sorted(cols)), np.array(sorted(rows))


def _full_size(wl, kind, batches, ncols=48, S=0, quantized=None, all_outputs_up_to=1):
    """Full-size parity.  One input: every output, against Algorithm 1 / 2 run literally.  A batch: every
    output against the written-out definition when the batch is at most `all_outputs_up_to`, else a
    structured sample.  `quantized` = (W, Wq, mask) lets several formats share one run of the oracle's
    quantizer."""
    if quantized is None:
        lf, Wq, mask = build_both(wl, kind, S)
    else:
        W, Wq, mask = quantized
        lf = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                       seed=wl.seed, seg_symbols=S).upload()
    check_decode(lf, Wq, mask)
    rng = np.random.default_rng(wl.seed)
    worst = 0.0
    for B in batches:
        X = si.inputs(wl, B)
        y = run_dot(lf, X)
        if B == 1:                                          # all outputs, via Algorithm 1 / 2
            ofmt = orc.hac_encode(Wq) if kind == "hac" else orc.shac_encode(Wq, mask)
            y_alg = (orc.dot_hac if kind == "hac" else orc.dot_shac)(ofmt, X[0])
            cols = np.sort(rng.choice(wl.m, size=min(ncols, wl.m), replace=False))
            y_ref, a = orc.dot_definition(Wq, X, cols=cols)
            assert np.array_equal(y_alg[cols], y_ref[0])
            a_all = np.abs(Wq.astype(np.float64)).T @ np.abs(X[0].astype(np.float64))
            worst = max(worst, check_outputs(y[0], y_alg, a_all * (1 + 1e-9)))
        elif B <= all_outputs_up_to:
            y_ref, a = orc.dot_definition(Wq, X)
            worst = max(worst, check_outputs(y, y_ref, a))
        else:
            cols, rows = _structured_sample(rng, wl.m, B, ncols)
            y_ref, a = orc.dot_definition(Wq, X[rows], cols=cols)
            worst = max(worst, check_outputs(y[np.ix_(rows, cols)], y_ref, a))
    return worst


def test_config2_dense_hac_full_size():
    _full_size(si.CFG2_DENSE_HAC, "hac", (1, 64), all_outputs_up_to=64)     # all 4096 x 64 outputs of the batch


def test_config3_fc_shac_full_size():
    _full_size(si.CFG3_FC_SHAC, "shac", (1, 16, 128), all_outputs_up_to=16)


def test_config4_conv_full_size():
    wl = dataclasses.replace(si.CFG4_CONV, batches=(6272,))
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    _full_size(wl, "shac", (1, 6272), quantized=(W, Wq, mask))
    _full_size(wl, "hac", (1, 6272), quantized=(W, Wq, mask))


SWEEP = [(c.sparsity, c.k) for c in si.sweep_cells()]


@pytest.mark.parametrize("sp,k", SWEEP, ids=[f"p{int(round(100 * sp))}-k{k}" for sp, k in SWEEP])
def test_config5_sweep_cells_full_size(sp, k):
    """Every cell of the sparsity x k sweep, both formats on one run of the oracle's quantizer."""
    cell = [c for c in si.sweep_cells() if c.sparsity == sp and c.k == k][0]
    W = si.weights(cell)
    Wq, mask = orc.quantize(W, cell.sparsity, cell.k, cell.quantizer, cell.kmeans_iters, cell.seed)
    for kind in ("hac", "shac"):
        _full_size(cell, kind, (1, 32), ncols=32, quantized=(W, Wq, mask))


PAPER_CELLS = si.paper_shaped_cells()


@pytest.mark.parametrize("cell", PAPER_CELLS, ids=[c.name for c in PAPER_CELLS])
def test_paper_shaped_cells_all_formats(cell):
    """The fully connected shapes of the paper's comparison of formats (Sect. V-C), one input and its eight inputs: HAC and
    sHAC on every output, and the index map and CSC of the same quantized matrix, all against the oracle."""
    from paper_2108_12704_b200.binding import Csc, IndexMap
    W = si.weights(cell)
    Wq, mask = orc.quantize(W, cell.sparsity, cell.k, cell.quantizer, cell.kmeans_iters, cell.seed)
    for kind in ("hac", "shac"):
        _full_size(cell, kind, (1, 8), ncols=min(32, cell.m), quantized=(W, Wq, mask), all_outputs_up_to=8)
    X = si.inputs(cell, 8)
    y_ref, a = orc.dot_definition(Wq, X)
    for fmt in (IndexMap(Wq, 8 if len(np.unique(Wq)) <= 256 else 16).upload(), Csc(Wq).upload()):
        check_outputs(run_dot(fmt, X), y_ref, a)
        check_outputs(run_dot(fmt, X[:1]), y_ref[:1], a[:1])


def test_chained_products_keep_stream_order():
    """Two layers back to back on one stream, the second reading what the first wrote, then the same
    buffers reused at once for another input: the kernels may start early (they are launched with
    programmatic stream serialization) but must not read x or write y before the kernel ahead of them
    is done."""
    wl = si.scaled(si.CFG2_DENSE_HAC, 1536, 1536)
    lf, Wq, mask = build_both(wl, "hac", 64)
    Wd = Wq.astype(np.float64)
    for B in (1, 64):
        X = si.inputs(wl, B)
        ws = torch.empty(max(16, lf.workspace_bytes(B)), dtype=torch.uint8, device="cuda")
        x0 = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
        shape = (wl.m,) if B == 1 else (wl.m, B)
        y1 = torch.empty(shape, device="cuda")
        y2 = torch.empty(shape, device="cuda")
        outs = []
        for rep in range(3):                       # no synchronisation between the launches
            lf.dot(x0, y1, ws)
            lf.dot(y1, y2, ws)
            outs.append(y2.clone())
            x0 = x0 * 0.5                          # a new input in a new buffer; y1, y2 and ws are reused
        torch.cuda.synchronize()
        Xd = X.astype(np.float64)
        for rep, got in enumerate(outs):
            h1 = (Xd * 0.5 ** rep) @ Wd
            ref = h1 @ Wd
            a = np.abs(h1) @ np.abs(Wd) + (np.abs(Xd * 0.5 ** rep) @ np.abs(Wd)) @ np.abs(Wd)
            g = got.cpu().numpy()
            g = g[None] if B == 1 else g.T
            check_outputs(g, ref, a)


def test_largest_sub_segments_with_wide_row_indices():
    """S = 1024 with 32-bit row indices: two staged segments do not fit the shared memory of an SM, so a
    single input goes through the batched kernel; the result must not change."""
    wl = dataclasses.replace(si.scaled(si.CFG3_FC_SHAC, 70000, 6), sparsity=0.2, k=64)
    lf, Wq, mask = build_both(wl, "shac", 1024)
    assert lf.sizes()["ri_bits"] == 32
    check_decode(lf, Wq, mask)
    for B in (1, 3):
        X = si.inputs(wl, B)
        y_ref, a = orc.dot_definition(Wq, X)
        check_outputs(run_dot(lf, X), y_ref, a)


def test_grouped_decode_with_unresolved_entries():
    """The kernels that decode three code words per window call a slower routine for a group that meets a
    first-level entry without its symbol.  With the magnitude table switched off (a diagnostic switch that is
    read once per process, hence the child process) a long-tailed code leaves such entries in the prefix table,
    rarely enough that those kernels still take the format: results must not change."""
    import os, subprocess, sys
    code = r'''
import dataclasses, numpy as np, torch
import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb
rng = np.random.default_rng(5)
k = 22
p = 0.35 ** np.arange(1, k + 1); p /= p.sum()          # code words beyond the 10-bit table: about 3 in 100000
values = np.sort(rng.standard_normal(k).astype(np.float32))
W = values[rng.choice(k, size=(4096, 300), p=p)].astype(np.float32)
W[:k, 0] = values
wl = dataclasses.replace(si.CFG1_TINY_SHAC, n=4096, m=300, sparsity=0.0, quantizer=si.QUANT_NONE)
Wq, mask = orc.quantize(W, 0.0, wl.k, si.QUANT_NONE, 0, 0)
for kind in ("hac", "shac"):
    lf = hb.Format(kind, W, sparsity=0.0, k=wl.k, quantizer=si.QUANT_NONE).upload()
    got = lf.debug_decode().cpu().numpy()
    want = np.ascontiguousarray(Wq.T) if kind == "hac" else Wq.T[mask.T]
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), kind
    for B in (1, 64):
        X = si.inputs(wl, B)
        y_ref, a = orc.dot_definition(Wq, X)
        xin = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
        y = lf.dot(xin).cpu().numpy()
        y = y[None] if B == 1 else y.T
        assert np.all(np.abs(y - y_ref) <= 1e-5 * a + 1e-7), (kind, B)
print("ok")
'''
    env = dict(os.environ, HAC_B200_XT="0")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout + out.stderr


def test_column_shards_give_the_whole_product():
    """Column sharding (one product split over several GPUs) on one GPU: the shards of two and three ranks are multiplied one
    after the other and their slices put side by side; the exchange itself is covered by the two-rank CPU test."""
    from paper_2108_12704_b200.sharded import ColumnSharded
    wl = si.scaled(si.CFG3_FC_SHAC, 3000, 101)
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    quant = dict(sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters, seed=wl.seed)
    X = si.inputs(wl, 5)
    y_ref, a = orc.dot_definition(Wq, X)
    for kind in ("shac", "hac"):
        for world in (1, 2, 3):
            slices = []
            for rank in range(world):
                sh = ColumnSharded(kind, W, rank, world, **quant).upload()
                slices.append(sh.format.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda()).cpu().numpy().T)
            check_outputs(np.concatenate(slices, axis=1), y_ref, a)
    one = ColumnSharded("shac", W, 0, 1, **quant).upload()
    check_outputs(one.dot(torch.from_numpy(X[0]).cuda()).cpu().numpy()[None], y_ref[:1], a[:1])


def test_no_bounded_wait_ran_out():
    """The batched kernel marks outputs NaN and counts the block when one of its bounded waits runs out; after batched products
    of both formats the count must still be zero and the outputs finite."""
    from paper_2108_12704_b200.binding import lost_waits
    for wl, kind in ((si.scaled(si.CFG2_DENSE_HAC, 2100, 300), "hac"), (si.scaled(si.CFG4_CONV, 1152, 128), "shac")):
        lf, Wq, mask = build_both(wl, kind)
        y = run_dot(lf, si.inputs(wl, 70))
        assert np.isfinite(y).all()
    assert lost_waits() == 0


def test_rowblock_kernel_forced_on_every_shape():
    """The batched sHAC kernel that stages rows of X is chosen only for many inputs and very sparse layers; here a
    diagnostic switch (read once per process, hence the child process) sends every batched sHAC product through it:
    ragged batches, unaligned X, several row splits, 32-bit row indices."""
    import os, subprocess, sys
    code = r'''
import dataclasses, numpy as np, torch
import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb
cases = [(si.scaled(si.CFG3_FC_SHAC, 6000, 200), 0, (5, 40, 64, 130)), (si.scaled(si.CFG4_CONV, 1152, 128), 0, (33, 200)),
         (si.scaled(si.CFG3_FC_SHAC, 70000, 24), 0, (64,)), (si.CFG1_TINY_SHAC, 0, (2, 70))]
for wl, S, batches in cases:
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    lf = hb.Format("shac", W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                   seed=wl.seed, seg_symbols=S).upload()
    for B in batches:
        X = si.inputs(wl, B)
        y_ref, a = orc.dot_definition(Wq, X)
        y = lf.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda()).cpu().numpy().T
        assert np.all(np.abs(y - y_ref) <= 1e-5 * a + 1e-7), (wl.name, B)
        bias = torch.linspace(-1, 1, wl.m, device="cuda")
        yb = lf.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda(), bias=bias, relu=True).cpu().numpy().T
        ref = np.maximum(y_ref + bias.cpu().numpy().astype(np.float64), 0)
        assert np.all(np.abs(yb - ref) <= 1e-5 * (a + 1) + 1e-6), (wl.name, B, "layer")
print("ok")
'''
    env = dict(os.environ, HAC_B200_SHAC_ROWS="2")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout + out.stderr
