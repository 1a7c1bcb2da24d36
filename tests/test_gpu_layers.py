"""Layer evaluation on the compressed formats (bias and activation applied in the product kernels, stacks
of layers as one chained submission) against the oracle's written-out definition, through the C ABI."""
import dataclasses

import numpy as np
import pytest

import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb
from golden_io import golden, read_sections

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

RTOL_A, ATOL = 1e-5, 1e-7


def _check(y, y_ref, a):
    err = np.abs(y.astype(np.float64) - y_ref)
    bound = RTOL_A * a + ATOL
    assert np.all(err <= bound), f"worst error / bound = {float((err / bound).max())}"


def _build(wl, kind, S=0):
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    lf = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                   seed=wl.seed, seg_symbols=S).upload()
    return lf, Wq


def test_hand_worked_layer_through_the_library():
    g = read_sections(golden("layer_hand_worked.txt"))
    num = lambda key: np.array([[float(v) for v in row] for row in g[key]])
    W = num("W").astype(np.float32); x = num("x")[0].astype(np.float32)
    bias = torch.tensor(num("bias")[0], dtype=torch.float32, device="cuda")
    for kind in ("hac", "shac"):
        f = hb.Format(kind, W, sparsity=0.0, k=16, quantizer=si.QUANT_NONE).upload()
        y = f.dot(torch.from_numpy(x).cuda(), bias=bias, relu=False).cpu().numpy()
        assert y.tolist() == num("linear")[0].tolist()
        y = f.dot(torch.from_numpy(x).cuda(), bias=bias, relu=True).cpu().numpy()
        assert y.tolist() == num("relu")[0].tolist()


CASES = [
    (si.scaled(si.CFG2_DENSE_HAC, 2100, 300), "hac", 64, (1, 64, 70)),       # rows kernel; cluster and plain batched kernels
    (si.scaled(si.CFG2_DENSE_HAC, 777, 45), "hac", 7, (1, 5)),               # older single-input kernel, several segments
    (si.scaled(si.CFG3_FC_SHAC, 6000, 200), "shac", 0, (1, 16)),
    (si.scaled(si.CFG3_FC_SHAC, 6000, 90), "shac", 3, (1, 40)),              # several segments per column: finishing kernel
    (si.scaled(si.CFG4_CONV, 1152, 128), "hac", 0, (1, 200)),
]


@pytest.mark.parametrize("wl,kind,S,batches", CASES, ids=[f"{c[0].name}-{c[1]}-S{c[2]}" for c in CASES])
def test_bias_and_relu_in_every_product_path(wl, kind, S, batches):
    lf, Wq = _build(wl, kind, S)
    rng = np.random.default_rng(wl.seed + 1)
    bias = (rng.standard_normal(wl.m) * 0.5).astype(np.float32)
    bias_d = torch.from_numpy(bias).cuda()
    for B in batches:
        X = si.inputs(wl, B)
        for use_bias, relu in ((True, True), (True, False), (False, True)):
            y_ref, a = orc.layer_definition(Wq, X, bias if use_bias else None, relu)
            for layout in (("nb", "bn") if B > 1 else ("nb",)):
                if B == 1:
                    y = lf.dot(torch.from_numpy(X[0]).cuda(), bias=bias_d if use_bias else None, relu=relu).cpu().numpy()[None]
                elif layout == "nb":
                    y = lf.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda(), layout="nb",
                               bias=bias_d if use_bias else None, relu=relu).cpu().numpy().T
                else:
                    y = lf.dot(torch.from_numpy(X).cuda(), layout="bn", bias=bias_d if use_bias else None,
                               relu=relu).cpu().numpy()
                _check(y, y_ref, a)
                if relu:
                    assert (y >= 0).all()


def test_empty_columns_get_their_bias():
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((300, 40)) * 0.1).astype(np.float32)
    W[:, 0] = 0; W[:, 17] = 0
    wl = dataclasses.replace(si.CFG1_TINY_SHAC, n=300, m=40, sparsity=0.5, k=8)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    bias = np.linspace(-1, 1, 40).astype(np.float32)
    for kind in ("shac", "hac"):
        lf = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters,
                       seed=wl.seed).upload()
        for B in (1, 9):
            X = si.inputs(wl, B)
            y_ref, a = orc.layer_definition(Wq, X, bias, True)
            xin = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
            y = lf.dot(xin, bias=torch.from_numpy(bias).cuda(), relu=True).cpu().numpy()
            y = y[None] if B == 1 else y.T
            _check(y, y_ref, a)
            assert np.all(y[:, 0] == max(bias[0], 0)) and np.all(y[:, 17] == max(bias[17], 0))


def fc_stack(scale=1):
    """The fully connected stack of the paper's VGG19 (512 -> 4096 -> 4096 -> 10, Sect. V), scaled down by `scale`:
    the first layer pruned and stored as sHAC, the second dense HAC, the last a small HAC layer."""
    d0, d1, d2 = 512 // scale, 4096 // scale, 10
    specs = [(dataclasses.replace(si.CFG3_FC_SHAC, n=d0, m=d1, sparsity=0.9, k=32, item=11), "shac", True),
             (dataclasses.replace(si.CFG2_DENSE_HAC, n=d1, m=d1, k=64, item=12), "hac", True),
             (dataclasses.replace(si.CFG2_DENSE_HAC, n=d1, m=d2, k=32, quantizer=si.QUANT_KMEANS, item=13), "hac", False)]
    return specs


@pytest.mark.parametrize("scale,batches", [(4, (1, 8)), (1, (1, 64))], ids=["quarter", "full"])
def test_chain_of_layers(scale, batches):
    layers, oracle_layers = [], []
    rng = np.random.default_rng(99)
    for wl, kind, relu in fc_stack(scale):
        lf, Wq = _build(wl, kind)
        bias = (rng.standard_normal(wl.m) * 0.1).astype(np.float32)
        layers.append((lf, torch.from_numpy(bias).cuda(), relu))
        oracle_layers.append((Wq, bias, relu))
    n0 = oracle_layers[0][0].shape[0]
    for B in batches:
        X = np.maximum(np.random.default_rng(B).standard_normal((B, n0)), 0).astype(np.float32)
        xin = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
        y, launches = hb.hac_chain(layers, xin)
        torch.cuda.synchronize()
        assert launches >= len(layers)
        # layer by layer: every layer of the chain is checked on the input it really saw
        cur = xin
        for (lf, bias_d, relu), (Wq, bias, _) in zip(layers, oracle_layers):
            got = lf.dot(cur, bias=bias_d, relu=relu)
            inp = cur.cpu().numpy()
            inp = inp[None] if B == 1 else inp.T
            y_ref, a = orc.layer_definition(Wq, inp, bias, relu)
            g = got.cpu().numpy()
            _check(g[None] if B == 1 else g.T, y_ref, a)
            cur = got
        assert torch.equal(cur, y), "the chained submission must give what the layers give one by one"


def test_chain_of_layers_with_one_dictionary():
    """The same stack (scaled down) quantized together (unified quantization, Sect. V-D): one codebook and one code for the
    three layers, every layer multiplied from its own stream, layer by layer against the oracle."""
    specs = fc_stack(4)
    Ws = [si.weights(wl) for wl, _, _ in specs]
    sparsity, k, iters, seed = 0.8, 48, 8, 5
    parts = orc.quantize_unified(Ws, sparsity, k, si.QUANT_KMEANS, iters, seed)
    lfs = hb.hac_build_unified([(kind, W) for (_, kind, _), W in zip(specs, Ws)], sparsity=sparsity, k=k,
                               quantizer=si.QUANT_KMEANS, kmeans_iters=iters, seed=seed)
    cb0 = lfs[0].export()["codebook"]
    rng = np.random.default_rng(98)
    layers, oracle_layers = [], []
    for lf, (wl, _, relu), (Wq, _) in zip(lfs, specs, parts):
        assert np.array_equal(lf.export()["codebook"], cb0)
        lf.upload()
        assert np.array_equal(lf.decode_host().view(np.uint32), Wq.view(np.uint32))
        if lf.kind == "hac":                                  # the kernels' decoder with a code that has unused symbols
            got = lf.debug_decode().cpu().numpy()
            assert np.array_equal(got.view(np.uint32), np.ascontiguousarray(Wq.T).view(np.uint32))
        bias = (rng.standard_normal(wl.m) * 0.1).astype(np.float32)
        layers.append((lf, torch.from_numpy(bias).cuda(), relu))
        oracle_layers.append((Wq, bias, relu))
    n0 = Ws[0].shape[0]
    for B in (1, 8):
        X = np.maximum(np.random.default_rng(B).standard_normal((B, n0)), 0).astype(np.float32)
        xin = torch.from_numpy(X[0] if B == 1 else np.ascontiguousarray(X.T)).cuda()
        y, _ = hb.hac_chain(layers, xin)
        cur = xin
        for (lf, bias_d, relu), (Wq, bias, _) in zip(layers, oracle_layers):
            got = lf.dot(cur, bias=bias_d, relu=relu)
            inp = cur.cpu().numpy()
            inp = inp[None] if B == 1 else inp.T
            y_ref, a = orc.layer_definition(Wq, inp, bias, relu)
            g = got.cpu().numpy()
            _check(g[None] if B == 1 else g.T, y_ref, a)
            cur = got
        assert torch.equal(cur, y)
