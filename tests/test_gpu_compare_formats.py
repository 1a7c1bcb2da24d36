"""The products of the comparison formats (index map, Sect. III-C.1; CSC, Sect. IV-A) on the device against the
oracle, element by element, on the quantized matrices the HAC / sHAC tests use."""
import numpy as np
import pytest

import synth_inputs as si
from oracle import hac_oracle as orc
from paper_2108_12704_b200.binding import Csc, IndexMap

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

RTOL_A, ATOL = 1e-5, 1e-7


def _check(y, y_ref, a):
    err = np.abs(y.astype(np.float64) - y_ref)
    assert np.all(err <= RTOL_A * a + ATOL), float((err / (RTOL_A * a + ATOL)).max())


def _quantized(wl):
    W = si.weights(wl)
    Wq, _ = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    return Wq


def _run(fmt, X, layout):
    if X.shape[0] == 1:
        return fmt.dot(torch.from_numpy(X[0]).cuda()).cpu().numpy()[None]
    if layout == "nb":
        return fmt.dot(torch.from_numpy(np.ascontiguousarray(X.T)).cuda(), layout="nb").cpu().numpy().T
    return fmt.dot(torch.from_numpy(X).cuda(), layout="bn").cpu().numpy()


CASES = [
    (si.scaled(si.CFG2_DENSE_HAC, 2096, 70), 8),           # n a multiple of 16: 128-bit loads of the pointers
    (si.scaled(si.CFG2_DENSE_HAC, 777, 45), 8),            # ragged: element loads
    (si.scaled(si.CFG2_DENSE_HAC, 1000, 130), 16),         # two-byte pointers, n a multiple of 8
    (si.scaled(si.CFG2_DENSE_HAC, 333, 20), 16),
    (si.scaled(si.CFG3_FC_SHAC, 6000, 200), 8),
]


@pytest.mark.parametrize("wl,bits", CASES, ids=[f"{c[0].name}-{c[1]}" for c in CASES])
@pytest.mark.parametrize("batch,layout", [(1, "nb"), (5, "nb"), (9, "bn")])
def test_index_map_product(wl, bits, batch, layout):
    Wq = _quantized(wl)
    im = IndexMap(Wq, bits).upload()
    X = si.inputs(wl, batch)
    y_ref, a = orc.dot_index_map(orc.index_map_encode(Wq), X)
    _check(_run(im, X, layout), y_ref, a)


CSC_CASES = [si.scaled(si.CFG3_FC_SHAC, 6000, 200), si.scaled(si.CFG4_CONV, 1152, 128), si.CFG1_TINY_SHAC]


@pytest.mark.parametrize("wl", CSC_CASES, ids=[c.name for c in CSC_CASES])
@pytest.mark.parametrize("batch,layout", [(1, "nb"), (6, "nb"), (7, "bn")])
def test_csc_product(wl, batch, layout):
    Wq = _quantized(wl)
    c = Csc(Wq).upload()
    X = si.inputs(wl, batch)
    nz, ri, cb = orc.csc(Wq, Wq != 0)
    y_ref, a = orc.dot_csc(nz, ri, cb, wl.n, X)
    _check(_run(c, X, layout), y_ref, a)


def test_csc_with_empty_columns_and_an_empty_matrix():
    W = np.zeros((50, 9), dtype=np.float32)
    x = torch.ones(50, device="cuda")
    assert not Csc(W).upload().dot(x).cpu().numpy().any()
    W[3, 2] = 2.0; W[49, 8] = -1.5
    y = Csc(W).upload().dot(x).cpu().numpy()
    assert y.tolist() == [0, 0, 2.0, 0, 0, 0, 0, 0, -1.5]


def test_full_size_dense_layer_index_map_equals_hac_inputs():
    """The 4096 x 4096 dense layer at full size: sampled columns against the oracle."""
    wl = si.CFG2_DENSE_HAC
    Wq = _quantized(wl)
    im = IndexMap(Wq, 8).upload()
    X = si.inputs(wl, 1)
    y = _run(im, X, "nb")
    cols = np.random.default_rng(5).choice(wl.m, 64, replace=False)
    y_ref, a = orc.dot_definition(Wq[:, cols], X)
    _check(y[:, cols], y_ref, a)
