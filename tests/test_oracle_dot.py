"""Pins of the oracle's dot procedures: Algorithms 1-3 must output x^T W (Sect. IV-B,
IV-C, IV-D), i.e. agree with the written-out definition, with a library fp64 product,
and with the special inputs whose answer is known (unit vectors, all ones)."""
import numpy as np
import pytest

from oracle import hac_oracle as orc


def quantized(seed, n, m, sparsity, k):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((n, m)) * np.sqrt(2.0 / n)).astype(np.float32)
    return orc.quantize(W, sparsity, k, 1, iters=5, seed=seed)


@pytest.mark.parametrize("n,m,sp,k", [(33, 17, 0.0, 8), (70, 40, 0.6, 16), (129, 65, 0.9, 32), (64, 31, 0.99, 4)])
def test_algorithms_equal_definition_bit_for_bit(n, m, sp, k):
    Wq, mask = quantized(n + m, n, m, sp, k)
    rng = np.random.default_rng(1)
    x = rng.uniform(-1, 1, n).astype(np.float32)
    y_def, a = orc.dot_definition(Wq, x)
    fh = orc.hac_encode(Wq)
    fs = orc.shac_encode(Wq, mask)
    y1 = orc.dot_hac(fh, x)
    y2 = orc.dot_shac(fs, x)
    # same order of additions; the null entries add exact zeros
    assert np.array_equal(y1, y_def[0])
    assert np.array_equal(y2, y_def[0])
    # a library product in fp64 agrees to rounding
    y_lib = x.astype(np.float64) @ Wq.astype(np.float64)
    assert np.all(np.abs(y_lib - y_def[0]) <= 1e-13 * a[0] + 1e-300)


def test_unit_vectors_return_rows_and_ones_return_column_sums():
    Wq, mask = quantized(3, 48, 20, 0.7, 8)
    fh = orc.hac_encode(Wq)
    fs = orc.shac_encode(Wq, mask)
    for i in (0, 17, 47):
        e = np.zeros(48, dtype=np.float32)
        e[i] = 1.0
        assert np.array_equal(orc.dot_hac(fh, e), Wq[i].astype(np.float64))
        assert np.array_equal(orc.dot_shac(fs, e), Wq[i].astype(np.float64))
    ones = np.ones(48, dtype=np.float32)
    col_sums = np.array([sum(float(v) for v in Wq[:, j]) for j in range(20)])
    assert np.array_equal(orc.dot_hac(fh, ones), col_sums)
    assert np.array_equal(orc.dot_shac(fs, ones), col_sums)


def test_transposed_operand_would_be_caught():
    # a non-square, non-symmetric case where x^T W differs from W x padded any way
    W = np.arange(1, 13, dtype=np.float32).reshape(4, 3)
    x = np.array([1, 0, 2, 0], dtype=np.float32)
    want = np.array([1 * 1 + 2 * 7, 1 * 2 + 2 * 8, 1 * 3 + 2 * 9], dtype=np.float64)
    assert np.array_equal(orc.dot_hac(orc.hac_encode(W), x), want)
    assert np.array_equal(orc.dot_shac(orc.shac_encode(W, W != 0), x), want)
    assert np.array_equal(orc.dot_definition(W, x)[0][0], want)


def test_empty_columns_and_empty_matrix():
    Wq, mask = quantized(9, 40, 12, 0.8, 4)
    Wq[:, 0] = 0; Wq[:, 5] = 0; Wq[:, 11] = 0          # first, middle and last column empty
    mask = Wq != 0
    x = np.random.default_rng(2).uniform(-1, 1, 40).astype(np.float32)
    y = orc.dot_shac(orc.shac_encode(Wq, mask), x)
    assert np.array_equal(y, orc.dot_definition(Wq, x)[0][0])
    assert y[0] == 0 and y[5] == 0 and y[11] == 0
    Z = np.zeros((6, 4), dtype=np.float32)
    assert np.array_equal(orc.dot_shac(orc.shac_encode(Z, Z != 0), x[:6]), np.zeros(4))
    assert np.array_equal(orc.dot_hac(orc.hac_encode(Z), x[:6]), np.zeros(4))   # one symbol, 1 bit each


def test_stored_zero_value_in_shac():
    # a surviving weight whose shared value is 0.0 stays a stored entry of sHAC
    Wq = np.array([[0.0, 2.0], [1.0, 0.0]], dtype=np.float32)
    mask = np.array([[True, True], [True, False]])
    fs = orc.shac_encode(Wq, mask)
    assert fs["cb"].tolist() == [0, 2, 3] and fs["nz"].tolist() == [0.0, 1.0, 2.0]
    x = np.array([3.0, 5.0], dtype=np.float32)
    assert orc.dot_shac(fs, x).tolist() == [5.0, 6.0]


@pytest.mark.parametrize("q", [1, 3, 8])
def test_pardot_equals_row_by_row(q):
    Wq, mask = quantized(21, 60, 25, 0.75, 8)
    X = np.random.default_rng(4).uniform(0, 1, (7, 60)).astype(np.float32)
    for fmt in (orc.hac_encode(Wq), orc.shac_encode(Wq, mask)):
        Y = orc.pardot(fmt, X, q)
        single = orc.dot_hac if fmt["kind"] == "hac" else orc.dot_shac
        for b in range(7):
            assert np.array_equal(Y[b], single(fmt, X[b]))
        assert np.array_equal(Y, orc.dot_definition(Wq, X)[0])


def test_definition_column_subset():
    Wq, _ = quantized(5, 30, 16, 0.5, 8)
    X = np.random.default_rng(6).uniform(-1, 1, (3, 30)).astype(np.float32)
    y, a = orc.dot_definition(Wq, X)
    cols = np.array([0, 7, 15])
    ys, as_ = orc.dot_definition(Wq, X, cols=cols)
    assert np.array_equal(ys, y[:, cols]) and np.array_equal(as_, a[:, cols])


# ---------------------------------------------------------------- layers (bias, activation, chains)
def test_layer_definition_against_the_hand_worked_example():
    from golden_io import golden, read_sections
    g = read_sections(golden("layer_hand_worked.txt"))
    num = lambda key: np.array([[float(v) for v in row] for row in g[key]])
    W = num("W").astype(np.float32); x = num("x")[0].astype(np.float32); bias = num("bias")[0]
    y, a = orc.layer_definition(W, x, bias, relu=False)
    assert y[0].tolist() == num("linear")[0].tolist() and a[0].tolist() == num("scale")[0].tolist()
    y, _ = orc.layer_definition(W, x, bias, relu=True)
    assert y[0].tolist() == num("relu")[0].tolist()
    V = num("V").astype(np.float32); bias2 = num("bias2")[0]
    outs = orc.chain_definition([(W, bias, True), (V, bias2, False)], x)
    assert outs[1][0][0].tolist() == num("chain_linear")[0].tolist()
    outs = orc.chain_definition([(W, bias, True), (V, bias2, True)], x)
    assert outs[1][0][0].tolist() == num("chain_relu")[0].tolist()


def test_layer_definition_properties():
    rng = np.random.default_rng(11)
    W = rng.standard_normal((40, 9)).astype(np.float32); X = rng.standard_normal((3, 40)).astype(np.float32)
    b = rng.standard_normal(9)
    y0, a0 = orc.dot_definition(W, X)
    y1, a1 = orc.layer_definition(W, X)                       # no bias, no activation: the product itself
    assert np.array_equal(y0, y1) and np.array_equal(a0, a1)
    yb, ab = orc.layer_definition(W, X, b)
    assert np.array_equal(yb, y0 + b) and np.array_equal(ab, a0 + np.abs(b))
    yr, _ = orc.layer_definition(W, X, b, relu=True)
    assert np.array_equal(yr, np.maximum(yb, 0.0)) and (yr >= 0).all()
    cols = np.array([1, 4, 8])
    yc, ac = orc.layer_definition(W, X, b, relu=True, cols=cols)
    assert np.array_equal(yc, yr[:, cols]) and np.array_equal(ac, ab[:, cols])
    # a chain equals the layers applied one after the other with fp32 activations in between
    V = rng.standard_normal((9, 4)).astype(np.float32)
    outs = orc.chain_definition([(W, b, True), (V, None, False)], X)
    want, _ = orc.dot_definition(V, yr.astype(np.float32))
    assert np.array_equal(outs[1][0], want)
