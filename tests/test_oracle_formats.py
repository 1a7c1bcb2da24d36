"""Pins of the oracle's format code: the examples the paper prints (Sect. IV-A Example 2,
Sect. IV-B address map), a stream worked out by hand from them, and the properties the
paper states for the formats (lossless, N = ceil(bits / b) words, Corollaries 1 and 2)."""
import numpy as np
import pytest

from oracle import hac_oracle as orc
from golden_io import golden, read_sections


def example2():
    g = read_sections(golden("example2_csc.txt"))
    W = np.array(g["W"], dtype=np.float32)
    nz = np.array(g["nz"][0], dtype=np.float32)
    ri = np.array(g["ri"][0], dtype=np.int64)
    cb = np.array(g["cb"][0], dtype=np.int64)
    return W, nz, ri, cb


def test_csc_matches_paper_example2():
    W, nz, ri, cb = example2()
    got_nz, got_ri, got_cb = orc.csc(W, W != 0)
    assert np.array_equal(got_nz, nz)
    assert np.array_equal(got_ri + 1, ri)          # the paper counts from 1
    assert np.array_equal(got_cb + 1, cb)


def test_hac_symbol_order_matches_paper_address_map():
    W, *_ = example2()
    tokens = read_sections(golden("example_address_map.txt"))[None][0]
    assert len(tokens) == 25
    fmt = orc.hac_encode(W)
    values = fmt["codebook"][fmt["sym"]]
    for tok, v in zip(tokens, values):
        want = 0.0 if tok == "0" else float(tok[2:-1])
        assert v == want
    # one code word per entry, zeros included: "q + 1 code words" for q distinct non-null values
    assert len(fmt["codebook"]) == len(np.unique(W[W != 0])) + 1


def test_hand_coded_example_hac():
    W, *_ = example2()
    g = read_sections(golden("example2_hand_coded.txt"))
    fmt = orc.hac_encode(W)
    assert np.array_equal(fmt["codebook"], np.array(g["hac_values"][0], dtype=np.float32))
    assert fmt["code_len"].tolist() == [int(t) for t in g["hac_lengths"][0]]
    assert [format(int(c), f"0{l}b") for c, l in zip(fmt["codes"], fmt["code_len"])] == g["hac_codes"][0]
    assert fmt["bits"] == int(g["hac_bits"][0][0])
    assert [f"{int(w):08X}" for w in fmt["words"]] == g["hac_words"][0]
    # one sub-segment per column (S = n): segment offsets are the column offsets
    idx = orc.hac_offset_index(fmt, S=5)
    want = [int(t) for t in g["hac_column_bit_offsets"][0]]
    assert idx["seg_bit_off"].tolist() == want[:-1]
    assert int(idx["seg_bit_off"][-1]) + int(idx["sub_bits"].reshape(-1, 32)[-1].sum()) == want[-1]


def test_hand_coded_example_shac_and_dot():
    W, *_ = example2()
    g = read_sections(golden("example2_hand_coded.txt"))
    fmt = orc.shac_encode(W, W != 0)
    assert np.array_equal(fmt["codebook"], np.array(g["shac_values"][0], dtype=np.float32))
    assert fmt["code_len"].tolist() == [int(t) for t in g["shac_lengths"][0]]
    assert [format(int(c), f"0{l}b") for c, l in zip(fmt["codes"], fmt["code_len"])] == g["shac_codes"][0]
    assert fmt["bits"] == int(g["shac_bits"][0][0])
    assert [f"{int(w):08X}" for w in fmt["words"]] == g["shac_words"][0]
    x = np.array(g["x"][0], dtype=np.float32)
    want = np.array(g["xTW"][0], dtype=np.float64)
    assert np.array_equal(orc.dot_shac(fmt, x), want)
    assert np.array_equal(orc.dot_hac(orc.hac_encode(W), x), want)
    assert np.array_equal(orc.dot_definition(W, x)[0][0], want)


def _random_quantized(rng, n, m, k, zero_frac):
    values = np.sort(rng.standard_normal(k).astype(np.float32))
    p = rng.dirichlet(np.ones(k) * 0.5)
    W = values[rng.choice(k, size=(n, m), p=p)]
    W[rng.random((n, m)) < zero_frac] = 0.0
    return W.astype(np.float32)


@pytest.mark.parametrize("n,m,k,zf", [(7, 5, 3, 0.5), (64, 33, 17, 0.0), (130, 70, 40, 0.9), (33, 9, 1, 0.0)])
def test_round_trip_is_lossless(n, m, k, zf):
    rng = np.random.default_rng(n * 1000 + m)
    W = _random_quantized(rng, n, m, k, zf)
    fh = orc.hac_encode(W)
    assert np.array_equal(orc.hac_decode(fh).view(np.uint32), W.view(np.uint32))
    fs = orc.shac_encode(W, W != 0)
    assert np.array_equal(orc.shac_decode(fs).view(np.uint32), W.view(np.uint32))


@pytest.mark.parametrize("n,m,k,zf", [(50, 20, 9, 0.3), (64, 64, 32, 0.8)])
def test_stream_length_and_padding(n, m, k, zf):
    rng = np.random.default_rng(5)
    W = _random_quantized(rng, n, m, k, zf)
    for fmt in (orc.hac_encode(W), orc.shac_encode(W, W != 0)):
        bits = int((fmt["counts"] * fmt["code_len"].astype(np.int64)).sum())
        assert fmt["bits"] == bits
        assert len(fmt["words"]) == -(-bits // 32)                       # N = ceil(|HAC| / b)
        pad = len(fmt["words"]) * 32 - bits
        if pad:
            assert int(fmt["words"][-1]) & ((1 << pad) - 1) == 0         # zero padding


def test_offset_index_segments_decode_alone():
    rng = np.random.default_rng(11)
    W = _random_quantized(rng, 300, 7, 12, 0.4)
    fmt = orc.hac_encode(W)
    S = 4
    idx = orc.hac_offset_index(fmt, S)
    n, m, G = fmt["n"], fmt["m"], idx["G"]
    assert idx["T"] == 75 and G == 3
    sym = fmt["sym"].reshape(m, n)
    for j in range(m):
        for g in range(G):
            u = j * G + g
            bit = int(idx["seg_bit_off"][u])
            for l in range(32):
                r0 = (g * 32 + l) * S
                cnt = max(0, min(S, n - r0))
                got, end = orc.decode_symbols(fmt, bit, cnt)
                assert np.array_equal(got, sym[j, r0:r0 + cnt])
                assert end - bit == int(idx["sub_bits"][u * 32 + l])
                bit = end
    last = len(idx["seg_bit_off"]) - 1
    assert int(idx["seg_bit_off"][last]) + int(idx["sub_bits"][last * 32:].sum()) == fmt["bits"]


def test_shac_offset_index_segments_decode_alone():
    rng = np.random.default_rng(12)
    W = _random_quantized(rng, 500, 9, 10, 0.6)
    W[:, 3] = 0.0                                       # an empty column
    fmt = orc.shac_encode(W, W != 0)
    S = 3
    idx = orc.shac_offset_index(fmt, S)
    cb = fmt["cb"]
    assert idx["seg_first"][3] == idx["seg_first"][4]
    for j in range(fmt["m"]):
        for u in range(int(idx["seg_first"][j]), int(idx["seg_first"][j + 1])):
            assert idx["seg_col"][u] == j
            g = u - int(idx["seg_first"][j])
            bit = int(idx["seg_bit_off"][u])
            for l in range(32):
                p0 = int(cb[j]) + (g * 32 + l) * S
                cnt = max(0, min(S, int(cb[j + 1]) - p0))
                got, end = orc.decode_symbols(fmt, bit, cnt)
                assert np.array_equal(got, fmt["sym"][p0:p0 + cnt])
                assert end - bit == int(idx["sub_bits"][u * 32 + l])
                bit = end
    assert len(idx["seg_col"]) == int(idx["seg_first"][-1])


@pytest.mark.parametrize("k", [2, 8, 32])
@pytest.mark.parametrize("zf", [0.0, 0.5, 0.9, 0.99])
def test_sizes_within_corollaries(k, zf):
    rng = np.random.default_rng(k * 100 + int(zf * 100))
    n, m = 256, 96
    W = _random_quantized(rng, n, m, k, zf)
    fh = orc.hac_encode(W)
    kk = len(fh["codebook"])
    assert orc.hac_paper_bits(fh) <= orc.cor1_bound_bits(n, m, kk) + 31      # + word padding
    fs = orc.shac_encode(W, W != 0)
    q = int(fs["cb"][-1])
    assert orc.shac_paper_bits(fs) <= orc.cor2_bound_bits(n, m, q, len(fs["codebook"])) + 31
    # occupancy bounds, Eq. (1) and Eq. (2), are the corollaries divided by b*n*m
    psi_hac = orc.hac_paper_bits(fh) / (32.0 * n * m)
    assert psi_hac <= (1 + np.log2(kk)) / 32 + 6 * kk / (n * m) + 31 / (32.0 * n * m)


def test_two_values_dense_is_one_bit_per_weight():
    # Table III of the paper: k = 2 on a dense matrix gives psi = 0.0313 = 1/32
    rng = np.random.default_rng(3)
    W = np.where(rng.random((128, 64)) < 0.3, np.float32(-0.5), np.float32(0.25)).astype(np.float32)
    fmt = orc.hac_encode(W)
    assert fmt["bits"] == W.size
    assert abs(fmt["bits"] / (32.0 * W.size)- 0.0313) <= 5.001e-5      # the printed value is 1/32 rounded


def test_crossover_formula_consistent_with_bounds():
    n, m, k = 4096, 4096, 32
    s_star = orc.shac_smaller_than_hac_threshold(n, m, k)
    for s in (s_star * 0.98, s_star * 1.02):
        q = int(s * n * m)
        shac_b = orc.cor2_bound_bits(n, m, q, k) - 6 * k * 32
        hac_b = orc.cor1_bound_bits(n, m, k) - 6 * k * 32
        assert (shac_b < hac_b) == (s < s_star)


# ---------------------------------------------------------------- index map and plain CSC (the comparison formats)
def test_index_map_on_the_papers_example_and_its_occupancy():
    W = example2_matrix() if "example2_matrix" in globals() else None
    if W is None:
        from golden_io import golden, read_sections
        g = read_sections(golden("layer_hand_worked.txt"))
        W = np.array([[float(v) for v in row] for row in g["W"]], dtype=np.float32)
    im = orc.index_map_encode(W)
    assert im["codebook"].tolist() == [0, 1, 2, 3, 4, 5, 6, 10] and im["b_bar"] == 8
    assert np.array_equal(orc.index_map_decode(im), W)
    # pi_ij points at the value: row 1 of the example holds 10 in column 1
    assert im["codebook"][im["index"][1, 1]] == 10 and im["index"][3].tolist() == [0] * 5
    # occupancy b_bar / b + k / (n m) (Sect. III-C.1): 8/32 + 8/25 here; about 1/4 for a large matrix with k <= 256
    assert orc.index_map_bits(im) == 8 * 25 + 8 * 32
    big = orc.index_map_encode((np.arange(300 * 200) % 256).reshape(300, 200).astype(np.float32))
    assert abs(orc.index_map_bits(big) / (32.0 * 300 * 200) - (0.25 + 256 / 60000)) < 1e-12
    wide = orc.index_map_encode(np.arange(400, dtype=np.float32).reshape(20, 20))
    assert wide["b_bar"] == 16                              # more than 256 values: two bytes per pointer
    x = np.array([1, 2, 3, 4, 5], dtype=np.float32)
    y, a = orc.dot_index_map(im, x)
    assert y[0].tolist() == [7, 29, 4, 0, 45] and a[0].tolist() == [7, 29, 4, 0, 45]


def test_csc_dot_and_size_on_the_papers_example():
    from golden_io import golden, read_sections
    g = read_sections(golden("layer_hand_worked.txt"))
    W = np.array([[float(v) for v in row] for row in g["W"]], dtype=np.float32)
    nz, ri, cb = orc.csc(W, W != 0)
    assert orc.csc_bits(nz, ri, cb) == (2 * 7 + 5 + 1) * 32       # (2q + m + 1) b, Sect. IV-A
    x = np.array([1, 2, 3, 4, 5], dtype=np.float32)
    y, a = orc.dot_csc(nz, ri, cb, 5, x)
    assert y[0].tolist() == [7, 29, 4, 0, 45]


def test_comparison_formats_agree_with_the_definition():
    rng = np.random.default_rng(21)
    W = rng.standard_normal((60, 17)).astype(np.float32)
    W[np.abs(W) < 0.8] = 0
    W = np.round(W * 4) / 4                                   # few distinct values
    X = rng.standard_normal((3, 60)).astype(np.float32)
    y_ref, a_ref = orc.dot_definition(W, X)
    y, a = orc.dot_index_map(orc.index_map_encode(W), X)
    assert np.array_equal(y, y_ref) and np.array_equal(a, a_ref)
    nz, ri, cb = orc.csc(W, W != 0)
    y, a = orc.dot_csc(nz, ri, cb, 60, X)
    assert np.array_equal(y, y_ref) and np.array_equal(a, a_ref)


# ---------------------------------------------------------------- unified quantization (Sect. V-D)
def _unified_golden():
    from golden_io import golden, read_sections
    g = read_sections(golden("unified_hand_worked.txt"))
    mat = lambda key: np.array([[float(v) for v in row] for row in g[key]], dtype=np.float32)
    ints = lambda key: [[int(v, 0) for v in row] for row in g[key]]
    return g, mat, ints


def test_unified_code_on_the_hand_worked_example():
    g, mat, ints = _unified_golden()
    A, B, Cm = mat("A"), mat("B"), mat("C")
    fmts = orc.unified_encode([("hac", A, A != 0), ("hac", B, B != 0), ("shac", Cm, Cm != 0)])
    for f, bits, word, own in zip(fmts, ints("bits")[0], ints("words")[0], ints("own_counts")):
        assert f["codebook"].tolist() == [float(v) for v in g["codebook"][0]]
        assert f["shared_counts"].tolist() == ints("counts")[0]
        assert f["code_len"].tolist() == ints("lengths")[0] and f["codes"].tolist() == ints("codes")[0]
        assert f["bits"] == bits and f["words"].tolist() == [word] and f["counts"].tolist() == own
    assert fmts[2]["ri"].tolist() == ints("ri")[0] and fmts[2]["cb"].tolist() == ints("cb")[0]
    assert orc.hac_encode(A)["bits"] == ints("A_alone_bits")[0][0]        # its own code would be shorter for A
    assert orc.unified_paper_bits(fmts) == ints("unified_paper_bits")[0][0]
    # every stream decodes back with the shared code
    assert np.array_equal(orc.hac_decode(fmts[0]), A) and np.array_equal(orc.hac_decode(fmts[1]), B)
    assert np.array_equal(orc.shac_decode(fmts[2]), Cm)


def test_unified_of_one_matrix_is_the_ordinary_format():
    rng = np.random.default_rng(3)
    W = rng.standard_normal((40, 12)).astype(np.float32)
    for quantizer in (1, 2, 3, 4):
        (Wq, mask), = orc.quantize_unified([W], 0.5, 8, quantizer, 5, 7)
        Wq1, mask1 = orc.quantize(W, 0.5, 8, quantizer, 5, 7)
        assert np.array_equal(Wq.view(np.uint32), Wq1.view(np.uint32)) and np.array_equal(mask, mask1)
    for kind in ("hac", "shac"):
        u, = orc.unified_encode([(kind, Wq1, mask1)])
        o = orc.hac_encode(Wq1) if kind == "hac" else orc.shac_encode(Wq1, mask1)
        for key in ("codebook", "code_len", "codes", "counts", "words"):
            assert np.array_equal(u[key], o[key]), key
        assert u["bits"] == o["bits"]


def test_unified_over_the_column_halves_of_a_matrix_is_the_matrix():
    """Cutting a matrix between two columns and quantizing the halves together must change nothing: the weights reach the
    sharing in the same order, the counts add up to the same code, and the two streams are the whole stream cut in two."""
    rng = np.random.default_rng(4)
    W = rng.standard_normal((30, 10)).astype(np.float32)
    W[np.abs(W) < 0.4] = 0                                   # already sparse: pruning (per matrix) stays off
    for quantizer in (1, 2, 4):
        whole, mask = orc.quantize(W, 0.0, 6, quantizer, 4, 9)
        (L, mL), (R, mR) = orc.quantize_unified([W[:, :4], W[:, 4:]], 0.0, 6, quantizer, 4, 9)
        assert np.array_equal(np.hstack([L, R]).view(np.uint32), whole.view(np.uint32))
        fw = orc.hac_encode(whole)
        fl, fr = orc.unified_encode([("hac", L, mL), ("hac", R, mR)])
        assert np.array_equal(fl["code_len"], fw["code_len"]) and np.array_equal(fl["codes"], fw["codes"])
        assert np.array_equal(np.concatenate([fl["sym"], fr["sym"]]), fw["sym"]) and fl["bits"] + fr["bits"] == fw["bits"]
        assert np.array_equal(fl["counts"] + fr["counts"], fw["counts"])


def test_unified_sharing_uses_one_set_of_values():
    rng = np.random.default_rng(5)
    Ws = [rng.standard_normal((20, 8)).astype(np.float32), (3 * rng.standard_normal((16, 5))).astype(np.float32)]
    parts = orc.quantize_unified(Ws, 0.25, 4, 1, 10, 1)
    values = np.unique(np.concatenate([Wq[mask] for Wq, mask in parts]))
    assert len(values) <= 4                                   # k values for all matrices together, not per matrix
    for (Wq, mask), W in zip(parts, Ws):
        assert abs((~mask).mean() - 0.25) < 0.02             # each matrix pruned on its own
