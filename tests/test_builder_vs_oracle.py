"""The library's host builder against the oracle: every array of the formats bit for bit
(codebook, code lengths, codes, stream words, ri, cb, offset index), on the same seeded
inputs.  No GPU needed: only host entry points of the C ABI are called."""
import dataclasses

import numpy as np
import pytest

import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb


def oracle_format(W, wl, kind):
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    fmt = orc.hac_encode(Wq) if kind == "hac" else orc.shac_encode(Wq, mask)
    return Wq, mask, fmt


def library_format(W, wl, kind, S=0, ri_bits=0):
    return hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer,
                     kmeans_iters=wl.kmeans_iters, seed=wl.seed, seg_symbols=S, ri_bits=ri_bits)


def assert_same_format(lib_fmt, ofmt, oidx, Wq):
    e = lib_fmt.export()
    assert np.array_equal(e["codebook"].view(np.uint32), ofmt["codebook"].view(np.uint32))
    assert np.array_equal(e["code_len"], ofmt["code_len"])
    assert np.array_equal(e["codes"], ofmt["codes"])
    assert np.array_equal(e["counts"], ofmt["counts"])
    assert e["stream_bits"] == ofmt["bits"]
    N = len(ofmt["words"])
    assert e["stream_words"] == N
    assert np.array_equal(e["stream"][:N], ofmt["words"])
    assert not e["stream"][N:].any() and e["stream_pad_words"] >= 4 and len(e["stream"]) % 4 == 0
    assert np.array_equal(e["seg_bit_off"], oidx["seg_bit_off"])
    assert np.array_equal(e["sub_bits"], oidx["sub_bits"])
    if lib_fmt.kind == "shac":
        assert np.array_equal(e["ri"].astype(np.int64), ofmt["ri"].astype(np.int64))
        assert np.array_equal(e["cb"].astype(np.int64), ofmt["cb"])
        assert np.array_equal(e["seg_first"], oidx["seg_first"])
        assert np.array_equal(e["seg_col"], oidx["seg_col"])
    else:
        assert e["segs_per_col"] == oidx["G"]
    assert np.array_equal(lib_fmt.decode_host().view(np.uint32), Wq.view(np.uint32))
    return e


CASES = [
    (si.CFG1_TINY_SHAC, "shac", 0),
    (si.CFG1_TINY_SHAC, "hac", 0),
    (si.scaled(si.CFG2_DENSE_HAC, 300, 70), "hac", 0),
    (si.scaled(si.CFG2_DENSE_HAC, 2100, 37), "hac", 64),      # two segments per column, ragged tail
    (si.scaled(si.CFG3_FC_SHAC, 3000, 96), "shac", 0),
    (si.scaled(si.CFG3_FC_SHAC, 3000, 96), "shac", 3),        # several segments per column
    (si.scaled(si.CFG4_CONV, 460, 64), "shac", 0),
    (si.scaled(si.CFG4_CONV, 460, 64), "hac", 16),
    (dataclasses.replace(si.scaled(si.CFG2_DENSE_HAC, 300, 70), quantizer=si.QUANT_GRID, k=64), "hac", 0),
    (dataclasses.replace(si.scaled(si.CFG3_FC_SHAC, 3000, 96), quantizer=si.QUANT_GRID, k=9), "shac", 0),
    (dataclasses.replace(si.scaled(si.CFG4_CONV, 460, 64), quantizer=si.QUANT_GRID, k=2), "hac", 16),
    (dataclasses.replace(si.scaled(si.CFG2_DENSE_HAC, 300, 70), quantizer=si.QUANT_PWS, k=64), "hac", 0),
    (dataclasses.replace(si.scaled(si.CFG3_FC_SHAC, 3000, 96), quantizer=si.QUANT_PWS, k=2), "shac", 0),
    (dataclasses.replace(si.scaled(si.CFG4_CONV, 460, 64), quantizer=si.QUANT_PWS, k=17), "shac", 5),
]


@pytest.mark.parametrize("wl,kind,S", CASES, ids=[f"{c[0].name}-{c[1]}-S{c[2]}" for c in CASES])
def test_formats_bit_exact(wl, kind, S):
    W = si.weights(wl)
    Wq, mask, ofmt = oracle_format(W, wl, kind)
    lf = library_format(W, wl, kind, S)
    S_eff = lf.sizes()["seg_symbols"]
    assert S_eff == S or (S == 0 and (S_eff == 64 if kind == "hac" else S_eff % 4 == 2))
    oidx = orc.hac_offset_index(ofmt, S_eff) if kind == "hac" else orc.shac_offset_index(ofmt, S_eff)
    assert_same_format(lf, ofmt, oidx, Wq)


@pytest.mark.parametrize("k", [2, 8, 1024])
@pytest.mark.parametrize("sp", [0.0, 0.9, 0.99])
def test_sweep_cells_small(k, sp):
    wl = dataclasses.replace(si.sweep_cells(192, 160)[0], sparsity=sp, k=k)
    W = si.weights(wl)
    for kind in ("hac", "shac"):
        Wq, mask, ofmt = oracle_format(W, wl, kind)
        lf = library_format(W, wl, kind)
        S_eff = lf.sizes()["seg_symbols"]
        oidx = orc.hac_offset_index(ofmt, S_eff) if kind == "hac" else orc.shac_offset_index(ofmt, S_eff)
        assert_same_format(lf, ofmt, oidx, Wq)


def test_sizes_report_matches_oracle_accounting():
    wl = si.scaled(si.CFG4_CONV, 460, 64)
    W = si.weights(wl)
    for kind in ("hac", "shac"):
        Wq, mask, ofmt = oracle_format(W, wl, kind)
        r = library_format(W, wl, kind).sizes()
        if kind == "hac":
            assert r["paper_bits"] == orc.hac_paper_bits(ofmt)
            assert r["bound_bits"] == pytest.approx(orc.cor1_bound_bits(wl.n, wl.m, len(ofmt["codebook"])), rel=1e-12)
        else:
            q = int(ofmt["cb"][-1])
            assert r["nnz"] == q
            assert r["paper_bits"] == orc.shac_paper_bits(ofmt)
            assert r["bound_bits"] == pytest.approx(orc.cor2_bound_bits(wl.n, wl.m, q, len(ofmt["codebook"])), rel=1e-12)
        assert r["paper_bits"] <= r["bound_bits"] + 31
        assert r["entropy"] <= r["avg_code_len"] <= r["entropy"] + 1
        assert r["total_bytes"] == (r["stream_bytes"] + r["pad_bytes"] + r["codebook_bytes"] + r["code_len_bytes"]
                                    + r["ri_bytes"] + r["cb_bytes"] + r["offset_index_bytes"])
        assert r["offset_index_bytes"] > 0


def test_quantizer_none_and_special_inputs():
    W = np.array([[1, 0, 4, 0, 0], [0, 10, 0, 0, 0], [2, 3, 0, 0, 5], [0, 0, 0, 0, 0], [0, 0, 0, 0, 6]],
                 dtype=np.float32)                                   # Example 2 of the paper
    lf = hb.Format("hac", W, quantizer=hb.QUANT_NONE, seg_symbols=5)
    e = lf.export()
    assert [f"{w:08X}" for w in e["stream"][:2]] == ["A5898680", "0E780000"]
    assert e["seg_bit_off"].tolist() == [0, 11, 21, 29, 34]
    ls = hb.Format("shac", W, quantizer=hb.QUANT_NONE)
    es = ls.export()
    assert f"{es['stream'][0]:08X}" == "4C977000"
    assert (es["ri"] + 1).tolist() == [1, 3, 2, 3, 1, 3, 5] and (es["cb"] + 1).tolist() == [1, 3, 5, 6, 6, 8]
    # all-zero matrix, single value, errors
    Z = np.zeros((4, 3), dtype=np.float32)
    assert hb.Format("shac", Z, quantizer=hb.QUANT_NONE).sizes()["nnz"] == 0
    assert hb.Format("hac", Z, quantizer=hb.QUANT_NONE).sizes()["stream_bits"] == 12
    with pytest.raises(hb.HacError) as ei:
        hb.Format("hac", np.array([[np.inf, 1.0]], dtype=np.float32), quantizer=hb.QUANT_NONE)
    assert ei.value.status == -3
    with pytest.raises(hb.HacError) as ei:
        hb.Format("hac", np.arange(5000, dtype=np.float32).reshape(50, 100) + 1, quantizer=hb.QUANT_NONE)
    assert ei.value.status == -4
    with pytest.raises(hb.HacError) as ei:
        hb.Format("hac", W, sparsity=1.5)
    assert ei.value.status == -1


def test_library_exports_every_declared_symbol():
    import re, os
    header = open(os.path.join(os.path.dirname(__file__), "..", "include", "hac.h")).read()
    declared = set(re.findall(r"\b(s?hac_[a-z_]+)\s*\(", header))
    declared -= {"hac_build_params"}
    lib = hb.load()
    assert declared == set(hb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_device_calls_fail_loudly_without_upload():
    W = si.weights(si.CFG1_TINY_SHAC)
    lf = hb.Format("shac", W, sparsity=0.9, k=8, kmeans_iters=2)
    lib = hb.load()
    rc = lib.shac_dot(lf._h, 16, 1, 1, 0, 16, 1, 0, None, 0, None)
    assert rc == -7          # HAC_ERR_NOT_UPLOADED: no silent fallback


def test_library_kmeans_on_the_hand_worked_example():
    """The library's own k-means reproduces the centroids of tests/golden/kmeans_hand_worked.txt."""
    from fractions import Fraction
    from golden_io import golden, read_sections
    g = read_sections(golden("kmeans_hand_worked.txt"))
    W = np.array([float(v) for v in g["data"][0]], dtype=np.float32).reshape(-1, 1)
    k, seed = int(g["k"][0][0]), int(g["seed"][0][0])
    for iters in (1, 2):
        want = sorted({np.float32(float(Fraction(v))) for v in g[f"centroids_after_{iters}"][0]})
        for kind in ("hac", "shac"):
            f = hb.Format(kind, W, sparsity=0.0, k=k, quantizer=si.QUANT_KMEANS, kmeans_iters=iters, seed=seed)
            assert f.export()["codebook"].tolist() == [float(v) for v in want]


def _geometric_matrix(rng, k, ratio, n=600, m=40):
    p = ratio ** np.arange(k)
    p /= p.sum()
    values = np.sort(rng.standard_normal(k).astype(np.float32))
    W = values[rng.choice(k, size=(n, m), p=p)].astype(np.float32)
    W.ravel()[:k] = values                                   # every value occurs
    return W


@pytest.mark.parametrize("k,ratio", [(22, 0.5), (60, 0.8), (200, 0.95), (247, 0.985), (8, 0.3), (33, 1.0)])
def test_first_level_table_of_the_kernels_decodes_every_window(k, ratio):
    """The table the kernels look code words up in (indexed by leading bits, or by the magnitude of the
    inverted window when code words are long) must give, for every code word followed by any bits,
    that code word's value and length, or say that it leaves it to the slower levels; where the kernels
    rely on it resolving everything, it must."""
    rng = np.random.default_rng(k)
    W = _geometric_matrix(rng, k, ratio)
    for kind in ("hac", "shac"):
        f = hb.Format(kind, W, sparsity=0.0, k=k, quantizer=si.QUANT_NONE)
        e = f.export()
        kinds = set()
        for s in range(e["k_eff"]):
            L = int(e["code_len"][s]); code = int(e["codes"][s])
            tails = [0, (1 << (32 - L)) - 1] + [int(t) for t in rng.integers(0, 1 << (32 - L), size=40)] if L < 32 else [0]
            for t in tails:
                window = (code << (32 - L)) | t
                value, length, tk, never = f.debug_table_lookup(window)
                kinds.add(tk)
                if length == 0:
                    assert not never, "an unresolved window in a table the kernels treat as complete"
                else:
                    assert length == L and np.float32(value) == e["codebook"][s]
        assert len(kinds) == 1


def test_long_tailed_code_takes_the_magnitude_table():
    rng = np.random.default_rng(3)
    f = hb.Format("hac", _geometric_matrix(rng, 40, 0.6, n=3000), sparsity=0.0, k=40, quantizer=si.QUANT_NONE)
    assert f.sizes()["max_code_len"] > 12
    assert f.debug_table_lookup(0)[2] == 1


# ---------------------------------------------------------------- serialization
def _same_arrays(a, b):
    assert a.keys() == b.keys()
    for k in a:
        if isinstance(a[k], np.ndarray):
            assert a[k].dtype == b[k].dtype and np.array_equal(a[k], b[k]), k
        else:
            assert a[k] == b[k], k


@pytest.mark.parametrize("kind", ["hac", "shac"])
def test_serialize_round_trip_and_rejection_of_altered_strings(kind):
    wl = si.scaled(si.CFG3_FC_SHAC, 700, 60)
    W = si.weights(wl)
    f = hb.Format(kind, W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, kmeans_iters=wl.kmeans_iters, seed=wl.seed)
    blob = f.serialize()
    g = hb.Format.deserialize(kind, blob)
    _same_arrays(f.export(), g.export())
    assert f.sizes() == g.sizes()
    assert np.array_equal(f.decode_host().view(np.uint32), g.decode_host().view(np.uint32))
    assert g.serialize() == blob
    for kk in ("xt", "l1"):
        pass
    # same tables: the first-level entry of a few windows
    for w in (0, 0x12345678, 0xffffffff, 0x80000000):
        assert f.debug_table_lookup(w) == g.debug_table_lookup(w)
    # every single flipped bit and every truncation is refused (checked on a sample of positions)
    rng = np.random.default_rng(1)
    positions = sorted(set([0, 8, 17, 100, 128, len(blob) - 9, len(blob) - 1] + rng.integers(0, len(blob), size=60).tolist()))
    for pos in positions:
        bad = bytearray(blob)
        bad[pos] ^= 1 << int(rng.integers(0, 8))
        with pytest.raises(hb.HacError) as ei:
            hb.Format.deserialize(kind, bytes(bad))
        assert ei.value.status == -10, pos
    for cut in (0, 7, 127, 136, len(blob) - 8, len(blob) - 1):
        with pytest.raises(hb.HacError) as ei:
            hb.Format.deserialize(kind, blob[:cut])
        assert ei.value.status == -10
    with pytest.raises(hb.HacError) as ei:
        hb.Format.deserialize("shac" if kind == "hac" else "hac", blob)
    assert ei.value.status == -1


def test_deserialize_checks_the_contents_not_only_the_checksum():
    """A string whose checksum was recomputed after tampering is still refused when its code or its index
    is not valid."""
    def fnv1a(b):
        h = 0xcbf29ce484222325
        for x in b:
            h = ((h ^ x) * 0x100000001b3) & 0xffffffffffffffff
        return h
    W = si.weights(si.scaled(si.CFG2_DENSE_HAC, 300, 20))
    f = hb.Format("hac", W, sparsity=0.0, k=16, quantizer=si.QUANT_UNIFORM)
    blob = bytearray(f.serialize())
    k = f.sizes()["k_eff"]
    def resealed(b):
        b = bytearray(b)
        b[-8:] = fnv1a(bytes(b[:-8])).to_bytes(8, "little")
        return bytes(b)
    hb.Format.deserialize("hac", resealed(blob))                       # untouched and resealed: accepted
    off_len = 128 + ((4 * k + 7) // 8) * 8                               # code lengths follow the codebook
    bad = bytearray(blob); bad[off_len] += 1                            # breaks the Kraft equality
    with pytest.raises(hb.HacError) as ei:
        hb.Format.deserialize("hac", resealed(bad))
    assert ei.value.status == -10
    bad = bytearray(blob); bad[128:132], bad[132:136] = blob[132:136], blob[128:132]      # codebook not ascending
    with pytest.raises(hb.HacError) as ei:
        hb.Format.deserialize("hac", resealed(bad))
    assert ei.value.status == -10


# ---------------------------------------------------------------- the comparison formats' encoders (host only)
def test_index_map_and_csc_encoders_against_the_oracle():
    from paper_2108_12704_b200.binding import IndexMap, Csc
    wl = si.scaled(si.CFG3_FC_SHAC, 300, 37)
    W = si.weights(wl)
    Wq, mask = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    ref = orc.index_map_encode(Wq)
    im = IndexMap(Wq, 8)
    assert im.k == len(ref["codebook"]) and np.array_equal(im.codebook.view(np.uint32), ref["codebook"].view(np.uint32))
    assert np.array_equal(im.index.reshape(wl.m, wl.n), ref["index"].T)             # column-major pointers
    assert abs(im.psi() - orc.index_map_bits(ref) / (32.0 * wl.n * wl.m)) < 1e-12
    im16 = IndexMap(Wq, 16)
    assert im16.index.dtype == np.uint16 and np.array_equal(im16.index.reshape(wl.m, wl.n), ref["index"].T)
    nz, ri, cb = orc.csc(Wq, Wq != 0)
    c = Csc(Wq)
    assert c.q == len(nz) and np.array_equal(c.nz.view(np.uint32), np.asarray(nz, np.float32).view(np.uint32))
    assert np.array_equal(c.ri.astype(np.int64), np.asarray(ri, np.int64)) and np.array_equal(c.cb.astype(np.int64), cb)
    assert abs(c.psi() - orc.csc_bits(nz, ri, cb) / (32.0 * wl.n * wl.m)) < 1e-12


def test_comparison_encoders_reject_bad_input():
    from paper_2108_12704_b200.binding import IndexMap, Csc
    many = np.arange(300, dtype=np.float32).reshape(20, 15)
    with pytest.raises(hb.HacError) as e:
        IndexMap(many, 8)                                    # 300 values do not fit one byte
    assert e.value.status == -4
    assert IndexMap(many, 16).k == 300
    bad = many.copy(); bad[3, 3] = np.nan
    for cls in (lambda w: IndexMap(w, 8), Csc):
        with pytest.raises(hb.HacError) as e:
            cls(bad)
        assert e.value.status == -3
    z = Csc(np.zeros((4, 3), dtype=np.float32))
    assert z.q == 0 and z.cb.tolist() == [0, 0, 0, 0]
    neg = IndexMap(np.array([[-0.0, 0.0], [1.0, 0.0]], dtype=np.float32), 8)
    assert neg.k == 2                                        # -0.0 and 0.0 are one value


# ---------------------------------------------------------------- unified quantization (Sect. V-D)
@pytest.mark.parametrize("quantizer,k", [(si.QUANT_KMEANS, 12), (si.QUANT_UNIFORM, 40), (si.QUANT_PWS, 9), (si.QUANT_GRID, 16)])
def test_unified_build_bit_exact(quantizer, k):
    """Three matrices of different shapes, HAC and sHAC mixed, quantized together: every array of every format against
    the oracle, and every format usable on its own (host decode, serialization)."""
    shapes = [("hac", si.scaled(si.CFG2_DENSE_HAC, 300, 40)), ("shac", si.scaled(si.CFG3_FC_SHAC, 900, 30)),
              ("hac", si.scaled(si.CFG4_CONV, 200, 10))]
    Ws = [si.weights(wl) for _, wl in shapes]
    sparsity, iters, seed = 0.7, 6, 11
    parts = orc.quantize_unified(Ws, sparsity, k, quantizer, iters, seed)
    ofmts = orc.unified_encode([(kind, Wq, mask) for (kind, _), (Wq, mask) in zip(shapes, parts)])
    lfs = hb.hac_build_unified([(kind, W) for (kind, _), W in zip(shapes, Ws)], sparsity=sparsity, k=k, quantizer=quantizer,
                               kmeans_iters=iters, seed=seed)
    for lf, ofmt, (Wq, mask) in zip(lfs, ofmts, parts):
        S_eff = lf.sizes()["seg_symbols"]
        oidx = orc.hac_offset_index(ofmt, S_eff) if lf.kind == "hac" else orc.shac_offset_index(ofmt, S_eff)
        assert_same_format(lf, ofmt, oidx, Wq)
        back = hb.Format.deserialize(lf.kind, lf.serialize())
        assert np.array_equal(back.decode_host().view(np.uint32), Wq.view(np.uint32))
    # the dictionary is one for all: the same codebook and code in every format
    e = [lf.export() for lf in lfs]
    assert all(np.array_equal(x["codebook"], e[0]["codebook"]) and np.array_equal(x["codes"], e[0]["codes"]) for x in e)
    total = sum(x["counts"] for x in e)
    assert np.array_equal(total, ofmts[0]["shared_counts"]) and (total > 0).all()


def test_unified_build_on_the_hand_worked_example_and_bad_arguments():
    from golden_io import golden, read_sections
    g = read_sections(golden("unified_hand_worked.txt"))
    mat = lambda key: np.array([[float(v) for v in row] for row in g[key]], dtype=np.float32)
    lfs = hb.hac_build_unified([("hac", mat("A")), ("hac", mat("B")), ("shac", mat("C"))], quantizer=si.QUANT_NONE)
    words = [int(v, 0) for v in g["words"][0]]
    for lf, word, bits, own in zip(lfs, words, g["bits"][0], g["own_counts"]):
        e = lf.export()
        assert e["stream"][0] == word and e["stream_bits"] == int(bits) and e["counts"].tolist() == [int(v) for v in own]
        assert e["code_len"].tolist() == [int(v) for v in g["lengths"][0]]
    one = hb.hac_build_unified([("hac", mat("A"))], quantizer=si.QUANT_NONE)[0].export()
    assert one["stream_bits"] == int(g["A_alone_bits"][0][0])
    with pytest.raises(hb.HacError):
        hb.hac_build_unified([], quantizer=si.QUANT_NONE)
    bad = mat("A").copy(); bad[0, 0] = np.inf
    with pytest.raises(hb.HacError) as err:
        hb.hac_build_unified([("hac", mat("B")), ("hac", bad)], quantizer=si.QUANT_NONE)
    assert err.value.status == -3
