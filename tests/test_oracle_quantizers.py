"""Pins of the oracle's lossy steps: magnitude pruning (Sect. III-B), k-means weight
sharing (Sect. III-C.1) and uniform quantization (Sect. III-C.3).

The paper prints no centroid values, so k-means is held by invariants only: the
objective never rises, the assignment is to a nearest centroid, closed forms for
k = 1 and k >= #distinct, and the exact 1-D optimum (dynamic programming) as a
lower bound on tiny inputs."""
import numpy as np
import pytest

from oracle import hac_oracle as orc


# ---------------------------------------------------------------- pruning
@pytest.mark.parametrize("seed", range(6))
def test_prune_brute_force(seed):
    rng = np.random.default_rng(seed)
    n, m = int(rng.integers(2, 9)), int(rng.integers(2, 9))
    W = rng.standard_normal((n, m)).astype(np.float32)
    if seed % 2:
        W = np.round(W * 2) / 2                      # many ties, some zeros
        W = W.astype(np.float32)
    for sparsity in (0.0, 0.1, 0.5, 0.9):
        z = int(np.floor(sparsity * n * m))
        got = orc.prune(W, sparsity)
        if z == 0:
            assert np.array_equal(got, W + np.float32(0.0))
            continue
        ordered = sorted(abs(float(v)) for v in W.ravel())
        tau = ordered[z - 1]
        for i in range(n):
            for j in range(m):
                want = W[i, j] if abs(float(W[i, j])) > tau else 0.0
                assert got[i, j] == want
        zeros = int((got == 0).sum())
        assert zeros >= z
        assert zeros == sum(1 for v in ordered if v <= tau)


def test_prune_rejects_non_finite_and_normalises_minus_zero():
    with pytest.raises(ValueError):
        orc.prune(np.array([[1.0, np.nan]], dtype=np.float32), 0.5)
    out = orc.prune(np.array([[-0.0, 1.0]], dtype=np.float32), 0.0)
    assert not np.signbit(out[0, 0])


def test_prune_hits_target_on_continuous_data():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((200, 100)).astype(np.float32)
    for s in (0.6, 0.9, 0.96, 0.99):
        got = orc.prune(W, s)
        assert abs((got == 0).mean() - s) < 1e-3
        assert np.array_equal(got[got != 0], W[got != 0])           # survivors untouched


# ---------------------------------------------------------------- splitmix64
def test_splitmix64_published_vectors():
    # outputs of the reference generator for seeds 0 and 1234567
    assert [orc.splitmix64(0, i) for i in range(3)] == [
        0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert [orc.splitmix64(1234567, i) for i in range(5)] == [
        6457827717110365317, 3203168211198807973, 9817491932198370423,
        4593380528125082431, 16408922859458223821]


# ---------------------------------------------------------------- k-means
def optimal_sse_1d(values, k):
    """Exact optimum of 1-D k-means by dynamic programming over the sorted data."""
    v = np.sort(np.asarray(values, dtype=np.float64))
    N = len(v)
    pre = np.concatenate(([0.0], np.cumsum(v)))
    pre2 = np.concatenate(([0.0], np.cumsum(v * v)))

    def cost(a, b):            # SSE of v[a:b] around its mean
        s = pre[b] - pre[a]
        return (pre2[b] - pre2[a]) - s * s / (b - a)

    INF = float("inf")
    D = [[INF] * (N + 1) for _ in range(k + 1)]
    D[0][0] = 0.0
    for c in range(1, k + 1):
        for b in range(c, N + 1):
            D[c][b] = min(D[c - 1][a] + cost(a, b) for a in range(c - 1, b))
    return D[k][N]


@pytest.mark.parametrize("seed", range(5))
def test_kmeans_invariants(seed):
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((40, 30)).astype(np.float32)
    Wp = orc.prune(W, 0.5)
    k = 8
    Wq, mask, c, sse = orc.kmeans_share(Wp, k, 20, seed=seed, return_trace=True)
    assert np.array_equal(mask, Wp != 0)
    assert np.all(Wq[~mask] == 0)
    assert np.all(np.diff(c) >= 0)                                   # centroids sorted
    assert np.all(np.diff(sse) <= 1e-12 * sse[0])                    # Lloyd never raises the SSE
    data = Wp[mask].astype(np.float64)
    assigned = Wq[mask].astype(np.float64)
    c32 = c.astype(np.float32).astype(np.float64)
    # each weight sits at a nearest centroid (up to the fp32 rounding of the centroid)
    dist_assigned = np.abs(data - assigned)
    dist_best = np.abs(data[:, None] - c[None, :]).min(axis=1)
    assert np.all(dist_assigned <= dist_best + 1e-6)
    assert set(np.unique(assigned)) <= set(c32)
    assert len(np.unique(Wq[mask])) <= k


def test_kmeans_at_least_exact_optimum_and_close():
    rng = np.random.default_rng(42)
    data = np.concatenate([rng.normal(-2, 0.1, 15), rng.normal(0.5, 0.1, 15), rng.normal(3, 0.1, 15)])
    W = data.astype(np.float32).reshape(9, 5)
    for k in (2, 3, 4):
        _, _, c, sse = orc.kmeans_share(W, k, 20, seed=7, return_trace=True)
        best = optimal_sse_1d(W.ravel().astype(np.float64), k)
        assert sse[-1] >= best - 1e-9
    # three well separated blobs and k = 3: a start with one centroid per blob is a fixed point
    # at the optimum, and among 20 seeded starts at least one is of that kind
    best3 = optimal_sse_1d(W.ravel().astype(np.float64), 3)
    finals = [orc.kmeans_share(W, 3, 20, seed=s, return_trace=True)[3][-1] for s in range(20)]
    assert min(finals) <= best3 * (1 + 1e-9)


def test_kmeans_closed_forms():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((12, 11)).astype(np.float32)
    # k = 1: the mean, accumulated in column-major order in fp64
    Wq, mask, c, _ = orc.kmeans_share(W, 1, 20, seed=0, return_trace=True)
    s = 0.0
    for v in W.T.ravel():
        s += float(v)
    assert c[0] == s / W.size
    assert np.all(Wq == np.float32(c[0]))
    # k >= number of distinct values: the data is its own codebook
    Wd = np.round(W * 2).astype(np.float32) / 2
    Wd[Wd == 0] = 0.5
    Wq, _ = orc.kmeans_share(Wd, 64, 20, seed=0)
    assert np.array_equal(Wq, Wd)


def test_kmeans_matches_a_python_restatement_in_storage_order():
    """Plain-Python Lloyd with the same rules on a tiny case: fixes summation order (column-major)
    and the tie rule, which decide the bits of the centroids."""
    rng = np.random.default_rng(8)
    W = (rng.integers(-6, 7, size=(9, 7)) / 4.0).astype(np.float32)
    W[W == 0] = 0.25
    k, iters, seed = 4, 5, 99
    _, _, c_got, _ = orc.kmeans_share(W, k, iters, seed=seed, return_trace=True)
    data = [float(v) for v in W.T.ravel()]
    u = sorted(set(data))
    idx = list(range(len(u)))
    for i in range(k):
        j = i + orc.splitmix64(seed, i) % (len(u) - i)
        idx[i], idx[j] = idx[j], idx[i]
    c = sorted(u[i] for i in idx[:k])
    for _ in range(iters):
        t = [(c[l] + c[l + 1]) * 0.5 for l in range(k - 1)]
        sums, cnts = [0.0] * k, [0] * k
        for w in data:
            l = sum(1 for tt in t if tt < w)
            sums[l] += w
            cnts[l] += 1
        c = sorted(sums[l] / cnts[l] if cnts[l] else c[l] for l in range(k))
    assert c_got.tolist() == c


# ---------------------------------------------------------------- uniform
@pytest.mark.parametrize("k", [2, 5, 16, 256])
def test_uniform_closed_form(k):
    rng = np.random.default_rng(k)
    W = rng.standard_normal((64, 48)).astype(np.float32)
    Wq, mask = orc.uniform_share(W, k)
    lo, hi = float(W.min()), float(W.max())
    delta = (hi - lo) / (k - 1)
    err = np.abs(Wq.astype(np.float64) - W.astype(np.float64))
    assert err.max() <= delta / 2 + np.spacing(np.float32(max(abs(lo), abs(hi))))
    assert len(np.unique(Wq)) <= k
    assert Wq.min() == W.min() and Wq.max() == W.max()              # the ends are levels
    levels = (Wq.astype(np.float64) - lo) / delta
    assert np.abs(levels - np.round(levels)).max() < 1e-4           # values lie on the grid


def test_uniform_on_pruned_matrix_keeps_zeros():
    rng = np.random.default_rng(2)
    W = rng.standard_normal((50, 40)).astype(np.float32)
    Wp = orc.prune(W, 0.8)
    Wq, mask = orc.uniform_share(Wp, 16)
    assert np.array_equal(mask, Wp != 0)
    assert np.all(Wq[~mask] == 0)
    assert Wq[mask].min() == Wp[mask].min() and Wq[mask].max() == Wp[mask].max()


# ---------------------------------------------------------------- zero-anchored grid (Sect. III-C.3 as printed, d = 0)
def test_grid_levels_round_half_up_on_a_hand_example():
    data = np.array([0.26, -0.26, 0.74, 0.75, -0.75, 1.0, 0.24, -0.25])
    # w / 0.5 = 0.52 -0.52 1.48 1.5 -1.5 2.0 0.48 -0.5 ; nearest integer, halves upwards
    assert orc.grid_levels(data, 0.5).tolist() == [1, -1, 1, 2, -1, 2, 0, 0]


@pytest.mark.parametrize("k", [2, 3, 16, 256])
def test_grid_share_invariants(k):
    rng = np.random.default_rng(100 + k)
    W = rng.standard_normal((96, 40)).astype(np.float32)
    Wq, mask = orc.grid_share(W, k)
    data = W.T[mask.T].astype(np.float64)
    delta = orc.grid_delta(data, k)
    assert mask.all() and len(np.unique(Wq)) <= k
    levels = Wq.astype(np.float64) / delta
    assert np.abs(levels - np.round(levels)).max() < 1e-4                 # multiples of delta: the grid passes through 0
    err = np.abs(Wq.astype(np.float64) - W.astype(np.float64))
    assert err.max() <= delta / 2 + np.spacing(np.float32(np.abs(W).max()))
    # delta is tuned: the next smaller double already leaves more than k values
    assert len(np.unique(orc.grid_levels(data, delta))) <= k
    assert len(np.unique(orc.grid_levels(data, np.nextafter(delta, 0.0)))) > k
    # and it sits where some weight crosses a rounding boundary: delta = |w| / (t - 1/2), t = 1, 2, ..
    t = np.round(np.abs(data) / delta + 0.5)
    t = t[t >= 1]
    cand = np.abs(data)[np.round(np.abs(data) / delta + 0.5) >= 1] / (t - 0.5)
    assert np.min(np.abs(cand - delta)) <= 4 * np.spacing(delta)


def test_grid_share_small_weights_become_stored_zeros_and_symmetry_holds():
    rng = np.random.default_rng(7)
    half = rng.standard_normal(300).astype(np.float32)
    W = np.concatenate([half, -half]).reshape(20, 30)
    Wp = orc.prune(W, 0.25)
    Wq, mask = orc.grid_share(Wp, 5)
    assert np.array_equal(mask, Wp != 0)
    assert np.all(Wq[~mask] == 0)
    assert np.any((Wq == 0) & mask)                     # survivors below delta/2 round to 0 but stay stored entries
    assert np.array_equal(np.unique(Wq), -np.unique(Wq)[::-1])
    # few distinct values: kept as they are
    V = np.array([[0.5, -1.25, 0.0], [3.0, 0.5, 3.0]], dtype=np.float32)
    Vq, vm = orc.grid_share(V, 4)
    assert np.array_equal(Vq, V) and np.array_equal(vm, V != 0)


# ---------------------------------------------------------------- PWS (Sect. III-C.2)
def test_splitmix64_many_equals_the_scalar_generator():
    for seed in (0, 1234567, (1 << 64) - 5):
        assert orc.splitmix64_many(seed, 50).tolist() == [orc.splitmix64(seed, i) for i in range(50)]


def test_pws_two_values_is_the_two_point_law_of_the_paper():
    # k = 2: every weight becomes min or max, the maximum with probability (w - min) / (max - min)
    rng = np.random.default_rng(11)
    W = rng.uniform(-1.0, 3.0, size=(30, 20)).astype(np.float32)
    lo, hi = np.float64(W.min()), np.float64(W.max())
    ups = np.zeros(W.shape)
    trials = 400
    for seed in range(trials):
        Wq, mask = orc.pws_share(W, 2, seed)
        assert set(np.unique(Wq).tolist()) <= {float(W.min()), float(W.max())}
        ups += Wq == W.max()
    p = (W.astype(np.float64) - lo) / (hi - lo)
    # frequencies within 5 standard deviations of the law, and the estimate is unbiased on average
    assert np.all(np.abs(ups / trials - p) <= 5 * np.sqrt(p * (1 - p) / trials) + 1e-12)
    est = lo + (hi - lo) * ups / trials
    assert abs(float((est - W).mean())) < 5 * (hi - lo) * 0.5 / np.sqrt(trials * W.size)


@pytest.mark.parametrize("k", [3, 8, 64])
def test_pws_values_bracket_the_weight_and_representatives_are_quantiles(k):
    rng = np.random.default_rng(k)
    W = rng.standard_normal((120, 50)).astype(np.float32)
    Wq, mask = orc.pws_share(W, k, seed=5)
    data = np.sort(W.ravel().astype(np.float64))
    q = data.size
    ext = np.unique([data[(i * (q - 1)) // (k - 1)] for i in range(k)])
    assert ext[0] == data[0] and ext[-1] == data[-1] and len(ext) <= k
    assert np.array_equal(orc.pws_extremes(W.T.ravel().astype(np.float64), k), ext)
    assert set(np.unique(Wq).tolist()) <= set(ext.astype(np.float32).tolist())
    # the two neighbours of w among the representatives, by brute force
    w64, q64 = W.astype(np.float64).ravel(), Wq.astype(np.float64).ravel()
    for w, v in zip(w64[::37], q64[::37]):
        below = ext[ext <= w].max()
        above = ext[ext > w].min() if (ext > w).any() else ext[-1]
        assert np.float32(v) in (np.float32(below), np.float32(above))
    # a representative is reproduced exactly
    hit = np.isin(w64, ext)
    assert np.array_equal(q64[hit].astype(np.float32), w64[hit].astype(np.float32))
    # the intervals between neighbouring representatives hold equal shares of the weights
    shares = np.array([((data >= a) & (data < b)).sum() for a, b in zip(ext[:-1], ext[1:])])
    assert np.all(np.abs(shares - (q - 1) / (k - 1)) <= 1.0)
    # same seed, same result; another seed, another draw
    assert np.array_equal(orc.pws_share(W, k, seed=5)[0], Wq)
    assert not np.array_equal(orc.pws_share(W, k, seed=6)[0], Wq)


def test_pws_with_256_values_codes_at_8_bits_like_the_papers_table():
    # equiprobable representatives: Huffman lengths close to log2 k, the occupancy 0.2500 = 8/32 the paper
    # reports for PWS at k = 256 on dense layers
    rng = np.random.default_rng(3)
    W = rng.standard_normal((512, 256)).astype(np.float32)
    Wq, mask = orc.pws_share(W, 256, seed=1)
    fmt = orc.hac_encode(Wq)
    assert 7.9 <= fmt["bits"] / W.size <= 8.05


# ---------------------------------------------------------------- k-means against a hand-worked example
def test_kmeans_two_iterations_worked_by_hand():
    """Pins the Lloyd rule itself (midpoint assignment, a weight on a midpoint goes down, mean update,
    exactly `iters` updates and one more assignment) against tests/golden/kmeans_hand_worked.txt,
    whose numbers were derived on paper as exact fractions."""
    from fractions import Fraction
    from golden_io import golden, read_sections
    g = read_sections(golden("kmeans_hand_worked.txt"))
    data = np.array([float(v) for v in g["data"][0]], dtype=np.float32)
    k, seed = int(g["k"][0][0]), int(g["seed"][0][0])
    start = [float(v) for v in g["start"][0]]
    assert orc.kmeans_init(np.unique(data.astype(np.float64)), k, seed).tolist() == start
    W = data.reshape(-1, 1)
    sse_want = [float(Fraction(v)) for v in g["sse"][0]]
    for iters in (1, 2):
        want_c = [Fraction(v) for v in g[f"centroids_after_{iters}"][0]]
        want_a = [int(v) for v in g[f"assign_iters_{iters}"][0]]
        Wq, mask, c, sse = orc.kmeans_share(W, k, iters, seed, return_trace=True)
        assert mask.all()
        # the centroids are the fractions rounded once to double
        assert c.tolist() == [float(f) for f in want_c]
        want_values = np.array([np.float32(float(want_c[a])) for a in want_a], dtype=np.float32)
        assert np.array_equal(Wq.ravel().view(np.uint32), want_values.view(np.uint32))
        assert np.allclose(sse[:iters + 1], sse_want[:iters + 1], rtol=1e-12, atol=0)
