"""CPU oracle for the HAC / sHAC formats and their compressed-domain product.

TEST INFRASTRUCTURE ONLY: the slow, plain fp64 reference that the CUDA library
is compared with.  It shares no code with that library; only tests, the smoke
check and the CPU-baseline leg of the benchmark may import it.

Each function states the passage of the paper it follows (Marino, Petrini,
Malchiodi, Frasca, "Compact representations of convolutional neural networks
via weight pruning and quantization").  Where the paper leaves a choice open
(ties, initialisation, bit order, which optimal Huffman code) the rule taken is
written in the docstring.  The loops that would be too slow in Python live in
hac_oracle.c (k-means sweeps, bit-by-bit packing, Algorithms 1-3).

Parity unpinned: `kmeans_share` has no value printed by the paper to compare
with; it is held by invariants only (see tests/test_oracle_quantizers.py).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from collections import deque

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hac_oracle.c")
_LIB = os.path.join(_HERE, "libhac_oracle.so")

B_WORD = 32          # b: bits of one memory word (FP32 weights), Sect. IV-A
MAX_SYMBOLS = 2048   # larger alphabets are rejected by both implementations


def build_native(force: bool = False) -> str:
    """Compile hac_oracle.c with gcc (plain C, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                               "-fno-fast-math", "-pthread", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _native():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build_native())
        _lib.orc_pack.restype = ctypes.c_int64
        _lib.orc_decode.restype = ctypes.c_int64
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


# ----------------------------------------------------------------------------
# Sect. III-B  weight pruning
# ----------------------------------------------------------------------------
def prune(W: np.ndarray, sparsity: float) -> np.ndarray:
    """Magnitude pruning (Sect. III-B): fix a percentile w_p of the magnitudes
    and keep w only where |w| > w_p.

    Reading: z = floor(sparsity * n*m) entries are to go; w_p is the z-th
    smallest magnitude itself (an order statistic, no interpolation); every
    entry with |w| <= w_p becomes 0, so ties at w_p are all pruned.  z = 0
    leaves W unchanged.  Non-finite inputs are rejected; -0.0 becomes +0.0.
    """
    W = np.asarray(W, dtype=np.float32)
    if not np.all(np.isfinite(W)):
        raise ValueError("non-finite weight")
    out = W.copy()
    out[out == 0] = np.float32(0.0)
    if not (0.0 <= sparsity < 1.0):
        raise ValueError("sparsity must be in [0, 1)")
    z = int(np.floor(np.float64(sparsity) * np.float64(W.size)))
    if z == 0:
        return out
    mag = np.abs(out).ravel()
    w_p = np.sort(mag)[z - 1]
    out[np.abs(out) <= w_p] = np.float32(0.0)
    return out


# ----------------------------------------------------------------------------
# SplitMix64 (Steele, Lea, Flood, "Fast splittable pseudorandom number
# generators", OOPSLA 2014), used as a counter-based generator: the i-th draw
# mixes seed + (i + 1) * gamma.  The k-means initialisation and PWS draw numbers.
# ----------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def splitmix64(seed: int, i: int) -> int:
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def kmeans_init(u: np.ndarray, k: int, seed: int) -> np.ndarray:
    """k distinct starting centroids: a partial Fisher-Yates shuffle of the
    sorted distinct values u, draw i swapping position i with position
    i + (r_i mod (len(u) - i)); the first k entries, sorted ascending."""
    idx = np.arange(len(u), dtype=np.int64)
    for i in range(k):
        j = i + splitmix64(seed, i) % (len(u) - i)
        idx[i], idx[j] = idx[j], idx[i]
    return np.sort(u[idx[:k]])


# ----------------------------------------------------------------------------
# Sect. III-C  weight sharing
# ----------------------------------------------------------------------------
def _nonnull_colmajor(Wp: np.ndarray):
    """Non-null weights of the pruned matrix listed by columns (the order of
    the CSC vector nz, Sect. IV-A), and the boolean mask they come from."""
    mask = Wp != 0
    return Wp.T[mask.T].astype(np.float64), mask


def _scatter_colmajor(mask: np.ndarray, values32: np.ndarray) -> np.ndarray:
    Wq = np.zeros(mask.shape, dtype=np.float32)
    WqT = Wq.T                      # view: assignment in column-major order
    WqT[mask.T] = values32
    Wq[Wq == 0] = np.float32(0.0)   # a centroid that rounds to -0.0 is stored as +0.0
    return Wq


def kmeans_share(Wp: np.ndarray, k: int, iters: int, seed: int, return_trace: bool = False):
    """CWS (Sect. III-C.1): k-means over the non-null weights (pruning and CWS
    in chain cluster only the weights that survived pruning), every weight
    replaced by its centroid.

    Reading (the paper only says "k-means"): Lloyd iterations, exactly `iters`
    of them, in fp64, on the weights in column-major storage order; seeded
    start from k distinct data values (kmeans_init); nearest centroid through
    midpoints, ties to the lower centroid; empty clusters keep their centroid;
    after the last update one more assignment.  If the data has at most k
    distinct values they are the codebook.  Centroids are rounded to fp32 when
    they replace the weights, so fewer than k shared values may remain.
    Returns (Wq, mask) with mask the positions of the non-null weights.
    """
    data, mask = _nonnull_colmajor(Wp)
    if k < 1:
        raise ValueError("k must be >= 1")
    if data.size == 0:
        return (np.zeros_like(Wp), mask) if not return_trace else (np.zeros_like(Wp), mask, None, None)
    u = np.unique(data)
    if len(u) <= k:
        Wq = _scatter_colmajor(mask, data.astype(np.float32))
        return (Wq, mask) if not return_trace else (Wq, mask, u, None)
    c = np.ascontiguousarray(kmeans_init(u, k, seed), dtype=np.float64)
    assign = np.empty(data.size, dtype=np.int32)
    sse = np.zeros(iters + 1, dtype=np.float64)
    data = np.ascontiguousarray(data)
    rc = _native().orc_kmeans(_p(data), ctypes.c_int64(data.size), _p(c), ctypes.c_int32(k),
                              ctypes.c_int32(iters), _p(assign), _p(sse))
    if rc != 0:
        raise RuntimeError(f"orc_kmeans failed: {rc}")
    Wq = _scatter_colmajor(mask, c.astype(np.float32)[assign])
    if return_trace:
        return Wq, mask, c, sse
    return Wq, mask


def uniform_share(Wp: np.ndarray, k: int):
    """UQ (Sect. III-C.3): representatives spaced uniformly in the weight domain,
    w = delta * round(w0 / delta) with the grid laid over the range of the
    non-null weights so that it has exactly k levels:
    lo = min, hi = max, delta = (hi - lo) / (k - 1),
    level(w) = floor((w - lo) / delta + 1/2) clamped to [0, k-1] (round half up),
    value = fp32(lo + level * delta).  Levels nobody falls in are not part of
    the codebook.  Returns (Wq, mask)."""
    data, mask = _nonnull_colmajor(Wp)
    if k < 2:
        raise ValueError("uniform quantization needs k >= 2")
    if data.size == 0:
        return np.zeros_like(Wp), mask
    lo = data.min()
    hi = data.max()
    if hi == lo:
        return _scatter_colmajor(mask, data.astype(np.float32)), mask
    delta = (hi - lo) / np.float64(k - 1)
    level = np.floor((data - lo) / delta + 0.5)
    level = np.clip(level, 0.0, np.float64(k - 1))
    values = (lo + level * delta).astype(np.float32)
    return _scatter_colmajor(mask, values), mask


def grid_levels(data: np.ndarray, delta: float) -> np.ndarray:
    """round(w / delta) of the formula of Sect. III-C.3 with d = 0, rounding half up."""
    return np.floor(data / np.float64(delta) + 0.5)


def grid_delta(data: np.ndarray, k: int, steps: int = 70) -> float:
    """The interval size delta of the zero-anchored grid, chosen so that the wanted number k of
    values results (the setting of uUQ in Sect. V; the paper gives no procedure): bisection on [0, 4 max|w|], `steps` halvings (enough to
    end on neighbouring doubles for k up to 2048); a trial
    delta that leaves at most k distinct values becomes the upper end, one that leaves more
    the lower end; the upper end is returned (it always satisfies the bound: at 4 max|w| every
    weight rounds to 0)."""
    a = np.float64(0.0)
    b = np.float64(4.0) * np.abs(data).max()
    for _ in range(steps):
        mid = np.float64(0.5) * (a + b)
        if len(np.unique(grid_levels(data, mid))) <= k:
            b = mid
        else:
            a = mid
    return float(b)


def grid_share(Wp: np.ndarray, k: int):
    """UQ exactly as printed in Sect. III-C.3, with the bias d = 0 of the paper's experiments:
    w = delta * round(w0 / delta) over the non-null weights, delta from grid_delta.  A weight that
    rounds to level 0 becomes the value 0.0 but stays a stored entry (it survived pruning).
    When the non-null weights already have at most k distinct values they are kept as they are.
    Returns (Wq, mask)."""
    data, mask = _nonnull_colmajor(Wp)
    if k < 2:
        raise ValueError("grid quantization needs k >= 2")
    if data.size == 0:
        return np.zeros_like(Wp), mask
    if len(np.unique(data)) <= k:
        return _scatter_colmajor(mask, data.astype(np.float32)), mask
    delta = np.float64(grid_delta(data, k))
    values = (grid_levels(data, delta) * delta).astype(np.float32)
    values[values == 0] = np.float32(0.0)                  # -0.0 -> +0.0
    return _scatter_colmajor(mask, values), mask


def splitmix64_many(seed: int, count: int) -> np.ndarray:
    """splitmix64(seed, i) for i = 0 .. count-1 (uint64 arithmetic wraps, as the generator wants)."""
    with np.errstate(over="ignore"):
        z = np.uint64(seed & _M64) + (np.arange(count, dtype=np.uint64) + np.uint64(1)) * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def pws_extremes(data: np.ndarray, k: int) -> np.ndarray:
    """The k representatives of PWS (Sect. III-C.2): the extremes of k - 1 intervals that hold equal
    shares of the weights, i.e. the i/(k-1) quantiles, i = 0 .. k-1, taken as order statistics
    s[floor(i (q-1) / (k-1))] of the sorted weights; equal ones are listed once."""
    srt = np.sort(data)
    q = len(srt)
    pos = [(i * (q - 1)) // (k - 1) for i in range(k)]
    return np.unique(srt[pos])


def pws_share(Wp: np.ndarray, k: int, seed: int):
    """PWS (Sect. III-C.2): a weight w inside the interval [lo, hi) of two neighbouring representatives
    becomes hi with probability (w - lo) / (hi - lo) and lo otherwise, which makes the result an
    unbiased estimate of w.  Weight p (column-major position among the non-null weights) uses the
    uniform number (splitmix64(seed, p) >> 11) * 2^-53.  Weights with at most k distinct values
    are kept as they are.  Returns (Wq, mask)."""
    data, mask = _nonnull_colmajor(Wp)
    if k < 2:
        raise ValueError("PWS needs k >= 2")
    if data.size == 0:
        return np.zeros_like(Wp), mask
    if len(np.unique(data)) <= k:
        return _scatter_colmajor(mask, data.astype(np.float32)), mask
    ext = pws_extremes(data, k)
    j = np.clip(np.searchsorted(ext, data, side="right") - 1, 0, len(ext) - 2)
    lo, hi = ext[j], ext[j + 1]
    p_hi = (data - lo) / (hi - lo)
    u = (splitmix64_many(seed, len(data)) >> np.uint64(11)).astype(np.float64) * np.float64(2.0 ** -53)
    values = np.where(u < p_hi, hi, lo).astype(np.float32)
    return _scatter_colmajor(mask, values), mask


def share_none(Wp: np.ndarray):
    """No weight sharing: the matrix already holds few distinct values."""
    Wq = Wp.copy()
    Wq[Wq == 0] = np.float32(0.0)
    return Wq, Wq != 0


def quantize(W: np.ndarray, sparsity: float, k: int, quantizer: int, iters: int = 20, seed: int = 0):
    """Pruning then weight sharing, as chained in Sect. III-C.1.  quantizer:
    0 none, 1 k-means (CWS), 2 uniform (UQ over [min, max]), 3 uniform (UQ on the zero-anchored
    grid of the printed formula), 4 probabilistic (PWS).  Returns (Wq, mask)."""
    Wp = prune(W, sparsity)
    if quantizer == 0:
        return share_none(Wp)
    if quantizer == 1:
        return kmeans_share(Wp, k, iters, seed)
    if quantizer == 2:
        return uniform_share(Wp, k)
    if quantizer == 3:
        return grid_share(Wp, k)
    if quantizer == 4:
        return pws_share(Wp, k, seed)
    raise ValueError("unknown quantizer")


# ----------------------------------------------------------------------------
# Sect. IV-B  Huffman code
# ----------------------------------------------------------------------------
def huffman_lengths(counts) -> np.ndarray:
    """Code word length of every symbol of a Huffman code for `counts`.

    Huffman's construction: repeatedly merge the two least frequent nodes.
    Which optimal code results depends on how ties are broken; the rule here:
    leaves sorted by (count, symbol id); merged nodes queue up in creation
    order; of two candidates with the same weight the leaf is taken before the
    merged node.  A single-symbol alphabet gets a 1-bit code word (a prefix
    code needs at least one bit per symbol to be countable in a stream).
    """
    counts = [int(c) for c in counts]
    k = len(counts)
    if k == 0:
        return np.zeros(0, dtype=np.uint8)
    if any(c <= 0 for c in counts):
        raise ValueError("every symbol of the alphabet must occur")
    if k == 1:
        return np.array([1], dtype=np.uint8)
    parent = {}
    leaves = deque(sorted(range(k), key=lambda s: (counts[s], s)))
    weight = {s: counts[s] for s in range(k)}
    merged = deque()
    nxt = k

    def take():
        if leaves and (not merged or weight[leaves[0]] <= weight[merged[0]]):
            return leaves.popleft()
        return merged.popleft()

    while len(leaves) + len(merged) > 1:
        a = take()
        b = take()
        weight[nxt] = weight[a] + weight[b]
        parent[a] = nxt
        parent[b] = nxt
        merged.append(nxt)
        nxt += 1
    lengths = np.zeros(k, dtype=np.int64)
    for s in range(k):
        v, d = s, 0
        while v in parent:
            v = parent[v]
            d += 1
        lengths[s] = d
    if lengths.max() > 32:
        raise ValueError("code word longer than 32 bits")
    return lengths.astype(np.uint8)


def canonical_codes(lengths) -> np.ndarray:
    """Code words for given lengths: symbols ordered by (length, id); the first
    gets 0...0, each next one the previous code word plus one, shifted left by
    the growth in length.  Code words are read most significant bit first.
    (The paper keeps the dictionaries H and H^-1 as B-trees; any prefix code
    with Huffman's lengths is an equally valid H.)"""
    lengths = np.asarray(lengths, dtype=np.int64)
    order = sorted(range(len(lengths)), key=lambda s: (int(lengths[s]), s))
    codes = np.zeros(len(lengths), dtype=np.uint32)
    code = 0
    prev = None
    for s in order:
        if prev is not None:
            code = (code + 1) << (int(lengths[s]) - prev)
        codes[s] = code
        prev = int(lengths[s])
    return codes


def entropy_bits(counts) -> float:
    p = np.asarray(counts, dtype=np.float64)
    p = p / p.sum()
    return float(-(p * np.log2(p)).sum())


# ----------------------------------------------------------------------------
# Sect. IV-A / IV-B / IV-C  the formats
# ----------------------------------------------------------------------------
def csc(Wq: np.ndarray, mask: np.ndarray):
    """CSC of Sect. IV-A: nz (stored values by column, rows ascending), ri (row
    of each), cb (cb[j] = number of stored entries in columns before j; the
    paper's cb is this plus one).  Stored entries are those of `mask`."""
    cols, rows = np.nonzero(mask.T)
    nz = Wq.T[mask.T].astype(np.float32)
    cb = np.zeros(mask.shape[1] + 1, dtype=np.int64)
    np.cumsum(np.bincount(cols, minlength=mask.shape[1]), out=cb[1:])
    return nz, rows.astype(np.int32), cb


def _pack(sym: np.ndarray, codes: np.ndarray, lengths: np.ndarray):
    total_bits = int(lengths.astype(np.int64)[sym].sum())
    nwords = (total_bits + B_WORD - 1) // B_WORD
    words = np.zeros(max(nwords, 1), dtype=np.uint32)
    sym = np.ascontiguousarray(sym, dtype=np.int32)
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    written = _native().orc_pack(_p(sym), ctypes.c_int64(sym.size), _p(codes), _p(lengths),
                                 _p(words), ctypes.c_int64(nwords))
    if written != total_bits:
        raise RuntimeError("orc_pack failed")
    return words[:nwords], total_bits


def _alphabet(values_in_stream_order: np.ndarray):
    codebook, sym, counts = np.unique(values_in_stream_order, return_inverse=True, return_counts=True)
    if len(codebook) > MAX_SYMBOLS:
        raise ValueError("too many distinct values")
    return codebook.astype(np.float32), sym.astype(np.int32).ravel(), counts.astype(np.int64)


def hac_encode(Wq: np.ndarray) -> dict:
    """HAC (Sect. IV-B): the address map of W in column order with a(z) the
    Huffman code word of z and the null entries coded like any other value;
    the bit string is cut into N = ceil(bits / 32) words, the last zero padded.
    Symbol id = rank of the value among the distinct values (ascending)."""
    n, m = Wq.shape
    seq = np.ascontiguousarray(Wq.T).ravel()          # column after column
    codebook, sym, counts = _alphabet(seq)
    lengths = huffman_lengths(counts)
    codes = canonical_codes(lengths)
    words, bits = _pack(sym, codes, lengths)
    return dict(kind="hac", n=n, m=m, codebook=codebook, counts=counts, code_len=lengths,
                codes=codes, sym=sym, words=words, bits=bits)


def shac_encode(Wq: np.ndarray, mask: np.ndarray) -> dict:
    """sHAC (Sect. IV-C): the CSC vectors of W with nz Huffman coded (code built
    on the stored values only, no code word for the null entries) and ri, cb
    kept as they are."""
    n, m = Wq.shape
    nz, ri, cb = csc(Wq, mask)
    if nz.size:
        codebook, sym, counts = _alphabet(nz)
        lengths = huffman_lengths(counts)
        codes = canonical_codes(lengths)
        words, bits = _pack(sym, codes, lengths)
    else:
        codebook = np.zeros(0, np.float32); sym = np.zeros(0, np.int32)
        counts = np.zeros(0, np.int64); lengths = np.zeros(0, np.uint8)
        codes = np.zeros(0, np.uint32); words = np.zeros(0, np.uint32); bits = 0
    return dict(kind="shac", n=n, m=m, codebook=codebook, counts=counts, code_len=lengths,
                codes=codes, sym=sym, words=words, bits=bits, nz=nz, ri=ri, cb=cb)


def decode_symbols(fmt: dict, bit0: int, count: int) -> tuple:
    """Read `count` symbols starting at bit `bit0` of the stream (tree walk)."""
    out = np.empty(max(count, 1), dtype=np.int32)
    words = np.ascontiguousarray(fmt["words"], dtype=np.uint32)
    end = _native().orc_decode(_p(words), ctypes.c_int64(words.size), ctypes.c_int64(bit0),
                               _p(np.ascontiguousarray(fmt["codes"])),
                               _p(np.ascontiguousarray(fmt["code_len"])),
                               ctypes.c_int32(len(fmt["codebook"])), ctypes.c_int64(count), _p(out))
    if end < 0:
        raise RuntimeError(f"orc_decode failed: {end}")
    return out[:count], int(end)


def hac_decode(fmt: dict) -> np.ndarray:
    """Rebuild the quantized matrix from a HAC stream (the format is lossless)."""
    sym, _ = decode_symbols(fmt, 0, fmt["n"] * fmt["m"])
    return fmt["codebook"][sym].reshape(fmt["m"], fmt["n"]).T.copy()


def shac_decode(fmt: dict) -> np.ndarray:
    sym, _ = decode_symbols(fmt, 0, int(fmt["cb"][-1]))
    W = np.zeros((fmt["n"], fmt["m"]), dtype=np.float32)
    cols = np.repeat(np.arange(fmt["m"]), np.diff(fmt["cb"]))
    W[fmt["ri"], cols] = fmt["codebook"][sym]
    return W


# ----------------------------------------------------------------------------
# Offset index (the column-offset vector the paper's conclusions propose for a
# finer parallelism, refined to sub-segments of S symbols)
# ----------------------------------------------------------------------------
def hac_offset_index(fmt: dict, S: int) -> dict:
    """Every column is cut into sub-segments of S symbols (the last shorter);
    32 consecutive sub-segments of a column form a segment.  seg_bit_off[u] is
    the bit at which segment u = j*G + g starts, sub_bits[u*32 + l] the bit
    length of its l-th sub-segment (0 where the column has ended)."""
    n, m = fmt["n"], fmt["m"]
    T = -(-n // S)
    G = -(-T // 32)
    lens = fmt["code_len"].astype(np.int64)[fmt["sym"]].reshape(m, n)
    padded = np.zeros((m, G * 32 * S), dtype=np.int64)
    padded[:, :n] = lens
    sub_bits = padded.reshape(m, G * 32, S).sum(axis=2)
    seg_bits = sub_bits.reshape(m * G, 32).sum(axis=1)
    seg_bit_off = np.concatenate(([0], np.cumsum(seg_bits)[:-1])).astype(np.uint64)
    return dict(S=S, T=T, G=G, seg_bit_off=seg_bit_off,
                sub_bits=sub_bits.reshape(-1).astype(np.uint16))


def shac_offset_index(fmt: dict, S: int) -> dict:
    """As for HAC, over each column's run of stored entries: column j with q_j
    entries has ceil(q_j / S) sub-segments and ceil(that / 32) segments.
    seg_first[j] = number of segments in columns before j, seg_col[u] = column
    of segment u."""
    m = fmt["m"]
    cb = fmt["cb"]
    lens = fmt["code_len"].astype(np.int64)[fmt["sym"]] if fmt["sym"].size else np.zeros(0, np.int64)
    seg_first = np.zeros(m + 1, dtype=np.uint32)
    seg_col, seg_bits_all, sub_all = [], [], []
    for j in range(m):
        l = lens[cb[j]:cb[j + 1]]
        T = -(-len(l) // S)
        G = -(-T // 32)
        seg_first[j + 1] = seg_first[j] + G
        if G == 0:
            continue
        padded = np.zeros(G * 32 * S, dtype=np.int64)
        padded[:len(l)] = l
        sb = padded.reshape(G * 32, S).sum(axis=1)
        sub_all.append(sb)
        seg_bits_all.append(sb.reshape(G, 32).sum(axis=1))
        seg_col.extend([j] * G)
    if seg_col:
        seg_bits = np.concatenate(seg_bits_all)
        seg_bit_off = np.concatenate(([0], np.cumsum(seg_bits)[:-1])).astype(np.uint64)
        sub_bits = np.concatenate(sub_all).astype(np.uint16)
    else:
        seg_bit_off = np.zeros(0, np.uint64); sub_bits = np.zeros(0, np.uint16)
    return dict(S=S, seg_first=seg_first, seg_col=np.asarray(seg_col, dtype=np.uint32),
                seg_bit_off=seg_bit_off, sub_bits=sub_bits)


# ----------------------------------------------------------------------------
# Space bounds (Corollaries 1 and 2) with the paper's accounting
# ----------------------------------------------------------------------------
def hac_paper_bits(fmt: dict) -> int:
    """|HAC(W)| as the paper counts it: stream words plus 6*k*b bits for the two
    dictionaries held as B-trees (proof of Theorem 1)."""
    return len(fmt["words"]) * B_WORD + 6 * len(fmt["codebook"]) * B_WORD


def cor1_bound_bits(n: int, m: int, k: int) -> float:
    """Corollary 1: |HAC(W)| <= nm (1 + log k) + 6 k b."""
    return n * m * (1.0 + np.log2(k)) + 6 * k * B_WORD


def shac_paper_bits(fmt: dict) -> int:
    """|sHAC(W)|: stream words, dictionaries, and ri, cb at b bits per entry."""
    q = int(fmt["cb"][-1])
    return (len(fmt["words"]) * B_WORD + 6 * len(fmt["codebook"]) * B_WORD
            + B_WORD * (q + fmt["m"] + 1))


def cor2_bound_bits(n: int, m: int, q: int, k: int) -> float:
    """Corollary 2 with s*n*m = q stored entries:
    |sHAC(W)| <= q (1 + log k) + b (6k + q + m + 1)."""
    return q * (1.0 + np.log2(max(k, 1))) + B_WORD * (6 * k + q + m + 1)


def shac_smaller_than_hac_threshold(n: int, m: int, k: int) -> float:
    """Non-zero ratio s below which the sHAC bound is under the HAC bound
    (the inequality after Algorithm 2)."""
    a = (1.0 + np.log2(k)) / B_WORD
    return (a - (m + 1) / (n * m)) / (1.0 + a)


# ----------------------------------------------------------------------------
# Sect. IV-B / IV-C / IV-D  the dot procedures
# ----------------------------------------------------------------------------
def _c32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def dot_hac(fmt: dict, x: np.ndarray) -> np.ndarray:
    """Algorithm 1 (Dot_HAC): sequential scan of the words, NCW pulling one code
    word at a time.  x has n entries; the result has m (one per column)."""
    out = np.zeros(fmt["m"], dtype=np.float64)
    words = np.ascontiguousarray(fmt["words"], dtype=np.uint32)
    rc = _native().orc_dot_hac(_p(words), ctypes.c_int64(words.size),
                               _p(np.ascontiguousarray(fmt["codes"])), _p(np.ascontiguousarray(fmt["code_len"])),
                               _p(_c32(fmt["codebook"])), ctypes.c_int32(len(fmt["codebook"])),
                               _p(_c32(x)), ctypes.c_int64(fmt["n"]), ctypes.c_int64(fmt["m"]), _p(out))
    if rc:
        raise RuntimeError(f"orc_dot_hac failed: {rc}")
    return out


def dot_shac(fmt: dict, x: np.ndarray) -> np.ndarray:
    """Algorithm 2 (Dot_sHAC)."""
    out = np.zeros(fmt["m"], dtype=np.float64)
    if fmt["cb"][-1] == 0:
        return out
    words = np.ascontiguousarray(fmt["words"], dtype=np.uint32)
    rc = _native().orc_dot_shac(_p(words), ctypes.c_int64(words.size),
                                _p(np.ascontiguousarray(fmt["codes"])), _p(np.ascontiguousarray(fmt["code_len"])),
                                _p(_c32(fmt["codebook"])), ctypes.c_int32(len(fmt["codebook"])),
                                _p(np.ascontiguousarray(fmt["ri"], dtype=np.int32)),
                                _p(np.ascontiguousarray(fmt["cb"], dtype=np.int64)),
                                _p(_c32(x)), ctypes.c_int64(fmt["m"]), _p(out))
    if rc:
        raise RuntimeError(f"orc_dot_shac failed: {rc}")
    return out


def pardot(fmt: dict, X: np.ndarray, q: int) -> np.ndarray:
    """Algorithm 3 (ParDot): X is B x n, one input per row; its rows are split
    into q chunks, each handled by one thread running Algorithm 1 or 2 once per
    row.  Returns B x m."""
    X = _c32(X)
    B = X.shape[0]
    out = np.zeros((B, fmt["m"]), dtype=np.float64)
    words = np.ascontiguousarray(fmt["words"], dtype=np.uint32)
    common = (_p(words), ctypes.c_int64(words.size), _p(np.ascontiguousarray(fmt["codes"])),
              _p(np.ascontiguousarray(fmt["code_len"])), _p(_c32(fmt["codebook"])),
              ctypes.c_int32(len(fmt["codebook"])))
    tail = (_p(X), ctypes.c_int64(B), ctypes.c_int64(fmt["n"]), ctypes.c_int64(fmt["m"]),
            ctypes.c_int32(q), _p(out))
    if fmt["kind"] == "hac":
        rc = _native().orc_pardot_hac(*common, *tail)
    else:
        if fmt["cb"][-1] == 0:
            return out
        rc = _native().orc_pardot_shac(*common, _p(np.ascontiguousarray(fmt["ri"], dtype=np.int32)),
                                       _p(np.ascontiguousarray(fmt["cb"], dtype=np.int64)), *tail)
    if rc:
        raise RuntimeError(f"pardot failed: {rc}")
    return out


def dot_definition(Wq: np.ndarray, X: np.ndarray, cols=None):
    """What the dot procedures output, written out: y[b, j] = sum_i Wq[i, j] X[b, i]
    in fp64 with i ascending, and a[b, j] = sum_i |Wq[i, j] X[b, i]|, the scale of the
    output tolerance.  With `cols`, only those columns (full-size spot checks)."""
    Wq = _c32(Wq)
    X = _c32(np.atleast_2d(X))
    n, m = Wq.shape
    B = X.shape[0]
    if cols is None:
        y = np.zeros((B, m)); a = np.zeros((B, m))
        _native().orc_dot_definition(_p(Wq), ctypes.c_int64(n), ctypes.c_int64(m), _p(X),
                                     ctypes.c_int64(B), _p(y), _p(a))
    else:
        cols = np.ascontiguousarray(cols, dtype=np.int64)
        y = np.zeros((B, cols.size)); a = np.zeros((B, cols.size))
        rc = _native().orc_dot_definition_cols(_p(Wq), ctypes.c_int64(n), ctypes.c_int64(m), _p(X),
                                               ctypes.c_int64(B), _p(cols), ctypes.c_int64(cols.size),
                                               _p(y), _p(a))
        if rc:
            raise RuntimeError("bad column index")
    return y, a


def layer_definition(Wq: np.ndarray, X: np.ndarray, bias=None, relu: bool = False, cols=None):
    """A fully connected layer evaluated on the compressed matrix, written out (Sect. V evaluates the
    networks with their fully connected layers kept in HAC / sHAC; the layer itself is the ordinary
    one): out[b, j] = act(sum_i Wq[i, j] X[b, i] + bias[j]) in fp64, act = identity or max(., 0).
    Returns (out, a) with a[b, j] = sum_i |Wq[i, j] X[b, i]| + |bias[j]|, the scale of the output
    tolerance (the activation does not enlarge an error)."""
    y, a = dot_definition(Wq, X, cols=cols)
    if bias is not None:
        b = np.asarray(bias, dtype=np.float64)
        if cols is not None:
            b = b[np.asarray(cols)]
        y = y + b[None, :]
        a = a + np.abs(b)[None, :]
    if relu:
        y = np.where(y < 0.0, 0.0, y)
    return y, a


def chain_definition(layers, X: np.ndarray):
    """A stack of such layers: `layers` is a list of (Wq, bias or None, relu); the input of layer l + 1 is
    the output of layer l rounded to fp32 (activations are stored as fp32).  Returns the list of every
    layer's (out, a)."""
    outs = []
    cur = np.atleast_2d(X)
    for Wq, bias, relu in layers:
        y, a = layer_definition(Wq, cur, bias, relu)
        outs.append((y, a))
        cur = y.astype(np.float32)
    return outs


# ----------------------------------------------------------------------------
# Sect. III-C.1 / IV-A  the formats HAC and sHAC are compared with (Sect. V, comparison of the formats):
# the index map and plain CSC
# ----------------------------------------------------------------------------
def index_map_encode(Wq: np.ndarray) -> dict:
    """Index map of Sect. III-C.1: the distinct values of Wq (zero included when it occurs) in a vector c,
    ascending, and the matrix Pi of pointers into it, pi_ij = position of Wq[i, j] in c, stored with
    b_bar = 8 bits when there are at most 256 values, else 16 (the paper's example), else 32."""
    Wq = _c32(Wq)
    c, inverse = np.unique(Wq, return_inverse=True)
    k = len(c)
    b_bar = 8 if k <= 256 else (16 if k <= 65536 else 32)
    dtype = {8: np.uint8, 16: np.uint16, 32: np.uint32}[b_bar]
    return {"n": Wq.shape[0], "m": Wq.shape[1], "codebook": c.astype(np.float32),
            "index": inverse.reshape(Wq.shape).astype(dtype), "b_bar": b_bar}


def index_map_bits(fmt: dict) -> int:
    """Size as the paper counts it: b_bar * n * m + k * b."""
    return fmt["b_bar"] * fmt["n"] * fmt["m"] + len(fmt["codebook"]) * B_WORD


def index_map_decode(fmt: dict) -> np.ndarray:
    return fmt["codebook"][fmt["index"].astype(np.int64)]


def dot_index_map(fmt: dict, X: np.ndarray):
    """x^T W with every weight fetched through its pointer, fp64, rows ascending; (y, a) as dot_definition."""
    X = np.atleast_2d(_c32(X)).astype(np.float64)
    n, m = fmt["n"], fmt["m"]
    c = fmt["codebook"].astype(np.float64)
    y = np.zeros((X.shape[0], m)); a = np.zeros((X.shape[0], m))
    idx = fmt["index"]
    for i in range(n):
        w = c[idx[i].astype(np.int64)]                  # row i of W through the map
        t = X[:, i:i + 1] * w[None, :]
        y += t; a += np.abs(t)
    return y, a


def csc_bits(nz, ri, cb) -> int:
    """Size of CSC as the paper counts it: (2 q + m + 1) b."""
    return (2 * len(nz) + len(cb)) * B_WORD


def dot_csc(nz, ri, cb, n: int, X: np.ndarray):
    """x^T W from the CSC vectors (Sect. IV-A): out[j] = sum over the stored entries p of column j of
    nz[p] * x[ri[p]], fp64, in storage order; (y, a) as dot_definition."""
    X = np.atleast_2d(_c32(X)).astype(np.float64)
    m = len(cb) - 1
    y = np.zeros((X.shape[0], m)); a = np.zeros((X.shape[0], m))
    nz64 = np.asarray(nz, dtype=np.float64)
    for j in range(m):
        for p in range(int(cb[j]), int(cb[j + 1])):
            t = X[:, int(ri[p])] * nz64[p]
            y[:, j] += t; a[:, j] += np.abs(t)
    return y, a


# ----------------------------------------------------------------------------
# Sect. V-D  unified quantization: all matrices quantized together, one dictionary
# ----------------------------------------------------------------------------
def quantize_unified(Ws, sparsity: float, k: int, quantizer: int, iters: int = 20, seed: int = 0):
    """Every matrix pruned on its own (Sect. III-B), then ONE run of the weight sharing over the non-null weights of all
    of them, listed matrix after matrix and column-major inside each (reading: the paper only says that the matrices are
    quantized together with a single k; the order only matters for the seeded start of k-means and the random draws of
    PWS).  Returns a list of (Wq, mask)."""
    pruned = [prune(W, sparsity) for W in Ws]
    parts = [_nonnull_colmajor(Wp) for Wp in pruned]
    if sum(d.size for d, _ in parts) == 0:
        return [(np.zeros_like(Wp), mask) for Wp, (_, mask) in zip(pruned, parts)]
    # the concatenated weights as one column: its column-major list of non-null weights is that concatenation
    column = np.concatenate([d for d, _ in parts]).astype(np.float32).reshape(-1, 1)
    if quantizer == 0:
        shared, _ = share_none(column)
    elif quantizer == 1:
        shared, _ = kmeans_share(column, k, iters, seed)
    elif quantizer == 2:
        shared, _ = uniform_share(column, k)
    elif quantizer == 3:
        shared, _ = grid_share(column, k)
    elif quantizer == 4:
        shared, _ = pws_share(column, k, seed)
    else:
        raise ValueError("unknown quantizer")
    out, at = [], 0
    for data, mask in parts:
        out.append((_scatter_colmajor(mask, shared[at:at + data.size, 0]), mask))
        at += data.size
    return out


def unified_encode(layers):
    """layers: list of (kind, Wq, mask).  One alphabet and one Huffman code on the symbol counts of all the streams together
    (HAC: every entry of the matrix, zeros included; sHAC: the stored entries), then each matrix coded with it.  Returns one
    format dict per layer (as hac_encode / shac_encode; `counts` are the layer's own, `shared_counts` those of the code)."""
    seqs = []
    for kind, Wq, mask in layers:
        seqs.append(np.ascontiguousarray(Wq.T).ravel() if kind == "hac" else csc(Wq, mask)[0])
    codebook, sym_all, counts = _alphabet(np.concatenate(seqs))
    lengths = huffman_lengths(counts)
    codes = canonical_codes(lengths)
    out, at = [], 0
    for (kind, Wq, mask), seq in zip(layers, seqs):
        sym = sym_all[at:at + seq.size]
        at += seq.size
        if seq.size:
            words, bits = _pack(sym, codes, lengths)
        else:
            words, bits = np.zeros(0, np.uint32), 0
        fmt = dict(kind=kind, n=Wq.shape[0], m=Wq.shape[1], codebook=codebook, code_len=lengths, codes=codes,
                   counts=np.bincount(sym, minlength=len(codebook)).astype(np.int64), shared_counts=counts, sym=sym,
                   words=words, bits=bits)
        if kind == "shac":
            nz, ri, cb = csc(Wq, mask)
            fmt.update(nz=nz, ri=ri, cb=cb)
        out.append(fmt)
    return out


def unified_paper_bits(fmts) -> int:
    """Size of a unified model as the paper counts it: every stream (and ri, cb of the sHAC ones), one dictionary."""
    k = len(fmts[0]["codebook"])
    total = 6 * k * B_WORD
    for f in fmts:
        total += len(f["words"]) * B_WORD
        if f["kind"] == "shac":
            total += B_WORD * (int(f["cb"][-1]) + f["m"] + 1)
    return total
