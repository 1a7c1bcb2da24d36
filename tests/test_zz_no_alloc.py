"""hac_dot_noalloc: the HAC product for hosts that may not allocate device memory (a server with a
fixed memory plan, a plugin without an allocator).  Its partial sums live in a buffer inside the
library image, so the call needs no workspace from the caller.  Checked here through the C ABI
against hac_dot on the same inputs, twice in a row (the buffer is shared between calls and keeps
the previous call's contents), and for the refusal of products that do not fit the buffer.

This file is collected last on purpose: a run that stops at the first failure has then already run
every other test."""
import ctypes as C

import numpy as np
import pytest

import synth_inputs as si
from oracle import hac_oracle as orc
import paper_2108_12704_b200 as hb

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

NOALLOC_BYTES = 4 << 20          # HAC_NOALLOC_SCRATCH_BYTES of include/hac.h


def _format(n, m, S):
    wl = si.scaled(si.CFG2_DENSE_HAC, n, m)
    W = si.weights(wl)
    fmt = hb.Format("hac", W, sparsity=wl.sparsity, k=wl.k, quantizer=wl.quantizer, seed=wl.seed,
                    seg_symbols=S).upload()
    Wq, _ = orc.quantize(W, wl.sparsity, wl.k, wl.quantizer, wl.kmeans_iters, wl.seed)
    return wl, fmt, Wq


def _raw_call(fmt, x, y, B, xs_i, xs_b, ys_j, ys_b):
    """The entry point itself, with plain pointers and strides, on torch's current stream."""
    lib = hb.load()
    st = torch.cuda.current_stream().cuda_stream
    return lib.hac_dot_noalloc(fmt._h, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b, st)


def test_noalloc_matches_hac_dot_twice_in_a_row():
    # 1000 rows in sub-segments of 8: four segments per column, so partial sums are really used
    wl, fmt, Wq = _format(1000, 96, 8)
    assert fmt.workspace_bytes(1) > 0 and fmt.workspace_bytes(5) <= NOALLOC_BYTES
    for round_ in range(2):
        for B in (1, 5):
            X = si.inputs(wl, B, salt=round_)
            y_ref, a = orc.dot_definition(Wq, X)
            if B == 1:
                x = torch.from_numpy(X[0]).cuda()
                want = fmt.dot(x)
                got = torch.full((wl.m,), float("nan"), device="cuda")
                assert _raw_call(fmt, x, got, 1, 1, 0, 1, 0) == 0
            else:
                x = torch.from_numpy(np.ascontiguousarray(X.T)).cuda()            # [n, B]
                want = fmt.dot(x)
                got = torch.full((wl.m, B), float("nan"), device="cuda")
                assert _raw_call(fmt, x, got, B, B, 1, B, 1) == 0
            torch.cuda.synchronize()
            got_h, want_h = got.cpu().numpy(), want.cpu().numpy()
            ref = y_ref[0] if B == 1 else y_ref.T
            tol = 1e-5 * (a[0] if B == 1 else a.T) + 1e-7
            assert np.all(np.abs(got_h - want_h) <= tol)            # against the existing entry point
            assert np.all(np.abs(got_h - ref) <= tol)               # and against the oracle


def test_noalloc_binding_and_refusal():
    wl, fmt, Wq = _format(1000, 96, 8)
    x = torch.from_numpy(si.inputs(wl, 1)[0]).cuda()
    assert torch.equal(fmt.dot_noalloc(x), fmt.dot(x))
    # a batch whose partial sums exceed the built-in buffer is refused, nothing is written
    B = NOALLOC_BYTES // fmt.workspace_bytes(1) + 1
    assert fmt.workspace_bytes(B) > NOALLOC_BYTES
    X = torch.zeros((wl.n, B), device="cuda")
    y = torch.full((wl.m, B), 7.0, device="cuda")
    rc = _raw_call(fmt, X, y, B, B, 1, B, 1)
    assert rc == -8                                                  # HAC_ERR_BUFFER_TOO_SMALL
    text = hb.load().hac_last_cuda_error().decode()
    assert "hac_dot_noalloc" in text and str(NOALLOC_BYTES) in text
    torch.cuda.synchronize()
    assert bool((y == 7.0).all())
    # the buffer is still good afterwards
    assert torch.equal(fmt.dot_noalloc(x), fmt.dot(x))
    # formats that were never uploaded are refused too
    cold = hb.Format("hac", si.weights(si.scaled(si.CFG2_DENSE_HAC, 64, 8)), k=8, quantizer=hb.QUANT_UNIFORM)
    assert hb.load().hac_dot_noalloc(cold._h, x.data_ptr(), 1, 1, 0, y.data_ptr(), 1, 0, None) == -7
