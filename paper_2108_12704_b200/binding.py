"""ctypes binding of libhac_b200.so: the same entry points as include/hac.h, argument
marshalling only.  Every step of the product runs in the library's CUDA kernels; there is
no CPU fallback: if the library is missing or a call fails, an exception is raised."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

QUANT_NONE, QUANT_KMEANS, QUANT_UNIFORM, QUANT_GRID, QUANT_PWS = 0, 1, 2, 3, 4


class HacError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: status {status} ({detail})")


class BuildParams(C.Structure):
    _fields_ = [("sparsity", C.c_double), ("k", C.c_uint32), ("quantizer", C.c_uint32),
                ("kmeans_iters", C.c_uint32), ("seg_symbols", C.c_uint32), ("seed", C.c_uint64),
                ("ri_bits", C.c_uint32), ("reserved", C.c_uint32)]


class SizeReport(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ("n", "m", "nnz", "symbols", "stream_bits", "stream_words", "stream_bytes", "pad_bytes",
                 "codebook_bytes", "code_len_bytes", "ri_bytes", "cb_bytes", "offset_index_bytes",
                 "total_bytes", "paper_bits")] + \
               [(n, C.c_double) for n in ("bound_bits", "entropy", "avg_code_len")] + \
               [(n, C.c_uint32) for n in ("k_eff", "max_code_len", "min_code_len", "seg_symbols", "ri_bits",
                                          "units")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class Epilogue(C.Structure):
    _fields_ = [("bias", C.c_void_p), ("relu", C.c_uint32), ("reserved", C.c_uint32)]


class Layer(C.Structure):
    _fields_ = [("hac", C.c_void_p), ("shac", C.c_void_p), ("epilogue", Epilogue)]


class UnifiedLayer(C.Structure):
    _fields_ = [("W", C.c_void_p), ("n", C.c_int64), ("m", C.c_int64), ("ldw", C.c_int64), ("sparse", C.c_int32),
                ("reserved", C.c_int32)]


class HostView(C.Structure):
    _fields_ = [("n", C.c_int64), ("m", C.c_int64), ("k_eff", C.c_uint32), ("seg_symbols", C.c_uint32),
                ("codebook", C.POINTER(C.c_float)), ("code_len", C.POINTER(C.c_uint8)),
                ("codes", C.POINTER(C.c_uint32)), ("counts", C.POINTER(C.c_int64)),
                ("stream", C.POINTER(C.c_uint32)),
                ("stream_bits", C.c_int64), ("stream_words", C.c_int64), ("stream_pad_words", C.c_int64),
                ("units", C.c_uint32), ("segs_per_col", C.c_uint32),
                ("seg_bit_off", C.POINTER(C.c_uint64)), ("sub_bits", C.POINTER(C.c_uint16))]


class SparseHostView(C.Structure):
    _fields_ = [("base", HostView), ("nnz", C.c_int64), ("ri_bits", C.c_uint32), ("ri", C.c_void_p),
                ("cb", C.POINTER(C.c_uint32)), ("seg_first", C.POINTER(C.c_uint32)),
                ("seg_col", C.POINTER(C.c_uint32))]


_lib = None

# every symbol include/hac.h declares
EXPORTS = (
    "hac_build", "shac_build", "hac_sizes", "shac_sizes", "hac_export", "shac_export",
    "hac_decode_host", "shac_decode_host", "hac_serialize_bytes", "shac_serialize_bytes", "hac_serialize",
    "shac_serialize", "hac_deserialize", "shac_deserialize", "hac_device_bytes", "shac_device_bytes", "hac_upload",
    "shac_upload", "hac_attach", "shac_attach", "hac_workspace_bytes", "shac_workspace_bytes", "hac_dot",
    "shac_dot", "hac_dot_noalloc", "hac_dot_layer", "shac_dot_layer", "hac_chain", "hac_dot_host_scratch_bytes", "shac_dot_host_scratch_bytes", "hac_dot_host",
    "shac_dot_host", "hac_dot_host_async", "shac_dot_host_async", "hac_debug_decode", "shac_debug_decode",
    "hac_debug_table_lookup", "shac_debug_table_lookup", "hac_last_launch_count",
    "shac_last_launch_count", "hac_free", "shac_free", "hac_status_string", "hac_last_cuda_error",
    "hac_index_map_encode", "hac_index_map_dot", "shac_csc_encode", "shac_csc_dot", "hac_build_unified", "hac_lost_waits",
)


def library_path() -> str:
    return _build.LIB


def load():
    """Load the shared library (built in-tree by build.build()); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise HacError(-1, "libhac_b200.so is not built", "run paper_2108_12704_b200.build.build()")
    lib = C.CDLL(path)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    fp = C.c_void_p
    for kind in ("hac", "shac"):
        getattr(lib, f"{kind}_build").argtypes = [fp, i64, i64, i64, C.POINTER(BuildParams), C.POINTER(vp)]
        getattr(lib, f"{kind}_sizes").argtypes = [vp, C.POINTER(SizeReport)]
        getattr(lib, f"{kind}_export").argtypes = [vp, vp]
        getattr(lib, f"{kind}_decode_host").argtypes = [vp, fp, i64]
        getattr(lib, f"{kind}_serialize_bytes").argtypes = [vp, C.POINTER(sz)]
        getattr(lib, f"{kind}_serialize").argtypes = [vp, vp, sz]
        getattr(lib, f"{kind}_deserialize").argtypes = [vp, sz, C.POINTER(vp)]
        getattr(lib, f"{kind}_device_bytes").argtypes = [vp, C.POINTER(sz)]
        getattr(lib, f"{kind}_upload").argtypes = [vp, vp, sz, vp]
        getattr(lib, f"{kind}_attach").argtypes = [vp, vp, sz]
        getattr(lib, f"{kind}_workspace_bytes").argtypes = [vp, i64, C.POINTER(sz)]
        getattr(lib, f"{kind}_dot").argtypes = [vp, fp, i64, i64, i64, fp, i64, i64, vp, sz, vp]
        getattr(lib, f"{kind}_dot_layer").argtypes = [vp, fp, i64, i64, i64, fp, i64, i64, C.POINTER(Epilogue), vp, sz, vp]
        getattr(lib, f"{kind}_dot_host_scratch_bytes").argtypes = [vp, i64, C.POINTER(sz)]
        getattr(lib, f"{kind}_dot_host").argtypes = [vp, fp, i64, fp, vp, sz, vp]
        getattr(lib, f"{kind}_dot_host_async").argtypes = [vp, fp, i64, fp, vp, sz, vp]
        getattr(lib, f"{kind}_debug_decode").argtypes = [vp, fp, vp]
        getattr(lib, f"{kind}_debug_table_lookup").argtypes = [vp, C.c_uint32, C.POINTER(C.c_float), C.POINTER(C.c_uint32),
                                                               C.POINTER(C.c_int), C.POINTER(C.c_int)]
        getattr(lib, f"{kind}_last_launch_count").argtypes = [vp]
        getattr(lib, f"{kind}_free").argtypes = [vp]
        getattr(lib, f"{kind}_free").restype = None
    lib.hac_dot_noalloc.argtypes = [vp, fp, i64, i64, i64, fp, i64, i64, vp]
    lib.hac_chain.argtypes = [C.POINTER(Layer), C.c_int, fp, i64, fp, fp, fp, sz, vp, sz, vp]
    lib.hac_index_map_encode.argtypes = [fp, i64, i64, i64, C.c_int, vp, fp, C.POINTER(C.c_int)]
    lib.hac_index_map_dot.argtypes = [vp, C.c_int, fp, C.c_int, i64, i64, fp, i64, i64, i64, fp, i64, i64, vp]
    lib.shac_csc_encode.argtypes = [fp, i64, i64, i64, fp, vp, vp, i64, C.POINTER(i64)]
    lib.shac_csc_dot.argtypes = [fp, vp, vp, i64, i64, fp, i64, i64, i64, fp, i64, i64, vp]
    lib.hac_build_unified.argtypes = [C.POINTER(UnifiedLayer), C.c_int, C.POINTER(BuildParams), C.POINTER(vp)]
    lib.hac_lost_waits.argtypes = [C.POINTER(C.c_uint)]
    lib.hac_status_string.argtypes = [C.c_int]
    lib.hac_status_string.restype = C.c_char_p
    lib.hac_last_cuda_error.restype = C.c_char_p
    _lib = lib
    return lib


def _check(status: int, what: str):
    if status != 0:
        lib = load()
        detail = lib.hac_status_string(status).decode()
        if status == -9:
            detail += ": " + lib.hac_last_cuda_error().decode()
        raise HacError(status, what, detail)


def _arr(ptr, count, dtype):
    if count == 0:
        return np.zeros(0, dtype=dtype)
    return np.ctypeslib.as_array(ptr, shape=(count,)).copy().astype(dtype, copy=False)


class Format:
    """A built HAC (kind='hac') or sHAC (kind='shac') format; thin wrapper over the opaque handle."""

    def __init__(self, kind: str, W: np.ndarray, sparsity=0.0, k=32, quantizer=QUANT_KMEANS, kmeans_iters=20,
                 seed=0, seg_symbols=0, ri_bits=0):
        assert kind in ("hac", "shac")
        self.kind = kind
        self._lib = load()
        self._h = C.c_void_p()
        W = np.ascontiguousarray(W, dtype=np.float32)
        if W.ndim != 2:
            raise ValueError("W must be a matrix")
        p = BuildParams(float(sparsity), int(k), int(quantizer), int(kmeans_iters), int(seg_symbols), int(seed),
                        int(ri_bits), 0)
        fn = getattr(self._lib, f"{kind}_build")
        _check(fn(W.ctypes.data, W.shape[0], W.shape[1], W.shape[1], C.byref(p), C.byref(self._h)),
               f"{kind}_build")
        self.n, self.m = W.shape
        self._device_buffer = None      # keeps the torch tensor alive

    def _fn(self, name):
        return getattr(self._lib, f"{self.kind}_{name}")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._fn("free")(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- host side -----------------------------------------------------------------------
    def sizes(self) -> dict:
        r = SizeReport()
        _check(self._fn("sizes")(self._h, C.byref(r)), "sizes")
        return r.as_dict()

    def export(self) -> dict:
        """Copies of every array of the format (numpy)."""
        if self.kind == "hac":
            v = HostView()
            _check(self._lib.hac_export(self._h, C.byref(v)), "hac_export")
            base, out = v, {}
        else:
            sv = SparseHostView()
            _check(self._lib.shac_export(self._h, C.byref(sv)), "shac_export")
            base = sv.base
            out = dict(nnz=sv.nnz, ri_bits=sv.ri_bits,
                       cb=_arr(sv.cb, base.m + 1, np.uint32), seg_first=_arr(sv.seg_first, base.m + 1, np.uint32),
                       seg_col=_arr(sv.seg_col, base.units, np.uint32))
            rt = C.c_uint16 if sv.ri_bits == 16 else C.c_uint32
            out["ri"] = _arr(C.cast(sv.ri, C.POINTER(rt)), sv.nnz, np.uint16 if sv.ri_bits == 16 else np.uint32)
        k = base.k_eff
        out.update(n=base.n, m=base.m, k_eff=k, seg_symbols=base.seg_symbols,
                   codebook=_arr(base.codebook, k, np.float32), code_len=_arr(base.code_len, k, np.uint8),
                   codes=_arr(base.codes, k, np.uint32), counts=_arr(base.counts, k, np.int64),
                   stream=_arr(base.stream, base.stream_words + base.stream_pad_words, np.uint32),
                   stream_bits=base.stream_bits, stream_words=base.stream_words,
                   stream_pad_words=base.stream_pad_words, units=base.units, segs_per_col=base.segs_per_col,
                   seg_bit_off=_arr(base.seg_bit_off, base.units, np.uint64),
                   sub_bits=_arr(base.sub_bits, base.units * 32, np.uint16))
        return out

    def serialize(self) -> bytes:
        """The format as one byte string (*_serialize of the C ABI)."""
        n = C.c_size_t()
        _check(self._fn("serialize_bytes")(self._h, C.byref(n)), "serialize_bytes")
        buf = (C.c_ubyte * n.value)()
        _check(self._fn("serialize")(self._h, buf, n.value), "serialize")
        return bytes(buf)

    @classmethod
    def deserialize(cls, kind: str, blob: bytes) -> "Format":
        """A handle from a byte string written by serialize() (*_deserialize of the C ABI)."""
        assert kind in ("hac", "shac")
        self = cls.__new__(cls)
        self.kind = kind
        self._lib = load()
        self._h = C.c_void_p()
        self._device_buffer = None
        buf = (C.c_ubyte * len(blob)).from_buffer_copy(blob)
        _check(getattr(self._lib, f"{kind}_deserialize")(buf, len(blob), C.byref(self._h)), f"{kind}_deserialize")
        sz = self.sizes()
        self.n, self.m = sz["n"], sz["m"]
        return self

    def decode_host(self) -> np.ndarray:
        Wq = np.empty((self.n, self.m), dtype=np.float32)
        _check(self._fn("decode_host")(self._h, Wq.ctypes.data, self.m), "decode_host")
        return Wq

    # ---- device side (torch supplies memory and streams) ---------------------------------
    def device_bytes(self) -> int:
        s = C.c_size_t()
        _check(self._fn("device_bytes")(self._h, C.byref(s)), "device_bytes")
        return s.value

    def upload(self, device="cuda"):
        import torch
        buf = torch.empty(self.device_bytes() + 256, dtype=torch.uint8, device=device)
        off = (-buf.data_ptr()) % 256
        self._device_buffer = buf
        self._image = buf[off:off + self.device_bytes()]
        st = torch.cuda.current_stream().cuda_stream
        _check(self._fn("upload")(self._h, self._image.data_ptr(), self._image.numel(), st), "upload")
        return self

    def image(self):
        """The device image as a torch uint8 tensor (for replication)."""
        return self._image

    def attach(self, image):
        """Use a byte-identical copy of the uploaded image that lives in `image` (torch uint8, 256-byte aligned)."""
        _check(self._fn("attach")(self._h, image.data_ptr(), image.numel()), "attach")
        self._image = image
        return self

    def workspace_bytes(self, batch: int) -> int:
        s = C.c_size_t()
        _check(self._fn("workspace_bytes")(self._h, int(batch), C.byref(s)), "workspace_bytes")
        return s.value

    def dot(self, x, y=None, workspace=None, layout="nb", bias=None, relu=False):
        """y = W^T x on the device.  x: torch float32 CUDA tensor, [n] or, for a batch, [n, B]
        (layout 'nb') or [B, n] (layout 'bn').  Returns y shaped [m], [m, B] or [B, m] alike.
        With `bias` (torch float32 CUDA tensor [m]) and / or relu=True the call goes through *_dot_layer:
        y = act(W^T x + bias)."""
        import torch
        assert x.is_cuda and x.dtype == torch.float32
        if x.dim() == 1:
            B, xs_i, xs_b = 1, x.stride(0), 0
            yshape = (self.m,)
        elif layout == "nb":
            B, xs_i, xs_b = x.shape[1], x.stride(0), x.stride(1)
            yshape = (self.m, B)
        else:
            B, xs_i, xs_b = x.shape[0], x.stride(1), x.stride(0)
            yshape = (B, self.m)
        if y is None:
            y = torch.empty(yshape, dtype=torch.float32, device=x.device)
        if y.dim() == 1:
            ys_j, ys_b = y.stride(0), 0
        elif layout == "nb":
            ys_j, ys_b = y.stride(0), y.stride(1)
        else:
            ys_j, ys_b = y.stride(1), y.stride(0)
        need = self.workspace_bytes(B)
        if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
            workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        wp = workspace.data_ptr() if workspace is not None else None
        wb = workspace.numel() * workspace.element_size() if workspace is not None else 0
        st = torch.cuda.current_stream().cuda_stream
        if bias is None and not relu:
            _check(self._fn("dot")(self._h, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b, wp, wb, st), "dot")
        else:
            epi = Epilogue(bias.data_ptr() if bias is not None else None, 1 if relu else 0, 0)
            _check(self._fn("dot_layer")(self._h, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b, C.byref(epi),
                                         wp, wb, st), "dot_layer")
        return y

    def dot_noalloc(self, x, y=None, layout="nb"):
        """hac_dot_noalloc of the C ABI: like dot(), but the partial sums go to the buffer built into
        the library instead of a workspace tensor (HAC only; refused with status -8 if they do not
        fit).  For hosts that are not allowed to allocate device memory; y is still the caller's, and
        is only created here as a convenience when it is not passed."""
        import torch
        assert self.kind == "hac" and x.is_cuda and x.dtype == torch.float32
        if x.dim() == 1:
            B, xs_i, xs_b, yshape = 1, x.stride(0), 0, (self.m,)
        elif layout == "nb":
            B, xs_i, xs_b, yshape = x.shape[1], x.stride(0), x.stride(1), (self.m, x.shape[1])
        else:
            B, xs_i, xs_b, yshape = x.shape[0], x.stride(1), x.stride(0), (x.shape[0], self.m)
        if y is None:
            y = torch.empty(yshape, dtype=torch.float32, device=x.device)
        if y.dim() == 1:
            ys_j, ys_b = y.stride(0), 0
        elif layout == "nb":
            ys_j, ys_b = y.stride(0), y.stride(1)
        else:
            ys_j, ys_b = y.stride(1), y.stride(0)
        st = torch.cuda.current_stream().cuda_stream
        _check(self._lib.hac_dot_noalloc(self._h, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b, st),
               "hac_dot_noalloc")
        return y

    def dot_host_scratch_bytes(self, batch: int) -> int:
        s = C.c_size_t()
        _check(self._fn("dot_host_scratch_bytes")(self._h, int(batch), C.byref(s)), "dot_host_scratch_bytes")
        return s.value

    def dot_host(self, X_host, Y_host, scratch, wait=True):
        """Host-to-host product: X_host [B, n] and Y_host [B, m] are CPU float32 tensors (pinned for
        speed) or numpy arrays, scratch a torch uint8 CUDA tensor.  Waits for completion; with
        wait=False (the *_dot_host_async entry points) the work is only enqueued on the current stream."""
        import torch
        B = X_host.shape[0] if X_host.ndim == 2 else 1
        xp = X_host.data_ptr() if hasattr(X_host, "data_ptr") else X_host.ctypes.data
        yp = Y_host.data_ptr() if hasattr(Y_host, "data_ptr") else Y_host.ctypes.data
        st = torch.cuda.current_stream().cuda_stream
        name = "dot_host" if wait else "dot_host_async"
        _check(self._fn(name)(self._h, xp, B, yp, scratch.data_ptr(), scratch.numel(), st), name)
        return Y_host

    def debug_decode(self):
        """TEST ONLY: the decoder's output as a device tensor (hac: [m, n] = Wq^T; shac: [nnz])."""
        import torch
        count = self.n * self.m if self.kind == "hac" else self.sizes()["nnz"]
        out = torch.zeros(max(count, 1), dtype=torch.float32, device=self._image.device)
        st = torch.cuda.current_stream().cuda_stream
        _check(self._fn("debug_decode")(self._h, out.data_ptr(), st), "debug_decode")
        out = out[:count]
        return out.view(self.m, self.n) if self.kind == "hac" else out

    def debug_table_lookup(self, window: int):
        """TEST ONLY: (value, length, kind, never_unresolved) of the kernels' first-level table for a 32-bit window."""
        v, l, k, nu = C.c_float(), C.c_uint32(), C.c_int(), C.c_int()
        _check(self._fn("debug_table_lookup")(self._h, C.c_uint32(window & 0xffffffff), C.byref(v), C.byref(l),
                                              C.byref(k), C.byref(nu)), "debug_table_lookup")
        return v.value, l.value, k.value, bool(nu.value)

    def last_launch_count(self) -> int:
        return self._fn("last_launch_count")(self._h)


def chain(layers, x, y=None, workspace=None):
    """hac_chain of the C ABI: `layers` is a list of (Format, bias or None, relu) evaluated one after the
    other on the current stream; x is a torch float32 CUDA tensor [n0] or [n0, B] (inputs of a batch
    contiguous), the result [m_last] or [m_last, B].  Returns (y, launches of the whole chain)."""
    import torch
    lib = load()
    B = 1 if x.dim() == 1 else x.shape[1]
    assert x.is_contiguous() and x.dtype == torch.float32
    arr = (Layer * len(layers))()
    for i, (fmt, bias, relu) in enumerate(layers):
        arr[i].hac = fmt._h if fmt.kind == "hac" else None
        arr[i].shac = fmt._h if fmt.kind == "shac" else None
        arr[i].epilogue = Epilogue(bias.data_ptr() if bias is not None else None, 1 if relu else 0, 0)
    last = layers[-1][0]
    if y is None:
        y = torch.empty((last.m,) if x.dim() == 1 else (last.m, B), dtype=torch.float32, device=x.device)
    widest = max([f.m for f, _, _ in layers[:-1]] + [1]) * B
    acts = torch.empty((2, widest), dtype=torch.float32, device=x.device)
    need = max(f.workspace_bytes(B) for f, _, _ in layers)
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=x.device)
    st = torch.cuda.current_stream().cuda_stream
    _check(lib.hac_chain(arr, len(layers), x.data_ptr(), B, y.data_ptr(), acts[0].data_ptr(), acts[1].data_ptr(), widest,
                         workspace.data_ptr(), workspace.numel(), st), "hac_chain")
    return y, last.last_launch_count()


def lost_waits() -> int:
    """hac_lost_waits of the C ABI."""
    n = C.c_uint()
    _check(load().hac_lost_waits(C.byref(n)), "hac_lost_waits")
    return n.value


def build_unified(layers, sparsity=0.0, k=32, quantizer=QUANT_KMEANS, kmeans_iters=20, seed=0, seg_symbols=0, ri_bits=0):
    """hac_build_unified of the C ABI: `layers` is a list of (kind, W); all matrices are quantized together and share one
    code.  Returns one Format per layer."""
    lib = load()
    mats = [np.ascontiguousarray(W, dtype=np.float32) for _, W in layers]
    arr = (UnifiedLayer * len(layers))()
    for i, ((kind, _), W) in enumerate(zip(layers, mats)):
        assert kind in ("hac", "shac") and W.ndim == 2
        arr[i] = UnifiedLayer(W.ctypes.data, W.shape[0], W.shape[1], W.shape[1], 1 if kind == "shac" else 0, 0)
    p = BuildParams(float(sparsity), int(k), int(quantizer), int(kmeans_iters), int(seg_symbols), int(seed), int(ri_bits), 0)
    out = (C.c_void_p * len(layers))()
    _check(lib.hac_build_unified(arr, len(layers), C.byref(p), out), "hac_build_unified")
    fmts = []
    for (kind, _), W, h in zip(layers, mats, out):
        f = Format.__new__(Format)
        f.kind, f._lib, f._h, f._device_buffer = kind, lib, C.c_void_p(h), None
        f.n, f.m = W.shape
        fmts.append(f)
    return fmts


def _dot_strides(x, y, m, layout):
    """(B, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b) for the x / y conventions of Format.dot."""
    import torch
    assert x.is_cuda and x.dtype == torch.float32
    if x.dim() == 1:
        B, xs_i, xs_b, yshape = 1, x.stride(0), 0, (m,)
    elif layout == "nb":
        B, xs_i, xs_b, yshape = x.shape[1], x.stride(0), x.stride(1), (m, x.shape[1])
    else:
        B, xs_i, xs_b, yshape = x.shape[0], x.stride(1), x.stride(0), (x.shape[0], m)
    if y is None:
        y = torch.empty(yshape, dtype=torch.float32, device=x.device)
    if y.dim() == 1:
        ys_j, ys_b = y.stride(0), 0
    elif layout == "nb":
        ys_j, ys_b = y.stride(0), y.stride(1)
    else:
        ys_j, ys_b = y.stride(1), y.stride(0)
    return B, xs_i, xs_b, y, ys_j, ys_b


class IndexMap:
    """hac_index_map_* of the C ABI (Sect. III-C.1): encode on the host, keep the arrays in device tensors, multiply."""

    def __init__(self, Wq: np.ndarray, index_bits: int = 8):
        lib = load()
        Wq = np.ascontiguousarray(Wq, dtype=np.float32)
        self.n, self.m, self.index_bits = Wq.shape[0], Wq.shape[1], int(index_bits)
        self.index = np.empty(self.n * self.m, dtype=np.uint8 if index_bits == 8 else np.uint16)
        codebook = np.zeros(1 << index_bits, dtype=np.float32)
        k = C.c_int()
        _check(lib.hac_index_map_encode(Wq.ctypes.data, self.n, self.m, Wq.strides[0] // 4, self.index_bits,
                                        self.index.ctypes.data, codebook.ctypes.data, C.byref(k)), "index_map_encode")
        self.k = k.value
        self.codebook = codebook[:self.k].copy()
        self._dev = None

    def psi(self) -> float:
        return self.index_bits / 32.0 + self.k / (self.n * self.m)

    def upload(self, device="cuda"):
        import torch
        self._dev = (torch.from_numpy(self.index.view(np.uint8)).to(device), torch.from_numpy(self.codebook).to(device))
        return self

    def dot(self, x, y=None, layout="nb"):
        import torch
        if self._dev is None:
            raise HacError(-7, "index_map_dot", "not uploaded")
        B, xs_i, xs_b, y, ys_j, ys_b = _dot_strides(x, y, self.m, layout)
        _check(load().hac_index_map_dot(self._dev[0].data_ptr(), self.index_bits, self._dev[1].data_ptr(), self.k, self.n,
                                        self.m, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b,
                                        torch.cuda.current_stream().cuda_stream), "index_map_dot")
        return y


class Csc:
    """shac_csc_* of the C ABI (Sect. IV-A): nz, ri, cb built on the host, kept in device tensors, multiplied."""

    def __init__(self, Wq: np.ndarray):
        lib = load()
        Wq = np.ascontiguousarray(Wq, dtype=np.float32)
        self.n, self.m = Wq.shape
        q = C.c_int64()
        ld = Wq.strides[0] // 4
        _check(lib.shac_csc_encode(Wq.ctypes.data, self.n, self.m, ld, None, None, None, 0, C.byref(q)), "csc_encode")
        self.q = q.value
        self.nz = np.empty(max(self.q, 1), dtype=np.float32)
        self.ri = np.empty(max(self.q, 1), dtype=np.uint32)
        self.cb = np.empty(self.m + 1, dtype=np.uint32)
        _check(lib.shac_csc_encode(Wq.ctypes.data, self.n, self.m, ld, self.nz.ctypes.data, self.ri.ctypes.data,
                                   self.cb.ctypes.data, self.q, C.byref(q)), "csc_encode")
        self.nz, self.ri = self.nz[:self.q], self.ri[:self.q]
        self._dev = None

    def psi(self) -> float:
        return (2 * self.q + self.m + 1) / (self.n * self.m)

    def upload(self, device="cuda"):
        import torch
        as_i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).to(device)
        self._dev = (torch.from_numpy(np.ascontiguousarray(self.nz)).to(device), as_i32(self.ri), as_i32(self.cb))
        return self

    def dot(self, x, y=None, layout="nb"):
        import torch
        if self._dev is None:
            raise HacError(-7, "csc_dot", "not uploaded")
        B, xs_i, xs_b, y, ys_j, ys_b = _dot_strides(x, y, self.m, layout)
        nz, ri, cb = self._dev
        _check(load().shac_csc_dot(nz.data_ptr() if self.q else None, ri.data_ptr() if self.q else None, cb.data_ptr(),
                                   self.n, self.m, x.data_ptr(), B, xs_i, xs_b, y.data_ptr(), ys_j, ys_b,
                                   torch.cuda.current_stream().cuda_stream), "csc_dot")
        return y
