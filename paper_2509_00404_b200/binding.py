"""ctypes binding of the C-ABI library (include/metis.h).  Argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the library's CUDA
kernels.  Loading fails loudly when the library has not been built: there is no CPU fallback.
"""
import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# METIS_DEBUG=1 selects the debug build of the same sources (index checks on every output store of the quantizing kernels)
LIB_PATH = os.path.join(_PKG, "libmetis_b200_debug.so" if os.environ.get("METIS_DEBUG") == "1" else "libmetis_b200.so")

OK = 0
BF16, FP32 = 0, 1
ROUND_RNE, ROUND_SR = 0, 1
BLOCKS_ALONG_COLS, BLOCKS_ALONG_ROWS, BLOCKS_BOTH = 1, 2, 3
TSCALE_AMAX_SELF, TSCALE_GIVEN = 0, 1
SKETCH_FULL, SKETCH_SAMPLED = 0, 1
SF_LINEAR, SF_TILED = 0, 1
STREAM_RESIDUAL, STREAM_LEFT, STREAM_RIGHT = 0x10, 0x11, 0x12
DEV_TIMEOUT, DEV_NUMERIC, DEV_NONFINITE, DEV_INDEX = 1, 2, 4, 8

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "ALIGNMENT", 4: "WORKSPACE", 5: "ARCH", 6: "CUDA",
                7: "NONFINITE", 8: "NUMERIC", 9: "TIMEOUT"}

EXPORTED = ["metis_create", "metis_destroy", "metis_last_device_status", "metis_debug_quantile_table",
            "metis_debug_launch_count", "metis_debug_timestamp", "metis_debug_wait_timeout", "metis_debug_build", "metis_debug_index_check",
            "metis_sf_bytes", "metis_workspace_bytes", "metis_default_sample_count", "metis_quantize_nvfp4", "metis_quantize_rht_nvfp4",
            "metis_split", "metis_requantize_operand", "metis_linear_fwd", "metis_linear_fwd_static_ws", "metis_linear_bwd", "metis_gemm_nvfp4"]


class MetisError(RuntimeError):
    def __init__(self, fn, code):
        super().__init__("%s failed: METIS_ERR_%s (%d)" % (fn, STATUS_NAMES.get(code, "?"), code))
        self.code = code


class NvFp4Struct(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("tensor_scale", ctypes.c_void_p),
                ("rows", ctypes.c_int64), ("k_len", ctypes.c_int64), ("sf_layout", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


class OperandStruct(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int32), ("reserved", ctypes.c_int32), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("left", ctypes.c_void_p), ("sigma", ctypes.c_void_p), ("right", ctypes.c_void_p),
                ("left_q", NvFp4Struct), ("right_q", NvFp4Struct), ("res_by_cols", NvFp4Struct),
                ("res_by_rows", NvFp4Struct)]


_lib = None


def lib():
    """Loads the shared library (once).  Raises if it is missing: build it with `python -m paper_2509_00404_b200.build`."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("CUDA library %s not built; run `python -m paper_2509_00404_b200.build`" % LIB_PATH)
    l = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64, u32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32,
                                  ctypes.c_size_t)
    P = ctypes.POINTER
    l.metis_create.argtypes = [P(vp), ctypes.c_int]
    l.metis_destroy.argtypes = [vp]
    l.metis_last_device_status.argtypes = [vp, P(u32), vp]
    l.metis_debug_quantile_table.argtypes = [vp, vp]
    l.metis_debug_launch_count.argtypes = []
    l.metis_debug_timestamp.argtypes = [vp, vp, vp]
    l.metis_debug_wait_timeout.argtypes = [vp, u32, vp, vp]
    l.metis_debug_launch_count.restype = u64
    l.metis_debug_build.argtypes = []
    l.metis_debug_build.restype = i32
    l.metis_debug_index_check.argtypes = [vp, i64, i64, i64, vp]
    l.metis_sf_bytes.argtypes = [i64, i64, i32]
    l.metis_sf_bytes.restype = sz
    l.metis_workspace_bytes.argtypes = [i32, i64, i64, i32, i32, P(sz)]
    l.metis_default_sample_count.argtypes = [i64, i32]
    l.metis_default_sample_count.restype = i64
    l.metis_quantize_nvfp4.argtypes = [vp, vp, i32, i64, i64, i64, i32, u64, u32, i32, P(NvFp4Struct), P(NvFp4Struct),
                                       vp, sz, vp]
    l.metis_quantize_rht_nvfp4.argtypes = [vp, vp, i32, i64, i64, i64, i32, u64, u32, P(NvFp4Struct), vp, sz, vp]
    l.metis_split.argtypes = [vp, vp, i32, i64, i64, i64, i32, i32, i32, i64, u64, i32, i32, vp, P(OperandStruct), vp, vp, sz, vp]
    l.metis_requantize_operand.argtypes = [vp, vp, i32, i64, i32, u64, i32, i32, P(OperandStruct), vp, sz, vp]
    l.metis_linear_fwd.argtypes = [vp, P(OperandStruct), P(OperandStruct), vp, i32, i64, vp, sz, vp]
    l.metis_linear_fwd_static_ws.argtypes = [vp, P(OperandStruct), P(OperandStruct), vp, i32, i64, vp]
    l.metis_linear_bwd.argtypes = [vp, P(OperandStruct), P(OperandStruct), P(OperandStruct), vp, i32, i64, vp, i32,
                                   i64, vp, vp, vp, vp, sz, vp]
    l.metis_gemm_nvfp4.argtypes = [vp, P(NvFp4Struct), P(NvFp4Struct), vp, i32, i64, i32, vp]
    for name in EXPORTED:
        if name not in ("metis_sf_bytes", "metis_default_sample_count", "metis_debug_launch_count", "metis_debug_build"):
            getattr(l, name).restype = ctypes.c_int
    _lib = l
    return l


def _check(fn, code):
    if code != OK:
        raise MetisError(fn, code)


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _dtype_code(t):
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    raise TypeError("expected a bfloat16 or float32 tensor")


def debug_build():
    """True when the loaded library is the debug build (METIS_DEBUG=1)."""
    return bool(lib().metis_debug_build())


def launch_count():
    return int(lib().metis_debug_launch_count())


def sf_bytes(rows, k_len, layout):
    return lib().metis_sf_bytes(rows, k_len, layout)


def default_sample_count(rows, q):
    return lib().metis_default_sample_count(rows, q)


def workspace_bytes(op, rows, cols, k, p):
    out = ctypes.c_size_t(0)
    _check("metis_workspace_bytes", lib().metis_workspace_bytes(op, rows, cols, k, p, ctypes.byref(out)))
    return out.value


class NvFp4:
    """Device buffers of one stored (rows x k_len) NVFP4 tensor."""

    def __init__(self, rows, k_len, layout=SF_TILED, device="cuda"):
        self.rows, self.k_len, self.layout = rows, k_len, layout
        self.codes = torch.zeros((rows, k_len // 2), dtype=torch.uint8, device=device)
        self.scales = torch.zeros(max(sf_bytes(rows, k_len, layout), 16), dtype=torch.uint8, device=device)
        self.tensor_scale = torch.zeros(1, dtype=torch.float32, device=device)

    def struct(self):
        return NvFp4Struct(self.codes.data_ptr(), self.scales.data_ptr(), self.tensor_scale.data_ptr(), self.rows,
                           self.k_len, self.layout, 0)

    def linear_scales(self):
        """Scale bytes as a (rows x k_len/16) uint8 tensor on the host, whatever the device layout."""
        s = self.scales.cpu()
        nb = self.k_len // 16
        if self.layout == SF_LINEAR:
            return s[: self.rows * nb].reshape(self.rows, nb)
        r = torch.arange(self.rows).reshape(-1, 1)
        b = torch.arange(nb).reshape(1, -1)
        off = ((r // 128) * (nb // 4) + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
        return s[off]


class Operand:
    """Device buffers of one split + quantized operand (rows x cols, rank k)."""

    def __init__(self, rows, cols, k, axes=BLOCKS_BOTH, layout=SF_TILED, device="cuda"):
        self.rows, self.cols, self.k, self.axes = rows, cols, k, axes
        kk = max(k, 1)
        self.left = torch.zeros((kk, rows), dtype=torch.float32, device=device)
        self.sigma = torch.zeros(kk, dtype=torch.float32, device=device)
        self.right = torch.zeros((kk, cols), dtype=torch.float32, device=device)
        self.left_q = NvFp4(kk, rows, layout, device)
        self.right_q = NvFp4(kk, cols, layout, device)
        self.res_by_cols = NvFp4(rows, cols, layout, device) if axes & BLOCKS_ALONG_COLS else None
        self.res_by_rows = NvFp4(cols, rows, layout, device) if axes & BLOCKS_ALONG_ROWS else None

    def struct(self):
        empty = NvFp4Struct(None, None, None, 0, 0, 0, 0)
        lq, rq = self.left_q.struct(), self.right_q.struct()
        lq.rows = rq.rows = self.k
        return OperandStruct(self.k, 0, self.rows, self.cols, self.left.data_ptr(), self.sigma.data_ptr(),
                             self.right.data_ptr(), lq, rq,
                             self.res_by_cols.struct() if self.res_by_cols else empty,
                             self.res_by_rows.struct() if self.res_by_rows else empty)


class Handle:
    """A library context on one device (metis_create / metis_destroy)."""

    def __init__(self, device=0):
        self._h = ctypes.c_void_p(0)
        if not torch.cuda.is_available():
            raise RuntimeError("the Metis B200 library needs a CUDA device; there is no CPU path")
        torch.cuda.set_device(device)
        torch.cuda.current_stream()          # make sure torch's primary context exists before the library binds to it
        _check("metis_create", lib().metis_create(ctypes.byref(self._h), device))
        self.device = device
        self._ws = None

    def close(self):
        if self._h:
            lib().metis_destroy(self._h)
            self._h = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, nbytes):
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda")
        return self._ws

    def device_status(self, stream=None):
        out = ctypes.c_uint32(0)
        _check("metis_last_device_status", lib().metis_last_device_status(self._h, ctypes.byref(out), _stream_ptr(stream)))
        return out.value

    def quantile_table(self):
        import numpy as np
        buf = np.zeros(65536, dtype=np.uint16)
        _check("metis_debug_quantile_table", lib().metis_debug_quantile_table(self._h, buf.ctypes.data_as(ctypes.c_void_p)))
        return buf

    # -- metis_quantize_nvfp4 ------------------------------------------------------------------
    def quantize_nvfp4(self, x, axes=BLOCKS_ALONG_COLS, rounding=ROUND_RNE, seed=0, stream_id=STREAM_RESIDUAL,
                       tensor_scale=None, layout=SF_TILED, out=None, stream=None):
        """Returns (by_cols, by_rows) NvFp4 objects (None for an orientation not requested)."""
        rows, cols = x.shape
        if out is None:
            bc = NvFp4(rows, cols, layout) if axes & BLOCKS_ALONG_COLS else None
            br = NvFp4(cols, rows, layout) if axes & BLOCKS_ALONG_ROWS else None
        else:
            bc, br = out
        mode = TSCALE_AMAX_SELF
        if tensor_scale is not None:
            mode = TSCALE_GIVEN
            for o in (bc, br):
                if o is not None:
                    o.tensor_scale.fill_(float(tensor_scale))
        sc = bc.struct() if bc else None
        sr = br.struct() if br else None
        ws = self.workspace(256)
        _check("metis_quantize_nvfp4", lib().metis_quantize_nvfp4(
            self._h, _ptr(x), _dtype_code(x), rows, cols, x.stride(0), rounding, seed, stream_id, mode,
            ctypes.byref(sc) if bc else None, ctypes.byref(sr) if br else None, _ptr(ws), ws.numel(), _stream_ptr(stream)))
        return bc, br

    def quantize_rht_nvfp4(self, x, rounding=ROUND_SR, seed=0, stream_id=STREAM_RESIDUAL, layout=SF_TILED, out=None, stream=None):
        """metis_quantize_rht_nvfp4: random Hadamard transform of every 16-block along the columns, then NVFP4 (the
        comparison recipe).  Returns the NvFp4 object."""
        rows, cols = x.shape
        t = out if out is not None else NvFp4(rows, cols, layout)
        st = t.struct()
        ws = self.workspace(256)
        _check("metis_quantize_rht_nvfp4", lib().metis_quantize_rht_nvfp4(
            self._h, _ptr(x), _dtype_code(x), rows, cols, x.stride(0), rounding, seed, stream_id, ctypes.byref(st), _ptr(ws), ws.numel(),
            _stream_ptr(stream)))
        return t

    # -- metis_split ---------------------------------------------------------------------------
    def split(self, x, k, p, sketch=SKETCH_SAMPLED, n_sample=0, seed=0, rounding=ROUND_RNE, axes=BLOCKS_BOTH,
              out=None, want_residual=False, stream=None, src_amax=None):
        """metis_split.  src_amax: optional one-element float32 CUDA tensor holding amax|x| (saves the library's own reduction)."""
        rows, cols = x.shape
        op = out if out is not None else Operand(rows, cols, k, axes)
        dense = torch.empty((rows, cols), dtype=torch.float32, device=x.device) if want_residual else None
        plain = x.dtype == torch.bfloat16 and x.stride(0) == cols
        need = workspace_bytes(1 if plain else 4, rows, cols, k, p)
        ws = self.workspace(need)
        st = op.struct()
        _check("metis_split", lib().metis_split(self._h, _ptr(x), _dtype_code(x), rows, cols, x.stride(0), k, p, sketch, n_sample, seed, rounding,
                                                axes, _ptr(src_amax), ctypes.byref(st), _ptr(dense), _ptr(ws), ws.numel(),
                                                _stream_ptr(stream)))
        return (op, dense) if want_residual else op

    def requantize_operand(self, op, residual, rounding=ROUND_RNE, seed=0, axes=BLOCKS_BOTH, given_scale=None, stream=None):
        """metis_requantize_operand: refreshes the NVFP4 members of `op` from its stored FP32 factors and the stored
        `residual` (rows x cols, float32 or bfloat16).  given_scale: tensor scale of the residual (None = its own amax/2688)."""
        mode = TSCALE_AMAX_SELF
        if given_scale is not None:
            mode = TSCALE_GIVEN
            for o in (op.res_by_cols, op.res_by_rows):
                if o is not None:
                    o.tensor_scale.fill_(float(given_scale))
        ws = self.workspace(256)
        st = op.struct()
        _check("metis_requantize_operand", lib().metis_requantize_operand(
            self._h, _ptr(residual), _dtype_code(residual), residual.stride(0), rounding, seed, axes, mode, ctypes.byref(st),
            _ptr(ws), ws.numel(), _stream_ptr(stream)))
        return op

    # -- metis_linear_fwd / metis_linear_bwd ---------------------------------------------------
    def linear_fwd(self, x_op, w_op, out_dtype=torch.float32, out=None, stream=None):
        l, n = x_op.rows, w_op.rows
        y = out if out is not None else torch.empty((l, n), dtype=out_dtype, device="cuda")
        ws = self.workspace(workspace_bytes(2, max(l, n), max(l, n), max(x_op.k, w_op.k), 0))
        sx, sw = x_op.struct(), w_op.struct()
        _check("metis_linear_fwd", lib().metis_linear_fwd(self._h, ctypes.byref(sx), ctypes.byref(sw), _ptr(y),
                                                          _dtype_code(y), y.stride(0), _ptr(ws), ws.numel(),
                                                          _stream_ptr(stream)))
        return y

    def linear_fwd_static_ws(self, x_op, w_op, out_dtype=torch.float32, out=None, stream=None):
        """metis_linear_fwd_static_ws: forward layer for callers that cannot supply scratch memory (for example
        because a framework pool already owns all device memory).  Allocates no workspace here either."""
        y = out if out is not None else torch.empty((x_op.rows, w_op.rows), dtype=out_dtype, device="cuda")
        sx, sw = x_op.struct(), w_op.struct()
        _check("metis_linear_fwd_static_ws", lib().metis_linear_fwd_static_ws(
            self._h, ctypes.byref(sx), ctypes.byref(sw), _ptr(y), _dtype_code(y), y.stride(0), _stream_ptr(stream)))
        return y

    def linear_bwd(self, dy_op, x_op, w_op, out_dtype=torch.float32, need_dx=True, need_dw=True, out=None, stream=None,
                   factor_grads=None):
        """dx, dw of the layer.  `factor_grads`: None, or a tuple (d_left, d_sigma, d_right) of FP32 CUDA tensors
        (k x n, k, k x m; any of them None) that receive the gradients of the weight factors."""
        l, n, m = dy_op.rows, dy_op.cols, (x_op.cols if x_op is not None else w_op.cols)
        dx = dw = None
        if out is not None:
            dx, dw = out
        else:
            if need_dx:
                dx = torch.empty((l, m), dtype=out_dtype, device="cuda")
            if need_dw:
                dw = torch.empty((n, m), dtype=out_dtype, device="cuda")
        big = max(l, n, m)
        ws = self.workspace(workspace_bytes(3, big, big, max(dy_op.k, x_op.k if x_op else 0, w_op.k if w_op else 0), 0))
        sd = dy_op.struct()
        sx = x_op.struct() if x_op is not None else None
        sw = w_op.struct() if w_op is not None else None
        _check("metis_linear_bwd", lib().metis_linear_bwd(
            self._h, ctypes.byref(sd), ctypes.byref(sx) if sx else None, ctypes.byref(sw) if sw else None,
            _ptr(dx), _dtype_code(dx) if dx is not None else FP32, dx.stride(0) if dx is not None else 0,
            _ptr(dw), _dtype_code(dw) if dw is not None else FP32, dw.stride(0) if dw is not None else 0,
            *(_ptr(t) for t in (factor_grads or (None, None, None))),
            _ptr(ws), ws.numel(), _stream_ptr(stream)))
        return dx, dw

    def timestamp(self, slot, stream=None):
        """Enqueues a kernel that writes the GPU nanosecond timer into the int64 CUDA tensor element `slot`."""
        _check("metis_debug_timestamp", lib().metis_debug_timestamp(self._h, _ptr(slot), _stream_ptr(stream)))

    def index_check(self, offset, nbytes, extent, stream=None):
        """metis_debug_index_check: the debug build's store check on a made-up store (nothing is accessed)."""
        _check("metis_debug_index_check", lib().metis_debug_index_check(self._h, offset, nbytes, extent, _stream_ptr(stream)))

    def wait_timeout(self, polls=256, stream=None):
        """metis_debug_wait_timeout: runs the bounded-wait hook; returns the two per-warp words as a CUDA int32 tensor."""
        seen = torch.zeros(2, dtype=torch.int32, device="cuda")
        _check("metis_debug_wait_timeout", lib().metis_debug_wait_timeout(self._h, polls, _ptr(seen), _stream_ptr(stream)))
        return seen

    # -- metis_gemm_nvfp4 ----------------------------------------------------------------------
    def gemm_nvfp4(self, a, b, out_dtype=torch.float32, impl=0, out=None, stream=None):
        d = out if out is not None else torch.empty((a.rows, b.rows), dtype=out_dtype, device="cuda")
        sa, sb = a.struct(), b.struct()
        _check("metis_gemm_nvfp4", lib().metis_gemm_nvfp4(self._h, ctypes.byref(sa), ctypes.byref(sb), _ptr(d),
                                                          _dtype_code(d), d.stride(0), impl, _stream_ptr(stream)))
        return d
