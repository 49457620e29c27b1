"""Thin Python face of the C-ABI library (include/zipml.h): argument marshalling only.

torch supplies device memory and streams; every step of the path runs in the library's CUDA
kernels.  The functions mirror the C names.  There is no fallback: if the shared library cannot be
loaded, or a call reports an error, a ZipmlError is raised.
"""
import ctypes as C
import os

import torch

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NONFINITE, ERR_CUDA, ERR_TIMEOUT, ERR_WORKSPACE = -1, -2, -3, -4, -5, -6
LEVELS_UNIFORM, LEVELS_TABLE = 0, 1
LOSS_DENSE, LOSS_CODES = 0, 1
LAYOUT_ROWS, LAYOUT_COLUMN_BLOCKS = 0, 1
GRID_RANGE, GRID_SYMMETRIC = 0, 1
NORM_L2, NORM_LINF = 0, 1
REG_NONE, REG_L2, REG_L1, REG_NONNEG, REG_LSSVM = 0, 1, 2, 3, 4
ENGINE_AUTO, ENGINE_STEPWISE, ENGINE_PERSISTENT, ENGINE_RING, ENGINE_LEAN, ENGINE_CLUSTER, ENGINE_STREAM, ENGINE_COLUMN = 0, 1, 2, 3, 4, 5, 6, 7

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "libzipml.so")
EXPORTS = ["zipml_up_row_bytes", "zipml_shared_base_encode", "zipml_shared_base_decode", "zipml_loss_shared_base",
           "zipml_sgd_epoch_shared_base", "zipml_sgd_apply_gradient", "zipml_quantize_draw", "zipml_poly_rows", "zipml_weighted_plane_mean", "zipml_column_blocks_bytes", "zipml_convert_layout", "zipml_create", "zipml_destroy", "zipml_sync", "zipml_kernel_launches", "zipml_last_engine", "zipml_barrier_latency", "zipml_wait_probe", "zipml_strerror", "zipml_row_bytes", "zipml_quantize",
           "zipml_optimal_levels", "zipml_sgd_epoch", "zipml_loss", "zipml_train_host",
           "zipml_loss_codes_static"]


class ZipmlError(RuntimeError):
    def __init__(self, code, what=""):
        self.code = code
        try:
            msg = lib().zipml_strerror(code).decode()
        except Exception:  # the library itself may be what is missing
            msg = "?"
        super().__init__(f"{what}: status {code} ({msg})")


class CDataset(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("bits", C.c_int32), ("level_mode", C.c_int32), ("layout", C.c_int32),
                ("m", C.c_int64), ("n", C.c_int64), ("row_bytes", C.c_int64),
                ("plane1", C.c_void_p), ("plane2", C.c_void_p),
                ("feat_lo", C.c_void_p), ("feat_step", C.c_void_p), ("levels", C.c_void_p)]


class CSharedBase(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("bits", C.c_int32), ("m", C.c_int64), ("n", C.c_int64),
                ("row_bytes", C.c_int64), ("up_row_bytes", C.c_int64), ("base", C.c_void_p), ("up1", C.c_void_p),
                ("up2", C.c_void_p), ("feat_lo", C.c_void_p), ("feat_step", C.c_void_p)]


class CSgdParams(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("model_bits", C.c_int32), ("grad_bits", C.c_int32), ("engine", C.c_int32),
                ("batch", C.c_int64), ("epoch", C.c_int64), ("first_step", C.c_int64), ("num_steps", C.c_int64),
                ("seed", C.c_uint64), ("batch_order", C.c_void_p), ("lr", C.c_float),
                ("grid_feature_parts", C.c_int32), ("grid_row_parts", C.c_int32), ("trace_steps", C.c_int32),
                ("trace", C.c_void_p), ("reg", C.c_int32), ("reg_param", C.c_float),
                ("model_out", C.c_void_p), ("cluster_contraction", C.c_int32), ("stream_prefetch", C.c_int32),
                ("column_chunk_rows", C.c_int32), ("vector_norm", C.c_int32)]


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1611_05402_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        L.zipml_create.argtypes = [C.POINTER(vp), C.c_int, vp]
        L.zipml_destroy.argtypes = [vp]
        L.zipml_sync.argtypes = [vp]
        L.zipml_kernel_launches.argtypes = [vp]
        L.zipml_kernel_launches.restype = i64
        L.zipml_last_engine.argtypes = [vp]
        L.zipml_last_engine.restype = C.c_int32
        L.zipml_barrier_latency.argtypes = [vp, i32, i32, i32, vp]
        L.zipml_wait_probe.argtypes = [vp, i64]
        L.zipml_strerror.argtypes = [C.c_int]
        L.zipml_strerror.restype = C.c_char_p
        L.zipml_row_bytes.argtypes = [i64, i32]
        L.zipml_row_bytes.restype = i64
        L.zipml_column_blocks_bytes.argtypes = [i64, i64]
        L.zipml_column_blocks_bytes.restype = i64
        L.zipml_convert_layout.argtypes = [vp, C.POINTER(CDataset), i32, vp, vp]
        L.zipml_up_row_bytes.argtypes = [i64]
        L.zipml_up_row_bytes.restype = i64
        L.zipml_shared_base_encode.argtypes = [vp, C.POINTER(CDataset), C.POINTER(CSharedBase)]
        L.zipml_shared_base_decode.argtypes = [vp, C.POINTER(CSharedBase), vp, vp]
        L.zipml_loss_shared_base.argtypes = [vp, C.POINTER(CSharedBase), vp, vp, vp]
        L.zipml_sgd_epoch_shared_base.argtypes = [vp, C.POINTER(CSharedBase), vp, vp, C.POINTER(CSgdParams), vp]
        L.zipml_sgd_apply_gradient.argtypes = [vp, vp, vp, C.c_int64, C.POINTER(CSgdParams), C.c_int64, vp]
        L.zipml_quantize_draw.argtypes = [vp, vp, i64, i64, i64, C.c_int32, C.c_int32, vp, C.c_uint64, C.c_uint32, C.c_int32, vp, vp, i64,
                                          vp, vp]
        L.zipml_poly_rows.argtypes = [vp, C.POINTER(CDataset), vp, C.c_int32, vp, vp, vp, vp]
        L.zipml_weighted_plane_mean.argtypes = [vp, C.POINTER(CDataset), vp, vp, vp]
        L.zipml_quantize.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, u64, vp, vp, i64, vp, vp]
        L.zipml_optimal_levels.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, vp]
        L.zipml_sgd_epoch.argtypes = [vp, C.POINTER(CDataset), vp, vp, C.POINTER(CSgdParams), vp]
        L.zipml_loss.argtypes = [vp, i32, vp, i64, i64, i64, C.POINTER(CDataset), vp, vp, vp]
        L.zipml_train_host.argtypes = [vp, vp, i64, i64, i64, vp, vp, i32, i32, i32, u64, C.POINTER(CSgdParams), i32, i32,
                                       vp]
        L.zipml_loss_codes_static.argtypes = [C.c_int, vp, C.POINTER(CDataset), vp, vp, vp]
        _lib = L
    return _lib


def _check(rc, what):
    if rc != OK:
        raise ZipmlError(rc, what)


def _ptr(t, dtype=None, device=None):
    if t is None:
        return None
    assert t.is_contiguous(), "tensor must be contiguous"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    if device is not None:
        assert t.device == device, f"expected a tensor on {device}, got {t.device}"
    return C.c_void_p(t.data_ptr())


class Dataset:
    """Two packed planes plus scales/levels, all torch tensors on the context's device."""

    def __init__(self, plane1, plane2, m, n, bits, level_mode, feat_lo, feat_step, levels, layout=LAYOUT_ROWS,
                 row_bytes=None):
        self.plane1, self.plane2 = plane1, plane2
        self.m, self.n, self.bits, self.level_mode, self.layout = m, n, bits, level_mode, layout
        self.row_bytes = plane1.shape[1] if row_bytes is None else row_bytes
        self.feat_lo, self.feat_step, self.levels = feat_lo, feat_step, levels

    def c_struct(self):
        d = CDataset()
        d.struct_size = C.sizeof(CDataset)
        d.bits, d.level_mode, d.m, d.n, d.row_bytes = self.bits, self.level_mode, self.m, self.n, self.row_bytes
        d.layout = self.layout
        d.plane1, d.plane2 = self.plane1.data_ptr(), self.plane2.data_ptr()
        d.feat_lo = self.feat_lo.data_ptr() if self.feat_lo is not None else None
        d.feat_step = self.feat_step.data_ptr() if self.feat_step is not None else None
        d.levels = self.levels.data_ptr() if self.levels is not None else None
        return d

    @property
    def packed_bytes(self):
        """Bytes one epoch has to read: both planes and the labels."""
        return 2 * self.m * self.row_bytes + 4 * self.m


class SharedBase:
    """Base plane plus two one-bit planes (see zipml_shared_base), all torch tensors on the context's device."""

    def __init__(self, base, up1, up2, m, n, bits, feat_lo, feat_step):
        self.base, self.up1, self.up2, self.m, self.n, self.bits = base, up1, up2, m, n, bits
        self.row_bytes, self.up_row_bytes = base.shape[1], up1.shape[1]
        self.feat_lo, self.feat_step = feat_lo, feat_step

    def c_struct(self):
        d = CSharedBase()
        d.struct_size = C.sizeof(CSharedBase)
        d.bits, d.m, d.n, d.row_bytes, d.up_row_bytes = self.bits, self.m, self.n, self.row_bytes, self.up_row_bytes
        d.base, d.up1, d.up2 = self.base.data_ptr(), self.up1.data_ptr(), self.up2.data_ptr()
        d.feat_lo = self.feat_lo.data_ptr() if self.feat_lo is not None else None
        d.feat_step = self.feat_step.data_ptr() if self.feat_step is not None else None
        return d

    @property
    def packed_bytes(self):
        """Bytes of the three planes and the labels."""
        return self.m * (self.row_bytes + 2 * self.up_row_bytes) + 4 * self.m


class Context:
    """zipml_create / zipml_destroy bound to torch's current stream of `device`."""

    def __init__(self, device="cuda:0", stream=None):
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise ZipmlError(ERR_CUDA, "zipml needs a CUDA device")
        self._h = C.c_void_p()
        if not torch.cuda.is_available():
            # let the library itself say so: there is nothing to fall back to
            _check(lib().zipml_create(C.byref(self._h), self.device.index or 0, None), "zipml_create")
            raise ZipmlError(ERR_CUDA, "zipml_create")
        index = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self.device = torch.device("cuda", index)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(lib().zipml_create(C.byref(self._h), index, C.c_void_p(self.stream.cuda_stream)), "zipml_create")

    def close(self):
        if getattr(self, "_h", None):
            lib().zipml_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # --- the calls of include/zipml.h ----------------------------------------------------------
    def zipml_sync(self):
        _check(lib().zipml_sync(self._h), "zipml_sync")

    def zipml_kernel_launches(self):
        return int(lib().zipml_kernel_launches(self._h))

    def zipml_last_engine(self):
        return int(lib().zipml_last_engine(self._h))

    def zipml_barrier_latency(self, ctas, floats_per_cta=0, iterations=1000):
        """Nanoseconds per step of the SGD step's communication skeleton on `ctas` CTAs."""
        out = torch.zeros(1, dtype=torch.int64, device=self.device)
        _check(lib().zipml_barrier_latency(self._h, ctas, floats_per_cta, iterations, _ptr(out)), "zipml_barrier_latency")
        self.zipml_sync()
        return out.item() / iterations

    def zipml_wait_probe(self, spin_limit=100000):
        """Enqueues a bounded wait that must give up; the next zipml_sync raises ZipmlError(ERR_TIMEOUT)."""
        _check(lib().zipml_wait_probe(self._h, spin_limit), "zipml_wait_probe")

    def zipml_quantize(self, A, bits, seed, level_mode=LEVELS_UNIFORM, levels=None, row_bytes=None, draw=0, grid=0):
        """Two packed quantizations of A; draw > 0: further independent pairs on the same grid (zipml_quantize_draw)."""
        m, n = A.shape
        assert A.stride(1) == 1 and A.dtype == torch.float32 and A.device == self.device
        rb = int(lib().zipml_row_bytes(n, bits)) if row_bytes is None else row_bytes
        if rb == 0:
            raise ZipmlError(ERR_UNSUPPORTED, "zipml_quantize")
        p1 = torch.empty((m, rb), dtype=torch.uint8, device=self.device)
        p2 = torch.empty((m, rb), dtype=torch.uint8, device=self.device)
        lo = torch.empty(n, dtype=torch.float32, device=self.device)
        step = torch.empty(n, dtype=torch.float32, device=self.device) if level_mode == LEVELS_UNIFORM else None
        if draw or grid:
            _check(lib().zipml_quantize_draw(self._h, C.c_void_p(A.data_ptr()), m, n, A.stride(0), bits, level_mode,
                                             _ptr(levels, torch.float32, self.device), seed, draw, grid, _ptr(p1), _ptr(p2), rb,
                                             _ptr(lo), _ptr(step)), "zipml_quantize_draw")
        else:
            _check(lib().zipml_quantize(self._h, C.c_void_p(A.data_ptr()), m, n, A.stride(0), bits, level_mode,
                                        _ptr(levels, torch.float32, self.device), seed, _ptr(p1), _ptr(p2), rb, _ptr(lo),
                                        _ptr(step)), "zipml_quantize")
        return Dataset(p1, p2, m, n, bits, level_mode, lo, step, levels)

    def zipml_convert_layout(self, data, to_layout):
        """A new Dataset with both planes in `to_layout` (scales and levels are shared with `data`)."""
        if to_layout == LAYOUT_COLUMN_BLOCKS:
            nbytes = int(lib().zipml_column_blocks_bytes(data.m, data.row_bytes))
            p1 = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            p2 = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        else:
            p1 = torch.empty((data.m, data.row_bytes), dtype=torch.uint8, device=self.device)
            p2 = torch.empty((data.m, data.row_bytes), dtype=torch.uint8, device=self.device)
        d = data.c_struct()
        _check(lib().zipml_convert_layout(self._h, C.byref(d), to_layout, _ptr(p1), _ptr(p2)), "zipml_convert_layout")
        return Dataset(p1, p2, data.m, data.n, data.bits, data.level_mode, data.feat_lo, data.feat_step, data.levels,
                       layout=to_layout, row_bytes=data.row_bytes)

    def zipml_shared_base_encode(self, data):
        urb = int(lib().zipml_up_row_bytes(data.n))
        base = torch.empty((data.m, data.row_bytes), dtype=torch.uint8, device=self.device)
        up1 = torch.empty((data.m, urb), dtype=torch.uint8, device=self.device)
        up2 = torch.empty((data.m, urb), dtype=torch.uint8, device=self.device)
        sb = SharedBase(base, up1, up2, data.m, data.n, data.bits, data.feat_lo, data.feat_step)
        d, o = data.c_struct(), sb.c_struct()
        _check(lib().zipml_shared_base_encode(self._h, C.byref(d), C.byref(o)), "zipml_shared_base_encode")
        return sb

    def zipml_shared_base_decode(self, sb):
        p1 = torch.empty((sb.m, sb.row_bytes), dtype=torch.uint8, device=self.device)
        p2 = torch.empty((sb.m, sb.row_bytes), dtype=torch.uint8, device=self.device)
        d = sb.c_struct()
        _check(lib().zipml_shared_base_decode(self._h, C.byref(d), _ptr(p1), _ptr(p2)), "zipml_shared_base_decode")
        return Dataset(p1, p2, sb.m, sb.n, sb.bits, LEVELS_UNIFORM, sb.feat_lo, sb.feat_step, None)

    def zipml_loss_shared_base(self, sb, b, x, out=None):
        out = torch.empty(1, dtype=torch.float64, device=self.device) if out is None else out
        d = sb.c_struct()
        _check(lib().zipml_loss_shared_base(self._h, C.byref(d), _ptr(b, torch.float32, self.device),
                                            _ptr(x, torch.float32, self.device), _ptr(out)), "zipml_loss_shared_base")
        return out

    def zipml_sgd_epoch_shared_base(self, sb, b, x, batch, lr, grad_out=None, **kw):
        p, keep = self.sgd_params(batch, lr, **kw)
        d = sb.c_struct()
        _check(lib().zipml_sgd_epoch_shared_base(self._h, C.byref(d), _ptr(b, torch.float32, self.device),
                                                 _ptr(x, torch.float32, self.device), C.byref(p),
                                                 _ptr(grad_out, torch.float32, self.device)), "zipml_sgd_epoch_shared_base")
        del keep

    def zipml_sgd_apply_gradient(self, x, g, step, lr, applied_out=None, **kw):
        """x <- R(x - lr * Q4(g)) in place (see zipml_sgd_apply_gradient); kw as for sgd_params."""
        p, keep = self.sgd_params(1, lr, **kw)
        _check(lib().zipml_sgd_apply_gradient(self._h, _ptr(x, torch.float32, self.device), _ptr(g, torch.float32, self.device),
                                              x.numel(), C.byref(p), step, _ptr(applied_out, torch.float32, self.device)),
               "zipml_sgd_apply_gradient")
        del keep

    def zipml_poly_rows(self, grid, planes, coef, x, scale=None, out=None):
        """Q(P) per sample from the planes Q_1 .. Q_d (device uint8 tensors of grid's shape), coef = (m_0 .. m_d)."""
        d = len(coef) - 1
        assert len(planes) >= d
        for p in planes[:d]:
            assert p.is_contiguous() and p.dtype == torch.uint8 and p.device == self.device
        ptrs = (C.c_void_p * max(d, 1))(*[p.data_ptr() for p in planes[:d]])
        cf = (C.c_double * (d + 1))(*[float(c) for c in coef])
        out = torch.empty(grid.m, dtype=torch.float64, device=self.device) if out is None else out
        g = grid.c_struct()
        _check(lib().zipml_poly_rows(self._h, C.byref(g), ptrs, d, cf, _ptr(x, torch.float32, self.device),
                                     _ptr(scale, torch.float32, self.device), _ptr(out, torch.float64, self.device)), "zipml_poly_rows")
        return out

    def zipml_weighted_plane_mean(self, grid, plane, c, out=None):
        """(1/m) sum_k c[k] Q(a_k) for the plane Q (n floats)."""
        out = torch.empty(grid.n, dtype=torch.float32, device=self.device) if out is None else out
        g = grid.c_struct()
        _check(lib().zipml_weighted_plane_mean(self._h, C.byref(g), _ptr(plane, torch.uint8, self.device),
                                               _ptr(c, torch.float64, self.device), _ptr(out, torch.float32, self.device)),
               "zipml_weighted_plane_mean")
        return out

    def zipml_optimal_levels(self, A, bits, hist_bins=1024, want_objective=False):
        m, n = A.shape
        assert A.stride(1) == 1 and A.dtype == torch.float32 and A.device == self.device
        lev = torch.empty((n, 1 << bits), dtype=torch.float32, device=self.device)
        obj = torch.empty(n, dtype=torch.int64, device=self.device) if want_objective else None
        _check(lib().zipml_optimal_levels(self._h, C.c_void_p(A.data_ptr()), m, n, A.stride(0), bits, hist_bins,
                                          _ptr(lev), _ptr(obj)), "zipml_optimal_levels")
        return (lev, obj) if want_objective else lev

    def sgd_params(self, batch, lr, model_bits=0, grad_bits=0, seed=0, epoch=0, first_step=0, num_steps=-1,
                   batch_order=None, engine=ENGINE_AUTO, grid_feature_parts=0, grid_row_parts=0, trace=None,
                   reg=REG_NONE, reg_param=0.0, model_out=None, cluster_contraction=0, stream_prefetch=0,
                   column_chunk_rows=0, vector_norm=NORM_L2):
        p = CSgdParams()
        p.struct_size = C.sizeof(CSgdParams)
        p.model_bits, p.grad_bits, p.engine = model_bits, grad_bits, engine
        p.batch, p.epoch, p.first_step, p.num_steps, p.seed, p.lr = batch, epoch, first_step, num_steps, seed, lr
        p.grid_feature_parts, p.grid_row_parts = grid_feature_parts, grid_row_parts
        p.reg, p.reg_param = reg, reg_param
        p.cluster_contraction, p.stream_prefetch = cluster_contraction, stream_prefetch
        p.column_chunk_rows = column_chunk_rows
        p.vector_norm = vector_norm
        if model_out is not None:  # (n,) fp32 device tensor
            assert model_out.dtype == torch.float32 and model_out.is_contiguous() and model_out.device == self.device
            p.model_out = model_out.data_ptr()
        if trace is not None:      # (steps, 8) int64 device tensor
            assert trace.dtype == torch.int64 and trace.is_contiguous() and trace.shape[1] == 8
            p.trace, p.trace_steps = trace.data_ptr(), trace.shape[0]
        keep = None
        if batch_order is not None:
            keep = torch.as_tensor(batch_order, dtype=torch.int32, device="cpu").contiguous()
            p.batch_order = keep.data_ptr()
        return p, keep

    def zipml_sgd_epoch(self, data, b, x, batch, lr, grad_out=None, **kw):
        """Updates x in place.  grad_out: optional (2, n) fp32 device tensor."""
        p, keep = self.sgd_params(batch, lr, **kw)
        d = data.c_struct()
        _check(lib().zipml_sgd_epoch(self._h, C.byref(d), _ptr(b, torch.float32, self.device),
                                     _ptr(x, torch.float32, self.device), C.byref(p),
                                     _ptr(grad_out, torch.float32, self.device)), "zipml_sgd_epoch")
        del keep

    def zipml_loss(self, mode, b, x, A=None, data=None, out=None):
        out = torch.empty(1, dtype=torch.float64, device=self.device) if out is None else out
        if mode == LOSS_DENSE:
            m, n = A.shape
            assert A.stride(1) == 1 and A.dtype == torch.float32
            rc = lib().zipml_loss(self._h, mode, C.c_void_p(A.data_ptr()), m, n, A.stride(0), None,
                                  _ptr(b, torch.float32, self.device), _ptr(x, torch.float32, self.device), _ptr(out))
        else:
            d = data.c_struct()
            rc = lib().zipml_loss(self._h, mode, None, 0, 0, 0, C.byref(d), _ptr(b, torch.float32, self.device),
                                  _ptr(x, torch.float32, self.device), _ptr(out))
        _check(rc, "zipml_loss")
        return out

    def zipml_train_host(self, A_host, b_host, x_host, bits, batch, lr, epochs, optimal_levels=False, hist_bins=1024,
                         quantize_seed=0, lr_decay=False, **kw):
        """All tensors on the CPU (pinned or not); x_host is updated in place; returns the dense loss."""
        m, n = A_host.shape
        for t in (A_host, b_host, x_host):
            assert t.device.type == "cpu" and t.dtype == torch.float32
        assert A_host.stride(1) == 1 and b_host.is_contiguous() and x_host.is_contiguous()
        p, keep = self.sgd_params(batch, lr, **kw)
        loss = torch.zeros(1, dtype=torch.float64)
        _check(lib().zipml_train_host(self._h, C.c_void_p(A_host.data_ptr()), m, n, A_host.stride(0), _ptr(b_host),
                                      _ptr(x_host), bits, int(optimal_levels), hist_bins, quantize_seed, C.byref(p),
                                      epochs, int(lr_decay), _ptr(loss)), "zipml_train_host")
        del keep
        return float(loss[0])


def zipml_loss_codes_static(data, b, x, out=None, stream=None):
    """Code-plane loss without any allocation inside the library (see include/zipml.h).

    For callers that cannot let the library call cudaMalloc: there is no context; the device and
    stream come from the tensors and from torch's current stream.  Problems larger than the
    library's fixed scratch raise ZipmlError(ERR_WORKSPACE).  Calls that overlap on the GPU race on
    that scratch, so keep them on one stream.
    """
    dev = b.device
    out = torch.empty(1, dtype=torch.float64, device=dev) if out is None else out
    stream = torch.cuda.current_stream(dev) if stream is None else stream
    d = data.c_struct()
    _check(lib().zipml_loss_codes_static(dev.index, C.c_void_p(stream.cuda_stream), C.byref(d),
                                         _ptr(b, torch.float32, dev), _ptr(x, torch.float32, dev), _ptr(out)),
           "zipml_loss_codes_static")
    return out
