"""ctypes face of the CPU oracle (oracle/zipml_oracle.cpp).

Test infrastructure only: imported by tests/, by the smoke check and by the benchmark's
cpu-baseline leg.  Nothing here imports the CUDA package, and the CUDA package never imports this.
All arrays are numpy arrays in host memory.
"""
import ctypes as C

import numpy as np

from .build import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NONFINITE = 0, -1, -2, -3
UNIFORM, TABLE = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _declare(_lib)
    return _lib


def _p(a, t=None):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _declare(L):
    vp, i32, i64, u32, u64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_uint32, C.c_uint64, C.c_float
    L.orc_philox4x32_10.argtypes = [vp, vp, vp]
    L.orc_philox4x32_10.restype = None
    L.orc_u24_sample.argtypes = [u64, u64, u32, u32]
    L.orc_u24_sample.restype = u32
    L.orc_u24_vector.argtypes = [u64, u32, u32, u32, u32]
    L.orc_u24_vector.restype = u32
    L.orc_container_bits.argtypes = [i32]
    L.orc_row_bytes.argtypes = [i64, i32]
    L.orc_row_bytes.restype = i64
    L.orc_pack_codes.argtypes = [vp, i64, i32, vp, i64]
    L.orc_pack_codes.restype = None
    L.orc_unpack_codes.argtypes = [vp, i64, i32, vp]
    L.orc_unpack_codes.restype = None
    L.orc_up_row_bytes.argtypes = [i64]
    L.orc_up_row_bytes.restype = i64
    L.orc_shared_base_encode.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp, i64]
    L.orc_shared_base_decode.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp, vp]
    L.orc_column_range.argtypes = [vp, i64, i64, i64, vp, vp]
    L.orc_quantize.argtypes = [vp, i64, i64, i64, i32, i32, vp, u64, vp, vp, i64, vp, vp]
    L.orc_quantize_pair.argtypes = [vp, i64, i64, i64, i32, i32, vp, u64, C.c_uint32, i32, vp, vp, i64, vp, vp]
    L.orc_poly_rows.argtypes = [vp, i32, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    L.orc_weighted_plane_mean.argtypes = [vp, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp]
    L.orc_dequantize_row.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp]
    L.orc_dequantize_row.restype = None
    L.orc_quantize_vector.argtypes = [vp, i64, i32, u64, u32, u32, u32, vp, vp]
    L.orc_quantize_vector.restype = None
    L.orc_quantize_vector_norm.argtypes = [vp, i64, i32, u64, u32, u32, u32, i32, vp, vp]
    L.orc_quantize_vector_norm.restype = None
    L.orc_sgd_epoch.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp, i64, f32, i32, i32,
                                u64, i64, i64, i64, vp, vp, i32, f32, i32]
    L.orc_estimator_mean.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp, i32, vp]
    L.orc_loss_dense.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    L.orc_loss_codes.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp, vp]
    L.orc_histogram.argtypes = [vp, i64, i64, i64, i32, vp, vp, vp]
    L.orc_interval_cost.argtypes = [vp, i32, i32]
    L.orc_interval_cost.restype = u64
    L.orc_interval_cost_prefix.argtypes = [vp, i32, i32, i32]
    L.orc_interval_cost_prefix.restype = u64
    L.orc_levels_dp.argtypes = [vp, i32, i32, vp, vp]
    L.orc_levels_bruteforce.argtypes = [vp, i32, i32, vp, vp]
    L.orc_total_variance.argtypes = [vp, i64, vp, i32]
    L.orc_total_variance.restype = C.c_double
    L.orc_levels_from_idx.argtypes = [vp, i32, i32, f32, f32, vp]
    L.orc_levels_from_idx.restype = None
    L.orc_optimal_levels.argtypes = [vp, i64, i64, i64, i32, i32, vp, vp]


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def u24_sample(seed, row, feature, copy):
    return int(lib().orc_u24_sample(seed, row, feature, copy))


def u24_vector(seed, epoch, step, coord, stream):
    return int(lib().orc_u24_vector(seed, epoch, step, coord, stream))


def container_bits(bits):
    return int(lib().orc_container_bits(bits))


def row_bytes(n, bits):
    return int(lib().orc_row_bytes(n, bits))


def pack_codes(codes, bits):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rb = row_bytes(codes.shape[0], bits)
    out = np.zeros(rb, dtype=np.uint8)
    lib().orc_pack_codes(_p(codes), codes.shape[0], bits, _p(out), rb)
    return out


def unpack_codes(row, n, bits):
    row = np.ascontiguousarray(row, dtype=np.uint8)
    out = np.zeros(n, dtype=np.uint8)
    lib().orc_unpack_codes(_p(row), n, bits, _p(out))
    return out


def unpack_plane(plane, n, bits):
    """(m, row_bytes) uint8 -> (m, n) uint8 codes."""
    return np.stack([unpack_codes(plane[k], n, bits) for k in range(plane.shape[0])])


def up_row_bytes(n):
    return int(lib().orc_up_row_bytes(n))


def shared_base_encode(ds):
    """(base, up1, up2) of a two-plane dataset: the smaller code once, one bit per sample."""
    urb = up_row_bytes(ds.n)
    base = np.zeros_like(ds.plane1)
    up1 = np.zeros((ds.m, urb), np.uint8)
    up2 = np.zeros((ds.m, urb), np.uint8)
    _check(lib().orc_shared_base_encode(_p(ds.plane1), _p(ds.plane2), ds.row_bytes, ds.m, ds.n, ds.bits, _p(base),
                                        _p(up1), _p(up2), urb))
    return base, up1, up2


def shared_base_decode(base, up1, up2, n, bits):
    base, up1, up2 = (np.ascontiguousarray(a, dtype=np.uint8) for a in (base, up1, up2))
    m, rb = base.shape
    p1 = np.zeros_like(base)
    p2 = np.zeros_like(base)
    _check(lib().orc_shared_base_decode(_p(base), _p(up1), _p(up2), rb, up1.shape[1], m, n, bits, _p(p1), _p(p2)))
    return p1, p2


def column_range(A):
    A = np.ascontiguousarray(A, dtype=np.float32)
    m, n = A.shape
    lo = np.zeros(n, np.float32)
    hi = np.zeros(n, np.float32)
    _check(lib().orc_column_range(_p(A), m, n, n, _p(lo), _p(hi)))
    return lo, hi


class Dataset:
    """Two packed code planes plus what dequantizes them (host arrays)."""

    def __init__(self, plane1, plane2, m, n, bits, mode, feat_lo, feat_step, levels):
        self.plane1, self.plane2 = plane1, plane2
        self.m, self.n, self.bits, self.mode = m, n, bits, mode
        self.row_bytes = plane1.shape[1]
        self.feat_lo, self.feat_step, self.levels = feat_lo, feat_step, levels

    def dequantize(self, which, k):
        plane = self.plane1 if which == 1 else self.plane2
        out = np.zeros(self.n, np.float64)
        lib().orc_dequantize_row(_p(plane[k]), self.n, self.bits, self.mode, _p(self.feat_lo),
                                 _p(self.feat_step), _p(self.levels), _p(out))
        return out


def quantize(A, bits, seed, mode=UNIFORM, levels=None):
    A = np.ascontiguousarray(A, dtype=np.float32)
    m, n = A.shape
    rb = row_bytes(n, bits)
    if rb == 0:
        raise OracleError(ERR_UNSUPPORTED)
    p1 = np.zeros((m, rb), np.uint8)
    p2 = np.zeros((m, rb), np.uint8)
    lo = np.zeros(n, np.float32)
    step = np.zeros(n, np.float32)
    if levels is not None:
        levels = np.ascontiguousarray(levels, dtype=np.float32)
    _check(lib().orc_quantize(_p(A), m, n, n, bits, mode, _p(levels), seed, _p(p1), _p(p2), rb, _p(lo), _p(step)))
    return Dataset(p1, p2, m, n, bits, mode, lo, step, levels)


def quantize_pair(A, bits, seed, pair, mode=UNIFORM, levels=None, symmetric=False):
    """Pair `pair` of independent quantizations of A on the grid of quantize(): planes 2 pair + 1, 2 pair + 2 of
    Q_1, Q_2, ... (Section 4.1); pair 0 is quantize()."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    m, n = A.shape
    rb = row_bytes(n, bits)
    p1, p2 = np.zeros((m, rb), np.uint8), np.zeros((m, rb), np.uint8)
    lo = np.zeros(n, np.float32)
    step = np.zeros(n, np.float32) if mode == UNIFORM else None
    if levels is not None:
        levels = np.ascontiguousarray(levels, dtype=np.float32)
    _check(lib().orc_quantize_pair(_p(A), m, n, n, bits, mode, _p(levels), seed, pair, int(symmetric), _p(p1), _p(p2), rb, _p(lo),
                                   _p(step)))
    return Dataset(p1, p2, m, n, bits, mode, lo, step, levels)


def poly_rows(planes, ds, x, coef, scale=None):
    """Q(P) per sample (Section 4.1) from the planes Q_1 .. Q_d (arrays like ds.plane1), coef = (m_0 .. m_d); times
    scale[k] where given."""
    d = len(coef) - 1
    assert len(planes) >= d
    planes = [np.ascontiguousarray(p) for p in planes[:d]]
    ptrs = (C.c_void_p * max(d, 1))(*[p.ctypes.data for p in planes])
    x = np.ascontiguousarray(x, dtype=np.float32)
    coef = np.ascontiguousarray(coef, dtype=np.float64)
    scale = None if scale is None else np.ascontiguousarray(scale, dtype=np.float32)
    out = np.zeros(ds.m, np.float64)
    _check(lib().orc_poly_rows(ptrs, d, ds.row_bytes, ds.m, ds.n, ds.bits, ds.mode, _p(ds.feat_lo), _p(ds.feat_step),
                               _p(ds.levels), _p(x), _p(coef), _p(scale), _p(out)))
    return out


def weighted_plane_mean(plane, ds, c):
    """(1/m) sum_k c_k Q(a_k) for the plane Q (Section 4.2: the gradient for factors c_k = b_k Q(P)_k)."""
    plane = np.ascontiguousarray(plane)
    c = np.ascontiguousarray(c, dtype=np.float64)
    g = np.zeros(ds.n, np.float64)
    _check(lib().orc_weighted_plane_mean(_p(plane), ds.row_bytes, ds.m, ds.n, ds.bits, ds.mode, _p(ds.feat_lo),
                                         _p(ds.feat_step), _p(ds.levels), _p(c), _p(g)))
    return g


NORM_L2, NORM_LINF = 0, 1


def quantize_vector(v, bits, seed, epoch, step, stream, norm=NORM_L2):
    v = np.ascontiguousarray(v, dtype=np.float32)
    out = np.zeros_like(v)
    codes = np.zeros(v.shape[0], np.int32)
    lib().orc_quantize_vector_norm(_p(v), v.shape[0], bits, seed, epoch, step, stream, norm, _p(out), _p(codes))
    return out, codes


REG_NONE, REG_L2, REG_L1, REG_NONNEG, REG_LSSVM = 0, 1, 2, 3, 4


def sgd_epoch(ds, b, x, batch, lr, model_bits=0, grad_bits=0, seed=0, epoch=0, first_step=0, num_steps=None,
              batch_order=None, want_grad=False, reg=REG_NONE, reg_param=0.0, vector_norm=NORM_L2):
    """Runs steps in place on a copy of x; returns (x_new, grad(2, n) or None)."""
    b = np.ascontiguousarray(b, dtype=np.float32)
    x = np.array(x, dtype=np.float32, copy=True)
    T = (ds.m + batch - 1) // batch
    if num_steps is None:
        num_steps = T - first_step
    if batch_order is not None:
        batch_order = np.ascontiguousarray(batch_order, dtype=np.int32)
    g = np.zeros((2, ds.n), np.float32) if want_grad else None
    _check(lib().orc_sgd_epoch(_p(ds.plane1), _p(ds.plane2), ds.row_bytes, ds.m, ds.n, ds.bits, ds.mode,
                               _p(ds.feat_lo), _p(ds.feat_step), _p(ds.levels), _p(b), _p(x), batch, lr,
                               model_bits, grad_bits, seed, epoch, first_step, num_steps, _p(batch_order), _p(g),
                               int(reg), C.c_float(reg_param), int(vector_norm)))
    return x, g


def estimator_mean(ds, b, x, which):
    b = np.ascontiguousarray(b, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.float32)
    g = np.zeros(ds.n, np.float64)
    _check(lib().orc_estimator_mean(_p(ds.plane1), _p(ds.plane2), ds.row_bytes, ds.m, ds.n, ds.bits, ds.mode,
                                    _p(ds.feat_lo), _p(ds.feat_step), _p(ds.levels), _p(b), _p(x), which, _p(g)))
    return g


def loss_dense(A, b, x):
    A = np.ascontiguousarray(A, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.zeros(1, np.float64)
    _check(lib().orc_loss_dense(_p(A), A.shape[0], A.shape[1], A.shape[1], _p(b), _p(x), _p(out)))
    return float(out[0])


def loss_codes(ds, b, x):
    b = np.ascontiguousarray(b, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.zeros(1, np.float64)
    _check(lib().orc_loss_codes(_p(ds.plane1), _p(ds.plane2), ds.row_bytes, ds.m, ds.n, ds.bits, ds.mode,
                                _p(ds.feat_lo), _p(ds.feat_step), _p(ds.levels), _p(b), _p(x), _p(out)))
    return float(out[0])


def histogram(A, M, lo, hi):
    A = np.ascontiguousarray(A, dtype=np.float32)
    m, n = A.shape
    counts = np.zeros((n, M), np.uint32)
    _check(lib().orc_histogram(_p(A), m, n, n, M, _p(lo), _p(hi), _p(counts)))
    return counts


def interval_cost(cnt, j, m):
    cnt = np.ascontiguousarray(cnt, dtype=np.uint32)
    return int(lib().orc_interval_cost(_p(cnt), j, m))


def interval_cost_prefix(cnt, j, m):
    cnt = np.ascontiguousarray(cnt, dtype=np.uint32)
    return int(lib().orc_interval_cost_prefix(_p(cnt), cnt.shape[0], j, m))


def levels_dp(cnt, s):
    cnt = np.ascontiguousarray(cnt, dtype=np.uint32)
    idx = np.zeros(s + 1, np.int32)
    obj = np.zeros(1, np.uint64)
    _check(lib().orc_levels_dp(_p(cnt), cnt.shape[0], s, _p(idx), _p(obj)))
    return idx, int(obj[0])


def levels_bruteforce(cnt, s):
    cnt = np.ascontiguousarray(cnt, dtype=np.uint32)
    idx = np.zeros(s + 1, np.int32)
    obj = np.zeros(1, np.uint64)
    _check(lib().orc_levels_bruteforce(_p(cnt), cnt.shape[0], s, _p(idx), _p(obj)))
    return idx, int(obj[0])


def total_variance(pts, edges):
    pts = np.ascontiguousarray(pts, dtype=np.float64)
    edges = np.ascontiguousarray(edges, dtype=np.float64)
    return float(lib().orc_total_variance(_p(pts), pts.shape[0], _p(edges), edges.shape[0] - 1))


def levels_from_idx(idx, M, lo, hi):
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.zeros(idx.shape[0], np.float32)
    lib().orc_levels_from_idx(_p(idx), idx.shape[0] - 1, M, lo, hi, _p(out))
    return out


def optimal_levels(A, bits, M):
    A = np.ascontiguousarray(A, dtype=np.float32)
    m, n = A.shape
    L = 1 << bits
    lev = np.zeros((n, L), np.float32)
    obj = np.zeros(n, np.uint64)
    _check(lib().orc_optimal_levels(_p(A), m, n, n, bits, M, _p(lev), _p(obj)))
    return lev, obj
