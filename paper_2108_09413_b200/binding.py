"""ctypes binding of libisc.so: same names and argument order as include/isc.h."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libisc.so")

EXPORTS = ["isc_load_qmodel", "isc_free_qmodel", "isc_plan_resident", "isc_predict", "isc_certify", "isc_certify_batch",
           "isc_sample_counts", "isc_sample_counts_static", "isc_decide_certify", "isc_decide_predict", "isc_certify_integer", "isc_decide_certify_integer", "isc_noise_table", "isc_noise_table_rounded", "isc_radius_integer", "isc_certified_metrics",
           "isc_debug_tensor", "isc_debug_wait_timeout", "isc_debug_residual_form", "isc_set_option", "isc_get_info", "isc_strerror"]


class IscError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"{what}: {code} ({lib().isc_strerror(code).decode()})")
        self.code = code


class _Layer(C.Structure):
    _fields_ = [("op", C.c_int32), ("in_tensor", C.c_int32), ("res_tensor", C.c_int32),
                ("cin", C.c_int32), ("cout", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32), ("relu", C.c_int32),
                ("zp_in", C.c_int32), ("zp_out", C.c_int32), ("zp_res", C.c_int32),
                ("w", C.c_void_p), ("bias", C.c_void_p), ("mult", C.c_void_p), ("shift", C.c_void_p),
                ("res_mult", C.c_int32), ("res_shift", C.c_int32)]


_lib = None


def lib():
    """Load libisc.so; raises if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2108_09413_b200.build`")
        L = C.CDLL(_LIB_PATH)
        vp, i32p, f64p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_double)
        L.isc_load_qmodel.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(vp)]
        L.isc_plan_resident.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i32p, C.POINTER(C.c_int64)]
        L.isc_free_qmodel.argtypes = [vp]
        L.isc_free_qmodel.restype = None
        L.isc_predict.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int64, C.c_double, C.c_double, vp,
                                  i32p, vp]
        L.isc_certify.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int64, C.c_int64, C.c_double,
                                  C.c_double, vp, i32p, f64p, vp, vp]
        L.isc_certify_batch.argtypes = [vp, vp, C.c_int, C.c_int, C.c_uint64, C.c_uint64, C.c_int64,
                                        C.c_int64, C.c_double, C.c_double, vp, vp, vp, vp, vp]
        L.isc_sample_counts.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int32, C.c_int64, C.c_int64,
                                        C.c_double, vp, vp, vp]
        L.isc_sample_counts_static.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int32, C.c_int64, C.c_int64,
                                               C.c_double, vp, vp]
        L.isc_decide_certify.argtypes = [vp, vp, C.c_int, C.c_int64, C.c_double, C.c_double, i32p, f64p, f64p]
        L.isc_decide_predict.argtypes = [vp, C.c_int, C.c_double, i32p]
        L.isc_decide_certify_integer.argtypes = [vp, vp, C.c_int, C.c_int64, C.c_double, C.c_double, C.c_int, i32p, i32p,
                                                 C.POINTER(C.c_int64)]
        L.isc_certify_integer.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int64, C.c_int64, C.c_double, C.c_double,
                                          C.c_int, vp, i32p, i32p, C.POINTER(C.c_int64), vp, vp]
        L.isc_noise_table.argtypes = [C.c_double, vp, C.c_int64, i32p]
        L.isc_noise_table_rounded.argtypes = [C.c_double, vp, C.c_int64, i32p]
        L.isc_radius_integer.argtypes = [C.c_double, C.c_uint32, i32p, C.POINTER(C.c_int64)]
        L.isc_certified_metrics.argtypes = [vp, vp, vp, C.c_int64, vp, C.c_int, C.POINTER(C.c_double), vp]
        L.isc_debug_tensor.argtypes = [vp, vp, C.c_uint64, C.c_uint64, C.c_int32, C.c_int64, C.c_double,
                                       C.c_int, vp, vp, C.c_int64]
        L.isc_debug_wait_timeout.argtypes = [vp, C.c_int64, vp, vp]
        L.isc_debug_residual_form.argtypes = [C.c_int32, C.c_int32, C.c_int32, vp, vp]
        L.isc_set_option.argtypes = [vp, C.c_char_p, C.c_int64]
        L.isc_get_info.argtypes = [vp, C.c_char_p, C.POINTER(C.c_int64)]
        L.isc_strerror.argtypes = [C.c_int]
        L.isc_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("isc_free_qmodel", "isc_strerror"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(code, what):
    if code != 0:
        raise IscError(code, what)


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _stream_ptr(stream):
    if stream is None:
        return None
    return C.c_void_p(int(getattr(stream, "cuda_stream", stream)))


def layer_array(layers):
    """isc_layer[] from a list of dicts; returns (array, keepalive list)."""
    arr = (_Layer * len(layers))()
    keep = []
    for i, d in enumerate(layers):
        s = arr[i]
        for k in ("op", "in_tensor", "res_tensor", "cin", "cout", "kh", "kw", "stride", "pad", "relu",
                  "zp_in", "zp_out", "zp_res", "res_mult", "res_shift"):
            setattr(s, k, int(d[k]))
        for k, dt in (("w", np.int8), ("bias", np.int32), ("mult", np.int32), ("shift", np.int8)):
            a = d.get(k)
            if a is None:
                setattr(s, k, None)
            else:
                a = np.ascontiguousarray(a, dtype=dt)
                keep.append(a)
                setattr(s, k, a.ctypes.data)
    return arr, keep


def plan_resident(model: dict):
    """(fits, rule, smem_bytes): isc_plan_resident on a model dict; host only."""
    arr, keep = layer_array(model["layers"])
    rule, smem = C.c_int32(), C.c_int64()
    rc = lib().isc_plan_resident(C.cast(arr, C.c_void_p), len(model["layers"]), *[int(v) for v in model["in_shape"]],
                                 int(model["n_classes"]), C.byref(rule), C.byref(smem))
    del keep
    if rc < 0:
        raise IscError(rc, "isc_plan_resident")
    return rc, rule.value, smem.value


class Model:
    """Handle of a loaded quantized classifier (isc_load_qmodel / isc_free_qmodel)."""

    def __init__(self, model: dict):
        self.in_shape = tuple(int(v) for v in model["in_shape"])
        self.n_classes = int(model["n_classes"])
        arr, keep = layer_array(model["layers"])
        h = C.c_void_p()
        _check(lib().isc_load_qmodel(C.cast(arr, C.c_void_p), len(model["layers"]), *self.in_shape,
                                     self.n_classes, C.byref(h)), "isc_load_qmodel")
        del keep
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().isc_free_qmodel(self._h)
            self._h = None

    __del__ = close

    def _x(self, x_u8, n=1):
        x = np.ascontiguousarray(x_u8, dtype=np.uint8)
        assert x.size == n * int(np.prod(self.in_shape)), "image size does not match the model input"
        return x

    def set_option(self, name, value):
        _check(lib().isc_set_option(self._h, name.encode(), int(value)), "isc_set_option")

    def get_info(self, name):
        v = C.c_int64()
        _check(lib().isc_get_info(self._h, name.encode(), C.byref(v)), "isc_get_info")
        return v.value

    def sample_counts(self, x_u8, seed, image_id, phase, first_sample, n_samples, sigma, stream=None,
                      want_logits=False):
        x = self._x(x_u8)
        counts = np.zeros(self.n_classes, dtype=np.int32)
        logits = np.zeros((n_samples, self.n_classes), dtype=np.int8) if want_logits else None
        _check(lib().isc_sample_counts(self._h, _ptr(x), seed, image_id, phase, first_sample, n_samples,
                                       float(sigma), _stream_ptr(stream), _ptr(counts), _ptr(logits)),
               "isc_sample_counts")
        return (counts, logits) if want_logits else counts

    def sample_counts_static(self, x_u8, seed, image_id, phase, first_sample, n_samples, sigma, stream=None):
        """isc_sample_counts_static: same counts, device work space taken from the library's fixed
        array instead of cudaMalloc (for callers that may not allocate device memory)."""
        x = self._x(x_u8)
        counts = np.zeros(self.n_classes, dtype=np.int32)
        _check(lib().isc_sample_counts_static(self._h, _ptr(x), seed, image_id, phase, first_sample,
                                              n_samples, float(sigma), _stream_ptr(stream), _ptr(counts)),
               "isc_sample_counts_static")
        return counts

    def predict(self, x_u8, seed, image_id, N, sigma, alpha, stream=None):
        x = self._x(x_u8)
        cls = C.c_int32()
        counts = np.zeros(self.n_classes, dtype=np.int32)
        _check(lib().isc_predict(self._h, _ptr(x), seed, image_id, N, float(sigma), float(alpha),
                                 _stream_ptr(stream), C.byref(cls), _ptr(counts)), "isc_predict")
        return cls.value, counts

    def certify(self, x_u8, seed, image_id, N0, N, sigma, alpha, stream=None):
        x = self._x(x_u8)
        cls, rad = C.c_int32(), C.c_double()
        c0 = np.zeros(self.n_classes, dtype=np.int32)
        c1 = np.zeros(self.n_classes, dtype=np.int32)
        _check(lib().isc_certify(self._h, _ptr(x), seed, image_id, N0, N, float(sigma), float(alpha),
                                 _stream_ptr(stream), C.byref(cls), C.byref(rad), _ptr(c0), _ptr(c1)),
               "isc_certify")
        return cls.value, rad.value, c0, c1

    def certify_integer(self, x_u8, seed, image_id, N0, N, sigma, alpha, two_sided=False, stream=None):
        """(class, q, q*q, counts0, counts): isc_certify_integer (Theorem 3.2 steps 2-3; Theorem 3.1 when two_sided)."""
        x = self._x(x_u8)
        cls, q, q2 = C.c_int32(), C.c_int32(), C.c_int64()
        c0 = np.zeros(self.n_classes, dtype=np.int32)
        c1 = np.zeros(self.n_classes, dtype=np.int32)
        _check(lib().isc_certify_integer(self._h, _ptr(x), seed, image_id, N0, N, float(sigma), float(alpha),
                                         int(bool(two_sided)), _stream_ptr(stream), C.byref(cls), C.byref(q), C.byref(q2),
                                         _ptr(c0), _ptr(c1)), "isc_certify_integer")
        return cls.value, q.value, q2.value, c0, c1

    def certify_batch(self, x_u8, n_images, seed, image_id0, N0, N, sigma, alpha, stream=None,
                      device_ptr=None):
        """x_u8: host array [n][C][H][W], or pass device_ptr (int) to read images resident on the GPU."""
        cls = np.zeros(n_images, dtype=np.int32)
        rad = np.zeros(n_images, dtype=np.float64)
        c0 = np.zeros((n_images, self.n_classes), dtype=np.int32)
        c1 = np.zeros((n_images, self.n_classes), dtype=np.int32)
        if device_ptr is not None:
            xp, on_dev = C.c_void_p(int(device_ptr)), 1
        else:
            x = self._x(x_u8, n_images)
            xp, on_dev = _ptr(x), 0
        _check(lib().isc_certify_batch(self._h, xp, on_dev, n_images, seed, image_id0, N0, N, float(sigma),
                                       float(alpha), _stream_ptr(stream), _ptr(cls), _ptr(rad), _ptr(c0),
                                       _ptr(c1)), "isc_certify_batch")
        return cls, rad, c0, c1

    def debug_wait_timeout(self, limit_ns, stream=None):
        """(status, [first wait, second wait, abort flag, ns]): isc_debug_wait_timeout; the status is returned, not raised."""
        out = np.zeros(4, dtype=np.int32)
        rc = lib().isc_debug_wait_timeout(self._h, int(limit_ns), _stream_ptr(stream), _ptr(out))
        return rc, out.tolist()

    def debug_tensor(self, x_u8, seed, image_id, phase, j, sigma, tensor, size, stream=None):
        x = self._x(x_u8)
        out = np.zeros(size, dtype=np.int32)
        _check(lib().isc_debug_tensor(self._h, _ptr(x), seed, image_id, phase, j, float(sigma), tensor,
                                      _stream_ptr(stream), _ptr(out), size), "isc_debug_tensor")
        return out


def certify_decide(counts0, counts, N, sigma, alpha):
    c0 = np.ascontiguousarray(counts0, dtype=np.int32)
    c1 = np.ascontiguousarray(counts, dtype=np.int32)
    cls, rad, pl = C.c_int32(), C.c_double(), C.c_double()
    _check(lib().isc_decide_certify(_ptr(c0), _ptr(c1), c0.size, int(N), float(sigma), float(alpha),
                                    C.byref(cls), C.byref(rad), C.byref(pl)), "isc_decide_certify")
    return cls.value, rad.value, pl.value


def certify_integer_decide(counts0, counts, N, sigma, alpha, two_sided=False):
    c0 = np.ascontiguousarray(counts0, dtype=np.int32)
    c1 = np.ascontiguousarray(counts, dtype=np.int32)
    cls, q, q2 = C.c_int32(), C.c_int32(), C.c_int64()
    _check(lib().isc_decide_certify_integer(_ptr(c0), _ptr(c1), c0.size, int(N), float(sigma), float(alpha),
                                            int(bool(two_sided)), C.byref(cls), C.byref(q), C.byref(q2)),
           "isc_decide_certify_integer")
    return cls.value, q.value, q2.value


def predict_decide(counts, alpha):
    c = np.ascontiguousarray(counts, dtype=np.int32)
    cls = C.c_int32()
    _check(lib().isc_decide_predict(_ptr(c), c.size, float(alpha), C.byref(cls)), "isc_decide_predict")
    return cls.value


def certified_metrics(classes, radii, labels, thresholds):
    """(CP, [CA(r) for r in thresholds]) over certification results (Sec. 4.1, Evaluation Metrics)."""
    c = np.ascontiguousarray(classes, dtype=np.int32)
    rd = np.ascontiguousarray(radii, dtype=np.float64)
    lb = np.ascontiguousarray(labels, dtype=np.int32)
    th = np.ascontiguousarray(thresholds, dtype=np.float64)
    ca = np.zeros(th.size, dtype=np.float64)
    cp = C.c_double()
    _check(lib().isc_certified_metrics(_ptr(c) if c.size else None, _ptr(rd) if rd.size else None, _ptr(lb) if lb.size else None,
                                       c.size, _ptr(th) if th.size else None, th.size, C.byref(cp),
                                       _ptr(ca) if ca.size else None), "isc_certified_metrics")
    return cp.value, ca.tolist()


def radius_integer(sigma, p_fx):
    """(q, q*q): integer-only quantile of the discrete Gaussian for p_fx = floor(p * 2^32) (Theorem 3.2 steps 2-3)."""
    q, q2 = C.c_int32(), C.c_int64()
    _check(lib().isc_radius_integer(float(sigma), int(p_fx), C.byref(q), C.byref(q2)), "isc_radius_integer")
    return q.value, q2.value


def residual_form(res_mult, res_shift, zp_res):
    """(k, c) of isc_debug_residual_form when the short form of the residual rescale exists, else None; host only."""
    k, c = C.c_int32(), C.c_int32()
    rc = lib().isc_debug_residual_form(int(res_mult), int(res_shift), int(zp_res), C.byref(k), C.byref(c))
    if rc < 0:
        raise IscError(rc, "isc_debug_residual_form")
    return (k.value, c.value) if rc == 1 else None


def noise_table(sigma, rounded=False):
    """Cumulative table of the noise law: Eq. 2, or the rounded continuous Gaussian when `rounded`."""
    f = lib().isc_noise_table_rounded if rounded else lib().isc_noise_table
    T = C.c_int32()
    _check(f(float(sigma), None, 0, C.byref(T)), "isc_noise_table")
    cum = np.zeros(2 * T.value + 1, dtype=np.uint32)
    _check(f(float(sigma), _ptr(cum), cum.size, C.byref(T)), "isc_noise_table")
    return cum
