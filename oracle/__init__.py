"""ctypes front end of the CPU oracle (``intrs_oracle.c``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library never does, and this package
never imports the CUDA library.  Models are passed as plain lists of dicts
holding numpy arrays (the format the workload generators emit).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "intrs_oracle.c")
_SRC2 = os.path.join(_HERE, "dgauss_rejection.c")
_LIB = os.path.join(_HERE, "libintrs_oracle.so")

OP_CONV2D, OP_FC, OP_GAVGPOOL, OP_MAXPOOL = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC2)):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-Wextra", "-o", _LIB, _SRC, _SRC2, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Layer(C.Structure):
    _fields_ = [("op", C.c_int32), ("in_tensor", C.c_int32), ("res_tensor", C.c_int32),
                ("cin", C.c_int32), ("cout", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32), ("relu", C.c_int32),
                ("zp_in", C.c_int32), ("zp_out", C.c_int32), ("zp_res", C.c_int32),
                ("w", C.c_void_p), ("bias", C.c_void_p), ("mult", C.c_void_p),
                ("shift", C.c_void_p), ("res_mult", C.c_int32), ("res_shift", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u32p, i32p = C.POINTER(C.c_uint32), C.POINTER(C.c_int32)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_uniform_u32.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64]
        L.orc_uniform_u32.restype = C.c_uint32
        L.orc_dgauss_halfwidth.argtypes = [C.c_double]
        L.orc_dgauss_halfwidth.restype = C.c_int32
        L.orc_dgauss_pmf.argtypes = [C.c_double, C.c_void_p]
        L.orc_dgauss_pmf.restype = None
        L.orc_dgauss_table.argtypes = [C.c_double, C.c_void_p]
        L.orc_dgauss_table.restype = None
        L.rej_dgauss_draws.argtypes = [C.c_double, C.c_uint64, C.c_int64, C.c_void_p]
        L.rej_dgauss_draws.restype = C.c_int64
        L.orc_rgauss_table.argtypes = [C.c_double, C.c_void_p]
        L.orc_rgauss_table.restype = None
        L.orc_set_noise_kind.argtypes = [C.c_int]
        L.orc_set_noise_kind.restype = None
        for f in (L.orc_dgauss_from_uniform, L.orc_dgauss_from_uniform_fast):
            f.argtypes = [C.c_uint32, C.c_void_p, C.c_int32]
            f.restype = C.c_int32
        L.orc_noise.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, C.c_double,
                                C.c_uint64, C.c_int64, C.c_void_p]
        L.orc_noise.restype = None
        L.orc_noisy_input.argtypes = [C.c_void_p, C.c_int64, C.c_uint64, C.c_uint64, C.c_uint32,
                                      C.c_uint64, C.c_double, C.c_void_p]
        L.orc_noisy_input.restype = None
        L.orc_requant.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        L.orc_requant.restype = C.c_int64
        L.orc_residual_term.argtypes = [C.c_int32] * 4
        L.orc_residual_term.restype = C.c_int64
        L.orc_forward.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                  C.c_void_p, C.c_int, C.c_void_p]
        L.orc_forward.restype = C.c_int
        L.orc_tensor_size.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]
        L.orc_tensor_size.restype = C.c_int64
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int]
        L.orc_argmax.restype = C.c_int32
        L.orc_sample_counts.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                        C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint32, C.c_int64,
                                        C.c_int64, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_sample_counts.restype = C.c_int
        L.orc_num_threads.restype = C.c_int
        L.orc_lower_conf_bound.argtypes = [C.c_int64, C.c_int64, C.c_double]
        L.orc_lower_conf_bound.restype = C.c_double
        L.orc_normal_quantile.argtypes = [C.c_double]
        L.orc_normal_quantile.restype = C.c_double
        L.orc_certify_decide.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_double,
                                         C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.orc_certify_decide.restype = C.c_int32
        L.orc_binom_pvalue_half.argtypes = [C.c_int64, C.c_int64]
        L.orc_binom_pvalue_half.restype = C.c_double
        L.orc_predict_decide.argtypes = [C.c_void_p, C.c_int, C.c_double]
        L.orc_predict_decide.restype = C.c_int32
        L.orc_dgauss_quantile_fx.argtypes = [C.c_uint32, C.c_void_p, C.c_int32]
        L.orc_dgauss_quantile_fx.restype = C.c_int32
        L.orc_certify_integer_decide.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_double, C.c_double,
                                                 C.c_int, i32p, C.POINTER(C.c_int64)]
        L.orc_certify_integer_decide.restype = C.c_int32
        L.orc_certify.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_void_p, C.c_uint64, C.c_uint64, C.c_int64, C.c_int64,
                                  C.c_double, C.c_double, i32p, C.POINTER(C.c_double),
                                  C.c_void_p, C.c_void_p]
        L.orc_certify.restype = C.c_int
        L.orc_predict.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_void_p, C.c_uint64, C.c_uint64, C.c_int64, C.c_double,
                                  C.c_double, i32p, C.c_void_p]
        L.orc_predict.restype = C.c_int
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


class Model:
    """Holds the C layer array plus the numpy buffers it points into."""

    def __init__(self, model: dict):
        self.in_c, self.in_h, self.in_w = model["in_shape"]
        self.n_classes = int(model["n_classes"])
        layers = model["layers"]
        self.n_layers = len(layers)
        self._keep = []
        self.arr = (_Layer * self.n_layers)()
        for i, d in enumerate(layers):
            s = self.arr[i]
            for k in ("op", "in_tensor", "res_tensor", "cin", "cout", "kh", "kw", "stride", "pad",
                      "relu", "zp_in", "zp_out", "zp_res", "res_mult", "res_shift"):
                setattr(s, k, int(d[k]))
            for k, dt in (("w", np.int8), ("bias", np.int32), ("mult", np.int32), ("shift", np.int8)):
                a = d.get(k)
                if a is None:
                    setattr(s, k, None)
                else:
                    a = np.ascontiguousarray(a, dtype=dt)
                    self._keep.append(a)
                    setattr(s, k, a.ctypes.data)

    @property
    def d(self):
        return self.in_c * self.in_h * self.in_w

    def _args(self):
        return (C.cast(self.arr, C.c_void_p), self.n_layers, self.in_c, self.in_h, self.in_w)


# ------------------------------------------------------------------ wrappers

def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(v) for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) for v in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def uniform_u32(seed, image_id, phase, j, e):
    return int(lib().orc_uniform_u32(seed, image_id, phase, j, e))


def dgauss_halfwidth(sigma):
    return int(lib().orc_dgauss_halfwidth(float(sigma)))


def dgauss_pmf(sigma):
    T = dgauss_halfwidth(sigma)
    p = np.zeros(2 * T + 1, dtype=np.float64)
    lib().orc_dgauss_pmf(float(sigma), _ptr(p))
    return p


def dgauss_table(sigma):
    T = dgauss_halfwidth(sigma)
    t = np.zeros(2 * T + 1, dtype=np.uint32)
    lib().orc_dgauss_table(float(sigma), _ptr(t))
    return t


def rgauss_table(sigma):
    """Cumulative table of the rounded continuous Gaussian (the FloatRS-quant comparison method's noise, Sec. 4.1)."""
    T = dgauss_halfwidth(sigma)
    t = np.zeros(2 * T + 1, dtype=np.uint32)
    lib().orc_rgauss_table(float(sigma), _ptr(t))
    return t


def rejection_dgauss(sigma, seed, n):
    """n draws of the discrete Gaussian with std 255 * sigma pixel levels from the table-free rejection sampler
    (dgauss_rejection.c); returns (draws, proposals made)."""
    out = np.zeros(n, dtype=np.int32)
    proposals = lib().rej_dgauss_draws(255.0 * float(sigma), int(seed), int(n), _ptr(out))
    return out, int(proposals)


def set_noise_kind(kind):
    """0: discrete Gaussian of Eq. 2 (default); 1: rounded continuous Gaussian.  Process-wide."""
    lib().orc_set_noise_kind(int(kind))


def dgauss_from_uniform(u, cum, fast=False):
    T = (len(cum) - 1) // 2
    f = lib().orc_dgauss_from_uniform_fast if fast else lib().orc_dgauss_from_uniform
    return int(f(int(u), _ptr(cum), T))


def noise(seed, image_id, phase, j, sigma, e0, n):
    out = np.zeros(n, dtype=np.int32)
    lib().orc_noise(seed, image_id, phase, j, float(sigma), e0, n, _ptr(out))
    return out


def noisy_input(x_u8, seed, image_id, phase, j, sigma):
    x = np.ascontiguousarray(x_u8, dtype=np.uint8).ravel()
    out = np.zeros(x.size, dtype=np.uint8)
    lib().orc_noisy_input(_ptr(x), x.size, seed, image_id, phase, j, float(sigma), _ptr(out))
    return out.reshape(np.shape(x_u8))


def requant(acc, mult, shift):
    return int(lib().orc_requant(int(acc), int(mult), int(shift)))


def residual_term(r, zp_res, res_mult, res_shift):
    return int(lib().orc_residual_term(int(r), int(zp_res), int(res_mult), int(res_shift)))


def tensor_size(m: Model, k):
    return int(lib().orc_tensor_size(*m._args(), k))


def forward(m: Model, a0, dump_tensor=-1):
    """a0: CHW values 0..255.  Returns logits (int32) and optionally a tensor dump."""
    a = np.ascontiguousarray(a0, dtype=np.int32).ravel()
    assert a.size == m.d
    n_last = tensor_size(m, m.n_layers)
    if n_last < 0:
        raise ValueError("oracle: bad layer list")
    logits = np.zeros(n_last, dtype=np.int32)
    dump = None
    if dump_tensor >= 0:
        dump = np.zeros(tensor_size(m, dump_tensor), dtype=np.int32)
    rc = lib().orc_forward(*m._args(), _ptr(a), _ptr(logits), dump_tensor,
                           _ptr(dump) if dump is not None else None)
    if rc:
        raise ValueError("oracle: bad layer list")
    return (logits, dump) if dump_tensor >= 0 else logits


def sample_counts(m: Model, x_u8, seed, image_id, phase, first, n, sigma, want_logits=False):
    x = np.ascontiguousarray(x_u8, dtype=np.uint8).ravel()
    assert x.size == m.d
    counts = np.zeros(m.n_classes, dtype=np.int32)
    logits = np.zeros((n, m.n_classes), dtype=np.int8) if want_logits else None
    rc = lib().orc_sample_counts(*m._args(), m.n_classes, _ptr(x), seed, image_id, phase, first, n,
                                 float(sigma), _ptr(counts), _ptr(logits) if want_logits else None)
    if rc:
        raise ValueError("oracle: bad layer list")
    return (counts, logits) if want_logits else counts


def num_threads():
    return int(lib().orc_num_threads())


def lower_conf_bound(k, n, alpha):
    return float(lib().orc_lower_conf_bound(int(k), int(n), float(alpha)))


def normal_quantile(p):
    return float(lib().orc_normal_quantile(float(p)))


def certify_decide(counts0, counts, N, sigma, alpha):
    c0 = np.ascontiguousarray(counts0, dtype=np.int32)
    c1 = np.ascontiguousarray(counts, dtype=np.int32)
    r, p = C.c_double(), C.c_double()
    cls = lib().orc_certify_decide(_ptr(c0), _ptr(c1), c0.size, int(N), float(sigma), float(alpha),
                                   C.byref(r), C.byref(p))
    return int(cls), r.value, p.value


def binom_pvalue_half(n_a, m):
    return float(lib().orc_binom_pvalue_half(int(n_a), int(m)))


def predict_decide(counts, alpha):
    c = np.ascontiguousarray(counts, dtype=np.int32)
    return int(lib().orc_predict_decide(_ptr(c), c.size, float(alpha)))


def dgauss_quantile_fx(p_fx, cum):
    T = (len(cum) - 1) // 2
    return int(lib().orc_dgauss_quantile_fx(int(p_fx), _ptr(cum), T))


def certify_integer_decide(counts0, counts, N, sigma, alpha, two_sided=False):
    """(class, q, q2): Algorithm 1's decision with the radius read off the discrete Gaussian's CDF table
    (Theorem 3.2 steps 2-3); two_sided: Theorem 3.1's form, q = twice the radius in pixel levels."""
    c0 = np.ascontiguousarray(counts0, dtype=np.int32)
    c1 = np.ascontiguousarray(counts, dtype=np.int32)
    q, q2 = C.c_int32(), C.c_int64()
    cls = lib().orc_certify_integer_decide(_ptr(c0), _ptr(c1), c0.size, int(N), float(sigma), float(alpha),
                                           int(bool(two_sided)), C.byref(q), C.byref(q2))
    return int(cls), q.value, q2.value


def certify(m: Model, x_u8, seed, image_id, N0, N, sigma, alpha):
    x = np.ascontiguousarray(x_u8, dtype=np.uint8).ravel()
    c0 = np.zeros(m.n_classes, dtype=np.int32)
    c1 = np.zeros(m.n_classes, dtype=np.int32)
    cls, rad = C.c_int32(), C.c_double()
    rc = lib().orc_certify(*m._args(), m.n_classes, _ptr(x), seed, image_id, N0, N, float(sigma),
                           float(alpha), C.byref(cls), C.byref(rad), _ptr(c0), _ptr(c1))
    if rc:
        raise ValueError("oracle: bad layer list")
    return cls.value, rad.value, c0, c1


def predict(m: Model, x_u8, seed, image_id, N, sigma, alpha):
    x = np.ascontiguousarray(x_u8, dtype=np.uint8).ravel()
    c = np.zeros(m.n_classes, dtype=np.int32)
    cls = C.c_int32()
    rc = lib().orc_predict(*m._args(), m.n_classes, _ptr(x), seed, image_id, N, float(sigma),
                           float(alpha), C.byref(cls), _ptr(c))
    if rc:
        raise ValueError("oracle: bad layer list")
    return cls.value, c


def certified_metrics(classes, radii, labels, thresholds):
    """Certified Percentage and Certified Accuracy at each radius threshold (Sec. 4.1, Evaluation Metrics,
    the two displayed equations): CP = share of inputs whose certification does not abstain (class != -1);
    CA(r) = among those, the share with the correct class and a certified radius >= r (0 when nothing certifies).
    Plain loops over the definition; test infrastructure like the rest of this package."""
    L = len(classes)
    certified = 0
    for i in range(L):
        if int(classes[i]) != -1:
            certified += 1
    cp = certified / L if L else 0.0
    ca = []
    for r in thresholds:
        hit = 0
        for i in range(L):
            if int(classes[i]) != -1 and int(classes[i]) == int(labels[i]) and float(radii[i]) >= float(r):
                hit += 1
        ca.append(hit / certified if certified else 0.0)
    return cp, ca
