"""CPU-only checks of libisc: it loads, exports every declared symbol, rejects bad arguments
before touching the GPU, and its host decision code agrees with the oracle bit for bit."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
import workloads as wl
import paper_2108_09413_b200 as isc
from paper_2108_09413_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_exports_match_header():
    hdr = open(os.path.join(ROOT, "include", "isc.h")).read()
    declared = set(re.findall(r"\b(isc_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    L = isc.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_strerror():
    L = isc.lib()
    assert L.isc_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert len(L.isc_strerror(code)) > 3
    assert L.isc_strerror(-99) == b"unknown error"


def test_noise_table_equals_oracle_entry_by_entry():
    for sigma in (0.12, 0.25, 0.5, 1.0, 0.01, 2.0):
        np.testing.assert_array_equal(isc.noise_table(sigma), oracle.dgauss_table(sigma))
    T = C.c_int32()
    assert isc.lib().isc_noise_table(0.0, None, 0, C.byref(T)) == -1
    small = np.zeros(4, np.uint32)
    assert isc.lib().isc_noise_table(0.25, small.ctypes.data, 4, C.byref(T)) == -1


def test_decisions_bit_equal_to_oracle():
    rng = np.random.default_rng(4)
    for _ in range(40):
        N = int(rng.choice([100, 1000, 10000, 100000]))
        nA = int(rng.integers(0, N + 1))
        rest = N - nA
        b = int(rng.integers(0, rest + 1))
        counts = [b, nA, rest - b]
        c0 = rng.integers(0, 100, 3).tolist()
        sigma = float(rng.choice([0.12, 0.25, 0.5, 1.0]))
        got = isc.certify_decide(c0, counts, N, sigma, 0.001)
        exp = oracle.certify_decide(c0, counts, N, sigma, 0.001)
        assert got == exp                                    # class, radius and p_lower: identical doubles
        assert isc.predict_decide(counts, 0.001) == oracle.predict_decide(counts, 0.001)
    for counts in ([0, 11, 0], [0, 10, 0], [50, 50], [7, 7, 7], [0, 0, 100000]):
        assert isc.predict_decide(counts, 0.001) == oracle.predict_decide(counts, 0.001)
    assert isc.certify_decide([0, 1], [0, 100000], 100000, 0.25, 0.001) == \
        oracle.certify_decide([0, 1], [0, 100000], 100000, 0.25, 0.001)


def test_decide_rejects_bad_arguments():
    L = isc.lib()
    c = np.array([1, 2], np.int32)
    cls, rad = C.c_int32(7), C.c_double(7.0)
    assert L.isc_decide_certify(None, c.ctypes.data, 2, 3, 0.25, 0.001, C.byref(cls), C.byref(rad), None) == -1
    assert L.isc_decide_certify(c.ctypes.data, c.ctypes.data, 2, 3, 0.25, 1.5, C.byref(cls), C.byref(rad), None) == -1
    assert L.isc_decide_certify(c.ctypes.data, c.ctypes.data, 2, 1, 0.25, 0.001, C.byref(cls), C.byref(rad), None) == -1
    assert L.isc_decide_predict(c.ctypes.data, 0, 0.001, C.byref(cls)) == -1
    assert cls.value == 7 and rad.value == 7.0               # outputs untouched on error


def _load(model):
    arr, keep = binding.layer_array(model["layers"])
    h = C.c_void_p()
    rc = isc.lib().isc_load_qmodel(C.cast(arr, C.c_void_p), len(model["layers"]), *model["in_shape"],
                                   model["n_classes"], C.byref(h))
    return rc, h


def test_load_rejects_malformed_models_without_a_gpu():
    base = wl.tiny_cnn()
    h = C.c_void_p()
    assert isc.lib().isc_load_qmodel(None, 4, 3, 32, 32, 10, C.byref(h)) == -1
    def variant(kw=None):
        m = dict(base, layers=[dict(l) for l in base["layers"]])
        for (i, k), v in (kw or {}).items():
            m["layers"][i][k] = v
        return m
    assert _load(variant({(1, "cin"): 8}))[0] == -2                 # channel mismatch
    assert _load(variant({(1, "in_tensor"): 3}))[0] == -2           # reads a later tensor
    assert _load(variant({(0, "op"): 9}))[0] == -1
    assert _load(variant({(0, "zp_out"): 300}))[0] == -1
    bad_shift = variant()
    bad_shift["layers"][0]["shift"] = np.full(16, 40, np.int8)
    assert _load(bad_shift)[0] == -1
    bad_mult = variant()
    bad_mult["layers"][0]["mult"] = np.full(16, 5, np.int32)
    assert _load(bad_mult)[0] == -1
    assert _load(dict(base, n_classes=11))[0] == -2                  # last tensor is not the logits
    no_w = variant()
    no_w["layers"][0]["w"] = None
    assert _load(no_w)[0] == -1
    assert h.value is None


def test_integer_radius_equals_oracle_lookup():
    """Theorem 3.2 steps 2-3: the library's table-lookup quantile and squared radius against the oracle's linear
    scan of its own table, on a sweep of probabilities (incl. both ends of the table and exact table values)."""
    rng = np.random.default_rng(7)
    for sigma in (0.12, 0.25, 0.5, 1.0):
        cum = oracle.dgauss_table(sigma)
        T = (cum.size - 1) // 2
        ps = [0, 1, 2 ** 31, 2 ** 32 - 1, int(0.9889 * 2 ** 32), int(0.99993 * 2 ** 32)]
        ps += [int(v) for v in cum[[0, 1, T - 1, T, T + 1, cum.size - 2, cum.size - 1]]]
        ps += [int(v) + 1 for v in cum[[0, T, cum.size - 2]] if int(v) + 1 < 2 ** 32]
        ps += [int(v) for v in rng.integers(0, 2 ** 32, size=200, dtype=np.uint64)]
        for p_fx in ps:
            q, q2 = isc.radius_integer(sigma, p_fx)
            assert q == oracle.dgauss_quantile_fx(p_fx, cum), (sigma, p_fx)
            assert q2 == q * q
    q = C.c_int32(123)
    assert isc.lib().isc_radius_integer(0.0, 5, C.byref(q), None) == -1 and q.value == 123
    assert isc.lib().isc_radius_integer(0.25, 5, None, None) == -1


def test_certified_metrics_equal_oracle():
    """Certified Percentage / Certified Accuracy (Sec. 4.1): the library's reduction against the oracle's loops."""
    rng = np.random.default_rng(11)
    th = [0.0, 0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75, 2.0]
    for n in (0, 1, 7, 500):
        classes = rng.integers(-1, 10, size=n)
        radii = np.where(classes == -1, 0.0, rng.random(n) * 2.0)
        labels = np.where(rng.random(n) < 0.7, np.maximum(classes, 0), rng.integers(0, 10, size=n))
        assert isc.certified_metrics(classes, radii, labels, th) == oracle.certified_metrics(classes, radii, labels, th)
    assert isc.certified_metrics([-1, -1], [0.0, 0.0], [1, 2], []) == (0.0, [])
    cp = C.c_double(9.0)
    assert isc.lib().isc_certified_metrics(None, None, None, 3, None, 0, C.byref(cp), None) == -1 and cp.value == 9.0


def test_plan_resident_accepts_cifar_resnets_and_names_the_refusing_rule():
    """Host-only planner query: the CIFAR-shaped networks fit the shared-memory-resident engine (227 KB per CTA at
    most), the 224x224 bottleneck network does not."""
    import workloads as wl
    for model in (wl.tiny_cnn(), wl.resnet20(), wl.resnet110(), wl.spread_model("resnet20")):
        fits, rule, smem = isc.plan_resident(model)
        assert (fits, rule) == (1, 0) and 0 < smem <= 227 * 1024, model["name"]
    fits, rule, smem = isc.plan_resident(wl.resnet50())
    assert fits == 0 and rule > 0 and smem == 0
    # a consumer whose zero-point differs from its producer's output zero-point reads wrong padding: refused
    model = wl.resnet20()
    model["layers"][1] = dict(model["layers"][1], zp_in=-100)
    fits, rule, _ = isc.plan_resident(model)
    assert fits == 0 and rule == 108
    # a layer list that does not type-check is an error, not a refusal
    model = wl.resnet20()
    model["layers"][1] = dict(model["layers"][1], cin=8)
    with pytest.raises(isc.IscError):
        isc.plan_resident(model)


def test_integer_certify_decisions_equal_the_oracle():
    rng = np.random.default_rng(11)
    for _ in range(60):
        n_classes = int(rng.integers(2, 12))
        N = int(rng.choice([100, 1000, 100_000]))
        top = int(rng.integers(N // 2 - N // 20, N + 1))
        rest = rng.multinomial(N - top, np.ones(n_classes - 1) / (n_classes - 1))
        counts = np.concatenate([[top], rest]).astype(np.int32)
        rng.shuffle(counts)
        counts0 = rng.integers(0, 50, n_classes).astype(np.int32)
        sigma = float(rng.choice([0.12, 0.25, 0.5, 1.0]))
        for two in (False, True):
            assert isc.certify_integer_decide(counts0, counts, N, sigma, 0.001, two) == \
                   oracle.certify_integer_decide(counts0, counts, N, sigma, 0.001, two)
    L = isc.lib()
    c = np.array([5, 5], np.int32)
    cls, q = C.c_int32(7), C.c_int32(7)
    assert L.isc_decide_certify_integer(c.ctypes.data, c.ctypes.data, 2, 10, 0.25, 1.5, 0, C.byref(cls), C.byref(q), None) == -1
    assert L.isc_decide_certify_integer(c.ctypes.data, c.ctypes.data, 2, 4, 0.25, 0.001, 0, C.byref(cls), C.byref(q), None) == -1
    assert (cls.value, q.value) == (7, 7)


def test_rounded_noise_table_equals_the_oracle():
    for sigma in (0.12, 0.25, 0.5, 1.0):
        np.testing.assert_array_equal(isc.noise_table(sigma, rounded=True), oracle.rgauss_table(sigma))
        np.testing.assert_array_equal(isc.noise_table(sigma), oracle.dgauss_table(sigma))


def test_residual_short_form_reproduces_the_rescale_on_every_byte():
    """The offset form of the residual rescale, floor((256 k + u) m2 / 2^32) - c, is used by the tensor-core engines only
    when it equals rs((r - zp_res) * res_mult, 31 - res_shift) for all 256 bytes: checked here with exact integers."""
    rng = np.random.default_rng(0x15174000)
    found = 0
    cases = [(1 << 30, 0, 0), (1 << 30, -1, -128), ((1 << 31) - 1, 0, 127), ((1 << 31) - 1, -1, -128)]
    cases += [(int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-1, 1)), int(rng.integers(-128, 128))) for _ in range(60)]
    for res_mult, res_shift, zp_res in cases:
        form = isc.residual_form(res_mult, res_shift, zp_res)
        if form is None:
            continue
        found += 1
        k, c = form
        assert 0 <= k < 4096
        n = 31 - res_shift
        m2 = res_mult << (32 - n)
        for r in range(-128, 128):
            want = ((r - zp_res) * res_mult + (1 << (n - 1))) >> n           # rs(): round half up, floor division
            assert (((256 * k + r + 128) * m2) >> 32) - c == want, (res_mult, res_shift, zp_res, r)
    assert found >= 50                                                        # the form exists for nearly every multiplier
    assert isc.residual_form(1 << 30, -3, 0) is None                         # rescale shifts the engines do not take
