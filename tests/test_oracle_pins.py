"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.stats as st

import oracle
import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
SIGMAS = (0.12, 0.25, 0.5, 1.0)          # the paper's noise levels (Sec. 4.2)


# ----------------------------------------------------------------- Philox

def test_philox_known_answers():
    """Published known-answer vectors of Philox4x32-10 (Salmon et al., SC'11)."""
    n = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        assert oracle.philox4x32_10(v[0:4], v[4:6]) == v[6:10]
        n += 1
    assert n == 3


def test_uniform_counter_layout():
    seed, img, ph, j = 0x1234567890ABCDEF, (0xBEEF << 32) | 77, 2, (0x5A << 32) | 123456
    for e in (0, 1, 2, 3, 4, 4097, 3071):
        ctr = [e >> 2, j & 0xFFFFFFFF, img & 0xFFFFFFFF,
               ph | (((j >> 32) & 0xFF) << 8) | (((img >> 32) & 0xFFFF) << 16)]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        assert oracle.uniform_u32(seed, img, ph, j, e) == oracle.philox4x32_10(ctr, key)[e & 3]
    # different phase / sample / image give different streams
    base = [oracle.uniform_u32(1, 0, 0, 0, e) for e in range(8)]
    assert base != [oracle.uniform_u32(1, 0, 1, 0, e) for e in range(8)]
    assert base != [oracle.uniform_u32(1, 0, 0, 1, e) for e in range(8)]
    assert base != [oracle.uniform_u32(1, 1, 0, 0, e) for e in range(8)]


# ------------------------------------------------- discrete Gaussian (Eq. 2)

def _pmf_direct(sigma, zs):
    """Eq. 2 evaluated directly with a far wider normalising sum than the table's."""
    s_int = 255.0 * sigma
    T = int(math.ceil(12 * s_int))
    h = np.arange(-T, T + 1, dtype=np.float64)
    norm = math.fsum(np.exp(-h * h / (2 * s_int * s_int)))
    zs = np.asarray(zs, dtype=np.float64)
    return np.exp(-zs * zs / (2 * s_int * s_int)) / norm


@pytest.mark.parametrize("sigma", SIGMAS)
def test_pmf_closed_forms(sigma):
    s_int = 255.0 * sigma
    T = oracle.dgauss_halfwidth(sigma)
    assert T == math.ceil(7 * s_int)
    p = oracle.dgauss_pmf(sigma)
    assert abs(p.sum() - 1.0) < 1e-12
    np.testing.assert_allclose(p, p[::-1], rtol=0, atol=0)                  # symmetry
    assert abs(p[T] - 1.0 / (s_int * math.sqrt(2 * math.pi))) < 1e-9       # P[0]
    z = np.arange(-40, 40)
    ratio = p[T + z + 1] / p[T + z]
    np.testing.assert_allclose(ratio, np.exp(-(2 * z + 1) / (2 * s_int * s_int)), rtol=1e-12)
    np.testing.assert_allclose(p, _pmf_direct(sigma, np.arange(-T, T + 1)), rtol=1e-9, atol=1e-18)
    # shift invariance of the normaliser on the lattice (Appendix H.1)
    h = np.arange(-T - 50, T + 51, dtype=np.float64)
    s0 = np.exp(-h * h / (2 * s_int * s_int)).sum()
    s7 = np.exp(-(h - 7) ** 2 / (2 * s_int * s_int)).sum()
    assert abs(s0 - s7) / s0 < 1e-12


@pytest.mark.parametrize("sigma", SIGMAS)
def test_table_matches_pmf(sigma):
    T = oracle.dgauss_halfwidth(sigma)
    cum = oracle.dgauss_table(sigma).astype(np.float64)
    assert np.all(np.diff(cum) >= 0) and cum[-1] == 2 ** 32 - 1
    mass = np.diff(np.concatenate(([0.0], cum))) / 2.0 ** 32
    np.testing.assert_allclose(mass, _pmf_direct(sigma, np.arange(-T, T + 1)), atol=5e-10)


def test_inverse_cdf_rule():
    cum = oracle.dgauss_table(0.12)
    T = (len(cum) - 1) // 2
    rng = np.random.default_rng(5)
    probes = set(int(v) for v in rng.integers(0, 2 ** 32, 2000))
    for k in range(T - 60, T + 60):                     # every boundary near the centre
        probes.update({int(cum[k]) - 1, int(cum[k]), int(cum[k]) + 1})
    probes.update({0, 1, 2 ** 32 - 1, 2 ** 32 - 2})
    for u in probes:
        if not 0 <= u < 2 ** 32:
            continue
        z = oracle.dgauss_from_uniform(u, cum)
        assert z == oracle.dgauss_from_uniform(u, cum, fast=True)
        idx = np.searchsorted(cum, u, side="right")     # first k with u < cum[k]
        assert z == (min(int(idx), 2 * T) - T)
    assert oracle.dgauss_from_uniform(2 ** 32 - 1, cum) == T


@pytest.mark.parametrize("sigma", SIGMAS)
def test_sampler_chi_square_1e7(sigma):
    """Exact-pmf chi-square of 10^7 draws of the oracle's sampler against Eq. 2."""
    n = 10_000_000
    T = oracle.dgauss_halfwidth(sigma)
    draws = oracle.noise(seed=99, image_id=3, phase=1, j=12345, sigma=sigma, e0=0, n=n)
    assert draws.min() >= -T and draws.max() <= T
    obs = np.bincount(draws + T, minlength=2 * T + 1).astype(np.float64)
    exp = _pmf_direct(sigma, np.arange(-T, T + 1)) * n
    keep = exp >= 5.0                                    # pool both thin tails
    lo, hi = np.argmax(keep), len(keep) - np.argmax(keep[::-1])
    o = np.concatenate(([obs[:lo].sum()], obs[lo:hi], [obs[hi:].sum()]))
    e = np.concatenate(([exp[:lo].sum()], exp[lo:hi], [exp[hi:].sum()]))
    e[0] += n - e.sum()                                  # mass outside +-T belongs to the tails
    chi2 = ((o - e) ** 2 / e).sum()
    p = st.chi2.sf(chi2, df=len(o) - 1)
    assert p > 1e-3, (chi2, len(o), p)
    s_int = 255.0 * sigma
    assert abs(draws.mean()) < 5 * s_int / math.sqrt(n)
    assert abs(draws.astype(np.float64).var() - s_int ** 2) < 5 * s_int ** 2 * math.sqrt(2.0 / n)


def test_noisy_input_is_clamped_sum():
    x = wl.images(1)[0]
    d = oracle.noise(7, 1, 0, 5, 0.5, 0, x.size).reshape(x.shape)
    a0 = oracle.noisy_input(x, 7, 1, 0, 5, 0.5)
    np.testing.assert_array_equal(a0, np.clip(x.astype(np.int32) + d, 0, 255))
    assert (a0 == 0).any() and (a0 == 255).any()


# ----------------------------------------------------------- layer arithmetic

def _rs_exact(num: int, n: int) -> int:
    """floor(num / 2^n + 1/2) in exact rational arithmetic."""
    return math.floor(Fraction(num, 1 << n) + Fraction(1, 2))


def test_requant_vs_exact_rationals():
    rng = np.random.default_rng(11)
    n = 200_000
    acc = rng.integers(-2 ** 31, 2 ** 31, n)
    mult = rng.integers(2 ** 30, 2 ** 31, n)
    shift = rng.integers(0, 32, n)
    for a, m, s in zip(acc.tolist(), mult.tolist(), shift.tolist()):
        assert oracle.requant(a, m, s) == _rs_exact(a * m, 31 + s)
    # exact ties: acc*mult == 2^(n-1) (mod 2^n), both signs -> rounds up (towards +inf)
    for s in range(0, 12):
        nbits = 31 + s
        m = 1 << 30
        for q in (-5, -1, 0, 1, 4):
            a = (2 * q + 1) << s                         # a*m = (2q+1) * 2^(nbits-1)
            assert (a * m) % (1 << nbits) == 1 << (nbits - 1)
            assert oracle.requant(a, m, s) == q + 1 == _rs_exact(a * m, nbits)
    assert oracle.requant(-3, 1 << 30, 0) == -1          # -1.5 -> -1 (half up)
    assert oracle.requant(3, 1 << 30, 0) == 2            # +1.5 -> 2


def test_residual_term_vs_exact_rationals():
    rng = np.random.default_rng(12)
    for _ in range(50_000):
        r = int(rng.integers(-128, 128)); zp = int(rng.integers(-128, 128))
        m = int(rng.integers(2 ** 30, 2 ** 31)); s = int(rng.integers(-4, 5))
        assert oracle.residual_term(r, zp, m, s) == _rs_exact((r - zp) * m, 31 - s)


def _brute_conv(a, L, res=None):
    """Second, independent statement of the conv rule: seven nested loops, exact rationals."""
    cin, H, W = a.shape
    kh, kw, st_, pad, cout = L["kh"], L["kw"], L["stride"], L["pad"], L["cout"]
    Ho = (H + 2 * pad - kh) // st_ + 1
    Wo = (W + 2 * pad - kw) // st_ + 1
    y = np.zeros((cout, Ho, Wo), dtype=np.int64)
    for o in range(cout):
        for oy in range(Ho):
            for ox in range(Wo):
                acc = int(L["bias"][o])
                for c in range(cin):
                    for r in range(kh):
                        for s in range(kw):
                            iy, ix = oy * st_ + r - pad, ox * st_ + s - pad
                            if 0 <= iy < H and 0 <= ix < W:
                                acc += (int(a[c, iy, ix]) - L["zp_in"]) * int(L["w"][o, c, r, s])
                v = _rs_exact(acc * int(L["mult"][o]), 31 + int(L["shift"][o]))
                if res is not None:
                    v += _rs_exact((int(res[o, oy, ox]) - L["zp_res"]) * L["res_mult"],
                                   31 - L["res_shift"])
                q = v + L["zp_out"]
                lo = max(-128, L["zp_out"]) if L["relu"] else -128
                y[o, oy, ox] = min(127, max(lo, q))
    return y


def _mk_conv(rng, cin, cout, k, stride, pad, relu, zp_in, zp_out, in_tensor=0, res_tensor=-1,
             zp_res=0, res_shift=0, shift_lo=0, shift_hi=6):
    return dict(op=wl.OP_CONV2D, in_tensor=in_tensor, res_tensor=res_tensor, cin=cin, cout=cout,
                kh=k, kw=k, stride=stride, pad=pad, relu=relu, zp_in=zp_in, zp_out=zp_out,
                zp_res=zp_res,
                w=rng.integers(-127, 128, (cout, cin, k, k)).astype(np.int8),
                bias=rng.integers(-4096, 4097, cout).astype(np.int32),
                mult=rng.integers(2 ** 30, 2 ** 31, cout).astype(np.int32),
                shift=rng.integers(shift_lo, shift_hi + 1, cout).astype(np.int8),
                res_mult=int(rng.integers(2 ** 30, 2 ** 31)) if res_tensor >= 0 else 0,
                res_shift=res_shift)


@pytest.mark.parametrize("cin,cout,k,stride,pad,hw,relu,zp_in,zp_out", [
    (1, 1, 3, 1, 1, 5, 0, 0, 0), (2, 3, 3, 1, 1, 5, 1, 0, -128), (2, 3, 3, 2, 1, 6, 1, 3, -20),
    (3, 2, 1, 2, 0, 5, 0, -7, 5), (2, 2, 5, 2, 2, 7, 1, 0, -128), (1, 2, 3, 1, 0, 4, 0, 9, 0),
])
def test_conv_vs_brute_force(cin, cout, k, stride, pad, hw, relu, zp_in, zp_out):
    rng = np.random.default_rng(cin * 100 + cout * 10 + k)
    L = _mk_conv(rng, cin, cout, k, stride, pad, relu, zp_in, zp_out)
    m = oracle.Model(dict(in_shape=(cin, hw, hw), n_classes=1, layers=[L]))
    a = rng.integers(0, 256, (cin, hw, hw))
    _, got = oracle.forward(m, a, dump_tensor=1)
    exp = _brute_conv(a, L)
    np.testing.assert_array_equal(got.reshape(exp.shape), exp)


def test_conv_identity_and_box_kernels():
    hw, zp = 6, 4
    rng = np.random.default_rng(3)
    a = rng.integers(0, 120, (1, hw, hw))
    base = dict(op=wl.OP_CONV2D, in_tensor=0, res_tensor=-1, cin=1, cout=1, stride=1, relu=0,
                zp_in=zp, zp_out=zp, zp_res=0, bias=np.zeros(1, np.int32),
                mult=np.array([1 << 30], np.int32), shift=np.zeros(1, np.int8),
                res_mult=0, res_shift=0)
    # weight 2 with mult 2^30 / 2^31 = 1/2: y = (a - zp) + zp = a
    ident = dict(base, kh=1, kw=1, pad=0, w=np.full((1, 1, 1, 1), 2, np.int8))
    _, got = oracle.forward(oracle.Model(dict(in_shape=(1, hw, hw), n_classes=1, layers=[ident])),
                            a, dump_tensor=1)
    np.testing.assert_array_equal(got.reshape(a.shape), a)
    # all-twos 3x3 kernel = box sum of (a - zp) over the valid neighbourhood
    box = dict(base, kh=3, kw=3, pad=1, w=np.full((1, 1, 3, 3), 2, np.int8), zp_out=0)
    small = rng.integers(0, 12, (1, hw, hw)) + zp
    _, got = oracle.forward(oracle.Model(dict(in_shape=(1, hw, hw), n_classes=1, layers=[box])),
                            small, dump_tensor=1)
    p = np.pad(small[0] - zp, 1)
    exp = sum(p[r:r + hw, s:s + hw] for r in range(3) for s in range(3))
    np.testing.assert_array_equal(got.reshape(hw, hw), exp)


def test_residual_pool_fc_chain_vs_brute_force():
    """conv -> conv(+residual from tensor 1, rescaled) -> global avg-pool -> FC."""
    rng = np.random.default_rng(21)
    hw = 4
    L1 = _mk_conv(rng, 2, 4, 3, 1, 1, 1, 0, -128, shift_lo=7, shift_hi=9)
    L2 = _mk_conv(rng, 4, 4, 3, 1, 1, 1, -128, -128, in_tensor=1, res_tensor=1, zp_res=-128,
                  res_shift=1, shift_lo=8, shift_hi=10)
    pool = wl._gavgpool(2, 4, hw * hw, -128)
    fc = _mk_conv(rng, 4, 3, 1, 1, 0, 0, -128, 0, in_tensor=3, shift_lo=4, shift_hi=6)
    fc["op"] = wl.OP_FC
    model = dict(in_shape=(2, hw, hw), n_classes=3, layers=[L1, L2, pool, fc])
    m = oracle.Model(model)
    a = rng.integers(0, 256, (2, hw, hw))
    t1 = _brute_conv(a, L1)
    t2 = _brute_conv(t1, L2, res=t1)
    assert (t2 != np.clip(_brute_conv(t1, L2), -128, 127)).any()      # the residual matters
    mult, s = int(pool["mult"][0]), int(pool["shift"][0])
    assert Fraction(mult, 1 << (31 + s)) == Fraction(1, hw * hw)
    t3 = np.array([min(127, max(-128, _rs_exact(int((t2[c] + 128).sum()) * mult, 31 + s) - 128))
                   for c in range(4)]).reshape(4, 1, 1)
    t4 = _brute_conv(t3, dict(fc, kh=1, kw=1, stride=1, pad=0))
    for k, exp in ((1, t1), (2, t2), (3, t3), (4, t4)):
        _, got = oracle.forward(m, a, dump_tensor=k)
        np.testing.assert_array_equal(got, exp.ravel())
    np.testing.assert_array_equal(oracle.forward(m, a), t4.ravel())


def test_maxpool_and_avgpool49():
    rng = np.random.default_rng(8)
    a = rng.integers(0, 256, (2, 7, 7))
    mp = wl._maxpool(0, 2, 3, 2, 1, 0)
    _, got = oracle.forward(oracle.Model(dict(in_shape=(2, 7, 7), n_classes=2, layers=[mp,
                            wl._gavgpool(1, 2, 16, 0)])), a, dump_tensor=1)
    p = np.pad(a, ((0, 0), (1, 1), (1, 1)), constant_values=-1)
    exp = np.stack([[[p[c, 2 * y:2 * y + 3, 2 * x:2 * x + 3].max() for x in range(4)]
                     for y in range(4)] for c in range(2)])
    np.testing.assert_array_equal(got.reshape(exp.shape), exp)
    ap = wl._gavgpool(0, 2, 49, 0)
    b = rng.integers(0, 128, (2, 7, 7))
    got = oracle.forward(oracle.Model(dict(in_shape=(2, 7, 7), n_classes=2, layers=[ap])), b)
    exp = [math.floor(Fraction(int(b[c].sum()), 49) + Fraction(1, 2)) for c in range(2)]
    assert np.abs(got - np.array(exp)).max() <= 0      # nearest multiplier is exact at this range
    v = np.array([3, 9, 9, 1], np.int32)
    assert oracle.lib().orc_argmax(v.ctypes.data, 4) == 1


def test_bad_layer_list_is_rejected():
    rng = np.random.default_rng(1)
    L = _mk_conv(rng, 2, 3, 3, 1, 1, 1, 0, -128)
    m = oracle.Model(dict(in_shape=(5, 4, 4), n_classes=3, layers=[L]))     # cin mismatch
    with pytest.raises(ValueError):
        oracle.forward(m, np.zeros((5, 4, 4)))


# ------------------------------------------------------- bound, radius, tests

ALPHA = 0.001


def test_lower_bound_closed_forms():
    for n, v in ((100, 0.933254300796991), (1000, 0.9931160484209338),
                 (10 ** 4, 0.9993094630025899), (10 ** 5, 0.9999309248330094)):
        assert abs(oracle.lower_conf_bound(n, n, ALPHA) - v) < 1e-15
        assert abs(oracle.lower_conf_bound(n, n, ALPHA) - ALPHA ** (1.0 / n)) < 1e-15
        assert oracle.lower_conf_bound(0, n, ALPHA) == 0.0
    prev = -1.0
    for k in range(0, 201):
        p = oracle.lower_conf_bound(k, 200, ALPHA)
        assert p > prev or (k == 0 and p == 0.0)
        assert p < k / 200 or k == 0
        prev = p
        if 0 < k < 200:                                   # tail at the bound is alpha
            assert abs(st.binom.sf(k - 1, 200, p) - ALPHA) < 1e-9


@pytest.mark.parametrize("k,n", [(99000, 100000), (50500, 100000), (50000, 100000), (700, 1000),
                                 (1, 100), (99, 100), (5100, 10000)])
def test_lower_bound_vs_scipy_beta(k, n):
    assert abs(oracle.lower_conf_bound(k, n, ALPHA) - st.beta.ppf(ALPHA, k, n - k + 1)) < 1e-9


def test_normal_quantile_vs_scipy():
    for p in (0.5, 0.500108, 0.6, 0.9, 0.98898934, 0.9999309248330094, 0.99999999):
        assert abs(oracle.normal_quantile(p) - st.norm.ppf(p)) < 1e-9 * max(1, st.norm.ppf(p))


def test_certify_decision_cases():
    c0 = [3, 90, 7]
    cls, rad, pl = oracle.certify_decide(c0, [100, 99000, 900], 100000, 0.25, ALPHA)
    assert cls == 1 and abs(pl - 0.98898934) < 1e-7 and abs(rad - 0.25 * st.norm.ppf(pl)) < 1e-9
    cls, rad, pl = oracle.certify_decide(c0, [0, 50500, 49500], 100000, 0.5, ALPHA)
    assert cls == 1 and 0 < rad < 1e-3 and pl > 0.5
    cls, rad, pl = oracle.certify_decide(c0, [0, 50000, 50000], 100000, 0.5, ALPHA)
    assert cls == -1 and rad == 0.0 and pl < 0.5
    # the class comes from the selection counts, the estimate from the second vector
    cls, rad, _ = oracle.certify_decide([50, 50, 0], [0, 100000, 0], 100000, 0.25, ALPHA)
    assert cls == -1                                        # tie -> class 0, which has no votes
    cls, rad, _ = oracle.certify_decide([0, 0, 100], [0, 0, 100000], 100000, 0.25, ALPHA)
    assert cls == 2


def test_max_radius_matches_paper_tables():
    """All N2 votes for one class gives the largest radius sigma*Phi^-1(alpha^(1/N2)); the
    paper's certified-accuracy tables are zero exactly from the first column beyond it."""
    rows = 0
    for line in open(os.path.join(GOLD, "certified_accuracy_zero_pattern.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, n2, sigma, last_nz, first_z, _ = line.split()
        n2, sigma, last_nz = int(n2), float(sigma), float(last_nz)
        cnt = [0, n2]
        cls, rmax, _ = oracle.certify_decide([0, 100], cnt, n2, sigma, ALPHA)
        assert cls == 1
        assert rmax >= last_nz, (sigma, n2, rmax)
        if first_z != "none":
            assert rmax < float(first_z), (sigma, n2, rmax)
        rows += 1
    assert rows == 8
    for sigma, v in ((0.12, 0.457), (0.25, 0.953), (0.5, 1.906), (1.0, 3.811)):
        assert abs(oracle.certify_decide([0, 1], [0, 10 ** 5], 10 ** 5, sigma, ALPHA)[1] - v) < 2e-3


def test_radius_monotone_in_pA_and_linear_in_sigma():
    N = 10000
    prev = -1.0
    for nA in range(4000, N + 1, 150):
        cls, r, _ = oracle.certify_decide([0, 1], [N - nA, nA], N, 0.25, ALPHA)
        assert r >= prev
        prev = r
    assert prev > 0
    base = oracle.certify_decide([0, 1], [500, 9500], N, 0.25, ALPHA)[1]
    for s in (0.12, 0.5, 1.0):
        r = oracle.certify_decide([0, 1], [500, 9500], N, s, ALPHA)[1]
        assert abs(r / s - base / 0.25) < 1e-12


def test_predict_closed_forms():
    for nA in range(1, 25):
        assert abs(oracle.binom_pvalue_half(nA, nA) - min(1.0, 2.0 ** (1 - nA))) < 1e-15
        assert oracle.predict_decide([0, nA, 0], ALPHA) == (1 if nA >= 11 else -1)
    assert oracle.binom_pvalue_half(50, 100) == 1.0
    assert oracle.predict_decide([50, 50], ALPHA) == -1
    for nA, nB in ((70, 30), (600, 400), (60, 40), (5300, 4700)):
        pv = oracle.binom_pvalue_half(nA, nA + nB)
        assert abs(pv - st.binomtest(nA, nA + nB, 0.5).pvalue) < 1e-9 * max(pv, 1e-300) + 1e-15
        assert oracle.predict_decide([nB, 3, nA], ALPHA) == (2 if pv <= ALPHA else -1)
    assert oracle.predict_decide([7, 7, 7], ALPHA) == -1


def test_integer_quantile_lookup_tracks_normal_quantile():
    """Theorem 3.2 step 2: the discrete-Gaussian quantile by table lookup is within 1.5
    pixel levels of sigma_int * Phi^-1(p) once sigma_int >= 30."""
    for sigma in SIGMAS:
        cum = oracle.dgauss_table(sigma)
        for p in (0.5, 0.6, 0.9, 0.9889, 0.99993):
            q = oracle.dgauss_quantile_fx(int(p * 2 ** 32), cum)
            assert abs(q - 255 * sigma * st.norm.ppf(p)) <= 1.5


def test_certified_metrics_closed_forms():
    """Sec. 4.1, Evaluation Metrics: closed forms of the two displayed equations."""
    L = 40
    labels = [i % 10 for i in range(L)]
    # everything certified and correct, radii i / L: CA(r) is the share of radii >= r, CP = 1
    radii = [i / L for i in range(L)]
    cp, ca = oracle.certified_metrics(labels, radii, labels, [0.0, 0.25, 0.5, 0.975, 1.0])
    assert cp == 1.0 and ca == [1.0, 0.75, 0.5, 1 / L, 0.0]
    # everything abstains: both are 0, whatever the labels
    cp, ca = oracle.certified_metrics([-1] * L, [0.0] * L, labels, [0.0, 0.5])
    assert cp == 0.0 and ca == [0.0, 0.0]
    # half abstain: CP = 1/2 and the denominator of CA is the certified half (the equation's own denominator)
    classes = [labels[i] if i % 2 == 0 else -1 for i in range(L)]
    cp, ca = oracle.certified_metrics(classes, [1.0] * L, labels, [0.5, 1.0, 1.5])
    assert cp == 0.5 and ca == [1.0, 1.0, 0.0]
    # wrong classes count as certified (CP) but never as accurate (CA)
    wrong = [(labels[i] + 1) % 10 for i in range(L)]
    cp, ca = oracle.certified_metrics(wrong, [1.0] * L, labels, [0.0])
    assert cp == 1.0 and ca == [0.0]
    # CA is non-increasing in r and invariant under a permutation of the inputs
    rng = np.random.default_rng(3)
    classes = rng.integers(-1, 10, size=200)
    radii = rng.random(200)
    lab = rng.integers(0, 10, size=200)
    th = [0.0, 0.1, 0.3, 0.6, 0.9]
    cp, ca = oracle.certified_metrics(classes, radii, lab, th)
    assert all(a >= b for a, b in zip(ca, ca[1:]))
    perm = rng.permutation(200)
    assert oracle.certified_metrics(classes[perm], radii[perm], lab[perm], th) == (cp, ca)
    assert oracle.certified_metrics([], [], [], [0.5]) == (0.0, [0.0])


# --------------------------------------------------------- whole-loop properties

def test_prefix_partition_and_limit_properties():
    model = wl.tiny_cnn()
    m = oracle.Model(model)
    x = wl.images(1)[0]
    full, lg = oracle.sample_counts(m, x, wl.NOISE_SEED, 0, 1, 0, 200, 0.25, want_logits=True)
    parts = sum(oracle.sample_counts(m, x, wl.NOISE_SEED, 0, 1, a, b - a, 0.25)
                for a, b in ((0, 1), (1, 64), (64, 177), (177, 200)))
    np.testing.assert_array_equal(full, parts)
    assert full.sum() == 200
    np.testing.assert_array_equal(np.bincount(lg.argmax(1), minlength=10), full)
    # sample j's logits are f(noisy_input(j))
    j = 17
    a0 = oracle.noisy_input(x, wl.NOISE_SEED, 0, 1, j, 0.25)
    np.testing.assert_array_equal(oracle.forward(m, a0), lg[j])
    # sigma -> 0: every sample is the clean image, all votes on f(x), radius maximal
    clean = int(np.argmax(oracle.forward(m, x)))
    cls, rad, c0, c1 = oracle.certify(m, x, 1, 0, 50, 300, 1e-4, ALPHA)
    assert c1[clean] == 300 and c0[clean] == 50 and cls == clean
    assert abs(rad - 1e-4 * st.norm.ppf(ALPHA ** (1 / 300))) < 1e-12
    # phases use different draws
    assert not np.array_equal(oracle.noise(1, 0, 0, 0, 0.25, 0, 64), oracle.noise(1, 0, 1, 0, 0.25, 0, 64))
    pc, pcounts = oracle.predict(m, x, wl.NOISE_SEED, 0, 120, 0.25, ALPHA)
    np.testing.assert_array_equal(pcounts, oracle.sample_counts(m, x, wl.NOISE_SEED, 0, 2, 0, 120, 0.25))
    assert pc == oracle.predict_decide(pcounts, ALPHA)


def test_workload_shapes():
    assert wl.macs_per_sample(wl.tiny_cnn()) == 1_622_336
    assert wl.macs_per_sample(wl.resnet20()) == 40_813_184
    m110 = wl.resnet110()
    assert wl.macs_per_sample(m110) == 253_149_824 and len(m110["layers"]) == 113
    a = wl.images(2, seed=5)
    b = wl.images(2, seed=5)
    np.testing.assert_array_equal(a, b)
    assert a.dtype == np.uint8 and a.shape == (2, 3, 32, 32) and a.min() == 0 and a.max() == 255


# ------------------------------------------------------------------ integer-only certification (Thm 3.2, Thm 3.1)

def test_integer_certify_decide_against_the_normal_radius_and_symmetry():
    """Theorem 3.2 steps 2-3: the table quantile q (pixel levels) must agree with Algorithm 1's sigma * Phi^-1(p_A)
    within 1.5 levels once the lattice is fine (255 sigma >= 30), abstain exactly when Algorithm 1 abstains, grow with
    the vote count; Theorem 3.1's two-sided form with a lone runner-up (n_B = N - n_A, so p_B^ub = 1 - p_A^lb) is the
    symmetric quantile: q_A - q_B within one level of 2 q_A."""
    N, alpha = 100_000, 0.001
    for sigma in (0.12, 0.25, 0.5, 1.0):
        prev_q = -1
        for n_a in (50_000, 50_600, 52_000, 60_000, 80_000, 99_000, 99_990, N):
            counts = [n_a, N - n_a, 0, 0]
            cls, radius, p_l = oracle.certify_decide([7, 1, 0, 0], counts, N, sigma, alpha)
            icls, q, q2 = oracle.certify_integer_decide([7, 1, 0, 0], counts, N, sigma, alpha)
            assert icls == cls
            if cls == -1:
                assert (q, q2) == (0, 0)
                continue
            assert q2 == q * q and q >= prev_q
            prev_q = q
            assert abs(q / 255.0 - radius) <= 1.5 / 255.0, (sigma, n_a, q, radius)
            tcls, d, d2 = oracle.certify_integer_decide([7, 1, 0, 0], counts, N, sigma, alpha, two_sided=True)
            assert tcls == cls and d2 == d * d and abs(d - 2 * q) <= 1
    # a runner-up weaker than the complement (votes spread over a third class): Theorem 3.1's radius exceeds
    # Algorithm 1's, and equals the normal form (sigma / 2)(Phi^-1(p_A^lb) - Phi^-1(p_B^ub)) within the lattice step
    from scipy.stats import norm
    counts = [70_000, 29_000, 1_000, 0]
    _, q, _ = oracle.certify_integer_decide([5, 1, 0, 0], counts, N, 0.5, alpha)
    _, d, _ = oracle.certify_integer_decide([5, 1, 0, 0], counts, N, 0.5, alpha, two_sided=True)
    p_a = oracle.lower_conf_bound(70_000, N, alpha)
    p_b = 1.0 - oracle.lower_conf_bound(N - 29_000, N, alpha)
    assert d > 2 * q
    assert abs(d / 255.0 - 0.5 * (norm.ppf(p_a) - norm.ppf(p_b))) <= 3.0 / 255.0
    # Theorem 3.1's premise fails (p_A^lb < p_B^ub) although Algorithm 1 would certify: cannot happen with p_A > 1/2
    # and n_B <= N - n_A, so the two forms abstain together
    for n_a in (50_100, 50_400):
        counts = [n_a, N - n_a, 0, 0]
        assert oracle.certify_integer_decide([3, 1, 0, 0], counts, N, 0.25, alpha, two_sided=True)[0] == \
               oracle.certify_integer_decide([3, 1, 0, 0], counts, N, 0.25, alpha)[0]


# ------------------------------------------------------------------ second samplers (Sec. 3.3, Sec. 4.1)

def _pooled_chi2_p(obs, exp, n):
    keep = exp >= 5.0
    lo, hi = np.argmax(keep), len(keep) - np.argmax(keep[::-1])
    o = np.concatenate(([obs[:lo].sum()], obs[lo:hi], [obs[hi:].sum()]))
    e = np.concatenate(([exp[:lo].sum()], exp[lo:hi], [exp[hi:].sum()]))
    e[0] += n - e.sum()
    return st.chi2.sf(((o - e) ** 2 / e).sum(), df=len(o) - 1)


@pytest.mark.parametrize("sigma", [0.12, 0.5])
def test_table_sampler_agrees_with_the_rejection_sampler(sigma):
    """The table-free rejection sampler the paper cites for its noise (Sec. 3.3) and the oracle's inverse-CDF table
    draw from the same law: each passes the exact-pmf chi-square of Eq. 2, and their two histograms pass a
    two-sample chi-square against each other."""
    n = 2_000_000
    T = oracle.dgauss_halfwidth(sigma)
    rej, proposals = oracle.rejection_dgauss(sigma, seed=4242, n=n)
    assert n <= proposals < 4 * n                       # the publication bounds the expected number of proposals
    assert np.abs(rej).max() <= T
    pmf = _pmf_direct(sigma, np.arange(-T, T + 1))
    h_rej = np.bincount(rej + T, minlength=2 * T + 1).astype(np.float64)
    assert _pooled_chi2_p(h_rej, pmf * n, n) > 1e-3
    tab = oracle.noise(seed=5, image_id=1, phase=0, j=77, sigma=sigma, e0=0, n=n)
    h_tab = np.bincount(tab + T, minlength=2 * T + 1).astype(np.float64)
    both = h_rej + h_tab
    use = both >= 10
    chi2 = (((h_rej - h_tab) ** 2)[use] / both[use]).sum()
    assert st.chi2.sf(chi2, df=int(use.sum()) - 1) > 1e-3
    s_int = 255.0 * sigma
    assert abs(rej.mean()) < 5 * s_int / math.sqrt(n)
    assert abs(rej.astype(np.float64).var() - s_int ** 2) < 5 * s_int ** 2 * math.sqrt(2.0 / n)


@pytest.mark.parametrize("sigma", [0.12, 1.0])
def test_rounded_gaussian_noise_of_the_comparison_method(sigma):
    """FloatRS-quant's noise (Sec. 4.1): continuous Gaussian, then quantised.  The oracle's table must be the CDF of
    round(255 sigma g) at the half-integers (SciPy's normal CDF), the draws must pass the chi-square of that law, and
    their variance must carry the rounding's 1/12 that the discrete Gaussian of Eq. 2 does not have."""
    s_int = 255.0 * sigma
    T = oracle.dgauss_halfwidth(sigma)
    cum = oracle.rgauss_table(sigma).astype(np.float64)
    z = np.arange(-T, T + 1)
    ref = np.floor(st.norm.cdf((z + 0.5) / s_int) * 2.0 ** 32)
    assert np.abs(cum[:-1] - ref[:-1]).max() <= 64           # the two erfc implementations differ in the last bits
    assert cum[-1] == 2.0 ** 32 - 1 and (np.diff(cum) >= 0).all()
    n = 2_000_000
    oracle.set_noise_kind(1)
    try:
        draws = oracle.noise(seed=8, image_id=2, phase=1, j=5, sigma=sigma, e0=0, n=n)
    finally:
        oracle.set_noise_kind(0)
    pmf = st.norm.cdf((z + 0.5) / s_int) - st.norm.cdf((z - 0.5) / s_int)
    obs = np.bincount(draws + T, minlength=2 * T + 1).astype(np.float64)
    assert _pooled_chi2_p(obs, pmf * n, n) > 1e-3
    var = draws.astype(np.float64).var()
    assert abs(var - (s_int ** 2 + 1.0 / 12.0)) < 5 * s_int ** 2 * math.sqrt(2.0 / n)
    # and it is not the law of Eq. 2: the default kind draws something else from the same uniforms
    assert (oracle.noise(seed=8, image_id=2, phase=1, j=5, sigma=sigma, e0=0, n=20000) != draws[:20000]).any()
