"""GPU parity on inputs that make the vote-level checks bite.

Random networks vote unanimously, so counts alone would pass for any kernel that keeps one logit on top.  The
models used here have a balanced final layer (workloads.spread_model): the votes of one image spread over most
classes, exact ties for the maximum are frequent, CERTIFY abstains or returns a radius below the maximum, and
PREDICT abstains.  Every logit row, every count, the class and the radius must equal the CPU oracle's
(Algorithm 1, Algorithm 2; ties go to the lowest class index).
"""
import numpy as np
import pytest

import oracle
import workloads as wl
import paper_2108_09413_b200 as isc

pytestmark = pytest.mark.gpu
SEED = wl.NOISE_SEED
ALPHA = 0.001
ENGINES = {"layerwise": 1, "line": 3}
BOOST = {"tiny_cnn": 160, "resnet20": 200}      # bias added to class 0: a majority that is not unanimous


def _rows_equal(got, exp, what):
    bad = np.nonzero((got != exp).any(axis=1))[0]
    assert bad.size == 0, f"{what}: {bad.size} logit rows differ, first {bad[:5]}"


@pytest.mark.parametrize("name,n", [("tiny_cnn", 4000), ("resnet20", 2000)])
def test_spread_logits_and_counts_every_engine(name, n):
    model = wl.spread_model(name)
    gm, om = isc.Model(model), oracle.Model(model)
    x = wl.spread_image()
    ecounts, elog = oracle.sample_counts(om, x, SEED, 0, 1, 0, n, 0.25, want_logits=True)
    # the inputs do what they are for: at least three classes with 5 % of the votes, exact ties for the maximum
    assert (ecounts >= 0.05 * n).sum() >= 3
    top = elog.max(axis=1)
    tied = ((elog == top[:, None]).sum(axis=1) > 1)
    assert tied.any()
    for ename, eng in ENGINES.items():
        gm.set_option("engine", eng)
        for batch in (0, 1000):
            gm.set_option("batch", batch)
            counts, log = gm.sample_counts(x, SEED, 0, 1, 0, n, 0.25, want_logits=True)
            _rows_equal(log, elog, f"{name} {ename} batch {batch}")
            np.testing.assert_array_equal(counts, ecounts, err_msg=f"{name} {ename} batch {batch}")
        # any partition of the range gives the same counts
        parts = sum(gm.sample_counts(x, SEED, 0, 1, a, b - a, 0.25) for a, b in ((0, 1), (1, 130), (130, 1031), (1031, n)))
        np.testing.assert_array_equal(parts, ecounts)


@pytest.mark.parametrize("name,N", [("tiny_cnn", 4000), ("resnet20", 1000)])
def test_spread_certify_and_predict_abstain_and_partial_radius(name, N):
    x = wl.spread_image()
    r_max = oracle.certify_decide([N] + [0] * 9, [N] + [0] * 9, N, 0.25, ALPHA)[1]
    seen = set()
    for boost in (0, BOOST[name]):
        model = wl.spread_model(name, boost=boost)
        gm, om = isc.Model(model), oracle.Model(model)
        ecls, erad, ec0, ec1 = oracle.certify(om, x, SEED, 3, 100, N, 0.25, ALPHA)
        epc, epcounts = oracle.predict(om, x, SEED, 3, 400, 0.25, ALPHA)
        seen.add("abstain" if ecls == -1 else "partial" if 0.0 < erad < r_max else "other")
        for ename, eng in ENGINES.items():
            gm.set_option("engine", eng)
            cls, rad, c0, c1 = gm.certify(x, SEED, 3, 100, N, 0.25, ALPHA)
            np.testing.assert_array_equal(c0, ec0, err_msg=ename)
            np.testing.assert_array_equal(c1, ec1, err_msg=ename)
            assert (cls, rad) == (ecls, erad), ename
            pc, pcounts = gm.predict(x, SEED, 3, 400, 0.25, ALPHA)
            np.testing.assert_array_equal(pcounts, epcounts, err_msg=ename)
            assert pc == epc, ename
        gm.close()
    assert seen == {"abstain", "partial"}, seen


def test_integer_certification_from_real_counts():
    """isc_certify_integer (Theorem 3.2 steps 2-3, Theorem 3.1) from the votes of the GPU loop: counts, class, q and
    q^2 equal the oracle's, for an abstaining image and for a majority that is not unanimous."""
    x = wl.spread_image()
    N = 4000
    seen = set()
    for boost in (0, BOOST["tiny_cnn"]):
        model = wl.spread_model("tiny_cnn", boost=boost)
        gm, om = isc.Model(model), oracle.Model(model)
        _, _, ec0, ec1 = oracle.certify(om, x, SEED, 3, 100, N, 0.25, ALPHA)
        for two in (False, True):
            cls, q, q2, c0, c1 = gm.certify_integer(x, SEED, 3, 100, N, 0.25, ALPHA, two_sided=two)
            np.testing.assert_array_equal(c0, ec0); np.testing.assert_array_equal(c1, ec1)
            assert (cls, q, q2) == oracle.certify_integer_decide(ec0, ec1, N, 0.25, ALPHA, two)
            seen.add(cls)
    assert seen == {-1, 0}


def test_resnet110_logits_where_a_cta_runs_several_groups():
    """One launch of 1776 samples = 444 groups of four: with one CTA per SM (148) every CTA carries three groups in
    turn.  Rows of the second and third turn are compared with the oracle; the counts of the whole launch follow from
    the logits (lowest index among the maxima)."""
    model = wl.spread_model("resnet110")
    gm, om = isc.Model(model), oracle.Model(model)
    gm.set_option("engine", ENGINES["line"])
    x = wl.spread_image()
    n = 1776
    counts, log = gm.sample_counts(x, SEED, 1, 1, 0, n, 0.25, want_logits=True)
    assert gm.get_info("engine") == 3
    for first in (0, 592, 1712):
        _, elog = oracle.sample_counts(om, x, SEED, 1, 1, first, 64, 0.25, want_logits=True)
        _rows_equal(log[first:first + 64], elog, f"samples {first}..{first + 63}")
    votes = np.bincount(np.argmax(log.astype(np.int32), axis=1), minlength=10)
    np.testing.assert_array_equal(counts, votes)
    assert (counts > 0).sum() >= 3


def test_resnet110_line_engine_many_launches_and_ragged_batches_spread():
    """Counts must not depend on how the samples are cut into launches: several hundred launches with group counts
    that do not divide the batch, on votes that fill every bin."""
    gm = isc.Model(wl.spread_model("resnet110"))
    gm.set_option("engine", ENGINES["line"])
    x = wl.spread_image()
    ref = None
    for batch in (0, 257, 4099):
        gm.set_option("batch", batch)
        c = gm.sample_counts(x, SEED, 2, 1, 3, 20001, 0.25)
        assert c.sum() == 20001
        ref = c if ref is None else ref
        np.testing.assert_array_equal(c, ref, err_msg=f"batch {batch}")
    assert (ref >= 1000).sum() >= 3


def test_full_n_certify_tiny_and_resnet20_ragged_tail():
    """Full-size sample counts against the oracle: N = 100,000 on the tiny CNN (the size of the paper's CIFAR-10
    runs, Sec. 4.1) and N = 20,001 in launches of 1024 (ragged tail) on ResNet-20."""
    x = wl.spread_image()
    model = wl.spread_model("tiny_cnn", boost=BOOST["tiny_cnn"])
    gm, om = isc.Model(model), oracle.Model(model)
    exp = oracle.certify(om, x, SEED, 9, 100, 100_000, 0.25, ALPHA)
    for eng in ENGINES.values():
        gm.set_option("engine", eng)
        got = gm.certify(x, SEED, 9, 100, 100_000, 0.25, ALPHA)
        assert (got[0], got[1]) == (exp[0], exp[1])
        np.testing.assert_array_equal(got[2], exp[2]); np.testing.assert_array_equal(got[3], exp[3])
    assert exp[0] == 0 and 0.0 < exp[1] < 0.953
    model = wl.spread_model("resnet20", boost=BOOST["resnet20"])
    gm, om = isc.Model(model), oracle.Model(model)
    gm.set_option("batch", 1024)
    exp = oracle.certify(om, x, SEED, 9, 100, 20_001, 0.25, ALPHA)
    got = gm.certify(x, SEED, 9, 100, 20_001, 0.25, ALPHA)
    assert gm.get_info("engine") == 3
    assert (got[0], got[1]) == (exp[0], exp[1])
    np.testing.assert_array_equal(got[2], exp[2]); np.testing.assert_array_equal(got[3], exp[3])


# ------------------------------------------------------------------ the resident engine's whole accepted range

def _conv(rng, in_tensor, cin, cout, k, stride, relu, zp_in, zp_out, res_tensor=-1, zp_res=0, shift_lo=1, shift_hi=20):
    return dict(op=wl.OP_CONV2D, in_tensor=in_tensor, res_tensor=res_tensor, cin=cin, cout=cout, kh=k, kw=k,
                stride=stride, pad=k // 2, relu=relu, zp_in=zp_in, zp_out=zp_out, zp_res=zp_res,
                w=rng.integers(-127, 128, (cout, cin, k, k)).astype(np.int8),
                bias=rng.integers(-(1 << 16), (1 << 16) + 1, cout).astype(np.int32),
                mult=rng.integers(2 ** 30, 2 ** 31, cout).astype(np.int32),
                shift=rng.integers(shift_lo, shift_hi + 1, cout).astype(np.int8),
                res_mult=int(rng.integers(2 ** 30, 2 ** 31)) if res_tensor >= 0 else 0,
                res_shift=int(rng.integers(-1, 1)) if res_tensor >= 0 else 0)


def random_cifar_net(seed):
    """32x32 input, three stages of basic blocks with stride-2 transitions and projection shortcuts, global average
    pool, FC -- with every parameter drawn from the whole range the line-tiled engine accepts.  The tensors that carry
    a stage's residual stream share one zero-point (the engine adds the residual in place, padding included, and keeps
    three 72 KB stage-1 tensors in shared memory only that way); everything else is drawn freely."""
    rng = np.random.default_rng(seed)
    in_c = int(rng.integers(1, 5))
    widths = (16, 32, 64) if seed % 3 else (16, int(rng.choice([16, 32])), int(rng.choice([16, 32, 64])))
    n_classes = int(rng.choice([1, 2, 7, 10, 33, 101, 128]))
    narrow = seed % 2 == 0                 # half of the networks keep mid-range shifts so that deep layers stay lively
    sl, sh = (7, 12) if narrow else (1, 20)
    zp = lambda: int(rng.integers(-128, 128))
    trunk = [zp(), zp(), zp()]
    zps = {0: int(rng.integers(0, 256))}
    L = [_conv(rng, 0, in_c, widths[0], int(rng.choice([1, 3])), 1, int(rng.integers(0, 2)), zps[0], trunk[0], shift_lo=sl, shift_hi=sh)]
    zps[1] = L[0]["zp_out"]
    cur, cin = 1, widths[0]
    for si, width in enumerate(widths):
        for b in range(int(rng.integers(1, 3))):
            stride = 2 if (si > 0 and b == 0) else 1
            L.append(_conv(rng, cur, cin, width, 3, stride, int(rng.integers(0, 2)), zps[cur], zp(), shift_lo=sl, shift_hi=sh))
            y1 = len(L); zps[y1] = L[-1]["zp_out"]
            if stride != 1 or cin != width:
                L.append(_conv(rng, cur, cin, width, 1, stride, int(rng.integers(0, 2)), zps[cur], trunk[si], shift_lo=sl, shift_hi=sh))
                short = len(L); zps[short] = L[-1]["zp_out"]
            else:
                short = cur
            zp_res = zps[short] if rng.integers(0, 2) else zp()
            L.append(_conv(rng, y1, width, width, int(rng.choice([3, 3, 1])), 1, int(rng.integers(0, 2)), zps[y1], trunk[si],
                           res_tensor=short, zp_res=zp_res, shift_lo=sl, shift_hi=sh))
            cur, cin = len(L), width
            zps[cur] = L[-1]["zp_out"]
    size = 8
    pool = wl._gavgpool(cur, cin, size * size, zps[cur])
    pool["zp_out"] = zp()
    pool["relu"] = int(rng.integers(0, 2))
    L.append(pool)
    fc = _conv(rng, len(L), cin, n_classes, 1, 1, int(rng.integers(0, 2)), pool["zp_out"], zp(), shift_lo=4, shift_hi=14)
    fc["op"] = wl.OP_FC
    L.append(fc)
    return dict(name=f"random_cifar_{seed}", in_shape=(in_c, 32, 32), n_classes=n_classes, layers=L), widths


@pytest.mark.parametrize("seed", range(12))
def test_random_cifar_nets_every_tensor_on_the_resident_engine(seed):
    model, widths = random_cifar_net(500 + seed)
    gm, om = isc.Model(model), oracle.Model(model)
    if widths == (16, 32, 64):
        assert gm.get_info("has_line_engine") == 1
    rng = np.random.default_rng(seed)
    x = rng.integers(0, 256, model["in_shape"]).astype(np.uint8)
    sizes = [oracle.tensor_size(om, k) for k in range(om.n_layers + 1)]
    engines = [1, 3] if gm.get_info("has_line_engine") == 1 else [1]
    sigma = float(rng.choice([0.12, 0.25, 0.5]))
    a0 = oracle.noisy_input(x, 5, seed, 1, 6, sigma)
    for eng in engines:
        gm.set_option("engine", eng)
        last = om.n_layers if eng == 1 else om.n_layers - 2        # the resident engine holds the convolution tensors
        for k in range(0 if eng == 3 else 1, last + 1):
            exp = a0.ravel().astype(np.int32) if k == 0 else oracle.forward(om, a0, dump_tensor=k)[1]
            got = gm.debug_tensor(x, 5, seed, 1, 6, sigma, k, sizes[k])
            bad = np.nonzero(got != exp)[0]
            assert bad.size == 0, f"engine {eng} tensor {k}: {bad.size} of {exp.size} differ, first at {bad[:8]}"
    ec, el = oracle.sample_counts(om, x, 5, seed, 1, 0, 44, sigma, want_logits=True)
    for eng in engines:
        gm.set_option("engine", eng)
        gc, gl = gm.sample_counts(x, 5, seed, 1, 0, 44, sigma, want_logits=True)
        _rows_equal(gl, el, f"engine {eng}")
        np.testing.assert_array_equal(gc, ec)
