"""GPU parity: every value the CUDA library returns through its C ABI is compared, bit for bit,
with the CPU oracle on the same seeded inputs."""
import ctypes as C

import numpy as np
import pytest

import oracle
import workloads as wl
import paper_2108_09413_b200 as isc

pytestmark = pytest.mark.gpu
SEED = wl.NOISE_SEED
ALPHA = 0.001
ENGINES = {"layerwise": 1, "line": 3}


def _pair(model):
    return isc.Model(model), oracle.Model(model)


def _tensor_sizes(om):
    return [oracle.tensor_size(om, k) for k in range(om.n_layers + 1)]


@pytest.mark.parametrize("sigma", [0.12, 0.25, 0.5, 1.0])
def test_noisy_input_matches(sigma):
    gm, om = _pair(wl.tiny_cnn())
    x = wl.images(1)[0]
    for image_id, phase, j in ((0, 0, 0), (5, 1, 77), ((3 << 32) | 9, 2, (1 << 33) + 12345), (1, 255, 99999)):
        got = gm.debug_tensor(x, SEED, image_id, phase, j, sigma, 0, x.size)
        np.testing.assert_array_equal(got, oracle.noisy_input(x, SEED, image_id, phase, j, sigma).ravel())


def test_tiny_cnn_every_tensor_and_full_certify():
    model = wl.CONFIGS[0]["model"]()
    gm, om = _pair(model)
    x = wl.images(1, seed=wl.CONFIGS[0]["image_seed"])[0]
    sizes = _tensor_sizes(om)
    for j in (0, 3, 1000):
        a0 = oracle.noisy_input(x, SEED, 0, 1, j, 0.25)
        for k in range(1, om.n_layers + 1):
            _, exp = oracle.forward(om, a0, dump_tensor=k)
            got = gm.debug_tensor(x, SEED, 0, 1, j, 0.25, k, sizes[k])
            np.testing.assert_array_equal(got, exp, err_msg=f"tensor {k} sample {j}")
    for name, eng in ENGINES.items():
        gm.set_option("engine", eng)
        cls, rad, c0, c1 = gm.certify(x, SEED, 0, 100, 1000, 0.25, ALPHA)
        ecls, erad, ec0, ec1 = oracle.certify(om, x, SEED, 0, 100, 1000, 0.25, ALPHA)
        np.testing.assert_array_equal(c0, ec0)
        np.testing.assert_array_equal(c1, ec1)
        assert (cls, rad) == (ecls, erad), name
        pc, pcounts = gm.predict(x, SEED, 0, 500, 0.25, ALPHA)
        epc, epcounts = oracle.predict(om, x, SEED, 0, 500, 0.25, ALPHA)
        np.testing.assert_array_equal(pcounts, epcounts)
        assert pc == epc


def _logit_parity(model, x, image_id, phase, first, n, sigma, engines=ENGINES):
    gm, om = _pair(model)
    ecounts, elog = oracle.sample_counts(om, x, SEED, image_id, phase, first, n, sigma, want_logits=True)
    for name, eng in engines.items():
        gm.set_option("engine", eng)
        counts, log = gm.sample_counts(x, SEED, image_id, phase, first, n, sigma, want_logits=True)
        bad = np.nonzero((log != elog).any(axis=1))[0]
        assert bad.size == 0, f"{name}: first mismatching sample {bad[:5]} of {n}"
        np.testing.assert_array_equal(counts, ecounts, err_msg=name)
    gm.close()


@pytest.mark.parametrize("sigma", [0.12, 0.25, 0.5])
def test_resnet20_logits_and_prefix_counts(sigma):
    cfg = wl.CONFIGS[1]
    xs = wl.images(3, seed=cfg["image_seed"])
    model = cfg["model"]()
    for i in (0, 2):
        _logit_parity(model, xs[i], i, 1, 0, 300, sigma)          # spans several tiles + ragged tail
    _logit_parity(model, xs[1], 1, 0, 0, 100, sigma)              # the selection phase


@pytest.mark.parametrize("engine", ["layerwise", "line"])
def test_resnet20_every_tensor(engine):
    model = wl.resnet20()
    gm, om = _pair(model)
    gm.set_option("engine", ENGINES[engine])
    x = wl.images(1, seed=77)[0]
    sizes = _tensor_sizes(om)
    a0 = oracle.noisy_input(x, SEED, 4, 1, 9, 0.5)
    last = om.n_layers if engine == "layerwise" else om.n_layers - 2     # resident: conv tensors only
    first = 1 if engine == "layerwise" else 0
    for k in range(first, last + 1):
        exp = a0.ravel().astype(np.int32) if k == 0 else oracle.forward(om, a0, dump_tensor=k)[1]
        got = gm.debug_tensor(x, SEED, 4, 1, 9, 0.5, k, sizes[k])
        bad = np.nonzero(got != exp)[0]
        assert bad.size == 0, f"{engine}: tensor {k}: {bad.size} of {exp.size} differ, first at {bad[:8]}"


def test_resident_engine_is_used_for_cifar_resnets():
    for model in (wl.tiny_cnn(), wl.resnet20(), wl.resnet110()):
        gm = isc.Model(model)
        assert gm.get_info("has_line_engine") == 1, model["name"]
        gm.sample_counts(wl.images(1)[0], SEED, 0, 1, 0, 8, 0.25)
        assert gm.get_info("engine") == 3
        gm.close()
    gm = isc.Model(wl.resnet50())
    assert gm.get_info("has_line_engine") == 0


def test_resnet110_logits_and_prefix_counts():
    cfg = wl.CONFIGS[2]
    xs = wl.images(2, seed=cfg["image_seed"])
    model = cfg["model"]()
    _logit_parity(model, xs[0], 0, 1, 0, 160, 0.25)
    _logit_parity(model, xs[1], 1, 1, 99_990, 10, 0.25)          # the tail of N = 100,000
    _logit_parity(model, xs[1], 1, 0, 0, 40, 1.0)                # sweep sigma of config 4


def test_resnet50_logits():
    """Config 3 (Sec. 4.1: ResNet-50 on 3 x 224 x 224 inputs, 101 classes): 64 samples on the tensor-core
    layer-by-layer engine (the automatic choice), a few on the plain one."""
    cfg = wl.CONFIGS[3]
    x = wl.images(1, seed=cfg["image_seed"], shape=cfg["shape"])[0]
    model = cfg["model"]()
    gm = isc.Model(model)
    assert gm.get_info("has_tensor_core_layers") == 1
    gm.sample_counts(x, SEED, 0, 1, 0, 2, 0.5)
    assert gm.get_info("engine") == 2
    gm.close()
    _logit_parity(model, x, 0, 1, 0, 64, 0.5, engines={"auto": 0})
    _logit_parity(model, x, 0, 1, 61, 6, 0.5, engines={"layerwise": 1, "tensorcore": 2})


def test_resnet50_every_tensor_on_the_tensor_core_engine():
    from concurrent.futures import ThreadPoolExecutor
    cfg = wl.CONFIGS[3]
    x = wl.images(2, seed=cfg["image_seed"], shape=cfg["shape"])[1]
    model = cfg["model"]()
    gm, om = _pair(model)
    gm.set_option("engine", 2)
    sizes = _tensor_sizes(om)
    a0 = oracle.noisy_input(x, SEED, 1, 1, 5, 0.5)
    with ThreadPoolExecutor(16) as pool:          # one oracle forward per tensor; the C call releases the GIL
        expected = list(pool.map(lambda k: oracle.forward(om, a0, dump_tensor=k)[1], range(1, om.n_layers + 1)))
    for k in range(1, om.n_layers + 1):
        got = gm.debug_tensor(x, SEED, 1, 1, 5, 0.5, k, sizes[k])
        bad = np.nonzero(got != expected[k - 1])[0]
        assert bad.size == 0, f"tensor {k}: {bad.size} of {got.size} differ, first at {bad[:8]}"


def _bottleneck_net(rng, fast=None):
    """Two bottleneck-style residual blocks on a small ragged image.  `fast` = (res_mult, res_shift, zp_res): every
    shift >= 2 and that residual rescale on both blocks, so that the 32-bit epilogue runs."""
    h, w = int(rng.integers(9, 23)), int(rng.integers(2, 6)) * 4
    zp = lambda: int(rng.integers(-128, 128))
    c0, c1 = int(rng.choice([64, 128])), int(rng.choice([64, 128, 256]))
    z = [int(rng.integers(0, 256)), zp(), zp(), zp(), zp(), zp()]
    if fast:
        z[4] = z[5] = fast[2]
    L = [_rand_conv(rng, 0, 3, c0, 3, 1, 1, 1, z[0], z[1]),
         _rand_conv(rng, 1, c0, c0, 1, 1, 0, int(rng.integers(0, 2)), z[1], z[2]),
         _rand_conv(rng, 2, c0, c0, 3, 2, 1, int(rng.integers(0, 2)), z[2], z[3]),
         _rand_conv(rng, 1, c0, c1, 1, 2, 0, 0, z[1], z[4])]
    L.append(_rand_conv(rng, 3, c0, c1, 1, 1, 0, 1, z[3], z[5], res_tensor=4, zp_res=z[4]))
    L.append(_rand_conv(rng, 5, c1, c1, 3, 1, 1, 1, z[5], z[1], res_tensor=5, zp_res=z[5]))
    if fast:
        for layer in L:
            layer["shift"] = np.maximum(layer["shift"], 2).astype(np.int8)
            if layer["res_tensor"] >= 0:
                layer["res_mult"], layer["res_shift"] = fast[0], fast[1]
    model = dict(in_shape=(3, h, w), n_classes=5, layers=L)
    om_tmp = oracle.Model(dict(model, n_classes=1))
    hw = oracle.tensor_size(om_tmp, 6) // c1
    L.append(wl._gavgpool(6, c1, hw, z[1]))
    fc = _rand_conv(rng, 7, c1, 5, 1, 1, 0, 0, z[1], zp())
    fc["op"] = wl.OP_FC
    L.append(fc)
    return model


def _bottleneck_parity(model, rng, seed, tensor_copy=1):
    gm, om = _pair(model)
    gm.set_option("engine", 2)
    gm.set_option("tensor_copy", tensor_copy)
    x = rng.integers(0, 256, model["in_shape"]).astype(np.uint8)
    sizes = _tensor_sizes(om)
    a0 = oracle.noisy_input(x, 5, seed, 1, 2, 0.25)
    for k in range(1, om.n_layers + 1):
        _, exp = oracle.forward(om, a0, dump_tensor=k)
        got = gm.debug_tensor(x, 5, seed, 1, 2, 0.25, k, sizes[k])
        np.testing.assert_array_equal(got, exp, err_msg=f"tensor {k}")
    ec, el = oracle.sample_counts(om, x, 5, seed, 1, 0, 37, 0.25, want_logits=True)
    gc, gl = gm.sample_counts(x, 5, seed, 1, 0, 37, 0.25, want_logits=True)
    assert gm.get_info("engine") == 2
    np.testing.assert_array_equal(gl, el)
    np.testing.assert_array_equal(gc, ec)


@pytest.mark.parametrize("seed", range(4))
def test_random_bottleneck_nets_on_the_tensor_core_engine(seed):
    """Small bottleneck networks with ragged sizes, strides, every zero-point and shift, residual rescales of all
    allowed shifts: the implicit-GEMM kernel's tiles end inside rows and images, its padding is a non-trivial
    zero-point."""
    rng = np.random.default_rng(900 + seed)
    _bottleneck_parity(_bottleneck_net(rng), rng, seed, tensor_copy=seed & 1)      # both ways of bringing 1 x 1 operand rows


@pytest.mark.parametrize("res", [(1304428746, 0, 77), (1334892440, -1, -63), (1 << 30, 0, 0),         # no offset form
                                 (1979951843, 0, 0), (1435772024, -1, -128)])                           # offset form
def test_bottleneck_nets_32_bit_epilogue_both_residual_forms(res):
    """The same networks with every shift >= 2, so that the kernel's 32-bit epilogue runs, and residual rescales
    with and without the offset form (isc_debug_residual_form): both forms of the residual term against the oracle."""
    has_form = isc.residual_form(*res) is not None
    assert has_form == (res[0] in (1979951843, 1435772024))
    rng = np.random.default_rng(950 + res[0] % 97)
    _bottleneck_parity(_bottleneck_net(rng, fast=res), rng, res[0] % 5, tensor_copy=res[0] % 2)


def test_partition_and_batch_invariance():
    model = wl.resnet20()
    gm = isc.Model(model)
    x = wl.images(1, seed=3)[0]
    n = 2500
    for eng in ENGINES.values():
        gm.set_option("engine", eng)
        gm.set_option("batch", 0)
        full = gm.sample_counts(x, SEED, 7, 1, 0, n, 0.25)
        assert full.sum() == n
        parts = sum(gm.sample_counts(x, SEED, 7, 1, a, b - a, 0.25)
                    for a, b in ((0, 1), (1, 130), (130, 1031), (1031, n)))
        np.testing.assert_array_equal(full, parts)
        for batch in (256, 1024, 4096, 16384):
            gm.set_option("batch", batch)
            np.testing.assert_array_equal(gm.sample_counts(x, SEED, 7, 1, 0, n, 0.25), full)
    gm.set_option("batch", 0)
    assert np.array_equal(gm.sample_counts(x, SEED, 7, 1, 0, 0, 0.25), np.zeros(10, np.int32))


def test_resnet110_line_engine_many_launches_and_ragged_batches():
    """Counts must not depend on how the samples are cut into launches (Algorithm 1 counts votes, nothing else):
    several hundred launches of the line-tiled engine with group counts that do not divide the batch."""
    gm = isc.Model(wl.resnet110())
    gm.set_option("engine", ENGINES["line"])
    xs = wl.images(2, seed=5)
    for sigma, img in ((0.12, 0), (1.0, 1)):
        ref = None
        for batch in (0, 257, 4099):
            gm.set_option("batch", batch)
            c = gm.sample_counts(xs[img], SEED, img, 1, 3, 20001, sigma)
            assert c.sum() == 20001
            ref = c if ref is None else ref
            np.testing.assert_array_equal(c, ref, err_msg=f"sigma {sigma} batch {batch}")
    assert gm.get_info("engine") == 3


def test_certify_batch_equals_single_calls_and_oracle_prefix():
    cfg = wl.CONFIGS[1]
    model = cfg["model"]()
    gm, om = _pair(model)
    xs = wl.images(4, seed=cfg["image_seed"])
    cls, rad, c0, c1 = gm.certify_batch(xs, 4, SEED, 10, 100, 700, 0.25, ALPHA)
    for i in range(4):
        s = gm.certify(xs[i], SEED, 10 + i, 100, 700, 0.25, ALPHA)
        assert (s[0], s[1]) == (cls[i], rad[i])
        np.testing.assert_array_equal(s[2], c0[i]); np.testing.assert_array_equal(s[3], c1[i])
        e = oracle.certify_decide(c0[i], c1[i], 700, 0.25, ALPHA)
        assert (e[0], e[1]) == (cls[i], rad[i])
    e = oracle.certify(om, xs[2], SEED, 12, 100, 700, 0.25, ALPHA)
    assert (e[0], e[1]) == (cls[2], rad[2])
    np.testing.assert_array_equal(e[2], c0[2]); np.testing.assert_array_equal(e[3], c1[2])
    # images resident on the device give the same answer
    import torch
    xd = torch.from_numpy(xs).cuda()
    d = gm.certify_batch(None, 4, SEED, 10, 100, 700, 0.25, ALPHA, device_ptr=xd.data_ptr(),
                         stream=torch.cuda.current_stream())
    np.testing.assert_array_equal(d[0], cls); np.testing.assert_array_equal(d[1], rad)
    np.testing.assert_array_equal(d[3], c1)


def test_sigma_to_zero_limit():
    model = wl.tiny_cnn()
    gm, om = _pair(model)
    x = wl.images(1, seed=2)[0]
    clean = int(np.argmax(oracle.forward(om, x)))
    cls, rad, c0, c1 = gm.certify(x, 1, 0, 50, 300, 1e-4, ALPHA)
    assert c1[clean] == 300 and cls == clean
    assert rad == oracle.certify_decide(c0, c1, 300, 1e-4, ALPHA)[1]


def _rand_conv(rng, in_tensor, cin, cout, k, stride, pad, relu, zp_in, zp_out, res_tensor=-1, zp_res=0):
    return dict(op=wl.OP_CONV2D, in_tensor=in_tensor, res_tensor=res_tensor, cin=cin, cout=cout, kh=k, kw=k,
                stride=stride, pad=pad, relu=relu, zp_in=zp_in, zp_out=zp_out, zp_res=zp_res,
                w=rng.integers(-127, 128, (cout, cin, k, k)).astype(np.int8),
                bias=rng.integers(-30000, 30001, cout).astype(np.int32),
                mult=rng.integers(2 ** 30, 2 ** 31, cout).astype(np.int32),
                shift=rng.integers(0, 14, cout).astype(np.int8),
                res_mult=int(rng.integers(2 ** 30, 2 ** 31)) if res_tensor >= 0 else 0,
                res_shift=int(rng.integers(-4, 5)) if res_tensor >= 0 else 0)


@pytest.mark.parametrize("seed", range(6))
def test_odd_shapes_zero_points_and_shifts(seed):
    """Ragged sizes, channel counts that are not multiples of 16, every zero-point and shift range."""
    rng = np.random.default_rng(100 + seed)
    h, w = int(rng.integers(5, 14)), int(rng.integers(5, 14)) // 4 * 4 + 4
    c1, c2 = int(rng.integers(3, 40)), int(rng.integers(3, 40))
    zp1, zp2 = int(rng.integers(-128, 100)), int(rng.integers(-128, 100))
    k0 = int(rng.choice([1, 3, 5]))
    L = [_rand_conv(rng, 0, 3, c1, k0, 1, k0 // 2, 1, int(rng.integers(0, 200)), zp1),
         _rand_conv(rng, 1, c1, c2, 3, 2, 1, int(rng.integers(0, 2)), zp1, zp2)]
    L.append(_rand_conv(rng, 2, c2, c2, 3, 1, 1, 1, zp2, zp1, res_tensor=2, zp_res=zp2))
    L.append(dict(wl._maxpool(3, c2, 3, 2, 1, zp1)))
    model = dict(in_shape=(3, h, w), n_classes=7, layers=L)
    om_tmp = oracle.Model(dict(model, n_classes=1))
    hw = oracle.tensor_size(om_tmp, 4) // c2
    L.append(wl._gavgpool(4, c2, hw, zp1))
    fc = _rand_conv(rng, 5, c2, 7, 1, 1, 0, 0, zp1, int(rng.integers(-20, 20)))
    fc["op"] = wl.OP_FC
    L.append(fc)
    gm, om = _pair(model)
    x = rng.integers(0, 256, (3, h, w)).astype(np.uint8)
    sizes = _tensor_sizes(om)
    a0 = oracle.noisy_input(x, 5, seed, 1, 2, 0.25)
    for k in range(1, om.n_layers + 1):
        _, exp = oracle.forward(om, a0, dump_tensor=k)
        got = gm.debug_tensor(x, 5, seed, 1, 2, 0.25, k, sizes[k])
        np.testing.assert_array_equal(got, exp, err_msg=f"tensor {k}")
    ec, el = oracle.sample_counts(om, x, 5, seed, 1, 0, 40, 0.25, want_logits=True)
    gc, gl = gm.sample_counts(x, 5, seed, 1, 0, 40, 0.25, want_logits=True)
    np.testing.assert_array_equal(gl, el)
    np.testing.assert_array_equal(gc, ec)


def test_argument_errors_leave_outputs_untouched():
    gm = isc.Model(wl.tiny_cnn())
    x = wl.images(1)[0]
    L = isc.lib()
    counts = np.full(10, -5, np.int32)
    for kw in (dict(sigma=0.0), dict(phase=256), dict(n=-1), dict(first=1 << 40)):
        rc = L.isc_sample_counts(gm._h, x.ctypes.data, 1, 0, kw.get("phase", 1), kw.get("first", 0),
                                 kw.get("n", 10), kw.get("sigma", 0.25), None, counts.ctypes.data, None)
        assert rc == -1 and (counts == -5).all()
    cls, rad = C.c_int32(9), C.c_double(9.0)
    assert L.isc_certify(gm._h, x.ctypes.data, 1, 0, 0, 10, 0.25, 0.001, None, C.byref(cls), C.byref(rad), None, None) == -1
    assert L.isc_certify(gm._h, x.ctypes.data, 1, 0, 10, 10, 0.25, 1.0, None, C.byref(cls), C.byref(rad), None, None) == -1
    assert L.isc_predict(gm._h, None, 1, 0, 10, 0.25, 0.001, None, C.byref(cls), None) == -1
    assert cls.value == 9 and rad.value == 9.0
    assert gm.get_info("gpu_launches") >= 0


def test_expired_wait_is_reported_and_the_handle_recovers():
    """Every device-side wait of the resident engine is bounded.  The harness runs the engine's own wait code on a
    barrier and a counter that nothing completes, with a 1 ms limit: the first wait must expire, raise the abort flag
    and the error word (ISC_ERR_TIMEOUT = -6 from the check), the second must fall through at once, and the handle must
    work afterwards.  Nothing here faults, traps or hangs the GPU."""
    model = wl.spread_model("resnet20")
    gm, om = _pair(model)
    x = wl.spread_image()
    before = gm.sample_counts(x, SEED, 0, 1, 0, 64, 0.25)
    rc, (first, second, abort_flag, ns) = gm.debug_wait_timeout(1_000_000)
    assert rc == -6
    assert (first, second, abort_flag) == (0, 0, 1)
    assert 1_000_000 <= ns < 200_000_000
    after, logits = gm.sample_counts(x, SEED, 0, 1, 0, 64, 0.25, want_logits=True)
    np.testing.assert_array_equal(after, before)
    np.testing.assert_array_equal(logits, oracle.sample_counts(om, x, SEED, 0, 1, 0, 64, 0.25, want_logits=True)[1])
    # out-of-range limits are refused before anything is launched
    assert gm.debug_wait_timeout(10)[0] == -1 and gm.debug_wait_timeout(10 ** 10)[0] == -1


def test_stalled_implicit_gemm_kernel_leaves_through_its_abort_path():
    """The layer-by-layer tensor-core engine: one launch of k_igemm whose weights are held back.  Every role's wait
    runs out after the kernel's own two-second limit (or sees the abort flag another role raised), in-flight copies
    are waited for, the tensor memory is freed, the error word is up (ISC_ERR_TIMEOUT = -6), and the same handle
    then computes the right logits.  Nothing here faults, traps or hangs the GPU."""
    model = wl.resnet50(hw=64, blocks=(1, 1, 1, 1))
    gm, om = _pair(model)
    gm.set_option("engine", 2)
    x = wl.images(1, shape=(3, 64, 64))[0]
    rc, (first, second, err_word, ns) = gm.debug_wait_timeout(1_000_000)
    assert rc == -6
    assert err_word >= 1
    assert 1_900_000_000 <= ns or ns == 0x7FFFFFFF
    got = gm.sample_counts(x, SEED, 3, 1, 0, 5, 0.5, want_logits=True)
    exp = oracle.sample_counts(om, x, SEED, 3, 1, 0, 5, 0.5, want_logits=True)
    assert gm.get_info("engine") == 2
    np.testing.assert_array_equal(got[1], exp[1])
    np.testing.assert_array_equal(got[0], exp[0])


def test_rounded_gaussian_noise_path():
    """The comparison method's noise (Sec. 4.1, FloatRS-quant: continuous Gaussian, then quantised) behind the same
    staging: with isc_set_option("noise", 1) every engine draws from the rounded-Gaussian table; noisy inputs, logits
    and counts equal the oracle's under the same law, and differ from the discrete-Gaussian ones."""
    model = wl.spread_model("resnet20")
    gm, om = _pair(model)
    x = wl.spread_image()
    base = gm.sample_counts(x, SEED, 0, 1, 0, 600, 0.5)
    gm.set_option("noise", 1)
    oracle.set_noise_kind(1)
    try:
        exp_in = oracle.noisy_input(x, SEED, 4, 1, 9, 0.5).ravel()
        ecounts, elog = oracle.sample_counts(om, x, SEED, 0, 1, 0, 600, 0.5, want_logits=True)
    finally:
        oracle.set_noise_kind(0)
    for eng in (1, 2, 3):
        gm.set_option("engine", eng)
        np.testing.assert_array_equal(gm.debug_tensor(x, SEED, 4, 1, 9, 0.5, 0, x.size), exp_in)
        counts, log = gm.sample_counts(x, SEED, 0, 1, 0, 600, 0.5, want_logits=True)
        np.testing.assert_array_equal(log, elog)
        np.testing.assert_array_equal(counts, ecounts)
    np.testing.assert_array_equal(gm.sample_counts_static(x, SEED, 0, 1, 0, 600, 0.5), ecounts)
    assert (ecounts != base).any()
    gm.set_option("noise", 0)
    gm.set_option("engine", 0)
    np.testing.assert_array_equal(gm.sample_counts(x, SEED, 0, 1, 0, 600, 0.5), base)
