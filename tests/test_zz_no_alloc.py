"""The allocation-free entry point (isc_sample_counts_static), collected last on purpose.

Callers that may not call cudaMalloc while running (pre-partitioned device memory, latency
budgets that rule out the synchronisation an allocation implies) use this variant; it must
return exactly what isc_sample_counts returns, call after call, although every call reuses
the same fixed device array and finds the previous call's data in it.
"""
import ctypes as C

import numpy as np
import pytest

import workloads as wl
import paper_2108_09413_b200 as isc

pytestmark = pytest.mark.gpu


def test_static_workspace_matches_allocating_entry_point_twice_in_a_row():
    # models whose votes spread over many classes: a miscounted or misplaced vote changes the histogram
    x = np.stack([wl.spread_image(), wl.images(1, seed=31)[0]])
    for model, n in ((wl.spread_model("tiny_cnn"), 700), (wl.spread_model("resnet20"), 2300)):
        gm = isc.Model(model)
        # two calls in a row with different arguments: the second one starts from the first one's leftovers
        for call, (img, phase, first, sigma) in enumerate(((0, 1, 0, 0.25), (1, 0, 17, 0.5), (0, 1, 0, 0.25))):
            expected = gm.sample_counts(x[img], wl.NOISE_SEED, 0, phase, first, n, sigma)
            got = gm.sample_counts_static(x[img], wl.NOISE_SEED, 0, phase, first, n, sigma)
            assert got.sum() == n
            np.testing.assert_array_equal(got, expected, err_msg=f"{model['name']} call {call}")
            assert gm.get_info("engine") == 1
            if img == 0:
                assert (got > 0).sum() >= 3
        gm.close()


def test_static_entry_point_leaves_free_device_memory_unchanged():
    """What the entry point is for: after the first call on the device (which looks up the array's address) further
    calls take no device memory, whatever their size."""
    import torch
    gm = isc.Model(wl.spread_model("resnet20"))
    x = wl.spread_image()
    gm.sample_counts_static(x, wl.NOISE_SEED, 0, 1, 0, 8, 0.25)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for n, sigma in ((5000, 0.25), (64, 1.0), (12000, 0.12)):
        assert gm.sample_counts_static(x, wl.NOISE_SEED, 0, 1, 0, n, sigma).sum() == n
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_workspace_rejects_what_does_not_fit():
    gm = isc.Model(wl.tiny_cnn())
    x = wl.images(1)[0]
    counts = np.full(10, -3, np.int32)
    L = isc.lib()
    # sigma = 10 needs a 35,702-entry noise table, beyond the 16,384 entries reserved for it
    rc = L.isc_sample_counts_static(gm._h, x.ctypes.data, 1, 0, 1, 0, 10, 10.0, None, counts.ctypes.data)
    assert rc == -3 and (counts == -3).all()
    rc = L.isc_sample_counts_static(gm._h, x.ctypes.data, 1, 0, 1, 0, -1, 0.25, None, counts.ctypes.data)
    assert rc == -1 and (counts == -3).all()
    np.testing.assert_array_equal(gm.sample_counts_static(x, 1, 0, 1, 0, 0, 0.25), np.zeros(10, np.int32))
    big = isc.Model(wl.resnet50())                 # one 224x224 sample needs several MiB: still fits
    xb = wl.images(1, shape=(3, 224, 224), seed=9)[0]
    np.testing.assert_array_equal(big.sample_counts_static(xb, 1, 0, 1, 0, 3, 0.5),
                                  big.sample_counts(xb, 1, 0, 1, 0, 3, 0.5))
