"""The spread-vote test models do what the GPU parity tests rely on (checked on the CPU oracle alone): the votes of
the balanced image fill several classes and the logits tie for the maximum, so that histogramming and the
lowest-index tie rule (Algorithm 1 step 2, Algorithm 2 step 2) decide results."""
import numpy as np

import oracle
import workloads as wl


def test_spread_models_fill_several_classes_and_tie():
    x = wl.spread_image()
    for name, n in (("tiny_cnn", 2000), ("resnet20", 600)):
        om = oracle.Model(wl.spread_model(name))
        counts, logits = oracle.sample_counts(om, x, wl.NOISE_SEED, 0, 1, 0, n, 0.25, want_logits=True)
        assert counts.sum() == n
        assert (counts >= 0.05 * n).sum() >= 3, counts
        top = logits.max(axis=1)
        tied = (logits == top[:, None]).sum(axis=1) > 1
        assert tied.any()
        # a tie is decisive: the lowest index among the maxima is the vote
        first_max = np.argmax(logits.astype(np.int32), axis=1)
        np.testing.assert_array_equal(np.bincount(first_max, minlength=om.n_classes), counts)
        assert abs(int(logits.max())) < 127 and int(logits.min()) > -128     # nothing saturates


def test_boosted_head_gives_a_majority_that_is_not_unanimous():
    x = wl.spread_image()
    om = oracle.Model(wl.spread_model("tiny_cnn", boost=160))
    cls, rad, c0, c1 = oracle.certify(om, x, wl.NOISE_SEED, 3, 100, 4000, 0.25, 0.001)
    r_max = oracle.certify_decide([4000], [4000], 4000, 0.25, 0.001)[1]
    assert cls == 0 and 0.0 < rad < r_max and c1[0] < 4000
    om = oracle.Model(wl.spread_model("tiny_cnn"))
    assert oracle.certify(om, x, wl.NOISE_SEED, 3, 100, 4000, 0.25, 0.001)[0] == -1
