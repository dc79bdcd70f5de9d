"""Small fixed case for profilers: `python -m paper_2108_09413_b200.profile_case [model] [n_samples] [engine]`.

Loads a seeded synthetic network (resnet110 by default), runs the Monte-Carlo loop of one image a few
times through isc_sample_counts and prints the vote counts.  Sized so that one kernel of the resident
engine lasts a few tens of milliseconds: short enough for a multi-pass ncu capture.
"""
import sys
import time

import numpy as np


def main():
    import workloads as wl
    import paper_2108_09413_b200 as isc
    name = sys.argv[1] if len(sys.argv) > 1 else "resnet110"
    n = int(sys.argv[2]) if len(sys.argv) > 2 else 148 * 8 * 4
    engine = int(sys.argv[3]) if len(sys.argv) > 3 else 0
    model = {"tiny": wl.tiny_cnn, "resnet20": wl.resnet20, "resnet110": wl.resnet110, "resnet50": wl.resnet50}[name]()
    x = wl.images(1, shape=model["in_shape"], seed=11)[0]
    gm = isc.Model(model)
    gm.set_option("engine", engine)
    for rep in range(3):
        t0 = time.perf_counter()
        counts = gm.sample_counts(x, wl.NOISE_SEED, 0, 1, 0, n, 0.25)
        dt = time.perf_counter() - t0
        print(f"rep {rep}: {n} samples in {dt * 1e3:.2f} ms -> {n / dt:.0f} samples/s, engine {gm.get_info('engine')}, "
              f"counts {counts.tolist()}")
    assert int(np.sum(counts)) == n


if __name__ == "__main__":
    main()
