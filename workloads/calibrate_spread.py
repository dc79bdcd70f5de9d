#!/usr/bin/env python
"""Writes spread_bias.json: FC biases that balance the spread-vote heads on the spread image.

Calls the CPU oracle only (never the CUDA library): for each base network it averages the
global-average-pool output of a few noisy copies of the image and sets each class's bias to
minus that class's mean accumulator, so that all classes start level and the noise decides.
Run from the repository root:  python workloads/calibrate_spread.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import workloads as wl  # noqa: E402

SIGMA, N_CAL = 0.25, 16


def main():
    out = {}
    x = wl.spread_image()
    for name, (delta, shift) in wl.SPREAD_HEADS.items():
        base = wl.spread_base(name)
        om = oracle.Model(base)
        pool_tensor = om.n_layers - 1                     # output of the global average pool
        feats = []
        for j in range(N_CAL):
            a0 = oracle.noisy_input(x, wl.NOISE_SEED, 0, 3, j, SIGMA)
            feats.append(oracle.forward(om, a0, dump_tensor=pool_tensor)[1])
        mean = np.mean(np.asarray(feats, dtype=np.float64), axis=0)
        head = wl.with_spread_head(base, np.zeros(base["n_classes"], np.int32), delta=delta, shift=shift)
        fc = head["layers"][-1]
        w = fc["w"].reshape(fc["cout"], fc["cin"]).astype(np.float64)
        out[name] = [int(v) for v in np.rint(-(w @ (mean - fc["zp_in"])))]
        print(name, out[name])
    with open(os.path.join(ROOT, "workloads", "spread_bias.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    main()
