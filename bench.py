#!/usr/bin/env python
"""Benchmark of the CERTIFY hot path (noise draw -> int8 network -> votes -> bound) on B200.

A step certifies `--images-per-step` synthetic images of the chosen workload (default: the
CIFAR-shaped int8 ResNet-110, N0 = 100, N = 100,000, sigma = 0.25, alpha = 0.001) through
`isc_certify_batch`.  `value` is noisy samples per second with the images already resident in
device memory; `e2e` is the same call given host buffers (host->device copy of the images and
device->host read of the vote counts inside the timed region).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

`--config 4` runs the throughput sweep (launch batch x sigma on the ResNet-110 model): one JSON
line per cell, then the summary line.  `--samples N` replaces the workload's N by a smaller
number (a short case for profilers; the line says so and is not a benchmark result).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

NOMINAL_INT8_TOPS = 4500.0      # dense int8 tensor-core figure for one B200 (context only)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(source="measured", hbm_gbs=p["hbm_gbs"], bf16=p["bf16_tflops"],
                    bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]))
    return dict(source="fallback", hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.samples, self._stop, self._t = index, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                     timeout=5).stdout.strip()
                if out:
                    self.samples.append([t.strip() for t in out.split(",")])
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        if not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        mhz = sorted(float(s[0]) for s in self.samples if s[0].replace(".", "").isdigit())
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return dict(sm_mhz=mhz[len(mhz) // 2] if mhz else None,
                    sm_max_mhz=float(self.samples[0][1]) if self.samples[0][1].replace(".", "").isdigit() else None,
                    reasons=reasons, samples=len(self.samples))


def workload(cfg_id, sigma=None):
    cfg = wl.CONFIGS[cfg_id]
    model = cfg["model"]()
    if sigma is None:
        sigma = 0.25 if 0.25 in cfg["sigmas"] else cfg["sigmas"][0]
    return cfg, model, sigma


def workload_name(cfg_id, model):
    return f"config {cfg_id}: {model['name']} CERTIFY"


def oracle_rate(model, cfg, sigma, n_samples, x):
    """Samples/s of the CPU oracle on n_samples of the estimation phase of one image."""
    import oracle
    om = oracle.Model(model)
    oracle.sample_counts(om, x, wl.NOISE_SEED, 0, 1, 0, max(1, oracle.num_threads()), sigma)   # warm caches
    t0 = time.perf_counter()
    oracle.sample_counts(om, x, wl.NOISE_SEED, 0, 1, 0, n_samples, sigma)
    dt = time.perf_counter() - t0
    return n_samples / dt, oracle.num_threads(), dt


def oracle_sample_size(model):
    macs = wl.macs_per_sample(model)
    # about 15 s at ~1.5 GMAC/s per core on 8 cores; at least a few samples per thread
    return int(max(16, min(4096, 1.8e11 / macs)))


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step = a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, model, sigma = workload(args.config, args.sigma)
    x = wl.images(1, shape=cfg["shape"], seed=cfg["image_seed"])[0]
    import oracle
    om = oracle.Model(model)
    per_step = max(oracle.num_threads(), oracle_sample_size(model) // 8)
    for _ in range(args.warmup):
        oracle.sample_counts(om, x, wl.NOISE_SEED, 0, 1, 0, oracle.num_threads(), sigma)
    t0 = time.perf_counter()
    for s in range(args.steps):
        oracle.sample_counts(om, x, wl.NOISE_SEED, 0, 1, s * per_step, per_step, sigma)
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    sample = f"{per_step} noisy samples of image 0 per step (estimation phase), {model['name']}"
    print(json.dumps({
        "impl": "reference", "metric": "noisy int8 samples/sec", "value": value, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload_name(args.config, model), "sigma": sigma,
                   "N0": cfg["N0"], "N": cfg["N"], "alpha": cfg["alpha"]},
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, choices=sorted(wl.CONFIGS))
    ap.add_argument("--images-per-step", type=int, default=0)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--engine", type=int, default=0, help="0 auto, 1 layer-by-layer, 3 resident tensor-core (line tiles)")
    ap.add_argument("--batch", type=int, default=0, help="noisy samples per launch (0: the library chooses)")
    ap.add_argument("--sigma", type=float, default=None, help="noise level (default: the workload's)")
    ap.add_argument("--samples", type=int, default=0, help="replace the workload's N (short case for profilers)")
    ap.add_argument("--spread", action="store_true",
                    help="the workload's network with the balanced final layer and its image (votes spread over the classes, "
                         "so the host bound runs its bisection instead of the closed form of unanimous votes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2108_09413_b200 as isc

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg, model, sigma = workload(args.config, args.sigma)
    if args.spread:
        model = wl.spread_model(model["name"])
    gm = isc.Model(model)
    gm.set_option("engine", args.engine)
    ctx = dict(torch=torch, dist=dist, rank=rank, local_rank=local_rank, world=world, gm=gm, cfg=cfg, model=model)

    if args.config == 4 and not args.samples:
        # the sweep: launch batch x sigma, 20 images per cell (2 steps of 10), device-resident images
        cells = []
        for batch in cfg["batches"]:
            for sg in cfg["sigmas"]:
                r = measure(ctx, args, sg, batch, steps=2, warmup=1, ips=10, e2e_arm=False)
                cell = {"cell": {"batch": batch, "sigma": sg}, "value": r["value"], "unit": r["unit"],
                        "certified_images_per_sec": r["certified_images_per_sec"], "ms_per_step": r["ms_per_step"],
                        "gpu_launches": r["gpu_launches"], "roofline_frac": r["roofline"]["frac"],
                        "frac_of_nominal_int8": r["roofline"]["frac_of_nominal_int8"],
                        "sampler_share": r.get("sampler_share"), "clocks": r["clocks"]}
                cells.append(cell)
                if rank == 0:
                    print(json.dumps(cell), flush=True)
        out = measure(ctx, args, sigma, args.batch, steps=args.steps, warmup=args.warmup, ips=args.images_per_step, e2e_arm=True)
        out["sweep"] = cells
    else:
        out = measure(ctx, args, sigma, args.batch, steps=args.steps, warmup=args.warmup, ips=args.images_per_step, e2e_arm=True)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_or = oracle_sample_size(model)
        probe = wl.images(1, shape=cfg["shape"], seed=cfg["image_seed"])
        rate, cores, dt = oracle_rate(model, cfg, sigma, n_or, probe[0])
        out["cpu_baseline"] = {"value": rate, "unit": "samples/s", "cores": cores, "kind": "oracle",
                               "sample": f"{n_or} noisy samples of one image (estimation phase), {dt:.1f} s"}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def measure(ctx, args, sigma, batch, steps, warmup, ips, e2e_arm):
    """One measurement: `steps` timed steps of `ips` certified images each, after `warmup` untimed ones."""
    torch, dist, rank, local_rank, world = ctx["torch"], ctx["dist"], ctx["rank"], ctx["local_rank"], ctx["world"]
    gm, cfg, model = ctx["gm"], ctx["cfg"], ctx["model"]
    gm.set_option("batch", batch)
    N0, alpha = cfg["N0"], cfg["alpha"]
    N = args.samples if args.samples else cfg["N"]
    macs = wl.macs_per_sample(model)

    # images per step: sized so that one step is about a second of GPU time
    total_steps = warmup + 2 * steps
    # every rank certifies its own images (weak scaling, no exchange)
    probe = wl.images(1, shape=cfg["shape"], seed=cfg["image_seed"])
    stream = torch.cuda.current_stream()
    if ips <= 0:
        xd = torch.from_numpy(probe).cuda()
        gm.certify_batch(None, 1, wl.NOISE_SEED, 0, N0, max(1, N // 50), sigma, alpha, stream, xd.data_ptr())
        t0 = time.perf_counter()
        gm.certify_batch(None, 1, wl.NOISE_SEED, 0, N0, max(1, N // 10), sigma, alpha, stream, xd.data_ptr())
        per_image = (time.perf_counter() - t0) * (N0 + N) / (N0 + max(1, N // 10))
        ips = int(max(1, min(cfg["n_images"], round(1.0 / max(per_image, 1e-4)))))
        if dist is not None:
            t = torch.tensor([ips], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MIN)
            ips = int(t.item())
    imgs = wl.images(ips * total_steps, shape=cfg["shape"], seed=cfg["image_seed"] + 7919 * rank)
    imgs = imgs.reshape(total_steps, ips, *cfg["shape"])
    if args.spread:                      # the image the head was balanced on, under a different image id each time
        imgs = np.broadcast_to(wl.spread_image(cfg["shape"]), imgs.shape).copy()
    dev_imgs = torch.from_numpy(imgs).cuda()
    pinned = torch.from_numpy(imgs).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2

    def step(i, host):
        id0 = (rank * total_steps + i) * ips
        if host:
            return gm.certify_batch(pinned[i].numpy(), ips, wl.NOISE_SEED, id0, N0, N, sigma, alpha, stream)
        return gm.certify_batch(None, ips, wl.NOISE_SEED, id0, N0, N, sigma, alpha, stream,
                                device_ptr=dev_imgs[i].data_ptr())

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(first, count, host):
        """Device time of `count` steps (events on the launching stream), L2 flushed between steps."""
        total_ms = 0.0
        for i in range(first, first + count):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            last_result[0] = step(i, host)
            e1.record(stream)
            e1.synchronize()
            total_ms += e0.elapsed_time(e1)
        return total_ms

    last_result = [None]

    def decide_ms():
        """Host time of the bound and radius (Algorithm 1 steps 5-7) per image, on the counts of the last step."""
        import paper_2108_09413_b200 as isc
        _, _, c0, c1 = last_result[0]
        t0 = time.perf_counter()
        for i in range(len(c0)):
            isc.certify_decide(c0[i], c1[i], N, sigma, alpha)
        return 1e3 * (time.perf_counter() - t0) / max(1, len(c0))

    def phase_cycles():
        try:
            return [gm.get_info(k) for k in ("cycles_fill", "cycles_noise", "cycles_conv", "cycles_tail")]
        except Exception:
            return None

    for i in range(warmup):
        step(i, False)
    launches0 = gm.get_info("gpu_launches")
    cyc0 = phase_cycles()
    barrier()
    with ClockSampler(local_rank) as clk:
        ms = timed(warmup, steps, False)
        barrier()
    launches = gm.get_info("gpu_launches") - launches0
    cyc1 = phase_cycles()
    barrier()
    ms_e2e = timed(warmup + steps, steps, True) if e2e_arm else ms
    barrier()
    if dist is not None:
        t = torch.tensor([ms, ms_e2e], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, ms_e2e = t.tolist()

    samples_per_step = ips * (N0 + N)
    total_samples = samples_per_step * steps * world
    value = total_samples / (ms * 1e-3)
    e2e = total_samples / (ms_e2e * 1e-3)
    peaks = load_peaks()
    int8_peak = 2.0 * peaks["bf16_sustained"]              # nominal int8 : bf16 ratio of the tensor cores is 2
    achieved = 2.0 * macs * samples_per_step * steps / (ms * 1e-3) / 1e12   # per GPU
    engine = gm.get_info("engine")
    name = workload_name(args.config, model)
    if args.spread:
        name += " (spread-vote head)"
    if args.samples:
        name += f" (short case: N = {N} instead of {cfg['N']}; not a benchmark result)"

    out = {
        "metric": "noisy int8 samples/sec", "value": value, "unit": "samples/s", "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic",
        "config": {"workload": name,
                   "sigma": sigma, "N0": N0, "N": N, "alpha": alpha, "images_per_step": ips, "batch": batch,
                   "engine": {1: "layer-by-layer", 3: "resident tensor-core, line tiles"}.get(engine, str(engine)),
                   "l2": "flushed between steps (256 MiB write)", "macs_per_sample": macs},
        "certified_images_per_sec": value / (N0 + N),
        "decide_ms_per_image": decide_ms(),
        "e2e": {"value": e2e, "unit": "samples/s", "h2d_bytes_per_step": int(ips * np.prod(cfg["shape"])),
                "d2h_bytes_per_step": int(ips * 2 * model["n_classes"] * 4)},
        "gpu_launches": int(launches),
        "clocks": clk.summary(),
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TFLOP/s",
                     "frac": achieved / int8_peak, "frac_of_nominal_int8": achieved / NOMINAL_INT8_TOPS, "traffic": None,
                     "peak_source": f"2 x {peaks['source']} sustained bf16 ({peaks['bf16_sustained']} TFLOP/s); "
                                    f"nominal dense int8 {NOMINAL_INT8_TOPS} TOP/s -> frac {achieved / NOMINAL_INT8_TOPS:.4f}",
                     "ops": "algorithmic: 2 x true MACs per noisy sample"},
    }
    if not e2e_arm:
        del out["e2e"]
    if cyc0 is not None and cyc1 is not None:
        d = [b - a for a, b in zip(cyc0, cyc1)]
        if sum(d) > 0:
            out["sampler_share"] = d[1] / sum(d)
            out["phase_shares"] = {"fill": d[0] / sum(d), "noise": d[1] / sum(d), "conv": d[2] / sum(d), "tail": d[3] / sum(d)}
    return out


if __name__ == "__main__":
    main()
