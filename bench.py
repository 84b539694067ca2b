#!/usr/bin/env python
"""Benchmark of the per-replica CNN training step (Algorithm 1's inner loop) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl b2c|reference] [--workload NAME]

A step is one pass of the whole hot path over one batch: for each micro-batch forward, loss,
backward with gradients summed on the device, then one fused average + SGD-momentum update.
The default workload is the ResNet-18-shaped CIFAR net at batch 1024 run as 8 micro-batches of
128.  Prints one JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_23186_b200 import workloads as wl  # noqa: E402

WORKLOADS = {
    # name: (spec builder, micro_batch, n_micro)
    "resnet18_cifar_b1024_8x128": (wl.resnet18_spec, 128, 8),
    "resnet18_cifar_b128": (wl.resnet18_spec, 128, 1),
    "wrn28_10_cifar_b256": (wl.wrn28_10_spec, 256, 1),
    "resnet50_cifar_b1024_8x128": (wl.resnet50_spec, 128, 8),
}
DEFAULT_WORKLOAD = "resnet18_cifar_b1024_8x128"
LR, MU, WD = 0.1, 0.9, 5e-4
METRIC, UNIT = "train_images_per_sec", "images/s"
NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0
FALLBACK_BF16_TFLOPS, FALLBACK_HBM_GBS = 1590.0, 6650.0


# ------------------------------------------------------------------------------------------------
# algorithmic work of one micro-batch (what the method must do; padding and halos not counted)
# ------------------------------------------------------------------------------------------------
# DRAM traffic of conv_kmajor_kernel (dram__bytes_read.sum + dram__bytes_write.sum, mean over the kernel's launches in one
# step) from the ncu capture summarised in the named profile, with the SHA-1 of the kernel source at the time of the
# capture: once the source differs the figure is stale and the line reports null.
KMAJOR_DRAM_CAPTURE = {
    "resnet18_cifar_b1024_8x128": {"bytes_per_launch": 91.01e6, "profile": "profiles/conv_kmajor_resnet18_b1024.md",
                                   "kernel_sha1": "6d268bd63002e0b945f04c138b0934e59871ad06"},
}


def kmajor_traffic(name):
    """(bytes per launch | None, where the figure comes from)."""
    import hashlib
    cap = KMAJOR_DRAM_CAPTURE.get(name)
    if cap is None:
        return None, "no ncu capture for this workload"
    src = os.path.join(ROOT, "paper_2503_23186_b200", "csrc", "conv_kmajor.cu")
    with open(src, "rb") as f:
        sha = hashlib.sha1(f.read()).hexdigest()
    if sha != cap["kernel_sha1"]:
        return None, f"stale: conv_kmajor.cu changed since the capture in {cap['profile']}"
    return cap["bytes_per_launch"], f"ncu capture summarised in {cap['profile']} (kernel source unchanged since)"


def algorithmic_work(spec, n):
    """Returns dict family -> (flops, bytes) for one micro-batch of n images."""
    w = {k: [0.0, 0.0] for k in ("conv_fwd", "conv_dgrad", "conv_wgrad", "bn_fwd", "bn_bwd", "update")}
    params = 0
    for L in spec:
        if L["kind"] == "conv":
            P, Q = L["H"] // L["stride"], L["W"] // L["stride"]
            flops = 2.0 * n * P * Q * L["K"] * L["R"] * L["R"] * L["C"]
            x_b, y_b, w_b = 2.0 * n * L["H"] * L["W"] * L["C"], 2.0 * n * P * Q * L["K"], 2.0 * L["K"] * L["R"] ** 2 * L["C"]
            w["conv_fwd"][0] += flops; w["conv_fwd"][1] += x_b + y_b + w_b
            w["conv_wgrad"][0] += flops; w["conv_wgrad"][1] += x_b + y_b + 2 * w_b
            if L["src"] != 0:
                w["conv_dgrad"][0] += flops; w["conv_dgrad"][1] += x_b + y_b + w_b
            params += L["K"] * L["R"] ** 2 * L["C"]
        elif L["kind"] == "bn":
            e = 2.0 * n * L["H"] * L["W"] * L["C"]          # bytes of one bf16 tensor of this shape
            res = 1 if L["res"] >= 0 else 0
            w["bn_fwd"][1] += e * (2 + res)                  # read y (+residual), write a
            w["bn_bwd"][1] += e * (5 + 3 * res)              # two passes over da, y (a, da2), write dy (dres)
            params += 2 * L["C"]
        elif L["kind"] == "fc":
            params += L["K"] * L["C"] + L["K"]
    w["update"][1] = 28.0 * params                           # per step, not per micro-batch
    return {k: tuple(v) for k, v in w.items()}, params


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), bf16_burst=float(p["bf16_tflops"]),
                    hbm=float(p["hbm_gbs"]), source="measured")
    return dict(bf16_sustained=1400.0, bf16_burst=FALLBACK_BF16_TFLOPS, hbm=FALLBACK_HBM_GBS, source="fallback")


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc, self.lines, self.index = None, [], device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def mark(self):
        """Start of the window whose samples count (the sampler itself is started earlier: nvidia-smi is slow to start)."""
        self.t0 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, line in self.lines:
            if stamp < getattr(self, "t0", 0.0):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(spec, params, images, labels, n_micro=1):
    from oracle import net as onet
    vel = {k: np.zeros_like(v) for k, v in params.items()}
    t = time.perf_counter()
    onet.train_step(spec, params, vel, images, labels, n_micro, LR, MU, WD, rounding=True)
    return time.perf_counter() - t


def cpu_baseline(spec, micro_batch: int, n_micro: int, target_s: float = 12.0):
    """The oracle as it stands, timed on this host on a bounded sample of the workload: a short probe of 8 images sizes
    the sample so that the timed run is roughly `target_s` seconds of CPU work (part of a micro-batch, or a few whole
    micro-batches of the step)."""
    import oracle
    oracle.lib()
    params = wl.init_params(spec, 0)
    images, labels = wl.image_batch(0, 8, tag="cpu_probe")
    probe = oracle_sample_step(spec, params, images.astype(np.float64), labels)
    want = 8 * round(target_s / max(probe, 1e-3))
    if want <= micro_batch:
        groups, sample_images = 1, int(max(8, want))
    else:
        groups = int(min(n_micro, max(1, want // micro_batch)))
        sample_images = groups * micro_batch
    images, labels = wl.image_batch(0, sample_images, tag="cpu")
    dt = oracle_sample_step(spec, params, images.astype(np.float64), labels, groups)
    return {"value": sample_images / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"one optimiser step on {groups} micro-batch(es), {sample_images} images in all (fp64, all layers, forward+backward+update), {dt:.1f} s"}


def run_reference(args, spec, name):
    """--impl reference: the oracle is the reference arm (there is no reference code to install)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.lib()
    sample = 16
    params = wl.init_params(spec, 0)
    images, labels = wl.image_batch(0, sample, tag="cpu")
    images = images.astype(np.float64)
    for _ in range(args.warmup):
        oracle_sample_step(spec, params, images, labels)
    times = [oracle_sample_step(spec, params, images, labels) for _ in range(args.steps)]
    total = sum(times)
    value = sample * args.steps / total
    desc = f"each step = one optimiser step of the oracle on one micro-batch of {sample} images of the workload"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": name, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
def run_b2c(args, spec, name, micro_batch, n_micro):
    import torch
    import torch.distributed as dist
    from paper_2503_23186_b200 import binding, data_parallel

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    ctx = binding.Context(local)
    net = binding.Net(ctx, spec, micro_batch, n_concurrent=args.concurrent if n_micro % args.concurrent == 0 else 1)
    net.load_params(wl.init_params(spec, 0))
    batch = micro_batch * n_micro
    images, labels = wl.image_batch(rank, batch, tag=f"r{rank}")        # each replica gets its own shard
    h_img = torch.from_numpy(images).to(torch.bfloat16).pin_memory()
    h_lab = torch.from_numpy(labels).pin_memory()
    d_img, d_lab = h_img.cuda(), h_lab.cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2

    def step(img, lab):
        # one replica: the fused single-call step; several: backward, NCCL sum of the gradient arrays, same update everywhere
        data_parallel.dp_train_step(net, img, lab, n_micro, LR, MU, WD)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step(d_img, d_lab)
    ctx.check_device()

    def timed_region():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        host_s = 0.0
        for a, b in ev:
            flush.zero_()            # untimed: evicts the previous step's lines from L2
            a.record()
            t_h = time.perf_counter()
            step(d_img, d_lab)
            host_s += time.perf_counter() - t_h
            b.record()
        timed_region.host_ms = 1e3 * host_s / args.steps   # host time to enqueue one step (no synchronisation inside)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = sum(a.elapsed_time(b) for a, b in ev)
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    # the headline: K steps as a user runs them
    sampler.mark()
    total_ms = timed_region()
    host_enqueue_ms = timed_region.host_ms
    clocks = sampler.stop() if rank == 0 else None
    # the same K steps again with CUDA events around every launch site (two event records per launch cost about 7 % of
    # the step, so they stay out of the headline): per-kernel-family times for the roofline figures
    net.profile_enable(True)
    profiled_ms = timed_region()
    fam_ms, fam_launches = net.profile_read()
    net.profile_enable(False)
    ctx.check_device()
    loss = float(net.loss.item())
    value = world * batch * args.steps / (total_ms * 1e-3)

    # end to end through the public call: host buffers in, loss out, copies inside the timed region
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        d_img.copy_(h_img, non_blocking=True)
        d_lab.copy_(h_lab, non_blocking=True)
        step(d_img, d_lab)
        _ = net.loss.cpu()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e = {"value": world * batch * args.steps / e2e_s, "unit": UNIT,
           "h2d_bytes_per_step": h_img.numel() * 2 + h_lab.numel() * 4, "d2h_bytes_per_step": 4}

    if rank != 0:
        return
    peaks = measured_peaks()
    # Which measured GEMM rate is the denominator: the burst figure when the timed region is short and ran at the top SM
    # clock (nothing like the seconds-long, power-capped loop the sustained figure comes from), else the sustained one.
    at_top_clock = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    use_burst = at_top_clock and total_ms < 1000.0
    bf16_peak = peaks["bf16_burst"] if use_burst else peaks["bf16_sustained"]
    peak_kind = "burst" if use_burst else "sustained"
    work, n_params = algorithmic_work(spec, micro_batch)
    reps = n_micro * args.steps        # algorithmic work is counted per micro-batch
    kernels = {}
    for fam in ("conv_fwd", "conv_dgrad", "conv_wgrad"):
        ms = fam_ms[fam]
        tf = work[fam][0] * reps / (ms * 1e-3) / 1e12 if ms > 0 else None
        kernels[fam] = {"ms_per_step": ms / args.steps, "tflops": tf, "frac_of_measured_burst": tf / peaks["bf16_burst"] if tf else None,
                        "frac_of_measured_sustained": tf / peaks["bf16_sustained"] if tf else None,
                        "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS if tf else None}
    for fam in ("bn_fwd", "bn_bwd", "update"):
        ms = fam_ms[fam]
        r = args.steps if fam == "update" else reps
        gbs = work[fam][1] * r / (ms * 1e-3) / 1e9 if ms > 0 else None
        kernels[fam] = {"ms_per_step": ms / args.steps, "gbs": gbs, "frac_of_measured": gbs / peaks["hbm"] if gbs else None}
    kernels["other"] = {"ms_per_step": fam_ms["other"] / args.steps}
    conv_flops = sum(work[f][0] for f in ("conv_fwd", "conv_dgrad", "conv_wgrad")) * reps
    conv_ms = sum(fam_ms[f] for f in ("conv_fwd", "conv_dgrad", "conv_wgrad"))
    conv_tf = conv_flops / (conv_ms * 1e-3) / 1e12 if conv_ms > 0 else None
    # dominant kernel: the K-major implicit-GEMM kernel (forward + data-gradient launches)
    km_ms = fam_ms["conv_fwd"] + fam_ms["conv_dgrad"]
    km_flops = (work["conv_fwd"][0] + work["conv_dgrad"][0]) * reps
    km_tf = km_flops / (km_ms * 1e-3) / 1e12 if km_ms > 0 else None
    km_launches = fam_launches["conv_fwd"] + fam_launches["conv_dgrad"]
    km_bytes = (work["conv_fwd"][1] + work["conv_dgrad"][1]) * reps
    traffic, traffic_source = kmajor_traffic(name)
    roofline = {"kernel": "conv_kmajor_kernel (forward + data-gradient launches)", "bound": "tensor", "achieved": km_tf,
                "peak": bf16_peak, "unit": "TFLOP/s", "frac": km_tf / bf16_peak if km_tf else None,
                "peak_source": f"{peaks['source']} {peak_kind} bf16 GEMM rate (timed region {total_ms:.0f} ms at a median SM clock of "
                               f"{clocks.get('sm_mhz') if clocks else None} MHz)",
                "frac_of_measured_burst": km_tf / peaks["bf16_burst"] if km_tf else None,
                "frac_of_measured_sustained": km_tf / peaks["bf16_sustained"] if km_tf else None,
                "frac_of_nominal": km_tf / NOMINAL_BF16_TFLOPS if km_tf else None,
                "timing": "kernel-family times come from the second, profiled region, where the event records around every launch site "
                          "serialise the launches (no overlap of one kernel's set-up with the previous kernel's tail): slightly pessimistic",
                "traffic": traffic, "traffic_source": traffic_source,
                "traffic_unit": "bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, mean over the kernel's launches of one step)",
                "algorithmic_bytes_per_launch": km_bytes / km_launches if km_launches else None,
                "all_conv_tflops": conv_tf, "all_conv_frac_of_measured_burst": conv_tf / peaks["bf16_burst"] if conv_tf else None,
                "all_conv_frac_of_measured_sustained": conv_tf / peaks["bf16_sustained"] if conv_tf else None,
                "all_conv_frac_of_nominal": conv_tf / NOMINAL_BF16_TFLOPS if conv_tf else None,
                "target": "north star: all convolution kernels together at 0.50 of nominal dense bf16"}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": name, "global_batch": world * batch, "micro_batch": micro_batch, "n_micro": n_micro, "micro_batches_per_pass": net.n_concurrent, "params": n_params,
                   "l2": "per-step working set (~0.5 GB of activations) exceeds the 126 MB L2; a 256 MB buffer is rewritten between timed steps (untimed)",
                   "timing": "CUDA events per step on the launching stream, summed, max over ranks; kernel-family times from a second region of the same steps with events around every launch site (b2c_net_profile_enable)",
                   "profiled_ms_per_step": profiled_ms / args.steps, "host_enqueue_ms_per_step": host_enqueue_ms},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(sum(fam_launches.values())),
        "roofline": roofline, "kernels": kernels, "loss": loss,
        "cpu_baseline": cpu_baseline(spec, micro_batch, n_micro) if world == 1 and not args.no_cpu_baseline else None,
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b2c", choices=["b2c", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--concurrent", type=int, default=8, help="micro-batches run side by side per pass")
    args = ap.parse_args()
    builder, micro_batch, n_micro = WORKLOADS[args.workload]
    spec = builder()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: launch one rank per GPU and let rank 0 print the line
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
               "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args, spec, args.workload)
    else:
        run_b2c(args, spec, args.workload, micro_batch, n_micro)


if __name__ == "__main__":
    main()
