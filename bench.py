#!/usr/bin/env python
"""Throughput of the PSB sampled-weight contraction on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload conv3x3|fc|resnet50|resnet50_adaptive|mobilenetv2]
                    [--k 8] [--impl reference]

One step = one pass of the whole hot path over one synthetic batch: draw fresh random bits
and build the integer filters (sampler), run the contraction, apply the fused output stage.
Prints ONE JSON line.  `value` is logical multiply-accumulates per second (one per
activation/weight pair, independent of k) with inputs resident in HBM; `e2e` is the same
through the public API from pinned host buffers, copies included.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "effective int MAC/s"
UNIT = "GMAC/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# --------------------------------------------------------------------------- workloads

class ConvWorkload:
    """3x3 stride-1 conv, 64 -> 64 channels on 56x56, batch 32, NCHW u8 activations in [0, 15]
    (half zeros), He-normal fp32 filter; k draws, 4-bit re-quantised output."""
    name = "conv3x3_c64_56x56_b32_nchw"
    oracle_images = 16

    def __init__(self, k, rank=0):
        from workloads import config2_conv

        self.k = k
        self.log2k = int(np.log2(k))
        self.cfg = config2_conv(seed=1 + 100 * rank)
        self.macs = self.cfg["macs"]
        self.images = self.cfg["x"].shape[0]
        self.planes = None

    def setup(self, ctx, psb, torch):
        self.ctx, self.psb, self.torch = ctx, psb, torch
        c, dev = self.cfg, ctx.device
        self.w = torch.from_numpy(c["w"]).to(dev)
        self.x = torch.from_numpy(c["x"]).to(dev)
        self.x_nhwc = self.x.permute(0, 2, 3, 1).contiguous()
        self.scale = torch.from_numpy(c["scale"]).to(dev)
        self.bias = torch.from_numpy(c["bias"]).to(dev)
        self.wt = ctx.sample_weights(self.w, seed=c["seed"], layer_id=0, level_mask=1 << self.log2k)
        ctx.set_sample_map(None, self.log2k)
        self.out = {"q": torch.empty((32, 64, 56, 56), dtype=torch.uint8, device=dev)}
        self.out_nhwc = {"q": torch.empty((32, 56, 56, 64), dtype=torch.uint8, device=dev)}
        # pinned host buffers for the end-to-end measurement
        self.x_host = torch.from_numpy(c["x"]).pin_memory()
        self.q_host = torch.empty((32, 64, 56, 56), dtype=torch.uint8).pin_memory()
        self.x_stage = torch.empty_like(self.x)
        span = 15 + self.log2k + 2
        self.planes = (span + 6) // 7

    def step(self, i):
        c, psb = self.cfg, self.psb
        self.ctx.sample_weights(self.w, seed=c["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt)
        self.ctx.conv2d(self.wt, self.x, psb.PSB_LAYOUT_NCHW, 1, 1, self.scale, self.bias, True,
                        c["inv_step"], 0, 15, in_max=15, out=self.out)

    def kernel_only(self):
        """The dominant kernel alone: contraction + output stage on channels-last input."""
        c, psb = self.cfg, self.psb
        self.ctx.conv2d(self.wt, self.x_nhwc, psb.PSB_LAYOUT_NHWC, 1, 1, self.scale, self.bias, True,
                        c["inv_step"], 0, 15, in_max=15, out=self.out_nhwc)

    def e2e_step(self, i):
        self.x_stage.copy_(self.x_host, non_blocking=True)
        c, psb = self.cfg, self.psb
        self.ctx.sample_weights(self.w, seed=c["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt)
        self.ctx.conv2d(self.wt, self.x_stage, psb.PSB_LAYOUT_NCHW, 1, 1, self.scale, self.bias, True,
                        c["inv_step"], 0, 15, in_max=15, out=self.out)
        self.q_host.copy_(self.out["q"], non_blocking=True)

    e2e_h2d = 32 * 64 * 56 * 56
    e2e_d2h = 32 * 64 * 56 * 56

    def roofline(self, kernel_ms, peaks):
        # algorithmic work of the contraction kernel: one int8 MAC per (activation, digit) pair,
        # P digit planes per weight, 2 operations per MAC; int8 dense peak = 2 x the measured bf16 peak
        ops = 2.0 * self.macs * self.planes
        achieved = ops / (kernel_ms * 1e-3) / 1e12
        peak = 2.0 * peaks["bf16_tflops"]
        # DRAM bytes of one launch from the ncu capture summarised in profiles/psb_mma_kernel_conv3x3_b32.md
        # (dram__bytes_read.sum + dram__bytes_write.sum; k does not change them); to be set back to None
        # whenever the kernel changes before the counters are taken again
        return dict(bound="tensor", kernel="psb_mma_kernel", achieved=achieved, peak=peak, unit="TOP/s (int8)",
                    frac=achieved / peak, traffic=6.63e6, traffic_unit="bytes per launch (ncu)",
                    peak_source=peaks["source"] + " bf16 burst x 2",
                    planes=self.planes, logical_gmacs=self.macs / (kernel_ms * 1e-3) / 1e9,
                    kernel_ms=kernel_ms)

    def oracle_sample(self, n_images=4):
        """Time the CPU oracle on the first n_images of the batch; returns (seconds, macs)."""
        from oracle import psb_oracle as orc

        c = self.cfg
        x = np.ascontiguousarray(c["x"][:n_images])
        t0 = time.perf_counter()
        W, eb, _ = orc.sample_level(c["w"], c["seed"], 0, self.log2k)
        g = orc.geom(x.shape, orc.NCHW, orc.U8, c["w"].shape, 1, 1, 1)
        acc = orc.conv_acc(x, g, {self.log2k: W}, uniform_log2k=self.log2k)
        orc.epilogue(acc, g, c["scale"], c["bias"], eb, True, c["inv_step"], 0, 15, uniform_log2k=self.log2k)
        dt = time.perf_counter() - t0
        return dt, self.macs * n_images // self.images, "first %d of %d images, all layers" % (n_images, self.images)


class FcWorkload:
    """Fully connected layer 256 -> 128, batch 16, k = 4, 8-bit output after ReLU: the small case.  Half a
    million multiply-accumulates per step, so a step is launch latency; what to read is microseconds."""
    name = "fc_256x128_b16"
    oracle_images = 16

    def __init__(self, k, rank=0):
        from workloads import config1_fc

        self.k = k
        self.log2k = int(np.log2(k))
        self.cfg = config1_fc(seed=100 * rank, k=k)
        self.macs = self.cfg["macs"]
        self.images = self.cfg["x"].shape[0]

    def setup(self, ctx, psb, torch):
        self.ctx, self.psb, self.torch = ctx, psb, torch
        c, dev = self.cfg, ctx.device
        self.w = torch.from_numpy(c["w"]).to(dev)
        self.x = torch.from_numpy(c["x"]).to(dev)
        self.scale = torch.from_numpy(c["scale"]).to(dev)
        self.bias = torch.from_numpy(c["bias"]).to(dev)
        self.wt = ctx.sample_weights(self.w, seed=c["seed"], layer_id=0, level_mask=1 << self.log2k)
        ctx.set_sample_map(None, self.log2k)
        self.out = {"q": torch.empty((self.images, c["w"].shape[0]), dtype=torch.uint8, device=dev)}
        self.x_host = torch.from_numpy(c["x"]).pin_memory()
        self.q_host = torch.empty((self.images, c["w"].shape[0]), dtype=torch.uint8).pin_memory()
        self.x_stage = torch.empty_like(self.x)
        self.e2e_h2d = self.x_host.numel()
        self.e2e_d2h = self.q_host.numel()

    def _gemm(self, x):
        c = self.cfg
        self.ctx.gemm(self.wt, x, self.scale, self.bias, True, c["inv_step"], 0, 255, in_max=15, out=self.out)

    def step(self, i):
        self.ctx.sample_weights(self.w, seed=self.cfg["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt)
        self._gemm(self.x)

    def kernel_only(self):
        self._gemm(self.x)

    def e2e_step(self, i):
        self.x_stage.copy_(self.x_host, non_blocking=True)
        self.ctx.sample_weights(self.w, seed=self.cfg["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt)
        self._gemm(self.x_stage)
        self.q_host.copy_(self.out["q"], non_blocking=True)

    def roofline(self, kernel_ms, peaks):
        # one launch of 2048 threads: neither bytes (35 KB) nor arithmetic matter, the launch does
        nbytes = self.images * 256 + 128 * 256 * 4 + self.images * 128
        achieved = nbytes / (kernel_ms * 1e-3) / 1e9
        return dict(bound="hbm", kernel="conv_direct_kernel (latency-bound: one launch of 2048 threads)",
                    achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                    traffic=None, peak_source=peaks["source"], kernel_ms=kernel_ms)

    def oracle_sample(self, n_images=16):
        from oracle import psb_oracle as orc

        c = self.cfg
        x = c["x"].reshape(self.images, 1, 1, 256)
        t0 = time.perf_counter()
        W, eb, _ = orc.sample_level(c["w"], c["seed"], 0, self.log2k)
        g = orc.geom(x.shape, orc.NHWC, orc.U8, c["w"].shape, 1, 1, 0)
        acc = orc.conv_acc(x, g, {self.log2k: W}, uniform_log2k=self.log2k)
        orc.epilogue(acc, g, c["scale"], c["bias"], eb, True, c["inv_step"], 0, 255, uniform_log2k=self.log2k)
        dt = time.perf_counter() - t0
        return dt, self.macs, "the whole batch of %d, sampling included" % self.images


class NetWorkload:
    """Network-shaped workloads: every conv / FC layer is a PSB layer, activations stay in HBM."""
    oracle_images = 1

    def __init__(self, kind, k, rank=0, batch=0):
        from workloads import mobilenetv2_layers, network_macs, resnet50_layers

        self.kind, self.k, self.rank = kind, k, rank
        self.log2k = int(np.log2(k))
        if kind == "mobilenetv2":
            self.layers, self.batch, self.qu, self.qs, self.prune, self.seed = mobilenetv2_layers(), batch or 64, 255, 127, 0.5, 3
        else:
            self.layers, self.qu, self.qs, self.prune = resnet50_layers(), 15, 15, 0.0
            self.batch, self.seed = (batch or 128, 4) if kind == "resnet50_adaptive" else (batch or 64, 2)
        self.adaptive = kind == "resnet50_adaptive"
        self.images = self.batch
        self.macs_per_image = network_macs(self.layers)
        self.macs = self.macs_per_image * self.batch
        self.name = "%s_b%d" % (kind, self.batch)
        self.mean_k = 4.0 if self.adaptive else float(k)

    def setup(self, ctx, psb, torch):
        from paper_1904_02205_b200.network import Network
        from workloads import build_network, saliency_kmaps

        self.ctx, self.psb, self.torch = ctx, psb, torch
        self.net = build_network(self.layers, 224, self.batch, self.seed + 100 * self.rank, self.qu, self.qs,
                                 prune_frac=self.prune)
        self.kmaps = saliency_kmaps(self.batch, [112, 56, 28, 14, 7], self.seed) if self.adaptive else None
        mask = 0b11111 if self.adaptive else 1 << self.log2k
        self.nw = Network(ctx, self.layers, self.net, self.batch, mask, kmaps=self.kmaps, uniform_log2k=self.log2k,
                          fc_log2k=4 if self.adaptive else None)
        self.nw.sample(self.seed)
        self.image_host = torch.from_numpy(self.net["image"]).pin_memory()
        self.image_dev = self.image_host.to(ctx.device)
        self.logits_host = torch.empty((self.batch, self.layers[-1]["cout"]), dtype=torch.float32).pin_memory()
        self.nw.forward(self.image_dev)
        self.e2e_h2d = self.image_host.numel()
        self.e2e_d2h = self.logits_host.numel() * 4
        self.layer_ms = None

    def step(self, i):
        self.nw.sample(self.seed + i)
        self.nw.forward()

    def kernel_only(self):
        """One forward pass with fixed filters and a pair of events around every layer."""
        ev = {}
        self.nw.forward(layer_events=ev)
        self.torch.cuda.synchronize()
        ms = {k: a.elapsed_time(b) for k, (a, b) in ev.items()}
        if self.layer_ms is None:
            self.layer_ms = {k: [] for k in ms}
        for k, v in ms.items():
            self.layer_ms[k].append(v)

    def e2e_step(self, i):
        self.nw.acts["image"].copy_(self.image_host, non_blocking=True)
        self.nw.sample(self.seed + i)
        self.nw.forward()
        self.logits_host.copy_(self.nw.logits, non_blocking=True)

    def roofline(self, _kernel_ms, peaks):
        """All launches of the tensor-core contraction in one forward pass, from per-layer events."""
        psb = self.psb
        span_bits = 15 + (4 if self.adaptive else self.log2k) + 2
        planes = (span_bits + 6) // 7
        t_ops, t_ms, s_ms, rows = 0.0, 0.0, 0.0, []
        for l in self.layers:
            ms = statistics.mean(self.layer_ms[l["name"]][1:] or self.layer_ms[l["name"]])
            if l["op"] != "conv":
                s_ms += ms
                continue
            macs = l["hout"] ** 2 * l["cout"] * (l["cin"] // l["groups"]) * l["k"] ** 2 * self.batch
            path = self.nw.paths[l["name"]]
            if path == psb.PSB_PATH_TENSOR:
                t_ops += 2.0 * macs * planes
                t_ms += ms
            else:
                s_ms += ms
            rows.append((l["name"], "tensor" if path == psb.PSB_PATH_TENSOR else "cuda-core", macs, ms))
        self.layer_rows = rows
        per_layer_ms = t_ms
        hook = getattr(self, "hook_ms", None)
        if hook:
            t_ms = statistics.mean(hook[1:] or hook)      # library events, one op-list forward pass
        achieved = t_ops / (t_ms * 1e-3) / 1e12 if t_ms else 0.0
        peak = 2.0 * peaks["bf16_tflops_sustained"]
        return dict(bound="tensor", kernel="psb_mma_kernel (all launches of one forward pass)", achieved=achieved,
                    peak=peak, unit="TOP/s (int8)", frac=achieved / peak, traffic=None,
                    peak_source=peaks["source"] + " bf16 sustained x 2", planes=planes, tensor_path_ms=t_ms,
                    tensor_path_ms_per_layer_events=per_layer_ms, other_layers_ms=s_ms)

    def oracle_sample(self, n_images=1):
        from oracle import psb_oracle as orc

        if not hasattr(self, "net"):
            from workloads import build_network, saliency_kmaps

            self.net = build_network(self.layers, 224, max(n_images, 2), self.seed, self.qu, self.qs, prune_frac=self.prune)
            self.kmaps = saliency_kmaps(max(n_images, 2), [112, 56, 28, 14, 7], self.seed) if self.adaptive else None
        t0 = time.perf_counter()
        orc.run_network(self.layers, self.net, self.net["image"][:n_images], self.seed, uniform_log2k=self.log2k,
                        fc_log2k=4 if self.adaptive else None,
                        kmaps=None if self.kmaps is None else {r: m[:n_images] for r, m in self.kmaps.items()})
        dt = time.perf_counter() - t0
        return dt, self.macs_per_image * n_images, "first %d of %d images, all layers, filters sampled once" % (n_images, self.batch)


def make_workload(args, rank):
    if args.workload == "conv3x3":
        return ConvWorkload(args.k, rank)
    if args.workload == "fc":
        return FcWorkload(args.k, rank)
    return NetWorkload(args.workload, args.k, rank, batch=args.batch)


# --------------------------------------------------------------------------- timing helpers

def aggregate_over_ranks(local_seconds, local_units, dist=None):
    """Whole-job throughput: units of all ranks divided by the slowest rank's time."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_seconds, local_units
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_seconds], dtype=torch.float64, device=dev)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = make_workload(args, 0)
    n_img = getattr(wl, "oracle_images", 1)
    times, macs, sample = [], 0, ""
    for i in range(args.warmup + args.steps):
        dt, macs, sample = wl.oracle_sample(n_img)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    val = macs / sec / 1e9
    line = dict(impl="reference", metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=sec * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="int64", data="synthetic",
                config=dict(workload=wl.name, k=args.k, sample=sample),
                cpu_baseline=dict(value=val, unit=UNIT, cores=1, kind="oracle", sample=sample),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))
    return 0


def run_int8_probe(ctx, index):
    """Ceiling of the dense path: back-to-back int8 MMAs from resident shared-memory tiles on every SM."""
    clocks = ClockSampler(index)
    clocks.start()
    rows = []
    for n_cols in (64, 128, 192, 256):
        for _ in range(3):
            mac_clk, tops = ctx.int8_mma_probe(n_cols, 20000)
        rows.append(dict(n_cols=n_cols, mac_per_clk_per_sm=mac_clk, tera_ops_per_s=tops))
    ctx.check_device()
    peaks = measured_peaks()
    print(json.dumps(dict(probe="tcgen05.mma.cta_group::1.kind::i8, M=128, K=32, operands resident in shared memory",
                          rows=rows, clocks=clocks.stop(),
                          bf16_x2_burst=2.0 * peaks["bf16_tflops"], bf16_x2_sustained=2.0 * peaks["bf16_tflops_sustained"],
                          peak_source=peaks["source"])))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="psb")
    ap.add_argument("--workload", default="conv3x3", choices=["conv3x3", "fc", "resnet50", "mobilenetv2", "resnet50_adaptive"])
    ap.add_argument("--k", type=int, default=8)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layer-table", default="", help="write per-layer times of the network workloads to this CSV")
    ap.add_argument("--probe-int8", action="store_true",
                    help="measure the bare tcgen05 int8 MMA issue rate instead of a workload and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    import paper_1904_02205_b200 as psb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    ctx = psb.Context(local_rank)
    if args.probe_int8:
        return run_int8_probe(ctx, local_rank)
    wl = make_workload(args, rank)
    wl.setup(ctx, psb, torch)
    # > L2 (126 MB); writing it also takes long enough (about 0.2 ms) for the host to have queued the whole
    # step behind it, so that the events see device time and not the host's launch rate
    flush = torch.empty(1 << 30, dtype=torch.uint8, device=ctx.device)

    def timed(fn, n, first=0):
        ms = []
        for i in range(n):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(first + i)
            e1.record()
            e1.synchronize()
            ms.append(e0.elapsed_time(e1))
        return ms

    for i in range(args.warmup):
        wl.step(i)
    ctx.check_device()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = ClockSampler(local_rank)
    clocks.start()
    launches0 = ctx.launch_count()
    step_ms = timed(wl.step, args.steps, first=args.warmup)
    torch.cuda.synchronize()
    launches = ctx.launch_count() - launches0      # kernels of the library inside the timed steps
    if world > 1:
        dist.barrier()
    kern_ms = timed(lambda i: wl.kernel_only(), max(args.steps, 10) if args.workload in ("conv3x3", "fc") else 4)
    in_step_ms = []
    if args.workload == "conv3x3":
        # the same steps once more with the library's own pair of events around the contraction kernel:
        # its duration inside the step (filters and converted input just written, output planar)
        for i in range(max(args.steps, 10)):
            flush.zero_()
            ctx.contraction_timing(True)          # a new sum for every step
            wl.step(args.warmup + args.steps + i)
            in_step_ms.append(ctx.contraction_time())
        ctx.contraction_timing(False)
    elif args.workload != "fc":
        # one forward pass issued as one op list with the library's events around every contraction launch:
        # the device time of the tensor path, independent of the host's per-layer call rate
        wl.hook_ms = []
        for i in range(3):
            flush.zero_()
            ctx.contraction_timing(True)
            wl.nw.forward()
            wl.hook_ms.append(ctx.contraction_time())
        ctx.contraction_timing(False)
    clk = clocks.stop()
    ctx.check_device()
    e2e_warm = timed(wl.e2e_step, 3)
    e2e_ms = timed(wl.e2e_step, args.steps, first=3)
    ctx.check_device()

    local_sec = sum(step_ms) * 1e-3
    sec, units = aggregate_over_ranks(local_sec, wl.macs * args.steps, dist if world > 1 else None)
    e2e_sec, e2e_units = aggregate_over_ranks(sum(e2e_ms) * 1e-3, wl.macs * args.steps, dist if world > 1 else None)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0
    peaks = measured_peaks()
    value = units / sec / 1e9
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=sec * 1e3 / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="int8 digits, int64 accumulators", data="synthetic",
                config=dict(workload=wl.name, k=args.k, l2="flushed between steps (1 GiB memset, untimed)",
                            images_per_step=wl.images * world, sampler="inside the timed step, fresh seed per step"),
                images_per_s=wl.images * world * args.steps / sec,
                gated_add_equiv_per_s=units * getattr(wl, "mean_k", args.k) / sec,
                clocks=clk, gpu_launches=launches * world,
                e2e=dict(value=e2e_units / e2e_sec / 1e9, unit=UNIT, h2d_bytes_per_step=wl.e2e_h2d,
                         d2h_bytes_per_step=wl.e2e_d2h),
                roofline=wl.roofline(statistics.mean(kern_ms), peaks))
    if in_step_ms:
        # for comparison: the same kernel inside the step, where it writes planar output and, with the events
        # around it, cannot start under the conversion kernel's tail (an empty pair of events reads 2.7 us)
        line["roofline"]["kernel_ms_in_step_planar_out"] = statistics.mean(in_step_ms)
    if not args.no_cpu_baseline and world == 1:
        dt, macs, sample = wl.oracle_sample(getattr(wl, "oracle_images", 4))
        line["cpu_baseline"] = dict(value=macs / dt / 1e9, unit=UNIT, cores=1, kind="oracle", sample=sample)
    print(json.dumps(line))
    if args.layer_table and hasattr(wl, "layer_rows"):
        with open(args.layer_table, "w") as f:
            f.write("layer,path,macs,ms,logical_gmacs\n")
            for name, path, macs, ms in wl.layer_rows:
                f.write("%s,%s,%d,%.5f,%.1f\n" % (name, path, macs, ms, macs / (ms * 1e-3) / 1e9))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
