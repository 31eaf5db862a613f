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
import hashlib
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


def measured_traffic(workload):
    """DRAM bytes per launch of the dominant kernel from the last ncu capture of this workload
    (profiles/traffic.json), or None when there is none or the kernel's source has changed since."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path)).get(workload)
    if not rec:
        return None
    src = os.path.join(ROOT, "paper_1904_02205_b200", "csrc", rec["source"])
    sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
    return rec["dram_bytes_per_launch"] if sha == rec["source_sha256"] else None


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

    def __init__(self, k, rank=0, sample_opts=None):
        from workloads import config2_conv

        self.k = k
        self.log2k = int(np.log2(k))
        self.sample_opts = dict(sample_opts or {})
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
        self.wt = ctx.sample_weights(self.w, seed=c["seed"], layer_id=0, level_mask=1 << self.log2k, **self.sample_opts)
        ctx.set_sample_map(None, self.log2k)
        self.out = {"q": torch.empty((32, 64, 56, 56), dtype=torch.uint8, device=dev)}
        self.out_nhwc = {"q": torch.empty((32, 56, 56, 64), dtype=torch.uint8, device=dev)}
        # pinned host buffers for the end-to-end measurement
        self.x_host = torch.from_numpy(c["x"]).pin_memory()
        self.q_host = torch.empty((32, 64, 56, 56), dtype=torch.uint8).pin_memory()
        self.x_stage = torch.empty_like(self.x)
        span = (1 << self.sample_opts.get("exp_bits", 4)) - 1 + self.log2k + 2
        self.planes = (span + 6) // 7

    def step(self, i):
        c, psb = self.cfg, self.psb
        self.ctx.sample_weights(self.w, seed=c["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt,
                                **self.sample_opts)
        self.ctx.conv2d(self.wt, self.x, psb.PSB_LAYOUT_NCHW, 1, 1, self.scale, self.bias, True,
                        c["inv_step"], 0, 15, in_max=15, out=self.out)

    def kernel_only(self):
        """The dominant kernel alone: contraction + output stage on channels-last input."""
        c, psb = self.cfg, self.psb
        self.ctx.conv2d(self.wt, self.x_nhwc, psb.PSB_LAYOUT_NHWC, 1, 1, self.scale, self.bias, True,
                        c["inv_step"], 0, 15, in_max=15, out=self.out_nhwc)

    def back_to_back(self, n_sets=24, rounds=4):
        """The dominant kernel launched back to back on a rotating set of input / output tensors larger than L2
        (24 x 12.8 MB): average device time per launch between one pair of events, i.e. without the gaps that a
        pair of events and an L2 flush put around a single launch."""
        c, psb, torch = self.cfg, self.psb, self.torch
        if not hasattr(self, "x_sets"):
            self.x_sets = [self.x_nhwc.clone() for _ in range(n_sets)]
            self.out_sets = [{"q": torch.empty_like(self.out_nhwc["q"])} for _ in range(n_sets)]
        def one(j):
            self.ctx.conv2d(self.wt, self.x_sets[j], psb.PSB_LAYOUT_NHWC, 1, 1, self.scale, self.bias, True,
                            c["inv_step"], 0, 15, in_max=15, out=self.out_sets[j])
        for j in range(n_sets):
            one(j)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(rounds):
            for j in range(n_sets):
                one(j)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / (rounds * n_sets)

    def e2e_step(self, i):
        self.x_stage.copy_(self.x_host, non_blocking=True)
        c, psb = self.cfg, self.psb
        self.ctx.sample_weights(self.w, seed=c["seed"] + i, layer_id=0, level_mask=1 << self.log2k, into=self.wt,
                                **self.sample_opts)
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
        # algorithmic bytes of the launch: activations in, codes out, digit planes once
        alg_bytes = 2.0 * 32 * 64 * 56 * 56 + self.planes * 64 * 576
        return dict(bound="tensor", kernel="psb_mma_kernel", achieved=achieved, peak=peak, unit="TOP/s (int8)",
                    frac=achieved / peak, frac_vs_sustained=achieved / (2.0 * peaks["bf16_tflops_sustained"]),
                    traffic=measured_traffic(self.name), traffic_unit="DRAM bytes per launch (ncu)",
                    algorithmic_bytes=alg_bytes, peak_source=peaks["source"] + " bf16 burst x 2",
                    planes=self.planes, logical_gmacs=self.macs / (kernel_ms * 1e-3) / 1e9,
                    kernel_ms=kernel_ms)

    def oracle_sample(self, n_images=4):
        """Time the CPU oracle on the first n_images of the batch; returns (seconds, macs)."""
        from oracle import psb_oracle as orc

        c = self.cfg
        x = np.ascontiguousarray(c["x"][:n_images])
        t0 = time.perf_counter()
        W, eb = orc.sample_level_ex(c["w"], c["seed"], 0, self.log2k, **self.sample_opts)[:2]
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

    def __init__(self, kind, k, rank=0, batch=0, sample_opts=None):
        from workloads import mobilenetv2_layers, network_macs, resnet50_layers

        self.kind, self.k, self.rank = kind, k, rank
        self.sample_opts = dict(sample_opts or {})
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
                          fc_log2k=4 if self.adaptive else None, sample_opts=self.sample_opts)
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
        span_bits = (1 << self.sample_opts.get("exp_bits", 4)) - 1 + (4 if self.adaptive else self.log2k) + 2
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

    def truncate_for_oracle(self, budget_macs):
        """Keep the longest prefix of the layer list whose work on one image fits the budget."""
        from workloads import network_macs

        keep = len(self.layers)
        while keep > 1 and network_macs(self.layers[:keep]) > budget_macs:
            keep -= 1
        self.oracle_layers = self.layers[:keep]

    def oracle_sample(self, n_images=1):
        from oracle import psb_oracle as orc

        layers = getattr(self, "oracle_layers", self.layers)
        if not hasattr(self, "net"):
            from workloads import build_network, saliency_kmaps

            self.net = build_network(self.layers, 224, max(n_images, 2), self.seed, self.qu, self.qs, prune_frac=self.prune)
            self.kmaps = saliency_kmaps(max(n_images, 2), [112, 56, 28, 14, 7], self.seed) if self.adaptive else None
        t0 = time.perf_counter()
        from workloads import network_macs

        orc.run_network(layers, self.net, self.net["image"][:n_images], self.seed, uniform_log2k=self.log2k,
                        fc_log2k=4 if self.adaptive else None,
                        kmaps=None if self.kmaps is None else {r: m[:n_images] for r, m in self.kmaps.items()})
        dt = time.perf_counter() - t0
        what = "all layers" if len(layers) == len(self.layers) else "the first %d of %d layers" % (len(layers), len(self.layers))
        return dt, network_macs(layers) * n_images, "first %d of %d images, %s, filters sampled once" % (n_images, self.batch, what)


def default_run_extras(args, ctx, psb, torch, timed):
    """What the default run reports beside config 2 at k = 8: the bare int8 issue rate, the draw-count sweep of
    the same layer, and the ResNet-50-shaped network at batch 64, k = 8 (per-launch device times from the
    library's own events)."""
    out = {}
    for _ in range(2):
        _, tops = ctx.int8_mma_probe(192, 20000)
    out["int8_probe_tops"] = tops
    sweep = {}
    for k in (1, 2, 4, 16):
        w = ConvWorkload(k, 0)
        w.setup(ctx, psb, torch)
        for i in range(3):
            w.step(i)
        ms = timed(w.step, 50, first=3)
        sec = sum(ms) * 1e-3
        sweep[str(k)] = dict(ms_per_step=sec * 1e3 / 50, gmacs=w.macs * 50 / sec / 1e9, images_per_s=w.images * 50 / sec)
        w.wt.free()
    out["k_sweep"] = sweep
    ctx.set_sample_map(None, 3)
    peaks = measured_peaks()
    net = NetWorkload("resnet50", 8, 0, batch=64)
    net.setup(ctx, psb, torch)
    for i in range(3):
        net.step(i)
    ms = timed(net.step, 10, first=3)
    sec = sum(ms) * 1e-3
    sample_ms = timed(lambda i: net.nw.sample(100 + i), 5)
    ctx.contraction_timing(True)
    net.nw.forward()
    per_launch = ctx.contraction_times()
    ctx.contraction_timing(False)
    planes = 3
    tensor_layers = [l for l in net.layers if l["op"] == "conv" and net.nw.paths[l["name"]] == psb.PSB_PATH_TENSOR]
    rec = dict(ms_per_step=sec * 1e3 / 10, images_per_s=net.batch * 10 / sec, gmacs=net.macs * 10 / sec / 1e9,
               sampler_ms=statistics.mean(sample_ms[1:]), contraction_launches=len(per_launch))
    if len(per_launch) == len(tensor_layers):
        dense_ops, dense_ms, hbm_bytes, hbm_ms = 0.0, 0.0, 0.0, 0.0
        for l, t in zip(tensor_layers, per_launch):
            d = (l["cin"] // l["groups"]) * l["k"] ** 2
            macs = l["hout"] ** 2 * l["cout"] * d * net.batch
            nbytes = net.batch * (l["hin"] ** 2 * l["cin"] + l["hout"] ** 2 * l["cout"] * (2 if l["residual"] else 1)) + 4 * l["cout"] * d
            # a layer is bound by bytes when its multiply-accumulates per byte, times the digit planes, stay
            # below the ridge of the machine (measured tensor peak over measured HBM bandwidth)
            ridge = 2.0 * peaks["bf16_tflops_sustained"] * 1e12 / 2.0 / (peaks["hbm_gbs"] * 1e9)
            if macs * planes / nbytes >= ridge and l["name"] != "conv1":
                dense_ops += 2.0 * macs * planes
                dense_ms += t
            else:
                hbm_bytes += nbytes
                hbm_ms += t
        rec["dense_convs"] = dict(tops=dense_ops / (dense_ms * 1e-3) / 1e12, ms=dense_ms,
                                  frac_of_2x_bf16_sustained=dense_ops / (dense_ms * 1e-3) / 1e12 / (2.0 * peaks["bf16_tflops_sustained"]),
                                  frac_of_int8_probe=dense_ops / (dense_ms * 1e-3) / 1e12 / tops)
        rec["bandwidth_bound_layers"] = dict(gbs=hbm_bytes / (hbm_ms * 1e-3) / 1e9, ms=hbm_ms,
                                             frac_of_hbm=hbm_bytes / (hbm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                             note="algorithmic bytes (input, output, shortcut, fp32 filter once) over the "
                                                  "contraction kernel's device time; the stem's gather pass is not in it")
    out["resnet50_b64_k8"] = rec
    net.nw.free()
    return out


def sample_options(args):
    opts = {}
    if args.exp_bits != 4:
        opts["exp_bits"] = args.exp_bits
    if args.underflow:
        opts["underflow"] = 1
    if args.prob_bits:
        opts["prob_bits"] = args.prob_bits
    return opts


class AttentionWorkload(NetWorkload):
    """The two-pass scheme of Sec. 4.5 on the ResNet-50-shaped network: a first pass with k = 8 everywhere, the
    pixelwise entropy of its last convolutional layer thresholded at the image mean, a second pass with k = 16
    inside the mask and k = 8 outside (psb8/16).  Both passes use one set of draws (levels share draws)."""

    def __init__(self, k, rank=0, batch=0, sample_opts=None):
        NetWorkload.__init__(self, "resnet50", 8, rank, batch=batch or 64, sample_opts=sample_opts)
        self.name = "resnet50_attention_b%d" % self.batch
        self.macs = 2 * self.macs_per_image * self.batch           # two passes
        self.mean_k = 8.0

    def setup(self, ctx, psb, torch):
        from paper_1904_02205_b200.network import Network
        from workloads import build_network

        self.ctx, self.psb, self.torch = ctx, psb, torch
        self.net = build_network(self.layers, 224, self.batch, self.seed + 100 * self.rank, self.qu, self.qs)
        res = [112, 56, 28, 14, 7]
        self.maps = {r: torch.full((self.batch, r, r), 3, dtype=torch.uint8, device=ctx.device) for r in res}
        self.first = Network(ctx, self.layers, self.net, self.batch, 0b11000, uniform_log2k=3, sample_opts=self.sample_opts)
        self.nw = Network(ctx, self.layers, self.net, self.batch, 0b11000, kmaps={r: m.cpu().numpy() for r, m in self.maps.items()},
                          uniform_log2k=3, fc_log2k=4, sample_opts=self.sample_opts, weights_from=self.first)
        self.nw.kmaps = self.maps                                  # the maps the producer writes, in place
        self.last = [l for l in self.layers if l["op"] == "conv" and l["hout"] == 7][-1]["dst"]
        self.last_step = float(self.net["steps"][self.last])
        self.entropy = torch.empty((self.batch, 7, 7), dtype=torch.float32, device=ctx.device)
        self.first.sample(self.seed)
        self.image_host = torch.from_numpy(self.net["image"]).pin_memory()
        self.image_dev = self.image_host.to(ctx.device)
        self.logits_host = torch.empty((self.batch, self.layers[-1]["cout"]), dtype=torch.float32).pin_memory()
        self.first.forward(self.image_dev)
        self.nw.acts["image"] = self.first.acts["image"]
        self._propose()
        self.nw.forward(self.image_dev)
        self.e2e_h2d = self.image_host.numel()
        self.e2e_d2h = self.logits_host.numel() * 4
        self.layer_ms = None

    def _propose(self):
        self.ctx.attention_entropy(self.first.acts[self.last], self.last_step, out=self.entropy)
        self.ctx.attention_maps(self.entropy, 3, 4, [112, 56, 28, 14, 7], out=self.maps)

    def step(self, i):
        self.first.sample(self.seed + i)
        self.first.forward()
        self._propose()
        self.nw.forward()

    def e2e_step(self, i):
        self.first.acts["image"].copy_(self.image_host, non_blocking=True)
        self.step(i)
        self.logits_host.copy_(self.nw.logits, non_blocking=True)

    def kernel_only(self):
        self.refined = float((self.maps[7] == 4).float().mean().item())
        NetWorkload.kernel_only(self)


def make_workload(args, rank):
    if args.workload == "resnet50_attention":
        return AttentionWorkload(args.k, rank, batch=args.batch, sample_opts=sample_options(args))
    if args.workload == "conv3x3":
        return ConvWorkload(args.k, rank, sample_options(args))
    if args.workload == "fc":
        return FcWorkload(args.k, rank)
    return NetWorkload(args.workload, args.k, rank, batch=args.batch, sample_opts=sample_options(args))


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
    # a bounded sample per step, so that the whole run stays within a few minutes whatever --steps is: the
    # oracle does about 0.6 G multiply-accumulates per second on one core
    budget_macs = 0.6e9 * 150.0 / max(1, args.warmup + args.steps)
    per_image = wl.macs / wl.images
    n_img = int(max(1, min(getattr(wl, "oracle_images", 1), budget_macs // per_image)))
    if isinstance(wl, NetWorkload) and per_image > budget_macs:
        wl.truncate_for_oracle(budget_macs)
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
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="psb")
    ap.add_argument("--workload", default="conv3x3", choices=["conv3x3", "fc", "resnet50", "mobilenetv2", "resnet50_adaptive", "resnet50_attention"])
    ap.add_argument("--k", type=int, default=8)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--exp-bits", type=int, default=4, help="octaves of the exponent window: 2^exp_bits (Sec. 4.4)")
    ap.add_argument("--underflow", action="store_true", help="Bernoulli gate below the window instead of flushing (Sec. 3.1)")
    ap.add_argument("--prob-bits", type=int, default=0, help="probabilities on a grid of 2^b points, packed draws (Sec. 4.4)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="default workload only: skip the draw-count sweep, the int8 probe and the network record")
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
    b2b_ms = wl.back_to_back() if args.workload == "conv3x3" else None
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
    extras = {}
    if args.workload == "conv3x3" and world == 1 and not args.no_extras:
        extras = default_run_extras(args, ctx, psb, torch, timed)
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
                config=dict(workload=wl.name, k=args.k, sampling=sample_options(args) or "defaults",
                            l2="flushed between steps (1 GiB memset, untimed)",
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
        r = line["roofline"]
        r["kernel_ms_in_step_planar_out"] = statistics.mean(in_step_ms)
        r["frac_in_step"] = r["frac"] * r["kernel_ms"] / r["kernel_ms_in_step_planar_out"]
    if b2b_ms:
        # the same kernel launched back to back on inputs that rotate through more than the L2 holds
        r = line["roofline"]
        r["kernel_ms_back_to_back"] = b2b_ms
        r["frac_back_to_back"] = r["frac"] * r["kernel_ms"] / b2b_ms
        r["back_to_back_note"] = "24 input/output sets of 12.8 MB in rotation (> L2), one pair of events around 96 launches"
    if clk.get("sm_mhz"):
        # kernel time x the SM clock sampled under load: comparable across runs whatever the clock was
        line["roofline"]["kernel_clocks"] = line["roofline"].get("kernel_ms", 0.0) * 1e-3 * clk["sm_mhz"] * 1e6
    if "int8_probe_tops" in extras:
        # the bare tcgen05 int8 issue rate measured in this process (zero operands, so the clocks stay up)
        line["roofline"]["int8_probe_tops"] = extras["int8_probe_tops"]
        line["roofline"]["frac_vs_int8_probe"] = line["roofline"]["achieved"] / extras["int8_probe_tops"]
    for key in ("k_sweep", "resnet50_b64_k8"):
        if key in extras:
            line[key] = extras[key]
    if hasattr(wl, "refined"):
        line["config"]["refined_fraction"] = wl.refined      # share of the locations the mask sends to k = 16
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
