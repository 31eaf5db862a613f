"""Runs a list of PSB layers (see ``workloads.nets``) through the library, layer by layer.

Only orchestration: every tensor operation is a call into the C ABI.  Activations stay
resident on the device, channels-last, one byte per element.
"""
import numpy as np
import torch

from . import binding as B


class Network:
    def __init__(self, ctx, layers, net, batch, level_mask, kmaps=None, uniform_log2k=3, fc_log2k=None,
                 path=B.PSB_PATH_AUTO):
        """layers/net: from workloads.build_network; kmaps: {resolution: u8 [batch, res, res]} or None."""
        self.ctx, self.layers, self.batch, self.level_mask, self.path = ctx, layers, batch, level_mask, path
        self.uniform_log2k = uniform_log2k
        self.fc_log2k = uniform_log2k if fc_log2k is None else fc_log2k
        dev = ctx.device
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.kmaps = None if kmaps is None else {r: t(m[:batch]) for r, m in kmaps.items()}
        self.params, self.weights, self.acts, self.qmax = {}, {}, {}, {"image": 255}
        hw = layers[0]["hin"]
        self.acts["image"] = torch.empty((batch, hw, hw, 3), dtype=torch.uint8, device=dev)
        for l in layers:
            p = net["params"].get(l["name"], {})
            if l["op"] == "conv":
                self.params[l["name"]] = dict(w=t(p["w"]), scale=t(p["scale"]), bias=t(p["bias"]), p=p)
                odt = torch.int8 if p["out_dtype"] == B.PSB_DT_S8 else torch.uint8
                shape = (batch, l["cout"]) if l["hin"] == 1 and l["k"] == 1 and l["src"] == "pooled" \
                    else (batch, l["hout"], l["hout"], l["cout"])
                self.acts[l["dst"]] = torch.empty(shape, dtype=odt, device=dev)
                self.qmax[l["dst"]] = max(abs(p["qmin"]), abs(p["qmax"]))
            elif l["op"] == "maxpool":
                self.acts[l["dst"]] = torch.empty((batch, l["hout"], l["hout"], l["c"]), dtype=torch.uint8, device=dev)
                self.qmax[l["dst"]] = self.qmax[l["src"]]
            else:
                self.params[l["name"]] = dict(p=p)
                self.acts[l["dst"]] = torch.empty((batch, l["c"]), dtype=torch.uint8, device=dev)
                self.qmax[l["dst"]] = p["qmax"]
        self.logits = torch.empty((batch, layers[-1]["cout"]), dtype=torch.float32, device=dev)
        self.paths = {}

    def sample(self, seed):
        """Fresh draws for every layer (psb_sample_weights; handles are created on first use)."""
        for l in self.layers:
            if l["op"] != "conv":
                continue
            pr = self.params[l["name"]]
            self.weights[l["name"]] = self.ctx.sample_weights(
                pr["w"], groups=l["groups"], seed=seed, layer_id=pr["p"]["layer_id"], level_mask=self.level_mask,
                into=self.weights.get(l["name"]))

    def forward(self, image=None, layer_events=None):
        """image: u8 CUDA tensor [batch, h, w, 3] (copied into the resident input buffer) or None.
        layer_events: optional dict that receives {layer name: (start, end)} CUDA events."""
        ctx = self.ctx
        if image is not None:
            self.acts["image"].copy_(image, non_blocking=True)
        prev_end = None
        for l in self.layers:
            if layer_events is not None:
                ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                if prev_end is not None:
                    prev_end.record()
                ev[0].record()
                layer_events[l["name"]] = ev
                prev_end = ev[1]
            x = self.acts[l["src"]]
            if l["op"] == "maxpool":
                ctx.maxpool2d_u8(x, B.PSB_LAYOUT_NHWC, l["k"], l["stride"], l["pad"], out=self.acts[l["dst"]])
                continue
            if l["op"] == "avgpool":
                p = self.params[l["name"]]["p"]
                ctx.global_avgpool_u8(x, B.PSB_LAYOUT_NHWC, p["pool_mul"], p["qmin"], p["qmax"], out=self.acts[l["dst"]])
                continue
            pr = self.params[l["name"]]
            p = pr["p"]
            is_fc = x.dim() == 2
            if self.kmaps is not None and not is_fc:
                ctx.set_sample_map(self.kmaps[l["hout"]])
            else:
                ctx.set_sample_map(None, self.fc_log2k if is_fc else self.uniform_log2k)
            res = None if l["residual"] is None else self.acts[l["residual"]]
            out = {"q": self.acts[l["dst"]]}
            if is_fc:
                out["f32"] = self.logits
                ctx.gemm(self.weights[l["name"]], x, pr["scale"], pr["bias"], l["relu"], p["inv_step"], p["qmin"],
                         p["qmax"], out_dtype=p["out_dtype"], in_max=self.qmax[l["src"]], path=self.path, out=out)
            else:
                ctx.conv2d(self.weights[l["name"]], x, B.PSB_LAYOUT_NHWC, l["stride"], l["pad"], pr["scale"],
                           pr["bias"], l["relu"], p["inv_step"], p["qmin"], p["qmax"], out_dtype=p["out_dtype"],
                           residual=res, residual_scale=p["res_scale"], in_max=self.qmax[l["src"]],
                           path=self.path, out=out)
            self.paths[l["name"]] = ctx.last_path()
        if prev_end is not None:
            prev_end.record()
        ctx.set_sample_map(None, 0)
        return self.logits

    def free(self):
        for w in self.weights.values():
            w.free()
        self.weights = {}
