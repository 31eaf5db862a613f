"""Runs a list of PSB layers (see ``workloads.nets``) through the library, layer by layer.

Only orchestration: every tensor operation is a call into the C ABI.  Activations stay
resident on the device, channels-last, one byte per element.
"""
import numpy as np
import torch

from . import binding as B


class Network:
    def __init__(self, ctx, layers, net, batch, level_mask, kmaps=None, uniform_log2k=3, fc_log2k=None,
                 path=B.PSB_PATH_AUTO, sample_opts=None, weights_from=None):
        """layers/net: from workloads.build_network; kmaps: {resolution: u8 [batch, res, res]} or None;
        sample_opts: keyword options of Context.sample_weights (exp_bits, underflow, prob_bits, ...);
        weights_from: another Network over the same layers whose sampled filters this one uses (two passes of one
        network with different draw counts share one set of draws)."""
        self.ctx, self.layers, self.batch, self.level_mask, self.path = ctx, layers, batch, level_mask, path
        self.sample_opts = dict(sample_opts or {})
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
        self._batch = None
        self._ops = None
        self._shared = weights_from
        if weights_from is not None:
            self.weights = weights_from.weights

    def sample(self, seed):
        """Fresh draws for every layer.  The first call creates the handles layer by layer
        (psb_sample_weights); later calls re-sample all layers in one psb_sample_batch_run."""
        if self._shared is not None:
            return self._shared.sample(seed)
        if self._batch is not None:
            self.ctx.sample_batch_run(self._batch, seed)
            return
        for l in self.layers:
            if l["op"] != "conv":
                continue
            pr = self.params[l["name"]]
            self.weights[l["name"]] = self.ctx.sample_weights(
                pr["w"], groups=l["groups"], seed=seed, layer_id=pr["p"]["layer_id"], level_mask=self.level_mask,
                into=self.weights.get(l["name"]), **self.sample_opts)
        convs = [l["name"] for l in self.layers if l["op"] == "conv"]
        self._batch = self.ctx.sample_batch_create([self.params[n]["w"] for n in convs],
                                                   [self.weights[n] for n in convs])

    def _build_ops(self):
        """The forward pass as one psb_run op list (same arguments as the per-layer calls)."""
        ops = (B.psb_op * len(self.layers))()
        for op, l in zip(ops, self.layers):
            x = self.acts[l["src"]]
            op.x_dev = x.data_ptr()
            if l["op"] != "conv":
                n, h, w, c = x.shape
                op.conv.layout, op.conv.n, op.conv.c, op.conv.h, op.conv.w = B.PSB_LAYOUT_NHWC, n, c, h, w
                op.pool_out_dev = self.acts[l["dst"]].data_ptr()
                if l["op"] == "maxpool":
                    op.kind, op.pool_k, op.conv.stride, op.conv.pad = B.PSB_OP_MAXPOOL, l["k"], l["stride"], l["pad"]
                else:
                    p = self.params[l["name"]]["p"]
                    op.kind, op.pool_mul, op.pool_qmin, op.pool_qmax = B.PSB_OP_AVGPOOL, float(p["pool_mul"]), p["qmin"], p["qmax"]
                continue
            pr = self.params[l["name"]]
            p = pr["p"]
            is_fc = x.dim() == 2
            op.weights = self.weights[l["name"]].handle.value
            if self.kmaps is not None and not is_fc:
                km = self.kmaps[l["hout"]]
                op.map_dev, op.map_n, op.map_oh, op.map_ow = km.data_ptr(), km.shape[0], km.shape[1], km.shape[2]
            else:
                op.uniform_log2k = self.fc_log2k if is_fc else self.uniform_log2k
            ep = B.psb_epilogue()
            ep.scale_dev, ep.bias_dev = pr["scale"].data_ptr(), pr["bias"].data_ptr()
            if l["residual"] is not None:
                res = self.acts[l["residual"]]
                ep.residual_dev, ep.residual_dtype = res.data_ptr(), B._dt_of(res)
            ep.residual_scale = float(p["res_scale"])
            ep.relu, ep.inv_step, ep.qmin, ep.qmax = int(l["relu"]), float(p["inv_step"]), p["qmin"], p["qmax"]
            ep.out_dtype = p["out_dtype"]
            ep.q_out_dev = self.acts[l["dst"]].data_ptr()
            if is_fc:
                ep.f32_out_dev = self.logits.data_ptr()
                op.kind = B.PSB_OP_GEMM
                op.gemm = B.psb_gemm_desc(B._dt_of(x), self.qmax[l["src"]], x.shape[0], x.shape[1], self.path, ep)
            else:
                n, h, w, c = x.shape
                op.kind = B.PSB_OP_CONV2D
                op.conv = B.psb_conv_desc(B.PSB_LAYOUT_NHWC, B._dt_of(x), self.qmax[l["src"]], n, c, h, w,
                                          l["stride"], l["pad"], self.path, ep)
        self._ops = ops

    def forward(self, image=None, layer_events=None):
        """image: u8 CUDA tensor [batch, h, w, 3] (copied into the resident input buffer) or None.
        layer_events: optional dict that receives {layer name: (start, end)} CUDA events."""
        ctx = self.ctx
        if image is not None:
            self.acts["image"].copy_(image, non_blocking=True)
        if layer_events is None and self.paths:
            # every later pass: one psb_run call over the whole layer list
            if self._ops is None:
                self._build_ops()
            ctx.run(self._ops, len(self.layers))
            return self.logits
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
        if self._shared is not None:
            self.weights = {}
            return
        if self._batch is not None:
            self.ctx.sample_batch_free(self._batch)
            self._batch = None
        for w in self.weights.values():
            w.free()
        self.weights = {}
