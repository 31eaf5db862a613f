"""Network-shaped workloads: layer lists, seeded parameters, draw-count maps.

A network is a list of layer dicts over named tensors (channels-last, one byte
per activation).  ``build_network`` fills in filters and the per-layer
constants (per-channel scale and bias, quantisation steps).  The steps are
calibrated once with an ordinary float32 forward pass of the same layer list on
a few images; that pass is part of the input recipe only and never serves as an
expected value.
"""
import numpy as np

U8, S8 = 0, 1


def _conv(name, src, dst, cin, cout, k, stride, hin, relu=True, residual=None, groups=1,
          signed_out=False, pad=None):
    pad = k // 2 if pad is None else pad
    hout = (hin + 2 * pad - k) // stride + 1
    return dict(op="conv", name=name, src=src, dst=dst, cin=cin, cout=cout, k=k, stride=stride,
                pad=pad, groups=groups, relu=relu, residual=residual, signed_out=signed_out,
                hin=hin, hout=hout)


def resnet_layers(blocks, widths, in_hw, stem_out=64, stem_k=7, n_classes=1000):
    """Bottleneck ResNet shape: stem conv /2, max-pool /2, stages of bottlenecks
    (1x1 -> w, 3x3 w -> w carrying the stage stride, 1x1 -> 4w, projection shortcut on
    the first block of a stage), global average pool, classifier."""
    L = [_conv("conv1", "image", "stem", 3, stem_out, stem_k, 2, in_hw)]
    h = L[-1]["hout"]
    hp = (h + 2 - 3) // 2 + 1
    L.append(dict(op="maxpool", name="pool1", src="stem", dst="p0", c=stem_out, k=3, stride=2, pad=1,
                  hin=h, hout=hp))
    h, cin, cur = hp, stem_out, "p0"
    for si, (n, wd) in enumerate(zip(blocks, widths)):
        for b in range(n):
            s = 2 if (b == 0 and si > 0) else 1
            pre = "s%db%d" % (si + 1, b)
            L.append(_conv(pre + "_a", cur, pre + "_ta", cin, wd, 1, 1, h))
            L.append(_conv(pre + "_b", pre + "_ta", pre + "_tb", wd, wd, 3, s, h))
            ho = L[-1]["hout"]
            if b == 0:
                L.append(_conv(pre + "_proj", cur, pre + "_sc", cin, wd * 4, 1, s, h, relu=False,
                               signed_out=True))
                res = pre + "_sc"
            else:
                res = cur
            L.append(_conv(pre + "_c", pre + "_tb", pre + "_out", wd, wd * 4, 1, 1, ho, residual=res))
            cur, cin, h = pre + "_out", wd * 4, ho
    L.append(dict(op="avgpool", name="gap", src=cur, dst="pooled", c=cin, hin=h, hout=1))
    L.append(_conv("fc", "pooled", "logits", cin, n_classes, 1, 1, 1, relu=False, signed_out=True))
    return L


def resnet50_layers():
    return resnet_layers([3, 4, 6, 3], [64, 128, 256, 512], 224)


def tiny_resnet_layers():
    """Same layer kinds as ResNet-50 at a size the CPU oracle finishes in seconds."""
    return resnet_layers([2, 1], [16, 32], 40, stem_out=16, stem_k=7, n_classes=24)


def mobilenet_layers(cfg, in_hw, stem_out=32, last=1280, n_classes=1000):
    """MobileNet-v2 shape: 3x3/2 stem, inverted residuals (expand 1x1, depthwise 3x3,
    linear 1x1 projection; shortcut when stride 1 and equal widths), 1x1 head, pool, classifier."""
    L = [_conv("conv0", "image", "t0", 3, stem_out, 3, 2, in_hw)]
    h, cin, cur = L[-1]["hout"], stem_out, "t0"
    for bi, (t, c, n, s) in enumerate(cfg):
        for i in range(n):
            st = s if i == 0 else 1
            hid = cin * t
            pre = "b%d_%d" % (bi, i)
            src = cur
            if t != 1:
                L.append(_conv(pre + "_exp", cur, pre + "_e", cin, hid, 1, 1, h))
                src = pre + "_e"
            L.append(_conv(pre + "_dw", src, pre + "_d", hid, hid, 3, st, h, groups=hid))
            h = L[-1]["hout"]
            res = cur if (st == 1 and cin == c) else None
            L.append(_conv(pre + "_proj", pre + "_d", pre + "_o", hid, c, 1, 1, h, relu=False,
                           residual=res, signed_out=True))
            cur, cin = pre + "_o", c
    L.append(_conv("conv_last", cur, "head", cin, last, 1, 1, h))
    L.append(dict(op="avgpool", name="gap", src="head", dst="pooled", c=last, hin=h, hout=1))
    L.append(_conv("fc", "pooled", "logits", last, n_classes, 1, 1, 1, relu=False, signed_out=True))
    return L


def mobilenetv2_layers():
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2),
           (6, 320, 1, 1)]
    return mobilenet_layers(cfg, 224)


def tiny_mobilenet_layers():
    cfg = [(1, 16, 1, 1), (6, 16, 2, 2), (6, 32, 2, 2)]
    return mobilenet_layers(cfg, 32, stem_out=16, last=64, n_classes=20)


def network_macs(layers):
    """Logical multiply-accumulates per image (one per activation/weight pair)."""
    total = 0
    for l in layers:
        if l["op"] == "conv":
            total += l["hout"] ** 2 * l["cout"] * (l["cin"] // l["groups"]) * l["k"] ** 2
    return total


def _pctl(a, pct):
    v = float(np.percentile(np.asarray(a, dtype=np.float64), pct))
    return v if v > 0 else 1.0


def build_network(layers, in_hw, batch, seed, act_qmax_unsigned, act_qmax_signed, prune_frac=0.0,
                  n_calib=2, image_step=1.0 / 128):
    """Seeded parameters for a layer list.

    Filters are He-normal N(0, 2/d) (optionally magnitude-pruned per layer), the folded
    batch-norm factor is U(0.5, 1.5) per channel, biases are N(0, 0.1^2) output steps, the
    image is uniform u8.  Output steps map the 99.9th percentile of each layer's float
    output on ``n_calib`` images to the top integer code.
    Returns dict(image=u8 [B,H,W,3], params={layer name: {...}}, steps={tensor: step}).
    """
    import torch
    import torch.nn.functional as F

    rng = np.random.default_rng(7000 + seed)
    image = rng.integers(0, 256, size=(batch, in_hw, in_hw, 3), dtype=np.uint8)
    nc = min(n_calib, batch)
    # calibration tensors: integer codes as float32 NCHW, with their step
    codes = {"image": torch.from_numpy(image[:nc].astype(np.float32)).permute(0, 3, 1, 2).contiguous()}
    steps = {"image": float(image_step)}
    dtypes = {"image": U8}
    params = {}
    lid = 0
    for l in layers:
        if l["op"] == "maxpool":
            codes[l["dst"]] = F.max_pool2d(codes[l["src"]], l["k"], l["stride"], l["pad"])
            steps[l["dst"]] = steps[l["src"]]
            dtypes[l["dst"]] = dtypes[l["src"]]
            continue
        if l["op"] == "avgpool":
            mean = codes[l["src"]].mean(dim=(2, 3), keepdim=True) * steps[l["src"]]
            out_step = _pctl(mean.numpy(), 99.9) / act_qmax_unsigned
            hw = l["hin"] * l["hin"]
            params[l["name"]] = dict(
                pool_mul=np.float32(np.float32(steps[l["src"]] / hw) * np.float32(1.0 / out_step)),
                qmin=0, qmax=act_qmax_unsigned)
            codes[l["dst"]] = torch.clamp(torch.round(mean / out_step), 0, act_qmax_unsigned)
            steps[l["dst"]] = out_step
            dtypes[l["dst"]] = U8
            continue
        cin_g = l["cin"] // l["groups"]
        d = cin_g * l["k"] * l["k"]
        w = rng.normal(0.0, np.sqrt(2.0 / d), size=(l["cout"], cin_g, l["k"], l["k"])).astype(np.float32)
        if prune_frac > 0:
            thr = np.quantile(np.abs(w), prune_frac)
            w[np.abs(w) <= thr] = 0.0
        bn = rng.uniform(0.5, 1.5, size=l["cout"]).astype(np.float32)
        in_step = np.float32(steps[l["src"]])
        scale = (bn * in_step).astype(np.float32)
        y = F.conv2d(codes[l["src"]], torch.from_numpy(w), None, l["stride"], l["pad"], 1, l["groups"])
        y = y * torch.from_numpy(scale).view(1, -1, 1, 1)
        res_scale = np.float32(0.0)
        if l["residual"] is not None:
            res_scale = np.float32(steps[l["residual"]])
            y = y + codes[l["residual"]] * float(res_scale)
        if l["relu"]:
            y = torch.relu(y)
        if l["signed_out"]:
            qmin, qmax = -act_qmax_signed, act_qmax_signed
            out_step = _pctl(np.abs(y.numpy()), 99.9) / act_qmax_signed
        else:
            qmin, qmax = 0, act_qmax_unsigned
            out_step = _pctl(np.maximum(y.numpy(), 0), 99.9) / act_qmax_unsigned
        bias = (rng.normal(0.0, 0.1, size=l["cout"]) * out_step).astype(np.float32)
        y = y + torch.from_numpy(bias).view(1, -1, 1, 1)
        if l["relu"]:
            y = torch.relu(y)
        codes[l["dst"]] = torch.clamp(torch.round(y / out_step), qmin, qmax)
        steps[l["dst"]] = out_step
        dtypes[l["dst"]] = S8 if l["signed_out"] else U8
        params[l["name"]] = dict(w=w, scale=scale, bias=bias, inv_step=np.float32(1.0 / out_step),
                                 qmin=qmin, qmax=qmax, res_scale=res_scale, layer_id=lid,
                                 out_dtype=dtypes[l["dst"]], in_dtype=dtypes[l["src"]],
                                 res_dtype=None if l["residual"] is None else dtypes[l["residual"]])
        lid += 1
    return dict(image=image, params=params, steps=steps, dtypes=dtypes)


def saliency_kmaps(batch, resolutions, seed, levels=(0, 1, 2, 3, 4), quantiles=(0.30, 0.55, 0.80, 0.925),
                   ref_res=56):
    """Per-image draw-count maps from a smooth random saliency field.

    f(u, v) = sum of three Gaussian blobs with random centre, width and height; the
    thresholds are quantiles of f on the image's ref_res x ref_res grid, so that
    levels log2 k = 0..4 cover 30 / 25 / 25 / 12.5 / 7.5 % of the locations (mean k = 4);
    the same thresholds are applied to f sampled at pixel centres of every resolution.
    Stands in for the entropy mask of Sec. 4.5.  Returns {res: u8 [batch, res, res]}.
    """
    rng = np.random.default_rng(9000 + seed)
    cx = rng.uniform(0, 1, size=(batch, 3))
    cy = rng.uniform(0, 1, size=(batch, 3))
    sg = rng.uniform(0.08, 0.25, size=(batch, 3))
    am = rng.uniform(0.5, 1.0, size=(batch, 3))

    def field(res):
        t = (np.arange(res) + 0.5) / res
        u, v = np.meshgrid(t, t, indexing="xy")
        f = np.zeros((batch, res, res))
        for b in range(3):
            f += am[:, b, None, None] * np.exp(
                -((u[None] - cx[:, b, None, None]) ** 2 + (v[None] - cy[:, b, None, None]) ** 2)
                / (2 * sg[:, b, None, None] ** 2))
        return f

    fref = field(ref_res).reshape(batch, -1)
    thr = np.quantile(fref, quantiles, axis=1).T  # [batch, 4]
    out = {}
    for res in resolutions:
        f = field(res)
        lvl = np.zeros(f.shape, dtype=np.int64)
        for q in range(thr.shape[1]):
            lvl += (f > thr[:, q, None, None])
        out[res] = np.asarray(levels, dtype=np.uint8)[lvl]
    return out
