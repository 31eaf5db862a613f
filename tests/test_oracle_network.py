"""Pins of the oracle's network walk (``psb_oracle.run_network``) on the CPU.

``run_network`` decides which tensor feeds a layer, which tensor is the shortcut, which draw-count
map (by resolution) and which level a layer uses and how codes are cast.  Here it is checked against
forward passes written out block by block from the network shapes themselves (stem, pooling, bottleneck
/ inverted-residual blocks, classifier) - they never read a layer's ``src`` / ``residual`` / ``hout``
entries - with the contraction done by a library routine (``torch.nn.functional.conv2d`` in float64,
exact on these integers).

1. Filters rounded to powers of two (p = 0 in Eq. 6, so every draw is deterministic and every level
   gives the same real weight) with power-of-two scales and steps: the whole forward pass is exact in
   float32 and must equal a plain float64 forward pass, code for code, for any seed, level or map.
2. Ordinary filters under per-resolution maps whose level sets differ per resolution: every layer's
   accumulators must equal the library convolution with the integer filter of the level that the map
   of the layer's own output resolution names at each location.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from workloads import build_network, tiny_mobilenet_layers, tiny_resnet_layers

RESNET = dict(blocks=[2, 1], widths=[16, 32], in_hw=40)
MOBILENET = dict(cfg=[(1, 16, 1, 1), (6, 16, 2, 2), (6, 32, 2, 2)], in_hw=32, stem_out=16)


def _pow2(v):
    """Nearest power of two in the log domain, sign kept, zeros kept."""
    v = np.asarray(v, dtype=np.float64)
    out = np.zeros_like(v)
    nz = v != 0
    out[nz] = np.sign(v[nz]) * 2.0 ** np.round(np.log2(np.abs(v[nz])))
    return out


def _make_exact(net):
    """Round every constant of a generated network so that its forward pass is exact in float32."""
    for name, p in net["params"].items():
        if "pool_mul" in p:
            p["pool_mul"] = np.float32(_pow2(p["pool_mul"]))
            continue
        w = _pow2(p["w"])
        top = np.abs(w).max()
        w[np.abs(w) < top / 8] = 0.0                       # four octaves: sums stay well inside 24 bits
        p["w"] = w.astype(np.float32)
        p["scale"] = _pow2(p["scale"]).astype(np.float32)
        p["inv_step"] = np.float32(_pow2(p["inv_step"]))
        step = 1.0 / float(p["inv_step"])
        p["bias"] = (np.round(p["bias"] / (step / 4)) * (step / 4)).astype(np.float32)
        p["res_scale"] = np.float32(_pow2(p["res_scale"])) if p["res_scale"] != 0 else np.float32(0)


class _Ref:
    """Float64 forward pass over codes; `filt(name, level)` gives the real-valued filter to use."""

    def __init__(self, net, check_exact):
        self.p, self.check_exact, self.codes = net["params"], check_exact, {}

    def _exact(self, t):
        if self.check_exact:
            a = t.numpy()
            assert np.array_equal(a.astype(np.float32).astype(np.float64), a), "the test's exactness assumption fails"

    def conv(self, name, x, stride, pad, groups=1, relu=True, res=None):
        p = self.p[name]
        y = F.conv2d(x, torch.from_numpy(p["w"].astype(np.float64)), None, stride, pad, 1, groups)
        self._exact(y)
        y = y * torch.from_numpy(p["scale"].astype(np.float64)).view(1, -1, 1, 1) \
            + torch.from_numpy(p["bias"].astype(np.float64)).view(1, -1, 1, 1)
        self._exact(y)
        if res is not None:
            y = y + res * float(p["res_scale"])
            self._exact(y)
        if relu:
            y = torch.relu(y)
        q = torch.clamp(torch.round(y * float(p["inv_step"])), p["qmin"], p["qmax"])    # round: ties to even
        self.codes[name] = q
        return q, y

    def avgpool(self, name, x):
        p = self.p[name]
        s = x.sum(dim=(2, 3))
        return torch.clamp(torch.round(s * float(p["pool_mul"])), p["qmin"], p["qmax"])


def _ref_resnet(net, image, spec, check_exact=True):
    r = _Ref(net, check_exact)
    out = {}
    x = torch.from_numpy(image.astype(np.float64)).permute(0, 3, 1, 2)
    x, _ = r.conv("conv1", x, 2, 3)
    out["stem"] = x
    x = F.max_pool2d(x, 3, 2, 1)
    out["p0"] = x
    for si, n in enumerate(spec["blocks"]):
        for b in range(n):
            pre = "s%db%d" % (si + 1, b)
            s = 2 if (b == 0 and si > 0) else 1
            a, _ = r.conv(pre + "_a", x, 1, 0)
            bb, _ = r.conv(pre + "_b", a, s, 1)
            if b == 0:
                sc, _ = r.conv(pre + "_proj", x, s, 0, relu=False)
                out[pre + "_sc"] = sc
            else:
                sc = x
            x, _ = r.conv(pre + "_c", bb, 1, 0, res=sc)
            out[pre + "_ta"], out[pre + "_tb"], out[pre + "_out"] = a, bb, x
    pooled = r.avgpool("gap", x)
    out["pooled"] = pooled
    q, y = r.conv("fc", pooled.view(pooled.shape[0], -1, 1, 1), 1, 0, relu=False)
    out["logits"] = q.view(q.shape[0], -1)
    return out, y.view(y.shape[0], -1)


def _ref_mobilenet(net, image, spec, check_exact=True):
    r = _Ref(net, check_exact)
    out = {}
    x = torch.from_numpy(image.astype(np.float64)).permute(0, 3, 1, 2)
    x, _ = r.conv("conv0", x, 2, 1)
    out["t0"] = x
    cin = spec["stem_out"]
    for bi, (t, c, n, s) in enumerate(spec["cfg"]):
        for i in range(n):
            pre = "b%d_%d" % (bi, i)
            st = s if i == 0 else 1
            h = x
            if t != 1:
                h, _ = r.conv(pre + "_exp", x, 1, 0)
                out[pre + "_e"] = h
            d, _ = r.conv(pre + "_dw", h, st, 1, groups=cin * t)
            out[pre + "_d"] = d
            res = x if (st == 1 and cin == c) else None
            x, _ = r.conv(pre + "_proj", d, 1, 0, relu=False, res=res)
            out[pre + "_o"] = x
            cin = c
    x, _ = r.conv("conv_last", x, 1, 0)
    out["head"] = x
    pooled = r.avgpool("gap", x)
    out["pooled"] = pooled
    q, y = r.conv("fc", pooled.view(pooled.shape[0], -1, 1, 1), 1, 0, relu=False)
    out["logits"] = q.view(q.shape[0], -1)
    return out, y.view(y.shape[0], -1)


def _same(acts, ref):
    for name, t in ref.items():
        got = acts[name]
        want = t.numpy()
        if want.ndim == 4:
            want = want.transpose(0, 2, 3, 1)
        assert got.shape == want.shape, name
        assert np.array_equal(got.astype(np.int64), want.astype(np.int64)), \
            "%s: %d of %d codes differ" % (name, int((got != want).sum()), want.size)


def _maps(n, resolutions, level_sets, seed):
    rng = np.random.default_rng(seed)
    return {r: rng.choice(level_sets[i % len(level_sets)], size=(n, r, r)).astype(np.uint8)
            for i, r in enumerate(resolutions)}


def test_run_network_resnet_shape_with_power_of_two_filters_is_an_exact_float_forward_pass(oracle):
    L = tiny_resnet_layers()
    net = build_network(L, RESNET["in_hw"], 3, 2, 15, 15)
    _make_exact(net)
    ref, ref_logits = _ref_resnet(net, net["image"][:3], RESNET)
    for seed, lv, fc in ((2, 3, None), (9, 0, 4)):
        acts, logits = oracle.run_network(L, net, net["image"][:3], seed, uniform_log2k=lv, fc_log2k=fc)
        _same(acts, ref)
        assert np.array_equal(logits.astype(np.float64), ref_logits.numpy())
    # per-resolution maps whose levels differ per resolution: with p = 0 the codes must not change
    kmaps = _maps(3, [20, 10, 5], [[0, 1], [2, 3], [4, 5]], 4)
    acts, logits = oracle.run_network(L, net, net["image"][:3], 5, uniform_log2k=3, fc_log2k=2, kmaps=kmaps)
    _same(acts, ref)
    assert np.array_equal(logits.astype(np.float64), ref_logits.numpy())


def test_run_network_mobilenet_shape_with_power_of_two_filters_is_an_exact_float_forward_pass(oracle):
    L = tiny_mobilenet_layers()
    net = build_network(L, MOBILENET["in_hw"], 3, 3, 255, 127, prune_frac=0.5)
    _make_exact(net)
    ref, ref_logits = _ref_mobilenet(net, net["image"][:3], MOBILENET)
    acts, logits = oracle.run_network(L, net, net["image"][:3], 3, uniform_log2k=4)
    _same(acts, ref)
    assert np.array_equal(logits.astype(np.float64), ref_logits.numpy())


def _layerwise(oracle, L, net, acts, seed, res_of, level_at, structure):
    """Every conv layer of `acts` recomputed from the tensors the *structure* names: accumulators by the
    library convolution with the integer filter of each level, selected per location, then the (separately
    pinned) output stage."""
    for name, src, residual, stride, pad, groups, relu in structure:
        p = net["params"][name]
        x = acts[src]
        is_fc = x.ndim == 2
        x4 = x.reshape(x.shape[0], 1, 1, -1) if is_fc else x
        xt = torch.from_numpy(x4.astype(np.float64)).permute(0, 3, 1, 2)
        km, lv = level_at(name, is_fc, res_of.get(name))
        levels = sorted(set(np.unique(km).tolist())) if km is not None else [lv]
        acc = None
        eb = None
        for l in levels:
            W, eb, _ = oracle.sample_level(p["w"], seed, p["layer_id"], l)
            a = F.conv2d(xt, torch.from_numpy(W.astype(np.float64)), None, stride, pad, 1, groups)
            a = a.permute(0, 2, 3, 1).numpy()
            assert np.abs(a).max() < 2.0 ** 52
            a = a.astype(np.int64)
            acc = a if acc is None else np.where((km == l)[..., None], a, acc) if km is not None else a
        g = oracle.geom(x4.shape, oracle.NHWC, oracle.U8 if x4.dtype == np.uint8 else oracle.S8, p["w"].shape,
                        groups, stride, pad)
        assert acc.shape == oracle.out_shape(g), name
        res = None if residual is None else acts[residual]
        y, q = oracle.epilogue(acc, g, p["scale"], p["bias"], eb, relu, p["inv_step"], p["qmin"], p["qmax"],
                               residual=res, residual_scale=p["res_scale"], kmap=km, uniform_log2k=lv)
        got = acts[[l for l in L if l["name"] == name][0]["dst"]]
        q = q.reshape(got.shape)
        assert np.array_equal(got.astype(np.int64), q.astype(np.int64)), \
            "%s: %d of %d codes differ" % (name, int((got != q).sum()), q.size)
        yield name, y


def _resnet_structure(spec):
    S = [("conv1", "image", None, 2, 3, 1, True)]
    res = {"conv1": spec["in_hw"] // 2}
    h = spec["in_hw"] // 4
    cur = "p0"
    for si, n in enumerate(spec["blocks"]):
        for b in range(n):
            pre = "s%db%d" % (si + 1, b)
            s = 2 if (b == 0 and si > 0) else 1
            S.append((pre + "_a", cur, None, 1, 0, 1, True))
            res[pre + "_a"] = h
            S.append((pre + "_b", pre + "_ta", None, s, 1, 1, True))
            h = h // s
            res[pre + "_b"] = h
            if b == 0:
                S.append((pre + "_proj", cur, None, s, 0, 1, False))
                res[pre + "_proj"] = h
            S.append((pre + "_c", pre + "_tb", pre + "_sc" if b == 0 else cur, 1, 0, 1, True))
            res[pre + "_c"] = h
            cur = pre + "_out"
    S.append(("fc", "pooled", None, 1, 0, 1, False))
    return S, res


def test_run_network_takes_each_layers_level_from_the_map_of_its_own_resolution(oracle):
    L = tiny_resnet_layers()
    net = build_network(L, RESNET["in_hw"], 2, 2, 15, 15)
    kmaps = _maps(2, [20, 10, 5], [[0, 2], [1, 3], [4, 5]], 6)      # disjoint level sets per resolution
    seed, fc_level = 13, 6
    acts, logits = oracle.run_network(L, net, net["image"][:2], seed, uniform_log2k=3, fc_log2k=fc_level, kmaps=kmaps)
    S, res_of = _resnet_structure(RESNET)

    def level_at(name, is_fc, res):
        return (None, fc_level) if is_fc else (kmaps[res], 3)

    ys = dict(_layerwise(oracle, L, net, acts, seed, res_of, level_at, S))
    assert len(ys) == sum(1 for l in L if l["op"] == "conv")
    assert np.array_equal(logits, ys["fc"].reshape(logits.shape))
    # pooling layers between them
    assert np.array_equal(acts["p0"], oracle.maxpool_u8(acts["stem"], oracle.NHWC, 3, 2, 1))
    last = "s%db%d_out" % (len(RESNET["blocks"]), RESNET["blocks"][-1] - 1)
    g = net["params"]["gap"]
    assert np.array_equal(acts["pooled"], oracle.global_avgpool_u8(acts[last], oracle.NHWC, g["pool_mul"], g["qmin"], g["qmax"]))
    # a planted mistake would show: the same walk with the maps of two resolutions swapped does not match
    swapped = {20: kmaps[20], 10: np.ascontiguousarray(kmaps[5].repeat(2, 1).repeat(2, 2)), 5: np.ascontiguousarray(kmaps[10][:, ::2, ::2])}

    def level_swapped(name, is_fc, res):
        return (None, fc_level) if is_fc else (swapped[res], 3)

    with pytest.raises(AssertionError):
        dict(_layerwise(oracle, L, net, acts, seed, res_of, level_swapped, S))
