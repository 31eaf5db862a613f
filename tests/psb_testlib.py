"""Helpers shared by the GPU parity tests: run one layer through the CUDA library and
through the CPU oracle on the same seeded inputs and compare element by element."""
import numpy as np


def oracle_layer(orc, w, x, layout, groups, stride, pad, seed, layer_id, levels, kmap, uniform_log2k,
                 scale, bias, relu, inv_step, qmin, qmax, residual=None, res_scale=0.0, exp_bits=4,
                 norm=0, opts=None):
    Ws, eb = {}, None
    for l in levels:
        if opts:
            Ws[l], eb = orc.sample_level_ex(w, seed, layer_id, l, exp_bits=exp_bits, norm=norm, **opts)[:2]
        else:
            Ws[l], eb, _ = orc.sample_level(w, seed, layer_id, l, exp_bits=exp_bits, norm=norm)
    lay = orc.NCHW if layout == 0 else orc.NHWC
    g = orc.geom(x.shape, lay, orc.U8 if x.dtype == np.uint8 else orc.S8, w.shape, groups, stride, pad)
    acc = orc.conv_acc(x, g, Ws, kmap=kmap, uniform_log2k=uniform_log2k)
    y, q = orc.epilogue(acc, g, scale, bias, eb, relu, inv_step, qmin, qmax, residual=residual,
                        residual_scale=res_scale, kmap=kmap, uniform_log2k=uniform_log2k)
    return dict(W=Ws, e_base=eb, acc=acc, f32=y, q=q)


def gpu_layer(psb, ctx, w, x, layout, groups, stride, pad, seed, layer_id, levels, kmap, uniform_log2k,
              scale, bias, relu, inv_step, qmin, qmax, out_dtype, residual=None, res_scale=0.0,
              exp_bits=4, norm=0, in_max=0, path=0, guard=True, want=("q", "f32", "acc"), opts=None):
    import torch

    dev = ctx.device
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    mask = 0
    for l in levels:
        mask |= 1 << l
    wt = ctx.sample_weights(t(w), groups=groups, seed=seed, layer_id=layer_id, level_mask=mask,
                            exp_bits=exp_bits, norm=norm, **(opts or {}))
    exported = {l: tuple(v.cpu().numpy() for v in ctx.weights_export(wt, l)) for l in levels}
    ctx.set_sample_map(None if kmap is None else t(kmap), uniform_log2k)
    O, KH, KW = w.shape[0], w.shape[2], w.shape[3]
    if layout == 0:
        n, c, h, ww = x.shape
    else:
        n, h, ww, c = x.shape
    oh, ow = (h + 2 * pad - KH) // stride + 1, (ww + 2 * pad - KW) // stride + 1
    oshape = (n, O, oh, ow) if layout == 0 else (n, oh, ow, O)
    numel = int(np.prod(oshape))
    G = 64  # guard band elements on both sides of every output
    qdt = torch.uint8 if out_dtype == psb.PSB_DT_U8 else torch.int8
    bufs = {"q": torch.full((numel + 2 * G,), 0x5A, dtype=qdt, device=dev),
            "f32": torch.full((numel + 2 * G,), -777.0, dtype=torch.float32, device=dev),
            "acc": torch.full((numel + 2 * G,), -(1 << 60) + 7, dtype=torch.int64, device=dev)}
    out = {k: v[G:G + numel].view(oshape) for k, v in bufs.items() if k in want}
    res = ctx.conv2d(wt, t(x), layout, stride, pad, t(scale), t(bias), relu, inv_step, qmin, qmax,
                     out_dtype=out_dtype, residual=None if residual is None else t(residual),
                     residual_scale=res_scale, in_max=in_max, path=path, want=want, out=out)
    status = ctx.device_status()
    used = ctx.last_path()
    host = {k: v.cpu().numpy() for k, v in res.items()}
    if guard:
        for k, v in bufs.items():
            full = v.cpu().numpy()
            fill = {"q": np.array(0x5A).astype(full.dtype), "f32": np.float32(-777.0),
                    "acc": np.int64(-(1 << 60) + 7)}[k]
            assert np.all(full[:G] == fill) and np.all(full[G + numel:] == fill), "guard band of %s overwritten" % k
    ctx.set_sample_map(None, 0)
    wt.free()
    return dict(W={l: exported[l][0] for l in levels}, e_base=exported[levels[0]][1], acc=host.get("acc"),
                f32=host.get("f32"), q=host.get("q"), status=status, path=used)


def compare(g, o, levels):
    assert g["status"] == 0, "device status %d" % g["status"]
    assert np.array_equal(g["e_base"], o["e_base"]), "e_base"
    for l in levels:
        assert np.array_equal(g["W"][l].astype(np.int64), o["W"][l]), "integer filter, level %d" % l
    if g["acc"] is not None:
        assert np.array_equal(g["acc"], o["acc"]), "accumulators: %d of %d differ" % (
            int((g["acc"] != o["acc"]).sum()), o["acc"].size)
    if g["q"] is not None:
        bad = int((g["q"].astype(np.int32) != o["q"]).sum())
        assert bad == 0, "re-quantised activations: %d of %d differ" % (bad, o["q"].size)
    # fp32: 1e-6 relative (both sides use correctly rounded IEEE operations, so expect equality)
    if g["f32"] is not None:
        assert np.allclose(g["f32"], o["f32"], rtol=1e-6, atol=0.0), "fp32 outputs"
