"""GPU parity: CUDA library (through the C ABI) against the CPU oracle, element by element.

Bit-exact on integer filters, base exponents, 64-bit accumulators and re-quantised
activations; 1e-6 relative on fp32 outputs.
"""
import numpy as np
import pytest

from psb_testlib import compare, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psb():
    import paper_1904_02205_b200 as p

    return p


@pytest.fixture(scope="module")
def ctx(psb):
    c = psb.Context(0)
    yield c
    c.close()


def _layer_inputs(rng, N, C, H, W, O, KH, KW, groups, layout, x_dtype=np.uint8, x_hi=16, w_sigma=None):
    d = (C // groups) * KH * KW
    sigma = np.sqrt(2.0 / d) if w_sigma is None else w_sigma
    w = rng.normal(0, sigma, size=(O, C // groups, KH, KW)).astype(np.float32)
    lo = 0 if x_dtype == np.uint8 else -x_hi
    shape = (N, C, H, W) if layout == 0 else (N, H, W, C)
    x = rng.integers(lo, x_hi, size=shape).astype(x_dtype)
    scale = rng.uniform(0.5, 1.5, O).astype(np.float32)
    bias = rng.normal(0, 0.5, O).astype(np.float32)
    return w, x, scale, bias


def _both(psb, ctx, oracle, w, x, layout, groups, stride, pad, levels, scale, bias, kmap=None,
          uniform=None, relu=True, inv_step=0.5, qmin=0, qmax=15, out_dtype=0, residual=None,
          res_scale=0.0, exp_bits=4, norm=0, in_max=0, path=0, seed=5, layer_id=3, want=("q", "f32", "acc"),
          opts=None):
    uniform = levels[0] if uniform is None else uniform
    o = oracle_layer(oracle, w, x, layout, groups, stride, pad, seed, layer_id, levels, kmap, uniform,
                     scale, bias, relu, np.float32(inv_step), qmin, qmax, residual, np.float32(res_scale),
                     exp_bits, norm, opts=opts)
    g = gpu_layer(psb, ctx, w, x, layout, groups, stride, pad, seed, layer_id, levels, kmap, uniform,
                  scale, bias, relu, np.float32(inv_step), qmin, qmax, out_dtype, residual,
                  np.float32(res_scale), exp_bits, norm, in_max, path, want=want, opts=opts)
    compare(g, o, levels)
    return g


# ------------------------------------------------------------------------ sampler

@pytest.mark.parametrize("shape,groups", [((128, 256, 1, 1), 1), ((64, 64, 3, 3), 1), ((96, 1, 3, 3), 96),
                                           ((16, 3, 7, 7), 1), ((5, 512, 3, 3), 1), ((1000, 40, 1, 1), 1),
                                           ((3, 2100, 1, 1), 1)])
@pytest.mark.parametrize("norm", [0, 1])
def test_sampler_all_levels(psb, ctx, oracle, shape, groups, norm):
    import torch

    rng = np.random.default_rng(abs(hash((shape, norm))) % 2 ** 31)
    w = rng.normal(0, 0.1, size=shape).astype(np.float32)
    flat = w.reshape(-1)
    flat[rng.random(flat.size) < 0.05] = 0.0
    flat[:4] = [0.5, -0.25, 1e-41, 3e-9]          # exact powers of two, a sub-normal, a flushed one
    for exp_bits in (4, 2):
        wt = ctx.sample_weights(torch.from_numpy(w).cuda(), groups=groups, seed=2 ** 40 + 17, layer_id=9,
                                level_mask=0x7F, exp_bits=exp_bits, norm=norm)
        for l in range(7):
            Wg, ebg = (v.cpu().numpy() for v in ctx.weights_export(wt, l))
            Wo, ebo, _ = oracle.sample_level(w, 2 ** 40 + 17, 9, l, exp_bits=exp_bits, norm=norm)
            assert np.array_equal(ebg, ebo)
            assert np.array_equal(Wg.astype(np.int64), Wo), (shape, norm, exp_bits, l)
        assert ctx.device_status() == 0
        wt.free()


def test_resampling_in_place_changes_with_the_seed_only(psb, ctx, oracle):
    import torch

    rng = np.random.default_rng(1)
    w = rng.normal(0, 0.1, size=(32, 32, 3, 3)).astype(np.float32)
    wd = torch.from_numpy(w).cuda()
    wt = ctx.sample_weights(wd, seed=1, layer_id=0, level_mask=0b1000)
    a = ctx.weights_export(wt, 3)[0].cpu().numpy()
    ctx.sample_weights(wd, seed=2, layer_id=0, level_mask=0b1000, into=wt)
    b = ctx.weights_export(wt, 3)[0].cpu().numpy()
    ctx.sample_weights(wd, seed=1, layer_id=0, level_mask=0b1000, into=wt)
    c = ctx.weights_export(wt, 3)[0].cpu().numpy()
    assert np.array_equal(a, c) and not np.array_equal(a, b)
    assert np.array_equal(b.astype(np.int64), oracle.sample_level(w, 2, 0, 3)[0])
    with pytest.raises(psb.PsbError):
        ctx.sample_weights(wd, seed=1, layer_id=0, level_mask=0b0100, into=wt)
    wt.free()


# ------------------------------------------------------------------ shift-add path

def test_config1_fully_connected(psb, ctx, oracle):
    from workloads import config1_fc

    c = config1_fc()
    x = c["x"].reshape(16, 1, 1, 256)
    _both(psb, ctx, oracle, c["w"], x, 1, 1, 1, 0, [c["log2k"]], c["scale"], c["bias"], relu=True,
          inv_step=c["inv_step"], qmin=0, qmax=255, seed=c["seed"], layer_id=0, path=psb.PSB_PATH_SHIFT_ADD)


@pytest.mark.parametrize("case", [
    dict(N=2, C=8, H=9, W=7, O=12, K=3, groups=1, stride=1, pad=1, layout=1),
    dict(N=1, C=12, H=10, W=10, O=8, K=3, groups=4, stride=2, pad=1, layout=0),
    dict(N=3, C=40, H=13, W=11, O=40, K=3, groups=40, stride=1, pad=1, layout=1),
    dict(N=2, C=40, H=13, W=11, O=40, K=3, groups=40, stride=2, pad=1, layout=0),
    dict(N=2, C=3, H=21, W=21, O=10, K=7, groups=1, stride=2, pad=3, layout=1),
    dict(N=2, C=20, H=5, W=6, O=7, K=1, groups=1, stride=1, pad=0, layout=0),
])
def test_shift_add_convolutions(psb, ctx, oracle, case):
    rng = np.random.default_rng(case["C"] * 31 + case["K"])
    w, x, scale, bias = _layer_inputs(rng, case["N"], case["C"], case["H"], case["W"], case["O"], case["K"],
                                      case["K"], case["groups"], case["layout"], x_hi=256)
    g = _both(psb, ctx, oracle, w, x, case["layout"], case["groups"], case["stride"], case["pad"], [4],
              scale, bias, inv_step=0.02, qmax=255, path=psb.PSB_PATH_SHIFT_ADD)
    assert g["path"] == psb.PSB_PATH_SHIFT_ADD


def test_shift_add_signed_input_residual_and_map(psb, ctx, oracle):
    rng = np.random.default_rng(77)
    w, x, scale, bias = _layer_inputs(rng, 2, 16, 8, 8, 24, 3, 3, 1, 1, x_dtype=np.int8, x_hi=128)
    res = rng.integers(-128, 128, size=(2, 8, 8, 24)).astype(np.int8)
    kmap = rng.choice([0, 1, 3, 6], size=(2, 8, 8)).astype(np.uint8)
    _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [0, 1, 3, 6], scale, bias, kmap=kmap, relu=False, inv_step=0.01,
          qmin=-128, qmax=127, out_dtype=1, residual=res, res_scale=0.07, path=psb.PSB_PATH_SHIFT_ADD)


# --------------------------------------------------------------------- tensor path

@pytest.mark.parametrize("case", [
    dict(N=2, C=64, H=9, W=15, O=64, K=1, stride=1, pad=0),      # plain GEMM, ragged last tile
    dict(N=1, C=256, H=12, W=12, O=128, K=1, stride=1, pad=0),   # 128-byte K block, two channel tiles
    dict(N=3, C=96, H=7, W=9, O=24, K=1, stride=1, pad=0),       # partial K block, ragged channels
    dict(N=2, C=32, H=10, W=10, O=80, K=1, stride=1, pad=0),     # 32-byte K block
    dict(N=2, C=64, H=14, W=14, O=64, K=3, stride=1, pad=1),     # 3x3 through the im2col loader
    dict(N=3, C=64, H=15, W=13, O=64, K=3, stride=2, pad=1),     # strided 3x3, odd sizes
    dict(N=2, C=128, H=14, W=14, O=256, K=1, stride=2, pad=0),   # strided projection
    dict(N=2, C=32, H=20, W=20, O=16, K=7, stride=2, pad=3),     # 7x7
    dict(N=1, C=160, H=9, W=9, O=64, K=3, stride=1, pad=1),      # 160 channels: K blocks 128 + 32
])
def test_tensor_path_layers(psb, ctx, oracle, case):
    rng = np.random.default_rng(case["C"] * 131 + case["K"] * 7 + case["stride"])
    w, x, scale, bias = _layer_inputs(rng, case["N"], case["C"], case["H"], case["W"], case["O"], case["K"],
                                      case["K"], 1, 1)
    g = _both(psb, ctx, oracle, w, x, 1, 1, case["stride"], case["pad"], [3], scale, bias, inv_step=0.6,
              in_max=15, path=psb.PSB_PATH_TENSOR)
    assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("case", [
    dict(N=3, C=3, H=37, W=41, O=64, K=7, stride=2, pad=3, dtype=np.uint8, hi=256),   # image stem
    dict(N=2, C=3, H=30, W=30, O=32, K=3, stride=2, pad=1, dtype=np.uint8, hi=256),   # 27 -> 32 columns
    dict(N=2, C=24, H=13, W=13, O=40, K=1, stride=1, pad=0, dtype=np.int8, hi=128),   # 24 channels, signed
    dict(N=2, C=20, H=11, W=9, O=70, K=3, stride=1, pad=1, dtype=np.uint8, hi=256),   # ragged everything
    dict(N=1, C=3, H=21, W=300, O=16, K=5, stride=2, pad=2, dtype=np.uint8, hi=256),  # two strips of output columns, odd row count
    dict(N=2, C=5, H=9, W=140, O=16, K=3, stride=1, pad=1, dtype=np.int8, hi=128),    # rows that start at odd byte addresses
])
def test_tensor_path_few_input_channels_full_range_bytes(psb, ctx, oracle, case):
    """Filters whose input-channel count is not a multiple of 16 run on the tensor cores through an
    explicitly gathered activation matrix; unsigned bytes up to 255 are fed with an offset of 128
    and corrected by 128 * sum(W)."""
    rng = np.random.default_rng(case["C"] * 17 + case["K"])
    w, x, scale, bias = _layer_inputs(rng, case["N"], case["C"], case["H"], case["W"], case["O"], case["K"],
                                      case["K"], 1, 1, x_dtype=case["dtype"], x_hi=case["hi"])
    for levels, kmap in (([3], None), ([0, 2, 4], "random")):
        km = None
        if kmap:
            oh = (case["H"] + 2 * case["pad"] - case["K"]) // case["stride"] + 1
            ow = (case["W"] + 2 * case["pad"] - case["K"]) // case["stride"] + 1
            km = rng.choice(levels, size=(case["N"], oh, ow)).astype(np.uint8)
        g = _both(psb, ctx, oracle, w, x, 1, 1, case["stride"], case["pad"], levels, scale, bias, kmap=km,
                  inv_step=0.02, qmax=255, path=psb.PSB_PATH_TENSOR)
        assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("case", [
    dict(N=2, C=96, H=13, W=11, stride=1, dtype=np.uint8, hi=256, res=None),
    dict(N=3, C=144, H=15, W=15, stride=2, dtype=np.uint8, hi=256, res=None),
    dict(N=2, C=32, H=9, W=9, stride=1, dtype=np.int8, hi=128, res=np.int8),
    dict(N=2, C=960, H=7, W=7, stride=1, dtype=np.uint8, hi=256, res=np.uint8),
])
def test_depthwise_codes_only(psb, ctx, oracle, case):
    """Depthwise 3x3 through the vectorised channels-last kernel (only re-quantised codes wanted)."""
    rng = np.random.default_rng(case["C"] + case["stride"])
    C = case["C"]
    w, x, scale, bias = _layer_inputs(rng, case["N"], C, case["H"], case["W"], C, 3, 3, C, 1,
                                      x_dtype=case["dtype"], x_hi=case["hi"])
    oh = (case["H"] + 2 - 3) // case["stride"] + 1
    ow = (case["W"] + 2 - 3) // case["stride"] + 1
    res = None
    if case["res"] is not None:
        lo, hi = (0, 256) if case["res"] == np.uint8 else (-128, 128)
        res = rng.integers(lo, hi, size=(case["N"], oh, ow, C)).astype(case["res"])
    g = _both(psb, ctx, oracle, w, x, 1, C, case["stride"], 1, [4], scale, bias, inv_step=0.03, qmax=255,
              residual=res, res_scale=0.2, want=("q",))
    assert g["path"] == psb.PSB_PATH_SHIFT_ADD


@pytest.mark.parametrize("case", [
    dict(N=2, C=96, H=14, W=14, O=32, K=1, stride=1),     # projection after a ReLU6: bytes up to 255
    dict(N=2, C=64, H=15, W=15, O=64, K=3, stride=2),     # taps but no padding
    dict(N=64, C=1280, H=1, W=1, O=1000, K=1, stride=1),  # classifier on pooled unsigned bytes
])
def test_tensor_path_full_range_unsigned_bytes_without_padding(psb, ctx, oracle, case):
    rng = np.random.default_rng(case["C"] + case["K"])
    w, x, scale, bias = _layer_inputs(rng, case["N"], case["C"], case["H"], case["W"], case["O"], case["K"],
                                      case["K"], 1, 1, x_hi=256)
    for want in (("q", "f32", "acc"), ("q",)):
        g = _both(psb, ctx, oracle, w, x, 1, 1, case["stride"], 0, [4], scale, bias, relu=False, inv_step=0.01,
                  qmin=-128, qmax=127, out_dtype=1, path=psb.PSB_PATH_TENSOR, want=want)
        assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("O,with_res,with_map", [(24, False, False), (24, True, False), (40, True, True), (72, False, True)])
def test_tensor_path_rows_of_odd_multiples_of_eight_channels(psb, ctx, oracle, O, with_res, with_map):
    """Output rows that are 8- but not 16-byte aligned keep the vector store path (codes only)."""
    rng = np.random.default_rng(O)
    N, C, H, W = 3, 96, 13, 12
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, 1, 1, 1, 1, x_hi=128)
    res = rng.integers(0, 256, size=(N, H, W, O)).astype(np.uint8) if with_res else None
    kmap = rng.integers(0, 5, size=(N, H, W)).astype(np.uint8) if with_map else None
    levels = [0, 1, 2, 3, 4] if with_map else [3]
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 0, levels, scale, bias, kmap=kmap, inv_step=0.02, qmax=255,
              residual=res, res_scale=0.1, in_max=127, path=psb.PSB_PATH_TENSOR, want=("q",))
    assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("O,with_res", [(64, False), (72, True), (20, True)])
def test_tensor_path_planar_layout_codes_only(psb, ctx, oracle, O, with_res):
    """[n][c][h][w] tensors in and out, only re-quantised codes wanted: planar stores from the tensor path."""
    rng = np.random.default_rng(O + 1)
    N, C, H, W = 3, 64, 14, 13
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, 3, 3, 1, 0, x_hi=16)
    res = rng.integers(0, 16, size=(N, O, H, W)).astype(np.uint8) if with_res else None
    g = _both(psb, ctx, oracle, w, x, 0, 1, 1, 1, [3], scale, bias, inv_step=0.4, qmax=15, residual=res,
              res_scale=0.3, in_max=15, path=psb.PSB_PATH_TENSOR, want=("q",))
    assert g["path"] == psb.PSB_PATH_TENSOR


# (N, C, H, W, O, KH, KW, pad, layout, signed input, shortcut): stride-1 filters with taps, one channel
# block and codes-only output take the band mode of the tensor kernel (a tile is 128 positions of one
# image in padded-row order); odd and even padded widths, no padding, wide filters, ragged last tiles,
# several images, two channel tiles, planar and channels-last outputs
@pytest.mark.parametrize("case", [(3, 64, 13, 11, 64, 3, 3, 1, 1, False, False),
                                  (2, 64, 30, 30, 128, 3, 3, 1, 1, False, True),
                                  (2, 128, 14, 9, 64, 2, 2, 1, 1, False, True),
                                  (2, 64, 12, 17, 64, 3, 3, 0, 1, False, False),
                                  (1, 64, 9, 21, 64, 2, 2, 1, 1, True, False),
                                  (2, 64, 10, 23, 48, 1, 3, 0, 0, False, True),
                                  (2, 128, 11, 6, 64, 3, 1, 0, 1, False, False),
                                  (5, 64, 7, 7, 64, 3, 3, 1, 0, False, False)])
def test_tensor_path_band_mode_codes_only(psb, ctx, oracle, case):
    N, C, H, W, O, KH, KW, pad, layout, signed, with_res = case
    rng = np.random.default_rng(abs(hash(case)) % 2 ** 31)
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, KH, KW, 1, layout, x_dtype=np.int8 if signed else np.uint8,
                                      x_hi=16)
    OH, OW = H + 2 * pad - KH + 1, W + 2 * pad - KW + 1
    res = None
    if with_res:
        res = rng.integers(0, 16, size=(N, O, OH, OW) if layout == 0 else (N, OH, OW, O)).astype(np.uint8)
    g = _both(psb, ctx, oracle, w, x, layout, 1, 1, pad, [3], scale, bias, inv_step=0.4, residual=res,
              res_scale=0.25 if with_res else 0.0, in_max=16 if signed else 15, path=psb.PSB_PATH_TENSOR, want=("q",))
    assert g["path"] == psb.PSB_PATH_TENSOR


def test_depthwise_5x5_codes_only(psb, ctx, oracle):
    rng = np.random.default_rng(55)
    C = 48
    w, x, scale, bias = _layer_inputs(rng, 2, C, 12, 10, C, 5, 5, C, 1, x_hi=256)
    _both(psb, ctx, oracle, w, x, 1, C, 1, 2, [3], scale, bias, inv_step=0.03, qmax=255, want=("q",))


def test_fully_connected_on_the_tensor_path(psb, ctx, oracle):
    rng = np.random.default_rng(5)
    w, x, scale, bias = _layer_inputs(rng, 64, 512, 1, 1, 1000, 1, 1, 1, 1)
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 0, [3], scale, bias, relu=False, inv_step=0.3, qmin=-128, qmax=127,
              out_dtype=1, in_max=15)
    assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("log2k", [0, 1, 2, 4, 5, 6])
def test_tensor_path_every_draw_count(psb, ctx, oracle, log2k):
    rng = np.random.default_rng(log2k)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 12, 12, 64, 3, 3, 1, 1)
    _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [log2k], scale, bias, inv_step=0.6, in_max=15,
          path=psb.PSB_PATH_TENSOR)


def test_tensor_path_per_location_draw_counts(psb, ctx, oracle):
    rng = np.random.default_rng(21)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 16, 16, 64, 3, 3, 1, 1)
    kmap = np.zeros((2, 16, 16), dtype=np.uint8)
    kmap[0, :8] = 3                       # tiles with a single level
    kmap[0, 8:] = rng.choice([0, 1, 2, 3, 4], size=(8, 16))   # mixed tiles
    kmap[1] = rng.choice([2, 4], size=(16, 16))
    _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [0, 1, 2, 3, 4], scale, bias, kmap=kmap, inv_step=0.6, in_max=15,
          path=psb.PSB_PATH_TENSOR)


@pytest.mark.parametrize("case", [(3, 64, 10, 16, 64, False), (2, 128, 7, 24, 72, True), (5, 32, 9, 8, 64, True)])
def test_tensor_path_per_location_draw_counts_1x1_patch_tiles(psb, ctx, oracle, case):
    """1x1 layers under a per-location map on channels-last tensors (rows sorted by level, gathered, scattered back
    in the output stage): ragged sizes, a smooth region with a single level, with and without a shortcut."""
    N, C, H, W, O, with_res = case
    rng = np.random.default_rng(abs(hash(case)) % 2 ** 31)
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, 1, 1, 1, 1)
    kmap = rng.choice([0, 1, 2, 3, 4], size=(N, H, W)).astype(np.uint8)
    kmap[0, : H // 2] = 2                       # a smooth region: whole tiles of one level
    res = rng.integers(0, 16, size=(N, H, W, O)).astype(np.uint8) if with_res else None
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 0, [0, 1, 2, 3, 4], scale, bias, kmap=kmap, inv_step=0.5,
              residual=res, res_scale=0.2 if with_res else 0.0, in_max=15, path=psb.PSB_PATH_TENSOR)
    assert g["path"] == psb.PSB_PATH_TENSOR


def test_tensor_path_signed_inputs_residual_nchw_and_exponent_options(psb, ctx, oracle):
    rng = np.random.default_rng(22)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 10, 10, 32, 3, 3, 1, 0, x_dtype=np.int8, x_hi=128)
    res = rng.integers(0, 256, size=(2, 32, 10, 10)).astype(np.uint8)
    _both(psb, ctx, oracle, w, x, 0, 1, 1, 1, [3], scale, bias, relu=False, inv_step=0.05, qmin=-128, qmax=127,
          out_dtype=1, residual=res, res_scale=0.3, norm=1, path=psb.PSB_PATH_TENSOR)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 10, 10, 32, 3, 3, 1, 1)
    res = rng.integers(-128, 128, size=(2, 10, 10, 32)).astype(np.int8)
    _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, inv_step=0.5, residual=res, res_scale=0.3,
          exp_bits=3, in_max=15, path=psb.PSB_PATH_TENSOR)


def test_auto_path_selection(psb, ctx, oracle):
    rng = np.random.default_rng(23)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 12, 12, 64, 3, 3, 1, 1)
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, in_max=15)
    assert g["path"] == psb.PSB_PATH_TENSOR
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [3], scale, bias)          # full-range u8: CUDA cores
    assert g["path"] == psb.PSB_PATH_SHIFT_ADD
    w, x, scale, bias = _layer_inputs(rng, 2, 48, 12, 12, 48, 3, 3, 48, 1)
    g = _both(psb, ctx, oracle, w, x, 1, 48, 1, 1, [3], scale, bias, in_max=15)
    assert g["path"] == psb.PSB_PATH_SHIFT_ADD


# ----------------------------------------------------- config 2 at its full size

@pytest.mark.parametrize("log2k", [0, 3])
def test_config2_full_size_sampled_outputs(psb, ctx, oracle, log2k):
    """The 3x3 64->64 conv on 56x56, batch 32, NCHW, with all three outputs wanted (the general output loop;
    the launch the benchmark times, codes only, is the next test): accumulators at 4000 sampled outputs
    against the oracle, all image borders included, plus whole-tensor properties."""
    import torch
    from workloads import config2_conv

    c = config2_conv()
    dev = ctx.device
    wt = ctx.sample_weights(torch.from_numpy(c["w"]).to(dev), seed=c["seed"], layer_id=0, level_mask=1 << log2k)
    ctx.set_sample_map(None, log2k)
    out = ctx.conv2d(wt, torch.from_numpy(c["x"]).to(dev), psb.PSB_LAYOUT_NCHW, 1, 1,
                     torch.from_numpy(c["scale"]).to(dev), torch.from_numpy(c["bias"]).to(dev), True,
                     c["inv_step"], 0, 15, in_max=15, want=("q", "f32", "acc"))
    assert ctx.device_status() == 0 and ctx.last_path() == psb.PSB_PATH_TENSOR
    acc, q, f32 = (out[k].cpu().numpy() for k in ("acc", "q", "f32"))
    W, eb, _ = oracle.sample_level(c["w"], c["seed"], 0, log2k)
    g = oracle.geom(c["x"].shape, oracle.NCHW, oracle.U8, c["w"].shape, 1, 1, 1)
    rng = np.random.default_rng(3)
    pts = np.stack([rng.integers(0, 32, 4000), rng.integers(0, 64, 4000), rng.integers(0, 56, 4000),
                    rng.integers(0, 56, 4000)], 1)
    pts[:500, 2] = rng.choice([0, 55], 500)
    pts[250:750, 3] = rng.choice([0, 55], 500)
    ref = oracle.conv_acc_points(c["x"], g, {log2k: W}, pts, uniform_log2k=log2k)
    got = acc[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]]
    assert np.array_equal(got, ref)
    for t in range(0, 4000, 40):
        n, o, oy, ox = pts[t]
        y = oracle.dequant_one(ref[t], c["scale"][o], eb[o], log2k, c["bias"][o], relu=True)
        assert f32[n, o, oy, ox] == np.float32(y)
        assert q[n, o, oy, ox] == oracle.requant_one(y, c["inv_step"], 0, 15)
    assert q.max() <= 15 and (f32 >= 0).all()
    wt.free()


# ---------------------------------------------------------------- errors and glue

def test_argument_errors_are_reported_not_launched(psb, ctx):
    import torch

    w = torch.randn(64, 64, 3, 3, device=ctx.device)
    wt = ctx.sample_weights(w, level_mask=0b100)
    x = torch.zeros(1, 8, 8, 64, dtype=torch.uint8, device=ctx.device)
    sc = torch.ones(64, device=ctx.device)
    ctx.set_sample_map(None, 3)                                 # level 3 was not sampled
    with pytest.raises(psb.PsbError) as e:
        ctx.conv2d(wt, x, 1, 1, 1, sc, sc, True, 1.0, 0, 15)
    assert e.value.status == psb.PSB_ERR_BAD_K
    ctx.set_sample_map(None, 2)
    with pytest.raises(psb.PsbError) as e:                      # channel mismatch
        ctx.conv2d(wt, torch.zeros(1, 8, 8, 32, dtype=torch.uint8, device=ctx.device), 1, 1, 1, sc, sc, True, 1.0, 0, 15)
    assert e.value.status == psb.PSB_ERR_INVALID_ARG
    with pytest.raises(psb.PsbError) as e:                      # code range beyond the container
        ctx.conv2d(wt, x, 1, 1, 1, sc, sc, True, 1.0, 0, 300)
    assert e.value.status == psb.PSB_ERR_INVALID_ARG
    with pytest.raises(psb.PsbError) as e:                      # full-range u8 cannot take the tensor path
        ctx.conv2d(wt, x, 1, 1, 1, sc, sc, True, 1.0, 0, 15, path=psb.PSB_PATH_TENSOR)
    assert e.value.status == psb.PSB_ERR_UNSUPPORTED
    kmap = torch.zeros(1, 4, 4, dtype=torch.uint8, device=ctx.device)
    ctx.set_sample_map(kmap)                                    # map of the wrong size
    with pytest.raises(psb.PsbError) as e:
        ctx.conv2d(wt, x, 1, 1, 1, sc, sc, True, 1.0, 0, 15)
    assert e.value.status == psb.PSB_ERR_INVALID_ARG
    with pytest.raises(psb.PsbError):
        ctx.sample_weights(w, level_mask=0)
    with pytest.raises(psb.PsbError):
        ctx.sample_weights(w, level_mask=1, exp_bits=5)
    ctx.set_sample_map(None, 0)
    assert ctx.device_status() == 0
    wt.free()


def test_device_side_errors_are_sticky_until_read(psb, ctx):
    import torch

    w = torch.randn(16, 16, 1, 1, device=ctx.device)
    w[3, 2, 0, 0] = float("nan")
    wt = ctx.sample_weights(w, level_mask=1)
    assert ctx.device_status() == psb.PSB_ERR_NONFINITE_WEIGHT
    assert ctx.device_status() == 0
    wt.free()
    w = torch.randn(64, 64, 1, 1, device=ctx.device)
    wt = ctx.sample_weights(w, level_mask=0b101)
    sc = torch.ones(64, device=ctx.device)
    for path, in_max in ((psb.PSB_PATH_SHIFT_ADD, 0), (psb.PSB_PATH_TENSOR, 15)):
        kmap = torch.full((2, 8, 8), 2, dtype=torch.uint8, device=ctx.device)
        kmap[1, 3, 3] = 1                                       # a level that was not sampled
        ctx.set_sample_map(kmap)
        x = torch.ones(2, 8, 8, 64, dtype=torch.uint8, device=ctx.device)
        ctx.conv2d(wt, x, 1, 1, 0, sc, sc, True, 1.0, 0, 15, in_max=in_max, path=path)
        assert ctx.device_status() == psb.PSB_ERR_BAD_K
    ctx.set_sample_map(None, 0)
    wt.free()


def test_pooling_kernels(psb, ctx, oracle):
    import torch

    rng = np.random.default_rng(31)
    for layout in (0, 1):
        x = rng.integers(0, 256, size=(3, 9, 13, 11) if layout == 0 else (3, 13, 11, 9), dtype=np.uint8)
        xd = torch.from_numpy(x).to(ctx.device)
        assert np.array_equal(ctx.maxpool2d_u8(xd, layout, 3, 2, 1).cpu().numpy(),
                              oracle.maxpool_u8(x, layout, 3, 2, 1))
        assert np.array_equal(ctx.global_avgpool_u8(xd, layout, 0.0123, 0, 255).cpu().numpy(),
                              oracle.global_avgpool_u8(x, layout, np.float32(0.0123), 0, 255))
    # channels-last with whole 16-channel groups: the vectorised kernels
    x = rng.integers(0, 256, size=(5, 7, 7, 48), dtype=np.uint8)
    xd = torch.from_numpy(x).to(ctx.device)
    assert np.array_equal(ctx.maxpool2d_u8(xd, 1, 3, 2, 1).cpu().numpy(), oracle.maxpool_u8(x, 1, 3, 2, 1))
    assert np.array_equal(ctx.global_avgpool_u8(xd, 1, 0.0201, 0, 15).cpu().numpy(),
                          oracle.global_avgpool_u8(x, 1, np.float32(0.0201), 0, 15))


def test_contraction_timing_hook(psb, oracle):
    """The measurement hook brackets the tensor-core kernel with events; results are unchanged by it."""
    c = psb.Context(0)
    with pytest.raises(psb.PsbError):
        c.contraction_time()                      # nothing timed yet
    rng = np.random.default_rng(31)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 12, 12, 64, 3, 3, 1, 1)
    c.contraction_timing(True)
    _both(psb, c, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, in_max=15, path=psb.PSB_PATH_TENSOR, want=("q",))
    ms = c.contraction_time()
    assert 0.0 < ms < 50.0
    c.contraction_timing(False)
    c.close()


def test_int8_issue_rate_probe_reports_a_plausible_ceiling(psb, ctx):
    """The measurement aid runs, leaves the device error word clear and reports between a quarter of and
    the full documented rate of 8192 int8 multiply-accumulates per SM clock."""
    mac_clk, tops = ctx.int8_mma_probe(192, 2000)
    assert ctx.device_status() == 0
    assert 2000.0 < mac_clk < 8300.0
    assert tops > 100.0
    with pytest.raises(psb.PsbError):
        ctx.int8_mma_probe(200, 10)      # columns must be a multiple of 16


# ------------------------------------- config 2 in the launch configuration the benchmark times

@pytest.mark.parametrize("log2k", [0, 1, 2, 3, 4])
def test_config2_full_size_codes_only_planar_as_benchmarked(psb, ctx, oracle, log2k):
    """The launch the default benchmark step makes: planar (NCHW) input, only re-quantised codes
    wanted, tensor path (band mode, planar stores), every draw count of the sweep.  Codes against the
    oracle at 4000 sampled outputs (image borders included) and on two whole images."""
    import torch
    from workloads import config2_conv

    c = config2_conv()
    dev = ctx.device
    wt = ctx.sample_weights(torch.from_numpy(c["w"]).to(dev), seed=c["seed"], layer_id=0, level_mask=1 << log2k)
    ctx.set_sample_map(None, log2k)
    q_buf = torch.full((32 * 64 * 56 * 56 + 128,), 0x5A, dtype=torch.uint8, device=dev)
    out = ctx.conv2d(wt, torch.from_numpy(c["x"]).to(dev), psb.PSB_LAYOUT_NCHW, 1, 1,
                     torch.from_numpy(c["scale"]).to(dev), torch.from_numpy(c["bias"]).to(dev), True,
                     c["inv_step"], 0, 15, in_max=15, want=("q",), out={"q": q_buf[64:-64].view(32, 64, 56, 56)})
    assert ctx.device_status() == 0 and ctx.last_path() == psb.PSB_PATH_TENSOR
    full = q_buf.cpu().numpy()
    assert (full[:64] == 0x5A).all() and (full[-64:] == 0x5A).all(), "guard band overwritten"
    q = out["q"].cpu().numpy()
    W, eb, _ = oracle.sample_level(c["w"], c["seed"], 0, log2k)
    g = oracle.geom(c["x"].shape, oracle.NCHW, oracle.U8, c["w"].shape, 1, 1, 1)
    rng = np.random.default_rng(30 + log2k)
    pts = np.stack([rng.integers(0, 32, 4000), rng.integers(0, 64, 4000), rng.integers(0, 56, 4000),
                    rng.integers(0, 56, 4000)], 1)
    pts[:500, 2] = rng.choice([0, 55], 500)
    pts[250:750, 3] = rng.choice([0, 55], 500)
    ref = oracle.conv_acc_points(c["x"], g, {log2k: W}, pts, uniform_log2k=log2k)
    for t in range(4000):
        n, o, oy, ox = pts[t]
        y = oracle.dequant_one(ref[t], c["scale"][o], eb[o], log2k, c["bias"][o], relu=True)
        assert q[n, o, oy, ox] == oracle.requant_one(y, c["inv_step"], 0, 15), (t, pts[t])
    for n in (0, 31):                                   # the first and the last image, every output
        xi = np.ascontiguousarray(c["x"][n:n + 1])
        g1 = oracle.geom(xi.shape, oracle.NCHW, oracle.U8, c["w"].shape, 1, 1, 1)
        acc = oracle.conv_acc(xi, g1, {log2k: W}, uniform_log2k=log2k)
        _, qo = oracle.epilogue(acc, g1, c["scale"], c["bias"], eb, True, c["inv_step"], 0, 15, uniform_log2k=log2k)
        assert np.array_equal(q[n].astype(np.int32), qo[0]), "image %d" % n
    wt.free()


# (N, C, H, W, O, K, pad, layout): codes-only output at k = 32 and 64 needs four digit planes; plain tiles
# (1x1, strided) and band mode (3x3 stride 1), channels-last and planar
@pytest.mark.parametrize("log2k", [5, 6])
@pytest.mark.parametrize("case", [(2, 64, 13, 12, 64, 1, 0, 1), (2, 64, 14, 13, 80, 3, 1, 1), (3, 128, 9, 11, 64, 3, 1, 0),
                                  (2, 256, 9, 9, 128, 1, 0, 1)])
def test_tensor_path_codes_only_four_planes(psb, ctx, oracle, log2k, case):
    N, C, H, W, O, K, pad, layout = case
    rng = np.random.default_rng(abs(hash((case, log2k))) % 2 ** 31)
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, K, K, 1, layout)
    OH, OW = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    res = rng.integers(0, 16, size=(N, O, OH, OW) if layout == 0 else (N, OH, OW, O)).astype(np.uint8)
    for r in (None, res):
        g = _both(psb, ctx, oracle, w, x, layout, 1, 1, pad, [log2k], scale, bias, inv_step=0.5, residual=r,
                  res_scale=0.3 if r is not None else 0.0, in_max=15, path=psb.PSB_PATH_TENSOR, want=("q",))
        assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("exp_bits", [2, 3])
@pytest.mark.parametrize("K", [1, 3])
def test_tensor_path_codes_only_map_one_and_two_planes(psb, ctx, oracle, exp_bits, K):
    """Narrow exponent windows need one or two digit planes; codes only under a per-location map."""
    rng = np.random.default_rng(100 * exp_bits + K)
    N, C, H, W, O = 2, 64, 11, 16, 72
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, K, K, 1, 1)
    levels = [0, 1, 2] if exp_bits == 2 else [0, 2, 3]
    kmap = rng.choice(levels, size=(N, H, W)).astype(np.uint8)
    kmap[0, :5] = levels[1]
    res = rng.integers(0, 16, size=(N, H, W, O)).astype(np.uint8)
    for r in (None, res):
        g = _both(psb, ctx, oracle, w, x, 1, 1, 1, K // 2, levels, scale, bias, kmap=kmap, inv_step=0.5, residual=r,
                  res_scale=0.3 if r is not None else 0.0, exp_bits=exp_bits, in_max=15, path=psb.PSB_PATH_TENSOR,
                  want=("q",))
        assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("norm", [0, 1])
def test_nonfinite_weight_is_flagged_and_leaves_the_other_weights_alone(psb, ctx, oracle, norm):
    """A NaN or Inf raises the error word; every finite weight keeps the integer it would have had with a
    zero in that place (the oracle refuses the filter, so it is given the zero)."""
    import torch

    rng = np.random.default_rng(8 + norm)
    w = rng.normal(0, 0.1, size=(24, 40, 3, 3)).astype(np.float32)
    w[5, 7, 1, 1] = 7.5                      # the largest weight of row 5 sits next to the NaN
    bad = w.copy()
    bad[5, 3, 0, 2] = np.nan
    bad[17, 0, 0, 0] = np.inf
    clean = w.copy()
    clean[5, 3, 0, 2] = 0.0
    clean[17, 0, 0, 0] = 0.0
    wt = ctx.sample_weights(torch.from_numpy(bad).cuda(), seed=3, layer_id=1, level_mask=0b1000, norm=norm)
    Wg, ebg = (v.cpu().numpy() for v in ctx.weights_export(wt, 3))
    assert ctx.device_status() == psb.PSB_ERR_NONFINITE_WEIGHT
    Wo, ebo, _ = oracle.sample_level(clean, 3, 1, 3, norm=norm)
    assert np.array_equal(ebg, ebo) and np.array_equal(Wg.astype(np.int64), Wo)
    wt.free()
    # the allocation-free entry point has no error word: same integers, nothing reported
    wint = torch.zeros(bad.shape, dtype=torch.int32, device=ctx.device)
    eb = torch.zeros(24, dtype=torch.int32, device=ctx.device)
    psb.sample_level_static(torch.from_numpy(bad).cuda(), wint, eb, seed=3, layer_id=1, log2k=3, norm=norm)
    assert np.array_equal(eb.cpu().numpy(), ebo) and np.array_equal(wint.cpu().numpy().astype(np.int64), Wo)
    assert ctx.device_status() == 0


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(psb, oracle):
    """The bounded wait of the kernels: a thread block waits on a barrier nobody arrives at, gives up after
    the bound, raises the error word and returns; the next ordinary call works."""
    c = psb.Context(0)
    c.set_wait_limit(100000)
    c.wait_selftest()
    assert c.device_status() == psb.PSB_ERR_TIMEOUT
    assert c.device_status() == 0
    rng = np.random.default_rng(41)
    w, x, scale, bias = _layer_inputs(rng, 2, 64, 12, 12, 64, 3, 3, 1, 1)
    _both(psb, c, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, in_max=15, path=psb.PSB_PATH_TENSOR)   # short bound kept
    c.set_wait_limit(0)
    _both(psb, c, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, in_max=15, path=psb.PSB_PATH_TENSOR, want=("q",))
    c.close()


def test_activation_beyond_in_max_is_reported(psb, ctx):
    """in_max is a promise; a byte beyond it is reported instead of silently changing the result."""
    import torch

    dev = ctx.device
    w = torch.randn(64, 64, 3, 3, device=dev)
    wt = ctx.sample_weights(w, level_mask=0b1000)
    ctx.set_sample_map(None, 3)
    sc = torch.ones(64, device=dev)
    good = torch.randint(0, 16, (2, 64, 12, 12), dtype=torch.uint8, device=dev)
    bad = good.clone()
    bad[1, 40, 7, 3] = 16
    # planar input: the layout conversion looks at every byte anyway
    ctx.conv2d(wt, good, psb.PSB_LAYOUT_NCHW, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15)
    assert ctx.device_status() == 0
    ctx.conv2d(wt, bad, psb.PSB_LAYOUT_NCHW, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15)
    assert ctx.device_status() == psb.PSB_ERR_RANGE
    # channels-last input goes straight to the copy engine: verified on request
    good_l, bad_l = good.permute(0, 2, 3, 1).contiguous(), bad.permute(0, 2, 3, 1).contiguous()
    ctx.conv2d(wt, bad_l, psb.PSB_LAYOUT_NHWC, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15)
    assert ctx.device_status() == 0
    ctx.set_checks(psb.PSB_CHECK_RANGE)
    for path in (psb.PSB_PATH_TENSOR, psb.PSB_PATH_SHIFT_ADD):
        ctx.conv2d(wt, good_l, psb.PSB_LAYOUT_NHWC, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15, path=path)
        assert ctx.device_status() == 0
        ctx.conv2d(wt, bad_l, psb.PSB_LAYOUT_NHWC, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15, path=path)
        assert ctx.device_status() == psb.PSB_ERR_RANGE
    # signed data: magnitudes
    sg = torch.randint(-15, 16, (2, 12, 12, 64), dtype=torch.int8, device=dev)
    ctx.conv2d(wt, sg, psb.PSB_LAYOUT_NHWC, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15)
    assert ctx.device_status() == 0
    sg[0, 0, 5, 63] = -16
    ctx.conv2d(wt, sg, psb.PSB_LAYOUT_NHWC, 1, 1, sc, sc, True, 1.0, 0, 15, in_max=15)
    assert ctx.device_status() == psb.PSB_ERR_RANGE
    ctx.set_checks(0)
    wt.free()
    # gathered stem (3 input channels): the gather verifies it
    w3 = torch.randn(16, 3, 3, 3, device=dev)
    wt3 = ctx.sample_weights(w3, level_mask=0b1000)
    img = torch.randint(0, 101, (2, 20, 20, 3), dtype=torch.uint8, device=dev)
    sc16 = torch.ones(16, device=dev)
    ctx.conv2d(wt3, img, psb.PSB_LAYOUT_NHWC, 2, 1, sc16, sc16, True, 1.0, 0, 255, in_max=100, path=psb.PSB_PATH_TENSOR)
    assert ctx.device_status() == 0
    img[1, 19, 19, 2] = 101
    ctx.conv2d(wt3, img, psb.PSB_LAYOUT_NHWC, 2, 1, sc16, sc16, True, 1.0, 0, 255, in_max=100, path=psb.PSB_PATH_TENSOR)
    assert ctx.device_status() == psb.PSB_ERR_RANGE
    ctx.set_sample_map(None, 0)
    wt3.free()


# (N, C, H, W, O, K, pad, layout, shortcut dtype or None)
@pytest.mark.parametrize("case", [(2, 64, 13, 12, 64, 1, 0, 1, None), (2, 64, 14, 13, 80, 3, 1, 1, np.uint8),
                                  (3, 128, 9, 11, 64, 3, 1, 0, np.uint8), (2, 256, 9, 9, 128, 1, 0, 1, np.int8)])
@pytest.mark.parametrize("signed_out", [False, True])
def test_tensor_path_codes_only_two_planes_and_signed_codes(psb, ctx, oracle, case, signed_out):
    """A window of eight octaves (exp_bits = 3) needs two digit planes at k = 8; the uniform codes-only output
    stage for it, plain tiles and band mode, unsigned codes from 0 and signed codes with both clamps."""
    N, C, H, W, O, K, pad, layout, res_dt = case
    rng = np.random.default_rng(abs(hash((case[:8], signed_out))) % 2 ** 31)
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, K, K, 1, layout)
    OH, OW = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    res = None
    if res_dt is not None:
        lo, hi = (0, 16) if res_dt == np.uint8 else (-15, 16)
        res = rng.integers(lo, hi, size=(N, O, OH, OW) if layout == 0 else (N, OH, OW, O)).astype(res_dt)
    kw = dict(relu=False, qmin=-15, qmax=15, out_dtype=1) if signed_out else dict(relu=True, qmin=0, qmax=15)
    g = _both(psb, ctx, oracle, w, x, layout, 1, 1, pad, [3], scale, bias, inv_step=0.5, residual=res,
              res_scale=0.3 if res is not None else 0.0, exp_bits=3, in_max=15, path=psb.PSB_PATH_TENSOR, want=("q",), **kw)
    assert g["path"] == psb.PSB_PATH_TENSOR


def test_tensor_path_codes_only_wide_accumulators(psb, ctx, oracle):
    """Large activations against a filter with large row sums: the 32-bit recombination of the output stage
    must not be chosen (the accumulators exceed 2^31), codes still exact."""
    rng = np.random.default_rng(99)
    N, C, H, W, O = 2, 512, 6, 6, 64
    w = rng.normal(0, 1.0, size=(O, C, 3, 3)).astype(np.float32)
    w = np.abs(w) * 0.9 + 0.5                       # same sign, all within one octave of the largest
    x = rng.integers(100, 128, size=(N, H, W, C)).astype(np.uint8)
    scale = np.ones(O, dtype=np.float32)
    bias = rng.normal(0, 0.5, O).astype(np.float32)
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, inv_step=0.008, qmax=255, in_max=127,
              path=psb.PSB_PATH_TENSOR)
    assert np.abs(g["acc"]).max() > 2 ** 31
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, 1, [3], scale, bias, inv_step=0.008, qmax=255, in_max=127,
              path=psb.PSB_PATH_TENSOR, want=("q",))
    assert g["q"].max() > 0


# ------------------------------------------- sampling options: gate below the window, b-bit probabilities

@pytest.mark.parametrize("opts", [dict(underflow=1), dict(prob_bits=4), dict(prob_bits=6), dict(prob_bits=8),
                                  dict(prob_bits=3, underflow=1), dict(prob_bits=4, deterministic=1),
                                  dict(prob_bits=8, underflow=1, deterministic=1), dict(prob_bits=1)])
@pytest.mark.parametrize("shape,groups,norm", [((64, 64, 3, 3), 1, 0), ((96, 1, 3, 3), 96, 1), ((130, 40, 1, 1), 1, 1),
                                                ((16, 3, 7, 7), 1, 0)])
def test_sampler_options_all_levels(psb, ctx, oracle, opts, shape, groups, norm):
    """The Bernoulli gate at the window floor (Sec. 3.1) and probabilities on a grid with packed draws and the
    deterministic variant (Sec. 4.4): integer filters of every level and base exponents against the oracle."""
    import torch

    rng = np.random.default_rng(abs(hash((shape, norm, tuple(sorted(opts.items()))))) % 2 ** 31)
    w = (rng.normal(0, 0.1, size=shape) * 2.0 ** rng.integers(-9, 1, size=shape)).astype(np.float32)
    flat = w.reshape(-1)
    flat[rng.random(flat.size) < 0.05] = 0.0
    flat[:6] = [0.5, -0.25, 1e-41, 3e-9, 0.99999994, -1.9999999]   # powers of two, sub-normal, tiny, p rounding to 1
    for exp_bits in (4, 3, 2):
        wt = ctx.sample_weights(torch.from_numpy(w).cuda(), groups=groups, seed=2 ** 41 + 3, layer_id=4,
                                level_mask=0x7F, exp_bits=exp_bits, norm=norm, **opts)
        for l in range(7):
            Wg, ebg = (v.cpu().numpy() for v in ctx.weights_export(wt, l))
            Wo, ebo = oracle.sample_level_ex(w, 2 ** 41 + 3, 4, l, exp_bits=exp_bits, norm=norm, **opts)[:2]
            assert np.array_equal(ebg, ebo), (exp_bits, l)
            assert np.array_equal(Wg.astype(np.int64), Wo), (shape, norm, exp_bits, l, opts)
        assert ctx.device_status() == 0
        wt.free()


@pytest.mark.parametrize("opts", [dict(), dict(underflow=1), dict(prob_bits=4), dict(prob_bits=5, underflow=1),
                                  dict(prob_bits=8, deterministic=1)])
@pytest.mark.parametrize("shape,norm", [((320, 1280, 1, 1), 0), ((320, 1280, 1, 1), 1), ((256, 192, 3, 3), 1)])
def test_large_layer_sampled_by_its_own_launch(psb, ctx, oracle, opts, shape, norm):
    """A layer large enough that a launch of its own gives every thread four weights (the sampler's vectorised
    loop, otherwise reached through the batched launch of a network only): integer filters of every level against
    the oracle under every option, and the digit planes through a contraction on a few locations."""
    import torch

    rng = np.random.default_rng(abs(hash((shape, norm, tuple(sorted(opts.items()))))) % 2 ** 31)
    w = (rng.normal(0, 0.05, size=shape) * 2.0 ** rng.integers(-7, 1, size=shape)).astype(np.float32)
    flat = w.reshape(-1)
    flat[rng.random(flat.size) < 0.05] = 0.0
    flat[:6] = [0.5, -0.25, 1e-41, 3e-9, 0.99999994, -1.9999999]
    for exp_bits in (4, 3):
        wt = ctx.sample_weights(torch.from_numpy(w).cuda(), seed=2 ** 33 + 9, layer_id=6, level_mask=0x7F,
                                exp_bits=exp_bits, norm=norm, **opts)
        for l in range(7):
            Wg, ebg = (v.cpu().numpy() for v in ctx.weights_export(wt, l))
            Wo, ebo = oracle.sample_level_ex(w, 2 ** 33 + 9, 6, l, exp_bits=exp_bits, norm=norm, **opts)[:2]
            assert np.array_equal(ebg, ebo), (exp_bits, l)
            assert np.array_equal(Wg.astype(np.int64), Wo), (shape, norm, exp_bits, l, opts)
        assert ctx.device_status() == 0
        wt.free()
    O, C, K, _ = shape
    x = rng.integers(0, 16, size=(1, 12, 11, C)).astype(np.uint8)
    scale = rng.uniform(0.5, 1.5, size=O).astype(np.float32)
    bias = rng.normal(0, 0.1, size=O).astype(np.float32)
    g = _both(psb, ctx, oracle, w, x, 1, 1, 1, K // 2, [3], scale, bias, inv_step=0.3, in_max=15, norm=norm,
              path=psb.PSB_PATH_TENSOR, opts=opts or None)
    assert g["path"] == psb.PSB_PATH_TENSOR


@pytest.mark.parametrize("exp_bits,opts", [(3, dict(underflow=1)), (2, dict(underflow=1)), (3, dict(underflow=1, prob_bits=4)),
                                           (4, dict(prob_bits=4))])
@pytest.mark.parametrize("case", [(2, 64, 14, 13, 80, 3, 1, 1), (3, 128, 9, 11, 64, 3, 1, 0), (2, 256, 9, 9, 128, 1, 0, 1),
                                  (2, 3, 21, 21, 32, 7, 3, 1)])
def test_layers_with_sampling_options(psb, ctx, oracle, exp_bits, opts, case):
    """Whole layers under the sampling options, all outputs and codes only: narrow windows with the gate run
    on two digit planes or one."""
    N, C, H, W, O, K, pad, layout = case
    rng = np.random.default_rng(abs(hash((case, exp_bits))) % 2 ** 31)
    w, x, scale, bias = _layer_inputs(rng, N, C, H, W, O, K, K, 1, layout, x_hi=16 if C >= 32 else 256)
    for want in (("q", "f32", "acc"), ("q",)):
        g = _both(psb, ctx, oracle, w, x, layout, 1, 1, pad, [3], scale, bias, inv_step=0.5 if C >= 32 else 0.02,
                  qmax=15 if C >= 32 else 255, exp_bits=exp_bits, in_max=15 if C >= 32 else 0,
                  path=psb.PSB_PATH_TENSOR, want=want, opts=opts)
        assert g["path"] == psb.PSB_PATH_TENSOR


def test_depthwise_and_fc_with_sampling_options(psb, ctx, oracle):
    rng = np.random.default_rng(61)
    C = 48
    w, x, scale, bias = _layer_inputs(rng, 2, C, 12, 10, C, 3, 3, C, 1, x_hi=256)
    _both(psb, ctx, oracle, w, x, 1, C, 1, 1, [4], scale, bias, inv_step=0.03, qmax=255, exp_bits=3, want=("q",),
          opts=dict(underflow=1, prob_bits=4))
    w, x, scale, bias = _layer_inputs(rng, 16, 256, 1, 1, 128, 1, 1, 1, 1)
    _both(psb, ctx, oracle, w, x, 1, 1, 1, 0, [2], scale, bias, inv_step=0.3, qmax=255, exp_bits=3, in_max=15,
          path=psb.PSB_PATH_SHIFT_ADD, opts=dict(underflow=1))


def test_bad_sampling_options_are_refused(psb, ctx):
    import torch

    w = torch.randn(16, 16, 1, 1, device=ctx.device)
    for bad in (dict(prob_bits=9), dict(deterministic=1), dict(underflow=2)):
        with pytest.raises(psb.PsbError) as e:
            ctx.sample_weights(w, level_mask=1, **bad)
        assert e.value.status == psb.PSB_ERR_INVALID_ARG


# ------------------------------------------------------------- attention proposal (Sec. 4.5)

@pytest.mark.parametrize("case", [(3, 7, 7, 2048, np.uint8, 15, 0.21), (2, 5, 9, 37, np.uint8, 255, 0.03),
                                  (2, 4, 4, 96, np.int8, 15, 0.4), (1, 14, 14, 1000, np.uint8, 15, 1.3)])
def test_attention_entropy_and_maps(psb, ctx, oracle, case):
    """Pixelwise entropy of the softmax over channels (fp32 on the device, float64 in the oracle: sums of up to
    2048 terms, so 2e-5 relative + 2e-5 absolute), the threshold at the image mean and the maps of every resolution.
    The threshold decides an integer from a floating-point value: locations whose entropy lies within 1e-4 of the
    mean may fall on either side; everywhere else the maps must be identical."""
    import torch

    N, H, W, C, dt, hi, step = case
    rng = np.random.default_rng(abs(hash(case[:4])) % 2 ** 31)
    lo = 0 if dt == np.uint8 else -hi
    q = rng.integers(lo, hi + 1, size=(N, H, W, C)).astype(dt)
    q[0, 0, 0] = q[0, 0, 0, 0]                   # equal activations: log C
    q[-1, -1, -1] = lo
    q[-1, -1, -1, C // 2] = hi                   # one dominant channel
    h_gpu = ctx.attention_entropy(torch.from_numpy(q).to(ctx.device), step)
    res = [H, 2 * H, 3, 11]
    maps, mean = ctx.attention_maps(h_gpu, 2, 4, res)
    assert ctx.device_status() == 0
    h_ref = oracle.attention_entropy(q, step)
    hg = h_gpu.cpu().numpy()
    assert np.allclose(hg, h_ref, rtol=2e-5, atol=2e-5)
    ref_maps, ref_mean = oracle.attention_maps(h_ref, 2, 4, res)
    assert np.allclose(mean.cpu().numpy(), ref_mean, rtol=2e-5, atol=2e-5)
    sure = np.abs(h_ref - ref_mean[:, None, None]) > 1e-4
    for r in res:
        got = maps[r].cpu().numpy()
        assert got.shape == (N, r, r) and set(np.unique(got)) <= {2, 4}
        ys, xs = (np.arange(r) * H) // r, (np.arange(r) * W) // r
        s = sure[:, ys][:, :, xs]
        assert np.array_equal(got[s], ref_maps[r][s])
        # and the map is what the device's own entropies and mean say
        own = np.where(hg[:, ys][:, :, xs] > mean.cpu().numpy()[:, None, None], 4, 2)
        assert np.array_equal(got, own)
    with pytest.raises(psb.PsbError):
        ctx.attention_maps(h_gpu, 2, 9, res)
