"""ctypes front end of the CPU oracle (``psb_oracle.cpp``).

TEST INFRASTRUCTURE ONLY.  The oracle is the slow, plain restatement of the
paper's definitions that the CUDA library is compared against.  Nothing in the
product path may import this module; it shares no code with the CUDA library.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psb_oracle.cpp")
_LIB = os.path.join(_HERE, "libpsb_oracle.so")

NCHW, NHWC = 0, 1
U8, S8 = 0, 1


def build(force=False):
    """Compile the oracle with the host compiler (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


class _Geom(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "layout", "x_dtype", "N", "C", "H", "W", "O", "KH", "KW", "groups", "stride", "pad", "OH", "OW")]


class _Epi(C.Structure):
    _fields_ = [("scale", C.c_void_p), ("bias", C.c_void_p), ("e_base", C.c_void_p),
                ("residual", C.c_void_p), ("residual_dtype", C.c_uint32),
                ("residual_scale", C.c_float), ("relu", C.c_uint32), ("inv_step", C.c_float),
                ("qmin", C.c_int32), ("qmax", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.psbo_decode.argtypes = [C.c_float, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_uint32)]
        _lib.psbo_decode.restype = C.c_int
        _lib.psbo_draw_bit.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32]
        _lib.psbo_draw_bit.restype = C.c_int
        _lib.psbo_dequant_one.argtypes = [C.c_int64, C.c_float, C.c_int32, C.c_uint32, C.c_float,
                                          C.c_int, C.c_int32, C.c_float, C.c_int]
        _lib.psbo_dequant_one.restype = C.c_float
        _lib.psbo_requant_one.argtypes = [C.c_float, C.c_float, C.c_int32, C.c_int32]
        _lib.psbo_requant_one.restype = C.c_int32
        _lib.psbo_sample_level.restype = C.c_int
        _lib.psbo_conv_acc.restype = C.c_int
        _lib.psbo_conv_acc_points.restype = C.c_int
        _lib.psbo_window.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().psbo_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def decode(w):
    """Eq. 5-7: returns (class, s, e, p * 2^23); class 0 = zero, 1 = normal, 2 = non-finite."""
    s, e, m = C.c_int(), C.c_int(), C.c_uint32()
    cls = lib().psbo_decode(C.c_float(float(np.float32(w))), C.byref(s), C.byref(e), C.byref(m))
    return cls, s.value, e.value, m.value


def draw_bit(seed, layer, index, j, p_num):
    return lib().psbo_draw_bit(seed, layer, index, j, p_num)


def sample_level(w, seed, layer, log2k, exp_bits=4, norm=0, counts_in=None):
    """Integer weights of level k = 2**log2k for a filter of shape [O, ...].

    Returns (W int64 of w's shape, e_base int32 [O], counts uint32 of w's shape).
    """
    w = np.ascontiguousarray(w, dtype=np.float32)
    O = w.shape[0]
    D = int(np.prod(w.shape[1:])) if w.ndim > 1 else 1
    W_out = np.zeros(w.shape, dtype=np.int64)
    e_base = np.zeros(O, dtype=np.int32)
    counts = np.zeros(w.shape, dtype=np.uint32)
    cin = None if counts_in is None else np.ascontiguousarray(counts_in, dtype=np.uint32)
    rc = lib().psbo_sample_level(_p(w), C.c_uint32(O), C.c_uint64(D), C.c_uint64(seed),
                                 C.c_uint32(layer), C.c_uint32(exp_bits), C.c_uint32(norm),
                                 C.c_uint32(log2k), _p(cin), _p(W_out), _p(e_base), _p(counts))
    if rc != 0:
        raise ValueError("non-finite weight")
    return W_out, e_base, counts


def sample_level_ex(w, seed, layer, log2k, exp_bits=4, norm=0, underflow=0, prob_bits=0, deterministic=0,
                    counts_in=None):
    """Integer weights of one level with the options of Sec. 3.1 (Bernoulli gate below the window) and
    Sec. 4.4 (b-bit probabilities, packed draws, deterministic variant).

    Returns (W int64, e_base int32 [O], counts uint32, cls uint8: 0 nothing, 1 inside the window, 2 gate).
    """
    w = np.ascontiguousarray(w, dtype=np.float32)
    O = w.shape[0]
    D = int(np.prod(w.shape[1:])) if w.ndim > 1 else 1
    W_out = np.zeros(w.shape, dtype=np.int64)
    e_base = np.zeros(O, dtype=np.int32)
    counts = np.zeros(w.shape, dtype=np.uint32)
    cls = np.zeros(w.shape, dtype=np.uint8)
    opts = np.array([exp_bits, norm, underflow, prob_bits, deterministic], dtype=np.uint32)
    cin = None if counts_in is None else np.ascontiguousarray(counts_in, dtype=np.uint32)
    lib().psbo_sample_level_ex.restype = C.c_int
    rc = lib().psbo_sample_level_ex(_p(w), C.c_uint32(O), C.c_uint64(D), C.c_uint64(seed), C.c_uint32(layer),
                                    _p(opts), C.c_uint32(log2k), _p(cin), _p(W_out), _p(e_base), _p(counts), _p(cls))
    if rc == -1:
        raise ValueError("non-finite weight")
    if rc != 0:
        raise ValueError("bad sampling options")
    return W_out, e_base, counts, cls


def quantise(w, prob_bits):
    """Sec. 4.4: (class, e, p * 2^prob_bits) of a weight after rounding p to the grid."""
    e, pq = C.c_int(), C.c_uint32()
    cls = lib().psbo_quantise(C.c_float(float(np.float32(w))), C.c_uint32(prob_bits), C.byref(e), C.byref(pq))
    return cls, e.value, pq.value


def classify(w, e_base, prob_bits=0, underflow=0):
    """(live, base, sh, thr) of one weight under a window with base exponent e_base."""
    out = np.zeros(4, dtype=np.uint32)
    lib().psbo_classify(C.c_float(float(np.float32(w))), C.c_int32(e_base), C.c_uint32(prob_bits),
                        C.c_uint32(underflow), _p(out))
    return tuple(int(v) for v in out)


def draw_bit_packed(seed, layer, index, j, thr, prob_bits):
    lib().psbo_draw_bit_packed.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
    return lib().psbo_draw_bit_packed(seed, layer, index, j, thr, prob_bits)


def geom(x_shape, layout, x_dtype, w_shape, groups, stride, pad):
    if layout == NCHW:
        N, Cc, H, W = x_shape
    else:
        N, H, W, Cc = x_shape
    O, Cg, KH, KW = w_shape
    assert Cg * groups == Cc and O % groups == 0
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (W + 2 * pad - KW) // stride + 1
    return _Geom(layout, x_dtype, N, Cc, H, W, O, KH, KW, groups, stride, pad, OH, OW)


def out_shape(g):
    return (g.N, g.O, g.OH, g.OW) if g.layout == NCHW else (g.N, g.OH, g.OW, g.O)


def _levels_array(W_levels):
    arr = (C.c_void_p * 7)()
    keep = []
    for lvl, Wk in W_levels.items():
        a = np.ascontiguousarray(Wk, dtype=np.int64)
        keep.append(a)
        arr[lvl] = a.ctypes.data
    return arr, keep


def conv_acc(x, g, W_levels, kmap=None, uniform_log2k=0):
    """Exact int64 accumulators of the whole layer; W_levels maps log2k -> int64 filter."""
    x = np.ascontiguousarray(x)
    arr, keep = _levels_array(W_levels)
    km = None if kmap is None else np.ascontiguousarray(kmap, dtype=np.uint8)
    acc = np.zeros(out_shape(g), dtype=np.int64)
    rc = lib().psbo_conv_acc(_p(x), C.byref(g), arr, _p(km), C.c_uint32(uniform_log2k), _p(acc))
    if rc != 0:
        raise ValueError("level not sampled")
    return acc


def conv_acc_points(x, g, W_levels, pts, kmap=None, uniform_log2k=0):
    """Accumulators at the rows of pts = [[n, o, oy, ox], ...] only."""
    x = np.ascontiguousarray(x)
    arr, keep = _levels_array(W_levels)
    km = None if kmap is None else np.ascontiguousarray(kmap, dtype=np.uint8)
    pts = np.ascontiguousarray(pts, dtype=np.uint32)
    acc = np.zeros(len(pts), dtype=np.int64)
    rc = lib().psbo_conv_acc_points(_p(x), C.byref(g), arr, _p(km), C.c_uint32(uniform_log2k),
                                    _p(pts), C.c_uint64(len(pts)), _p(acc))
    if rc != 0:
        raise ValueError("level not sampled")
    return acc


def epilogue(acc, g, scale, bias, e_base, relu, inv_step, qmin, qmax, residual=None,
             residual_scale=0.0, kmap=None, uniform_log2k=0):
    """Dequantise, add bias and shortcut, ReLU, re-quantise.  Returns (y float32, q int32)."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    e_base = np.ascontiguousarray(e_base, dtype=np.int32)
    res = None
    rdt = 0
    if residual is not None:
        res = np.ascontiguousarray(residual)
        assert res.shape == acc.shape and res.dtype in (np.uint8, np.int8)
        rdt = U8 if res.dtype == np.uint8 else S8
    km = None if kmap is None else np.ascontiguousarray(kmap, dtype=np.uint8)
    ep = _Epi(scale.ctypes.data, bias.ctypes.data, e_base.ctypes.data,
              None if res is None else res.ctypes.data, rdt, residual_scale, int(relu),
              inv_step, qmin, qmax)
    y = np.zeros(acc.shape, dtype=np.float32)
    q = np.zeros(acc.shape, dtype=np.int32)
    lib().psbo_epilogue_apply(_p(acc), C.byref(g), C.byref(ep), _p(km), C.c_uint32(uniform_log2k),
                              _p(y), _p(q))
    return y, q


def dequant_one(acc, scale, e_base, log2k, bias, res_q=None, res_scale=0.0, relu=False):
    return lib().psbo_dequant_one(int(acc), float(np.float32(scale)), int(e_base), int(log2k),
                                  float(np.float32(bias)), 0 if res_q is None else 1,
                                  0 if res_q is None else int(res_q), float(np.float32(res_scale)),
                                  int(relu))


def requant_one(y, inv_step, qmin, qmax):
    return lib().psbo_requant_one(float(np.float32(y)), float(np.float32(inv_step)), qmin, qmax)


def maxpool_u8(x, layout, ksize, stride, pad):
    x = np.ascontiguousarray(x, dtype=np.uint8)
    if layout == NCHW:
        N, Cc, H, W = x.shape
    else:
        N, H, W, Cc = x.shape
    OH = (H + 2 * pad - ksize) // stride + 1
    OW = (W + 2 * pad - ksize) // stride + 1
    out = np.zeros((N, Cc, OH, OW) if layout == NCHW else (N, OH, OW, Cc), dtype=np.uint8)
    lib().psbo_maxpool_u8(_p(x), C.c_uint32(layout), C.c_uint32(N), C.c_uint32(Cc), C.c_uint32(H),
                          C.c_uint32(W), C.c_uint32(ksize), C.c_uint32(stride), C.c_uint32(pad), _p(out))
    return out


def global_avgpool_u8(x, layout, pool_mul, qmin, qmax):
    x = np.ascontiguousarray(x, dtype=np.uint8)
    if layout == NCHW:
        N, Cc, H, W = x.shape
    else:
        N, H, W, Cc = x.shape
    out = np.zeros((N, Cc), dtype=np.uint8)
    lib().psbo_global_avgpool_u8(_p(x), C.c_uint32(layout), C.c_uint32(N), C.c_uint32(Cc),
                                 C.c_uint32(H), C.c_uint32(W), C.c_float(pool_mul), C.c_int32(qmin),
                                 C.c_int32(qmax), _p(out))
    return out


def run_network(layers, net, images, seed, uniform_log2k=3, fc_log2k=None, kmaps=None, levels=None):
    """The oracle's forward pass of a layer list (workloads.nets) on u8 images [n, h, w, 3].

    Returns ({tensor name: integer codes}, logits float32).  kmaps: {resolution: u8 [n, res, res]}.
    """
    fc_log2k = uniform_log2k if fc_log2k is None else fc_log2k
    acts = {"image": np.ascontiguousarray(images)}
    logits = None
    for l in layers:
        x = acts[l["src"]]
        if l["op"] == "maxpool":
            acts[l["dst"]] = maxpool_u8(x, NHWC, l["k"], l["stride"], l["pad"])
            continue
        p = net["params"][l["name"]]
        if l["op"] == "avgpool":
            acts[l["dst"]] = global_avgpool_u8(x, NHWC, p["pool_mul"], p["qmin"], p["qmax"])
            continue
        is_fc = x.ndim == 2
        if is_fc:
            x = x.reshape(x.shape[0], 1, 1, x.shape[1])
        kmap = None if (kmaps is None or is_fc) else np.ascontiguousarray(kmaps[l["hout"]][:x.shape[0]])
        lv = fc_log2k if is_fc else uniform_log2k
        need = sorted(set(int(v) for v in np.unique(kmap))) if kmap is not None else [lv]
        Ws, eb = {}, None
        for lev in need:
            Ws[lev], eb, _ = sample_level(p["w"], seed, p["layer_id"], lev)
        g = geom(x.shape, NHWC, U8 if x.dtype == np.uint8 else S8, p["w"].shape, l["groups"], l["stride"], l["pad"])
        acc = conv_acc(x, g, Ws, kmap=kmap, uniform_log2k=lv)
        res = None if l["residual"] is None else acts[l["residual"]]
        y, q = epilogue(acc, g, p["scale"], p["bias"], eb, l["relu"], p["inv_step"], p["qmin"], p["qmax"],
                        residual=res, residual_scale=p["res_scale"], kmap=kmap, uniform_log2k=lv)
        q = q.astype(np.int8 if p["out_dtype"] == S8 else np.uint8)
        if is_fc:
            q, logits = q.reshape(q.shape[0], -1), y.reshape(y.shape[0], -1)
        acts[l["dst"]] = q
    return acts, logits


# ---- attention proposal (Sec. 4.5, "Computational Attention") ---------------------------------
# Plain numpy in float64, written out from the definitions.

def attention_entropy(codes, step):
    """Pixelwise entropy of the softmax over the channels of a layer's activations a = codes * step
    (channels-last [n, h, w, c]):  h_xy = - sum_c softmax(a_xy)_c * log softmax(a_xy)_c."""
    a = np.asarray(codes, dtype=np.float64) * float(step)
    a = a - a.max(axis=-1, keepdims=True)
    e = np.exp(a)
    sm = e / e.sum(axis=-1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(sm > 0, sm * np.log(sm), 0.0)
    return -t.sum(axis=-1)


def attention_maps(entropy, lo_log2k, hi_log2k, resolutions):
    """Hard threshold at the mean entropy of each image: locations above it get the higher draw count.  The
    mask of the layer's own resolution serves every other resolution by nearest-neighbour sampling:
    location (y, x) of an r x r map reads mask[floor(y * h / r), floor(x * w / r)].
    Returns ({r: uint8 [n, r, r] of log2 k}, mean entropy per image)."""
    h = np.asarray(entropy, dtype=np.float64)
    n, H, W = h.shape
    mean = h.reshape(n, -1).mean(axis=1)
    mask = h > mean[:, None, None]
    out = {}
    for r in resolutions:
        ys = (np.arange(r) * H) // r
        xs = (np.arange(r) * W) // r
        m = mask[:, ys][:, :, xs]
        out[r] = np.where(m, hi_log2k, lo_log2k).astype(np.uint8)
    return out, mean
