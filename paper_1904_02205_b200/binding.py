"""Thin ctypes binding of the C ABI in ``include/psb.h``.

Argument marshalling only: every step of the method runs inside the CUDA
library.  PyTorch is used for device memory and streams.  There is no CPU
fallback: loading fails loudly if the library has not been built, and
``Context`` fails if no B200 is usable.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpsb_b200.so")

PSB_OK = 0
PSB_ERR_INVALID_ARG, PSB_ERR_BAD_K, PSB_ERR_UNSUPPORTED, PSB_ERR_ALLOC = -1, -2, -3, -4
PSB_ERR_CUDA, PSB_ERR_TIMEOUT, PSB_ERR_NONFINITE_WEIGHT, PSB_ERR_RANGE = -5, -6, -7, -8
PSB_CHECK_RANGE = 1
PSB_LAYOUT_NCHW, PSB_LAYOUT_NHWC = 0, 1
PSB_DT_U8, PSB_DT_S8 = 0, 1
PSB_PATH_AUTO, PSB_PATH_SHIFT_ADD, PSB_PATH_TENSOR = 0, 1, 2

EXPORTS = ["psb_create", "psb_destroy", "psb_status_string", "psb_device_status", "psb_sample_weights",
           "psb_weights_export", "psb_weights_free", "psb_set_sample_map", "psb_conv2d", "psb_gemm",
           "psb_last_path", "psb_maxpool2d_u8", "psb_global_avgpool_u8", "psb_sample_level_static",
           "psb_sample_batch_create", "psb_sample_batch_run", "psb_sample_batch_free", "psb_run",
           "psb_launch_count", "psb_int8_mma_probe", "psb_contraction_timing", "psb_contraction_time",
           "psb_set_checks", "psb_set_wait_limit", "psb_wait_selftest", "psb_contraction_times",
           "psb_attention_entropy", "psb_attention_maps"]


class psb_wshape(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("out_ch", "in_ch_per_group", "kh", "kw", "groups")]


class psb_sample_cfg(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("layer_id", C.c_uint32), ("level_mask", C.c_uint32),
                ("exp_bits", C.c_uint32), ("norm", C.c_uint32), ("underflow", C.c_uint32),
                ("prob_bits", C.c_uint32), ("deterministic", C.c_uint32), ("reserved", C.c_uint32)]


class psb_epilogue(C.Structure):
    _fields_ = [("scale_dev", C.c_void_p), ("bias_dev", C.c_void_p), ("residual_dev", C.c_void_p),
                ("residual_scale", C.c_float), ("residual_dtype", C.c_uint32), ("relu", C.c_uint32),
                ("inv_step", C.c_float), ("qmin", C.c_int32), ("qmax", C.c_int32),
                ("out_dtype", C.c_uint32), ("q_out_dev", C.c_void_p), ("f32_out_dev", C.c_void_p),
                ("acc_out_dev", C.c_void_p)]


class psb_conv_desc(C.Structure):
    _fields_ = [("layout", C.c_uint32), ("in_dtype", C.c_uint32), ("in_max", C.c_uint32),
                ("n", C.c_uint32), ("c", C.c_uint32), ("h", C.c_uint32), ("w", C.c_uint32),
                ("stride", C.c_uint32), ("pad", C.c_uint32), ("path", C.c_uint32), ("ep", psb_epilogue)]


class psb_gemm_desc(C.Structure):
    _fields_ = [("in_dtype", C.c_uint32), ("in_max", C.c_uint32), ("batch", C.c_uint32),
                ("in_features", C.c_uint32), ("path", C.c_uint32), ("ep", psb_epilogue)]


class psb_op(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("weights", C.c_void_p), ("x_dev", C.c_void_p), ("map_dev", C.c_void_p),
                ("map_n", C.c_uint32), ("map_oh", C.c_uint32), ("map_ow", C.c_uint32),
                ("uniform_log2k", C.c_uint32), ("conv", psb_conv_desc), ("gemm", psb_gemm_desc),
                ("pool_k", C.c_uint32), ("pool_mul", C.c_float), ("pool_qmin", C.c_int32),
                ("pool_qmax", C.c_int32), ("pool_out_dev", C.c_void_p)]


PSB_OP_CONV2D, PSB_OP_GEMM, PSB_OP_MAXPOOL, PSB_OP_AVGPOOL = 0, 1, 2, 3

_lib = None


def load_library():
    """Load libpsb_b200.so; raises if it is missing (build it with ``build.build()``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("CUDA library %s is missing: run paper_1904_02205_b200.build.build()" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, u32, i32 = C.c_void_p, C.c_uint32, C.c_int32
    lib.psb_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.psb_destroy.argtypes = [vp]
    lib.psb_status_string.argtypes = [i32]
    lib.psb_status_string.restype = C.c_char_p
    lib.psb_device_status.argtypes = [vp, vp]
    lib.psb_sample_weights.argtypes = [vp, vp, C.POINTER(psb_wshape), C.POINTER(psb_sample_cfg),
                                       C.POINTER(vp), vp]
    lib.psb_weights_export.argtypes = [vp, vp, u32, vp, vp, vp]
    lib.psb_weights_free.argtypes = [vp, vp]
    lib.psb_set_sample_map.argtypes = [vp, vp, u32, u32, u32, u32]
    lib.psb_conv2d.argtypes = [vp, vp, vp, C.POINTER(psb_conv_desc), vp]
    lib.psb_gemm.argtypes = [vp, vp, vp, C.POINTER(psb_gemm_desc), vp]
    lib.psb_last_path.argtypes = [vp]
    lib.psb_int8_mma_probe.argtypes = [vp, u32, u32, C.POINTER(C.c_double), C.POINTER(C.c_double), vp]
    lib.psb_contraction_timing.argtypes = [vp, u32]
    lib.psb_contraction_time.argtypes = [vp, C.POINTER(C.c_float)]
    lib.psb_contraction_times.argtypes = [vp, C.POINTER(C.c_float), u32, C.POINTER(u32)]
    lib.psb_set_checks.argtypes = [vp, u32]
    lib.psb_set_wait_limit.argtypes = [vp, C.c_uint64]
    lib.psb_wait_selftest.argtypes = [vp, vp]
    lib.psb_attention_entropy.argtypes = [vp, vp, u32, u32, u32, u32, u32, C.c_float, vp, vp]
    lib.psb_attention_maps.argtypes = [vp, vp, u32, u32, u32, u32, u32, u32, C.POINTER(u32), C.POINTER(vp), vp, vp]
    lib.psb_launch_count.argtypes = []
    lib.psb_launch_count.restype = C.c_uint64
    lib.psb_maxpool2d_u8.argtypes = [vp, vp, u32, u32, u32, u32, u32, u32, u32, u32, vp, vp]
    lib.psb_global_avgpool_u8.argtypes = [vp, vp, u32, u32, u32, u32, u32, C.c_float, i32, i32, vp, vp]
    lib.psb_sample_level_static.argtypes = [vp, C.POINTER(psb_wshape), C.POINTER(psb_sample_cfg), u32, vp, vp, vp]
    lib.psb_sample_batch_create.argtypes = [vp, u32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
    lib.psb_sample_batch_run.argtypes = [vp, vp, C.c_uint64, vp]
    lib.psb_sample_batch_free.argtypes = [vp, vp]
    lib.psb_run.argtypes = [vp, C.POINTER(psb_op), u32, vp]
    for name in EXPORTS:
        if name not in ("psb_status_string", "psb_launch_count"):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


class PsbError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        name = load_library().psb_status_string(status).decode()
        super().__init__("%s failed: %s (%d)" % (where, name, status))


def _check(status, where):
    if status != PSB_OK:
        raise PsbError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


_TORCH_DT = {PSB_DT_U8: torch.uint8, PSB_DT_S8: torch.int8}


def _dt_of(t):
    if t.dtype == torch.uint8:
        return PSB_DT_U8
    if t.dtype == torch.int8:
        return PSB_DT_S8
    raise TypeError("activations must be uint8 or int8")


PSB_STATIC_MAX_OUT_CH = 4096


def sample_level_static(w, wint_out, e_base_out, groups=1, seed=0, layer_id=0, log2k=0, exp_bits=4,
                        norm=0, stream=None):
    """psb_sample_level_static: sample one level into tensors the caller already owns.

    For callers that must not allocate (real-time loops, work next to a graph capture, fixed
    memory budgets): needs no Context and allocates nothing; w is a float32 CUDA tensor
    [out_ch, in_ch/groups, kh, kw], wint_out an int32 CUDA tensor of the same shape, e_base_out
    int32 [out_ch] (either output may be None).  Calls that may overlap on the GPU must be
    serialised by the caller; they share one fixed scratch array inside the library.
    """
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    shape = psb_wshape(w.shape[0], w.shape[1], w.shape[2], w.shape[3], groups)
    cfg = psb_sample_cfg(seed, layer_id, 0, exp_bits, norm, 0, 0, 0, 0)
    with torch.cuda.device(w.device):
        _check(load_library().psb_sample_level_static(_ptr(w), C.byref(shape), C.byref(cfg), log2k,
                                                      _ptr(wint_out), _ptr(e_base_out), _stream(stream)),
               "psb_sample_level_static")


class Weights:
    """Handle of one layer's sampled integer filters (library-owned device memory)."""

    def __init__(self, ctx, handle, shape, level_mask):
        self.ctx, self.handle, self.shape, self.level_mask = ctx, handle, shape, level_mask

    def free(self):
        if self.handle is not None:
            _check(self.ctx.lib.psb_weights_free(self.ctx.handle, self.handle), "psb_weights_free")
            self.handle = None


class Context:
    """One per device and host thread; wraps psb_ctx."""

    def __init__(self, device=0):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the PSB library has no CPU path")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        h = C.c_void_p()
        _check(self.lib.psb_create(C.byref(h), device), "psb_create")
        self.handle = h
        self._kmap = None

    def close(self):
        if self.handle is not None:
            self.lib.psb_destroy(self.handle)
            self.handle = None

    def device_status(self, stream=None):
        return self.lib.psb_device_status(self.handle, _stream(stream))

    def check_device(self, stream=None):
        _check(self.device_status(stream), "psb_device_status")

    def last_path(self):
        return self.lib.psb_last_path(self.handle)

    def set_checks(self, flags):
        """PSB_CHECK_RANGE: verify every input byte against in_max on the device."""
        _check(self.lib.psb_set_checks(self.handle, flags), "psb_set_checks")

    def set_wait_limit(self, sm_clocks):
        """Bound of every device-side wait in SM clocks (0 restores the default)."""
        _check(self.lib.psb_set_wait_limit(self.handle, sm_clocks), "psb_set_wait_limit")

    def wait_selftest(self, stream=None):
        """One small thread block waits on a barrier nobody arrives at; the wait runs out."""
        _check(self.lib.psb_wait_selftest(self.handle, _stream(stream)), "psb_wait_selftest")

    def int8_mma_probe(self, n_cols=192, groups=4000, stream=None):
        """Returns (int8 MAC per clock per SM, tera-operations per second) of bare MMA issue."""
        a, b = C.c_double(0.0), C.c_double(0.0)
        _check(self.lib.psb_int8_mma_probe(self.handle, n_cols, groups, C.byref(a), C.byref(b), _stream(stream)),
               "psb_int8_mma_probe")
        return a.value, b.value

    def contraction_timing(self, enable):
        """Bracket every launch of the contraction kernel with CUDA events (measurement aid)."""
        _check(self.lib.psb_contraction_timing(self.handle, 1 if enable else 0), "psb_contraction_timing")

    def contraction_time(self):
        """Summed device time in milliseconds of the contraction launches made since timing was switched on."""
        ms = C.c_float(0.0)
        _check(self.lib.psb_contraction_time(self.handle, C.byref(ms)), "psb_contraction_time")
        return float(ms.value)

    def contraction_times(self):
        """Device time in milliseconds of each contraction launch made since timing was switched on."""
        buf, n = (C.c_float * 256)(), C.c_uint32(0)
        _check(self.lib.psb_contraction_times(self.handle, buf, 256, C.byref(n)), "psb_contraction_times")
        return [float(buf[i]) for i in range(min(n.value, 256))]

    def launch_count(self):
        """Kernels launched by the library in this process so far."""
        return int(self.lib.psb_launch_count())

    # -- psb_sample_weights --------------------------------------------------
    def sample_weights(self, w, groups=1, seed=0, layer_id=0, level_mask=1, exp_bits=4, norm=0,
                       into=None, stream=None, underflow=0, prob_bits=0, deterministic=0):
        """w: float32 CUDA tensor [out_ch, in_ch/groups, kh, kw] (or [out, in] for a FC layer)."""
        assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
        if w.dim() == 2:
            w = w.view(w.shape[0], w.shape[1], 1, 1)
        shape = psb_wshape(w.shape[0], w.shape[1], w.shape[2], w.shape[3], groups)
        cfg = psb_sample_cfg(seed, layer_id, level_mask, exp_bits, norm, underflow, prob_bits, deterministic, 0)
        h = C.c_void_p(into.handle.value if into is not None else None)
        _check(self.lib.psb_sample_weights(self.handle, _ptr(w), C.byref(shape), C.byref(cfg),
                                           C.byref(h), _stream(stream)), "psb_sample_weights")
        if into is not None:
            return into
        return Weights(self, h, tuple(w.shape) + (groups,), level_mask)

    def weights_export(self, weights, log2k, stream=None):
        O, Cg, KH, KW, _ = weights.shape
        wint = torch.empty((O, Cg, KH, KW), dtype=torch.int32, device=self.device)
        e_base = torch.empty((O,), dtype=torch.int32, device=self.device)
        _check(self.lib.psb_weights_export(self.handle, weights.handle, log2k, _ptr(wint), _ptr(e_base),
                                           _stream(stream)), "psb_weights_export")
        return wint, e_base

    # -- psb_set_sample_map --------------------------------------------------
    def set_sample_map(self, log2k_map=None, uniform_log2k=0):
        """log2k_map: uint8 CUDA tensor [n, oh, ow] (kept alive by the context) or None."""
        if log2k_map is None:
            _check(self.lib.psb_set_sample_map(self.handle, None, 0, 0, 0, uniform_log2k),
                   "psb_set_sample_map")
            self._kmap = None
        else:
            assert log2k_map.is_cuda and log2k_map.dtype == torch.uint8 and log2k_map.is_contiguous()
            n, oh, ow = log2k_map.shape
            _check(self.lib.psb_set_sample_map(self.handle, _ptr(log2k_map), n, oh, ow, 0),
                   "psb_set_sample_map")
            self._kmap = log2k_map

    # -- psb_conv2d / psb_gemm ----------------------------------------------
    def _epilogue(self, out_shape, scale, bias, relu, inv_step, qmin, qmax, out_dtype, residual,
                  residual_scale, want, out):
        out = dict(out or {})
        if "q" in want and "q" not in out:
            out["q"] = torch.empty(out_shape, dtype=_TORCH_DT[out_dtype], device=self.device)
        if "f32" in want and "f32" not in out:
            out["f32"] = torch.empty(out_shape, dtype=torch.float32, device=self.device)
        if "acc" in want and "acc" not in out:
            out["acc"] = torch.empty(out_shape, dtype=torch.int64, device=self.device)
        ep = psb_epilogue()
        ep.scale_dev, ep.bias_dev = scale.data_ptr(), bias.data_ptr()
        ep.residual_dev = None if residual is None else residual.data_ptr()
        ep.residual_scale = float(residual_scale)
        ep.residual_dtype = PSB_DT_U8 if residual is None else _dt_of(residual)
        ep.relu, ep.inv_step, ep.qmin, ep.qmax, ep.out_dtype = int(relu), float(inv_step), qmin, qmax, out_dtype
        ep.q_out_dev = out["q"].data_ptr() if "q" in out else None
        ep.f32_out_dev = out["f32"].data_ptr() if "f32" in out else None
        ep.acc_out_dev = out["acc"].data_ptr() if "acc" in out else None
        return ep, out

    def conv2d(self, weights, x, layout, stride, pad, scale, bias, relu, inv_step, qmin, qmax,
               out_dtype=PSB_DT_U8, residual=None, residual_scale=0.0, in_max=0, path=PSB_PATH_AUTO,
               want=("q",), out=None, stream=None):
        """x: uint8/int8 CUDA tensor, [n,c,h,w] (NCHW) or [n,h,w,c] (NHWC).  Returns a dict with
        the requested outputs among 'q', 'f32', 'acc', laid out like x."""
        assert x.is_cuda and x.is_contiguous()
        O, Cg, KH, KW, groups = weights.shape
        if layout == PSB_LAYOUT_NCHW:
            n, c, h, w = x.shape
        else:
            n, h, w, c = x.shape
        oh, ow = (h + 2 * pad - KH) // stride + 1, (w + 2 * pad - KW) // stride + 1
        oshape = (n, O, oh, ow) if layout == PSB_LAYOUT_NCHW else (n, oh, ow, O)
        ep, out = self._epilogue(oshape, scale, bias, relu, inv_step, qmin, qmax, out_dtype, residual,
                                 residual_scale, want, out)
        d = psb_conv_desc(layout, _dt_of(x), in_max, n, c, h, w, stride, pad, path, ep)
        _check(self.lib.psb_conv2d(self.handle, weights.handle, _ptr(x), C.byref(d), _stream(stream)),
               "psb_conv2d")
        return out

    def gemm(self, weights, x, scale, bias, relu, inv_step, qmin, qmax, out_dtype=PSB_DT_U8,
             residual=None, residual_scale=0.0, in_max=0, path=PSB_PATH_AUTO, want=("q",), out=None,
             stream=None):
        """x: uint8/int8 CUDA tensor [batch, in_features]; outputs are [batch, out]."""
        assert x.is_cuda and x.is_contiguous() and x.dim() == 2
        batch, fin = x.shape
        ep, out = self._epilogue((batch, weights.shape[0]), scale, bias, relu, inv_step, qmin, qmax,
                                 out_dtype, residual, residual_scale, want, out)
        d = psb_gemm_desc(_dt_of(x), in_max, batch, fin, path, ep)
        _check(self.lib.psb_gemm(self.handle, weights.handle, _ptr(x), C.byref(d), _stream(stream)),
               "psb_gemm")
        return out

    # -- attention proposal (Sec. 4.5) -----------------------------------------
    def attention_entropy(self, act, step, out=None, stream=None):
        """act: uint8/int8 CUDA tensor [n, h, w, c] of codes; returns float32 [n, h, w]."""
        assert act.is_cuda and act.is_contiguous() and act.dim() == 4
        n, h, w, c = act.shape
        if out is None:
            out = torch.empty((n, h, w), dtype=torch.float32, device=self.device)
        _check(self.lib.psb_attention_entropy(self.handle, _ptr(act), _dt_of(act), n, h, w, c, float(step), _ptr(out),
                                              _stream(stream)), "psb_attention_entropy")
        return out

    def attention_maps(self, entropy, lo_log2k, hi_log2k, resolutions, out=None, stream=None):
        """entropy: float32 CUDA tensor [n, h, w]; returns ({res: uint8 [n, res, res]}, mean float32 [n])."""
        n, h, w = entropy.shape
        res = list(resolutions)
        maps = out or {r: torch.empty((n, r, r), dtype=torch.uint8, device=self.device) for r in res}
        mean = torch.empty((n,), dtype=torch.float32, device=self.device)
        ra = (C.c_uint32 * len(res))(*res)
        pa = (C.c_void_p * len(res))(*[maps[r].data_ptr() for r in res])
        _check(self.lib.psb_attention_maps(self.handle, _ptr(entropy), n, h, w, lo_log2k, hi_log2k, len(res), ra, pa,
                                           _ptr(mean), _stream(stream)), "psb_attention_maps")
        return maps, mean

    # -- whole networks -------------------------------------------------------
    def sample_batch_create(self, filters, weights):
        """filters: float32 CUDA tensors; weights: the Weights handles sampled from them before."""
        n = len(filters)
        wp = (C.c_void_p * n)(*[f.data_ptr() for f in filters])
        hp = (C.c_void_p * n)(*[w.handle.value for w in weights])
        b = C.c_void_p()
        _check(self.lib.psb_sample_batch_create(self.handle, n, wp, hp, C.byref(b)), "psb_sample_batch_create")
        return b

    def sample_batch_run(self, batch, seed, stream=None):
        _check(self.lib.psb_sample_batch_run(self.handle, batch, seed, _stream(stream)), "psb_sample_batch_run")

    def sample_batch_free(self, batch):
        _check(self.lib.psb_sample_batch_free(self.handle, batch), "psb_sample_batch_free")

    def run(self, ops, n_ops, stream=None):
        """ops: ctypes array of psb_op."""
        _check(self.lib.psb_run(self.handle, ops, n_ops, _stream(stream)), "psb_run")

    # -- glue ----------------------------------------------------------------
    def maxpool2d_u8(self, x, layout, k, stride, pad, out=None, stream=None):
        if layout == PSB_LAYOUT_NCHW:
            n, c, h, w = x.shape
        else:
            n, h, w, c = x.shape
        oh, ow = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
        if out is None:
            out = torch.empty((n, c, oh, ow) if layout == PSB_LAYOUT_NCHW else (n, oh, ow, c),
                              dtype=torch.uint8, device=self.device)
        _check(self.lib.psb_maxpool2d_u8(self.handle, _ptr(x), layout, n, c, h, w, k, stride, pad,
                                         _ptr(out), _stream(stream)), "psb_maxpool2d_u8")
        return out

    def global_avgpool_u8(self, x, layout, pool_mul, qmin, qmax, out=None, stream=None):
        if layout == PSB_LAYOUT_NCHW:
            n, c, h, w = x.shape
        else:
            n, h, w, c = x.shape
        if out is None:
            out = torch.empty((n, c), dtype=torch.uint8, device=self.device)
        _check(self.lib.psb_global_avgpool_u8(self.handle, _ptr(x), layout, n, c, h, w, float(pool_mul),
                                              qmin, qmax, _ptr(out), _stream(stream)),
               "psb_global_avgpool_u8")
        return out
