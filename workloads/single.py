"""Single-layer workloads: one fully connected layer and one 3x3 convolution."""
import numpy as np


def _inv_step_from(y_float, qmax, pct=99.9):
    """1/step such that the given percentile of the non-negative part maps to qmax."""
    pos = np.maximum(np.asarray(y_float, dtype=np.float64), 0.0)
    top = float(np.percentile(pos, pct))
    if top <= 0.0:
        top = 1.0
    return np.float32(qmax / top)


def config1_fc(seed=0, batch=16, d_in=256, d_out=128, k=4):
    """FC 256 -> 128, batch 16; N(0, 0.05^2) weights with 5% exact zeros; u8 inputs in
    [0, 15]; bias ~ N(0, 0.01^2); scale 1; 8-bit unsigned output after ReLU."""
    rng = np.random.default_rng(1000 + seed)
    w = rng.normal(0.0, 0.05, size=(d_out, d_in)).astype(np.float32)
    zero = rng.random(size=w.shape) < 0.05
    w[zero] = 0.0
    x = rng.integers(0, 16, size=(batch, d_in), dtype=np.uint8)
    bias = rng.normal(0.0, 0.01, size=d_out).astype(np.float32)
    scale = np.ones(d_out, dtype=np.float32)
    y_float = x.astype(np.float64) @ w.astype(np.float64).T + bias
    return dict(name="fc_256x128_b16", w=w.reshape(d_out, d_in, 1, 1), x=x, bias=bias, scale=scale,
                log2k=int(np.log2(k)), seed=seed, layer_id=0, relu=True,
                inv_step=_inv_step_from(y_float, 255), qmin=0, qmax=255,
                macs=batch * d_in * d_out)


def config2_conv(seed=1, batch=32, c=64, o=64, hw=56, layout="NCHW"):
    """3x3 stride 1 pad 1 conv, 64 -> 64 channels on 56x56, batch 32; He-normal weights;
    ReLU-like u8 activations: half zeros, the rest uniform in [1, 15]."""
    rng = np.random.default_rng(1000 + seed)
    d = c * 9
    w = rng.normal(0.0, np.sqrt(2.0 / d), size=(o, c, 3, 3)).astype(np.float32)
    shape = (batch, c, hw, hw) if layout == "NCHW" else (batch, hw, hw, c)
    x = rng.integers(1, 16, size=shape, dtype=np.uint8)
    x[rng.random(size=shape) < 0.5] = 0
    scale = np.ones(o, dtype=np.float32)
    bias = np.zeros(o, dtype=np.float32)
    # pre-activations are roughly N(0, 2 * E[x^2]); map about +3 sigma to the top code
    ex2 = float(np.mean(x.astype(np.float64) ** 2))
    inv_step = np.float32(15.0 / (3.0 * np.sqrt(2.0 * ex2)))
    return dict(name="conv3x3_64_56_b%d" % batch, w=w, x=x, bias=bias, scale=scale, seed=seed,
                layer_id=0, relu=True, inv_step=inv_step, qmin=0, qmax=15, stride=1, pad=1,
                layout=layout, macs=batch * hw * hw * o * d)
