"""Bias and spread of a PSB layer's output under the sampling options, from the CPU oracle.

    python oracle/window_stats.py [--seeds 300] [--k 8]

For the 3x3, 64 -> 64 layer of the default benchmark (He-normal filter, activations 0..15, half of them zero) the
real-valued output sum_i x_i W_k[i] 2^e_base / k of 64 output channels at one location is sampled over many
seeds and compared with the float product: relative bias of the mean and relative standard deviation, for
exponent windows of 16, 8 and 4 octaves (exp_bits 4, 3, 2), flushing below the window or with the Bernoulli
gate at its floor (Sec. 3.1), full or 4-bit probabilities (Sec. 4.4).  TEST INFRASTRUCTURE: reads only oracle/ and
workloads/.
"""
import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import psb_oracle as orc  # noqa: E402
from workloads import config2_conv  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seeds", type=int, default=300)
    ap.add_argument("--k", type=int, default=8)
    args = ap.parse_args()
    orc.build()
    c = config2_conv(batch=1)
    w = c["w"].reshape(64, -1)
    x = c["x"][0, :, 20:23, 20:23].reshape(-1).astype(np.float64)      # one 3x3 patch, 576 values
    ref = (w.astype(np.float64) * x).sum(1)
    log2k = int(np.log2(args.k))
    print("options                               planes  rel. bias of the mean   rel. std of one sample   share of weights: window / gate / dropped")
    for exp_bits in (4, 3, 2):
        for underflow in (0, 1):
            for pb in (0, 4):
                outs = np.zeros((args.seeds, 64))
                for s in range(args.seeds):
                    W, eb, _, cls = orc.sample_level_ex(w, s, 0, log2k, exp_bits=exp_bits, underflow=underflow, prob_bits=pb)
                    outs[s] = (W * x).sum(1) * 2.0 ** eb.astype(np.float64) / args.k
                scale = np.abs(ref).mean()
                bias = np.abs(outs.mean(0) - ref).mean() / scale
                std = outs.std(0).mean() / scale
                planes = ((1 << exp_bits) - 1 + log2k + 2 + 6) // 7
                nz = w != 0
                print("exp_bits %d underflow %d prob_bits %d   %d       %.4f                  %.4f                   %.2f / %.2f / %.2f" % (
                    exp_bits, underflow, pb, planes, bias, std, (cls == 1)[nz].mean(), (cls == 2)[nz].mean(), (cls == 0)[nz].mean()))


if __name__ == "__main__":
    main()
