"""Writes tests/golden/tiny_path_oracle.txt: stored results of the CPU oracle on one tiny seeded case.

The paper prints no worked example (it gives topology and widths only), so nothing here is a value of the paper;
the file pins the oracle against drift: tests/test_oracle_golden.py recomputes every entry from the same seeds
and compares.  This script calls only `oracle/` and the seeded input generators.  Run it again only when a change
to the oracle's arithmetic is justified by the paper (Sec. 2.2 for the network, Sec. 3 for the training set-up),
and say so in the commit.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import ops, unet as O                      # noqa: E402
from paper_2006_12575_b200 import synth                # noqa: E402


def entries():
    """(name, value) pairs; every value is a float computed by the oracle in fp64."""
    out = []
    x = synth.normal_bf16((1, 4, 5, 6, 8), 11).astype(np.float64)
    w = synth.kaiming_bf16(27, 16, 8, 27 * 8, 12).astype(np.float64)
    b = synth.rng(13).standard_normal(16)
    y = ops.conv3d_fwd(x, w, b, 3, 1, 1)
    dy = synth.normal_bf16(y.shape, 14).astype(np.float64)
    dx = ops.conv3d_dgrad(dy, w, (4, 5, 6), 3, 1, 1)
    dw, db = ops.conv3d_wgrad(x, dy, 3, 1, 1)
    for name, a in (("conv3 s1 fwd", y), ("conv3 s1 dgrad", dx), ("conv3 s1 wgrad", dw), ("conv3 s1 dbias", db)):
        out += [(name + " sum", float(a.sum())), (name + " sumsq", float((a * a).sum())), (name + " first", float(a.ravel()[0])),
                (name + " last", float(a.ravel()[-1]))]
    y2 = ops.conv3d_fwd(x, w, None, 3, 2, 1)
    out += [("conv3 s2 fwd sum", float(y2.sum())), ("conv3 s2 fwd sumsq", float((y2 * y2).sum()))]
    mu, var, rstd = ops.instnorm_stats(y, 1e-5)
    z = ops.instnorm_relu_fwd(y, mu, rstd)
    out += [("instnorm relu fwd sum", float(z.sum())), ("instnorm relu fwd sumsq", float((z * z).sum()))]
    spec = O.UNetSpec(2, [8, 16], 1, 1, 3)
    lay = O.unet_layers(spec)
    ws = [a.astype(np.float64) for a in synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], 15)]
    bs = [np.zeros(l.c_out) for l in lay]
    vol = synth.bf16_round(synth.blurred_noise((4, 4, 4), 1.0, 16))[None, ..., None].astype(np.float64)
    lab = synth.labels_quartiles((4, 4, 4), 17, 3)[None]
    loss, dW, dB, p = O.train_step(spec, ws, bs, vol, lab)
    out += [("tiny unet loss", float(loss)), ("tiny unet probs sumsq", float((p * p).sum()))]
    for i, g in enumerate(dW):
        out.append((f"tiny unet dW[{i}] sumsq", float((g * g).sum())))
    out.append(("window starts 512/64/0.25 count", float(len(O.window_starts(512, 64, 0.25)))))
    out.append(("gaussian window 8 min", float(O.gaussian_window((8, 8, 8)).min())))
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_path_oracle.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_golden.py from oracle/ alone (fp64); not values of the paper,\n")
        f.write("# which prints no worked example (network of Sec. 2.2)\n")
        for name, v in entries():
            f.write("%s\t%.17g\n" % (name, v))
    print(path)
