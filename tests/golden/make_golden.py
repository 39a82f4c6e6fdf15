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
    out.append(("gaussian window 8 [2,3,4]", float(O.gaussian_window((8, 8, 8))[2, 3, 4])))
    # squeeze-and-excitation residual block (the SEU-Net variant named in Sec. 1 / Sec. 3; the block is this build's reading)
    g = synth.rng(18)
    zz = np.maximum(g.standard_normal((2, 3, 4, 5, 8)), 0.0)
    rr = np.maximum(g.standard_normal((2, 3, 4, 5, 8)), 0.0)
    W1, b1, W2, b2 = g.standard_normal((2, 8)) * 0.5, g.standard_normal(2) * 0.2 + 0.3, g.standard_normal((8, 2)) * 0.5, g.standard_normal(8) * 0.2
    o, cache = ops.se_block_fwd(zz, rr, W1, b1, W2, b2)
    dz, dr, dW1, db1, dW2, db2 = ops.se_block_bwd(g.standard_normal(zz.shape), cache)
    out += [("se block out sumsq", float((o * o).sum())), ("se block excitation sum", float(cache["e"].sum())),
            ("se block dz sumsq", float((dz * dz).sum())), ("se block dW1 sumsq", float((dW1 * dW1).sum())),
            ("se block dW2 sumsq", float((dW2 * dW2).sum())), ("se block db2 sum", float(db2.sum()))]
    sspec = O.UNetSpec(2, [8, 16], 2, 1, 3, se_ratio=4)
    slay = O.unet_layers(sspec)
    sws = [a.astype(np.float64) for a in synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in slay], 19)]
    sbs = [np.zeros(l.c_out) for l in slay]
    sse = [None if not l.se_cr else (g.standard_normal((l.se_cr, l.c_out)) * 0.4, np.full(l.se_cr, 0.2),
                                     g.standard_normal((l.c_out, l.se_cr)) * 0.4, np.zeros(l.c_out)) for l in slay]
    sloss, sdW, sdB, sp, sdS = O.train_step(sspec, sws, sbs, vol, lab, se=sse)
    out += [("tiny seunet loss", float(sloss)), ("tiny seunet probs sumsq", float((sp * sp).sum())),
            ("tiny seunet dW[0] sumsq", float((sdW[0] * sdW[0]).sum()))]
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_path_oracle.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_golden.py from oracle/ alone (fp64); not values of the paper,\n")
        f.write("# which prints no worked example (network of Sec. 2.2)\n")
        for name, v in entries():
            f.write("%s\t%.17g\n" % (name, v))
    print(path)
