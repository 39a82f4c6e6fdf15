"""CPU oracle for the parameter update (TEST INFRASTRUCTURE, fp64).

The paper trains with "RMSProp ... learning rate of 1e-3" (Sec. 3, training setup) and cites Tieleman & Hinton's
lecture for the method; it gives no other hyper-parameter.  Reading used here: the update of that lecture,

    v <- alpha * v + (1 - alpha) * g^2
    w <- w - lr * g / (sqrt(v) + eps)

without momentum and without centring, with alpha and eps as arguments (callers default to alpha = 0.99,
eps = 1e-8, the defaults of the framework the paper's experiments ran on).  The parameters are kept as a master
copy; the bf16 copy the convolution kernels read is the master copy rounded to nearest-even.

Nothing here is shared with the CUDA library, and the library never imports this package.
"""
from __future__ import annotations

import numpy as np

from .ops import bf16_round


def rmsprop_step(w, g, v, lr=1e-3, alpha=0.99, eps=1e-8):
    """One update of every element.  Returns (w_new, v_new, w_bf16) as float64 arrays; the inputs are not modified."""
    w = np.asarray(w, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    v_new = alpha * v + (1.0 - alpha) * g * g
    w_new = w - lr * g / (np.sqrt(v_new) + eps)
    return w_new, v_new, bf16_round(w_new)
