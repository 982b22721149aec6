"""Choice of the paper's two hyper-parameters for a synthetic cache.

The paper leaves sigmaS_max and sigmaX_max (Section 4.1) as hyper-parameters.  For the
synthetic workloads they are found once per configuration by bisection on the mean
selected width (keys ~4 bits, values ~3 bits by default), using the library's own
selection kernel; only scalar bookkeeping happens here.
"""
from __future__ import annotations

import math

from . import qaq


def _mean_bits(cfg, pol, K, V, ring, nvalid, thr):
    bK, bV = qaq.qaq_select_bits(cfg, pol, K, V, ring, nvalid, thr)
    return float(bK.float().mean()), float(bV.float().mean())


def calibrate(cfg, K, V, ring, nvalid, thr, T, qnorm2, target_k=4.0, target_v=3.0, iters=24):
    """Returns (sigmaS_max, sigmaX_max, policy) whose mean widths on this layer are close to the targets."""
    lo_s, hi_s, lo_x, hi_x = -12.0, 2.0, -12.0, 4.0   # log10 brackets
    for _ in range(iters):
        ms, mx = 0.5 * (lo_s + hi_s), 0.5 * (lo_x + hi_x)
        pol = qaq.qaq_policy_from_hyper(10.0 ** ms, 10.0 ** mx, qnorm2, T)
        mk, mv = _mean_bits(cfg, pol, K, V, ring, nvalid, thr)
        # a larger error budget gives fewer bits
        if mk > target_k: lo_s = ms
        else: hi_s = ms
        if mv > target_v: lo_x = mx
        else: hi_x = mx
    sS, sX = 10.0 ** (0.5 * (lo_s + hi_s)), 10.0 ** (0.5 * (lo_x + hi_x))
    return sS, sX, qaq.qaq_policy_from_hyper(sS, sX, qnorm2, T)
