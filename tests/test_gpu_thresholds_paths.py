"""Every path of qaq_outlier_thresholds (Section 4.2, "Outliers": order statistics at the alpha/2 tails) gives the exact
order statistic: inputs built so that the sample's bracket fails in each possible way."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import u16

pytestmark = pytest.mark.gpu


def check(K, V, wl, alpha):
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, K.shape[2], 2, 8, wl.window, alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, K.cuda(), V.cuda()).cpu().numpy()
    Ku, Vu = u16(K).reshape(wl.bh, K.shape[2], wl.head_dim), u16(V).reshape(wl.bh, K.shape[2], wl.head_dim)
    for bh in range(wl.bh):
        want = np.array([*oracle.thresholds(Ku[bh], alpha), *oracle.thresholds(Vu[bh], alpha)], dtype=np.float32)
        assert np.array_equal(thr[bh], want), (bh, thr[bh], want)


def sampled_tokens(T):
    return [s * T // 64 for s in range(64)]      # the 64 tokens the bracket is taken from


def test_bracket_collapses_and_the_candidate_lists_overflow():
    # the sampled tokens are all zero: the bracket is [0, 0], every non-zero entry is a candidate, the lists overflow
    # and the problem is redone by the exact two-pass select over its data
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=4096)
    K, V = synth.make_kv(wl, 0)
    K[:, :, sampled_tokens(4096)] = 0
    V[:, :, sampled_tokens(4096)] = 0
    check(K, V, wl, wl.alpha)


def test_bracket_too_wide_to_hold_rank_k():
    # the sampled tokens are a hundred times larger than the rest: the bracket lies far outside the bulk and fewer
    # than k+1 entries fall beyond it
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=4096)
    K, V = synth.make_kv(wl, 0)
    K[:, :, sampled_tokens(4096)] *= 100
    V[:, :, sampled_tokens(4096)] *= 100
    check(K, V, wl, wl.alpha)


def test_more_candidates_than_the_select_kernel_keeps_on_chip():
    # alpha = 8 % of 4096 x 128 entries: about 40 thousand candidates per tail, above the 16384 keys held in shared
    # memory but inside the list: rank select over the list in global memory
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=4096)
    K, V = synth.make_kv(wl, 0)
    check(K, V, wl, 0.08)


def test_constant_tensor_and_single_distinct_tail_value():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=1024)
    K, V = synth.make_kv(wl, 0)
    K[:] = 1.5                       # every entry equal: both thresholds are that value, no outliers
    V[:, :, :, ::2] = -2.0           # half of the entries tie at the lower tail
    check(K, V, wl, wl.alpha)


@pytest.mark.parametrize("alpha", [0.3, 0.5, 1.0])
def test_tails_so_heavy_that_every_scan_block_overflows(alpha):
    # a third of the entries (or more) beyond the bracket per tail: every block of the scan finds more candidates
    # than it can hold, while the global list would have room for the count - the holes must send the problem to the
    # exact select over its data
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=2048)
    K, V = synth.make_kv(wl, 0)
    check(K, V, wl, alpha)
