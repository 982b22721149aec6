"""GPU parity of the score window after a prefill (Section 4.2, attention score prediction) against the CPU
oracle: causal softmax rows of the last n queries, newest first, and the rows-per-token counts."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import oracle_thresholds, u16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D,window,tokens", [(128, 32, 1000), (64, 5, 300), (32, 64, 517), (128, 40, 23), (128, 64, 4096), (64, 32, 4500)])
def test_window_rows_match_the_oracle(D, window, tokens):
    # 1000 and 517 tokens: several chunks with a ragged tail; 23 tokens: fewer tokens than window rows; 4096 tokens: the
    # largest sequence the one-pass kernel takes (a cluster of 8 CTAs per (b,h)), with 64 rows; 4500: the two-kernel path
    wl = synth.scaled(synth.CONFIGS["C1"], batch=2, heads=2, head_dim=D, tokens=tokens, window=window, seed=70 + D)
    K, _ = synth.make_kv(wl)
    g = torch.Generator().manual_seed(D + window)
    Q = torch.randn((wl.bh, window, D), generator=g).to(torch.float16)
    scale = 1.0 / math.sqrt(D)
    cfg = qaq.make_config(wl.batch, wl.heads, D, tokens, 2, 8, window, wl.alpha)
    ring, nvalid, qn = qaq.qaq_prefill_window(cfg, Q.cuda(), K.cuda(), scale, want_qnorm2=True)
    ring = ring.cpu().numpy().reshape(wl.bh, window, tokens).astype(np.float64)
    nvalid = nvalid.cpu().numpy().reshape(wl.bh, tokens)
    ku, qu = u16(K).reshape(wl.bh, tokens, D), u16(Q)
    for bh in range(wl.bh):
        want, nv, qn2 = oracle.prefill_window(qu[bh], ku[bh], scale)
        assert np.array_equal(nvalid[bh], nv)
        assert np.all(ring[bh][want == 0] == 0)                           # nothing where a query cannot see
        assert np.all(np.abs(ring[bh] - want) <= 1e-6 + 1e-2 * want)
        assert np.allclose(qn.cpu().numpy()[bh], qn2, rtol=1e-5)
        live = min(window, tokens)
        assert np.allclose(ring[bh][:live].sum(axis=1), 1.0, atol=1e-4)   # the rows of queries that exist


def test_window_feeds_the_width_selection_like_any_ring():
    # the ring made on the device, used for selection on the device, equals selection by the oracle on the oracle's ring
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=700)
    K, V = synth.make_kv(wl)
    D, W, T = wl.head_dim, wl.window, 700
    g = torch.Generator().manual_seed(3)
    Q = (2.0 * torch.randn((wl.bh, W, D), generator=g)).to(torch.float16)
    scale = 1.0 / math.sqrt(D)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T, wl.bits_min, wl.bits_max, W, wl.alpha)
    Kd, Vd = K.cuda(), V.cuda()
    ring, nvalid = qaq.qaq_prefill_window(cfg, Q.cuda(), Kd, scale)
    hyper = (0.002, 0.01, 128.0)
    pol = qaq.qaq_policy_from_hyper(*hyper, T)
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    bK, bV = qaq.qaq_select_bits(cfg, pol, Kd, Vd, ring, nvalid, thr)
    cK, cV = oracle.policy(*hyper, T)
    ku, vu, qu = u16(K).reshape(wl.bh, T, D), u16(V).reshape(wl.bh, T, D), u16(Q)
    thr_h = oracle_thresholds(wl, K, V, thr)
    agree = total = 0
    for bh in range(wl.bh):
        r, nv, _ = oracle.prefill_window(qu[bh], ku[bh], scale)
        wk, wv = oracle.select_bits(ku[bh], vu[bh], thr_h[bh], r.astype(np.float32), nv, cK, cV, wl.bits_min, wl.bits_max)
        assert np.array_equal(bK.cpu().numpy()[bh], wk)                  # keys do not depend on the scores
        got = bV.cpu().numpy()[bh]
        # a score within rounding of a ladder boundary may tip a value width by one; everything else is equal
        assert np.all(np.abs(got.astype(int) - wv.astype(int)) <= 1)
        agree += int((got == wv).sum()); total += T
    assert agree >= 0.995 * total


@pytest.mark.parametrize("n", [1, 7, 1000, 262144])
def test_qnorm2_quantile_equals_the_oracle(n):
    """qaq_qnorm2_quantile (Section 4.1, squared query norm quantile) against the oracle's order statistic, bit for bit:
    ties, negative values, zeros of both signs and NaNs in the list."""
    rng = np.random.default_rng(100 + n)
    v = np.round(rng.chisquare(8, size=n), 2).astype(np.float32)
    if n >= 7:
        v[::5] = -v[::5]
        v[3] = np.nan
        v[4] = 0.0
        v[5] = -0.0
    for frac in (0.1, 0.0, 0.5):
        got = qaq.qaq_qnorm2_quantile(torch.from_numpy(v).cuda(), frac).cpu().numpy()[0]
        want = np.float32(oracle.qnorm2_quantile(v, frac))
        assert got == want, (n, frac, got, want)


def test_policy_from_the_window_queries():
    """The chain a caller runs after a prefill: window rows and per-query squared norms (qaq_prefill_window), their upper
    10 % quantile (qaq_qnorm2_quantile), the policy constants; against the same chain on the oracle."""
    wl = synth.scaled(synth.CONFIGS["C2"], tokens=640, heads=4)
    K, _ = synth.make_kv(wl)
    BH, D, W, T = wl.bh, wl.head_dim, wl.window, wl.tokens
    g = torch.Generator().manual_seed(11)
    Q = torch.randn((BH, W, D), generator=g).to(torch.float16)
    scale = 1.0 / math.sqrt(D)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T, wl.bits_min, wl.bits_max, W, wl.alpha)
    _, _, qn = qaq.qaq_prefill_window(cfg, Q.cuda(), K.cuda(), scale, want_qnorm2=True)
    qd = float(qaq.qaq_qnorm2_quantile(qn, 0.1).cpu()[0])
    qf = (Q.double() * scale) ** 2
    want = oracle.qnorm2_quantile(qf.sum(-1).numpy().astype(np.float32), 0.1)
    assert abs(qd - want) <= 1e-5 * want                                     # binary32 sums in another order
    pd = qaq.qaq_policy_from_hyper(0.002, 0.01, qd, T)
    cK, cV = oracle.policy(0.002, 0.01, want, T)
    assert abs(pd.cK - cK) <= 1e-5 * cK and pd.cV == np.float32(cV)
