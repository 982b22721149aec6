"""The remaining benchmark configurations at their full per-layer sizes, in the launch configuration the
library uses for them; the oracle checks every (b,h) where that is cheap and a sample of (b,h) otherwise."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import assert_attention_close, compare_export, gpu_pipeline, make_inputs, oracle_batch
from test_gpu_parity import HYPER, full_case

pytestmark = pytest.mark.gpu


def test_c2_7b_layer_batch_1_all_heads():
    full_case(synth.CONFIGS["C2"], HYPER["C2"])


def test_c4_13b_shaped_layer_heavy_tails_sampled():
    # 4 x 40 (b,h), 8192 tokens, Student-t data with 5 % planted outliers, window 64, alpha = 5 %
    wl = synth.scaled(synth.CONFIGS["C4"], layers=1)
    full_case(wl, HYPER["C4"], bh_sel=[0, 83, 159])


def test_c5_long_prefill_then_one_token_appends_sampled():
    # 32 heads, prefill 32768 tokens, then single-token appends whose values take bits_max (no score seen yet);
    # thresholds frozen at prefill; decode after the appends against the oracle on a sample of heads
    wl = synth.scaled(synth.CONFIGS["C5"], grow_to=0)
    n_app = 70
    T0, T1 = wl.tokens, wl.tokens + n_app
    wl_all = synth.scaled(wl, tokens=T1)
    K, V, q, ring, nv = make_inputs(wl_all)
    nv[:, :, T0:] = 0
    hyper = HYPER["C2"]
    pol = qaq.qaq_policy_from_hyper(*hyper, T1)
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, T1, 2, 8, wl.window, wl.alpha)
    Kd, Vd, qd, rd, nd = (t.cuda() for t in (K, V, q, ring, nv))
    thr = qaq.qaq_outlier_thresholds(cfg, Kd[:, :, :T0], Vd[:, :, :T0])
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, Kd[:, :, :T0], Vd[:, :, :T0], thr, policy=pol,
                            ring=rd[:, :, :, :T0].contiguous(), nvalid=nd[:, :, :T0].contiguous())
    for t in range(T0, T1):
        qaq.qaq_quantize_append(cache, Kd[:, :, t:t + 1], Vd[:, :, t:t + 1], thr, policy=pol,
                                ring=rd[:, :, :, t:t + 1].contiguous(), nvalid=nd[:, :, t:t + 1].contiguous())
    assert cache.tokens == T1
    out = qaq.qaq_decode_attention(cache, qd, 1.0 / math.sqrt(wl.head_dim))
    torch.cuda.synchronize()
    sel = [0, 13, 31]
    ref = oracle_batch(wl_all, K, V, q, ring, nv, pol.cK, pol.cV, thr=thr.cpu().numpy(), bh_sel=sel)
    compare_export(cache, ref, sel)
    assert_attention_close(out.cpu().numpy()[sel], ref.X)
    ex = qaq.qaq_cache_export(cache, 1)
    assert (ex["bits"][:, T0:] == 8).all()
    assert qaq.qaq_cache_stats(cache).device_status == 0
