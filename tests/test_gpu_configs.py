"""The remaining benchmark configurations at their full per-layer sizes, in the launch configuration the
library uses for them; the oracle checks every (b,h) where that is cheap and a sample of (b,h) otherwise."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import assert_attention_close, compare_export, gpu_pipeline, make_inputs, oracle_batch, oracle_thresholds
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
    thr_o = oracle_thresholds(wl_all, K, V, thr, sel, tokens=T0)      # frozen at the prefill
    full = np.zeros((wl.bh, 4), np.float32); full[sel] = thr_o
    ref = oracle_batch(wl_all, K, V, q, ring, nv, pol.cK, pol.cV, thr=full, bh_sel=sel)
    compare_export(cache, ref, sel)
    assert_attention_close(out.cpu().numpy()[sel], ref.X)
    ex = qaq.qaq_cache_export(cache, 1)
    assert (ex["bits"][:, T0:] == 8).all()
    assert qaq.qaq_cache_stats(cache).device_status == 0


def test_c3_layer_generation_step_loop_sampled():
    # one LLaMA-7B-shaped layer at the benchmark's size (8 x 32 (b,h), 4096 tokens): the score window made from the
    # prefill's last queries, quantization with widths by the rules, then the per-step re-quantization in both
    # directions with a second window and compaction; a sample of (b,h) against the oracle at every stage
    wl = synth.scaled(synth.CONFIGS["C3"], layers=1)
    K, V = synth.make_kv(wl)
    q = synth.make_query(wl)
    T, D, W = wl.tokens, wl.head_dim, wl.window
    scale = 1.0 / math.sqrt(D)
    g = torch.Generator().manual_seed(21)
    Qw = (1.5 * torch.randn((wl.bh, W, D), generator=g)).to(torch.float16)
    # room for tiles that move when widths are raised
    cfg = qaq.make_config(wl.batch, wl.heads, D, 2 * T, wl.bits_min, wl.bits_max, W, wl.alpha)
    Kd, Vd, qd = K.cuda(), V.cuda(), q.cuda()
    sel = [0, 101, 255]
    # the window the device makes from the prefill's last queries, against the oracle's own
    ring_d, nvalid_d = qaq.qaq_prefill_window(cfg, Qw.cuda(), Kd, scale)
    ku = K.numpy().view(np.uint16).reshape(wl.bh, T, D); qu = Qw.numpy().view(np.uint16)
    for bh in sel:
        want, nv_want, _ = oracle.prefill_window(qu[bh], ku[bh], scale)
        got = ring_d.reshape(wl.bh, W, T)[bh].cpu().numpy().astype(np.float64)
        assert np.array_equal(nvalid_d.reshape(wl.bh, T)[bh].cpu().numpy(), nv_want)
        assert np.all(np.abs(got - want) <= 1e-6 + 1e-2 * want)
    # quantization with widths by the rules; both sides are fed the same synthetic window
    ring, nvalid = synth.make_score_ring(wl, 0)
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    hyper = HYPER["C2"]
    pol = qaq.qaq_policy_from_hyper(*hyper, T)
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, Kd, Vd, thr, policy=pol, ring=ring.cuda(), nvalid=nvalid.cuda())
    thr_h = np.zeros((wl.bh, 4), np.float32); thr_h[sel] = oracle_thresholds(wl, K, V, thr, sel)
    ref = oracle_batch(wl, K, V, q, ring, nvalid, *oracle.policy(*hyper, T), thr=thr_h, bh_sel=sel)
    compare_export(cache, ref, sel)
    # second window (as if made of later decode rows), looser budgets: most widths go down, some values go up
    ring2, nv2 = synth.make_score_ring(wl, 9)
    hyper2 = (0.004, 0.008, 128.0)
    pol2 = qaq.qaq_policy_from_hyper(*hyper2, T)
    qaq.qaq_requantize(cache, Kd, Vd, thr, policy=pol2, ring=ring2.cuda(), nvalid=nv2.cuda())
    ref2 = oracle_batch(wl, K, V, q, ring2, nv2, *oracle.policy(*hyper2, T), thr=thr_h, bh_sel=sel)
    compare_export(cache, ref2, sel)
    out = qaq.qaq_decode_attention(cache, qd, scale)
    assert_attention_close(out.cpu().numpy()[sel], ref2.X)
    up = sum(int((a.bits > b.bits).sum()) for a, b in zip(ref2.K + ref2.V, ref.K + ref.V))
    down = sum(int((a.bits < b.bits).sum()) for a, b in zip(ref2.K + ref2.V, ref.K + ref.V))
    assert up > 50 and down > 50, (up, down)
    qaq.qaq_cache_compact(cache)
    compare_export(cache, ref2, sel)
    assert qaq.qaq_cache_stats(cache).device_status == 0
