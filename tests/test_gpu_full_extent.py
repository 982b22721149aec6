"""The benchmark configurations at the extent they are stated with: every layer of the 7B- and 13B-shaped caches,
the streaming configuration through all of its one-token appends.  Inputs are generated on the device (seeded per
layer) and copied to the host for the CPU oracle, so both sides see the same bits."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import assert_attention_close, compare_export, u16
from test_gpu_parity import HYPER

pytestmark = pytest.mark.gpu
CORES = os.cpu_count() or 8


def layer_case(wl, hyper, layer, bh_sel=None, window_from_attention=False):
    """thresholds -> fused selection + quantization -> decode of one layer on the device against the oracle on all
    (b,h) or on bh_sel.  window_from_attention: the score rows of the checked (b,h) are the oracle's own causal
    softmax rows of `window` queries on the unquantized keys (Section 4.2, attention score prediction), fed to both
    sides; otherwise the synthetic window."""
    dev = torch.device("cuda")
    BH, T, D, W = wl.bh, wl.tokens, wl.head_dim, wl.window
    scale = 1.0 / math.sqrt(D)
    K, V = synth.make_kv(wl, layer, device=dev)
    q = synth.make_query(wl, layer, device=dev)
    ring, nv = synth.make_score_ring(wl, layer, device=dev)
    rows = list(range(BH)) if bh_sel is None else list(bh_sel)
    Kh = u16(K).reshape(BH, T, D)[rows]
    Vh = u16(V).reshape(BH, T, D)[rows]
    if window_from_attention:
        g = torch.Generator().manual_seed(wl.seed + layer + 77)
        Qw = torch.randn((len(rows), W, D), generator=g).to(torch.float16).numpy().view(np.uint16)
        ring4 = ring.reshape(BH, W, T)
        nv2 = nv.reshape(BH, T)
        for j, bh in enumerate(rows):
            w_rows, nv_rows, _ = oracle.prefill_window(Qw[j], Kh[j], scale)
            ring4[bh] = torch.from_numpy(np.asarray(w_rows, dtype=np.float32)).to(dev)
            nv2[bh] = torch.from_numpy(np.asarray(nv_rows, dtype=np.uint8)).to(dev)
    pol = qaq.qaq_policy_from_hyper(*hyper, T)
    cK, cV = oracle.policy(*hyper, T)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T, wl.bits_min, wl.bits_max, W, wl.alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, K, V)
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, K, V, thr, policy=pol, ring=ring, nvalid=nv)
    out = qaq.qaq_decode_attention(cache, q, scale)
    torch.cuda.synchronize()
    ref = oracle.run_batch(Kh, Vh, u16(q).reshape(BH, D)[rows], ring.reshape(BH, W, T)[rows].cpu().numpy(),
                           nv.reshape(BH, T)[rows].cpu().numpy(), alpha=wl.alpha, cK=cK, cV=cV, bmin=wl.bits_min,
                           bmax=wl.bits_max, scale=scale, n_threads=CORES, out_cap=max(1024, T * D // 2), want_scores=False)
    assert np.array_equal(thr.cpu().numpy()[rows], ref.thr), "thresholds differ from the oracle's order statistics"
    compare_export(cache, ref, None if bh_sel is None else rows)
    assert_attention_close(out.cpu().numpy()[rows], ref.X)
    assert qaq.qaq_cache_stats(cache).device_status == 0
    return ref


@pytest.mark.parametrize("layer", range(32))
def test_c3_7b_full_cache_every_layer_all_256_heads(layer):
    # 32 layers x (8 x 32 (b,h), 4096 tokens, head_dim 128), seeded per layer: widths, outlier lists, packed codes
    # bit for bit and the decode output of every (b,h) of every layer
    layer_case(synth.scaled(synth.CONFIGS["C3"], layers=1), HYPER["C2"], layer)


@pytest.mark.parametrize("layer", range(40))
def test_c4_13b_cache_every_layer_8_heads_window_of_64_attention_rows(layer):
    # 40 layers x (4 x 40 (b,h), 8192 tokens), Student-t data with 5 % planted outliers, alpha = 5 %; the widths of
    # the checked (b,h) are selected from attention rows of 64 queries (the oracle's), window 64
    wl = synth.scaled(synth.CONFIGS["C4"], layers=1)
    sel = sorted({(17 * layer + 19 * i) % wl.bh for i in range(8)})
    ref = layer_case(wl, HYPER["C4"], layer, bh_sel=sel, window_from_attention=True)
    if layer == 0:
        assert len({int(b) for r in ref.V for b in np.unique(r.bits)}) >= 3      # the attention rows do spread the widths


def test_c1_tiny_layer_widths_from_attention_rows_of_5_queries():
    layer_case(synth.CONFIGS["C1"], HYPER["C1"], 0, window_from_attention=True)


def prefix(qt, T):
    """The first T tokens of a canonical quantized tensor."""
    no = int(qt.rowptr[T])
    return oracle.QuantTensor(T, qt.D, qt.bits[:T], qt.mn[:T], qt.step[:T], qt.off[:T + 1], qt.stream[:int(qt.off[T])],
                              qt.rowptr[:T + 1], qt.ch[:no], qt.val[:no])


def test_c5_streaming_32768_prefill_then_all_98304_one_token_appends_with_decode_every_step():
    # one 7B-shaped layer (32 heads), prefill of 32768 tokens, then 98304 single-token appends, each followed by
    # packed decode attention on the device.  Thresholds are frozen at the prefill; appended tokens have no score yet
    # (values at bits_max).  The oracle quantizes all 131072 tokens of three heads and checks the decode output at
    # steps 0, 1, 2, every 8192nd and the last (T = 131072), then the whole cache of those heads bit for bit.
    wl = synth.CONFIGS["C5"]
    T0, T1 = wl.tokens, wl.grow_to
    wl_all = synth.scaled(wl, tokens=T1, grow_to=0)
    dev = torch.device("cuda")
    BH, D, W = wl.bh, wl.head_dim, wl.window
    scale = 1.0 / math.sqrt(D)
    K, V = synth.make_kv(wl_all, 0, device=dev)
    ring, nv = synth.make_score_ring(wl_all, 0, device=dev)
    nv[:, :, T0:] = 0
    hyper = HYPER["C2"]
    pol = qaq.qaq_policy_from_hyper(*hyper, T1)          # one policy for the whole run (the caller's choice of T)
    cK, cV = oracle.policy(*hyper, T1)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T1, 2, 8, W, wl.alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, K[:, :, :T0], V[:, :, :T0])
    sel = [0, 13, 31]
    Kh = u16(K).reshape(BH, T1, D)[sel]
    Vh = u16(V).reshape(BH, T1, D)[sel]
    thr_o = np.array([[*oracle.thresholds(Kh[j][:T0], wl.alpha), *oracle.thresholds(Vh[j][:T0], wl.alpha)] for j in range(len(sel))],
                     dtype=np.float32)
    assert np.array_equal(thr.cpu().numpy()[sel], thr_o)
    q0 = synth.make_query(wl_all, 0, device=dev)
    ref = oracle.run_batch(Kh, Vh, u16(q0).reshape(BH, D)[sel], ring.reshape(BH, W, T1)[sel].cpu().numpy(),
                           nv.reshape(BH, T1)[sel].cpu().numpy(), alpha=wl.alpha, cK=cK, cV=cV, bmin=2, bmax=8, scale=scale,
                           thr=thr_o, run_decode=False, n_threads=CORES, out_cap=T1 * D // 2)
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, K[:, :, :T0], V[:, :, :T0], thr, policy=pol, ring=ring[:, :, :, :T0].contiguous(),
                            nvalid=nv[:, :, :T0].contiguous())
    out = torch.empty((BH, D), dtype=torch.float32, device=dev)
    r1 = torch.zeros((wl.batch, wl.heads, W, 1), dtype=torch.float32, device=dev)
    n1 = torch.zeros((wl.batch, wl.heads, 1), dtype=torch.uint8, device=dev)
    n_steps = T1 - T0
    checks = sorted({0, 1, 2, n_steps - 1} | set(range(8192 - 1, n_steps, 8192)))
    worst = 0.0
    for step in range(n_steps):
        t = T0 + step
        qaq.qaq_quantize_append(cache, K[:, :, t:t + 1], V[:, :, t:t + 1], thr, policy=pol, ring=r1, nvalid=n1)
        check = step in checks
        q = synth.make_query(wl_all, 0, step=step + 1, device=dev) if check else q0
        qaq.qaq_decode_attention(cache, q, scale, out=out)
        if check:
            got = out.cpu().numpy()[sel]
            qh = u16(q).reshape(BH, D)[sel]
            want = np.stack([oracle.decode(qh[j], prefix(ref.K[j], t + 1), prefix(ref.V[j], t + 1), scale)[0] for j in range(len(sel))])
            worst = max(worst, assert_attention_close(got, want))
    assert cache.tokens == T1
    compare_export(cache, ref, sel)
    ex = qaq.qaq_cache_export(cache, 1)
    assert (ex["bits"][:, T0:] == 8).all()
    assert qaq.qaq_cache_stats(cache).device_status == 0
