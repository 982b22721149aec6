"""The generation step with the token count kept in device memory (Section 4.2, integration in the text generation
process): one append + decode pair is captured in a CUDA graph once and replayed for every step while the cache grows
across tile boundaries; the decode outputs, the score rows and the final cache are checked against the CPU oracle."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import assert_attention_close, compare_export, u16
from test_gpu_full_extent import prefix
from test_gpu_parity import HYPER

pytestmark = pytest.mark.gpu
CORES = os.cpu_count() or 8


def stream_case(D, T0, n_steps, use_graph, heads=3, batch=2, window=8, alpha=0.02):
    dev = torch.device("cuda")
    T1 = T0 + n_steps
    wl = synth.scaled(synth.CONFIGS["C1"], batch=batch, heads=heads, head_dim=D, tokens=T1, window=window, alpha=alpha)
    BH, W = wl.bh, wl.window
    scale = 1.0 / math.sqrt(D)
    K, V = synth.make_kv(wl, 0, device=dev)
    ring, nv = synth.make_score_ring(wl, 0, device=dev, ragged=True)     # appended tokens have 0..W scores of their own
    hyper = HYPER["C1"]
    pol = qaq.qaq_policy_from_hyper(*hyper, T1)
    cK, cV = oracle.policy(*hyper, T1)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T1, wl.bits_min, wl.bits_max, W, wl.alpha)
    Tq = max(T0, 32)                 # the thresholds are frozen: those of the prefill (of the first 32 tokens without one)
    thr = qaq.qaq_outlier_thresholds(cfg, K[:, :, :Tq], V[:, :, :Tq])
    Kh, Vh = u16(K).reshape(BH, T1, D), u16(V).reshape(BH, T1, D)
    thr_o = np.array([[*oracle.thresholds(Kh[j][:Tq], wl.alpha), *oracle.thresholds(Vh[j][:Tq], wl.alpha)] for j in range(BH)],
                     dtype=np.float32)
    assert np.array_equal(thr.cpu().numpy(), thr_o)
    q0 = synth.make_query(wl, 0, device=dev)
    ref = oracle.run_batch(Kh, Vh, u16(q0).reshape(BH, D), ring.reshape(BH, W, T1).cpu().numpy(), nv.reshape(BH, T1).cpu().numpy(),
                           alpha=wl.alpha, cK=cK, cV=cV, bmin=wl.bits_min, bmax=wl.bits_max, scale=scale, thr=thr_o,
                           run_decode=False, n_threads=CORES, out_cap=T1 * D // 2)

    # the kernels are loaded by one eager step on a scratch cache, so that the capture below records launches only
    warm = qaq.Cache(cfg)
    k1 = torch.zeros((wl.batch, wl.heads, 1, D), dtype=torch.float16, device=dev)
    v1 = torch.zeros_like(k1)
    r1 = torch.zeros((wl.batch, wl.heads, W, 1), dtype=torch.float32, device=dev)
    n1 = torch.zeros((wl.batch, wl.heads, 1), dtype=torch.uint8, device=dev)
    qb = torch.zeros((wl.batch, wl.heads, D), dtype=torch.float16, device=dev)
    out = torch.zeros((BH, D), dtype=torch.float32, device=dev)
    scores = torch.zeros((BH, T1), dtype=torch.float32, device=dev)
    out.fill_(1.0)
    qaq.qaq_stream_begin(warm)
    qaq.qaq_stream_decode(warm, qb, scale, out, scores_out=scores)        # count 0: zeros, nothing read
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0
    qaq.qaq_stream_append(warm, k1, v1, thr, policy=pol, score_col=r1, nvalid=n1)
    qaq.qaq_stream_decode(warm, qb, scale, out, scores_out=scores)
    assert qaq.qaq_stream_end(warm) == 1
    warm.close()

    cache = qaq.Cache(cfg)
    if T0:
        qaq.qaq_quantize_append(cache, K[:, :, :T0], V[:, :, :T0], thr, policy=pol, ring=ring[:, :, :, :T0].contiguous(),
                                nvalid=nv[:, :, :T0].contiguous())
    cache.workspace()
    qaq.qaq_stream_begin(cache)

    def step():
        qaq.qaq_stream_append(cache, k1, v1, thr, policy=pol, score_col=r1, nvalid=n1)
        qaq.qaq_stream_decode(cache, qb, scale, out, scores_out=scores)

    graph = None
    if use_graph:
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):        # recorded, not run: the count is still T0
            step()

    checks = sorted({0, 1, n_steps - 1} | {s for s in range(n_steps) if (T0 + s + 1) % 64 in (0, 1)})
    for s in range(n_steps):
        t = T0 + s
        k1.copy_(K[:, :, t:t + 1]); v1.copy_(V[:, :, t:t + 1])
        r1.copy_(ring[:, :, :, t:t + 1]); n1.copy_(nv[:, :, t:t + 1])
        q = synth.make_query(wl, 0, step=s + 1, device=dev)
        qb.copy_(q)
        if graph is not None:
            graph.replay()
        else:
            step()
        if s in checks:
            got, sc = out.cpu().numpy(), scores.cpu().numpy()
            qh = u16(q).reshape(BH, D)
            for j in range(BH):
                X, S = oracle.decode(qh[j], prefix(ref.K[j], t + 1), prefix(ref.V[j], t + 1), scale)
                assert_attention_close(got[j], X)
                assert_attention_close(sc[j, :t + 1], S)
    assert qaq.qaq_stream_end(cache) == T1
    assert cache.tokens == T1
    compare_export(cache, ref)
    assert qaq.qaq_cache_stats(cache).device_status == 0

    # one step too many: nothing is stored, the count stays, the device status says why
    qaq.qaq_stream_begin(cache)
    if graph is not None:
        graph.replay()
    else:
        step()
    assert qaq.qaq_stream_end(cache) == T1
    compare_export(cache, ref)
    assert qaq.qaq_cache_stats(cache).device_status == 3
    # the host-driven calls carry on from the count that came back
    got = qaq.qaq_decode_attention(cache, qb, scale).cpu().numpy()
    assert np.array_equal(got, out.cpu().numpy())     # same kernel arithmetic, same split: same bits
    cache.close()


@pytest.mark.parametrize("D,T0,n_steps", [(128, 100, 200), (64, 64, 70), (32, 1, 130)])
def test_captured_step_replayed_across_tile_boundaries(D, T0, n_steps):
    stream_case(D, T0, n_steps, use_graph=True)


def test_stream_calls_launched_one_by_one_from_an_empty_cache():
    stream_case(128, 0, 67, use_graph=False)
