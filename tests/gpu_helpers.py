"""Shared helpers of the GPU parity tests: run the CUDA path through the binding and
the CPU checker on the same seeded inputs, and compare."""
import math

import numpy as np
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

ATOL, RTOL = 2e-3, 1e-2   # attention output: |gpu - ref| <= ATOL + RTOL * |ref|


def u16(t):
    return t.detach().cpu().contiguous().numpy().view(np.uint16)


def make_inputs(wl, layer=0, ragged=False):
    K, V = synth.make_kv(wl, layer)
    q = synth.make_query(wl, layer)
    ring, nv = synth.make_score_ring(wl, layer, ragged=ragged)
    return K, V, q, ring, nv


def oracle_batch(wl, K, V, q, ring, nv, cK, cV, thr=None, bitsK=None, bitsV=None, bh_sel=None, n_threads=8):
    BH, T, D, W = wl.bh, K.shape[2], wl.head_dim, wl.window
    k = u16(K).reshape(BH, T, D); v = u16(V).reshape(BH, T, D); qq = u16(q).reshape(BH, D)
    r = ring.numpy().reshape(BH, W, T); n = nv.numpy().reshape(BH, T)
    if bh_sel is not None:
        k, v, qq, r, n = k[bh_sel], v[bh_sel], qq[bh_sel], r[bh_sel], n[bh_sel]
        if thr is not None: thr = thr[bh_sel]
        if bitsK is not None: bitsK, bitsV = bitsK[bh_sel], bitsV[bh_sel]
    return oracle.run_batch(k, v, qq, r, n, alpha=wl.alpha, cK=cK, cV=cV, bmin=wl.bits_min, bmax=wl.bits_max,
                            scale=1.0 / math.sqrt(D), thr=thr, bitsK=bitsK, bitsV=bitsV, n_threads=n_threads,
                            out_cap=max(1024, T * D // 2))


def oracle_thresholds(wl, K, V, thr_gpu, bh_sel=None, tokens=None):
    """Thresholds computed by the oracle for the chosen (b,h); the device's must equal them bit for bit.  Returns
    the oracle's values (what the oracle is fed with afterwards never comes from the device)."""
    T = K.shape[2] if tokens is None else tokens
    ku = u16(K).reshape(wl.bh, K.shape[2], wl.head_dim)[:, :T]; vu = u16(V).reshape(wl.bh, V.shape[2], wl.head_dim)[:, :T]
    rows = range(wl.bh) if bh_sel is None else bh_sel
    out = np.array([[*oracle.thresholds(ku[bh], wl.alpha), *oracle.thresholds(vu[bh], wl.alpha)] for bh in rows], dtype=np.float32)
    got = thr_gpu.detach().cpu().numpy()[list(rows)]
    assert np.array_equal(got, out), "thresholds differ from the oracle's order statistics"
    return out


def compare_export(cache, ref, bh_sel=None):
    """Bit-exact comparison of the canonical arrays of both tensors with the oracle's."""
    for x, refs in ((0, ref.K), (1, ref.V)):
        ex = qaq.qaq_cache_export(cache, x)
        g = {k: v.cpu().numpy() for k, v in ex.items() if k != "stats"}
        rows = range(len(refs)) if bh_sel is None else bh_sel
        for j, bh in enumerate(rows):
            r = refs[j]
            T = r.T
            assert np.array_equal(g["bits"][bh], r.bits), f"bits tensor {x} bh {bh}"
            assert np.array_equal(g["mn"][bh].view(np.uint32), r.mn.view(np.uint32)), f"min tensor {x} bh {bh}"
            assert np.array_equal(g["step"][bh], r.step), f"step tensor {x} bh {bh}"
            assert np.array_equal(g["off"][bh].astype(np.uint32), r.off), f"off tensor {x} bh {bh}"
            nb = int(r.off[T])
            assert np.array_equal(g["codes"][bh, :nb], r.stream), f"codes tensor {x} bh {bh}"
            assert np.array_equal(g["rowptr"][bh].astype(np.uint32), r.rowptr), f"rowptr tensor {x} bh {bh}"
            no = int(r.rowptr[T])
            assert np.array_equal(g["ch"][bh, :no], r.ch), f"outlier channels tensor {x} bh {bh}"
            assert np.array_equal(g["val"][bh, :no].view(np.uint16), r.val), f"outlier values tensor {x} bh {bh}"


def assert_attention_close(got, ref):
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    bound = ATOL + RTOL * np.abs(ref)
    assert np.all(err <= bound), f"max abs err {err.max():.3e}, worst ratio {(err / bound).max():.3f}"
    return float(err.max())


def gpu_pipeline(wl, K, V, q, ring, nv, policy, bits=None, max_tokens=None, max_outliers=0):
    """thresholds -> (select) -> fused quantize_append -> decode, all through the C ABI."""
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, max_tokens or K.shape[2], wl.bits_min, wl.bits_max, wl.window,
                          wl.alpha, max_outliers)
    Kd, Vd, qd, rd, nd = (t.cuda() for t in (K, V, q, ring, nv))
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    cache = qaq.Cache(cfg)
    if bits is None:
        qaq.qaq_quantize_append(cache, Kd, Vd, thr, policy=policy, ring=rd, nvalid=nd)
    else:
        qaq.qaq_quantize_append(cache, Kd, Vd, thr, bitsK=bits[0].cuda(), bitsV=bits[1].cuda())
    scores = torch.empty((wl.bh, K.shape[2]), dtype=torch.float32, device="cuda")
    out = qaq.qaq_decode_attention(cache, qd, 1.0 / math.sqrt(wl.head_dim), scores_out=scores)
    torch.cuda.synchronize()
    return cfg, cache, thr, out, scores, (Kd, Vd, qd, rd, nd)
