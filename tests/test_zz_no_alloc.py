"""The allocation-free decode entry point against the regular one.

`qaq_decode_attention_static` is for callers that cannot get device memory when they call
(all memory handed out at start-up, or no tolerance for the stalls an allocation can cause):
its split partials live in a fixed device array inside the library.  Here it is called twice
in a row through the C ABI, on two different caches so that the second call finds the first
call's leftovers in the shared array, and each result must equal what `qaq_decode_attention`
(caller-supplied workspace) returns, within the attention tolerance used by the parity tests.
This file is named so that it is collected last.
"""
import math

import numpy as np
import pytest
import torch

from paper_2403_04643_b200 import qaq, synth

pytestmark = pytest.mark.gpu

ATOL, RTOL = 2e-3, 1e-2


def _filled_cache(wl, hyper):
    K, V = synth.make_kv(wl)
    ring, nv = synth.make_score_ring(wl)
    T = wl.tokens
    pol = qaq.qaq_policy_from_hyper(*hyper, T)
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, T, wl.bits_min, wl.bits_max, wl.window, wl.alpha)
    Kd, Vd, rd, nd = (t.cuda() for t in (K, V, ring, nv))
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    cache = qaq.Cache(cfg)
    qaq.qaq_quantize_append(cache, Kd, Vd, thr, policy=pol, ring=rd, nvalid=nd)
    return cache


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    cases = [
        (synth.scaled(synth.CONFIGS["C2"], heads=4, tokens=1500), (0.002, 0.01, 128.0)),   # many splits
        (synth.scaled(synth.CONFIGS["C1"], batch=3, heads=5, tokens=333, seed=21), (0.006, 0.03, 64.0)),
    ]
    caches = [(wl, _filled_cache(wl, hy)) for wl, hy in cases]
    for call in range(2):                       # two calls in a row, the second over the first one's leftovers
        wl, cache = caches[call]
        q = synth.make_query(wl, step=call).cuda()
        scale = 1.0 / math.sqrt(wl.head_dim)
        want = qaq.qaq_decode_attention(cache, q, scale).cpu().numpy()
        out = torch.full((wl.bh, wl.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        qaq.qaq_decode_attention_static(cache, q, scale, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got - want) <= ATOL + RTOL * np.abs(want)), np.abs(got - want).max()
        # both entry points run the same kernels with the same split, and every sum in them is either an exact
        # integer sum or taken in a fixed order: the results are the same bit for bit
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # and once more on the first cache, after the other shape has used the array
    wl, cache = caches[0]
    q = synth.make_query(wl, step=7).cuda()
    want = qaq.qaq_decode_attention(cache, q, 1.0 / math.sqrt(wl.head_dim)).cpu().numpy()
    out = torch.empty((wl.bh, wl.head_dim), dtype=torch.float32, device="cuda")
    qaq.qaq_decode_attention_static(cache, q, 1.0 / math.sqrt(wl.head_dim), out)
    assert np.all(np.abs(out.cpu().numpy() - want) <= ATOL + RTOL * np.abs(want))


def _one_tile_cache(B, H, D=128, T=64):
    cfg = qaq.make_config(B, H, D, T, 2, 8, 1, 0.0)
    cache = qaq.Cache(cfg)
    K = torch.zeros((B, H, T, D), dtype=torch.float16, device="cuda")
    thr = torch.tensor([[-1.0, 1.0, -1.0, 1.0]], device="cuda").repeat(B * H, 1).contiguous()
    bits = torch.full((B * H, T), 2, dtype=torch.uint8, device="cuda")
    qaq.qaq_quantize_append(cache, K, K, thr, bitsK=bits, bitsV=bits)
    return cache


def test_static_scratch_limit_is_exact_and_a_warm_call_takes_no_device_memory():
    # one tile per (b,h): the partials take (b,h) x (2 x 131 + 2) floats, so 3971 (b,h) fit the 4 MiB and 3972 do not
    D = 128
    fits, too_large = _one_tile_cache(11, 361), _one_tile_cache(12, 331)
    for cache, bh, ok in ((fits, 3971, True), (too_large, 3972, False)):
        q = torch.zeros((bh, D), dtype=torch.float16, device="cuda")
        out = torch.empty((bh, D), dtype=torch.float32, device="cuda")
        if ok:
            qaq.qaq_decode_attention_static(cache, q, 1.0, out)          # first call on this device: symbol look-up, module load
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            qaq.qaq_decode_attention_static(cache, q, 1.0, out)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before
        else:
            with pytest.raises(qaq.QaqError) as e:
                qaq.qaq_decode_attention_static(cache, q, 1.0, out)
            assert e.value.code == 5


def test_static_scratch_rejects_shapes_beyond_its_limit():
    # 8320 (b,h) of one tile each: 8320 CTAs x 2 partials x 131 floats do not fit the 4 MiB built in: refused on the host, nothing launched
    B, H, D, T = 128, 65, 128, 64
    cfg = qaq.make_config(B, H, D, T, 2, 8, 1, 0.0)
    cache = qaq.Cache(cfg)
    K = torch.zeros((B, H, T, D), dtype=torch.float16, device="cuda")
    thr = torch.tensor([[-1.0, 1.0, -1.0, 1.0]], device="cuda").repeat(B * H, 1).contiguous()
    bits = torch.full((B * H, T), 2, dtype=torch.uint8, device="cuda")
    qaq.qaq_quantize_append(cache, K, K, thr, bitsK=bits, bitsV=bits)
    q = torch.zeros((B * H, D), dtype=torch.float16, device="cuda")
    out = torch.empty((B * H, D), dtype=torch.float32, device="cuda")
    with pytest.raises(qaq.QaqError) as e:
        qaq.qaq_decode_attention_static(cache, q, 1.0, out)
    assert e.value.code == 5
    qaq.qaq_decode_attention(cache, q, 1.0, out)      # the regular entry point still serves this shape
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0
