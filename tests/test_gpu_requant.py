"""GPU parity of the in-place further quantization to lower widths (Section 4.2, integration in the
generation process) against the CPU oracle: widths, scales, byte offsets and packed codes bit for bit,
attention over the lowered cache within the usual tolerance."""
import math
from types import SimpleNamespace

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import assert_attention_close, compare_export, gpu_pipeline, make_inputs, oracle_batch, oracle_thresholds, u16

pytestmark = pytest.mark.gpu

HYPER = (0.002, 0.01, 128.0)        # mixed widths on the C2-shaped synthetic cache
LOOSER = (0.02, 0.05, 128.0)        # larger variance budgets: lower widths


def _decode_ref(wl, q, qk, qv):
    qq = u16(q).reshape(wl.bh, wl.head_dim)
    return np.stack([oracle.decode(qq[bh], qk[bh], qv[bh], 1.0 / math.sqrt(wl.head_dim))[0] for bh in range(wl.bh)])


def test_widths_recomputed_by_the_rules_and_lowered_in_place():
    # 1000 tokens = 15 full tiles + an open tile of 40; second window and looser budgets for the second selection
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=1000)
    K, V, q, ring, nv = make_inputs(wl, ragged=True)
    T = K.shape[2]
    polA = qaq.qaq_policy_from_hyper(*HYPER, T)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, polA)
    ref = oracle_batch(wl, K, V, q, ring, nv, *oracle.policy(*HYPER, T))
    compare_export(cache, ref)

    ring2, nv2 = synth.make_score_ring(wl, 7, ragged=True)
    polB = qaq.qaq_policy_from_hyper(*LOOSER, T)
    cKb, cVb = oracle.policy(*LOOSER, T)
    qaq.qaq_requantize_down(cache, policy=polB, ring=ring2.cuda(), nvalid=nv2.cuda())
    r2 = ring2.numpy().reshape(wl.bh, wl.window, T); n2 = nv2.numpy().reshape(wl.bh, T)
    qk, qv = [], []
    lowered = kept = 0
    for bh in range(wl.bh):
        bk = oracle.reselect_bits(ref.K[bh], False, None, None, cKb, wl.bits_min, wl.bits_max)
        bv = oracle.reselect_bits(ref.V[bh], True, r2[bh], n2[bh], cVb, wl.bits_min, wl.bits_max)
        qk.append(oracle.requantize_down(ref.K[bh], bk)); qv.append(oracle.requantize_down(ref.V[bh], bv))
        for a, b in ((qk[-1], ref.K[bh]), (qv[-1], ref.V[bh])):
            lowered += int((a.bits < b.bits).sum()); kept += int((a.bits == b.bits).sum())
    assert lowered > 100 and kept > 100
    compare_export(cache, SimpleNamespace(K=qk, V=qv))
    out2 = qaq.qaq_decode_attention(cache, dev[2], 1.0 / math.sqrt(wl.head_dim))
    assert_attention_close(out2.cpu().numpy(), _decode_ref(wl, q, qk, qv))
    st = qaq.qaq_cache_stats(cache)
    assert st.device_status == 0
    assert st.code_bytes[0] == sum(int(t.off[T]) for t in qk) and st.code_bytes[1] == sum(int(t.off[T]) for t in qv)
    # a second pass with the same inputs changes nothing
    qaq.qaq_requantize_down(cache, policy=polB, ring=ring2.cuda(), nvalid=nv2.cuda())
    compare_export(cache, SimpleNamespace(K=qk, V=qv))


@pytest.mark.parametrize("D", [32, 64, 128])
def test_given_widths_then_appends_continue_behind_the_shrunk_open_tile(D):
    wl = synth.scaled(synth.CONFIGS["C1"], batch=2, heads=2, head_dim=D, tokens=150, seed=40 + D)
    K, V, q, ring, nv = make_inputs(wl)
    first, T = 100, 150                                   # 100 = one full tile + an open tile of 36
    rng = np.random.default_rng(D)
    b0 = rng.integers(3, 9, (2, wl.bh, T)).astype(np.uint8)       # widths at quantization time
    req = rng.integers(0, 10, (2, wl.bh, first)).astype(np.uint8)  # requested later (0 counts as 1, 9 lowers nothing)
    cfg = qaq.make_config(wl.batch, wl.heads, D, T, wl.bits_min, wl.bits_max, wl.window, wl.alpha)
    Kd, Vd = K.cuda(), V.cuda()
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    cache = qaq.Cache(cfg)
    tb = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    qaq.qaq_quantize_append(cache, Kd[:, :, :first], Vd[:, :, :first], thr, bitsK=tb(b0[0][:, :first]), bitsV=tb(b0[1][:, :first]))
    qaq.qaq_requantize_down(cache, bitsK=tb(req[0]), bitsV=tb(req[1]))
    qaq.qaq_quantize_append(cache, Kd[:, :, first:], Vd[:, :, first:], thr, bitsK=tb(b0[0][:, first:]), bitsV=tb(b0[1][:, first:]))
    # expected: every token quantized directly at its final width (the nesting property pinned on the CPU side)
    final = b0.copy()
    final[:, :, :first] = np.minimum(b0[:, :, :first], np.maximum(req, 1))
    thr_h = oracle_thresholds(wl, K, V, thr)
    ku, vu = u16(K).reshape(wl.bh, T, D), u16(V).reshape(wl.bh, T, D)
    qk = [oracle.quantize(ku[bh], thr_h[bh, 0], thr_h[bh, 1], final[0, bh]) for bh in range(wl.bh)]
    qv = [oracle.quantize(vu[bh], thr_h[bh, 2], thr_h[bh, 3], final[1, bh]) for bh in range(wl.bh)]
    compare_export(cache, SimpleNamespace(K=qk, V=qv))
    out = qaq.qaq_decode_attention(cache, q.cuda(), 1.0 / math.sqrt(D))
    assert_attention_close(out.cpu().numpy(), _decode_ref(wl, q, qk, qv))
    assert qaq.qaq_cache_stats(cache).device_status == 0


def test_argument_errors_and_empty_cache():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=64)
    cfg = qaq.make_config(1, 1, 128, 64, 2, 8, wl.window, wl.alpha)
    cache = qaq.Cache(cfg)
    bits = torch.full((1, 64), 4, dtype=torch.uint8, device="cuda")
    qaq.qaq_requantize_down(cache, bitsK=bits, bitsV=bits)          # empty cache: nothing to do
    K, V = synth.make_kv(wl)
    thr = qaq.qaq_outlier_thresholds(cfg, K.cuda(), V.cuda())
    qaq.qaq_quantize_append(cache, K.cuda(), V.cuda(), thr, bitsK=bits, bitsV=bits)
    with pytest.raises(qaq.QaqError) as e:
        qaq.qaq_requantize_down(cache, bitsK=bits[:, :32].contiguous(), bitsV=bits[:, :32].contiguous())   # fewer columns than tokens
    assert e.value.code == 1
    with pytest.raises(qaq.QaqError):
        qaq.qaq_requantize_down(cache, nvalid=bits)                 # rules asked for, policy and window missing


def _quantized(wl, K, V, thr_h, bits, T):
    ku, vu = u16(K).reshape(wl.bh, -1, wl.head_dim)[:, :T], u16(V).reshape(wl.bh, -1, wl.head_dim)[:, :T]
    qk = [oracle.quantize(ku[bh], thr_h[bh, 0], thr_h[bh, 1], bits[0, bh, :T]) for bh in range(wl.bh)]
    qv = [oracle.quantize(vu[bh], thr_h[bh, 2], thr_h[bh, 3], bits[1, bh, :T]) for bh in range(wl.bh)]
    return qk, qv


@pytest.mark.parametrize("D,shadow", [(32, "device"), (64, "device"), (128, "device"), (128, "pinned")])
def test_both_directions_leave_the_cache_as_if_filled_at_the_new_widths(D, shadow):
    # widths go up and down at random, twice, with appends in between: tiles that grow move to the end of their
    # pool, the open tile stays the last thing in it.  Expected: direct quantization at the final widths.
    wl = synth.scaled(synth.CONFIGS["C1"], batch=2, heads=2, head_dim=D, tokens=300, seed=90 + D)
    K, V, q, ring, nv = make_inputs(wl)
    T0, T1, T2 = 150, 180, 300                            # 150 = two closed tiles + an open one of 22
    rng = np.random.default_rng(D + 1)
    bits = rng.integers(1, 9, (2, wl.bh, T2)).astype(np.uint8)
    # token capacity three times what is appended: tiles that grow leave their old bytes unused in the pool
    cfg = qaq.make_config(wl.batch, wl.heads, D, 3 * T2, wl.bits_min, wl.bits_max, wl.window, wl.alpha)
    Kd, Vd = K.cuda(), V.cuda()
    Ks, Vs = (Kd, Vd) if shadow == "device" else (K.pin_memory(), V.pin_memory())
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    thr_h = oracle_thresholds(wl, K, V, thr)
    cache = qaq.Cache(cfg)
    tb = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    scale = 1.0 / math.sqrt(D)

    def append(lo, hi):
        qaq.qaq_quantize_append(cache, Kd[:, :, lo:hi], Vd[:, :, lo:hi], thr, bitsK=tb(bits[0][:, lo:hi]), bitsV=tb(bits[1][:, lo:hi]))

    def requantize(T):
        new = rng.integers(1, 9, (2, wl.bh, T)).astype(np.uint8)
        try:
            qaq.qaq_requantize(cache, Ks, Vs, thr, bitsK=tb(new[0]), bitsV=tb(new[1]))
        except qaq.QaqError as e:
            if shadow == "pinned" and e.code == 1:
                pytest.skip("pinned host memory is not mapped into the device's address space here")
            raise
        bits[:, :, :T] = new

    def check(T):
        qk, qv = _quantized(wl, K, V, thr_h, bits, T)
        compare_export(cache, SimpleNamespace(K=qk, V=qv))
        out = qaq.qaq_decode_attention(cache, q.cuda(), scale)
        qq = u16(q).reshape(wl.bh, D)
        ref = np.stack([oracle.decode(qq[bh], qk[bh], qv[bh], scale)[0] for bh in range(wl.bh)])
        assert_attention_close(out.cpu().numpy(), ref)
        assert qaq.qaq_cache_stats(cache).device_status == 0

    append(0, T0); requantize(T0); check(T0)
    append(T0, T1); check(T1)                             # continues behind the (moved or resized) open tile
    requantize(T1); check(T1)
    append(T1, T2); requantize(T2); check(T2)
    # the moves left gaps in the pools; compaction closes them without changing what the cache holds
    before = qaq.qaq_cache_pool_use(cache)
    qaq.qaq_cache_compact(cache)
    after = qaq.qaq_cache_pool_use(cache)
    check(T2)
    assert after[0] < before[0] and after[1] < before[1] and after[2] == before[2]
    # nothing but the tiles, 16-byte aligned each.  A tile has a 32-byte header (which slots have a piece of each width);
    # a tile of keys then takes the bytes of its tokens; a tile of values stores the pieces of each width (8, 4, 2, 1)
    # in groups of four tokens, the last group of a width padded.
    def tile_bytes(b, is_v):
        if not is_v:
            return 32 + int(b.astype(np.int64).sum()) * D // 8
        return 32 + sum(-(-int(np.count_nonzero(b & w)) // 4) * 4 * D * w // 8 for w in (8, 4, 2, 1))
    per_bh = [max(sum((tile_bytes(bits[x][bh, i:min(i + 64, T2)], x == 1) + 15) // 16 * 16 for i in range(0, T2, 64))
                  for bh in range(wl.bh)) for x in range(2)]
    assert after[0] <= per_bh[0] and after[1] <= per_bh[1]
    requantize(T2); check(T2)                                       # and the cache goes on working


def test_widths_by_the_rules_raise_and_lower():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=500)
    K, V, q, ring, nv = make_inputs(wl)
    T = K.shape[2]
    polA = qaq.qaq_policy_from_hyper(*LOOSER, T)          # filled at low widths
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, polA, max_tokens=2 * T)   # room for tiles that move
    ring2, nv2 = synth.make_score_ring(wl, 5)
    polB = qaq.qaq_policy_from_hyper(*HYPER, T)           # tighter budgets: most widths go up
    qaq.qaq_requantize(cache, dev[0], dev[1], thr, policy=polB, ring=ring2.cuda(), nvalid=nv2.cuda())
    thr_h = oracle_thresholds(wl, K, V, thr)
    ref = oracle_batch(wl, K, V, q, ring2, nv2, *oracle.policy(*HYPER, T), thr=thr_h)
    assert qaq.qaq_cache_stats(cache).device_status == 0
    compare_export(cache, ref)                            # as if selected and quantized with the second window and policy
    out2 = qaq.qaq_decode_attention(cache, dev[2], 1.0 / math.sqrt(wl.head_dim))
    assert_attention_close(out2.cpu().numpy(), ref.X)
    first = oracle_batch(wl, K, V, q, ring, nv, *oracle.policy(*LOOSER, T), thr=thr_h)
    up = sum(int((a.bits > b.bits).sum()) for a, b in zip(ref.K + ref.V, first.K + first.V))
    down = sum(int((a.bits < b.bits).sum()) for a, b in zip(ref.K + ref.V, first.K + first.V))
    assert up > 200 and qaq.qaq_cache_stats(cache).device_status == 0, (up, down)


def test_pageable_host_memory_is_refused():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=64)
    K, V = synth.make_kv(wl)
    cfg = qaq.make_config(1, 1, 128, 64, 2, 8, wl.window, wl.alpha)
    cache = qaq.Cache(cfg)
    bits = torch.full((1, 64), 4, dtype=torch.uint8, device="cuda")
    thr = qaq.qaq_outlier_thresholds(cfg, K.cuda(), V.cuda())
    qaq.qaq_quantize_append(cache, K.cuda(), V.cuda(), thr, bitsK=bits, bitsV=bits)
    with pytest.raises(qaq.QaqError) as e:
        qaq.qaq_requantize(cache, K, V, thr, bitsK=bits, bitsV=bits)    # plain CPU tensors: the GPU cannot read them
    assert e.value.code == 1


def test_a_full_pool_is_reported_and_every_tile_stays_consistent():
    # token capacity exactly what is cached: tiles that grow find no room at the end of the pool sooner or later.
    # Those tiles stay as they were; whatever width a token ends up with, its codes are the ones for that width.
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=500)
    K, V, q, ring, nv = make_inputs(wl)
    T = K.shape[2]
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, qaq.qaq_policy_from_hyper(*LOOSER, T))
    ring2, nv2 = synth.make_score_ring(wl, 5)
    qaq.qaq_requantize(cache, dev[0], dev[1], thr, policy=qaq.qaq_policy_from_hyper(*HYPER, T), ring=ring2.cuda(), nvalid=nv2.cuda())
    assert qaq.qaq_cache_stats(cache).device_status == 3
    got = np.stack([qaq.qaq_cache_export(cache, x)["bits"].cpu().numpy() for x in range(2)])
    qk, qv = _quantized(wl, K, V, oracle_thresholds(wl, K, V, thr), got, T)
    compare_export(cache, SimpleNamespace(K=qk, V=qv))
    out2 = qaq.qaq_decode_attention(cache, dev[2], 1.0 / math.sqrt(wl.head_dim))
    assert_attention_close(out2.cpu().numpy(), _decode_ref(wl, q, qk, qv))


def test_compaction_of_a_pool_with_many_moved_tiles():
    # 5000 tokens = 78 closed tiles + an open one; raising the widths moves most tiles, compaction brings the pool
    # back to the size of its contents and later appends and decodes work on it
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=5100)
    K, V, q, ring, nv = make_inputs(wl)
    T, D = 5000, wl.head_dim
    rng = np.random.default_rng(17)
    bits = rng.integers(1, 5, (2, wl.bh, 5100)).astype(np.uint8)
    cfg = qaq.make_config(wl.batch, wl.heads, D, 3 * 5100, wl.bits_min, wl.bits_max, wl.window, wl.alpha)
    Kd, Vd = K.cuda(), V.cuda()
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    cache = qaq.Cache(cfg)
    tb = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    qaq.qaq_quantize_append(cache, Kd[:, :, :T], Vd[:, :, :T], thr, bitsK=tb(bits[0][:, :T]), bitsV=tb(bits[1][:, :T]))
    filled = qaq.qaq_cache_pool_use(cache)
    bits[:, :, :T] = rng.integers(3, 9, (2, wl.bh, T)).astype(np.uint8)
    qaq.qaq_requantize(cache, Kd, Vd, thr, bitsK=tb(bits[0][:, :T]), bitsV=tb(bits[1][:, :T]))
    moved = qaq.qaq_cache_pool_use(cache)
    qaq.qaq_cache_compact(cache)
    packed = qaq.qaq_cache_pool_use(cache)
    assert moved[0] > 1.5 * filled[0] and packed[0] < 0.8 * moved[0] and packed[1] < 0.8 * moved[1]
    qaq.qaq_quantize_append(cache, Kd[:, :, T:], Vd[:, :, T:], thr, bitsK=tb(bits[0][:, T:]), bitsV=tb(bits[1][:, T:]))
    qk, qv = _quantized(wl, K, V, oracle_thresholds(wl, K, V, thr), bits, 5100)
    compare_export(cache, SimpleNamespace(K=qk, V=qv))
    out = qaq.qaq_decode_attention(cache, q.cuda(), 1.0 / math.sqrt(D))
    assert_attention_close(out.cpu().numpy(), _decode_ref(wl, q, qk, qv))
    assert qaq.qaq_cache_stats(cache).device_status == 0


def test_appends_and_decode_after_a_pool_ran_full():
    # Raising widths moves tiles to the end of their pool until it is full; appends that find no room afterwards are
    # reported (device status QAQ_ERR_CAPACITY), publish nothing, and decode and export keep working on what the
    # cache holds: tokens that were not stored count with zero width.
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=640)
    K, V, q, ring, nv = make_inputs(wl)
    T0 = 500
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, 640, wl.bits_min, wl.bits_max, wl.window, wl.alpha)
    Kd, Vd, qd = K.cuda(), V.cuda(), q.cuda()
    thr = qaq.qaq_outlier_thresholds(cfg, Kd[:, :, :T0], Vd[:, :, :T0])
    cache = qaq.Cache(cfg)
    low = torch.full((wl.bh, T0), 2, dtype=torch.uint8, device="cuda")
    qaq.qaq_quantize_append(cache, Kd[:, :, :T0], Vd[:, :, :T0], thr, bitsK=low, bitsV=low)
    for b in (3, 5, 6, 7, 8):          # every step makes the closed tiles grow and move
        up = torch.full((wl.bh, T0), b, dtype=torch.uint8, device="cuda")
        qaq.qaq_requantize(cache, Kd[:, :, :T0], Vd[:, :, :T0], thr, bitsK=up, bitsV=up)
    assert qaq.qaq_cache_stats(cache).device_status == 3
    wide = torch.full((wl.bh, 1), 8, dtype=torch.uint8, device="cuda")
    for t in range(T0, 640):
        qaq.qaq_quantize_append(cache, Kd[:, :, t:t + 1], Vd[:, :, t:t + 1], thr, bitsK=wide, bitsV=wide)
    assert cache.tokens == 640
    out = qaq.qaq_decode_attention(cache, qd, 1.0 / math.sqrt(wl.head_dim))
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    use = qaq.qaq_cache_pool_use(cache)
    assert use[0] <= use[2] and use[1] <= use[2]
    for x in range(2):
        ex = qaq.qaq_cache_export(cache, x)
        bits = ex["bits"].cpu().numpy()
        assert set(np.unique(bits)) <= {0, 2, 3, 5, 6, 7, 8}
    qaq.qaq_cache_compact(cache)
    out2 = qaq.qaq_decode_attention(cache, qd, 1.0 / math.sqrt(wl.head_dim))
    assert np.array_equal(out2.cpu().numpy().view(np.uint32), out.cpu().numpy().view(np.uint32))
