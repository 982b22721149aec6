"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Widths, outlier lists, scales and packed codes must match bit for bit;
attention outputs within 2e-3 absolute + 1e-2 relative."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import qaq, synth

from gpu_helpers import (assert_attention_close, compare_export, gpu_pipeline, make_inputs, oracle_batch, u16)

pytestmark = pytest.mark.gpu

# hyper-parameters (sigmaS_max, sigmaX_max, qnorm2) that give mixed widths on the synthetic caches
HYPER = {"C1": (0.006, 0.03, 64.0), "C2": (0.002, 0.01, 128.0), "C4": (0.004, 0.05, 128.0)}


def full_case(wl, hyper, ragged=False, bh_sel=None, layer=0):
    K, V, q, ring, nv = make_inputs(wl, layer, ragged)
    T = K.shape[2]
    pol = qaq.qaq_policy_from_hyper(*hyper, T)
    cK, cV = oracle.policy(*hyper, T)
    assert (pol.cK, pol.cV) == (cK, cV)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    ref = oracle_batch(wl, K, V, q, ring, nv, cK, cV, bh_sel=bh_sel)
    sel = slice(None) if bh_sel is None else bh_sel
    # thresholds: exact order statistics
    assert np.array_equal(thr.cpu().numpy()[sel], ref.thr)
    # separate selection kernel = fused selection = oracle
    bK, bV = qaq.qaq_select_bits(cfg, pol, dev[0], dev[1], dev[3], dev[4], thr)
    assert np.array_equal(bK.cpu().numpy()[sel], ref.bitsK) and np.array_equal(bV.cpu().numpy()[sel], ref.bitsV)
    compare_export(cache, ref, bh_sel)
    assert_attention_close(out.cpu().numpy()[sel], ref.X)
    S = scores.cpu().numpy()[sel].astype(np.float64)
    assert np.all(np.abs(S - ref.S) <= 1e-6 + 1e-2 * ref.S)
    assert np.allclose(S.sum(1), 1.0, atol=1e-3)
    st = qaq.qaq_cache_stats(cache)
    assert st.device_status == 0 and st.tokens == T
    return cache, ref, st


def test_c1_tiny_layer_full_parity():
    wl = synth.CONFIGS["C1"]
    cache, ref, st = full_case(wl, HYPER["C1"])
    # compression ratio from bit counts, as the oracle computes it
    cbk = sum(oracle.code_bits(r.bits, wl.head_dim) for r in ref.K); cbv = sum(oracle.code_bits(r.bits, wl.head_dim) for r in ref.V)
    nok = sum(r.ch.size for r in ref.K); nov = sum(r.ch.size for r in ref.V)
    assert st.cr_paper == pytest.approx(oracle.cr_paper(cbk, cbv, nok, nov, wl.tokens * wl.bh, wl.head_dim), rel=1e-12)
    assert st.code_bytes[0] * 8 == cbk and st.outliers[1] == nov
    assert len([b for b in range(9) if st.hist[1][b]]) >= 4           # several widths exercised


def test_c2_shaped_ragged_tail_and_ragged_window():
    # 7B head geometry, fewer heads; 1000 tokens = 15 full tiles + a tail of 40; window rows partly missing
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=1000)
    full_case(wl, HYPER["C2"], ragged=True)


def test_heavy_tails_many_outliers():
    # Student-t data, 5 % planted outliers, window 64; alpha = 10 % makes a tile hold more outliers than are staged on chip
    wl = synth.scaled(synth.CONFIGS["C4"], batch=1, heads=2, tokens=640, alpha=0.10)
    full_case(wl, HYPER["C4"])


def test_head_dim_32_and_64_batch_gt_1():
    for D in (32, 64):
        wl = synth.scaled(synth.CONFIGS["C1"], batch=2, heads=3, head_dim=D, tokens=200, seed=11 + D)
        full_case(wl, HYPER["C1"])


def test_every_width_given_bits_and_no_outliers():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=257, alpha=0.0, bits_min=1)
    K, V, q, ring, nv = make_inputs(wl)
    g = torch.Generator().manual_seed(5)
    bK = torch.randint(1, 9, (wl.bh, 257), generator=g, dtype=torch.uint8)
    bV = torch.randint(1, 9, (wl.bh, 257), generator=g, dtype=torch.uint8)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 257)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol, bits=(bK, bV))
    ref = oracle_batch(wl, K, V, q, ring, nv, pol.cK, pol.cV, bitsK=bK.numpy(), bitsV=bV.numpy())
    compare_export(cache, ref)
    assert sum(r.ch.size for r in ref.K) == 0
    assert_attention_close(out.cpu().numpy(), ref.X)


def test_appends_equal_bulk_quantization():
    # prefill 100, then 70 single-token appends (crossing tile boundaries), then a bulk of 150:
    # the cache must equal the quantization of all 320 tokens at once
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=320, window=4)
    K, V, q, ring, nv = make_inputs(wl, ragged=True)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 320)
    cfg = qaq.make_config(1, 2, 128, 320, 2, 8, 4, wl.alpha)
    Kd, Vd, qd, rd, nd = (t.cuda() for t in (K, V, q, ring, nv))
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    cache = qaq.Cache(cfg)
    pieces = [(0, 100)] + [(100 + i, 101 + i) for i in range(70)] + [(170, 320)]
    for a, b in pieces:
        qaq.qaq_quantize_append(cache, Kd[:, :, a:b], Vd[:, :, a:b], thr, policy=pol,
                                ring=rd[:, :, :, a:b].contiguous(), nvalid=nd[:, :, a:b].contiguous())
    assert cache.tokens == 320
    ref = oracle_batch(wl, K, V, q, ring, nv, pol.cK, pol.cV)
    compare_export(cache, ref)
    out = qaq.qaq_decode_attention(cache, qd, 1 / math.sqrt(128))
    assert_attention_close(out.cpu().numpy(), ref.X)
    # decode after every growth step equals the oracle on the prefix (sampled)
    cache.reset()
    for a, b in pieces[:40]:
        qaq.qaq_quantize_append(cache, Kd[:, :, a:b], Vd[:, :, a:b], thr, policy=pol,
                                ring=rd[:, :, :, a:b].contiguous(), nvalid=nd[:, :, a:b].contiguous())
    Tp = cache.tokens
    wlp = synth.scaled(wl, tokens=Tp)
    refp = oracle_batch(wlp, K[:, :, :Tp], V[:, :, :Tp], q, ring[:, :, :, :Tp].contiguous(), nv[:, :, :Tp].contiguous(),
                        pol.cK, pol.cV, thr=ref.thr)              # the oracle's own thresholds of the full sequence, frozen
    out = qaq.qaq_decode_attention(cache, qd, 1 / math.sqrt(128))
    assert_attention_close(out.cpu().numpy(), refp.X)


def test_new_tokens_without_scores_take_bmax_for_values():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=64)
    K, V, q, ring, nv = make_inputs(wl)
    nv[:] = 0
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 64)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    ex = qaq.qaq_cache_export(cache, 1)
    assert (ex["bits"] == 8).all()
    ref = oracle_batch(wl, K, V, q, ring, nv, pol.cK, pol.cV)
    compare_export(cache, ref)


def test_single_token_and_constant_tokens():
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=1, heads=1)
    K, V, q, ring, nv = make_inputs(wl)
    K[:] = 0.75   # zero range: step 0, all codes 0
    pol = qaq.qaq_policy_from_hyper(*HYPER["C1"], 1)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    ref = oracle_batch(wl, K, V, q, ring, nv, pol.cK, pol.cV)
    compare_export(cache, ref)
    assert_attention_close(out.cpu().numpy(), ref.X)
    assert scores.cpu().numpy()[0, 0] == pytest.approx(1.0)


def test_runs_of_tiles_that_straddle_two_heads():
    # 3 (b,h) x 10 tiles are cut into runs of 4 tiles: the third run ends one head and begins the next
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=600)
    full_case(wl, HYPER["C2"])


def test_split_count_does_not_change_the_result_beyond_rounding():
    # same cache content decoded with different cuts of the tile sequence (runs of 4 tiles inside a head;
    # runs of 5 tiles, some of which straddle two heads)
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=2048)
    K, V, q, ring, nv = make_inputs(wl)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 2048)
    outs = []
    for rep in (1, 40):   # 2 (b,h) -> 16 runs of 4 tiles;  80 (b,h) -> 512 runs of 5 tiles
        wlr = synth.scaled(wl, batch=rep)
        Kr, Vr, qr = K.repeat(rep, 1, 1, 1), V.repeat(rep, 1, 1, 1), q.repeat(rep, 1, 1)
        rr, nr = ring.repeat(rep, 1, 1, 1), nv.repeat(rep, 1, 1)
        cfg, cache, thr, out, scores, dev = gpu_pipeline(wlr, Kr, Vr, qr, rr, nr, pol)
        outs.append(out.cpu().numpy()[:2])
        if rep > 1:
            # replicas are cut at different tiles, so they agree up to the rounding of the value weights to
            # 11 significant bits: at most 2^-12 * sum_t p_t |v_t - X|, and the attention here is peaked on
            # a few tokens whose values differ by up to ~4, so no averaging helps
            assert np.allclose(out.cpu().numpy()[:2], out.cpu().numpy()[-2:], rtol=0, atol=1e-3)
    assert np.allclose(outs[0], outs[1], rtol=0, atol=1e-3)


def test_capacity_errors_are_reported_not_faulted():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=128)
    K, V, q, ring, nv = make_inputs(wl)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 128)
    cfg = qaq.make_config(1, 1, 128, 100, 2, 8, wl.window, wl.alpha)
    cache = qaq.Cache(cfg)
    Kd, Vd, rd, nd = K.cuda(), V.cuda(), ring.cuda(), nv.cuda()
    thr = qaq.qaq_outlier_thresholds(cfg, Kd, Vd)
    with pytest.raises(qaq.QaqError) as e:
        qaq.qaq_quantize_append(cache, Kd, Vd, thr, policy=pol, ring=rd, nvalid=nd)   # 128 > 100 tokens
    assert e.value.code == 3 and cache.tokens == 0
    with pytest.raises(qaq.QaqError):
        qaq.qaq_decode_attention(cache, q.cuda(), 0.1)                                  # empty cache
    # outlier list too small: surplus outliers are dropped and the device status says so
    cfg2 = qaq.make_config(1, 1, 128, 128, 2, 8, wl.window, 0.2, max_outliers_per_bh=1)
    cache2 = qaq.Cache(cfg2)
    thr2 = qaq.qaq_outlier_thresholds(cfg2, Kd, Vd)
    qaq.qaq_quantize_append(cache2, Kd, Vd, thr2, policy=pol, ring=rd, nvalid=nd)
    st = qaq.qaq_cache_stats(cache2)
    assert st.device_status == 3
    torch.cuda.synchronize()


def test_host_buffer_entry_points_match_device_path():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=192)
    K, V, q, ring, nv = make_inputs(wl)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C2"], 192)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    cache_h = qaq.Cache(cfg)
    pin = lambda t: t.contiguous().pin_memory()
    qaq.qaq_quantize_append_host(cache_h, pin(K), pin(V), pol, pin(ring), pin(nv), pin(thr.cpu()))
    out_h = torch.empty((wl.bh, 128), dtype=torch.float32).pin_memory()
    qaq.qaq_decode_attention_host(cache_h, pin(q), 1 / math.sqrt(128), out_h)
    assert np.array_equal(out_h.numpy(), out.cpu().numpy())


def test_c3_shaped_full_size_layer_sampled():
    # the launch configuration the benchmark times: 8 x 32 (b,h), 4096 tokens; the oracle checks a sample of (b,h)
    wl = synth.scaled(synth.CONFIGS["C3"], layers=1)
    sel = [0, 97, 255]
    full_case(wl, HYPER["C2"], bh_sel=sel)


@pytest.mark.parametrize("tokens", [48, 64, 1000])
def test_thresholds_with_nans_of_both_signs(tokens):
    # NaNs are left out of the population (the oracle's reading); 48 and 64 tokens are solved from the
    # sample alone, 1000 tokens go through bracket, scan and select.  One head is NaN only.
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, tokens=tokens)
    K, V = synth.make_kv(wl, 0)
    rng = np.random.default_rng(5)
    Ku, Vu = u16(K).copy(), u16(V).copy()
    for arr, frac in ((Ku, 0.02), (Vu, 0.3)):
        m = rng.random(arr.shape) < frac
        arr[m] = np.where(rng.random(int(m.sum())) < 0.5, 0x7E00, 0xFE01).astype(np.uint16)   # +NaN, -NaN
    Vu[0, 2] = 0xFFFF
    Kn = torch.from_numpy(Ku.view(np.float16)).cuda()
    Vn = torch.from_numpy(Vu.view(np.float16)).cuda()
    cfg = qaq.make_config(wl.batch, wl.heads, wl.head_dim, tokens, 2, 8, wl.window, wl.alpha)
    thr = qaq.qaq_outlier_thresholds(cfg, Kn, Vn).cpu().numpy()
    for bh in range(wl.bh):
        b, h = divmod(bh, wl.heads)
        want = (*oracle.thresholds(Ku[b, h], wl.alpha), *oracle.thresholds(Vu[b, h], wl.alpha))
        assert np.array_equal(thr[bh], np.array(want, dtype=np.float32)), (bh, thr[bh], want)


def test_decode_twice_gives_the_same_bits():
    # outlier corrections are summed with integer atomics and everything else in a fixed order: a repeat of the call,
    # and a call with the score row requested, return the same output bit for bit
    wl = synth.scaled(synth.CONFIGS["C4"], batch=2, heads=3, tokens=1500, alpha=0.10)      # many outliers per tile
    K, V, q, ring, nv = make_inputs(wl)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C4"], wl.tokens)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    first = out.cpu().numpy().view(np.uint32).copy()
    for _ in range(3):
        again = qaq.qaq_decode_attention(cache, dev[2], 1.0 / math.sqrt(wl.head_dim))
        assert np.array_equal(again.cpu().numpy().view(np.uint32), first)


@pytest.mark.parametrize("D,n_q", [(128, 1), (128, 3), (128, 8), (64, 5), (32, 4), (64, 6), (32, 2)])
def test_batched_multi_query_decode(D, n_q):
    # several queries per (b,h) in one call (Section 4.2, integration: every later query reads the same packed cache):
    # each against the oracle's attention for that query, and against the single-query entry point; 1000 tokens with
    # a ragged tail, CTAs that straddle two (b,h), eight queries in two passes
    wl = synth.scaled(synth.CONFIGS["C2"], heads=3, head_dim=D, tokens=1000, seed=40 + D)
    K, V, q, ring, nv = make_inputs(wl)
    hyper = HYPER["C2"]
    pol = qaq.qaq_policy_from_hyper(*hyper, wl.tokens)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    ref = oracle_batch(wl, K, V, q, ring, nv, *oracle.policy(*hyper, wl.tokens))
    g = torch.Generator().manual_seed(7 + n_q)
    Q = (torch.randn((wl.bh, n_q, D), generator=g) * torch.linspace(0.5, 2.0, n_q).view(1, n_q, 1)).to(torch.float16)
    Q[:, 0] = q.reshape(wl.bh, D)
    scale = 1.0 / math.sqrt(D)
    got = qaq.qaq_decode_attention_multi(cache, Q.cuda(), scale).cpu().numpy()
    Qu = Q.numpy().view(np.uint16)
    for j in range(n_q):
        want = np.stack([oracle.decode(Qu[bh, j], ref.K[bh], ref.V[bh], scale)[0] for bh in range(wl.bh)])
        assert_attention_close(got[:, j], want)
        single = qaq.qaq_decode_attention(cache, Q[:, j].contiguous().cuda(), scale).cpu().numpy()
        assert np.all(np.abs(got[:, j] - single) <= 1e-3 + 5e-3 * np.abs(single))     # two roundings of the same sums
    with pytest.raises(qaq.QaqError):
        qaq.qaq_decode_attention_multi(cache, torch.zeros((wl.bh, 9, D), dtype=torch.float16, device="cuda"), scale)


@pytest.mark.parametrize("tokens,alpha", [(1, 0.01), (65, 0.01), (640, 0.10)])
def test_batched_decode_edge_cases(tokens, alpha):
    # a single token, one token past a tile, and tiles with more outliers than one pass over the threads handles
    wl = synth.scaled(synth.CONFIGS["C4"], batch=1, heads=2, tokens=tokens, alpha=alpha)
    K, V, q, ring, nv = make_inputs(wl)
    pol = qaq.qaq_policy_from_hyper(*HYPER["C4"], tokens)
    cfg, cache, thr, out, scores, dev = gpu_pipeline(wl, K, V, q, ring, nv, pol)
    ref = oracle_batch(wl, K, V, q, ring, nv, *oracle.policy(*HYPER["C4"], tokens))
    D, scale = wl.head_dim, 1.0 / math.sqrt(wl.head_dim)
    g = torch.Generator().manual_seed(3)
    Q = torch.randn((wl.bh, 2, D), generator=g).to(torch.float16)
    got = qaq.qaq_decode_attention_multi(cache, Q.cuda(), scale).cpu().numpy()
    Qu = Q.numpy().view(np.uint16)
    for j in range(2):
        want = np.stack([oracle.decode(Qu[bh, j], ref.K[bh], ref.V[bh], scale)[0] for bh in range(wl.bh)])
        assert_attention_close(got[:, j], want)
