"""Pins for the CPU oracle: each check ties a part of oracle/ to something other than
itself -- closed forms and hand-worked cases of the paper's formulas, invariants the
paper states, brute force on small inputs, and library routines (numpy sort, torch
softmax attention) on the special cases that reduce to them."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2403_04643_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F16_INF = np.float32(np.inf)


def f16bits(a):
    return np.asarray(a, dtype=np.float16).view(np.uint16)


def rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(v) for v in line.split()])
    return out


# ---------------------------------------------------------------------------- fp16
def test_half_to_float_matches_numpy_for_every_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    ref = allbits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in allbits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


# ---------------------------------------------------------------- bit count (E-B)
def test_bit_count_golden_cases():
    for r, c, b in rows("bit_count_cases.txt"):
        assert oracle.bits_ladder(r, c, 1, 16) == int(b)


def test_bit_ladder_boundaries_and_clamp():
    c = np.float32(0.3711)
    for b in range(2, 9):
        r = np.float32(math.ldexp(float(c), b))              # exactly c * 2^b -> b
        assert oracle.bits_ladder(r, c, 2, 8) == b
        up = np.nextafter(r, np.float32(np.inf), dtype=np.float32)
        assert oracle.bits_ladder(up, c, 2, 8) == min(b + 1, 8)
    assert oracle.bits_ladder(0.0, c, 2, 8) == 2                # zero range -> b_min
    assert oracle.bits_ladder(1e30, c, 2, 8) == 8               # clamp above
    assert oracle.bits_ladder(1.0, 0.0, 2, 8) == 8              # no bound -> b_max


def test_bit_ladder_equals_ceil_log2_away_from_boundaries():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        r = np.float32(rng.uniform(1e-3, 50.0))
        c = np.float32(rng.uniform(1e-3, 2.0))
        x = math.log2(float(r) / float(c))
        if abs(x - round(x)) < 1e-4:
            continue
        want = min(8, max(2, math.ceil(x)))
        assert oracle.bits_ladder(r, c, 2, 8) == want


def test_value_bits_monotone_in_score_and_range_key_bits_ignore_score():
    cV = np.float32(0.01)
    prev = 0
    for s in np.geomspace(1e-6, 1.0, 60):
        b = oracle.value_bits(-1.0, 2.0, np.float32(s), cV, 2, 8)
        assert b >= prev
        prev = b
    assert prev == 8
    prev = 0
    for r in np.geomspace(1e-3, 100.0, 60):
        b = oracle.value_bits(0.0, np.float32(r), np.float32(0.01), cV, 2, 8)
        assert b >= prev
        prev = b
    # larger sigma budget -> fewer bits
    assert oracle.value_bits(-1.0, 2.0, 0.01, np.float32(0.1), 2, 8) <= oracle.value_bits(-1.0, 2.0, 0.01, cV, 2, 8)
    # unknown score (no row observed yet) -> b_max
    assert oracle.value_bits(-1.0, 2.0, F16_INF, cV, 2, 8) == 8
    # the key rule has no S_t in it: select_bits must not change K widths when scores change
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=64)
    K, V = synth.make_kv(wl)
    ring, nv = synth.make_score_ring(wl)
    k = K[0, 0].numpy().view(np.uint16); v = V[0, 0].numpy().view(np.uint16)
    thr = np.array([-1e9, 1e9, -1e9, 1e9], np.float32)
    b1 = oracle.select_bits(k, v, thr, ring[0, 0].numpy(), nv[0, 0].numpy(), 0.05, 1e-3, 2, 8)
    b2 = oracle.select_bits(k, v, thr, ring[0, 0].numpy() * 0.01, nv[0, 0].numpy(), 0.05, 1e-3, 2, 8)
    assert np.array_equal(b1[0], b2[0])
    assert (b2[1] <= b1[1]).all() and (b2[1] < b1[1]).any()


def test_policy_closed_forms():
    # Key bound substituted back into the variance approximation of Section 4.1 gives sigma2(S)_max:
    #   var(S_t) ~ T^-2 (1 - 1/T) (exp(sum_d Q_d^2 * var(K_t)) - 1)
    for sS, sX, qn, T in [(1e-4, 0.05, 130.0, 4096), (3e-3, 0.2, 11.5, 512), (1e-5, 1.0, 64.0, 131072)]:
        cK, cV = oracle.policy(sS, sX, qn, T)
        varK = (float(cK) / (2 * math.sqrt(3))) ** 2
        varS = (1.0 / T**2) * (1 - 1.0 / T) * math.expm1(qn * varK)
        assert varS == pytest.approx(sS**2, rel=1e-5)
        # Value bound: with sigma(V_t) = sigmaX / (sqrt(T) S_t), sum_t S_t^2 var(V_t) = sigmaX^2
        S = np.random.default_rng(1).dirichlet(np.ones(T))
        sigV = (float(cV) / (2 * math.sqrt(3))) / S
        assert float(np.sum(S**2 * sigV**2)) == pytest.approx(sX**2, rel=1e-5)
    assert oracle.policy(1e-3, 0.1, 10.0, 1)[0] == 0.0        # T = 1: key bound undefined -> b_max


def test_value_rule_keeps_output_variance_under_budget():
    # Unclamped widths from the value rule => sum_t S_t^2 * step_t^2 / 12 <= sigmaX_max^2 (Section 4.1)
    rng = np.random.default_rng(3)
    T = 1024
    S = rng.dirichlet(np.full(T, 0.3)).astype(np.float32)
    r = rng.uniform(0.5, 8.0, T).astype(np.float32)
    sX = 0.02
    _, cV = oracle.policy(1e-3, sX, 100.0, T)
    tot = 0.0
    for t in range(T):
        b = oracle.value_bits(0.0, r[t], S[t], cV, 0, 40)
        step = float(r[t]) / 2.0**b
        tot += float(S[t]) ** 2 * step**2 / 12.0
    assert tot <= sX**2 * (1 + 1e-5)


# ---------------------------------------------------------------- quantizer (E-Q)
def test_midpoint_golden_cases():
    for B, x, code, xhat in rows("midpoint_cases.txt"):
        tok = f16bits([0.0, 8.0, x] + [4.0] * 29)
        mn, step, codes, flag = oracle.token_codes(tok, -np.inf, np.inf, int(B))
        assert mn == 0.0 and step == np.float32(8.0 / 2 ** int(B))
        assert codes[2] == int(code)
        assert float(oracle.dequant(codes[2], mn, step)) == xhat
        assert not flag.any()


def test_quantizer_bruteforce_error_bound_all_widths():
    # every binary16 value in [-2, 2) as data, in shuffled tokens of 32 channels
    vals = np.arange(65536, dtype=np.uint16).view(np.float16)
    vals = vals[np.isfinite(vals) & (np.abs(vals.astype(np.float32)) < 2.0)]
    rng = np.random.default_rng(0)
    vals = rng.permutation(vals)
    vals = vals[: (vals.size // 32) * 32].reshape(-1, 32)[:600]
    errs = {}
    for B in range(2, 9):
        e_all = []
        for tok in vals:
            x = tok.astype(np.float64)
            mn, step, codes, _ = oracle.token_codes(tok.view(np.uint16), -np.inf, np.inf, B)
            r = x.max() - x.min()
            assert float(mn) == x.min() and float(step) == pytest.approx(r / 2**B, rel=1e-7)
            assert codes.max() <= 2**B - 1
            assert codes[np.argmin(x)] == 0 and codes[np.argmax(x)] == 2**B - 1
            xhat = np.array([float(oracle.dequant(c, mn, step)) for c in codes])
            delta = r / 2 ** (B + 1)
            assert np.all(np.abs(x - xhat) <= delta * (1 + 1e-5) + 1e-7)
            e_all.append((x - xhat) / max(float(step), 1e-30))
        errs[B] = np.concatenate(e_all)
    # spread-out data: errors are uniform over a segment, sigma = Delta / sqrt 3 = step / (2 sqrt 3)
    u = np.random.default_rng(1).uniform(-1, 1, (400, 128)).astype(np.float16)
    e = []
    for tok in u:
        mn, step, codes, _ = oracle.token_codes(tok.view(np.uint16), -np.inf, np.inf, 3)
        e.append((tok.astype(np.float64) - (float(mn) + (codes + 0.5) * float(step))) / float(step))
    assert np.std(np.concatenate(e)) == pytest.approx(1 / (2 * math.sqrt(3)), rel=0.02)


def test_codes_nest_from_higher_to_lower_width():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=48)
    K, _ = synth.make_kv(wl)
    for tok in K[0, 0].numpy().view(np.uint16):
        ref = {B: oracle.token_codes(tok, -4.0, 4.0, B)[2] for B in range(2, 9)}
        for B in range(3, 9):
            for Bl in range(2, B):
                assert np.array_equal(ref[B] >> (B - Bl), ref[Bl])


def test_degenerate_tokens():
    tok = f16bits([1.5] * 32)
    mn, step, codes, flag = oracle.token_codes(tok, -np.inf, np.inf, 4)
    assert mn == 1.5 and step == 0.0 and not codes.any()
    assert float(oracle.dequant(0, mn, step)) == 1.5
    # every entry an outlier -> range [0,0]
    mn, step, codes, flag = oracle.token_codes(tok, -1.0, 1.0, 4)
    assert mn == 0.0 and step == 0.0 and flag.all() and not codes.any()


# ---------------------------------------------------------------- outliers
def test_thresholds_are_order_statistics():
    rng = np.random.default_rng(5)
    x = rng.standard_normal(64 * 128).astype(np.float16)
    for alpha in (0.0, 0.01, 0.05, 0.5):
        lo, hi = oracle.thresholds(x.view(np.uint16), alpha)
        s = np.sort(x.astype(np.float32))
        k = int(math.floor(alpha * x.size / 2))
        assert lo == s[k] and hi == s[x.size - 1 - k]
        n_out = int(np.sum((x.astype(np.float32) < lo) | (x.astype(np.float32) > hi)))
        assert n_out <= alpha * x.size
    # ties at the threshold are not outliers
    y = np.array([0.0] * 90 + [5.0] * 10, np.float16)
    lo, hi = oracle.thresholds(y.view(np.uint16), 0.1)
    assert (lo, hi) == (0.0, 5.0)


def test_thresholds_leave_nans_of_both_signs_out_of_the_population():
    # Section 4.2 "Outliers": the quantile is taken over the values of the tensor; a NaN has no rank, so the
    # population is the non-NaN values and k = floor(alpha * N / 2) counts only them.
    rng = np.random.default_rng(17)
    x = rng.standard_normal(40 * 64).astype(np.float16)
    u = x.view(np.uint16).copy()
    nan_pos = rng.choice(u.size, 300, replace=False)
    u[nan_pos[:150]] = 0x7E00 | rng.integers(0, 0x1FF, 150).astype(np.uint16)   # +NaN, several payloads
    u[nan_pos[150:]] = 0xFE00 | rng.integers(0, 0x1FF, 150).astype(np.uint16)   # -NaN
    xf = u.view(np.float16).astype(np.float32)
    good = np.sort(xf[~np.isnan(xf)])               # numpy's sort of the values that have a rank
    N = good.size
    assert N == u.size - 300
    for alpha in (0.0, 0.01, 0.05, 0.3):
        lo, hi = oracle.thresholds(u, alpha)
        k = int(math.floor(alpha * N / 2))
        assert lo == good[k] and hi == good[N - 1 - k]
        assert int(np.sum((good < lo) | (good > hi))) <= alpha * N
    # a tiny case where counting the NaNs in N would move the rank
    tiny = np.array([1, 2, 3, 4, 5, 6, 7, 8, 9, 10], np.float16).view(np.uint16).copy()
    with_nan = np.concatenate([tiny, np.array([0x7E00, 0xFE00, 0x7FFF, 0xFFFF], np.uint16)])
    # alpha = 0.4: N = 10 -> k = 2 -> (3, 8); counting the NaNs (N = 14) would give k = 2.8 -> 2 as well,
    # alpha = 0.6: N = 10 -> k = 3 -> (4, 7); with N = 14, k = 4 -> (5, 6): this one tells them apart
    assert oracle.thresholds(with_nan, 0.4) == (3.0, 8.0)
    assert oracle.thresholds(with_nan, 0.6) == (4.0, 7.0)
    # NaNs must not sort to either end either: the extremes at alpha = 0 are the finite ones
    assert oracle.thresholds(with_nan, 0.0) == (1.0, 10.0)
    # nothing but NaNs: no population, thresholds (0, 0)
    assert oracle.thresholds(np.array([0x7E00, 0xFE01, 0x7FFF], np.uint16), 0.01) == (0.0, 0.0)
    # alpha at a tie: the k-th values are repeated, equal values are not outliers, so the count stays <= alpha N
    t = np.array([-2.0] * 5 + [0.0] * 10 + [2.0] * 5, np.float16).view(np.uint16)
    lo, hi = oracle.thresholds(np.concatenate([t, np.array([0xFE00], np.uint16)]), 0.5)   # k = 5: first of the zeros
    assert (lo, hi) == (0.0, 0.0)
    lo, hi = oracle.thresholds(np.concatenate([t, np.array([0x7E00], np.uint16)]), 0.4)   # k = 4: inside the tie at -2 / 2
    assert (lo, hi) == (-2.0, 2.0)


def test_planted_outliers_are_split_off_and_kept_exactly():
    wl = synth.scaled(synth.CONFIGS["C2"], heads=2, tokens=256)
    K, _ = synth.make_kv(wl)
    x = K[0, 1].numpy()
    xb = x.view(np.uint16)
    lo, hi = oracle.thresholds(xb, 0.02)            # alpha above the planted 1 %
    xf = x.astype(np.float32)
    planted = np.abs(xf) > 9.0 * np.exp(0.5 * 3.5)   # far beyond any N(0,1)*scale draw of this size
    bits = np.full(256, 4, np.uint8)
    qt = oracle.quantize(xb, lo, hi, bits)
    mask = np.zeros_like(planted)
    for t in range(256):
        for o in range(qt.rowptr[t], qt.rowptr[t + 1]):
            mask[t, qt.ch[o]] = True
            assert qt.val[o] == xb[t, qt.ch[o]]                      # bit-identical binary16
        chs = qt.ch[qt.rowptr[t]: qt.rowptr[t + 1]]
        assert np.all(np.diff(chs.astype(int)) > 0)                 # channel order inside a token
    assert np.array_equal(mask, (xf < lo) | (xf > hi))
    assert mask[planted].all()
    assert qt.rowptr[-1] <= 0.02 * x.size
    # the range of what is left shrinks
    for t in range(0, 256, 17):
        mn, mx = oracle.masked_range(xb[t], lo, hi)
        assert mn >= xf[t].min() and mx <= xf[t].max() and lo <= mn <= mx <= hi
    # reconstruction restores outliers exactly and everything else within Delta
    xh = oracle.reconstruct(qt)
    assert np.array_equal(xh[mask], xf[mask])
    delta = (qt.step / 2)[:, None]
    assert np.all(np.abs(xh - xf)[~mask] <= (np.broadcast_to(delta, xf.shape) * (1 + 1e-5))[~mask] + 1e-7)


# ---------------------------------------------------------------- packing
@pytest.mark.parametrize("D", [32, 64, 128])
def test_pack_roundtrip_and_size(D):
    rng = np.random.default_rng(D)
    for B in range(1, 9):
        codes = rng.integers(0, 2**B, D).astype(np.uint8)
        data = oracle.pack_token(codes, B)
        assert data.size == D * B // 8
        assert np.array_equal(oracle.unpack_token(data, D, B), codes)
        assert int(np.unpackbits(data).sum()) == int(np.unpackbits(codes).sum())   # every code bit stored once


def test_plane_layout_byte_lane_property():
    """Independent statement of the layout: in the plane of width w, AND-ing a 32-bit word with the mask
    (2^w-1) replicated in the four byte lanes and shifted by w*m selects, in byte lane i, channel
    32*p + 4*r + i with r = (8/w)*j + m, where j is the word's index inside part p (w words per part)."""
    D = 128
    rng = np.random.default_rng(7)
    for B in (1, 2, 4, 8, 3, 5, 6, 7):
        codes = rng.integers(0, 2**B, D).astype(np.uint8)
        words = oracle.pack_token(codes, B).view("<u4")
        base = 0
        rebuilt = np.zeros(D, np.uint32)
        for w in (8, 4, 2, 1):
            if not (B & w):
                continue
            shift = B & (w - 1)
            per = 8 // w
            for p in range(D // 32):
                for j in range(w):
                    word = int(words[base + p * w + j])
                    for m in range(per):
                        lanes = (word >> (w * m)) & (0x01010101 * (2**w - 1))
                        for i in range(4):
                            f = (lanes >> (8 * i)) & 0xFF
                            rebuilt[32 * p + 4 * (per * j + m) + i] |= f << shift
            base += (D // 32) * w
        assert np.array_equal(rebuilt.astype(np.uint8), codes)


def test_stream_offsets_are_prefix_sums():
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=100)
    K, _ = synth.make_kv(wl)
    rng = np.random.default_rng(2)
    bits = rng.integers(2, 9, 100).astype(np.uint8)
    qt = oracle.quantize(K[0, 2].numpy().view(np.uint16), -3.0, 3.0, bits)
    assert np.array_equal(qt.off, np.concatenate([[0], np.cumsum(bits.astype(np.int64) * 64 // 8)]).astype(np.uint32))
    assert qt.stream.size == qt.off[-1]
    for t in (0, 13, 99):
        _, _, codes, _ = oracle.token_codes(K[0, 2, t].numpy().view(np.uint16), -3.0, 3.0, int(bits[t]))
        assert np.array_equal(oracle.unpack_token(qt.stream[qt.off[t]: qt.off[t + 1]], 64, int(bits[t])), codes)


# ---------------------------------------------------------------- attention window
def test_window_max_and_unknown_scores():
    rng = np.random.default_rng(4)
    ring = rng.random((5, 40)).astype(np.float32)
    nv = rng.integers(0, 6, 40).astype(np.uint8)
    got = oracle.window_max(ring, nv)
    for t in range(40):
        if nv[t] == 0:
            assert np.isinf(got[t])
        else:
            assert got[t] == ring[: nv[t], t].max()
    # window of one row = the current score itself ("no window")
    assert np.array_equal(oracle.window_max(ring[:1], np.ones(40, np.uint8)), ring[0])


# ---------------------------------------------------------------- attention
def test_attention_matches_torch_softmax_attention_fp64():
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=300)
    K, V = synth.make_kv(wl)
    q = synth.make_query(wl)
    k = K[0, 1].numpy().view(np.uint16); v = V[0, 1].numpy().view(np.uint16)
    bits = np.random.default_rng(0).integers(2, 9, 300).astype(np.uint8)
    lo, hi = oracle.thresholds(k, 0.01)
    qk = oracle.quantize(k, lo, hi, bits)
    lo, hi = oracle.thresholds(v, 0.01)
    qv = oracle.quantize(v, lo, hi, bits[::-1].copy())
    scale = 1 / math.sqrt(64)
    X, S = oracle.decode(q[0, 1].numpy().view(np.uint16), qk, qv, scale)
    Kh = torch.from_numpy(oracle.reconstruct(qk)).double()
    Vh = torch.from_numpy(oracle.reconstruct(qv)).double()
    qq = q[0, 1].double()[None, None, None, :]
    ref = torch.nn.functional.scaled_dot_product_attention(qq, Kh[None, None], Vh[None, None], scale=scale)[0, 0, 0]
    assert np.allclose(X, ref.numpy(), rtol=1e-12, atol=1e-13)
    assert S.sum() == pytest.approx(1.0, abs=1e-12)
    Sref = torch.softmax((Kh @ q[0, 1].double()) * scale, 0).numpy()
    assert np.allclose(S, Sref, rtol=1e-12, atol=1e-15)
    # splitting T and merging the halves by log-sum-exp gives the same result
    h = 170
    def part(a, b):
        logit = (Kh[a:b] @ q[0, 1].double()).numpy() * scale
        m = logit.max(); p = np.exp(logit - m)
        return m, p.sum(), p @ Vh[a:b].numpy()
    m1, l1, a1 = part(0, h); m2, l2, a2 = part(h, 300)
    M = max(m1, m2)
    merged = (a1 * math.exp(m1 - M) + a2 * math.exp(m2 - M)) / (l1 * math.exp(m1 - M) + l2 * math.exp(m2 - M))
    assert np.allclose(X, merged, rtol=1e-12, atol=1e-13)


def test_eight_bit_cache_is_close_to_fp16_attention():
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=256)
    K, V = synth.make_kv(wl); q = synth.make_query(wl)
    k = K[0, 0].numpy().view(np.uint16); v = V[0, 0].numpy().view(np.uint16); qq = q[0, 0].numpy().view(np.uint16)
    bits = np.full(256, 8, np.uint8)
    lo, hi = oracle.thresholds(k, 0.01); qk = oracle.quantize(k, lo, hi, bits)
    lo, hi = oracle.thresholds(v, 0.01); qv = oracle.quantize(v, lo, hi, bits)
    X, S = oracle.decode(qq, qk, qv, 0.125)
    X0, S0 = oracle.attention_fp16(qq, k, v, 0.125)
    # first-order bound from dX_j/dV_tj = S_t: |dX_j| <= sum_t S_t * Delta_t (+ the key-side term, also small)
    assert np.max(np.abs(X - X0)) < 0.05 and np.sum((S - S0) ** 2) < 1e-3
    b2 = np.full(256, 2, np.uint8)
    X2, _ = oracle.decode(qq, oracle.quantize(k, *oracle.thresholds(k, 0.01), b2),
                          oracle.quantize(v, *oracle.thresholds(v, 0.01), b2), 0.125)
    assert np.sum((X2 - X0) ** 2) > np.sum((X - X0) ** 2)


# ---------------------------------------------------------------- accounting
def test_compression_ratio_from_bit_counts_two_ways():
    rng = np.random.default_rng(9)
    T, D = 200, 128
    bK = rng.integers(2, 9, T).astype(np.uint8); bV = rng.integers(2, 9, T).astype(np.uint8)
    wl = synth.scaled(synth.CONFIGS["C2"], heads=1, tokens=T)
    K, V = synth.make_kv(wl)
    k = K[0, 0].numpy().view(np.uint16); v = V[0, 0].numpy().view(np.uint16)
    qk = oracle.quantize(k, *oracle.thresholds(k, 0.01), bK)
    qv = oracle.quantize(v, *oracle.thresholds(v, 0.01), bV)
    cbk, cbv = oracle.code_bits(bK, D), oracle.code_bits(bV, D)
    assert cbk == 8 * qk.stream.size and cbv == 8 * qv.stream.size        # histogram vs stream length
    cr = oracle.cr_paper(cbk, cbv, qk.ch.size, qv.ch.size, T, D)
    assert cr == pytest.approx(32 * T * D / (8 * (qk.stream.size + qv.stream.size) + 16 * (qk.ch.size + qv.ch.size)))
    # uniform 4-bit, no outliers: exactly 16/4
    assert oracle.cr_paper(4 * T * D, 4 * T * D, 0, 0, T, D) == 4.0


# ---------------------------------------------------------------- batch runner
def test_batch_runner_equals_single_calls_and_threads_agree():
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=96)
    K, V = synth.make_kv(wl); q = synth.make_query(wl); ring, nv = synth.make_score_ring(wl, ragged=True)
    k = K.numpy().view(np.uint16).reshape(4, 96, 64); v = V.numpy().view(np.uint16).reshape(4, 96, 64)
    qq = q.numpy().view(np.uint16).reshape(4, 64)
    cK, cV = oracle.policy(0.03, 0.035, 70.0, 96)
    kw = dict(alpha=0.01, cK=cK, cV=cV, bmin=2, bmax=8, scale=0.125)
    r1 = oracle.run_batch(k, v, qq, ring.numpy().reshape(4, 5, 96), nv.numpy().reshape(4, 96), n_threads=1, **kw)
    r3 = oracle.run_batch(k, v, qq, ring.numpy().reshape(4, 5, 96), nv.numpy().reshape(4, 96), n_threads=3, **kw)
    assert r3.threads == 3 and np.array_equal(r1.X, r3.X) and np.array_equal(r1.bitsV, r3.bitsV)
    i = 2
    lo, hi = oracle.thresholds(k[i], 0.01)
    assert (r1.thr[i, 0], r1.thr[i, 1]) == (lo, hi)
    bK, bV = oracle.select_bits(k[i], v[i], r1.thr[i], ring.numpy()[0, i], nv.numpy()[0, i], cK, cV, 2, 8)
    assert np.array_equal(bK, r1.bitsK[i]) and np.array_equal(bV, r1.bitsV[i])
    assert len(set(bK.tolist())) >= 2 and len(set(bV.tolist())) >= 3
    qt = oracle.quantize(k[i], lo, hi, bK)
    assert np.array_equal(qt.stream, r1.K[i].stream) and np.array_equal(qt.val, r1.K[i].val)


# ---- further quantization to lower widths (Section 4.2, integration in the generation process)
def _requant_case(seed, T=40, D=64):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((T, D)) * rng.lognormal(0, 0.5, (1, D))).astype(np.float16)
    x[rng.random((T, D)) < 0.02] *= 12                       # a few entries beyond the thresholds
    x[3] = x[3, 0]                                           # a constant token
    xu = x.view(np.uint16)
    lo, hi = oracle.thresholds(xu, 0.02)
    bits = rng.integers(1, 9, T).astype(np.uint8)
    return xu, lo, hi, bits, rng


def test_requantize_down_equals_quantizing_the_original_at_the_lower_width():
    # independent route to the same result: quantize the binary16 values directly at min(old, requested)
    for seed in range(4):
        xu, lo, hi, bits, rng = _requant_case(seed)
        req = rng.integers(0, 10, bits.size).astype(np.uint8)            # 0 is treated as 1; 9 is above every width
        got = oracle.requantize_down(oracle.quantize(xu, lo, hi, bits), req)
        want_bits = np.minimum(bits, np.maximum(req, 1)).astype(np.uint8)
        want = oracle.quantize(xu, lo, hi, want_bits)
        assert np.array_equal(got.bits, want_bits)
        assert np.array_equal(got.step.view(np.uint32), want.step.view(np.uint32))
        assert np.array_equal(got.mn.view(np.uint32), want.mn.view(np.uint32))
        assert np.array_equal(got.off, want.off) and np.array_equal(got.stream, want.stream)
        assert np.array_equal(got.rowptr, want.rowptr) and np.array_equal(got.ch, want.ch) and np.array_equal(got.val, want.val)
        assert (want_bits < bits).any() and (want_bits == bits).any()


def test_requantize_down_drops_low_code_bits_and_never_raises_a_width():
    xu, lo, hi, bits, rng = _requant_case(11)
    q0 = oracle.quantize(xu, lo, hi, bits)
    same = oracle.requantize_down(q0, np.full(bits.size, 8, np.uint8))   # nothing to lower
    assert np.array_equal(same.bits, q0.bits) and np.array_equal(same.stream, q0.stream) and np.array_equal(same.step, q0.step)
    req = np.full(bits.size, 2, np.uint8)
    q1 = oracle.requantize_down(q0, req)
    for t in range(q0.T):
        B, Bn = int(q0.bits[t]), int(q1.bits[t])
        assert Bn == min(B, 2)
        c0 = oracle.unpack_token(q0.stream[q0.off[t]:q0.off[t + 1]], q0.D, B)
        c1 = oracle.unpack_token(q1.stream[q1.off[t]:q1.off[t + 1]], q1.D, Bn)
        assert np.array_equal(c1, c0 >> (B - Bn))
        assert q1.step[t] == q0.step[t] * 2.0 ** (B - Bn)
    # reconstruction error grows with the dropped bits but stays inside half a (new) step
    x = xu.view(np.float16).astype(np.float64)
    inl = (x >= lo) & (x <= hi)
    err = np.abs(oracle.reconstruct(q1).astype(np.float64) - x)
    assert np.all(err[inl] <= (0.5 * q1.step.astype(np.float64)[:, None] * np.ones_like(x))[inl] * (1 + 1e-3) + 1e-6)
    assert np.all(err[~inl] == 0)                                         # outliers stay exact


def test_reselect_from_stored_form_equals_selection_on_the_original_values():
    rng = np.random.default_rng(3)
    T, D, W = 48, 64, 6
    K = (rng.standard_normal((T, D)) * 1.5).astype(np.float16).view(np.uint16)
    V = (rng.standard_normal((T, D)) * 0.7).astype(np.float16).view(np.uint16)
    thr = (*oracle.thresholds(K, 0.02), *oracle.thresholds(V, 0.02))
    ring = rng.random((W, T)).astype(np.float32) * 0.05
    nvalid = rng.integers(0, W + 1, T).astype(np.uint8)
    cK, cV = oracle.policy(0.03, 0.035, 70.0, T)
    bK, bV = oracle.select_bits(K, V, np.array(thr, np.float32), ring, nvalid, cK, cV, 2, 8)
    top = np.full(T, 8, np.uint8)                                         # stored at the top width
    qk, qv = oracle.quantize(K, thr[0], thr[1], top), oracle.quantize(V, thr[2], thr[3], top)
    assert np.array_equal(oracle.reselect_bits(qk, False, None, None, cK, 2, 8), bK)
    assert np.array_equal(oracle.reselect_bits(qv, True, ring, nvalid, cV, 2, 8), bV)
    assert len(set(bK.tolist()) | set(bV.tolist())) >= 3


def test_prefill_window_rows_are_causal_softmax_rows_newest_first():
    rng = np.random.default_rng(8)
    T, n, D = 37, 5, 32
    Q = rng.standard_normal((n, D)).astype(np.float16); K = rng.standard_normal((T, D)).astype(np.float16)
    scale = 1.0 / math.sqrt(D)
    ring, nvalid, qn2 = oracle.prefill_window(Q.view(np.uint16), K.view(np.uint16), scale)
    logits = torch.from_numpy(Q.astype(np.float64)) @ torch.from_numpy(K.astype(np.float64)).T * scale   # [n, T]
    for i in range(n):
        vis = T - n + i + 1
        want = torch.softmax(logits[i, :vis], dim=0).numpy()
        row = ring[n - 1 - i]
        assert np.allclose(row[:vis], want, rtol=1e-12, atol=1e-15) and np.all(row[vis:] == 0)
    for t in range(T):                                   # the rows holding token t are exactly 0..nvalid[t]-1
        assert np.all(ring[: nvalid[t], t] > 0) and np.all(ring[nvalid[t]:, t] == 0)
    assert np.allclose(qn2, (Q.astype(np.float64) ** 2).sum(1) * scale * scale)
    # feeds the window maximum like any other ring
    shat = oracle.window_max(ring.astype(np.float32), nvalid)
    assert np.allclose(shat, ring.astype(np.float32).max(axis=0))


# ----------------------------------------------------------------------------- squared query norm quantile
def test_qnorm2_quantile_closed_form_counts_and_nans():
    """Section 4.1, end of "Key cache quantization": the upper 10 % quantile of the squared query norms.  Pinned by a
    closed form (1..100: ten values lie above 90), by the counting rule on random data with ties (at most frac*N
    values above the result, more than frac*N at or above it), by a plain Python sort, and by NaNs being left out."""
    assert oracle.qnorm2_quantile(np.arange(1, 101, dtype=np.float32), 0.1) == 90.0
    assert oracle.qnorm2_quantile(np.arange(1, 101, dtype=np.float32)[::-1].copy(), 0.1) == 90.0
    assert oracle.qnorm2_quantile(np.array([3.0], dtype=np.float32), 0.1) == 3.0
    assert oracle.qnorm2_quantile(np.array([], dtype=np.float32), 0.1) == 0.0
    rng = np.random.default_rng(5)
    for n, frac in ((10, 0.1), (37, 0.1), (1000, 0.1), (1000, 0.25), (513, 0.0)):
        v = np.round(rng.chisquare(8, size=n), 1).astype(np.float32)        # rounded: many ties
        q = oracle.qnorm2_quantile(v, frac)
        above, at_or_above = int(np.count_nonzero(v > q)), int(np.count_nonzero(v >= q))
        assert above <= frac * n < at_or_above
        k = int(math.floor(frac * n))
        assert q == sorted(float(x) for x in v)[n - 1 - k]
    v = np.array([np.nan, 1.0, -np.nan, 5.0, 2.0, np.nan, 4.0, 3.0], dtype=np.float32)
    assert oracle.qnorm2_quantile(v, 0.2) == 4.0                            # five values count: sorted[5-1-1]
    assert oracle.qnorm2_quantile(np.full(4, np.nan, dtype=np.float32), 0.1) == 0.0
