"""Pins for the CPU oracle: each oracle function is checked against something
other than itself -- the constants the paper states, closed forms, brute force
on tiny inputs, and library routines on special cases."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import vidkv_oracle as O
from workloads import CONFIGS, make_layer_kv, make_saliency

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


def rng(seed=0):
    return np.random.default_rng(seed)


def fp16_values(shape, seed=0, scale=1.0):
    return (rng(seed).standard_normal(shape) * scale).astype(np.float16).astype(np.float32)


# ------------------------------------------------------------------ constants
def test_paper_constants():
    assert O.G == GOLD["group_size_G"]["value"]
    assert O.R == GOLD["residual_length_R"]["value"]
    assert float(O.GAMMA) == pytest.approx(GOLD["gamma"]["value"], abs=1e-7)


def test_bit_accounting():
    k = fp16_values((64, 128), 1)
    abn, nom = O.select_channels(k, 0.5)
    assert len(abn) == 64 and len(nom) == 64
    assert (2 * len(abn) + 1 * len(nom)) / 128 == GOLD["key_bits_at_k_0p5"]["value"]
    abn75, nom75 = O.select_channels(k, 0.75)
    assert (2 * len(abn75) + len(nom75)) / 128 == GOLD["key_bits_at_k_0p75"]["value"]
    # ternary information content and the p = 0.2 mix
    assert round(math.log2(3), 2) == GOLD["value_bits_ternary"]["value"]
    assert round(0.2 * 2 + 0.8 * 1.58, 2) == GOLD["value_bits_at_p_0p2"]["value"]
    # 5 trits fit one byte
    assert 3 ** 5 <= 256 < 3 ** 6


def test_alphabets():
    x = fp16_values((32, 16), 2)
    q, _, _ = O.gquant(x, 2)
    assert set(np.unique(q)) <= set(GOLD["two_bit_alphabet"]["value"])
    b, _ = O.fft_1bit(fp16_values((32, 64), 3))
    assert set(np.unique(b)) <= set(GOLD["one_bit_alphabet"]["value"])
    t, _ = O.quant_1p58(x)
    assert set(np.unique(t)) <= set(GOLD["ternary_alphabet"]["value"])
    assert set(np.unique(t)) == {-1, 0, 1}


# ------------------------------------------------------------------ Eq. 4
@pytest.mark.parametrize("bits", [1, 2, 4])
def test_gquant_extremes_and_error_bound(bits):
    x = fp16_values((32, 40), 4, scale=3.0)
    q, s, z = O.gquant(x, bits)
    lv = 2 ** bits - 1
    xd = O.gdequant(q, s, z)
    amin, amax = x.argmin(0), x.argmax(0)
    cols = np.arange(x.shape[1])
    assert (q[amin, cols] == 0).all()
    assert (q[amax, cols] == lv).all()
    # the group minimum is reproduced exactly (z = min, code 0)
    assert (xd[amin, cols] == x.min(0).astype(np.float64)).all()
    # every element within half a step (+ the binary16 rounding of s over lv steps)
    s64 = s.astype(np.float64)
    bound = s64 / 2 + lv * s64 * 2.0 ** -11 + 1e-12
    assert (np.abs(xd - x) <= bound[None, :]).all()


def test_gquant_is_nearest_level_bruteforce():
    # code = argmin_j |x - (z + j s)| wherever that argmin is not a near-tie
    x = fp16_values((7, 50), 5, scale=2.0)
    q, s, z = O.gquant(x, 2)
    s64, z64 = s.astype(np.float64), z.astype(np.float64)
    levels = z64[None, None, :] + np.arange(4)[:, None, None] * s64[None, None, :]
    dist = np.abs(x[None].astype(np.float64) - levels)           # [4, n, C]
    best = dist.argmin(0)
    srt = np.sort(dist, axis=0)
    clear = (srt[1] - srt[0]) > 1e-3 * s64[None, :]
    assert clear.mean() > 0.99
    assert (q[clear] == best[clear]).all()


def test_gquant_constant_group_exact():
    x = np.full((32, 5), np.float32(np.float16(1.2345)))
    q, s, z = O.gquant(x, 2)
    assert (q == 0).all() and (s == 0).all()
    assert (O.gdequant(q, s, z) == x).all()


def test_gquant_known_values():
    # hand-computed: column {0, 1, 2, 3} -> s = 1, z = 0, codes 0..3;
    # column {-1, -0.5, 0.5, 2} -> s = 1, z = -1, (x - z)/s = 0, .5, 1.5, 3 -> half-to-even 0, 0, 2, 3
    x = np.array([[0, -1.0], [1, -0.5], [2, 0.5], [3, 2.0]], dtype=np.float32)
    q, s, z = O.gquant(x, 2)
    assert s.tolist() == [1.0, 1.0] and z.tolist() == [0.0, -1.0]
    assert q[:, 0].tolist() == [0, 1, 2, 3]
    assert q[:, 1].tolist() == [0, 0, 2, 3]


def test_gquant_groups_are_independent():
    x = fp16_values((70, 6), 6)
    q, s, z = O.gquant_groups(x, 2)
    assert s.shape == (3, 6)
    for g, sl in enumerate([slice(0, 32), slice(32, 64), slice(64, 70)]):
        qg, sg, zg = O.gquant(x[sl], 2)
        assert (q[sl] == qg).all() and (s[g] == sg).all() and (z[g] == zg).all()


# ------------------------------------------------------------------ channel selection
def test_select_channels_matches_sort_and_is_permutation_invariant():
    k = fp16_values((96, 128), 7) * (1 + np.arange(128, dtype=np.float32)[None, :] % 5)
    abn, nom = O.select_channels(k, 0.5)
    r = k.max(0) - k.min(0)
    ref = np.sort(np.lexsort((np.arange(128), -r))[:64])
    assert (abn == ref).all()
    assert sorted(set(abn) | set(nom)) == list(range(128)) and not (set(abn) & set(nom))
    perm = rng(8).permutation(96)
    abn2, _ = O.select_channels(k[perm], 0.5)
    assert (abn2 == abn).all()


def test_channel_variance_and_outliers():
    k = fp16_values((200, 6), 71, scale=3.0)
    var = O.channel_variance(k)
    np.testing.assert_allclose(var, np.var(k.astype(np.float64), axis=0), rtol=1e-12)     # library routine
    for c in range(6):                                                                        # brute force
        col = [float(x) for x in k[:, c]]
        m = sum(col) / len(col)
        assert var[c] == pytest.approx(sum((x - m) ** 2 for x in col) / len(col), rel=1e-12)
    # closed forms: a constant channel has variance 0, +-a alternating has a^2; a shift changes nothing
    z = np.zeros((64, 2), np.float32)
    z[:, 0] = 1.5
    z[0::2, 1], z[1::2, 1] = 2.0, -2.0
    assert O.channel_variance(z).tolist() == [0.0, 4.0]
    np.testing.assert_allclose(O.channel_variance(k + 7.0), var, rtol=1e-9)
    # outliers: element by element, M = 3 (the paper's setting)
    out = O.channel_outliers(k)
    for c in range(6):
        a = [abs(float(x)) for x in k[:, c]]
        assert out[c] == sum(1 for x in a if x > 3.0 * (sum(a) / len(a)))
    # planted: 5 values of 100 among 995 ones -> mean |K| = 1.495, threshold 4.485, exactly the 5 planted ones count
    p = np.ones((1000, 1), np.float32)
    p[::200, 0] = -100.0
    assert O.channel_outliers(p)[0] == 5
    assert O.channel_outliers(np.ones((50, 3), np.float32)).tolist() == [0, 0, 0]


def test_select_channels_tie_break():
    k = np.zeros((4, 8), dtype=np.float32)
    k[0, :] = 1.0           # all ranges equal -> lowest indices win
    abn, nom = O.select_channels(k, 0.5)
    assert abn.tolist() == [0, 1, 2, 3] and nom.tolist() == [4, 5, 6, 7]
    k[1, 6] = 5.0           # channel 6 has the largest range
    abn, _ = O.select_channels(k, 0.5)
    assert abn.tolist() == [0, 1, 2, 6]


def test_planted_outlier_channels_are_selected():
    from workloads.synth import _outlier_channels
    cfg = CONFIGS["tiny"]
    K, _ = make_layer_kv(cfg, 0)
    ids, _ = _outlier_channels(cfg, 0)
    for h in range(4):
        abn, _ = O.select_channels(K[0, h].float().numpy(), 0.5)
        assert set(ids[h].tolist()) <= set(abn.tolist())


# ------------------------------------------------------------------ DFT
def test_dft_matches_library_and_roundtrip():
    x = rng(9).standard_normal((5, 64))
    xf = O.dft64(x)
    assert np.allclose(xf, np.fft.fft(x, norm="ortho"), atol=1e-12)
    assert np.allclose(O.idft64(xf).real, x, atol=1e-12)        # FFT -> IFFT restores the input
    assert np.abs(O.idft64(xf).imag).max() < 1e-12
    assert np.allclose((np.abs(xf) ** 2).sum(-1), (x ** 2).sum(-1))   # Parseval (orthonormal)


def test_dft_closed_forms():
    imp = np.zeros(64); imp[0] = 1.0
    assert np.allclose(O.dft64(imp), np.full(64, 1 / 8))         # impulse -> flat 1/sqrt(64)
    const = np.ones(64)
    ref = np.zeros(64, dtype=complex); ref[0] = 8.0               # constant -> DC only, sqrt(64)
    assert np.allclose(O.dft64(const), ref, atol=1e-12)
    m = np.arange(64)
    tone = np.cos(2 * np.pi * 3 * m / 64)
    ref = np.zeros(64, dtype=complex); ref[3] = ref[61] = 4.0     # cosine at bin 3 -> 8/2 at +-3
    assert np.allclose(O.dft64(tone), ref, atol=1e-12)
    stone = np.sin(2 * np.pi * 5 * m / 64)
    ref = np.zeros(64, dtype=complex); ref[5] = -4.0j; ref[59] = 4.0j   # forward sign convention
    assert np.allclose(O.dft64(stone), ref, atol=1e-12)


# ------------------------------------------------------------------ Eq. 5
def test_fft_1bit_definition_and_hermitian_packing():
    x = fp16_values((32, 64), 10)
    bits, s = O.fft_1bit(x)
    xf = np.fft.fft(x.astype(np.float64), norm="ortho")
    cols = np.concatenate([xf.real, xf.imag], -1)
    far = np.abs(cols) > 1e-9
    assert (bits[far] == (cols[far] > 0)).all()
    assert np.allclose(s.astype(np.float64), np.abs(cols).mean(0), rtol=2.0 ** -11, atol=1e-7)
    # mirrored bins: equal real part (same bit, same scale); imaginary part flips sign
    for k in range(1, 32):
        assert (bits[:, k] == bits[:, 64 - k]).all() and s[k] == s[64 - k]
        assert (bits[:, 64 + k] != bits[:, 128 - k]).all() and s[64 + k] == s[128 - k]
    assert s[64] == 0 and s[64 + 32] == 0                    # Im of DC and Nyquist vanish
    # so the dequantized signal is real, and the 64 packed columns determine it
    xr, imag_max = O.fft_1bit_dequant(bits, s)
    assert imag_max < 1e-9
    pk = O.hermitian_pack_columns(64)
    assert len(pk) == 64 and len(set(pk.tolist())) == 64
    vals = (2.0 * bits[:, pk] - 1.0) * s[pk].astype(np.float64)
    half = np.zeros((32, 33), dtype=complex)
    half[:, 0] = vals[:, 0]
    half[:, 32] = vals[:, 1]
    half[:, 1:32] = vals[:, 2::2] + 1j * vals[:, 3::2]
    assert np.allclose(np.fft.irfft(half, n=64, norm="ortho"), xr, atol=1e-9)


def test_one_bit_code_is_l2_optimal_bruteforce():
    # min over b in {+-1}^n, a >= 0 of ||x - a b||^2 is attained at b = sign(x), a = mean|x|
    x = rng(11).standard_normal(7)
    best = None
    for b in itertools.product([-1.0, 1.0], repeat=7):
        b = np.array(b)
        a = max(0.0, float(b @ x) / 7)
        err = float(((x - a * b) ** 2).sum())
        if best is None or err < best[0]:
            best = (err, b, a)
    assert (best[1] == np.sign(x)).all()
    assert best[2] == pytest.approx(np.abs(x).mean())
    # the oracle's per-column code is exactly that choice (up to binary16 rounding of s)
    X = fp16_values((32, 64), 12)
    bits, s = O.fft_1bit(X)
    cols = np.concatenate([O.dft64(X).real, O.dft64(X).imag], -1)
    deq = (2.0 * bits - 1) * s.astype(np.float64)
    live = s > 0
    assert np.allclose(np.abs(deq).mean(0)[live], s[live].astype(np.float64))
    inner = (deq * cols).sum(0)[live]
    assert np.allclose(inner, 32 * s[live].astype(np.float64) * np.abs(cols).mean(0)[live], rtol=1e-9)


def test_fft_1bit_group_and_token_independence():
    # the transform is per token: permuting tokens inside a group permutes bits, keeps scales
    x = fp16_values((32, 64), 13)
    bits, s = O.fft_1bit(x)
    perm = rng(14).permutation(32)
    bits2, s2 = O.fft_1bit(x[perm])
    assert (bits2 == bits[perm]).all() and (s2 == s).all()


# ------------------------------------------------------------------ MixQuant
def test_mixquant_structure_and_dequant():
    cfg = CONFIGS["tiny"]
    K, _ = make_layer_kv(cfg, 0, T=160)
    k = K[0, 1].float().numpy()
    mq = O.mixquant(k, 0.5)
    assert mq["codes2"].shape == (160, 64) and mq["bits1"].shape == (160, 128)
    assert mq["s2"].shape == (5, 64) and mq["s1"].shape == (5, 128)
    kd = O.mixquant_dequant(mq)
    # 2-bit channels: independent GQuant per column
    assert np.allclose(kd[:, mq["abn_idx"]],
                       O.gdequant_groups(*O.gquant_groups(k[:, mq["abn_idx"]], 2)))
    # 1-bit channels: the reconstruction lies in the span and beats the zero signal
    nom = mq["nom_idx"]
    err = ((kd[:, nom] - k[:, nom]) ** 2).sum()
    assert err < (k[:, nom] ** 2).sum()
    # and the 2-bit outlier channels reconstruct much better than the 1-bit ones, relatively
    abn = mq["abn_idx"]
    rel_abn = ((kd[:, abn] - k[:, abn]) ** 2).sum() / (k[:, abn] ** 2).sum()
    rel_nom = err / (k[:, nom] ** 2).sum()
    assert rel_abn < rel_nom


def test_mixquant_dequant_scatters_a_hand_built_chunk_to_its_channels():
    """DeQuant of a chunk written by hand, against closed forms: the anomalous channels are a constant
    (s = 0, so every code dequantizes to z), the normal channels hold a spectrum with a single real
    bin k0 (every other column has scale 0), i.e. a cosine over the normal channels in ascending
    channel order, which numpy's inverse real FFT gives independently.  Two groups with different
    amplitudes and per-token signs catch a transposed or mis-scattered result."""
    T, k0 = 40, 5                                             # one full group and a short one
    r = rng(77)
    abn = np.sort(r.permutation(128)[:64])
    nom = np.setdiff1d(np.arange(128), abn)
    z2 = np.stack([np.linspace(-3, 3, 64), np.linspace(5, -5, 64)]).astype(np.float16)
    amp = np.array([2.0, 0.75])
    s1 = np.zeros((2, 128), dtype=np.float16)
    s1[:, k0] = amp; s1[:, 64 - k0] = amp                      # Re X[k0] and its mirror bin
    sign = r.integers(0, 2, size=T)
    bits1 = np.zeros((T, 128), dtype=np.uint8)
    bits1[:, k0] = sign; bits1[:, 64 - k0] = sign
    mq = dict(T=T, abn_idx=abn, nom_idx=nom, codes2=np.zeros((T, 64), dtype=np.int8),
              s2=np.zeros((2, 64), dtype=np.float16), z2=z2, bits1=bits1, s1=s1)
    kd = O.mixquant_dequant(mq)
    assert kd.shape == (T, 128)
    for t in range(T):
        g = t // 32
        assert np.array_equal(kd[t, abn], z2[g].astype(np.float64))
        spec = np.zeros(33)
        spec[k0] = (2 * sign[t] - 1) * amp[g]
        want = np.fft.irfft(spec, n=64, norm="ortho")        # = +-(amp / 4) cos(2 pi k0 n / 64)
        assert np.allclose(kd[t, nom], want, atol=1e-12)
        assert np.allclose(want, (2 * sign[t] - 1) * amp[g] / 4 * np.cos(2 * np.pi * k0 * np.arange(64) / 64), atol=1e-12)


def test_dequant_1p58_groups_closed_form():
    """trit * s per (32-token group, channel): hand values, with a short second group."""
    trits = np.zeros((33, 3), dtype=np.int8)
    trits[0] = [1, 0, -1]
    trits[31] = [-1, -1, 1]
    trits[32] = [1, -1, 0]
    s = np.array([[2.0, 7.0, 0.5], [3.0, 0.25, 9.0]], dtype=np.float16)
    out = O.dequant_1p58_groups(trits, s)
    assert out.shape == (33, 3)
    assert np.array_equal(out[0], [2.0, 0.0, -0.5])
    assert np.array_equal(out[31], [-2.0, -7.0, 0.5])
    assert np.array_equal(out[32], [3.0, -0.25, 0.0])         # the second group's scales
    assert np.count_nonzero(out[1:31]) == 0


def test_mixquant_chunks_do_not_see_each_other():
    k = fp16_values((64, 128), 15)
    k[:32, 5] *= 50            # channel 5 is anomalous only in the first half
    a = O.mixquant(k[:32], 0.5)
    b = O.mixquant(k[32:], 0.5)
    assert 5 in a["abn_idx"]
    whole = O.mixquant(k, 0.5)
    assert 5 in whole["abn_idx"]
    # selection is per chunk: computed from that chunk's tokens only
    assert (b["abn_idx"] == O.select_channels(k[32:], 0.5)[0]).all()


# ------------------------------------------------------------------ Eq. 6
def test_ternary_definition_and_symmetry():
    v = fp16_values((32, 128), 16)
    t, s = O.quant_1p58(v)
    mean_abs = np.abs(v.astype(np.float64)).mean(0)
    assert np.allclose(s.astype(np.float64), mean_abs, rtol=2.0 ** -11)
    alpha = 0.7 * s.astype(np.float64)
    clear = np.abs(np.abs(v) - alpha[None]) > 1e-3 * s.astype(np.float64)[None]
    expect = np.sign(v) * (np.abs(v) > alpha[None])
    assert (t[clear] == expect[clear]).all()
    assert ((t == 0) == ~((v > (np.float32(0.7) * s.astype(np.float32))[None]) |
                          (v < -(np.float32(0.7) * s.astype(np.float32))[None]))).all()
    t2, s2 = O.quant_1p58(-v)
    assert (t2 == -t).all() and (s2 == s).all()


def test_ternary_gamma_limits():
    v = fp16_values((32, 64), 17)
    t0, _ = O.quant_1p58(v, gamma=np.float32(0.0))
    assert (t0 == np.sign(v)).all()
    t_big, _ = O.quant_1p58(v, gamma=np.float32(100.0))
    assert (t_big == 0).all()


def test_ternary_nonzero_fraction_gaussian():
    # |v| > 0.7 E|v| for v ~ N(0,1): 2 (1 - Phi(0.7 sqrt(2/pi))) = 0.5765...
    v = fp16_values((32 * 400, 128), 18)
    t, _ = O.quant_1p58_groups(v)
    expect = math.erfc(0.7 * math.sqrt(2 / math.pi) / math.sqrt(2))
    assert expect == pytest.approx(0.5765, abs=1e-3)
    assert (t != 0).mean() == pytest.approx(expect, abs=5e-3)


def test_ternary_nonzero_mean_scale():
    v = fp16_values((32, 16), 61, scale=2.0)
    t, s = O.quant_1p58(v)
    t2, s2 = O.quant_1p58(v, scale="nonzero_mean")
    assert (t == t2).all()                                   # the codes do not depend on the stored scale
    # brute force per channel
    for c in range(16):
        vals = [abs(float(v[i, c])) for i in range(32) if t[i, c] != 0]
        want = np.float16(sum(vals) / len(vals)) if vals else np.float16(0)
        assert s2[c] == want
    # least squares: for fixed codes the unrounded non-zero mean minimises |v - s t|^2, so it cannot lose to Mean|v|
    vv, tt = v.astype(np.float64), t.astype(np.float64)
    nz = tt != 0
    s_opt = (np.abs(vv) * nz).sum(0) / np.maximum(nz.sum(0), 1)
    err_opt = ((vv - s_opt * tt) ** 2).sum(0)
    err_mean = ((vv - s.astype(np.float64) * tt) ** 2).sum(0)
    assert (err_opt <= err_mean + 1e-12).all()
    # closed form: equal magnitudes m with some zeros -> the non-zero mean is m itself
    w = np.zeros((32, 1), np.float32)
    w[:8, 0] = 3.0
    w[8:12, 0] = -3.0
    t3, s3 = O.quant_1p58(w, scale="nonzero_mean")
    assert t3[:8, 0].tolist() == [1] * 8 and t3[8:12, 0].tolist() == [-1] * 4 and not t3[12:].any()
    assert float(s3[0]) == 3.0
    # a channel of zeros has no non-zero code: scale 0
    z = np.zeros((32, 2), np.float32)
    assert (O.quant_1p58(z, scale="nonzero_mean")[1] == 0).all()


def test_ternary_short_group_uses_present_elements():
    v = fp16_values((40, 4), 19)
    t, s = O.quant_1p58_groups(v)
    assert s.shape == (2, 4)
    assert np.allclose(s[1].astype(np.float64), np.abs(v[32:].astype(np.float64)).mean(0), rtol=2.0 ** -11)


# ------------------------------------------------------------------ token protection
def test_select_tokens_matches_argsort_and_counts():
    for name, n_expect in [("tiny", 313), ("llava", 1254), ("qwen", 2508), ("batched", 2508),
                           ("stress", 39200)]:
        assert O.n_protected(0.2, CONFIGS[name].l_v) == n_expect
    cfg = CONFIGS["tiny"]
    sal = make_saliency(cfg)[0].numpy()
    E = O.select_tokens(sal, 0.2, 0, cfg.T)
    assert E.sum() == 313 and not E[cfg.l_v:].any()
    ref = np.argsort(-sal, kind="stable")[:313]
    assert set(np.nonzero(E)[0].tolist()) == set(ref.tolist())
    assert O.select_tokens(sal, 0.0, 0, cfg.T).sum() == 0
    # ties: lower index first
    tie = np.array([1.0, 2.0, 2.0, 2.0, 0.0], dtype=np.float32)
    E = O.select_tokens(tie, 0.4, 3, 10)
    assert np.nonzero(E)[0].tolist() == [4, 5]


def test_stp_saliency_brute_force_and_closed_forms():
    r = rng(41)
    x_v = fp16_values((7, 12), 42)
    x_t = fp16_values((5, 12), 43)
    got = O.stp_saliency(x_v, x_t)
    # Eq. 7 element by element, then the row sums
    want = np.zeros(7)
    for i in range(7):
        for j in range(5):
            want[i] += sum(float(x_v[i, c]) * float(x_t[j, c]) for c in range(12))
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # text tokens that are unit vectors pick coordinates of the visual tokens
    e = np.zeros((3, 12), np.float32)
    e[0, 2] = e[1, 5] = e[2, 5] = 1.0
    np.testing.assert_allclose(O.stp_saliency(x_v, e), x_v[:, 2].astype(np.float64) + 2.0 * x_v[:, 5], rtol=0, atol=1e-12)
    # the order of the text tokens does not matter; the score is linear in the visual token
    np.testing.assert_allclose(O.stp_saliency(x_v, x_t[r.permutation(5)]), got, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O.stp_saliency(2.0 * x_v, x_t), 2.0 * got, rtol=1e-12, atol=1e-12)
    # a single text token: one matrix-vector product (library routine)
    np.testing.assert_allclose(O.stp_saliency(x_v, x_t[:1]), np.dot(x_v.astype(np.float64), x_t[0].astype(np.float64)),
                               rtol=1e-12, atol=1e-12)


def test_stp_saliency_ranks_planted_tokens_first():
    # visual tokens aligned with the text direction must come out on top of the ranking
    r = rng(44)
    d, l_v, l_t = 64, 200, 9
    direction = r.standard_normal(d)
    direction /= np.linalg.norm(direction)
    x_t = (direction[None, :] * r.uniform(1.0, 2.0, (l_t, 1)) + 0.01 * r.standard_normal((l_t, d))).astype(np.float32)
    x_v = (0.1 * r.standard_normal((l_v, d))).astype(np.float32)
    planted = np.sort(r.choice(l_v, 40, replace=False))
    x_v[planted] += 3.0 * direction[None, :].astype(np.float32)
    E = O.select_tokens(O.stp_saliency(x_v, x_t), 0.2, 0, l_v)
    assert np.array_equal(np.nonzero(E)[0], planted)


def test_stpquant_streams():
    v = fp16_values((96, 16), 20)
    E = np.zeros(96, dtype=bool)
    E[[3, 10, 11, 50, 95]] = True
    sq = O.stpquant(v, E)
    assert sq["codes2"].shape == (5, 16) and sq["trits"].shape == (91, 16)
    assert sq["st"].shape == (3, 16)           # 91 tokens -> groups of 32, 32, 27 in gathered order
    vd = O.stp_dequant(sq)
    assert np.allclose(vd[E], O.gdequant_groups(*O.gquant_groups(v[E], 2)))
    rest = v[~E]
    assert np.allclose(vd[~E], O.dequant_1p58_groups(*O.quant_1p58_groups(rest)))
    # protected tokens are reconstructed more precisely than ternary ones
    assert np.abs(vd[E] - v[E]).mean() < np.abs(vd[~E] - v[~E]).mean()
    # p = 0: STPQuant degenerates to 1.58Quant
    sq0 = O.stpquant(v, np.zeros(96, dtype=bool))
    t, s = O.quant_1p58_groups(v)
    assert (sq0["trits"] == t).all() and (sq0["st"] == s).all()


# ------------------------------------------------------------------ Eq. 3 / Algorithm 1
def test_attention_matches_library():
    q = rng(21).standard_normal((7, 128))
    K = rng(22).standard_normal((50, 128))
    V = rng(23).standard_normal((50, 128))
    out = O.attention(q, K, V, 1 / math.sqrt(128))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None])[0]
    assert np.allclose(out, ref.numpy(), atol=1e-12)
    # all-equal value rows -> that row, whatever the scores
    Vc = np.tile(V[:1], (50, 1))
    assert np.allclose(O.attention(q, K, Vc, 0.3), np.tile(V[:1], (7, 1)))
    # a huge logit on one key -> that key's value row
    K2 = K.copy(); K2[17] = q[2] * 100
    assert np.allclose(O.attention(q[2:3], K2, V, 1.0), V[17:18], atol=1e-9)


def test_prefill_residual_split_and_decode_against_library():
    cfg = CONFIGS["tiny"]
    K, V = make_layer_kv(cfg, 0, T=77)        # r = 77 % 32 = 13 tokens stay in the residual
    k, v = K[0, 0].float().numpy(), V[0, 0].float().numpy()
    c = O.SlabCache()
    c.prefill(k, v)
    assert c.n_quantized == 64 and c.k_res.shape[0] == 13 and c.v_res.shape[0] == 13
    assert (c.k_res == k[64:]).all() and (c.v_res == v[64:]).all()
    q = rng(24).standard_normal((7, 128))
    kn, vn = rng(25).standard_normal(128), rng(26).standard_normal(128)
    Kd, Vd = c.dequant_k(), c.dequant_v()
    out = c.decode_step(q, kn, vn)
    Kall = np.concatenate([Kd, k[64:], kn.astype(np.float32)[None]])
    Vall = np.concatenate([Vd, v[64:], vn.astype(np.float32)[None]])
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(Kall)[None], torch.from_numpy(Vall)[None])[0]
    assert np.allclose(out, ref.numpy(), atol=1e-10)
    assert c.k_res.shape[0] == 14


def test_residual_flush_after_R_tokens():
    cfg = CONFIGS["tiny"]
    K, V = make_layer_kv(cfg, 0, T=64)
    c = O.SlabCache()
    c.prefill(K[0, 0].float().numpy(), V[0, 0].float().numpy())
    g = rng(27)
    news = []
    for step in range(O.R):
        assert len(c.k_chunks) == 1 and c.k_res.shape[0] == step
        kn = g.standard_normal(128).astype(np.float16).astype(np.float32)
        vn = g.standard_normal(128).astype(np.float16).astype(np.float32)
        news.append((kn, vn))
        c.decode_step(g.standard_normal((7, 128)), kn, vn)
    # after R steps: one more 128-token chunk with its own channel split, empty residual
    assert len(c.k_chunks) == 2 and c.k_chunks[1]["T"] == 128
    assert c.k_res.shape[0] == 0 and c.v_res.shape[0] == 0 and len(c.v_flush) == 1
    kres = np.stack([a for a, _ in news])
    vres = np.stack([b for _, b in news])
    assert (c.k_chunks[1]["abn_idx"] == O.select_channels(kres, 0.5)[0]).all()
    t, s = O.quant_1p58_groups(vres)            # decode-time tokens: 1.58Quant, never protected
    assert (c.v_flush[0][0] == t).all() and (c.v_flush[0][1] == s).all()
    assert c.dequant_k().shape == (192, 128) and c.dequant_v().shape == (192, 128)
    # step R+1 attends over 192 quantized tokens + 1 residual token
    q = g.standard_normal((7, 128))
    Kd, Vd = c.dequant_k(), c.dequant_v()
    out = c.decode_step(q, news[0][0], news[0][1])
    ref = O.attention(q, np.concatenate([Kd, news[0][0][None]]),
                      np.concatenate([Vd, news[0][1][None]]), 1 / math.sqrt(128))
    assert np.allclose(out, ref)


def test_fft_1bit_codes_the_hermitian_half():
    # mirror bins follow from the half for any input ...
    x = fp16_values((32, 64), 81)
    bits, s = O.fft_1bit(x)
    for k in range(1, 32):
        assert (bits[:, 64 - k] == bits[:, k]).all() and (bits[:, 128 - k] == 1 - bits[:, 64 + k]).all()
        assert s[64 - k] == s[k] and s[128 - k] == s[64 + k]
    # ... so the dequantized spectrum is Hermitian and its inverse transform real, also when imaginary
    # coefficients are exactly zero (an input that is even in the channel index has a real spectrum):
    # coding each mirror bin by its own sign would give both the bit of +0 and leave an imaginary part
    e = np.zeros((32, 64), np.float32)
    e[:, 0] = fp16_values((32,), 82)
    e[:, 32] = fp16_values((32,), 83)
    for c in range(1, 32):
        e[:, c] = e[:, 64 - c] = fp16_values((32,), 84 + c)
    e[1] += x[1]                                   # one generic row so that the imaginary columns have a scale
    xr, imag_max = O.fft_1bit_dequant(*O.fft_1bit(e))
    assert imag_max <= 1e-12
    assert xr.shape == e.shape


def test_fft_smooths_one_bit_error_direction():
    # Direction of the paper's Fig. 5 only (its numbers come from a real model's
    # key channel): for tokens with a sharp outlier at a varying channel, sign coding in the
    # frequency domain loses less than sign coding in place.
    g = rng(28)
    x = g.standard_normal((32, 64)) * 0.1
    for t in range(32):                                    # one sharp spike per token, moving channel
        x[t, g.integers(0, 64)] += g.choice([-4.0, 4.0])
    x = x.astype(np.float16).astype(np.float32)
    bits, s = O.fft_1bit(x)
    xr, _ = O.fft_1bit_dequant(bits, s)
    err_fft = ((xr - x) ** 2).mean()
    plain = np.sign(x) * np.abs(x).mean(0)[None]
    err_plain = ((plain - x) ** 2).mean()
    assert err_fft < err_plain


def test_attention_over_token_shards_merges_to_the_whole():
    """Pins attention_partial / merge_partials to the plain definition: any cut of the token axis into
    shards (an empty one included) merges to Softmax(q K^T) V of the whole, and to torch's
    scaled_dot_product_attention."""
    import torch
    r = rng(91)
    q = r.standard_normal((7, 128)) * 2
    K = r.standard_normal((300, 128)) * 3          # logits spread over tens of units: the maxima matter
    V = r.standard_normal((300, 128))
    scale = 1.0 / np.sqrt(128.0)
    whole = O.attention(q, K, V, scale)
    for cuts in ([0, 300], [0, 1, 300], [0, 130, 130, 300], [0, 64, 200, 299, 300]):
        parts = [O.attention_partial(q, K[a:b], V[a:b], scale) for a, b in zip(cuts[:-1], cuts[1:])]
        assert np.allclose(O.merge_partials(parts), whole, rtol=1e-12, atol=1e-13)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q)[None], torch.from_numpy(K)[None],
                                                           torch.from_numpy(V)[None])[0].numpy()
    assert np.allclose(whole, ref, atol=1e-10)
    m, l, o = O.attention_partial(q, K[:0], V[:0], scale)
    assert np.isneginf(m).all() and (l == 0).all() and (o == 0).all()



# ------------------------------------------------------------------ other bit widths (Algorithm 3 with other k)
def test_bit_accounting_of_the_other_ratios():
    k = fp16_values((64, 128), 11)
    for ratio, key in ((0.25, "key_bits_at_k_0p25"), (1.0, "key_bits_at_k_1p0")):
        abn, nom = O.select_channels(k, ratio)
        assert len(abn) + len(nom) == 128 and not set(abn) & set(nom)
        assert (2 * len(abn) + len(nom)) / 128 == GOLD[key]["value"]
    for ratio in (0.25, 0.5, 0.75, 1.0):
        assert (O.one_bit_mode(ratio) == "fft") == (ratio in GOLD["fft_one_bit_ratios"]["value"])


def test_one_bit_minmax_is_the_two_level_code():
    # GQuant with n = 1 (Eq. 4): levels z = min and z + s = max; every element goes to the nearer one
    x = fp16_values((32, 24), 12, scale=3.0)
    q, s, z = O.gquant(x, 1)
    assert set(np.unique(q)) == {0, 1}
    s32, z32 = s.astype(np.float64), z.astype(np.float64)
    for c in range(x.shape[1]):
        col = x[:, c].astype(np.float64)
        assert q[col.argmin(), c] == 0 and q[col.argmax(), c] == 1
        nearer = (np.abs(col - (z32[c] + s32[c])) < np.abs(col - z32[c])).astype(np.int8)
        undecided = np.abs(np.abs(col - (z32[c] + s32[c])) - np.abs(col - z32[c])) < 1e-3 * s32[c]
        assert np.array_equal(q[:, c][~undecided], nearer[~undecided])
    d = O.gdequant(q, s, z)
    assert np.all(np.abs(d - x) <= 0.5 * s32 + np.abs(x) * 2.0 ** -10 + 1e-6)


@pytest.mark.parametrize("ratio,n_abn", [(0.25, 32), (0.5, 64), (0.75, 96)])
def test_mixquant_minmax_mode(ratio, n_abn):
    cfg = CONFIGS["tiny"]
    K, _ = make_layer_kv(cfg, 0, T=96)
    k = K[0, 2].float().numpy()
    mq = O.mixquant(k, ratio, one_bit="minmax")
    assert mq["mode"] == "minmax" and len(mq["abn_idx"]) == n_abn and len(mq["nom_idx"]) == 128 - n_abn
    assert mq["codes1"].shape == (96, 128 - n_abn) and mq["s1"].shape == (3, 128 - n_abn) == mq["z1"].shape
    kd = O.mixquant_dequant(mq)
    nom, abn = mq["nom_idx"], mq["abn_idx"]
    # normal channels: every dequantized element is one of the group's two levels, which are the
    # binary16 roundings of the group's minimum and of minimum + (maximum - minimum)
    for g in range(3):
        blk = k[32 * g:32 * g + 32][:, nom]
        lo = blk.min(axis=0).astype(np.float16).astype(np.float64)
        rng_h = (blk.max(axis=0) - blk.min(axis=0)).astype(np.float16).astype(np.float64)
        got = kd[32 * g:32 * g + 32][:, nom]
        assert np.all((got == lo) | (got == lo + rng_h))
        assert np.all(np.abs(got - blk) <= 0.5 * rng_h + np.abs(blk) * 2.0 ** -10 + 1e-6)
    # anomalous channels are untouched by the mode
    ref = O.mixquant(k, ratio, one_bit="fft")
    assert np.array_equal(ref["abn_idx"], abn) and np.array_equal(ref["codes2"], mq["codes2"])
    assert np.array_equal(kd[:, abn], O.mixquant_dequant(ref)[:, abn])


def test_mixquant_all_channels_two_bit():
    k = fp16_values((64, 128), 13, scale=2.0)
    mq = O.mixquant(k, 1.0)
    assert len(mq["nom_idx"]) == 0 and np.array_equal(mq["abn_idx"], np.arange(128))
    kd = O.mixquant_dequant(mq)
    c, s, z = O.gquant_groups(k, 2)
    assert np.array_equal(kd, O.gdequant_groups(c, s, z))
    s_tok = np.repeat(s.astype(np.float64), 32, axis=0)
    assert np.all(np.abs(kd - k) <= 0.5 * s_tok + np.abs(k) * 2.0 ** -10 + 1e-6)


def test_mixquant_fft_on_32_normal_channels():
    # k = 0.75: the transform runs over the 32 normal channels; a chunk whose normal channels hold one
    # cosine of the channel position has a single spectral line, so the sign code keeps its phase
    T = 32
    k = np.zeros((T, 128), dtype=np.float32)
    k[:, :96] = (np.arange(96) % 7 + 1.0) * 4.0 * np.where(np.arange(T)[:, None] % 2, 1.0, -1.0)   # wide range: anomalous
    pos = np.arange(32)
    k[:, 96:] = np.cos(2 * np.pi * 3 * pos / 32)[None, :].astype(np.float16)
    mq = O.mixquant(k, 0.75)
    assert mq["mode"] == "fft" and np.array_equal(mq["nom_idx"], np.arange(96, 128))
    assert mq["bits1"].shape == (T, 64) and mq["s1"].shape == (1, 64)
    # the library transform of the same rows: the code's scales are the mean magnitudes of its parts
    spec = np.fft.fft(k[:, 96:].astype(np.float64), axis=1, norm="ortho")
    assert np.allclose(mq["s1"][0, :32].astype(np.float64), np.abs(spec.real).mean(axis=0), rtol=2e-3, atol=1e-4)
    assert np.allclose(mq["s1"][0, 32:].astype(np.float64), np.abs(spec.imag).mean(axis=0), rtol=2e-3, atol=1e-4)
    kd = O.mixquant_dequant(mq)[:, 96:]
    # bins 3 and 29 dominate the reconstruction: it correlates strongly with the input
    corr = (kd * k[:, 96:]).sum() / np.sqrt((kd ** 2).sum() * (k[:, 96:] ** 2).sum())
    assert corr > 0.9


def test_slabcache_carries_ratio_and_mode_through_a_flush():
    cfg = CONFIGS["tiny"]
    K, V = make_layer_kv(cfg, 0, T=64 + O.R)
    k, v = K[0, 0].float().numpy(), V[0, 0].float().numpy()
    sc = O.SlabCache(ratio=0.25, one_bit="auto")
    sc.prefill(k[:64], v[:64])
    q = fp16_values((7, 128), 14)
    for t in range(O.R):
        sc.decode_step(q, k[64 + t], v[64 + t])
    assert len(sc.k_chunks) == 2 and all(c["mode"] == "minmax" and len(c["abn_idx"]) == 32 for c in sc.k_chunks)
    assert sc.dequant_k().shape == (64 + O.R, 128)
