"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on seeded inputs that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

from oracle import vidkv_oracle as O
from tests import unpack as U
from tests.helpers import (Pair, TOL_ABS, check_stats, compare_key_chunk, compare_ternary, f16_ulp_distance,
                           new_stats, to_np)
from workloads import CONFIGS, make_layer_kv, make_saliency, make_step_inputs

pytestmark = pytest.mark.gpu


def _compare_prefill(pair: Pair):
    cache = pair.cache_bytes()
    stats = new_stats()
    Tq = pair.T - pair.T % 32
    r = pair.T % 32
    for (layer, b, h), sc in pair.slabs.items():
        slab = U.slab_bytes(cache, pair.lay, pair.cfg, layer, b, h)
        k = to_np(pair.K[layer][b, h])
        v = to_np(pair.V[layer][b, h])
        if Tq:
            ties = compare_key_chunk(slab, pair.lay, 0, 0, sc.k_chunks[0], k[:Tq], stats)
            if len(ties):
                assert len(ties) <= max(2, 2e-3 * Tq), "too many tokens with a sign bit at a tie"
                pair.sign_tie_tokens[(layer, b, h)] = ties
        sq = sc.v_prefill
        n_rest = len(sq["rest_idx"])
        if n_rest:
            ng = (n_rest + 31) // 32
            trits, s = U.ternary_groups(slab, pair.lay, 0, ng)
            thr = None if pair.ternary_scale == "mean_abs" else O.quant_1p58_groups(v[sq["rest_idx"]])[1]
            compare_ternary(trits, s, sq["trits"], sq["st"], v[sq["rest_idx"]], stats, o_s_thr=thr)
        n_prot = len(sq["prot_idx"])
        if n_prot:
            E, prefix = U.selection_mask(cache, pair.lay, b, Tq)
            assert (np.nonzero(E)[0] == sq["prot_idx"]).all(), "protected token set differs"
            assert prefix[Tq // 32] == n_prot
            npg = (n_prot + 31) // 32
            codes, s, z = U.protected_groups(slab, pair.lay, npg)
            assert (codes[:n_prot] == sq["codes2"]).all()
            assert (s.view(np.int16) == sq["s2"].view(np.int16)).all()
            assert (z.view(np.int16) == sq["z2"].view(np.int16)).all()
        if r:
            assert (U.residual(slab, pair.lay, "k", r, pair.wl.torch_dtype) == k[Tq:]).all()
            assert (U.residual(slab, pair.lay, "v", r, pair.wl.torch_dtype) == v[Tq:]).all()
    check_stats(stats)
    return stats


def _compare_dequant(pair: Pair):
    """Dequantized K and V within 2e-3 of the oracle's, element by element.  Where the two sides hold
    different codes or metadata for an element, which the matching rules allow only at ties and for
    mean-based scales one binary16 step apart, the bound for exactly the affected elements grows by
    what that difference is worth:
      - a stored Eq. 5 scale that differs by d moves every normal channel of the group's tokens by
        at most w d / 8 (orthonormal 64-point transform; w = 2 for a column that stands for a
        conjugate pair, 1 for the two real bins);
      - a sign bit that differs at a tie flips a coefficient of magnitude s: w 2 s / 8 per channel;
      - a ternary scale that differs by d moves the group's non-zero elements of that channel by d;
      - a trit that differs at a tie moves its element by s.
    The library's dequantizers return float32, so each element also gets the rounding of its own
    float32 evaluation: 4 units of 2^-24 of its magnitude (code * s + z), and for a normal channel,
    a sum of 64 spectrum terms, 64 * 2^-24 times the sum of the terms' magnitudes.  For keys and
    values of ordinary size both are far below 2e-3; they matter for inputs of several thousand.
    Everything else holds 2e-3 as it is."""
    cache = pair.cache_bytes()
    pk = O.hermitian_pack_columns(64)
    w = np.full(64, 2.0)
    w[:2] = 1.0
    for layer in range(pair.L):
        Kd = pair.cache.dequantize_keys(layer).cpu().numpy().astype(np.float64)
        Vd = pair.cache.dequantize_values(layer).cpu().numpy().astype(np.float64)
        for b in range(pair.B):
            for h in range(pair.cfg.H_kv):
                sc = pair.slabs[(layer, b, h)]
                ok, ov = sc.dequant_k(), sc.dequant_v()
                assert Kd[b, h].shape == ok.shape and Vd[b, h].shape == ov.shape
                if ok.size == 0:
                    continue
                slab = U.slab_bytes(cache, pair.lay, pair.cfg, layer, b, h)
                # ---- keys
                tolK = TOL_ABS + 4.0 * 2.0 ** -24 * np.abs(ok)
                t0 = g0 = 0
                for c in sc.k_chunks:
                    Tc, ng = c["T"], c["T"] // 32
                    _, bits1, _, _, s1 = U.key_groups(slab, pair.lay, g0, ng)
                    o_s1 = c["s1"][:, pk].astype(np.float64)
                    per_group = (np.abs(s1.astype(np.float64) - o_s1) * w).sum(axis=1) / 8.0
                    extra = np.repeat(per_group + 64.0 * 2.0 ** -24 * (o_s1 * w).sum(axis=1) / 8.0, 32)
                    bad = bits1 != c["bits1"][:, pk]
                    if bad.any():
                        extra = extra + (bad * np.repeat(o_s1, 32, axis=0) * w).sum(axis=1) / 4.0
                    tolK[t0:t0 + Tc, c["nom_idx"]] += extra[:, None]
                    t0 += Tc
                    g0 += ng
                assert (np.abs(Kd[b, h] - ok) <= tolK).all(), float((np.abs(Kd[b, h] - ok) - tolK).max())
                # ---- values
                tolV = TOL_ABS + 4.0 * 2.0 ** -24 * np.abs(ov)
                sq = sc.v_prefill
                n_rest = len(sq["rest_idx"])
                runs = []                                    # (token ids of the run, first stream group, oracle trits, oracle scales)
                if n_rest:
                    runs.append((np.asarray(sq["rest_idx"]), 0, sq["trits"], sq["st"]))
                tq0 = sq["T"]
                for i, (ft, fs) in enumerate(sc.v_flush):
                    runs.append((tq0 + 128 * i + np.arange(128), (n_rest + 31) // 32 + 4 * i, ft, fs))
                for tok, gb, o_t, o_s in runs:
                    ng = (len(tok) + 31) // 32
                    trits, s = U.ternary_groups(slab, pair.lay, gb, ng)
                    ds = np.repeat(np.abs(s.astype(np.float64) - o_s.astype(np.float64)), 32, axis=0)[:len(tok)]
                    flip = (trits[:len(tok)] != o_t) * np.repeat(o_s.astype(np.float64), 32, axis=0)[:len(tok)]
                    tolV[tok] += ds + flip
                assert (np.abs(Vd[b, h] - ov) <= tolV).all(), float((np.abs(Vd[b, h] - ov) - tolV).max())


@pytest.mark.parametrize("name,T,B,p", [
    ("tiny", 1632, 1, 0.0),        # the named config: 51 groups, 10.2 supergroups, 12.75 encode tiles
    ("tiny", 1632, 1, 0.2),        # with semantic token protection (313 protected tokens)
    ("tiny", 77, 2, 0.0),          # ragged: 64 quantized tokens + 13 residual tokens
    ("tiny", 31, 1, 0.0),          # nothing quantized, everything in the residual
    ("llava", 352, 1, 0.2),        # heavy-tailed values, +-5 outlier offsets
    ("qwen", 480, 2, 0.2),         # bf16 inputs, rotary-structured keys
    ("tiny", 1632, 1, 0.9),        # nearly every visual token protected
    ("tiny", 800, 1, 0.002),       # a single protected token
])
def test_prefill_codes_and_dequant(name, T, B, p):
    pair = Pair(CONFIGS[name], T, B=B, L=1, p=p).prefill()
    _compare_prefill(pair)
    _compare_dequant(pair)
    assert pair.cache.status() == 0


@pytest.mark.parametrize("name,T,p,steps", [("tiny", 300, 0.2, 0), ("qwen", 101, 0.0, 130), ("tiny", 250, 0.3, 125)])
def test_exports_agree_with_the_documented_layout_and_the_oracle(name, T, p, steps):
    """vidkv_export_codes / vidkv_get_selection against (a) the independent reader of the byte layout
    in tests/unpack.py and (b) the oracle's codes, after prefill and after a residual flush."""
    pair = Pair(CONFIGS[name], T, B=2, L=1, p=p, max_new=steps + 1).prefill()
    for _ in range(steps):
        pair.decode()
    ex = {k: v.cpu().numpy() for k, v in pair.cache.export_codes(0, T).items()}
    dmask, E = (x.cpu().numpy() for x in pair.cache.get_selection(0, T))
    cache = pair.cache_bytes()
    Tq = T - T % 32
    for (layer, b, h), sc in pair.slabs.items():
        slab = U.slab_bytes(cache, pair.lay, pair.cfg, layer, b, h)
        ng = sc.n_quantized // 32
        codes2, bits1, s2, z2, s1 = U.key_groups(slab, pair.lay, 0, ng)
        assert (ex["k2"][b, h] == codes2).all() and (ex["k1bits"][b, h] == bits1).all()
        assert (ex["k_s2"][b, h].view(np.int16) == s2.view(np.int16)).all()
        assert (ex["k_z2"][b, h].view(np.int16) == z2.view(np.int16)).all()
        assert (ex["k_s1"][b, h].view(np.int16) == s1.view(np.int16)).all()
        t0 = 0
        for ci, c in enumerate(sc.k_chunks):
            assert (ex["k2"][b, h][t0:t0 + c["T"]] == c["codes2"]).all()         # the oracle's Eq. 4 codes
            want = np.zeros(128, dtype=np.uint8)
            want[c["abn_idx"]] = 1
            assert (dmask[b, h, ci if Tq else ci + 1] == want).all()             # the oracle's D-mask
            t0 += c["T"]
        nt = ex["v_trits"].shape[2] // 32
        trits, s = U.ternary_groups(slab, pair.lay, 0, nt)
        assert (ex["v_trits"][b, h] == trits).all() and (ex["v_s"][b, h].view(np.int16) == s.view(np.int16)).all()
        npg = ex["v2"].shape[2] // 32
        if npg:
            codes, s, z = U.protected_groups(slab, pair.lay, npg)
            assert (ex["v2"][b, h] == codes).all()
            assert (ex["v2_s"][b, h].view(np.int16) == s.view(np.int16)).all()
            assert (ex["v2_z"][b, h].view(np.int16) == z.view(np.int16)).all()
            n_prot = len(sc.v_prefill["prot_idx"])
            assert (ex["v2"][b, h][:n_prot] == sc.v_prefill["codes2"]).all()     # the oracle's protected codes
        want_E = np.zeros(T, dtype=np.uint8)
        if pair.E is not None:
            want_E[:Tq] = pair.E[b]
        assert (E[b] == want_E).all()                                             # the oracle's mask E
    assert pair.cache.status() == 0


def test_prefill_is_deterministic_and_leaves_other_regions_alone():
    a = Pair(CONFIGS["tiny"], 1632, L=1, p=0.2).prefill()
    b = Pair(CONFIGS["tiny"], 1632, L=1, p=0.2).prefill()
    ca, cb = a.cache_bytes(), b.cache_bytes()
    assert (ca == cb).all()
    # header magic and a clean status word
    assert ca[:4].view("<u4")[0] == 0x564B4456 and ca[8:12].view("<i4")[0] == 0


def _decode_steps(pair: Pair, n_steps, tol=TOL_ABS):
    worst = 0.0
    for _ in range(n_steps):
        out, ref = pair.decode()
        err = np.abs(out - ref).max()
        worst = max(worst, err)
        assert err <= tol, f"step {pair.step - 1}: max abs error {err}"
    return worst


@pytest.mark.parametrize("name,T,B,p,steps", [
    ("tiny", 1632, 1, 0.0, 16),    # the named config
    ("tiny", 1632, 1, 0.2, 16),
    ("tiny", 77, 2, 0.0, 5),
    ("tiny", 31, 1, 0.0, 3),
    ("qwen", 480, 2, 0.2, 4),
    ("qwen", 480, 2, 0.0, 4),      # bf16 inputs without protection: the tensor-core kernel
    ("tiny", 2000, 1, 0.0, 3),     # 1984 quantized tokens = 3.1 splits of 640, plus 16 residual tokens
    ("tiny", 1300, 2, 0.0, 3),     # last split starts inside a supergroup (1280) and ends in the residual
    ("tiny", 1632, 1, 0.9, 3),     # nearly every visual token protected: long protected stream, short ternary one
    ("tiny", 800, 1, 0.002, 3),    # a single protected token
    ("tiny", 1568, 1, 1.0, 3),     # every token is visual and protected: the ternary stream is empty
])
def test_decode_attention_parity(name, T, B, p, steps):
    pair = Pair(CONFIGS[name], T, B=B, L=1, p=p, max_new=steps).prefill()
    _decode_steps(pair, steps)
    assert pair.cache.status() == 0


def _random_cases(n, seed):
    r = np.random.default_rng(seed)
    cases = []
    for _ in range(n):
        name = ["tiny", "llava", "qwen"][int(r.integers(0, 3))]
        cases.append((name, int(r.integers(1, 1500)), int(r.integers(1, 3)), int(r.integers(1, 3)),
                      [0.0, 0.0, 0.1, 0.5][int(r.integers(0, 4))], int(r.integers(1, 4)),
                      ["mean_abs", "nonzero_mean"][int(r.integers(0, 2))]))
    return cases


@pytest.mark.parametrize("name,T,B,L,p,steps,ternary_scale", _random_cases(10, 20250316))
def test_seeded_random_shapes(name, T, B, L, p, steps, ternary_scale):
    """Shapes nobody picked by hand: token counts anywhere in [1, 1500) (any remainder modulo 32, 128, 160 and
    640), one or two sequences and layers, with and without protected tokens, both scale modes."""
    wl = CONFIGS[name]
    if min(wl.l_v, T - T % 32) < 1:
        p = 0.0                                      # no quantized visual token to protect
    pair = Pair(wl, T, B=B, L=L, p=p, max_new=steps, ternary_scale=ternary_scale).prefill()
    _compare_prefill(pair)
    _compare_dequant(pair)
    for _ in range(steps):
        out, ref = pair.decode()
        # as in the heavy-tail tests: where the outputs are large the bound scales with their magnitude
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    assert pair.cache.status() == 0


def test_decode_parity_heavy_tailed():
    # Student-t inputs: outputs are large, so the tolerance scales with their magnitude
    pair = Pair(CONFIGS["llava"], 352, B=1, L=2, p=0.2, max_new=4).prefill()
    for _ in range(4):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())


def test_decode_parity_heavy_tailed_without_protection():
    # Student-t keys and values through the tensor-core kernel, three splits
    pair = Pair(CONFIGS["llava"], 1504, B=1, L=1, p=0.0, max_new=3).prefill()
    for _ in range(3):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("name,T,p,k_mul,q_mul", [
    ("tiny", 300, 0.0, 100.0, 1.0),     # outlier channels reach +-6000: key scales near 2000 meet query entries near 40
    ("tiny", 704, 0.25, 100.0, 1.0),
    ("qwen", 480, 0.0, 10.0, 64.0),     # bfloat16; query entries of several hundred
    ("tiny", 300, 0.0, 1.0, 2.0 ** -12),  # a tiny query: its binary16 image must not lose its bits
])
def test_large_keys_and_queries_stay_finite(monkeypatch, name, T, p, k_mul, q_mul):
    """q_j * s_j would leave the binary16 range if the query went into the score operands as it
    is; the kernels normalise each query head by a power of two, so the result stays an ordinary
    number and still matches the oracle."""
    from tests import helpers as Hm
    make_kv, make_step = Hm.make_layer_kv, Hm.make_step_inputs

    def big_kv(wl, layer, device="cpu", T=None, B=None):
        K, V = make_kv(wl, layer, device, T=T, B=B)
        return (K.float() * k_mul).clamp(-60000, 60000).to(K.dtype), V

    def big_step(wl, layer, step, device="cpu", T=None, B=None):
        q, k, v = make_step(wl, layer, step, device, T=T, B=B)
        return (q.float() * q_mul).to(q.dtype), k, v

    monkeypatch.setattr(Hm, "make_layer_kv", big_kv)
    monkeypatch.setattr(Hm, "make_step_inputs", big_step)
    pair = Pair(CONFIGS[name], T, B=1, L=1, p=p, max_new=3).prefill()
    for _ in range(3):
        out, ref = pair.decode()
        assert np.isfinite(out).all()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    assert pair.cache.status() == 0


def _degenerate(kind, K, V):
    K, V = K.clone(), V.clone()
    if kind == "zeros":                       # zero range everywhere: s = 0, every code 0
        K.zero_(); V.zero_()
    elif kind == "constant_channels":         # zero-range groups next to ordinary ones
        K[..., 5] = 1.5; K[..., 77] = -2.0; V[..., 9] = 0.0; V[..., 100] = 3.0
    elif kind == "huge":                      # near the end of the binary16 range
        K = (K.float() * 6000).clamp(-60000, 60000).to(K.dtype); V = (V.float() * 6000).clamp(-60000, 60000).to(V.dtype)
    elif kind == "tiny_values":               # subnormal binary16 (flushed to zero in bfloat16)
        K = (K.float() * 1e-6).to(K.dtype); V = (V.float() * 1e-6).to(V.dtype)
    elif kind == "equal_rows":                # every token the same: all ranges zero, nothing to rank
        K[:, :, 1:] = K[:, :, :1]; V[:, :, 1:] = V[:, :, :1]
    return K, V


@pytest.mark.parametrize("kind", ["zeros", "constant_channels", "huge", "tiny_values", "equal_rows"])
@pytest.mark.parametrize("name,T,p", [("tiny", 300, 0.0), ("tiny", 300, 0.2), ("qwen", 200, 0.2)])
def test_degenerate_inputs(monkeypatch, kind, name, T, p):
    """The degenerate cases of the method: zero-range groups (s = 0), constant channels, values at
    both ends of the binary16 range, identical tokens.  Codes, metadata, dequantized tensors and
    two decode steps against the oracle."""
    from tests import helpers as Hm
    make_kv = Hm.make_layer_kv
    monkeypatch.setattr(Hm, "make_layer_kv",
                        lambda wl, layer, device="cpu", T=None, B=None: _degenerate(kind, *make_kv(wl, layer, device, T=T, B=B)))
    pair = Pair(CONFIGS[name], T, B=1, L=1, p=p, max_new=3).prefill()
    _compare_prefill(pair)
    _compare_dequant(pair)
    for _ in range(2):
        out, ref = pair.decode()
        assert np.isfinite(out).all()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    assert pair.cache.status() == 0


def test_full_size_slabs_in_the_benchmark_launch_shape():
    """The benchmark's configuration (batched long video: T = 12544, batch 16, 640-token splits),
    two layers in one call; the oracle recomputes four sampled (layer, batch, KV head) slabs."""
    import paper_2503_16257_b200 as P
    from workloads import make_layer_kv, make_step_inputs
    wl = CONFIGS["batched"]
    L, B, T, steps = 2, wl.batch, wl.T, 2
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=steps, p_ratio=0.0,
                        in_dtype=P.VIDKV_F16, out_dtype=P.VIDKV_F32)
    cache = P.VidKVCache(cfg, device="cuda")
    samples = [(0, 0, 0), (0, 7, 2), (1, 15, 3), (1, 3, 1)]
    slabs = {}
    for layer in range(L):
        K, V = make_layer_kv(wl, layer, "cuda")
        cache.quantize_keys(layer, K)
        cache.quantize_values(layer, V)
        for (sl, b, h) in samples:
            if sl == layer:
                sc = O.SlabCache()
                sc.prefill(to_np(K[b, h]), to_np(V[b, h]), None)
                slabs[(sl, b, h)] = sc
        del K, V
    for step in range(steps):
        q, k, v = (torch.stack(t) for t in zip(*[make_step_inputs(wl, layer, step, "cuda") for layer in range(L)]))
        out = torch.empty((L, B, 28, 128), dtype=torch.float32, device="cuda")
        cache.decode_attention(0, L, q, k, v, out)
        out = out.cpu().numpy().astype(np.float64)
        for (sl, b, h), sc in slabs.items():
            ref = sc.decode_step(to_np(q[sl, b, 7 * h:7 * h + 7]), to_np(k[sl, b, h]), to_np(v[sl, b, h]))
            assert np.abs(out[sl, b, 7 * h:7 * h + 7] - ref).max() <= TOL_ABS
    assert cache.status() == 0


def test_longest_sequence_slab():
    """The stress configuration's token count (1000 frames = 196 000 tokens, 307 splits per slab) on
    one layer and one batch element; the oracle recomputes one KV head."""
    import paper_2503_16257_b200 as P
    from workloads import make_layer_kv, make_step_inputs
    wl = CONFIGS["stress"]
    T = wl.T
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=T, max_new_tokens=2, p_ratio=0.0,
                        in_dtype=P.VIDKV_F16, out_dtype=P.VIDKV_F32)
    cache = P.VidKVCache(cfg, device="cuda")
    K, V = make_layer_kv(wl, 0, "cuda", T=T, B=1)
    cache.quantize_keys(0, K)
    cache.quantize_values(0, V)
    h = 2
    sc = O.SlabCache()
    sc.prefill(to_np(K[0, h]), to_np(V[0, h]), None)
    q, k, v = make_step_inputs(wl, 0, 0, "cuda", T=T, B=1)
    out = torch.empty((1, 1, 28, 128), dtype=torch.float32, device="cuda")
    cache.decode_attention(0, 1, q[None], k[None], v[None], out)
    ref = sc.decode_step(to_np(q[0, 7 * h:7 * h + 7]), to_np(k[0, h]), to_np(v[0, h]))
    assert np.abs(out[0, 0, 7 * h:7 * h + 7].cpu().numpy().astype(np.float64) - ref).max() <= TOL_ABS
    assert cache.layer_state(0) == dict(n_quantized=196000 - 196000 % 32, n_residual=196000 % 32 + 1, n_chunks=1, n_protected=0)
    assert cache.status() == 0


@pytest.mark.parametrize("H_kv,H_q,p", [(2, 16, 0.0), (2, 16, 0.25), (8, 8, 0.0), (1, 4, 0.25), (4, 8, 0.0), (4, 12, 0.25), (2, 10, 0.0), (1, 6, 0.25), (3, 9, 0.0), (16, 16, 0.25)])
def test_other_head_counts(H_kv, H_q, p):
    """GQA ratios 8, 1 and 4 (the named workloads all use 7): seeded Gaussian K, V, q with a few
    wide key channels, two decode steps, every slab against the oracle."""
    import paper_2503_16257_b200 as P
    T, B, rep = 704, 2, H_q // H_kv
    g = torch.Generator().manual_seed(1234 + 17 * H_kv + H_q)
    wide = torch.ones(128); wide[torch.randperm(128, generator=g)[:6]] = 8.0
    K = (torch.randn((B, H_kv, T, 128), generator=g) * wide).to(torch.float16)
    V = torch.randn((B, H_kv, T, 128), generator=g).to(torch.float16)
    cfg = P.VidKVConfig(B=B, L=1, H_kv=H_kv, H_q=H_q, max_prefill_tokens=T, max_new_tokens=2, p_ratio=p,
                        in_dtype=P.VIDKV_F16, out_dtype=P.VIDKV_F32)
    cache = P.VidKVCache(cfg, device="cuda")
    E = [None] * B
    if p > 0:
        sal = torch.randn((B, 640), generator=g)
        cache.select_tokens(sal.cuda(), 0, 640, T)
        for b in range(B):
            E[b] = np.zeros(T, dtype=bool)
            E[b][:T - T % 32] = O.select_tokens(sal[b].numpy(), p, 0, T - T % 32)
    cache.quantize_keys(0, K.cuda())
    cache.quantize_values(0, V.cuda())
    slabs = {}
    for b in range(B):
        for h in range(H_kv):
            sc = O.SlabCache()
            sc.prefill(to_np(K[b, h]), to_np(V[b, h]), E[b])
            slabs[(b, h)] = sc
    for step in range(2):
        q = (torch.randn((1, B, H_q, 128), generator=g)).to(torch.float16)
        k = (torch.randn((1, B, H_kv, 128), generator=g) * wide).to(torch.float16)
        v = torch.randn((1, B, H_kv, 128), generator=g).to(torch.float16)
        out = torch.empty((1, B, H_q, 128), dtype=torch.float32, device="cuda")
        cache.decode_attention(0, 1, q.cuda(), k.cuda(), v.cuda(), out)
        out = out.cpu().numpy().astype(np.float64)
        for (b, h), sc in slabs.items():
            ref = sc.decode_step(to_np(q[0, b, h * rep:(h + 1) * rep]), to_np(k[0, b, h]), to_np(v[0, b, h]))
            assert np.abs(out[0, b, h * rep:(h + 1) * rep] - ref).max() <= TOL_ABS
    assert cache.status() == 0


@pytest.mark.parametrize("name,T,B,p", [
    ("tiny", 1632, 1, 0.0), ("tiny", 77, 2, 0.0), ("llava", 352, 1, 0.2), ("qwen", 480, 2, 0.2),
])
def test_nonzero_mean_ternary_scale_prefill(name, T, B, p):
    """The optional stored scale (mean of |v| over the non-zero codes): same codes, other scales."""
    pair = Pair(CONFIGS[name], T, B=B, L=1, p=p, ternary_scale="nonzero_mean").prefill()
    _compare_prefill(pair)
    _compare_dequant(pair)
    ref = Pair(CONFIGS[name], T, B=B, L=1, p=p).prefill()
    a, b = pair.cache_bytes(), ref.cache_bytes()
    assert (a != b).any()                       # the scales differ from the default mode's ...
    for key, sc in pair.slabs.items():          # ... the codes do not
        assert (sc.v_prefill["trits"] == ref.slabs[key].v_prefill["trits"]).all()
    assert pair.cache.status() == 0


@pytest.mark.parametrize("ternary_scale", ["mean_abs", "nonzero_mean"])
def test_residual_flush_parity(ternary_scale):
    # 64 quantized + 5 residual tokens; the residual fills at step 123 and is flushed
    wl = CONFIGS["tiny"]
    pair = Pair(wl, 69, B=1, L=2, p=0.0, max_new=140, ternary_scale=ternary_scale).prefill()
    _decode_steps(pair, 123)
    st = pair.cache.layer_state(0)
    assert st == dict(n_quantized=192, n_residual=0, n_chunks=2, n_protected=0)
    cache = pair.cache_bytes()
    stats = new_stats()
    for (layer, b, h), sc in pair.slabs.items():
        assert len(sc.k_chunks) == 2 and sc.k_res.shape[0] == 0
        slab = U.slab_bytes(cache, pair.lay, pair.cfg, layer, b, h)
        kin, vin = pair.flushed_in[(layer, b, h)]
        compare_key_chunk(slab, pair.lay, 1, 2, sc.k_chunks[1], kin, stats)
        trits, s = U.ternary_groups(slab, pair.lay, 2, 4)
        o_t, o_s = sc.v_flush[0]
        compare_ternary(trits, s, o_t, o_s, vin, stats,
                        o_s_thr=None if ternary_scale == "mean_abs" else O.quant_1p58_groups(vin)[1])
    check_stats(stats)
    _compare_dequant(pair)
    _decode_steps(pair, 10)          # attention over two chunks + a fresh residual
    assert pair.cache.layer_state(1)["n_residual"] == 10


@pytest.mark.parametrize("name,T,B,p,ternary_scale", [
    ("qwen", 577, 2, 0.2, "nonzero_mean"),      # bf16, protected tokens, the flush lands at stream group 18.4
    ("llava", 475, 2, 0.0, "nonzero_mean"),     # heavy-tailed, 27 residual tokens at prefill
    ("tiny", 118, 2, 0.0, "mean_abs"),
    ("tiny", 320, 1, 1.0, "mean_abs"),          # the flush appends to a ternary stream that was empty
])
def test_decode_across_a_flush_on_other_shapes(name, T, B, p, ternary_scale):
    steps = 128 - T % 32 + 3
    pair = Pair(CONFIGS[name], T, B=B, L=1, p=p, max_new=steps + 1, ternary_scale=ternary_scale).prefill()
    for _ in range(steps):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    st = pair.cache.layer_state(0)
    assert st["n_chunks"] == 2 and st["n_residual"] == 3 and pair.cache.status() == 0


@pytest.mark.parametrize("name,T,p,ternary_scale,steps", [
    ("tiny", 69, 0.0, "mean_abs", 262), ("qwen", 200, 0.2, "nonzero_mean", 270),
])
def test_decode_across_two_flushes(name, T, p, ternary_scale, steps):
    """Three key chunks with their own channel splits, two appended value runs, a residual on top."""
    pair = Pair(CONFIGS[name], T, B=1, L=1, p=p, max_new=steps + 1, ternary_scale=ternary_scale).prefill()
    for _ in range(steps):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    st = pair.cache.layer_state(0)
    assert st["n_chunks"] == 3 and st["n_quantized"] == T - T % 32 + 256 and pair.cache.status() == 0


def test_flush_with_protected_tokens_keeps_streams_apart():
    wl = CONFIGS["tiny"]
    pair = Pair(wl, 256, B=1, L=1, p=0.2, max_new=135).prefill()     # 51 protected, 205 ternary (6.4 groups)
    _decode_steps(pair, 130)
    assert pair.cache.layer_state(0) == dict(n_quantized=384, n_residual=2, n_chunks=2, n_protected=51)
    _compare_dequant(pair)


@pytest.mark.parametrize("name,p", [("tiny", 0.2), ("qwen", 0.0)])
def test_strided_inputs_give_the_same_cache(name, p):
    """K and V kept token-major ([B, T, H, D], as a projection writes them) and handed over as a
    [B, H, T, D] view must pack to the same bytes as contiguous copies."""
    import paper_2503_16257_b200 as P
    wl = CONFIGS[name]
    T, B = 1000, 2
    K, V = make_layer_kv(wl, 0, "cuda", T=T, B=B)
    in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
    cfg = P.VidKVConfig(B=B, L=1, max_prefill_tokens=T, max_new_tokens=1, p_ratio=p, in_dtype=in_dt, out_dtype=P.VIDKV_F32)
    caches = []
    for strided in (False, True):
        c = P.VidKVCache(cfg, device="cuda")
        if p > 0:
            c.select_tokens(make_saliency(wl, "cuda", l_v=960, B=B), 0, 960, T)
        if strided:
            Kt = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)     # [B, H, T, D] view of [B, T, H, D]
            Vt = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            assert not Kt.is_contiguous() and Kt.stride(2) == K.shape[1] * 128
            c.quantize_keys(0, Kt); c.quantize_values(0, Vt)
        else:
            c.quantize_keys(0, K); c.quantize_values(0, V)
        torch.cuda.synchronize()
        assert c.status() == 0
        caches.append(c.cache.cpu().numpy())
    assert np.array_equal(caches[0], caches[1])


@pytest.mark.parametrize("name,T,p", [("tiny", 1003, 0.2), ("qwen", 640, 0.0)])
def test_layer_range_quantization_gives_the_same_cache(name, T, p):
    """vidkv_quantize_keys_layers / vidkv_quantize_values_layers on [n_layers, B, H, T, D] tensors pack
    the same bytes as one call per layer (each layer keeps its own channel split and scales)."""
    import paper_2503_16257_b200 as P
    wl = CONFIGS[name]
    B, L = 2, 3
    in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=1, p_ratio=p, in_dtype=in_dt, out_dtype=P.VIDKV_F32)
    KV = [make_layer_kv(wl, layer, "cuda", T=T, B=B) for layer in range(L)]
    sal = make_saliency(wl, "cuda", l_v=T - T % 32, B=B) if p > 0 else None
    caches = []
    for ranged in (False, True):
        c = P.VidKVCache(cfg, device="cuda")
        if sal is not None:
            c.select_tokens(sal, 0, T - T % 32, T)
        if ranged:
            c.quantize_keys_layers(0, torch.stack([kv[0] for kv in KV]))
            c.quantize_values_layers(1, torch.stack([kv[1] for kv in KV[1:]]))      # a range that starts at layer 1
            c.quantize_values_layers(0, KV[0][1][None])
        else:
            for layer in range(L):
                c.quantize_keys(layer, KV[layer][0])
                c.quantize_values(layer, KV[layer][1])
        torch.cuda.synchronize()
        assert c.status() == 0 and c.layer_state(2)["n_quantized"] == T - T % 32
        caches.append(c.cache.cpu().numpy())
    assert np.array_equal(caches[0], caches[1])


def test_two_caches_on_two_streams():
    """Two caches worked on from two streams at once (prefill and decode interleaved) end up exactly
    as when each runs alone: the library keeps no per-call state outside the handle."""
    import paper_2503_16257_b200 as P
    wl = CONFIGS["tiny"]
    T, B, L = 1632, 2, 2
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=4, p_ratio=0.0, in_dtype=P.VIDKV_F16, out_dtype=P.VIDKV_F32)
    KV = [make_layer_kv(wl, layer, "cuda", T=T, B=B) for layer in range(L)]
    from workloads import make_step_inputs
    steps = [[make_step_inputs(wl, layer, s, "cuda", T=T, B=B) for layer in range(L)] for s in range(3)]

    def calls(cache, outs):
        """The work on one cache as a list of calls."""
        todo = []
        for layer in range(L):
            todo.append(lambda layer=layer: cache.quantize_keys(layer, KV[layer][0]))
            todo.append(lambda layer=layer: cache.quantize_values(layer, KV[layer][1]))
        for s in range(3):
            def step(s=s):
                q = torch.stack([steps[s][layer][0] for layer in range(L)])
                k = torch.stack([steps[s][layer][1] for layer in range(L)])
                v = torch.stack([steps[s][layer][2] for layer in range(L)])
                out = torch.empty((L, B, 28, 128), dtype=torch.float32, device="cuda")
                cache.decode_attention(0, L, q, k, v, out)
                outs.append(out)
            todo.append(step)
        return todo

    alone = P.VidKVCache(cfg, device="cuda")
    ref = []
    for f in calls(alone, ref):
        f()
    torch.cuda.synchronize()
    a, b = P.VidKVCache(cfg, device="cuda"), P.VidKVCache(cfg, device="cuda")
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    s1.wait_stream(torch.cuda.current_stream()); s2.wait_stream(torch.cuda.current_stream())
    oa, ob = [], []
    # call by call, alternating streams, so that kernels of both caches are in flight together
    for fa, fb in zip(calls(a, oa), calls(b, ob)):
        with torch.cuda.stream(s1):
            fa()
        with torch.cuda.stream(s2):
            fb()
    torch.cuda.synchronize()
    for x, y, z in zip(ref, oa, ob):
        assert torch.equal(x, y) and torch.equal(x, z)
    assert torch.equal(alone.cache, a.cache) and torch.equal(alone.cache, b.cache)
    assert a.status() == 0 and b.status() == 0


def test_multi_layer_call_equals_per_layer_calls():
    wl = CONFIGS["tiny"]
    a = Pair(wl, 320, B=2, L=3, p=0.0, max_new=2).prefill()
    out_all, ref = a.decode()
    assert np.abs(out_all - ref).max() <= TOL_ABS
    b = Pair(wl, 320, B=2, L=3, p=0.0, max_new=2).prefill()
    from workloads import make_step_inputs
    for layer in range(3):
        q, k, v = make_step_inputs(wl, layer, 0, "cpu", T=320, B=2)
        out = torch.empty((1, 2, 28, 128), dtype=torch.float32, device="cuda")
        b.cache.decode_attention(layer, 1, q[None].cuda(), k[None].cuda(), v[None].cuda(), out)
        assert np.array_equal(out.cpu().numpy()[0].astype(np.float64), out_all[layer])


def test_output_dtypes():
    import paper_2503_16257_b200 as P
    wl = CONFIGS["tiny"]
    from workloads import make_layer_kv, make_step_inputs
    K, V = make_layer_kv(wl, 0, "cpu", T=160)
    q, k, v = make_step_inputs(wl, 0, 0, "cpu", T=160)
    outs = {}
    for od, tdt in [(P.VIDKV_F32, torch.float32), (P.VIDKV_F16, torch.float16), (P.VIDKV_BF16, torch.bfloat16)]:
        cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=160, max_new_tokens=1, out_dtype=od)
        c = P.VidKVCache(cfg)
        c.quantize_keys(0, K.cuda()); c.quantize_values(0, V.cuda())
        out = torch.empty((1, 1, 28, 128), dtype=tdt, device="cuda")
        c.decode_attention(0, 1, q[None].cuda(), k[None].cuda(), v[None].cuda(), out)
        outs[od] = out.float().cpu()
    assert torch.equal(outs[P.VIDKV_F32].half().float(), outs[P.VIDKV_F16])
    assert torch.equal(outs[P.VIDKV_F32].bfloat16().float(), outs[P.VIDKV_BF16])


def test_call_order_and_capacity_errors():
    import paper_2503_16257_b200 as P
    wl = CONFIGS["tiny"]
    from workloads import make_layer_kv, make_step_inputs
    K, V = make_layer_kv(wl, 0, "cpu", T=96)
    q, k, v = make_step_inputs(wl, 0, 0, "cpu", T=96)
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=96, max_new_tokens=1, p_ratio=0.2)
    c = P.VidKVCache(cfg)
    out = torch.empty((1, 1, 28, 128), dtype=torch.float32, device="cuda")
    args = (0, 1, q[None].cuda(), k[None].cuda(), v[None].cuda(), out)
    with pytest.raises(P.VidKVError) as e:
        c.decode_attention(*args)                       # nothing quantized yet
    assert e.value.status == -5
    c.quantize_keys(0, K.cuda())
    with pytest.raises(P.VidKVError) as e:
        c.quantize_keys(0, K.cuda())                    # twice
    assert e.value.status == -5
    with pytest.raises(P.VidKVError) as e:
        c.quantize_values(0, V.cuda())                  # p > 0 but no token selection yet
    assert e.value.status == -5
    c.select_tokens(None, 0, 0, 96)
    with pytest.raises(P.VidKVError) as e:
        c.quantize_values(0, V[:, :, :64].contiguous().cuda())     # T differs from the keys'
    assert e.value.status == -5
    big = torch.zeros((1, 4, 128, 128), dtype=torch.float16, device="cuda")
    c2 = P.VidKVCache(cfg)
    with pytest.raises(P.VidKVError) as e:
        c2.quantize_keys(0, big)                        # more tokens than the cache was sized for
    assert e.value.status == -4
    with pytest.raises(P.VidKVError) as e:
        c2.quantize_keys(0, K.cuda()[:, :, :, 1:])      # misaligned view
    assert e.value.status in (-3, -1)
    c.quantize_values(0, V.cuda())
    c.decode_attention(*args)
    with pytest.raises(P.VidKVError) as e:
        c.decode_attention(*args)                       # max_new_tokens = 1
    assert e.value.status == -4
    assert c.status() == 0


def test_token_mask_entry_point_matches_saliency_selection():
    import paper_2503_16257_b200 as P
    from workloads import make_layer_kv, make_saliency
    wl = CONFIGS["tiny"]
    T = 320
    K, V = make_layer_kv(wl, 0, "cpu", T=T, B=2)
    sal = make_saliency(wl, "cpu", l_v=256, B=2)
    cfg = P.VidKVConfig(B=2, L=1, max_prefill_tokens=T, max_new_tokens=1, p_ratio=0.2)
    a = P.VidKVCache(cfg)
    a.select_tokens(sal.cuda(), 32, 256, T)
    a.quantize_values(0, V.cuda())
    E = np.stack([O.select_tokens(sal[b].numpy(), 0.2, 32, T) for b in range(2)]).astype(np.uint8)
    b = P.VidKVCache(cfg)
    b.set_token_mask(torch.from_numpy(E).cuda(), T)
    b.quantize_values(0, V.cuda())
    torch.cuda.synchronize()
    assert torch.equal(a.cache, b.cache)
    assert a.layer_state(0)["n_protected"] == 51
    # with the count stated the call does not synchronise and gives the same cache
    b2 = P.VidKVCache(cfg)
    b2.set_token_mask(torch.from_numpy(E).cuda(), T, n_protected=51)
    b2.quantize_values(0, V.cuda())
    torch.cuda.synchronize()
    assert torch.equal(a.cache, b2.cache) and b2.status() == 0
    # a mask whose rows protect different numbers of tokens is rejected: on the host when the
    # library counts, through the status word when the caller stated the count
    E[1, 40] ^= 1
    c = P.VidKVCache(cfg)
    with pytest.raises(P.VidKVError):
        c.set_token_mask(torch.from_numpy(E).cuda(), T)
    d = P.VidKVCache(cfg)
    d.set_token_mask(torch.from_numpy(E).cuda(), T, n_protected=51)
    assert d.status() == -1


def test_saliency_ties_take_lower_index():
    import paper_2503_16257_b200 as P
    T = 64
    sal = torch.zeros((1, 64), dtype=torch.float32)
    sal[0, 10] = 2.0
    sal[0, 20:30] = 1.0                 # ten-way tie for the remaining 11 places of n = 12
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=T, max_new_tokens=1, p_ratio=0.1875)
    c = P.VidKVCache(cfg)
    c.select_tokens(sal.cuda(), 0, 64, T)
    torch.cuda.synchronize()
    E, _ = U.selection_mask(c.cache.cpu().numpy(), c.layout, 0, T)
    ref = O.select_tokens(sal[0].numpy(), 0.1875, 0, T)
    assert (E == ref).all() and E.sum() == 12 and E[0] and not E[2]


@pytest.mark.parametrize("name,p", [("tiny", 0.2), ("qwen", 0.0)])
def test_values_quantized_on_a_second_stream_give_the_same_cache(name, p):
    """The key and the value quantizer write disjoint parts of the cache and workspace: with the values on a
    second stream beside the keys (selection before both, streams joined afterwards) the cache holds the
    same bytes as with everything on one stream, and decodes to the same output."""
    import paper_2503_16257_b200 as P
    wl = CONFIGS[name]
    T, B, L = 1100, 2, 3
    in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=2, p_ratio=p, in_dtype=in_dt, out_dtype=P.VIDKV_F32)
    KV = [make_layer_kv(wl, layer, "cuda", T=T, B=B) for layer in range(L)]
    side = torch.cuda.Stream()
    images, outs = [], []
    for two_streams in (False, True):
        c = P.VidKVCache(cfg, device="cuda")
        if p > 0:
            c.select_tokens(make_saliency(wl, "cuda", l_v=960, B=B), 0, 960, T)
        main = torch.cuda.current_stream()
        side.wait_stream(main)
        for layer in range(L):
            c.quantize_keys(layer, KV[layer][0])
            if two_streams:
                with torch.cuda.stream(side):
                    c.quantize_values(layer, KV[layer][1])
            else:
                c.quantize_values(layer, KV[layer][1])
        main.wait_stream(side)
        q, k, v = [torch.stack(x) for x in zip(*[make_step_inputs(wl, layer, 0, "cuda", T=T, B=B) for layer in range(L)])]
        out = torch.empty((L, B, cfg.H_q, 128), dtype=torch.float32, device="cuda")
        c.decode_attention(0, L, q, k, v, out)
        torch.cuda.synchronize()
        assert c.status() == 0
        images.append(c.cache.cpu().numpy())
        outs.append(out.cpu().numpy())
    assert np.array_equal(images[0], images[1])
    assert np.array_equal(outs[0], outs[1])
