"""GPU parity of the other key bit widths (Algorithm 3 with k = 0.25, 0.75, 1 and the plain min/max
1-bit code of 1BitQuant's other branch; Table 2's 1.25-, 1.75- and 2-bit rows) against the oracle:
channel split, codes and metadata bit-exact (Eq. 5 bits up to ties), dequantized keys and attention
outputs within the stated bound, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import vidkv_oracle as O
from tests import unpack as U
from tests.helpers import Pair, TOL_ABS, TIE_REL, f16_ulp_distance, to_np
from workloads import CONFIGS

pytestmark = pytest.mark.gpu

FORMATS = [(0.25, "minmax"), (0.5, "minmax"), (0.75, "minmax"), (0.75, "fft"), (1.0, "fft")]


def _fmt_id(f):
    return f"k{f[0]}-{f[1]}"


def _check_chunk(exp, raw, mq, b, h, g0, k_in):
    """One key chunk of slab (b, h): exported arrays `exp`, raw-byte reading `raw`, oracle dict `mq`."""
    ng = mq["T"] // 32
    rows = slice(32 * g0, 32 * (g0 + ng))
    grp = slice(g0, g0 + ng)
    n1 = len(mq["nom_idx"])
    codes2, bits1, s2, z2, s1, z1 = raw
    k2 = exp["k2"][b, h, rows].cpu().numpy()
    assert np.array_equal(k2, codes2) and np.array_equal(k2, mq["codes2"]), "2-bit codes differ"
    for name, mine, ref in (("k_s2", s2, mq["s2"]), ("k_z2", z2, mq["z2"])):
        got = exp[name][b, h, grp].cpu().numpy()
        assert np.array_equal(got.view(np.int16), mine.view(np.int16))
        assert np.array_equal(got.view(np.int16), ref.view(np.int16)), name + " differs"
    if n1 == 0:
        return 0
    k1 = exp["k1bits"][b, h, rows].cpu().numpy()
    assert np.array_equal(k1, bits1)
    if mq["mode"] == "minmax":
        es = exp["k_s1"][b, h, grp].cpu().numpy()
        assert np.array_equal(es[:, 0].view(np.int16), s1.view(np.int16)) and np.array_equal(es[:, 1].view(np.int16), z1.view(np.int16))
        assert np.array_equal(s1.view(np.int16), mq["s1"].view(np.int16)), "1-bit scales differ"
        assert np.array_equal(z1.view(np.int16), mq["z1"].view(np.int16)), "1-bit zero points differ"
        assert np.array_equal(k1, mq["codes1"]), "1-bit codes differ"
        return 0
    pk = O.hermitian_pack_columns(n1)
    o_bits, o_s1 = mq["bits1"][:, pk], mq["s1"][:, pk]
    assert np.array_equal(exp["k_s1"][b, h, grp].cpu().numpy().view(np.int16), s1.view(np.int16))
    assert f16_ulp_distance(s1, o_s1).max() <= 1, "Eq. 5 scales differ by more than one binary16 step"
    bad = k1 != o_bits
    if bad.any():
        xf = O.dft64(k_in[:, mq["nom_idx"]])
        cols = np.concatenate([xf.real, xf.imag], -1)[:, pk]
        scale = np.repeat(o_s1.astype(np.float64), 32, axis=0)
        assert (np.abs(cols[bad]) <= TIE_REL * scale[bad] + 1e-12).all(), "a sign bit differs away from zero"
    return int(bad.sum())


def _check_layer(pair, layer=0):
    cfg = pair.cfg
    n2 = int(round(pair.k_ratio * 128))
    plain = pair.one_bit == "minmax" and n2 < 128
    exp = pair.cache.export_codes(layer, pair.T)
    dmask, _ = pair.cache.get_selection(layer, pair.T)
    deq = pair.cache.dequantize_keys(layer).cpu().numpy().astype(np.float64)
    cache = pair.cache_bytes()
    n_bad = n_all = 0
    for b in range(pair.B):
        for h in range(cfg.H_kv):
            sc = pair.slabs[(layer, b, h)]
            slab = U.slab_bytes(cache, pair.lay, cfg, layer, b, h)
            g0 = 0
            k_all = to_np(pair.K[layer][b, h])
            tq0 = pair.T - pair.T % 32
            for ci, mq in enumerate(sc.k_chunks):
                chunk = ci if tq0 > 0 else ci + 1
                abn, nom = U.chunk_perm_general(slab, pair.lay, chunk, n2)
                assert np.array_equal(abn, mq["abn_idx"]) and np.array_equal(nom, mq["nom_idx"]), "channel split differs"
                dm = dmask[b, h, chunk].cpu().numpy()
                assert np.array_equal(np.nonzero(dm)[0], mq["abn_idx"])
                ng = mq["T"] // 32
                raw = U.key_groups_general(slab, pair.lay, g0, ng, n2, plain)
                k_in = k_all[:tq0] if ci == 0 and tq0 > 0 else pair.flushed_chunks[(layer, b, h)][ci - (1 if tq0 > 0 else 0)]
                n_bad += _check_chunk(exp, raw, mq, b, h, g0, k_in)
                n_all += mq["T"] * len(mq["nom_idx"])
                g0 += ng
            ref = sc.dequant_k()
            got = deq[b, h]
            assert got.shape == ref.shape
            if n_bad == 0:
                # elements whose codes and metadata agree: the float32 evaluation of the same formula; a
                # mean-based scale one binary16 step apart moves a token's normal channels by a fraction of it
                tol = TOL_ABS * max(1.0, np.abs(ref).max())
                assert np.abs(got - ref).max() <= tol, np.abs(got - ref).max()
    assert n_bad <= max(1, 1e-4 * n_all)


@pytest.mark.parametrize("fmt", FORMATS, ids=_fmt_id)
@pytest.mark.parametrize("name,T,B", [("tiny", 363, 2), ("qwen", 224, 1)])
def test_prefill_codes_and_dequantized_keys(fmt, name, T, B):
    pair = Pair(CONFIGS[name], T, B=B, L=1, max_new=4, k_ratio=fmt[0], one_bit=fmt[1])
    pair.flushed_chunks = {}
    pair.prefill()
    assert pair.cache.status() == 0
    _check_layer(pair)


@pytest.mark.parametrize("fmt", FORMATS, ids=_fmt_id)
@pytest.mark.parametrize("p", [0.0, 0.2])
def test_decode_across_a_flush(fmt, p):
    T = 200
    steps = 128 - T % 32 + 3
    pair = Pair(CONFIGS["tiny"], T, B=1, L=1, p=p, max_new=steps + 1, k_ratio=fmt[0], one_bit=fmt[1]).prefill()
    pair.flushed_chunks = {}
    for _ in range(steps):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
        for key, (fk, _) in pair.flushed_in.items():
            pair.flushed_chunks.setdefault(key, [fk])
    st = pair.cache.layer_state(0)
    assert st["n_chunks"] == 2 and st["n_residual"] == 3 and pair.cache.status() == 0
    _check_layer(pair)


@pytest.mark.parametrize("fmt", [(0.25, "minmax"), (0.75, "fft"), (1.0, "fft")], ids=_fmt_id)
@pytest.mark.parametrize("name,p", [("qwen", 0.0), ("llava", 0.2)])
def test_decode_over_several_units_layers_and_run_lengths(fmt, name, p):
    """Long enough that a warp's run crosses units and slabs; forced run lengths cover the joins."""
    T, B, L = 1700, 2, 2
    pair = Pair(CONFIGS[name], T, B=B, L=L, p=p, max_new=8, k_ratio=fmt[0], one_bit=fmt[1]).prefill()
    for run_units in (0, 1, 3, 7):
        pair.cache.debug_set_decode_plan(run_units)
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max()), (run_units, np.abs(out - ref).max())
    assert pair.cache.status() == 0


def test_workspace_free_attention_on_another_key_format():
    import paper_2503_16257_b200 as P
    pair = Pair(CONFIGS["tiny"], 500, B=2, L=1, p=0.0, max_new=4, k_ratio=0.75, one_bit="fft").prefill()
    out, ref = pair.decode()
    st = pair.cache.layer_state(0)
    q = torch.randn((1, 2, pair.cfg.H_q, 128), device="cuda", generator=torch.Generator("cuda").manual_seed(5)).half()
    o1 = torch.empty((1, 2, pair.cfg.H_q, 128), dtype=torch.float32, device="cuda")
    P.vidkv_attend_noalloc(pair.cfg, pair.cache.cache, 500 - 500 % 32, 0, st["n_residual"], 0, 0, 1, q, o1)
    torch.cuda.synchronize()
    rep = pair.cfg.H_q // pair.cfg.H_kv
    for b in range(2):
        for h in range(pair.cfg.H_kv):
            sc = pair.slabs[(0, b, h)]
            K = np.concatenate([sc.dequant_k(), sc.k_res.astype(np.float64)])
            V = np.concatenate([sc.dequant_v(), sc.v_res.astype(np.float64)])
            want = O.attention(to_np(q[0, b, h * rep:(h + 1) * rep]), K, V, 1.0 / np.sqrt(128.0))
            got = o1[0, b, h * rep:(h + 1) * rep].cpu().numpy()
            assert np.abs(got - want).max() <= TOL_ABS * max(1.0, np.abs(want).max())


def _random_cases(n, seed):
    r = np.random.default_rng(seed)
    cases = []
    for _ in range(n):
        fmt = FORMATS[int(r.integers(0, len(FORMATS)))]
        name = ["tiny", "llava", "qwen"][int(r.integers(0, 3))]
        cases.append((fmt, name, int(r.integers(1, 1500)), int(r.integers(1, 3)), int(r.integers(1, 3)),
                      [0.0, 0.0, 0.1, 0.5][int(r.integers(0, 4))], int(r.integers(1, 4))))
    return cases


@pytest.mark.parametrize("fmt,name,T,B,L,p,steps", _random_cases(12, 20250317),
                         ids=lambda v: _fmt_id(v) if isinstance(v, tuple) else str(v))
def test_seeded_random_shapes(fmt, name, T, B, L, p, steps):
    """Shapes nobody picked by hand: any token count below 1500 (any remainder modulo 32 and 160), one or two
    sequences and layers, with and without protected tokens, every key format."""
    wl = CONFIGS[name]
    if min(wl.l_v, T - T % 32) < 1:
        p = 0.0
    pair = Pair(wl, T, B=B, L=L, p=p, max_new=steps, k_ratio=fmt[0], one_bit=fmt[1])
    pair.flushed_chunks = {}
    pair.prefill()
    if T >= 32:
        for layer in range(L):
            _check_layer(pair, layer)
    for _ in range(steps):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS * max(1.0, np.abs(ref).max())
    assert pair.cache.status() == 0
