"""CPU-side checks of libvidkv.so: it loads, exports every function the header declares,
and its host-only entry points (sizing, layout, argument validation) behave."""
import ctypes
import os
import re

import pytest

import paper_2503_16257_b200 as P
from paper_2503_16257_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.load_library()


def _header_functions():
    text = open(os.path.join(ROOT, "include", "vidkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vidkv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _header_functions()
    assert len(names) >= 14
    raw = ctypes.CDLL(P.library_path())
    for n in names:
        assert hasattr(raw, n), f"{n} declared in include/vidkv.h but not exported"
    assert set(names) == set(P.exported_symbols())


def test_version(lib):
    assert P.vidkv_version() >= 100


def test_bytes_per_token_accounting(lib):
    # one 32-token key group: 64 ch x 2 bit + 64 ch x 1 bit + (s, z, s) binary16 x 64
    assert 32 * (64 * 2 + 64 * 1) // 8 + 3 * 64 * 2 == 1152          # 36 B / token / head -> 1.5 bit + metadata
    assert (64 * 2 + 64 * 1) / 128 == 1.5
    # one ternary supergroup: 160 tokens x 128 ch x 1.6 bit + 5 x 128 binary16 scales
    assert 160 * 128 // 5 + 5 * 128 * 2 == 5376                      # 33.6 B / token / head
    assert 8 / 5 == 1.6 and 3 ** 5 <= 256
    # one protected group: 32 tokens x 128 ch x 2 bit + (s, z) binary16 x 128
    assert 32 * 128 * 2 // 8 + 2 * 128 * 2 == 1536                   # 48 B / token / head
    cfg = P.VidKVConfig(B=4, L=28, max_prefill_tokens=196000, max_new_tokens=64)
    lay = P.vidkv_cache_layout(cfg)
    assert lay["max_kgroups"] == 6125 and lay["max_chunks"] == 1
    packed = lay["max_kgroups"] * 1152 + lay["max_supergroups"] * 5376
    fp16 = 196000 * 128 * 2 * 2
    assert 0.13 < packed / fp16 < 0.14                               # ~86 % smaller than FP16 K+V
    cache_bytes, ws_bytes = P.vidkv_cache_bytes(cfg)
    assert cache_bytes == lay["total_bytes"] and cache_bytes < 0.15 * fp16 * 4 * 4 * 28
    assert ws_bytes > 0


def test_layout_regions_do_not_overlap(lib):
    for p in (0.0, 0.2):
        cfg = P.VidKVConfig(B=2, L=3, max_prefill_tokens=1000, max_new_tokens=300, p_ratio=p)
        lay = P.vidkv_cache_layout(cfg)
        regions = [
            (lay["chunk_table_offset"], lay["max_chunks"] * 128),
            (lay["kgroup_offset"], lay["max_kgroups"] * 1152),
            (lay["tern_offset"], lay["max_supergroups"] * 5376),
            (lay["prot_offset"], lay["max_pgroups"] * 1536),
            (lay["kres_offset"], 128 * 128 * 2),
            (lay["vres_offset"], 128 * 128 * 2),
        ]
        end = 0
        for off, size in regions:
            assert off >= end and off % 128 == 0
            end = off + size
        assert end <= lay["slab_stride"] and lay["slab_stride"] % 256 == 0
        assert lay["slab_offset"] >= lay["sel_offset"] + 2 * lay["sel_stride_b"]
        assert lay["total_bytes"] == lay["slab_offset"] + lay["slab_stride"] * 3 * 2 * 4
        # 1000 prefill tokens -> 31 groups; (31 + 300) // 128 = 2 flushes possible
        assert lay["max_chunks"] == 3 and lay["max_kgroups"] == 31 + 8
        assert lay["max_pgroups"] == (0 if p == 0 else (200 + 31) // 32)


@pytest.mark.parametrize("kw,status", [
    (dict(D=64), -2), (dict(G=64), -2), (dict(R=64), -2), (dict(k_ratio=0.6), -2),
    (dict(H_q=30), -2), (dict(H_q=64), -2), (dict(key_1bit_mode=2), -1), (dict(k_ratio=0.25, key_1bit_mode=0), -2),
    (dict(B=0), -1), (dict(p_ratio=1.5), -1), (dict(p_ratio=-0.1), -1), (dict(in_dtype=2), -1),
    (dict(out_dtype=7), -1), (dict(max_new_tokens=-1), -1), (dict(gamma=float("nan")), -1),
    (dict(ternary_scale=2), -1),
])
def test_config_validation(lib, kw, status):
    base = dict(B=1, L=1, max_prefill_tokens=64, max_new_tokens=4)
    base.update(kw)
    with pytest.raises(P.VidKVError) as e:
        P.vidkv_cache_bytes(P.VidKVConfig(**base))
    assert e.value.status == status


@pytest.mark.parametrize("k_ratio,mode,group_bytes", [
    (0.5, 0, 1152), (0.25, 1, 1152), (0.5, 1, 1280), (0.75, 1, 1408), (0.75, 0, 1344), (1.0, 0, 1536), (1.0, 1, 1536)])
def test_key_group_bytes_follow_the_key_format(lib, k_ratio, mode, group_bytes):
    """2 bits per anomalous channel, 1 bit per normal one, a binary16 (s, z) pair per two-bit channel,
    one binary16 scale per spectrum column or an (s, z) pair per plain one-bit channel, per 32 tokens."""
    n2 = int(k_ratio * 128)
    n1 = 128 - n2
    assert group_bytes == (2 * n2 + n1) * 32 // 8 + 4 * n2 + (4 if mode == 1 else 2) * n1
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=320, max_new_tokens=0, k_ratio=k_ratio, key_1bit_mode=mode)
    lay = P.vidkv_cache_layout(cfg)
    assert lay["max_kgroups"] == 10
    assert lay["tern_offset"] - lay["kgroup_offset"] == -(-10 * group_bytes // 256) * 256


def test_null_arguments_are_rejected_without_a_device(lib):
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=64, max_new_tokens=4).to_c()
    assert lib.vidkv_cache_bytes(ctypes.byref(cfg), None, None) == -1
    assert lib.vidkv_cache_layout(None, None) == -1
    h = ctypes.c_void_p()
    assert lib.vidkv_cache_init(ctypes.byref(cfg), None, 0, None, 0, None, ctypes.byref(h)) == -1
    assert lib.vidkv_cache_init(ctypes.byref(cfg), ctypes.c_void_p(0x1001), 1 << 30, ctypes.c_void_p(0x1000), 1 << 30,
                                None, ctypes.byref(h)) == -3
    assert lib.vidkv_cache_init(ctypes.byref(cfg), ctypes.c_void_p(0x1000), 16, ctypes.c_void_p(0x1000), 16,
                                None, ctypes.byref(h)) == -4
    assert lib.vidkv_cache_destroy(None) == -1
    assert lib.vidkv_decode_attention(None, 0, 1, None, None, None, None, 0.0, None) == -1


def test_saliency_scores_argument_checks_without_a_device(lib):
    f = lib.vidkv_saliency_scores
    a = ctypes.c_void_p(0x1000)
    assert f(7, a, a, 1, 4, 2, 64, a, a, None) == -1                      # unknown dtype
    assert f(P.VIDKV_F16, a, a, -1, 4, 2, 64, a, a, None) == -1           # negative size
    assert f(P.VIDKV_F16, None, a, 1, 4, 2, 64, a, a, None) == -1         # null input
    assert f(P.VIDKV_F16, a, a, 0, 4, 2, 64, a, a, None) == 0             # nothing to do
    assert f(P.VIDKV_F16, a, a, 1, 4, 2, 12, a, a, None) == -2            # d not a multiple of 8
    assert f(P.VIDKV_F16, a, a, 1, 4, 2, 32768, a, a, None) == -2         # d beyond the supported width
    assert f(P.VIDKV_F16, ctypes.c_void_p(0x1004), a, 1, 4, 2, 64, a, a, None) == -3   # misaligned


def test_channel_metrics_argument_checks_without_a_device(lib):
    f = lib.vidkv_channel_metrics
    a = ctypes.c_void_p(0x1000)
    ok = (P.VIDKV_F16, a, 1, 4, 64, 4 * 64 * 128, 64 * 128, 128, P.VIDKV_METRIC_VARIANCE, 3.0, a, a, None)
    def call(**kw):
        names = ["dtype", "K", "B", "H", "T", "sb", "sh", "st", "metric", "M", "scratch", "out", "stream"]
        args = list(ok)
        for k, v in kw.items():
            args[names.index(k)] = v
        return f(*args)
    assert call(dtype=5) == -1 and call(metric=0) == -1 and call(metric=3) == -1     # unknown dtype / metric
    assert call(T=0) == -1 and call(M=0.0) == -1 and call(M=float("nan")) == -1
    assert call(K=None) == -1 and call(out=None) == -1
    assert call(B=0) == 0                                                              # nothing to do
    assert call(st=100) == -3 and call(sh=4) == -3                                     # strides
    assert call(K=ctypes.c_void_p(0x1002)) == -3                                       # misaligned


@pytest.mark.parametrize("B,L,T_max,max_new,p", [
    (4, 1, 24000, 16, 0.2),      # a shorter prompt picks shorter splits and needs about twice the records
    (1, 1, 100000, 16, 0.2),
    (4, 1, 24000, 16, 0.0),
    (16, 28, 12544, 128, 0.2),   # the batched workload
    (1, 28, 6400, 256, 0.0),
    (2, 3, 700, 300, 0.5),
])
def test_partial_records_fit_the_workspace_for_every_token_count(lib, B, L, T_max, max_new, p):
    """The workspace is sized once, from the configured maxima; how a decode call is cut into work
    depends on the live token count and on how many layers the call covers.  Whatever they are,
    the records the plan needs must fit what was reserved."""
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T_max, max_new_tokens=max_new, p_ratio=p)
    step = max(32, (T_max // 400) // 32 * 32)
    tokens = sorted(set(list(range(0, T_max + 1, step)) + [T_max - T_max % 32] +
                        [t for t in (32, 160, 320, 640, 1280, 18912, 18944, 23008, 23040) if t <= T_max]))
    worst = 0
    for n_layers in sorted({1, L, max(1, L // 2)}):
        for sm in (1, 132, 148, 1000):
            for T in tokens:
                T = T - T % 32
                n_prot = int(p * T) // 2
                for n_flush, n_res in ((0, 1), (0, 128), (max_new // 128, 77)):
                    for prot in sorted({0, n_prot}):
                        pl = P.vidkv_debug_decode_plan(cfg, T, n_flush, n_res, prot, n_layers, sm_count=sm)
                        assert pl["records"] <= pl["records_capacity"], (n_layers, sm, T, n_flush, n_res, prot, pl)
                        worst = max(worst, pl["records"])
                        if T > 0:
                            assert pl["n_units"] == n_layers * B * 4 * pl["units_per_slab"]
                            assert pl["n_runs"] * pl["run_units"] >= pl["n_units"]
                            assert pl["parts_stride"] >= -(-pl["units_per_slab"] // pl["run_units"]) + 1
    assert worst > 0
    # a plan forced through the test hook may need more than was reserved (the decode call then
    # returns VIDKV_ERR_CAPACITY); on problems with fewer units than the largest launch has warps, one
    # unit per run still fits
    T = T_max - T_max % 32
    if B * L * 4 * (-(-T // 160)) <= 256 * 12:
        assert P.vidkv_debug_decode_plan(cfg, T, 0, 1, 0, L, run_units=1)["records"] <= \
            P.vidkv_debug_decode_plan(cfg, T, 0, 1, 0, L)["records_capacity"]


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2503_16257_b200.api as api
    monkeypatch.setattr(api, "_LIB", None)
    monkeypatch.setattr(api, "library_path", lambda: "/nonexistent/libvidkv.so")
    with pytest.raises(RuntimeError):
        api.load_library()
