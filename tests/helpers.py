"""Shared helpers of the GPU parity tests: run the oracle and the library on the same
seeded inputs and compare packed codes, metadata, dequantized tensors and outputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import vidkv_oracle as O
from tests import unpack as U
from workloads import make_layer_kv, make_saliency, make_step_inputs

TOL_ABS = 2e-3          # dequantized K/V and attention outputs (max-abs)
TIE_REL = 1e-3          # a code may differ only within TIE_REL * scale of its threshold
TIE_FRAC = 1e-4         # ... and on at most this fraction of the elements


def f16_ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    def key(x):
        i = x.astype(np.float16).view(np.int16).astype(np.int32)
        return np.where(i < 0, -(i & 0x7FFF), i)
    return np.abs(key(a) - key(b))


def to_np(x: torch.Tensor) -> np.ndarray:
    return x.detach().float().cpu().numpy()


class Pair:
    """One configuration run through both implementations (all layers, all slabs)."""

    def __init__(self, wl, T, B=None, L=None, p=0.0, max_new=16, device="cuda", ternary_scale="mean_abs",
                 k_ratio=0.5, one_bit="fft"):
        import paper_2503_16257_b200 as P
        self.P = P
        self.wl, self.T, self.p = wl, T, p
        self.B = wl.batch if B is None else B
        self.L = wl.layers if L is None else L
        self.device = device
        in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
        self.cfg = P.VidKVConfig(B=self.B, L=self.L, max_prefill_tokens=T, max_new_tokens=max_new, p_ratio=p,
                                 in_dtype=in_dt, out_dtype=P.VIDKV_F32, k_ratio=k_ratio,
                                 key_1bit_mode=P.VIDKV_KEY1BIT_PLAIN_MINMAX if one_bit == "minmax" else P.VIDKV_KEY1BIT_FFT_SIGN,
                                 ternary_scale=P.VIDKV_TERNARY_SCALE_NONZERO_MEAN if ternary_scale == "nonzero_mean"
                                 else P.VIDKV_TERNARY_SCALE_MEAN_ABS)
        self.ternary_scale = ternary_scale
        self.k_ratio, self.one_bit = k_ratio, one_bit
        self.cache = P.VidKVCache(self.cfg, device=device)
        self.lay = self.cache.layout
        self.l_v = min(wl.l_v, T - T % 32)
        self.K, self.V = [], []
        self.slabs = {}
        self.E = None
        self.step = 0
        self.sign_tie_tokens = {}  # per slab: prefill tokens whose sign bits differ from the oracle's at a tie
        self.res_in = {}          # inputs currently in the residual, per slab
        self.flushed_in = {}      # inputs of the most recent flush, per slab

    # ---- prefill on both sides
    def prefill(self):
        sal = None
        if self.p > 0:
            sal = make_saliency(self.wl, "cpu", l_v=self.l_v, B=self.B)
            self.cache.select_tokens(sal.to(self.device), 0, self.l_v, self.T)
            self.E = [O.select_tokens(sal[b].numpy(), self.p, 0, self.T - self.T % 32) for b in range(self.B)]
        for layer in range(self.L):
            K, V = make_layer_kv(self.wl, layer, "cpu", T=self.T, B=self.B)
            self.K.append(K); self.V.append(V)
            Kd, Vd = K.to(self.device), V.to(self.device)
            self.cache.quantize_keys(layer, Kd)
            self.cache.quantize_values(layer, Vd)
            for b in range(self.B):
                for h in range(self.cfg.H_kv):
                    sc = O.SlabCache(ratio=self.k_ratio, ternary_scale=self.ternary_scale, one_bit=self.one_bit)
                    E = None
                    if self.E is not None:
                        E = np.zeros(self.T, dtype=bool)
                        E[: self.T - self.T % 32] = self.E[b]
                    sc.prefill(to_np(K[b, h]), to_np(V[b, h]), E)
                    self.slabs[(layer, b, h)] = sc
                    self.res_in[(layer, b, h)] = (list(sc.k_res), list(sc.v_res))
        torch.cuda.synchronize()
        return self

    def cache_bytes(self) -> np.ndarray:
        torch.cuda.synchronize()
        return self.cache.cache.cpu().numpy()

    # ---- one decode step on both sides; returns (lib_out, oracle_out) as [L, B, H_q, D] arrays
    def decode(self):
        qs, ks, vs = [], [], []
        for layer in range(self.L):
            q, k, v = make_step_inputs(self.wl, layer, self.step, "cpu", T=self.T, B=self.B)
            qs.append(q); ks.append(k); vs.append(v)
        q, k, v = torch.stack(qs), torch.stack(ks), torch.stack(vs)
        out = torch.empty((self.L, self.B, self.cfg.H_q, self.cfg.D), dtype=torch.float32, device=self.device)
        self.cache.decode_attention(0, self.L, q.to(self.device), k.to(self.device), v.to(self.device), out)
        rep = self.cfg.H_q // self.cfg.H_kv
        ref = np.zeros((self.L, self.B, self.cfg.H_q, self.cfg.D))
        for layer in range(self.L):
            for b in range(self.B):
                for h in range(self.cfg.H_kv):
                    sc = self.slabs[(layer, b, h)]
                    rk, rv = self.res_in[(layer, b, h)]
                    rk.append(to_np(k[layer, b, h])); rv.append(to_np(v[layer, b, h]))
                    if len(rk) == O.R:
                        self.flushed_in[(layer, b, h)] = (np.stack(rk), np.stack(rv))
                        self.res_in[(layer, b, h)] = ([], [])
                    ref[layer, b, h * rep:(h + 1) * rep] = sc.decode_step(
                        to_np(q[layer, b, h * rep:(h + 1) * rep]), to_np(k[layer, b, h]), to_np(v[layer, b, h]))
        self.step += 1
        torch.cuda.synchronize()
        return out.cpu().numpy().astype(np.float64), ref


# ---------------------------------------------------------------------------- comparisons
def compare_key_chunk(slab, lay, chunk_idx, g_begin, mq, k_chunk, stats):
    """Packed key chunk vs the oracle's MixQuant dict; k_chunk [T, D] are the chunk's inputs."""
    abn, nom = U.chunk_perm(slab, lay, chunk_idx)
    assert (abn == mq["abn_idx"]).all(), "anomalous channel list differs"
    assert (nom == mq["nom_idx"]).all(), "normal channel list differs"
    T = mq["T"]
    ng = T // 32
    codes2, bits1, s2, z2, s1 = U.key_groups(slab, lay, g_begin, ng)
    assert (s2.view(np.int16) == mq["s2"].view(np.int16)).all(), "2-bit scales differ"
    assert (z2.view(np.int16) == mq["z2"].view(np.int16)).all(), "2-bit zero points differ"
    assert (codes2 == mq["codes2"]).all(), "2-bit codes differ"
    pk = O.hermitian_pack_columns(64)
    o_bits, o_s1 = mq["bits1"][:, pk], mq["s1"][:, pk]
    ulp = f16_ulp_distance(s1, o_s1)
    assert ulp.max() <= 1, f"1-bit scales differ by {ulp.max()} ulp"
    stats["s1_n"] += ulp.size; stats["s1_off"] += int((ulp > 0).sum())
    bad = bits1 != o_bits
    stats["bits_n"] += bad.size; stats["bits_off"] += int(bad.sum())
    if bad.any():
        xf = O.dft64(k_chunk[:, nom])
        cols = np.concatenate([xf.real, xf.imag], -1)[:, pk]
        scale = np.repeat(o_s1.astype(np.float64), 32, axis=0)
        assert (np.abs(cols[bad]) <= TIE_REL * scale[bad] + 1e-12).all(), "a sign bit differs away from zero"
    return np.nonzero(bad.any(axis=1))[0]          # tokens of the chunk with a sign bit at a tie


def compare_ternary(trits, s, o_trits, o_s, v_stream, stats, gamma=0.7, o_s_thr=None):
    """o_s_thr: the oracle's Mean |v| scales where the stored scale is a different statistic (the
    threshold always comes from Mean |v|)."""
    n = o_trits.shape[0]
    bad = trits[:n] != o_trits
    ulp = f16_ulp_distance(s, o_s)
    if o_s_thr is not None and bad.any():
        # a stored scale that averages over the non-zero codes moves when a code at a tie differs
        ng = o_s.shape[0]
        pad = np.zeros((ng * 32, bad.shape[1]), dtype=bool)
        pad[:n] = bad
        ulp = np.where(pad.reshape(ng, 32, -1).any(axis=1), 0, ulp)
    assert ulp.max() <= 1, f"ternary scales differ by {ulp.max()} ulp"
    stats["st_n"] += ulp.size; stats["st_off"] += int((ulp > 0).sum())
    stats["trit_n"] += bad.size; stats["trit_off"] += int(bad.sum())
    if bad.any():
        thr_s = o_s if o_s_thr is None else o_s_thr
        ulp_thr = ulp if o_s_thr is None else np.ones_like(ulp)
        ng = o_s.shape[0]
        srow = np.repeat(thr_s.astype(np.float64), 32, axis=0)[:n]
        urow = np.repeat(ulp_thr, 32, axis=0)[:n]
        dist = np.abs(np.abs(v_stream.astype(np.float64)) - gamma * srow)
        tol = TIE_REL * srow + urow * srow * 2.0 ** -10
        assert (dist[bad] <= tol[bad] + 1e-12).all(), "a trit differs away from the threshold"


def new_stats():
    return dict(s1_n=0, s1_off=0, bits_n=0, bits_off=0, st_n=0, st_off=0, trit_n=0, trit_off=0)


def check_stats(stats):
    if stats["bits_n"]:
        assert stats["bits_off"] <= max(1, TIE_FRAC * stats["bits_n"]), stats
    if stats["trit_n"]:
        assert stats["trit_off"] <= max(1, TIE_FRAC * stats["trit_n"]), stats
    # binary16 rounding of mean-based scales: float32 vs float64 summation may land on
    # neighbouring binary16 values for a small share of the scales
    if stats["s1_n"]:
        assert stats["s1_off"] <= max(2, 1e-2 * stats["s1_n"]), stats
    if stats["st_n"]:
        assert stats["st_off"] <= max(2, 1e-2 * stats["st_n"]), stats
