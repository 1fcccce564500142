"""Plain CPU oracle for the VidKV hot path (key / value quantizers, decode).

TEST INFRASTRUCTURE ONLY -- the product package never imports this module and
this module imports nothing from the product.  numpy only; slow on purpose.

What follows the paper, step by step, in its notation:

* ``gquant``            Eq. 4   n-bit asymmetric min/max quantizer ("GQuant")
* ``select_channels``   Algorithm 3 (range / TopK / D-mask / N-mask), Sec. 3.2(1)
* ``channel_variance`` / ``channel_outliers``   the two other channel metrics of Sec. 4.1(1)
* ``dft64`` / ``idft64``        the discrete Fourier transform written out as
                                 its defining matrix (no FFT routine)
* ``fft_1bit``          Eq. 5   sign code + mean-|.| scale in the frequency domain
* ``mixquant``          Algorithm 3 MixQuant (k = 0.5 : 64 two-bit + 64 one-bit; other k and the
                        plain min/max 1-bit code of 1BitQuant's other branch as parameters)
* ``quant_1p58``        Eq. 6 / Algorithm 2 "1.58Quant" (ternary, gamma = 0.7)
* ``stp_saliency``      Eq. 7   cross-modal scores I = X_v X_t^T, summed over the text tokens
* ``select_tokens``     Eq. 7 / Sec. 3.3(2): top n = floor(p * l_v) visual tokens
* ``stpquant``          Algorithm 2 STPQuant
* ``SlabCache``         Algorithm 1 Prefill / Decoding for one (layer, batch,
                        KV head); ``decode_step`` is Eq. 3 on the dequantized
                        cache plus the residual flush.

Precision.  Everything is float64 except the places where a floating-point
number decides an integer code.  Those decisions are taken in float32, the
precision the kernels use, exactly as stated here:

* stored metadata (scales ``s``, zero points ``z``) is IEEE binary16, rounded
  to nearest-even from the float32 (min/max based) or float64 (mean based)
  statistic; codes and thresholds are computed from the *rounded* metadata;
* Eq. 4 codes: ``rint((x - z) / s)`` with x, z, s widened to float32 and the
  subtraction, division and rounding done in float32 (rint = half to even);
* Eq. 6 threshold: ``alpha = float32(0.7) * float32(s)``, compared in float32;
* channel ranges: ``float32(max) - float32(min)`` in float32.

Readings of the paper that it leaves open (each is also listed in the design
notes of the repository):

* Eq. 5's ``sign(.)+1 in {0,1}`` is read as bit = [x >= 0]; the dequantized
  coefficient is ``(2*bit-1) * s`` (symmetric binary code, zero offset 0);
* the transform runs along the channel axis over the 64 normal channels of one
  token in ascending channel order, orthonormal (1/sqrt(N)) both ways;
* real and imaginary parts are separate columns (Algorithm 3 reshapes to
  ``[l, d*2]``); every statistic is per column per group of G = 32 tokens;
* Algorithm 2's ``Mean(|X|, dim=channel)`` is the per-channel mean over the
  (up to) 32 tokens of a group; the ternary code dequantizes to ``trit * s``;
* a zero-range group has s = 0, all codes 0, and dequantizes to z;
* a short last group takes its statistics over the elements present;
* TopK ties: larger value first, then lower index; index lists ascending.

Pins: every function here is checked in the CPU test-suite against closed
forms, brute force on tiny inputs, library routines on special cases and the
constants the paper prints.  The paper prints no worked numeric example, so
end-to-end values are "parity unpinned" by the paper itself; the pins are the
mathematical ones.
"""
from __future__ import annotations

import math

import numpy as np

G = 32          # group size (Sec. 4.1, implementation details)
R = 128         # residual length (Sec. 4.1)
GAMMA = np.float32(0.7)   # ternary threshold factor (Sec. 4.1, ablation on gamma)
N_FFT = 64      # number of normal (1-bit) channels at k = 0.5 with head_dim 128


# --------------------------------------------------------------------------
# Eq. 4 : n-bit asymmetric quantizer
# --------------------------------------------------------------------------
def gquant(x: np.ndarray, bits: int):
    """Eq. 4 applied to one group: x is [n_tokens, C]; statistics per column.

    Returns (codes int8 [n, C], s float16 [C], z float16 [C]).
    """
    x = np.asarray(x, dtype=np.float32)
    levels = np.float32(2 ** bits - 1)
    mn = x.min(axis=0)
    mx = x.max(axis=0)
    s_h = ((mx - mn) / levels).astype(np.float16)      # s = (max-min)/(2^n-1)
    z_h = mn.astype(np.float16)                        # z = min
    s = s_h.astype(np.float32)
    z = z_h.astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        q = np.rint((x - z) / s)                       # float32 throughout
    q = np.clip(q, np.float32(0), levels)
    q = np.where(s == 0, np.float32(0), q)
    return q.astype(np.int8), s_h, z_h


def gdequant(codes, s_h, z_h):
    """Eq. 4, second half: X' = Q * s + z (float64)."""
    return codes.astype(np.float64) * s_h.astype(np.float64) + z_h.astype(np.float64)


def gquant_groups(x: np.ndarray, bits: int):
    """Eq. 4 group-wise along tokens: x [T, C] -> codes [T, C], s, z [n_groups, C]."""
    T = x.shape[0]
    ng = (T + G - 1) // G
    codes = np.zeros(x.shape, dtype=np.int8)
    s = np.zeros((ng, x.shape[1]), dtype=np.float16)
    z = np.zeros((ng, x.shape[1]), dtype=np.float16)
    for g in range(ng):
        sl = slice(g * G, min((g + 1) * G, T))
        codes[sl], s[g], z[g] = gquant(x[sl], bits)
    return codes, s, z


def gdequant_groups(codes, s, z):
    out = np.zeros(codes.shape, dtype=np.float64)
    for g in range(s.shape[0]):
        sl = slice(g * G, min((g + 1) * G, codes.shape[0]))
        out[sl] = gdequant(codes[sl], s[g], z[g])
    return out


# --------------------------------------------------------------------------
# Algorithm 3, first lines : range-based channel selection
# --------------------------------------------------------------------------
def topk_indices(score: np.ndarray, n: int) -> np.ndarray:
    """Indices of the n largest entries; ties: larger first, then lower index.
    Returned in ascending index order."""
    score = np.asarray(score)
    order = sorted(range(score.shape[0]), key=lambda i: (-float(score[i]), i))
    return np.array(sorted(order[:n]), dtype=np.int64)


def channel_range(k: np.ndarray) -> np.ndarray:
    """Sec. 3.2(1): R = max(K) - min(K) per channel over all tokens (float32)."""
    k = np.asarray(k, dtype=np.float32)
    return k.max(axis=0) - k.min(axis=0)


def channel_variance(k: np.ndarray) -> np.ndarray:
    """Sec. 4.1(1), the Variance metric: population variance of each channel over the tokens (float64)."""
    k = np.asarray(k, dtype=np.float64)
    mean = k.sum(axis=0) / k.shape[0]
    return ((k - mean) ** 2).sum(axis=0) / k.shape[0]


def channel_outliers(k: np.ndarray, M: float = 3.0) -> np.ndarray:
    """Sec. 4.1(1), the Outliers metric: N = sum_i 1[K_i > M * mean(K)] per channel with M = 3.  The paper
    writes the comparison without magnitudes; for channels that are centred near zero that would count
    about half of the tokens whatever their spread, so the reading taken here compares magnitudes:
    |K_i| > M * mean_i |K_i|."""
    a = np.abs(np.asarray(k, dtype=np.float64))
    return (a > M * (a.sum(axis=0) / a.shape[0])).sum(axis=0).astype(np.int64)


def select_channels(k: np.ndarray, ratio: float = 0.5):
    """Algorithm 3: D-mask = TopK(range, k); N-mask = ~D-mask.

    Returns (abn_idx, nom_idx): ascending channel lists (2-bit / 1-bit)."""
    d = k.shape[1]
    n_abn = int(math.ceil(ratio * d))
    abn = topk_indices(channel_range(k), n_abn)
    mask = np.zeros(d, dtype=bool)
    mask[abn] = True
    nom = np.nonzero(~mask)[0].astype(np.int64)
    return abn, nom


# --------------------------------------------------------------------------
# Eq. 5 : frequency-domain 1-bit quantizer
# --------------------------------------------------------------------------
def dft_matrix(n: int) -> np.ndarray:
    """W[k, m] = exp(-2 pi i k m / n) / sqrt(n): the orthonormal DFT."""
    k = np.arange(n).reshape(n, 1)
    m = np.arange(n).reshape(1, n)
    return np.exp(-2j * np.pi * (k * m) / n) / np.sqrt(n)


def dft64(x: np.ndarray) -> np.ndarray:
    """Orthonormal DFT along the last axis, by its definition (matrix product)."""
    n = x.shape[-1]
    return np.asarray(x, dtype=np.float64) @ dft_matrix(n).T


def idft64(xf: np.ndarray) -> np.ndarray:
    """Inverse of ``dft64`` (conjugate matrix)."""
    n = xf.shape[-1]
    return xf @ np.conj(dft_matrix(n)).T


def fft_1bit(x: np.ndarray):
    """Eq. 5 on one group: x is [n_tokens, N] real (N normal channels).

    FFT along channels; the real and imaginary parts form 2N real columns
    (Algorithm 3, reshape to [l, d*2]); per column bit = [col >= 0] and
    s = Mean(|col|) over the group's tokens, stored in binary16.

    Returns (bits uint8 [n, 2N], s float16 [2N]); columns 0..N-1 are the real
    parts of bins 0..N-1, columns N..2N-1 the imaginary parts."""
    xf = dft64(x)
    cols = np.concatenate([xf.real, xf.imag], axis=-1)           # [n, 2N]
    bits = (cols >= 0).astype(np.uint8)
    s_h = np.abs(cols).mean(axis=0).astype(np.float16)
    # The input is real, so bins N/2+1 .. N-1 are the conjugates of bins N/2-1 .. 1, and one bit per
    # normal channel (the paper's bit count) pays for the N columns of the Hermitian half only
    # (``hermitian_pack_columns``).  The mirror bins are therefore not coded on their own: their bits
    # and scales follow from the half (real part equal, imaginary part negated).  This differs from
    # coding every column by its own sign only where a coefficient is exactly zero.
    n = x.shape[-1]
    for k in range(1, n // 2):
        bits[..., n - k] = bits[..., k]
        bits[..., n + n - k] = 1 - bits[..., n + k]
        s_h[n - k] = s_h[k]
        s_h[n + n - k] = s_h[n + k]
    return bits, s_h


def fft_1bit_dequant(bits, s_h):
    """Eq. 5, second half: X' = IFFT[(2 bit - 1) * s]; returns the real part and
    the largest imaginary magnitude (zero up to rounding by Hermitian symmetry)."""
    n2 = bits.shape[-1]
    n = n2 // 2
    vals = (2.0 * bits.astype(np.float64) - 1.0) * s_h.astype(np.float64)
    xf = vals[..., :n] + 1j * vals[..., n:]
    x = idft64(xf)
    return x.real, float(np.abs(x.imag).max()) if x.size else 0.0


def hermitian_pack_columns(n: int = N_FFT) -> np.ndarray:
    """Which of the 2n full-spectrum columns carry information for a real
    input, in storage order: Re0, Re(n/2), then Re_k, Im_k for k = 1..n/2-1.
    (The other columns follow from X[n-k] = conj(X[k]); Im0 = Im(n/2) = 0.)"""
    cols = [0, n // 2]
    for k in range(1, n // 2):
        cols += [k, n + k]
    return np.array(cols, dtype=np.int64)


# --------------------------------------------------------------------------
# Algorithm 3 : MixQuant
# --------------------------------------------------------------------------
def one_bit_mode(ratio: float) -> str:
    """Algorithm 3, 1BitQuant, and Sec. 4.1 (Implementation Details): the normal channels go through
    the FFT only at k = 0.5 and k = 0.75; every other k uses the plain 1-bit quantizer."""
    return "fft" if ratio in (0.5, 0.75) else "minmax"


def mixquant(k: np.ndarray, ratio: float = 0.5, one_bit: str = "auto"):
    """Algorithm 3 MixQuant on one chunk k [T, D] (T a multiple of G or not).

    one_bit: "fft" = Eq. 5 on the transformed normal channels, "minmax" = GQuant(bit=1) (Eq. 4 with
    n = 1) on the normal channels as they are, "auto" = the paper's choice for this k
    (``one_bit_mode``).  k = 1 leaves no normal channel.

    Returns a dict: abn_idx, nom_idx, codes2 [T, n_abn], s2, z2 [ng, n_abn], mode, and for "fft"
    bits1 [T, 2*n_nom] (full complex columns), s1 [ng, 2*n_nom]; for "minmax" codes1 [T, n_nom],
    s1 and z1 [ng, n_nom]."""
    k = np.asarray(k, dtype=np.float32)
    T = k.shape[0]
    mode = one_bit_mode(ratio) if one_bit == "auto" else one_bit
    abn, nom = select_channels(k, ratio)
    codes2, s2, z2 = gquant_groups(k[:, abn], 2)          # GQuant(X_abn, bit=2)
    ng = (T + G - 1) // G
    out = dict(abn_idx=abn, nom_idx=nom, codes2=codes2, s2=s2, z2=z2, T=T, mode=mode)
    if mode == "minmax":                                   # 1BitQuant without the transform
        out["codes1"], out["s1"], out["z1"] = gquant_groups(k[:, nom], 1)
        return out
    bits1 = np.zeros((T, 2 * len(nom)), dtype=np.uint8)
    s1 = np.zeros((ng, 2 * len(nom)), dtype=np.float16)
    for g in range(ng):                                    # 1BitQuant(X_nom)
        sl = slice(g * G, min((g + 1) * G, T))
        if len(nom):
            bits1[sl], s1[g] = fft_1bit(k[sl][:, nom])
    out["bits1"], out["s1"] = bits1, s1
    return out


def mixquant_dequant(mq) -> np.ndarray:
    """DeQuant of a MixQuant chunk -> K' [T, D] float64."""
    T = mq["T"]
    d = len(mq["abn_idx"]) + len(mq["nom_idx"])
    out = np.zeros((T, d), dtype=np.float64)
    out[:, mq["abn_idx"]] = gdequant_groups(mq["codes2"], mq["s2"], mq["z2"])
    if len(mq["nom_idx"]) == 0:
        return out
    if mq.get("mode", "fft") == "minmax":
        out[:, mq["nom_idx"]] = gdequant_groups(mq["codes1"], mq["s1"], mq["z1"])
        return out
    for g in range(mq["s1"].shape[0]):
        sl = slice(g * G, min((g + 1) * G, T))
        xr, _ = fft_1bit_dequant(mq["bits1"][sl], mq["s1"][g])
        out[sl.start:sl.stop, mq["nom_idx"]] = xr
    return out


# --------------------------------------------------------------------------
# Eq. 6 / Algorithm 2 : 1.58-bit (ternary) quantizer
# --------------------------------------------------------------------------
def quant_1p58(v: np.ndarray, gamma=GAMMA, scale: str = "mean_abs"):
    """Eq. 6 on one group v [n_tokens, C]: s = Mean|v| per channel (binary16),
    alpha = gamma * s, trit = +1 if v > alpha, -1 if v < -alpha, else 0.

    The paper gives the codes only; the scale that multiplies them back is a reading.
    ``scale="mean_abs"`` (the default) stores the same s.  ``scale="nonzero_mean"`` stores
    the mean of |v| over the elements whose trit is not 0 (0 where there is none), the
    least-squares scale for the given codes as in ternary weight networks, from which
    Eq. 6 takes its threshold; the codes are the same in both modes."""
    v = np.asarray(v, dtype=np.float32)
    s_h = np.abs(v.astype(np.float64)).mean(axis=0).astype(np.float16)
    alpha = np.float32(gamma) * s_h.astype(np.float32)
    trit = np.zeros(v.shape, dtype=np.int8)
    trit[v > alpha] = 1
    trit[v < -alpha] = -1
    if scale == "mean_abs":
        return trit, s_h
    assert scale == "nonzero_mean"
    nz = trit != 0
    total = (np.abs(v.astype(np.float64)) * nz).sum(axis=0)
    count = nz.sum(axis=0)
    s_nz = np.where(count > 0, total / np.maximum(count, 1), 0.0).astype(np.float16)
    return trit, s_nz


def quant_1p58_groups(v: np.ndarray, gamma=GAMMA, scale: str = "mean_abs"):
    T = v.shape[0]
    ng = (T + G - 1) // G
    trits = np.zeros(v.shape, dtype=np.int8)
    s = np.zeros((ng, v.shape[1]), dtype=np.float16)
    for g in range(ng):
        sl = slice(g * G, min((g + 1) * G, T))
        trits[sl], s[g] = quant_1p58(v[sl], gamma, scale)
    return trits, s


def dequant_1p58_groups(trits, s):
    out = np.zeros(trits.shape, dtype=np.float64)
    for g in range(s.shape[0]):
        sl = slice(g * G, min((g + 1) * G, trits.shape[0]))
        out[sl] = trits[sl].astype(np.float64) * s[g].astype(np.float64)
    return out


# --------------------------------------------------------------------------
# Eq. 7 / Sec. 3.3(2) : semantic token protection
# --------------------------------------------------------------------------
def n_protected(p, l_v: int) -> int:
    """n = floor(p * l_v) with p held in float32 (the config stores a float)."""
    return int(math.floor(float(np.float32(p)) * l_v))


def stp_saliency(x_v: np.ndarray, x_t: np.ndarray) -> np.ndarray:
    """Eq. 7: the cross-modal score matrix I[i, j] = X_v(i) . X_t(j) between the hidden
    states of the l_v visual tokens (x_v [l_v, d]) and of the l_t text tokens (x_t [l_t, d]).
    The paper ranks visual tokens by these scores without saying how the text axis is
    reduced; the reading taken here is the sum over the text tokens (the mean up to a
    constant, which does not change a ranking).  Returns the l_v row sums, float64."""
    I = x_v.astype(np.float64) @ x_t.astype(np.float64).T
    return I.sum(axis=1)


def select_tokens(saliency: np.ndarray, p, vis_begin: int, T: int) -> np.ndarray:
    """Mask E over T tokens: the top n visual tokens by saliency are protected.
    saliency [l_v] scores the visual tokens vis_begin .. vis_begin+l_v-1."""
    l_v = saliency.shape[0]
    n = n_protected(p, l_v)
    E = np.zeros(T, dtype=bool)
    if n > 0:
        E[vis_begin + topk_indices(saliency, n)] = True
    return E


def stpquant(v: np.ndarray, E: np.ndarray, gamma=GAMMA, scale: str = "mean_abs"):
    """Algorithm 2 STPQuant: X[E] -> 2-bit GQuant per channel, X[~E] -> 1.58Quant;
    both streams keep ascending token order and are grouped by 32 in that order."""
    v = np.asarray(v, dtype=np.float32)
    prot_idx = np.nonzero(E)[0]
    rest_idx = np.nonzero(~E)[0]
    codes2, s2, z2 = gquant_groups(v[prot_idx], 2) if len(prot_idx) else (
        np.zeros((0, v.shape[1]), np.int8), np.zeros((0, v.shape[1]), np.float16),
        np.zeros((0, v.shape[1]), np.float16))
    trits, st = quant_1p58_groups(v[rest_idx], gamma, scale)
    return dict(prot_idx=prot_idx, rest_idx=rest_idx, codes2=codes2, s2=s2, z2=z2,
                trits=trits, st=st, T=v.shape[0])


def stp_dequant(sq) -> np.ndarray:
    d = sq["trits"].shape[1]
    out = np.zeros((sq["T"], d), dtype=np.float64)
    if len(sq["prot_idx"]):
        out[sq["prot_idx"]] = gdequant_groups(sq["codes2"], sq["s2"], sq["z2"])
    out[sq["rest_idx"]] = dequant_1p58_groups(sq["trits"], sq["st"])
    return out


# --------------------------------------------------------------------------
# Eq. 3 : attention of one query token over a cache
# --------------------------------------------------------------------------
def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """A = Softmax(q K^T * scale) V for q [n_q, D], K, V [T, D]; float64."""
    logits = (np.asarray(q, np.float64) @ np.asarray(K, np.float64).T) * scale
    logits -= logits.max(axis=-1, keepdims=True)
    w = np.exp(logits)
    w /= w.sum(axis=-1, keepdims=True)
    return w @ np.asarray(V, np.float64)


def attention_partial(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float):
    """Eq. 3 restricted to a shard of the token axis, left unnormalised: per query row the largest
    logit m (natural units, -inf for an empty shard), l = sum_t exp(logit_t - m) and
    o = sum_t exp(logit_t - m) V_t.  Softmax(q K^T) V over the union of shards follows from these
    triples alone (merge_partials)."""
    q = np.asarray(q, np.float64)
    K = np.asarray(K, np.float64)
    V = np.asarray(V, np.float64)
    if K.shape[0] == 0:
        return np.full(q.shape[0], -np.inf), np.zeros(q.shape[0]), np.zeros((q.shape[0], V.shape[1]))
    logits = (q @ K.T) * scale
    m = logits.max(axis=-1)
    w = np.exp(logits - m[:, None])
    return m, w.sum(axis=-1), w @ V


def merge_partials(parts):
    """Combine (m, l, o) triples of disjoint token shards: out = sum_p e^(m_p - M) o_p / sum_p e^(m_p - M) l_p."""
    M = np.max(np.stack([p[0] for p in parts]), axis=0)
    num = sum(np.where(np.isfinite(p[0]), np.exp(p[0] - M), 0.0)[:, None] * p[2] for p in parts)
    den = sum(np.where(np.isfinite(p[0]), np.exp(p[0] - M), 0.0) * p[1] for p in parts)
    return num / den[:, None]


# --------------------------------------------------------------------------
# Algorithm 1 : Prefill / Decoding for one (layer, batch element, KV head)
# --------------------------------------------------------------------------
class SlabCache:
    """KV cache of one (layer, batch element, KV head): the 4-tuple of
    Algorithm 1, Q(X_Kq), X_Kr, Q(X_Vq), X_Vr, with the key part kept as a list
    of independently MixQuant-ed chunks (prefill chunk, then one per flush)."""

    def __init__(self, ratio: float = 0.5, gamma=GAMMA, ternary_scale: str = "mean_abs", one_bit: str = "auto"):
        self.ratio = ratio
        self.one_bit = one_bit
        self.gamma = gamma
        self.ternary_scale = ternary_scale
        self.k_chunks = []        # list of mixquant dicts
        self.v_prefill = None     # stpquant dict of the prefill tokens
        self.v_flush = []         # list of (trits, s) per flushed residual
        self.k_res = None         # [r, D] float32 (exact input values)
        self.v_res = None

    # Algorithm 1, procedure Prefill
    def prefill(self, k: np.ndarray, v: np.ndarray, E: np.ndarray | None = None):
        k = np.asarray(k, dtype=np.float32)
        v = np.asarray(v, dtype=np.float32)
        l = k.shape[0]
        r = l % G
        kq, self.k_res = k[:l - r], k[l - r:].copy()
        vq, self.v_res = v[:l - r], v[l - r:].copy()
        if E is None:
            E = np.zeros(l, dtype=bool)
        self.v_prefill = stpquant(vq, np.asarray(E[:l - r], dtype=bool), self.gamma, self.ternary_scale)
        self.k_chunks = [mixquant(kq, self.ratio, self.one_bit)] if l - r > 0 else []

    def dequant_k(self) -> np.ndarray:
        """DeQuant(Q(X_Kq)); each chunk's result is kept once computed."""
        for c in self.k_chunks:
            if "_deq" not in c:
                c["_deq"] = mixquant_dequant(c)
        parts = [c["_deq"] for c in self.k_chunks]
        d = self.k_res.shape[1]
        return np.concatenate(parts, axis=0) if parts else np.zeros((0, d))

    def dequant_v(self) -> np.ndarray:
        if self.v_prefill["T"] and "_deq" not in self.v_prefill:
            self.v_prefill["_deq"] = stp_dequant(self.v_prefill)
        parts = [self.v_prefill["_deq"]] if self.v_prefill["T"] else []
        parts += [dequant_1p58_groups(t, s) for (t, s) in self.v_flush]
        d = self.v_res.shape[1]
        return np.concatenate(parts, axis=0) if parts else np.zeros((0, d))

    @property
    def n_quantized(self) -> int:
        return sum(c["T"] for c in self.k_chunks)

    # Algorithm 1, procedure Decoding
    def decode_step(self, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                    scale: float | None = None) -> np.ndarray:
        """q [n_q, D] are the query heads served by this KV head."""
        d = self.k_res.shape[1]
        if scale is None:
            scale = 1.0 / math.sqrt(d)
        self.k_res = np.concatenate([self.k_res, np.asarray(k_new, np.float32).reshape(1, d)])
        self.v_res = np.concatenate([self.v_res, np.asarray(v_new, np.float32).reshape(1, d)])
        K = np.concatenate([self.dequant_k(), self.k_res.astype(np.float64)])
        V = np.concatenate([self.dequant_v(), self.v_res.astype(np.float64)])
        out = attention(q, K, V, scale)
        if self.v_res.shape[0] == R:                      # residual flush
            self.v_flush.append(quant_1p58_groups(self.v_res, self.gamma, self.ternary_scale))
            self.k_chunks.append(mixquant(self.k_res, self.ratio, self.one_bit))
            self.k_res = np.zeros((0, d), dtype=np.float32)
            self.v_res = np.zeros((0, d), dtype=np.float32)
        return out
