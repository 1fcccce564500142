"""Test-side reader of the packed cache format documented in include/vidkv.h.

Written from the format description only: it turns the bytes of one slab back into
plain integer codes and binary16 metadata so that they can be compared with the
oracle's unpacked codes.  It contains no quantizer arithmetic."""
from __future__ import annotations

import numpy as np

G, R, D = 32, 128, 128
KG_BYTES, SG_BYTES, PG_BYTES, CHUNK_BYTES = 1152, 5376, 1536, 128


def _tern_offsets():
    """Byte offset of (stream token j, channel c) inside the 4096-byte plane of a supergroup."""
    j = np.arange(G)[:, None]
    c = np.arange(D)[None, :]
    m = j // 2
    kt, u, r = m // 8, (m // 4) % 2, m % 4
    w, rho, e = c // 32, (c // 4) % 8, c % 4
    return (((((kt * 2 + u) * 4 + w) * 4 + r) * 8 + rho) * 8) + 2 * e + j % 2


TERN_OFF = _tern_offsets()


def slab_bytes(cache: np.ndarray, lay: dict, cfg, layer: int, b: int, h: int) -> np.ndarray:
    idx = (layer * cfg.B + b) * cfg.H_kv + h
    off = lay["slab_offset"] + idx * lay["slab_stride"]
    return cache[off: off + lay["slab_stride"]]


def chunk_perm(slab: np.ndarray, lay: dict, chunk: int):
    e = slab[lay["chunk_table_offset"] + chunk * CHUNK_BYTES:][:CHUNK_BYTES]
    return e[:64].astype(np.int64), e[64:].astype(np.int64)


def key_groups(slab: np.ndarray, lay: dict, g_begin: int, n_groups: int):
    """-> codes2 [32*n, 64] int8, bits1 [32*n, 64] uint8, s2, z2, s1 [n, 64] float16."""
    codes2 = np.zeros((n_groups * G, 64), np.int8)
    bits1 = np.zeros((n_groups * G, 64), np.uint8)
    s2 = np.zeros((n_groups, 64), np.float16)
    z2 = np.zeros((n_groups, 64), np.float16)
    s1 = np.zeros((n_groups, 64), np.float16)
    j = np.arange(64)
    t = np.arange(G)
    # word / half-word index of (token t, slot or column j): ((t % 8) * 4 + j // 16) * 4 + t // 8
    idx = ((t[:, None] % 8) * 4 + j[None, :] // 16) * 4 + t[:, None] // 8
    bit2 = 2 * ((j % 16) // 2) + 16 * (j % 2)
    bit1 = 15 - j % 16
    for g in range(n_groups):
        rec = slab[lay["kgroup_offset"] + (g_begin + g) * KG_BYTES:][:KG_BYTES]
        w2 = rec[0:512].view("<u4")
        codes2[g * G:(g + 1) * G] = (w2[idx] >> bit2[None, :]) & 3
        w1 = rec[512:768].view("<u2")
        bits1[g * G:(g + 1) * G] = (w1[idx] >> bit1[None, :]) & 1
        s2[g] = rec[768:896].view("<f2")
        z2[g] = rec[896:1024].view("<f2")
        s1[g] = rec[1024:1152].view("<f2")
    return codes2, bits1, s2, z2, s1


def ternary_groups(slab: np.ndarray, lay: dict, g_begin: int, n_groups: int):
    """-> trits [32*n, 128] int8, s [n, 128] float16 for ternary stream groups g_begin.."""
    trits = np.zeros((n_groups * G, D), np.int8)
    s = np.zeros((n_groups, D), np.float16)
    for k in range(n_groups):
        gi = g_begin + k
        rec = slab[lay["tern_offset"] + (gi // 5) * SG_BYTES:][:SG_BYTES]
        slot = gi % 5
        q = rec[:4096].astype(np.int64)[TERN_OFF]
        bval = (q * 243) >> 8
        digit = (bval // 3 ** (4 - slot)) % 3
        trits[k * G:(k + 1) * G] = digit - 1
        s[k] = rec[4096 + slot * 256: 4096 + (slot + 1) * 256].view("<f2")
    return trits, s


def protected_groups(slab: np.ndarray, lay: dict, n_groups: int):
    codes = np.zeros((n_groups * G, D), np.int8)
    s = np.zeros((n_groups, D), np.float16)
    z = np.zeros((n_groups, D), np.float16)
    j = np.arange(G)[:, None]
    c = np.arange(D)[None, :]
    widx = (((j // 16) * 4 + c // 32) * 4 + (j // 2) % 4) * 8 + (c // 4) % 8
    bit = 2 * (4 * ((j // 8) % 2) + c % 4) + 16 * (j % 2)
    for g in range(n_groups):
        rec = slab[lay["prot_offset"] + g * PG_BYTES:][:PG_BYTES]
        w = rec[:1024].view("<u4")
        codes[g * G:(g + 1) * G] = (w[widx] >> bit) & 3
        s[g] = rec[1024:1280].view("<f2")
        z[g] = rec[1280:1536].view("<f2")
    return codes, s, z


def residual(slab: np.ndarray, lay: dict, which: str, n: int, torch_dtype):
    import torch
    off = lay["kres_offset"] if which == "k" else lay["vres_offset"]
    raw = slab[off: off + n * D * 2].copy()
    return torch.from_numpy(raw).view(torch_dtype).reshape(n, D).float().numpy()


def selection_mask(cache: np.ndarray, lay: dict, b: int, T_q: int):
    off = lay["sel_offset"] + b * lay["sel_stride_b"]
    words = cache[off: off + 4 * lay["sel_words"]].view("<u4")
    prefix = cache[off + 4 * lay["sel_words"]: off + 8 * lay["sel_words"]].view("<u4")
    t = np.arange(T_q)
    E = ((words[t // 32] >> (t % 32)) & 1).astype(bool)
    return E, prefix


def general_key_group_bytes(n2: int, plain: bool) -> int:
    """Bytes of one 32-token key group in the general layout (other k, plain 1-bit code)."""
    n1 = D - n2
    return n2 * 8 + n1 * 4 + n2 * 4 + n1 * 2 * (2 if plain else 1)


def chunk_perm_general(slab: np.ndarray, lay: dict, chunk: int, n2: int):
    e = slab[lay["chunk_table_offset"] + chunk * CHUNK_BYTES:][:CHUNK_BYTES]
    return e[:n2].astype(np.int64), e[n2:].astype(np.int64)


def key_groups_general(slab: np.ndarray, lay: dict, g_begin: int, n_groups: int, n2: int, plain: bool):
    """General key layout -> codes2 [32n, n2], bits1 [32n, n1], s2, z2 [n, n2], s1 [n, n1], z1 [n, n1] or None.

    Blocks of 32 channels.  Two-bit region: byte (block, lane = 4 (t % 8) + (j % 32) // 8, tile t // 8,
    parity j % 2) at block * 256 + lane * 8 + tile * 2 + parity, field (j % 8) // 2.  One-bit region:
    byte (block, lane, tile) at block * 128 + lane * 4 + tile, column j % 8 at bit 7 - j % 8."""
    n1 = D - n2
    gb = general_key_group_bytes(n2, plain)
    t = np.arange(G)[:, None]
    j2 = np.arange(n2)[None, :]
    off2 = (j2 // 32) * 256 + ((t % 8) * 4 + (j2 % 32) // 8) * 8 + (t // 8) * 2 + j2 % 2
    sh2 = 2 * ((j2 % 8) // 2)
    j1 = np.arange(n1)[None, :]
    off1 = (j1 // 32) * 128 + ((t % 8) * 4 + (j1 % 32) // 8) * 4 + t // 8
    sh1 = 7 - j1 % 8
    o_b1 = n2 * 8
    o_s2 = o_b1 + n1 * 4
    o_z2 = o_s2 + n2 * 2
    o_s1 = o_z2 + n2 * 2
    o_z1 = o_s1 + n1 * 2
    codes2 = np.zeros((n_groups * G, n2), np.int8)
    bits1 = np.zeros((n_groups * G, n1), np.uint8)
    s2 = np.zeros((n_groups, n2), np.float16); z2 = np.zeros((n_groups, n2), np.float16)
    s1 = np.zeros((n_groups, n1), np.float16); z1 = np.zeros((n_groups, n1), np.float16) if plain else None
    for g in range(n_groups):
        rec = slab[lay["kgroup_offset"] + (g_begin + g) * gb:][:gb]
        codes2[g * G:(g + 1) * G] = (rec[off2].astype(np.int64) >> sh2) & 3
        if n1:
            bits1[g * G:(g + 1) * G] = (rec[o_b1:][off1].astype(np.int64) >> sh1) & 1
        s2[g] = rec[o_s2:o_z2].view("<f2")
        z2[g] = rec[o_z2:o_s1].view("<f2")
        s1[g] = rec[o_s1:o_z1].view("<f2")
        if plain:
            z1[g] = rec[o_z1:o_z1 + n1 * 2].view("<f2")
    return codes2, bits1, s2, z2, s1, z1
