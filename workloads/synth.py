"""Seeded synthetic KV-cache workloads shaped like video-LLM prompts.

The five named configurations stand in for the key/value caches that
LLaVA-OV-7B / Qwen2.5-VL-7B would produce on long video prompts (196 visual
tokens per frame, 28 layers, 4 KV heads x head_dim 128, 28 query heads).  No
model weights or benchmark items are involved: every tensor is drawn from a
seeded ``torch.Generator``, one generator per (config, layer, tensor), with
seed ``seed * 1_000_003 + layer * 16 + tensor_id``.  The tensor is generated
once in float32, cast to the storage dtype, and those bits are what every
consumer sees.

Tokens are ordered visual first, then text.  Layout is ``[B, H, T, D]``.
"""
from __future__ import annotations

import functools
from dataclasses import dataclass

import torch

H_KV = 4
H_Q = 28
D = 128
TOKENS_PER_FRAME = 196

_T_K, _T_V, _T_CH, _T_MU, _T_SIG, _T_SAL, _T_STEP, _T_HV, _T_HT = 0, 1, 2, 3, 4, 5, 6, 7, 8
D_MODEL = 3584   # hidden size of the 7B video LLMs the workloads are shaped after


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    layers: int
    batch: int
    frames: int
    text_tokens: int
    dtype: str            # "fp16" | "bf16"
    k_dist: str           # "normal" | "student_t3" | "rope"
    v_dist: str           # "normal" | "student_t3" | "scaled_normal"
    n_outlier: int        # planted outlier key channels per (layer, head)
    outlier_sign: str     # "plus" (10x+5) | "pm" (10x +-5) | "scale" (10x)
    steps: int
    seed: int = 0

    @property
    def l_v(self) -> int:
        return self.frames * TOKENS_PER_FRAME

    @property
    def T(self) -> int:
        return self.l_v + self.text_tokens

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16


CONFIGS = {
    "tiny": WorkloadConfig("tiny", 1, 1, 8, 64, "fp16", "normal", "normal", 8, "plus", 16),
    "llava": WorkloadConfig("llava", 28, 1, 32, 128, "fp16", "student_t3", "student_t3", 6, "pm", 256),
    "qwen": WorkloadConfig("qwen", 28, 1, 64, 256, "bf16", "rope", "scaled_normal", 6, "scale", 256),
    "batched": WorkloadConfig("batched", 28, 16, 64, 0, "fp16", "normal", "normal", 6, "plus", 128),
    "stress": WorkloadConfig("stress", 28, 4, 1000, 0, "fp16", "normal", "normal", 6, "plus", 64),
}


def _gen(cfg: WorkloadConfig, layer: int, tensor_id: int, device, extra: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + layer * 16 + tensor_id + extra * 7919 * 16)
    return g


def _student_t3(shape, gen, device):
    z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    c = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(3):
        w = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        c += w * w
    return (z / torch.sqrt(c / 3.0)).clamp_(-6.0e4, 6.0e4)


def _outlier_channels(cfg: WorkloadConfig, layer: int):
    """[H_KV, n_outlier] planted channel ids and their +-1 signs (CPU, tiny)."""
    g = _gen(cfg, layer, _T_CH, "cpu")
    ids = torch.stack([torch.randperm(D, generator=g)[:cfg.n_outlier] for _ in range(H_KV)])
    sign = torch.randint(0, 2, (H_KV, cfg.n_outlier), generator=g) * 2 - 1
    return ids, sign


@functools.lru_cache(maxsize=256)
def _outlier_affine(cfg: WorkloadConfig, layer: int):
    """Per-head channel-wise (scale, offset) [H_KV, D] that plants the outlier channels."""
    ids, sign = _outlier_channels(cfg, layer)
    scale = torch.ones((H_KV, D), dtype=torch.float32)
    offset = torch.zeros((H_KV, D), dtype=torch.float32)
    for h in range(H_KV):
        for c, sg in zip(ids[h].tolist(), sign[h].tolist()):
            scale[h, c] = 10.0
            if cfg.outlier_sign == "plus":
                offset[h, c] = 5.0
            elif cfg.outlier_sign == "pm":
                offset[h, c] = 5.0 * sg
    return scale, offset


def _plant_outliers(cfg: WorkloadConfig, layer: int, x: torch.Tensor, head_of_dim1):
    """x [B, n_heads, T_or_1, D]: scale/shift the planted channels of each head."""
    scale, offset = _outlier_affine(cfg, layer)
    idx = torch.tensor(list(head_of_dim1), dtype=torch.long)
    sc = scale[idx].to(x.device).view(1, len(idx), 1, D)
    of = offset[idx].to(x.device).view(1, len(idx), 1, D)
    return x.mul_(sc).add_(of)


def _rope_params(cfg: WorkloadConfig, layer: int, device):
    g = _gen(cfg, layer, _T_MU, "cpu")
    mu = (torch.randn((H_KV, D), generator=g) * 2.0).to(device)
    theta = (1.0e6 ** (-torch.arange(D // 2, dtype=torch.float64) / (D // 2))).to(device)
    return mu, theta


def _key_like(cfg: WorkloadConfig, layer: int, gen, device, B: int, heads, t0: int, n_tok: int):
    """Draw [B, len(heads), n_tok, D] float32 from the key distribution of the
    KV heads listed in ``heads`` (token positions t0 .. t0+n_tok-1)."""
    shape = (B, len(heads), n_tok, D)
    if cfg.k_dist == "normal":
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    elif cfg.k_dist == "student_t3":
        x = _student_t3(shape, gen, device)
    else:  # rope-structured: per-channel mean + noise, pairs (i, i+64) rotated by t*theta_i
        mu, theta = _rope_params(cfg, layer, device)
        a = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        a += mu[list(heads)].view(1, len(heads), 1, D)
        pos = torch.arange(t0, t0 + n_tok, device=device, dtype=torch.float64)
        ang = pos.view(n_tok, 1) * theta.view(1, D // 2)
        cs, sn = torch.cos(ang).float(), torch.sin(ang).float()
        lo, hi = a[..., : D // 2], a[..., D // 2:]
        x = torch.cat([lo * cs - hi * sn, lo * sn + hi * cs], dim=-1)
    return _plant_outliers(cfg, layer, x, heads)


def _value_like(cfg: WorkloadConfig, layer: int, gen, device, B: int, heads, n_tok: int):
    shape = (B, len(heads), n_tok, D)
    if cfg.v_dist == "normal":
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if cfg.v_dist == "student_t3":
        return _student_t3(shape, gen, device)
    g = _gen(cfg, layer, _T_SIG, "cpu")
    sigma = (torch.rand((H_KV, D), generator=g) * 1.5 + 0.5).to(device)
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    return x * sigma[list(heads)].view(1, len(heads), 1, D)


def make_layer_kv(cfg: WorkloadConfig, layer: int, device="cpu", T: int | None = None,
                  B: int | None = None):
    """K, V of one layer: ``[B, H_KV, T, D]`` in the config's storage dtype."""
    T = cfg.T if T is None else T
    B = cfg.batch if B is None else B
    heads = list(range(H_KV))
    K = _key_like(cfg, layer, _gen(cfg, layer, _T_K, device), device, B, heads, 0, T)
    V = _value_like(cfg, layer, _gen(cfg, layer, _T_V, device), device, B, heads, T)
    return K.to(cfg.torch_dtype).contiguous(), V.to(cfg.torch_dtype).contiguous()


def make_step_inputs(cfg: WorkloadConfig, layer: int, step: int, device="cpu",
                     T: int | None = None, B: int | None = None):
    """Decode-step inputs of one layer: q ``[B, H_Q, D]``, k_new, v_new
    ``[B, H_KV, D]``, drawn from the per-channel distribution of the cache
    (query head h uses the key distribution of KV head h // 7)."""
    T = cfg.T if T is None else T
    B = cfg.batch if B is None else B
    gen = _gen(cfg, layer, _T_STEP, device, extra=step + 1)
    q_heads = [h // (H_Q // H_KV) for h in range(H_Q)]
    q = _key_like(cfg, layer, gen, device, B, q_heads, T + step, 1)[:, :, 0, :]
    k_new = _key_like(cfg, layer, gen, device, B, list(range(H_KV)), T + step, 1)[:, :, 0, :]
    v_new = _value_like(cfg, layer, gen, device, B, list(range(H_KV)), 1)[:, :, 0, :]
    dt = cfg.torch_dtype
    return q.to(dt).contiguous(), k_new.to(dt).contiguous(), v_new.to(dt).contiguous()


def make_saliency(cfg: WorkloadConfig, device="cpu", l_v: int | None = None,
                  B: int | None = None) -> torch.Tensor:
    """Per-visual-token saliency scores ``[B, l_v]`` float32 ~ N(0, 1)."""
    l_v = cfg.l_v if l_v is None else l_v
    B = cfg.batch if B is None else B
    return torch.randn((B, l_v), generator=_gen(cfg, 0, _T_SAL, device), device=device,
                       dtype=torch.float32)


def make_hidden_states(cfg: WorkloadConfig, device="cpu", l_v: int | None = None, l_t: int | None = None,
                       B: int | None = None, d_model: int = D_MODEL):
    """Hidden states of the visual tokens ``[B, l_v, d_model]`` and of the text tokens
    ``[B, l_t, d_model]`` in the config's storage dtype, ~ N(0, 1); the text tokens share a
    common direction (scale 0.5) so that their sum does not average out."""
    l_v = cfg.l_v if l_v is None else l_v
    l_t = cfg.text_tokens if l_t is None else l_t
    B = cfg.batch if B is None else B
    x_v = torch.randn((B, l_v, d_model), generator=_gen(cfg, 0, _T_HV, device), device=device, dtype=torch.float32)
    g = _gen(cfg, 0, _T_HT, device)
    common = torch.randn((B, 1, d_model), generator=g, device=device, dtype=torch.float32)
    x_t = torch.randn((B, l_t, d_model), generator=g, device=device, dtype=torch.float32) + 0.5 * common
    dt = cfg.torch_dtype
    return x_v.to(dt).contiguous(), x_t.to(dt).contiguous()
