"""Sequence-sharded decode (caches beyond one device, Sec. 1): the token axis is cut into shards,
each held by its own cache; vidkv_decode_attention_partial leaves a shard's (max, sum, out) triples,
vidkv_merge_partials combines them.  One GPU stands in for the devices here: the shards are two
caches on it and the exchange is a concatenation; the result is compared with the oracle's attention
over the shards' dequantized tokens (each shard quantized on its own) plus the residual."""
import numpy as np
import pytest
import torch

from oracle import vidkv_oracle as O
from tests.helpers import TOL_ABS, to_np
from workloads import CONFIGS, make_layer_kv, make_saliency, make_step_inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,T,cut,p,steps", [
    ("tiny", 2000, 1024, 0.0, 3),      # shard A: 1024 tokens; shard B: 960 quantized + 16 residual + the new tokens
    ("tiny", 2000, 992, 0.2, 3),       # protected tokens in both shards (each shard selects among its own visual tokens)
    ("qwen", 1200, 640, 0.0, 130),     # bfloat16; shard B flushes its residual on the way
])
def test_two_token_shards_merge_to_the_oracle(name, T, cut, p, steps):
    import paper_2503_16257_b200 as P
    wl = CONFIGS[name]
    B, L = 2, 2
    in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
    spans = [(0, cut), (cut, T)]
    caches, slabs = [], [{}, {}]
    KV = [make_layer_kv(wl, layer, "cpu", T=T, B=B) for layer in range(L)]
    for si, (lo, hi) in enumerate(spans):
        n = hi - lo
        cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=n, max_new_tokens=steps + 1, p_ratio=p, in_dtype=in_dt,
                            out_dtype=P.VIDKV_F32)
        c = P.VidKVCache(cfg)
        E = [None] * B
        if p > 0:
            l_v = n - n % 32
            sal = make_saliency(wl, "cpu", l_v=l_v, B=B) + si          # different scores per shard
            c.select_tokens(sal.cuda(), 0, l_v, n)
            for b in range(B):
                E[b] = np.zeros(n, dtype=bool)
                E[b][:l_v] = O.select_tokens(sal[b].numpy(), p, 0, l_v)
        for layer in range(L):
            K, V = KV[layer][0][:, :, lo:hi].contiguous(), KV[layer][1][:, :, lo:hi].contiguous()
            c.quantize_keys(layer, K.cuda())
            c.quantize_values(layer, V.cuda())
            for b in range(B):
                for h in range(4):
                    sc = O.SlabCache()
                    sc.prefill(to_np(K[b, h]), to_np(V[b, h]), E[b])
                    slabs[si][(layer, b, h)] = sc
        caches.append(c)
    scale = 1.0 / np.sqrt(128.0)
    for step in range(steps):
        q, k, v = (torch.stack(t) for t in zip(*[make_step_inputs(wl, layer, step, "cpu", T=T, B=B) for layer in range(L)]))
        parts = torch.full((2, L, B, 28, 130), float("nan"), dtype=torch.float32, device="cuda")
        caches[0].decode_attention_partial(0, L, q.cuda(), None, None, parts[0])
        caches[1].decode_attention_partial(0, L, q.cuda(), k.cuda(), v.cuda(), parts[1])
        out = torch.empty((L, B, 28, 128), dtype=torch.float32, device="cuda")
        P.vidkv_merge_partials(parts, out)
        out = out.cpu().numpy().astype(np.float64)
        check = step < 3 or step >= steps - 3
        for layer in range(L):
            for b in range(B):
                for h in range(4):
                    a, bb = slabs[0][(layer, b, h)], slabs[1][(layer, b, h)]
                    qs = to_np(q[layer, b, 7 * h:7 * h + 7])
                    # shard B's step on the oracle side (append, attend, flush) keeps its state in step
                    bb.decode_step(qs, to_np(k[layer, b, h]), to_np(v[layer, b, h]))
                    if not check:
                        continue
                    Kb = np.concatenate([bb.dequant_k(), bb.k_res.astype(np.float64)])
                    Vb = np.concatenate([bb.dequant_v(), bb.v_res.astype(np.float64)])
                    if bb.k_res.shape[0] == 0:
                        continue      # the step that flushed: the library attended before the flush, the oracle state is after it
                    ref = O.merge_partials([O.attention_partial(qs, a.dequant_k(), a.dequant_v(), scale),
                                            O.attention_partial(qs, Kb, Vb, scale)])
                    err = np.abs(out[layer, b, 7 * h:7 * h + 7] - ref).max()
                    assert err <= TOL_ABS * max(1.0, np.abs(ref).max()), (step, layer, b, h, err)
    assert caches[0].status() == 0 and caches[1].status() == 0
    # shard A was only attended to: its token counts did not move
    assert caches[0].layer_state(0)["n_residual"] == cut % 32
