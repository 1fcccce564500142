"""The workspace-free attention entry point, for callers that cannot allocate device memory
(they get their tensors from a host framework and have no scratch buffer to offer).

It must give what the regular decode call gives.  The regular call appends the new token and
then attends; the workspace-free call attends over the cache as it then stands, so calling it
right after a regular step with the same query repeats that step's attention.  Checked on two
steps in a row, because the library's internal scratch array is shared by all calls and keeps
the previous call's contents.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_attend_noalloc_matches_decode_attention_twice():
    import paper_2503_16257_b200 as P
    from tests.helpers import TOL_ABS
    from workloads import CONFIGS, make_layer_kv, make_saliency, make_step_inputs

    wl = CONFIGS["tiny"]
    T, B, L = 1000, 2, 2                       # 992 quantized tokens + 8 residual, several splits
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=4, p_ratio=0.2)
    cache = P.VidKVCache(cfg)
    sal = make_saliency(wl, "cuda", l_v=960, B=B)
    cache.select_tokens(sal, 0, 960, T)
    for layer in range(L):
        K, V = make_layer_kv(wl, layer, "cuda", T=T, B=B)
        cache.quantize_keys(layer, K)
        cache.quantize_values(layer, V)
    for step in range(2):
        q, k, v = (torch.stack(t) for t in zip(*[make_step_inputs(wl, layer, step, "cuda", T=T, B=B)
                                                  for layer in range(L)]))
        ref = torch.empty((L, B, 28, 128), dtype=torch.float32, device="cuda")
        cache.decode_attention(0, L, q, k, v, ref)
        st = cache.layer_state(0)
        out = torch.full_like(ref, float("nan"))
        P.vidkv_attend_noalloc(cfg, cache.cache, 992, 0, st["n_residual"], st["n_protected"], 0, L, q, out)
        torch.cuda.synchronize()
        assert st["n_residual"] == 8 + step + 1 and st["n_protected"] == 192
        assert torch.isfinite(out).all()
        assert float((out - ref).abs().max()) <= TOL_ABS
        # one layer at a time gives the same rows
        one = torch.empty((1, B, 28, 128), dtype=torch.float32, device="cuda")
        P.vidkv_attend_noalloc(cfg, cache.cache, 992, 0, st["n_residual"], st["n_protected"], 1, 1, q[1:2], one)
        assert float((one[0] - ref[1]).abs().max()) <= TOL_ABS


def test_attend_noalloc_rejects_what_does_not_fit():
    import paper_2503_16257_b200 as P
    cfg = P.VidKVConfig(B=16, L=28, max_prefill_tokens=12544, max_new_tokens=1)
    cache = torch.zeros(256, dtype=torch.uint8, device="cuda")
    q = torch.zeros((28, 16, 28, 128), dtype=torch.float16, device="cuda")
    out = torch.zeros((28, 16, 28, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(P.VidKVError) as e:          # 28 * 16 * 28 heads * 20 splits records: too many
        P.vidkv_attend_noalloc(cfg, cache, 12544, 0, 1, 0, 0, 28, q, out)
    assert e.value.status == -4
    with pytest.raises(P.VidKVError) as e:          # token count beyond what the cache was sized for
        P.vidkv_attend_noalloc(cfg, cache, 12544 + 32, 0, 1, 0, 0, 1, q, out)
    assert e.value.status == -4
    with pytest.raises(P.VidKVError) as e:
        P.vidkv_attend_noalloc(cfg, cache, 100, 0, 1, 0, 0, 1, q, out)     # not a multiple of G
    assert e.value.status == -1


@pytest.mark.parametrize("p", [0.0, 0.2])
def test_attend_noalloc_matches_the_oracle(p):
    """The workspace-free call against the oracle itself (not only against the regular call): after a
    regular step the cache holds that step's token, so the same query through the workspace-free call
    must reproduce the oracle's output of that step.  Without and with protected tokens."""
    import paper_2503_16257_b200 as P
    from tests.helpers import Pair, TOL_ABS
    from workloads import CONFIGS, make_step_inputs

    wl = CONFIGS["tiny"]
    T, B, L = 1000, 2, 2
    pair = Pair(wl, T, B=B, L=L, p=p, max_new=3).prefill()
    for step in range(2):
        _, ref = pair.decode()
        q = torch.stack([make_step_inputs(wl, layer, step, "cpu", T=T, B=B)[0] for layer in range(L)]).cuda()
        st = pair.cache.layer_state(0)
        out = torch.full((L, B, 28, 128), float("nan"), dtype=torch.float32, device="cuda")
        P.vidkv_attend_noalloc(pair.cfg, pair.cache.cache, 992, 0, st["n_residual"], st["n_protected"], 0, L, q, out)
        torch.cuda.synchronize()
        assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= TOL_ABS
