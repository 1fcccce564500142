"""GPU parity of vidkv_channel_metrics (the Variance and Outliers metrics of Sec. 4.1(1)) against the
CPU oracle, through the C ABI, on the workloads' key tensors."""
import numpy as np
import pytest
import torch

import paper_2503_16257_b200 as P
from oracle import vidkv_oracle as O
from workloads import CONFIGS, make_layer_kv

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,T,B", [
    ("tiny", 1632, 1),       # 3.2 blocks of 512 tokens per slab, planted outlier channels
    ("tiny", 1, 2),          # a single token: variance 0, no outliers
    ("llava", 1000, 1),      # heavy-tailed keys: many outliers, ragged last block
    ("qwen", 777, 2),        # bfloat16 inputs, channels with large means (one-pass variance in float64)
])
def test_metrics_match_the_oracle(name, T, B):
    wl = CONFIGS[name]
    K, _ = make_layer_kv(wl, 0, "cuda", T=T, B=B)
    var = P.vidkv_channel_metrics(K, P.VIDKV_METRIC_VARIANCE).cpu().numpy()
    out = P.vidkv_channel_metrics(K, P.VIDKV_METRIC_OUTLIERS).cpu().numpy()
    Kc = K.float().cpu().numpy()
    for b in range(B):
        for h in range(K.shape[1]):
            want_var = O.channel_variance(Kc[b, h])
            # float64 sums on both sides; the one-pass formula loses (mean^2 / variance) * 2^-52, the float32 result 2^-24
            tol = 1e-6 * want_var + 1e-9 * (Kc[b, h].astype(np.float64) ** 2).mean(axis=0) + 1e-30
            assert np.all(np.abs(var[b, h] - want_var) <= tol)
            assert np.array_equal(out[b, h].astype(np.int64), O.channel_outliers(Kc[b, h]))


def test_metrics_on_a_strided_view_and_other_threshold():
    wl = CONFIGS["tiny"]
    K, _ = make_layer_kv(wl, 0, "cuda", T=640, B=2)
    big = torch.zeros((2, K.shape[1], 700, 128), dtype=K.dtype, device="cuda")
    big[:, :, 30:670] = K
    view = big[:, :, 30:670]                      # same values behind other strides and a base offset
    a = P.vidkv_channel_metrics(K, P.VIDKV_METRIC_OUTLIERS, M=2.0)
    b = P.vidkv_channel_metrics(view, P.VIDKV_METRIC_OUTLIERS, M=2.0)
    assert torch.equal(a, b)
    Kc = K.float().cpu().numpy()
    assert np.array_equal(a[1, 0].cpu().numpy().astype(np.int64), O.channel_outliers(Kc[1, 0], M=2.0))


def test_full_size_metrics_on_sampled_slabs():
    """One layer of the batched workload as a whole launch (64 slabs x 12544 tokens); three slabs against the oracle."""
    wl = CONFIGS["batched"]
    K, _ = make_layer_kv(wl, 0, "cuda")
    var = P.vidkv_channel_metrics(K, P.VIDKV_METRIC_VARIANCE).cpu().numpy()
    out = P.vidkv_channel_metrics(K, P.VIDKV_METRIC_OUTLIERS).cpu().numpy()
    for (b, h) in [(0, 0), (7, 2), (wl.batch - 1, 3)]:
        k = K[b, h].float().cpu().numpy()
        want = O.channel_variance(k)
        assert np.all(np.abs(var[b, h] - want) <= 1e-6 * want + 1e-9 * (k.astype(np.float64) ** 2).mean(axis=0))
        assert np.array_equal(out[b, h].astype(np.int64), O.channel_outliers(k))
