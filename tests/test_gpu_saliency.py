"""GPU parity of the Eq. 7 score entry point (vidkv_saliency_scores) against the CPU oracle,
through the C ABI, on seeded hidden states."""
import numpy as np
import pytest
import torch

import paper_2503_16257_b200 as P
from oracle import vidkv_oracle as O
from workloads import CONFIGS, D_MODEL, make_hidden_states

pytestmark = pytest.mark.gpu


def _tolerance(x_v, x_t):
    """Float32 accumulation against the float64 oracle: the text sums carry l_t roundings, the
    dot product d more, each relative 2^-24 of the running magnitude, which sum_c |x_v[c]| |t[c]|
    bounds.  (l_t + d) * 2^-24 of that bound, doubled."""
    t = np.abs(x_t.astype(np.float64)).sum(axis=0)
    bound = np.abs(x_v.astype(np.float64)) @ t
    return 2.0 * (x_t.shape[0] + x_v.shape[1]) * 2.0 ** -24 * bound + 1e-30


@pytest.mark.parametrize("name,B,l_v,l_t,d", [
    ("tiny", 2, 1000, 64, 256),       # several blocks of 64 rows and a ragged tail (1000 = 15 * 64 + 40)
    ("tiny", 1, 1, 1, 8),             # the smallest problem
    ("tiny", 1, 63, 3, 3584),         # the models' hidden size, odd row count inside one block
    ("qwen", 2, 321, 17, 3584),       # bfloat16 inputs
    ("llava", 1, 130, 0, 64),         # no text tokens: every score is zero
    ("tiny", 1, 70, 5, 16384),        # the widest supported hidden size (64 KB of shared memory)
])
def test_scores_match_the_oracle(name, B, l_v, l_t, d):
    wl = CONFIGS[name]
    x_v, x_t = make_hidden_states(wl, "cuda", l_v=l_v, l_t=l_t, B=B, d_model=d)
    got = P.vidkv_saliency_scores(x_v, x_t).cpu().numpy()
    assert got.shape == (B, l_v)
    for b in range(B):
        xv = x_v[b].float().cpu().numpy()
        xt = x_t[b].float().cpu().numpy()
        want = O.stp_saliency(xv, xt)
        tol = _tolerance(xv, xt) if l_t else np.zeros(l_v)
        assert np.all(np.abs(got[b] - want) <= tol), float(np.max(np.abs(got[b] - want) / (tol + 1e-30)))


def test_scores_drive_the_same_token_selection():
    """Scores from the device fed to vidkv_select_tokens protect the tokens the oracle picks from
    its own scores; a token may differ only if its score is within the tolerance of the n-th one."""
    wl = CONFIGS["tiny"]
    B, T = 2, wl.T
    l_v = min(wl.l_v, T - T % 32)
    x_v, x_t = make_hidden_states(wl, "cuda", l_v=l_v, B=B, d_model=512)
    sal = P.vidkv_saliency_scores(x_v, x_t)
    cfg = P.VidKVConfig(B=B, L=1, max_prefill_tokens=T, max_new_tokens=1, p_ratio=0.2, in_dtype=P.VIDKV_F16,
                        out_dtype=P.VIDKV_F32)
    cache = P.VidKVCache(cfg, device="cuda")
    cache.select_tokens(sal, 0, l_v, T)
    got_scores = sal.cpu().numpy()
    for b in range(B):
        xv, xt = x_v[b].float().cpu().numpy(), x_t[b].float().cpu().numpy()
        want_scores = O.stp_saliency(xv, xt)
        E_want = O.select_tokens(want_scores, 0.2, 0, T)
        E_got = O.select_tokens(got_scores[b].astype(np.float64), 0.2, 0, T)
        diff = np.nonzero(E_want != E_got)[0]
        if diff.size:
            n = int(E_want.sum())
            kth = np.sort(want_scores)[::-1][n - 1]
            tol = _tolerance(xv, xt)
            assert np.all(np.abs(want_scores[diff] - kth) <= 2 * tol[diff])
    assert cache.status() == 0


def test_argument_checks():
    x_v = torch.zeros((1, 4, 12), dtype=torch.float16, device="cuda")     # d not a multiple of 8
    x_t = torch.zeros((1, 2, 12), dtype=torch.float16, device="cuda")
    with pytest.raises(P.VidKVError):
        P.vidkv_saliency_scores(x_v, x_t)


def test_full_size_scores_on_sampled_rows():
    """The batched workload's shape as bench.py launches it (16 sequences, every visual token, hidden
    size 3584): sampled rows against the oracle, which handles a row at a time."""
    wl = CONFIGS["batched"]
    x_v, x_t = make_hidden_states(wl, "cuda", l_t=wl.text_tokens if wl.text_tokens > 0 else 64)
    assert x_v.shape == (wl.batch, wl.l_v, D_MODEL) and x_t.shape[1] > 0
    got = P.vidkv_saliency_scores(x_v, x_t).cpu().numpy()
    r = np.random.default_rng(5)
    for b in (0, wl.batch // 2, wl.batch - 1):
        rows = np.unique(np.concatenate([[0, 63, 64, wl.l_v - 1], r.integers(0, wl.l_v, 60)]))
        xv = x_v[b, torch.as_tensor(rows, device="cuda")].float().cpu().numpy()
        xt = x_t[b].float().cpu().numpy()
        want = O.stp_saliency(xv, xt)
        assert np.all(np.abs(got[b, rows] - want) <= _tolerance(xv, xt))
