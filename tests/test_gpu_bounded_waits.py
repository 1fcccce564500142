"""The two device-side waits of the library are bounded: when what they wait for never comes they
give up, record VIDKV_ERR_TIMEOUT in the cache's status word and leave in order, and the device
stays usable.  The test hook withholds the awaited event with nothing outstanding (no products
issued, no copy in flight), so nothing here faults, traps or waits without a limit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _fresh_run_is_fine():
    from tests.helpers import Pair, TOL_ABS
    from workloads import CONFIGS
    pair = Pair(CONFIGS["tiny"], 352, B=1, L=1, p=0.0, max_new=2).prefill()
    out, ref = pair.decode()
    assert np.abs(out - ref).max() <= TOL_ABS
    assert pair.cache.status() == 0


def test_key_encoder_wait_runs_out_and_reports_timeout():
    import paper_2503_16257_b200 as P
    from workloads import CONFIGS, make_layer_kv
    wl = CONFIGS["tiny"]
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=640, max_new_tokens=1)
    cache = P.VidKVCache(cfg)
    K, _ = make_layer_kv(wl, 0, "cuda", T=640, B=1)
    P.vidkv_debug_withhold_once(1)
    cache.quantize_keys(0, K)
    assert cache.status() == -7                    # VIDKV_ERR_TIMEOUT, read after a stream synchronisation
    # the hook cleared itself: a fresh cache quantizes and decodes as usual
    _fresh_run_is_fine()


def test_stream_kernel_wait_runs_out_and_reports_timeout():
    import paper_2503_16257_b200 as P
    from workloads import CONFIGS, make_layer_kv, make_step_inputs
    wl = CONFIGS["tiny"]
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=640, max_new_tokens=2)
    cache = P.VidKVCache(cfg)
    K, V = make_layer_kv(wl, 0, "cuda", T=640, B=1)
    cache.quantize_keys(0, K)
    cache.quantize_values(0, V)
    assert cache.status() == 0
    q, k, v = make_step_inputs(wl, 0, 0, "cuda", T=640, B=1)
    out = torch.empty((1, 1, 28, 128), dtype=torch.float32, device="cuda")
    P.vidkv_debug_withhold_once(2)
    cache.decode_attention(0, 1, q[None], k[None], v[None], out)
    assert cache.status() == -7
    _fresh_run_is_fine()
