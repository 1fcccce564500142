"""GPU parity at the launch shapes the benchmark times and at every way a decode call can be cut
into work: the named workloads at their full sizes (the oracle recomputes sampled slabs), and
small inputs on which every slab is checked while the test hook forces several run lengths of the
stream kernels (without and with protected tokens), including runs that end inside slabs, on slab
boundaries and span several slabs, and steps after a residual flush."""
import numpy as np
import pytest
import torch

from oracle import vidkv_oracle as O
from tests.helpers import Pair, TOL_ABS, to_np
from workloads import CONFIGS, make_layer_kv, make_saliency, make_step_inputs

pytestmark = pytest.mark.gpu


def _rel_tol(ref):
    """2e-3 absolute; where the outputs are large (heavy-tailed values) the bound scales with
    their magnitude."""
    return TOL_ABS * max(1.0, float(np.abs(ref).max()))


class SampledRun:
    """A workload at full size on the GPU; the oracle holds only the sampled (layer, b, h) slabs."""

    def __init__(self, name, L, B, T, p, max_new, samples):
        import paper_2503_16257_b200 as P
        self.P, self.wl, self.L, self.B, self.T, self.p = P, CONFIGS[name], L, B, T, p
        wl = self.wl
        in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
        self.cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=max_new, p_ratio=p,
                                 in_dtype=in_dt, out_dtype=P.VIDKV_F32)
        self.cache = P.VidKVCache(self.cfg, device="cuda")
        self.samples = samples
        self.slabs = {}
        self.step = 0
        Tq = T - T % 32
        E = {}
        if p > 0:
            l_v = min(wl.l_v, Tq)
            sal = make_saliency(wl, "cpu", l_v=l_v, B=B)
            self.cache.select_tokens(sal.cuda(), 0, l_v, T)
            for (_, b, _) in samples:
                if b not in E:
                    e = np.zeros(T, dtype=bool)
                    e[:Tq] = O.select_tokens(sal[b].numpy(), p, 0, Tq)
                    E[b] = e
        for layer in range(L):
            K, V = make_layer_kv(wl, layer, "cuda", T=T, B=B)
            self.cache.quantize_keys(layer, K)
            self.cache.quantize_values(layer, V)
            for (sl, b, h) in samples:
                if sl == layer:
                    sc = O.SlabCache()
                    sc.prefill(to_np(K[b, h]), to_np(V[b, h]), E.get(b))
                    self.slabs[(sl, b, h)] = sc
            del K, V

    def decode(self, check=True):
        wl, L, B = self.wl, self.L, self.B
        q, k, v = (torch.stack(t) for t in zip(*[make_step_inputs(wl, layer, self.step, "cuda", T=self.T, B=B)
                                                  for layer in range(L)]))
        out = torch.empty((L, B, self.cfg.H_q, 128), dtype=torch.float32, device="cuda")
        self.cache.decode_attention(0, L, q, k, v, out)
        out = out.cpu().numpy().astype(np.float64)
        rep = self.cfg.H_q // self.cfg.H_kv
        worst = 0.0
        for (sl, b, h), sc in self.slabs.items():
            ref = sc.decode_step(to_np(q[sl, b, rep * h:rep * (h + 1)]), to_np(k[sl, b, h]), to_np(v[sl, b, h]))
            if check:
                err = np.abs(out[sl, b, rep * h:rep * (h + 1)] - ref).max()
                assert err <= _rel_tol(ref), f"step {self.step} slab {(sl, b, h)}: max abs error {err}"
                worst = max(worst, err)
        self.step += 1
        return worst


def _plan(run: SampledRun, n_residual):
    st = run.cache.layer_state(0)
    n_prefill_q = run.T - run.T % 32
    n_flush = (st["n_quantized"] - n_prefill_q) // 128
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    return run.P.vidkv_debug_decode_plan(run.cfg, n_prefill_q, n_flush, n_residual, st["n_protected"], run.L, sm_count=sm)


# ------------------------------------------------------------------ the benchmark's own shape
@pytest.mark.parametrize("L,p,steps", [
    (8, 0.0, 2),       # runs of about 23 units: three to four runs per slab
    (28, 0.0, 2),      # the launch bench.py times: runs of 80 units, every run crosses a slab boundary
    (28, 0.2, 2),      # the launch bench.py --p 0.2 times: runs of 120 units (two thirds of the warps)
])
def test_batched_workload_at_the_timed_launch_shape(L, p, steps):
    wl = CONFIGS["batched"]
    samples = [(0, 0, 0), (L // 2, 7, 2), (L - 1, 15, 3), (L - 1, 3, 1)]
    run = SampledRun("batched", L, wl.batch, wl.T, p, steps, samples)
    plan = _plan(run, 1)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    assert plan["run_units"] == -(-(L * 64 * 79) // (sm * (12 if p == 0 else 8)))      # 80 / 120 at L = 28 on 148 SMs
    for _ in range(steps):
        run.decode()
    assert run.cache.status() == 0


@pytest.mark.parametrize("p", [0.0, 0.2])
def test_batched_shape_through_the_flush(p):
    """Two layers at batch 16 (128 slabs): 129 steps, so the 128-token residual is flushed and the step
    after it attends to the flushed chunk.  With p = 0.2 (2508 protected tokens per sequence) unit and
    run boundaries fall inside ternary supergroups and protected groups."""
    wl = CONFIGS["batched"]
    run = SampledRun("batched", 2, wl.batch, wl.T, p, 130, [(0, 0, 0), (1, 9, 2)])
    assert _plan(run, 1)["run_units"] > 2
    for s in range(129):
        run.decode(check=(s < 2 or s >= 126))
    assert run.cache.layer_state(1) == dict(n_quantized=wl.T + 128, n_residual=1, n_chunks=2,
                                            n_protected=int(np.float32(p) * wl.T) if p else 0)
    assert run.cache.status() == 0


# ------------------------------------------------------------------ the other named workloads
@pytest.mark.parametrize("name,p", [("llava", 0.0), ("llava", 0.2), ("qwen", 0.0), ("qwen", 0.2)])
def test_named_workload_one_layer_through_the_flush(name, p):
    """LLaVA-shaped (T = 6400, Student-t) and Qwen-shaped (T = 12 800, bfloat16, rotary keys) caches,
    one layer, every KV head against the oracle, through step 129 (the flush happens at step 128)."""
    wl = CONFIGS[name]
    run = SampledRun(name, 1, 1, wl.T, p, 130, [(0, 0, h) for h in range(4)])
    for s in range(129):
        run.decode(check=(s < 3 or s >= 126 or s % 16 == 0))
    assert run.cache.layer_state(0)["n_chunks"] == 2 and run.cache.status() == 0


@pytest.mark.parametrize("p", [0.0, 0.2])
def test_stress_length_slab(p):
    """196 000 tokens (1000 frames) on one sequence; the oracle recomputes one KV head."""
    wl = CONFIGS["stress"]
    run = SampledRun("stress", 1, 1, wl.T, p, 2, [(0, 0, 2)])
    for _ in range(2):
        run.decode()
    st = run.cache.layer_state(0)
    assert st["n_quantized"] == wl.T - wl.T % 32 and st["n_protected"] == (int(np.float32(0.2) * wl.l_v) if p else 0)
    assert run.cache.status() == 0


# ------------------------------------------------------------------ every plan on small inputs, all slabs checked
@pytest.mark.parametrize("run_units", [1, 2, 3, 5, 13, 40])
@pytest.mark.parametrize("name,T,B,L,p", [
    ("tiny", 2000, 2, 2, 0.2),       # 1984 quantized tokens = 12.4 units per slab, 16 residual tokens
    ("qwen", 1311, 1, 1, 0.5),       # bfloat16, half the visual tokens protected
    ("tiny", 1632, 1, 1, 0.9),       # long protected stream, short ternary one
])
def test_stream_kernel_with_protected_tokens_at_every_run_length(run_units, name, T, B, L, p):
    """Runs of 1 .. 40 units over caches with protected tokens: runs end inside ternary supergroups and
    protected groups, which both neighbours then multiply with their own probabilities."""
    pair = Pair(CONFIGS[name], T, B=B, L=L, p=p, max_new=4).prefill()
    pair.cache.debug_set_decode_plan(run_units=run_units)
    for _ in range(3):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= _rel_tol(ref)
    assert pair.cache.status() == 0


@pytest.mark.parametrize("run_units", [1, 3])
def test_stream_kernel_with_protected_tokens_across_a_flush(run_units):
    pair = Pair(CONFIGS["tiny"], 1000, B=1, L=1, p=0.2, max_new=125).prefill()    # 992 + 8; flush at step 120
    pair.cache.debug_set_decode_plan(run_units=run_units)
    for s in range(123):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= _rel_tol(ref), s
    assert pair.cache.layer_state(0)["n_chunks"] == 2 and pair.cache.status() == 0


@pytest.mark.parametrize("run_units", [1, 2, 3, 5, 13, 40])
def test_stream_kernel_at_every_run_length(run_units):
    """2000 tokens = 12.4 units per slab, 16 slabs: runs of 1 .. 40 units, so runs end inside slabs, on
    slab boundaries and span several slabs; every slab is checked."""
    pair = Pair(CONFIGS["tiny"], 2000, B=2, L=2, p=0.0, max_new=4).prefill()
    pair.cache.debug_set_decode_plan(run_units=run_units)
    for _ in range(3):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= TOL_ABS
    assert pair.cache.status() == 0


@pytest.mark.parametrize("run_units", [1, 4])
def test_stream_kernel_across_two_flushes(run_units):
    """Chunks with their own channel splits inside one unit: 96 prefill tokens, then two flushed
    128-token chunks (a unit of 160 tokens then holds groups of two or three chunks)."""
    pair = Pair(CONFIGS["qwen"], 101, B=2, L=1, p=0.0, max_new=260).prefill()
    pair.cache.debug_set_decode_plan(run_units=run_units)
    for s in range(255):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= _rel_tol(ref), s
    assert pair.cache.layer_state(0)["n_chunks"] == 3 and pair.cache.status() == 0


def _random_plans(n, seed):
    r = np.random.default_rng(seed)
    cases = []
    for _ in range(n):
        name = ["tiny", "llava", "qwen"][int(r.integers(0, 3))]
        T = int(r.integers(33, 2600))
        steps = int(r.integers(1, 4)) if r.random() < 0.75 else 128 - T % 32 + int(r.integers(1, 4))
        cases.append((name, T, int(r.integers(1, 3)), int(r.integers(1, 3)), [0.0, 0.05, 0.2, 0.5, 0.97][int(r.integers(0, 5))],
                      [1, 2, 3, 7, 19][int(r.integers(0, 5))], steps))
    return cases


@pytest.mark.parametrize("name,T,B,L,p,run_units,steps", _random_plans(14, 20250317))
def test_seeded_random_shapes_and_run_lengths(name, T, B, L, p, run_units, steps):
    """Shapes, protection ratios and run lengths nobody picked by hand (a quarter of the cases decode
    across a residual flush), every slab against the oracle."""
    pair = Pair(CONFIGS[name], T, B=B, L=L, p=p, max_new=steps + 1).prefill()
    pair.cache.debug_set_decode_plan(run_units=run_units)
    for s in range(steps):
        out, ref = pair.decode()
        assert np.abs(out - ref).max() <= _rel_tol(ref), s
    assert pair.cache.status() == 0


# ------------------------------------------------------------------ prompts shorter than one group
@pytest.mark.parametrize("T", [31, 0])
def test_flushes_after_a_prompt_with_nothing_to_quantize(T):
    """Fewer than 32 prompt tokens: chunk 0 of the chunk table stays empty and the flushed chunks
    follow it.  Decoded across two flushes through vidkv_decode_attention, and after each flush
    through vidkv_attend_noalloc as well."""
    import paper_2503_16257_b200 as P
    wl = CONFIGS["tiny"]
    steps = 2 * 128 - T + 3
    cfg = P.VidKVConfig(B=1, L=1, max_prefill_tokens=32, max_new_tokens=steps + 1, p_ratio=0.0, out_dtype=P.VIDKV_F32)
    cache = P.VidKVCache(cfg)
    K, V = make_layer_kv(wl, 0, "cpu", T=32, B=1)
    K, V = K[:, :, :T].contiguous(), V[:, :, :T].contiguous()
    cache.quantize_keys(0, K.cuda())
    cache.quantize_values(0, V.cuda())
    slabs = []
    for h in range(4):
        sc = O.SlabCache()
        sc.prefill(to_np(K[0, h]), to_np(V[0, h]), None)
        slabs.append(sc)
    flushes = 0
    for s in range(steps):
        q, k, v = make_step_inputs(wl, 0, s, "cpu", T=32, B=1)
        out = torch.empty((1, 1, 28, 128), dtype=torch.float32, device="cuda")
        cache.decode_attention(0, 1, q[None].cuda(), k[None].cuda(), v[None].cuda(), out)
        ref = np.concatenate([slabs[h].decode_step(to_np(q[0, 7 * h:7 * h + 7]), to_np(k[0, h]), to_np(v[0, h]))
                              for h in range(4)])
        assert np.abs(out[0, 0].cpu().numpy().astype(np.float64) - ref).max() <= TOL_ABS, s
        st = cache.layer_state(0)
        if st["n_quantized"] // 128 > flushes or s == steps - 1:
            flushes = st["n_quantized"] // 128
            # the same attention once more, without the append, through the workspace-free entry point
            again = torch.full((1, 1, 28, 128), float("nan"), dtype=torch.float32, device="cuda")
            P.vidkv_attend_noalloc(cfg, cache.cache, 0, flushes, st["n_residual"], 0, 0, 1, q[None].cuda(), again)
            if st["n_residual"] > 0:          # right after a flush the residual is empty and the attended set differs
                assert float((again - out).abs().max()) <= TOL_ABS
            else:
                # the flushed tokens are now read from their packed form: compare with the oracle's dequantized view
                Kd = [sl.dequant_k() for sl in slabs]
                Vd = [sl.dequant_v() for sl in slabs]
                r2 = np.concatenate([O.attention(to_np(q[0, 7 * h:7 * h + 7]), Kd[h], Vd[h], 1.0 / np.sqrt(128.0))
                                     for h in range(4)])
                assert np.abs(again[0, 0].cpu().numpy().astype(np.float64) - r2).max() <= TOL_ABS
    assert cache.layer_state(0) == dict(n_quantized=256, n_residual=T + steps - 256, n_chunks=2, n_protected=0)
    assert cache.status() == 0
