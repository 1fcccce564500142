#!/usr/bin/env python
"""Benchmark of the VidKV hot path on B200: KV quantization + packed-cache decode attention.

One "step" is one pass of the whole hot path over one batch of synthetic input:
token selection (when p > 0), MixQuant of the keys and 1.58Quant / STPQuant of the values
of every layer, then the workload's decode steps (append, attention over the packed cache,
residual flush), every layer of a decode step in one library call.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload batched] [--p 0.0]
    python bench.py --impl reference      # the CPU oracle on a bounded sample, same metric

Prints one JSON line (rank 0).  `value` is the packed-KV decode-attention throughput in
GB/s of algorithmic bytes (packed codes + metadata + FP16 residual + q/out per decode step),
summed over ranks; the quantizer's tokens/s rides along in `quantize`.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NOMINAL_HBM_GBS = 8000.0          # the 8 TB/s the targets are quoted against
FALLBACK_HBM_GBS = 6650.0         # earlier measurement on this machine, used if MEASURED_PEAKS.json is absent
# DRAM bytes per cached token per KV head moved by one launch of the decode attention kernel, from the
# ncu captures summarised in profiles/decode_stream_kernel_batched_4layers.txt (p = 0) and
# profiles/decode_stream_stp_kernel_batched_4layers_p02.txt (p > 0): a 4-layer cut of the batched workload
# (3 211 264 cached token-heads per launch), scaled to the launch by the token-heads it processes
# (traffic is proportional to them).
NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD = {"decode_stream_kernel": 71.75, "decode_stream_stp_kernel": 79.28}


KERNEL_TIMING_STRIDE = 4
KG_BYTES = 1152      # bytes of one 32-token key group; follows --k-ratio / --key-1bit (set in main)
KEY_FORMAT = {"k_ratio": 0.5, "one_bit": "fft"}


def key_group_bytes(k_ratio, one_bit):
    """2 bits per anomalous channel and 1 per normal one for 32 tokens, a binary16 (s, z) pair per 2-bit channel,
    a binary16 scale per spectrum column or an (s, z) pair per plain 1-bit channel."""
    n2 = int(round(k_ratio * 128))
    n1 = 128 - n2
    return (2 * n2 + n1) * 4 + 4 * n2 + (4 if one_bit == "minmax" else 2) * n1


def algorithmic_decode_bytes(B, L, H_kv, H_q, T_q0, n_flush, n_res, n_prot, elem=2):
    """Bytes one decode step must read/write per the packed layout (all layers)."""
    kgroups = T_q0 // 32 + 4 * n_flush
    n_rest = T_q0 - n_prot
    tgroups = (n_rest + 31) // 32 + 4 * n_flush
    pgroups = (n_prot + 31) // 32
    per_slab = kgroups * KG_BYTES + tgroups * (5376 / 5) + pgroups * 1536 + n_res * 128 * elem * 2 \
        + (1 + n_flush) * 128
    io = H_q * 128 * (elem + 4) + 2 * H_kv * 128 * elem
    return L * B * (H_kv * per_slab + io)


def algorithmic_quantize_bytes(B, L, H_kv, T, n_prot, elem=2):
    T_q = T - T % 32
    read = 2 * T * 128 * elem
    write = (T_q // 32) * KG_BYTES + ((T_q - n_prot + 31) // 32) * (5376 / 5) + ((n_prot + 31) // 32) * 1536
    return L * B * H_kv * (read + write)


def max_over_ranks(values, device, world):
    """Element-wise maximum over the ranks of a list of floats (one all-reduce on `device`,
    with whatever process group is initialised); the list itself at world == 1.  Every rank
    processes the same amount of work, so job throughput = world * units / this maximum."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    tt = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return tt.tolist()


def whole_job_throughput(units_per_rank, ms, world):
    """Units per second of the whole job: every rank did `units_per_rank` in at most `ms`."""
    return world * units_per_rank / (ms * 1e-3)


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(wl, p, device_tensors=None, max_batch=8, n_steps=8):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload (about ten seconds of
    host time on the batched shape): layer 0, up to 8 batch elements, all KV heads, full T, K+V
    quantize once and 8 decode steps."""
    import numpy as np
    from oracle import vidkv_oracle as O
    from workloads import make_layer_kv, make_saliency, make_step_inputs
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    T = min(wl.T, 12544)
    nb = min(wl.batch, max_batch)
    if device_tensors is not None:
        K, V = device_tensors
        K, V = K[:nb, :, :T].float().cpu(), V[:nb, :, :T].float().cpu()
    else:
        K, V = make_layer_kv(wl, 0, "cpu", T=T, B=nb)
    l_v = min(wl.l_v, T - T % 32)
    E = None
    n_prot = 0
    if p > 0:
        sal = make_saliency(wl, "cpu", l_v=l_v, B=nb)
        E = [O.select_tokens(sal[b].numpy(), p, 0, T) for b in range(nb)]
        n_prot = int(E[0].sum())
    H = K.shape[1]
    t0 = time.perf_counter()
    slabs = []
    for b in range(nb):
        for h in range(H):
            sc = O.SlabCache(ratio=KEY_FORMAT["k_ratio"], one_bit=KEY_FORMAT["one_bit"])
            sc.prefill(K[b, h].float().numpy(), V[b, h].float().numpy(), E[b] if E is not None else None)
            slabs.append(sc)
    t_quant = time.perf_counter() - t0
    rep = 7   # query heads per KV head in every workload
    t0 = time.perf_counter()
    for s in range(n_steps):
        q, k, v = make_step_inputs(wl, 0, s, "cpu", T=T, B=nb)
        for b in range(nb):
            for h in range(H):
                slabs[b * H + h].decode_step(q[b, rep * h:rep * h + rep].float().numpy(), k[b, h].float().numpy(),
                                             v[b, h].float().numpy())
    t_dec = (time.perf_counter() - t0) / n_steps
    dec_bytes = algorithmic_decode_bytes(nb, 1, H, rep * H, T - T % 32, 0, T % 32 + 1, n_prot)
    return {
        "decode_gbs": dec_bytes / t_dec / 1e9,
        "quantize_tokens_per_s": nb * T / t_quant,
        "seconds": t_quant + t_dec * n_steps,
        "cores": threads,
        "sample": f"layer 0, batch elements 0..{nb - 1}, {H} KV heads, T={T}: K+V quantize once, {n_steps} decode steps "
                  f"(first step includes the oracle's one-time dequantization)",
    }


def run_reference(args, wl):
    """--impl reference: the oracle on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, ms = [], []
    res = None
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        res = oracle_sample(wl, args.p)
        if i >= args.warmup:
            vals.append(res["decode_gbs"]); ms.append((time.perf_counter() - t0) * 1e3)
    value = sum(vals) / len(vals)
    line = {
        "impl": "reference", "metric": "packed_kv_decode_attention_GBps", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sum(ms) / len(ms),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args.p),
        "quantize": {"tokens_per_s": res["quantize_tokens_per_s"], "unit": "tokens/s"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": res["cores"], "kind": "oracle", "sample": res["sample"]},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(wl, p):
    return {"workload": wl.name, "layers": wl.layers, "batch_per_gpu": wl.batch, "tokens": wl.T, "kv_heads": 4,
            "query_heads": 28, "head_dim": 128, "decode_steps": wl.steps, "dtype": wl.dtype, "p": p,
            "k_ratio": KEY_FORMAT["k_ratio"], "key_1bit": KEY_FORMAT["one_bit"],
            "cache": "inputs larger than L2 (no flush needed)" if wl.name in ("batched", "stress")
            else "packed cache fits L2: rotated over copies larger than L2"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="batched")
    ap.add_argument("--p", type=float, default=0.0, help="fraction of visual tokens protected at 2 bits")
    ap.add_argument("--k-ratio", type=float, default=0.5, choices=[0.25, 0.5, 0.75, 1.0],
                    help="fraction of key channels at 2 bits (Algorithm 3's k)")
    ap.add_argument("--key-1bit", default=None, choices=["fft", "minmax"],
                    help="1-bit code of the normal key channels; default: the paper's choice for the k (Sec. 4.1)")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (profiling captures)")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the decode steps per bench step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-token-scores", action="store_true", help="skip the stand-alone timing of vidkv_saliency_scores")
    ap.add_argument("--no-variants", action="store_true", help="skip the warm / cold and per-layer-launch figures of "
                    "the workloads whose packed cache fits L2")
    args = ap.parse_args()
    global KG_BYTES
    one_bit = args.key_1bit or ("fft" if args.k_ratio in (0.5, 0.75) else "minmax")
    if one_bit == "fft" and args.k_ratio == 0.25:
        ap.error("the FFT 1-bit code is built for k = 0.5 and 0.75 (Sec. 4.1); use --key-1bit minmax")
    KEY_FORMAT.update(k_ratio=args.k_ratio, one_bit=one_bit)
    KG_BYTES = key_group_bytes(args.k_ratio, one_bit)

    from dataclasses import replace
    from workloads import CONFIGS
    wl = CONFIGS[args.workload]
    if args.layers is not None:
        wl = replace(wl, layers=args.layers)
    if args.decode_steps is not None:
        wl = replace(wl, steps=args.decode_steps)

    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import paper_2503_16257_b200 as P
    from workloads import make_layer_kv, make_saliency, make_step_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    L, B, T, H, HQ = wl.layers, wl.batch, wl.T, 4, 28
    steps_dec = wl.steps
    in_dt = P.VIDKV_F16 if wl.dtype == "fp16" else P.VIDKV_BF16
    cfg = P.VidKVConfig(B=B, L=L, max_prefill_tokens=T, max_new_tokens=steps_dec, p_ratio=args.p,
                        in_dtype=in_dt, out_dtype=P.VIDKV_F32, k_ratio=args.k_ratio,
                        key_1bit_mode=P.VIDKV_KEY1BIT_PLAIN_MINMAX if KEY_FORMAT["one_bit"] == "minmax" else P.VIDKV_KEY1BIT_FFT_SIGN)
    # Small workloads: rotate over enough independent caches that one decode step never finds its
    # cache in L2 (126 MB); large ones exceed L2 by themselves.
    one_cache = algorithmic_decode_bytes(B, L, H, HQ, T - T % 32, 0, 1, 0)
    n_caches = 1 if one_cache > 400e6 else int(min(8, -(-400e6 // one_cache)))
    caches = [P.VidKVCache(cfg, device=dev) for _ in range(n_caches)]

    # ---- inputs resident in HBM before the timed region
    Ks, Vs = [], []
    for layer in range(L):
        K, V = make_layer_kv(wl, layer, dev)
        Ks.append(K); Vs.append(V)
    qs, ks, vs = [], [], []
    for s in range(steps_dec):
        ql, kl, vl = zip(*[make_step_inputs(wl, layer, s, dev) for layer in range(L)])
        qs.append(torch.stack(ql)); ks.append(torch.stack(kl)); vs.append(torch.stack(vl))
    sal = make_saliency(wl, dev) if args.p > 0 else None
    out = torch.empty((L, B, HQ, 128), dtype=torch.float32, device=dev)
    n_prot = int(args.p * wl.l_v) if args.p > 0 else 0
    stream = torch.cuda.current_stream()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    k_b, k_e = ev(), ev()
    k_b.record(); k_e.record()
    torch.cuda.synchronize()

    # workloads whose layers are small hand all layers to the quantizer in one call (fewer launches);
    # the large ones go layer by layer, as a model produces them
    layers_in_one_call = one_cache < 400e6
    Kall = torch.stack(Ks) if layers_in_one_call else None
    Vall = torch.stack(Vs) if layers_in_one_call else None

    side_stream = torch.cuda.Stream()

    def quantize(cache):
        cache.reset()
        if sal is not None:
            cache.select_tokens(sal, 0, wl.l_v, T)
        # keys and values of a layer go to disjoint parts of the cache: the value quantizer runs on a second
        # stream beside the key quantizer (the token selection before both, the decode steps after both)
        main = torch.cuda.current_stream()
        side_stream.wait_stream(main)
        if layers_in_one_call:
            cache.quantize_keys_layers(0, Kall)
            with torch.cuda.stream(side_stream):
                cache.quantize_values_layers(0, Vall)
        else:
            for layer in range(L):
                cache.quantize_keys(layer, Ks[layer])
                with torch.cuda.stream(side_stream):
                    cache.quantize_values(layer, Vs[layer])
        main.wait_stream(side_stream)

    def one_step(timers=None):
        """Whole hot path once.  Returns the algorithmic decode bytes of the step."""
        if timers is not None:
            e0, e1, e2 = ev(), ev(), ev()
            e0.record()
        for c in caches:
            quantize(c)
        if timers is not None:
            e1.record()
        dec_bytes = 0.0
        kern = []
        for s in range(steps_dec):
            c = caches[s % n_caches]
            st = c.layer_state(0)
            if timers is not None:
                # the dominant kernel is timed on every fourth decode step; events around it make that step's
                # launches ordinary ones, the other steps run as a user's would (dependent launches)
                if s % KERNEL_TIMING_STRIDE == 0:
                    a, b_ = ev(), ev()
                    a.record(); b_.record()            # materialise the CUDA events
                    c.set_profile_events(a, b_)
                    kern.append((a, b_))
                else:
                    c.set_profile_events(None, None)
            c.decode_attention(0, L, qs[s], ks[s], vs[s], out)
            dec_bytes += algorithmic_decode_bytes(B, L, H, HQ, T - T % 32, (st["n_quantized"] - (T - T % 32)) // 128,
                                                  st["n_residual"] + 1, n_prot)
        if timers is not None:
            e2.record()
            timers.append((e0, e1, e2, kern))
        return dec_bytes

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches0 = P.vidkv_launch_count()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    timers = []
    t_b, t_e = ev(), ev()
    torch.cuda.synchronize()
    t_b.record()
    dec_bytes = 0.0
    for _ in range(args.steps):
        dec_bytes = one_step(timers)
    t_e.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if sampler else None
    launches = P.vidkv_launch_count() - launches0
    for c in caches:
        c.set_profile_events(None, None)

    total_ms = t_b.elapsed_time(t_e)
    q_ms = sum(t[0].elapsed_time(t[1]) for t in timers) / len(timers)
    d_ms = sum(t[1].elapsed_time(t[2]) for t in timers) / len(timers)
    kern_ms = [a.elapsed_time(b_) for t in timers for (a, b_) in t[3]]
    kern_avg_ms = sum(kern_ms) / len(kern_ms)
    total_ms, q_ms, d_ms, kern_avg_ms = max_over_ranks([total_ms, q_ms, d_ms, kern_avg_ms], dev, world)
    ms_per_step = total_ms / args.steps

    peak, peak_kind = read_peaks()
    decode_gbs = whole_job_throughput(dec_bytes, d_ms, world) / 1e9
    q_bytes = n_caches * algorithmic_quantize_bytes(B, L, H, T, n_prot)
    q_tokens = n_caches * B * T * L
    kern_bytes = dec_bytes / steps_dec
    kern_gbs = kern_bytes / (kern_avg_ms * 1e-3) / 1e9
    kernel_name = "decode_stream_stp_kernel" if n_prot > 0 else "decode_stream_kernel"
    general_fmt = not (KEY_FORMAT["k_ratio"] == 0.5 and KEY_FORMAT["one_bit"] == "fft")
    if general_fmt:
        kernel_name += "<general key format>"          # the same kernel, instantiated for the general key layout
    traffic = NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD.get(kernel_name)   # counters exist for the default format only
    if traffic is not None:
        traffic = traffic * B * L * H * (T - T % 32)

    line = {
        "metric": "packed_kv_decode_attention_GBps", "value": decode_gbs, "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, args.p),
        "pct_of_8TBps": 100.0 * decode_gbs / world / NOMINAL_HBM_GBS,
        "pct_of_measured_hbm": 100.0 * decode_gbs / world / peak,
        "decode": {"ms_per_bench_step": d_ms, "decode_steps": steps_dec, "bytes_per_decode_step": kern_bytes,
                   "caches_rotated": n_caches},
        "quantize": {"tokens_per_s": world * q_tokens / (q_ms * 1e-3), "unit": "tokens/s (one position, 4 KV heads, "
                     "one layer, K and V)", "calls": ("one call for all layers" if layers_in_one_call else "one call per layer") + "; values on a second stream beside the keys",
                     "ms_per_bench_step": q_ms, "GBps": world * q_bytes / (q_ms * 1e-3) / 1e9,
                     "pct_of_8TBps": 100.0 * q_bytes / (q_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
        "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": kern_gbs, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": kern_gbs / peak, "traffic": traffic,
                     "avg_launch_ms": kern_avg_ms, "launches_timed": len(kern_ms),
                     "timed": "every %dth launch of the timed region" % KERNEL_TIMING_STRIDE},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    # what the packed cache saves: FP16 K and V of the prompt against the bytes the layout holds for it
    fp16_bytes = 2 * 2 * 128 * H * B * L * T
    packed_bytes = B * L * H * ((T // 32) * KG_BYTES + ((T - T % 32 - n_prot + 31) // 32) * (5376 / 5) + ((n_prot + 31) // 32) * 1536
                                + (T % 32) * 512)
    line["memory"] = {"fp16_kv_bytes": fp16_bytes, "packed_kv_bytes": packed_bytes,
                      "bytes_saved_vs_fp16": fp16_bytes - packed_bytes, "saved_frac": 1.0 - packed_bytes / fp16_bytes}
    if rank == 0 and world == 1 and one_cache < 400e6 and not args.no_variants:
        line["l2_sized_variants"] = run_variants(P, torch, wl, cfg, caches, qs, ks, vs, out, n_prot, quantize)

    if rank == 0 and not args.no_e2e:
        line["e2e"] = run_e2e(P, torch, wl, cfg, caches[0], Ks, Vs, qs, ks, vs, sal, out, n_prot, dev, world)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        res = oracle_sample(wl, args.p, device_tensors=(Ks[0], Vs[0]))
        line["cpu_baseline"] = {"value": res["decode_gbs"], "unit": "GB/s", "cores": res["cores"], "kind": "oracle",
                                "sample": res["sample"], "quantize_tokens_per_s": res["quantize_tokens_per_s"],
                                "seconds": res["seconds"]}
        try:                                           # the same oracle on one thread, on a quarter of the sample
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                one = oracle_sample(wl, args.p, device_tensors=(Ks[0], Vs[0]), max_batch=2, n_steps=4)
            line["cpu_baseline"]["single_thread"] = {"value": one["decode_gbs"], "unit": "GB/s", "cores": 1,
                                                     "quantize_tokens_per_s": one["quantize_tokens_per_s"],
                                                     "seconds": one["seconds"], "sample": one["sample"]}
        except Exception as e:                         # threadpoolctl missing: say so instead of guessing
            line["cpu_baseline"]["single_thread"] = {"unavailable": repr(e)}
    if rank == 0 and not args.no_token_scores:
        line["token_scores"] = run_token_scores(P, torch, wl, dev, peak)
        line["channel_metrics"] = run_channel_metrics(P, torch, Ks, peak)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_variants(P, torch, wl, cfg, caches, qs, ks, vs, out, n_prot, quantize):
    """Workloads whose packed cache fits the 126 MB L2 (tiny, LLaVA-shaped, Qwen-shaped): decode GB/s of
    algorithmic bytes with the cache cold (rotating over copies larger than L2 in sum) and warm (the same
    cache every step), and with one library call per decode step for all layers or one call per layer."""
    L, B, T, H, HQ = wl.layers, wl.batch, wl.T, 4, 28
    n_steps = min(32, wl.steps)
    res = {}
    # per-layer views made once, outside the timed loops (slicing a tensor costs microseconds of host time)
    layer_args = [[(qs[i][l:l + 1], ks[i][l:l + 1], vs[i][l:l + 1], out[l:l + 1]) for l in range(L)] for i in range(n_steps)]
    for cold in (True, False):
        for per_layer in (False, True):
            use = caches if cold else caches[:1]
            for c in use:
                quantize(c)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            nbytes = 0.0
            e0.record()
            for s in range(n_steps * len(use)):
                c = use[s % len(use)]
                st = c.layer_state(0)
                i = s // len(use)
                if per_layer:
                    for layer in range(L):
                        c.decode_attention(layer, 1, *layer_args[i][layer])
                else:
                    c.decode_attention(0, L, qs[i], ks[i], vs[i], out)
                nbytes += algorithmic_decode_bytes(B, L, H, HQ, T - T % 32, 0, st["n_residual"] + 1, n_prot)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            res[("cold" if cold else "warm") + ("_per_layer_calls" if per_layer else "_one_call")] = {
                "GBps": nbytes / (ms * 1e-3) / 1e9, "us_per_decode_step": 1e3 * ms / (n_steps * len(use))}
    res["note"] = ("cold: every step reads a cache that is not in L2 (rotation over %d copies); warm: one cache, L2-resident; "
                   "per_layer_calls: %d library calls per decode step instead of one" % (len(caches), L))
    return res


def run_channel_metrics(P, torch, Ks, peak):
    """Upstream of the hot path: the Variance and Outliers channel metrics of one layer's keys, timed alone
    with CUDA events, alternating between two layers' tensors when there are two.  Bytes = K read once
    (variance) or twice (outliers: a mean pass and a counting pass).  The arithmetic is float64."""
    res = {}
    for metric, name, passes in ((P.VIDKV_METRIC_VARIANCE, "variance", 1), (P.VIDKV_METRIC_OUTLIERS, "outliers", 2)):
        for i in range(4):
            P.vidkv_channel_metrics(Ks[i % min(2, len(Ks))], metric)
        times = []
        for i in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            P.vidkv_channel_metrics(Ks[i % min(2, len(Ks))], metric)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = sum(times) / len(times)
        gbs = passes * Ks[0].numel() * 2 / (ms * 1e-3) / 1e9
        res[name] = {"GBps": gbs, "frac_of_measured_hbm": gbs / peak, "ms_per_call": ms}
    return res


def run_token_scores(P, torch, wl, dev, peak):
    """Upstream of the hot path (not part of a step): the Eq. 7 scores of the visual tokens from hidden
    states of the workload's shape, timed alone with CUDA events; two input copies alternate so that
    no call finds its input in L2.  Algorithmic bytes = the two inputs read once + the scores written."""
    from workloads import make_hidden_states
    l_t = wl.text_tokens if wl.text_tokens > 0 else 64    # a 64-token text query where the workload has none
    x_v, x_t = make_hidden_states(wl, dev, l_t=l_t)
    xs = [x_v, x_v.clone()] if x_v.numel() * 2 < 400e6 else [x_v]
    B, l_v, d = x_v.shape
    text_sum = torch.empty((B, d), dtype=torch.float32, device=dev)
    sal = torch.empty((B, l_v), dtype=torch.float32, device=dev)
    for i in range(8):
        P.vidkv_saliency_scores(xs[i % len(xs)], x_t, text_sum, sal)
    times = []
    for i in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        P.vidkv_saliency_scores(xs[i % len(xs)], x_t, text_sum, sal)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = sum(times) / len(times)
    nbytes = x_v.numel() * 2 + x_t.numel() * 2 + sal.numel() * 4
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"GBps": gbs, "frac_of_measured_hbm": gbs / peak, "pct_of_8TBps": 100.0 * gbs / NOMINAL_HBM_GBS, "ms_per_call": ms,
            "bytes_per_call": nbytes, "shape": {"B": B, "l_v": l_v, "l_t": int(x_t.shape[1]), "d_model": d},
            "launches_per_call": 2, "ms_each": [round(t, 4) for t in times]}


def run_e2e(P, torch, wl, cfg, cache, Ks, Vs, qs, ks, vs, sal, out, n_prot, dev, world):
    """The same step through the public API with HOST buffers: every step copies K, V (and
    the saliency) from pinned host memory before quantizing, every decode step copies q, k_new,
    v_new in and the attention output back out.  One warm-up step, two timed steps."""
    L, B, T, H, HQ = wl.layers, wl.batch, wl.T, 4, 28
    steps_dec = wl.steps
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, device="cpu", pin_memory=True).copy_(t)
    hK, hV = [pin(k) for k in Ks], [pin(v) for v in Vs]
    hq, hk, hv = [pin(t) for t in qs], [pin(t) for t in ks], [pin(t) for t in vs]
    hsal = pin(sal) if sal is not None else None
    hout = torch.empty(out.shape, dtype=out.dtype, device="cpu", pin_memory=True)
    dK, dV = torch.empty_like(Ks[0]), torch.empty_like(Vs[0])
    dq, dk, dv = torch.empty_like(qs[0]), torch.empty_like(ks[0]), torch.empty_like(vs[0])
    dsal = torch.empty_like(sal) if sal is not None else None
    h2d = sum(t.numel() * t.element_size() for t in hK + hV + hq + hk + hv) + (hsal.numel() * 4 if hsal is not None else 0)
    d2h = steps_dec * hout.numel() * hout.element_size()

    def step():
        cache.reset()
        if hsal is not None:
            dsal.copy_(hsal, non_blocking=True)
            cache.select_tokens(dsal, 0, wl.l_v, T)
        for layer in range(L):
            dK.copy_(hK[layer], non_blocking=True)
            cache.quantize_keys(layer, dK)
            dV.copy_(hV[layer], non_blocking=True)
            cache.quantize_values(layer, dV)
        e_mid = torch.cuda.Event(enable_timing=True)
        e_mid.record()
        dec_bytes = 0.0
        for s in range(steps_dec):
            st = cache.layer_state(0)
            dq.copy_(hq[s], non_blocking=True); dk.copy_(hk[s], non_blocking=True); dv.copy_(hv[s], non_blocking=True)
            cache.decode_attention(0, L, dq, dk, dv, out)
            hout.copy_(out, non_blocking=True)
            torch.cuda.current_stream().synchronize()          # the caller reads the result every step
            dec_bytes += algorithmic_decode_bytes(B, L, H, HQ, T - T % 32, (st["n_quantized"] - (T - T % 32)) // 128,
                                                  st["n_residual"] + 1, n_prot)
        return e_mid, dec_bytes

    step()
    torch.cuda.synchronize()
    n = 2
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    dms, tot = 0.0, 0.0
    for _ in range(n):
        t0.record()
        e_mid, dec_bytes = step()
        t1.record()
        torch.cuda.synchronize()
        dms += e_mid.elapsed_time(t1); tot += t0.elapsed_time(t1)
    return {"value": world * dec_bytes / (dms / n * 1e-3) / 1e9, "unit": "GB/s",
            "scope": "decode part of the step: per decode step H2D of q, k_new, v_new, the attention call, D2H of the output "
                     "and a stream synchronisation; the H2D of the prompt's K and V sits in the quantize part",
            "whole_step_value": world * dec_bytes / (tot / n * 1e-3) / 1e9,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": tot / n,
            "decode_ms_per_step": dms / n, "steps": n,
            "quantize_tokens_per_s": world * B * T * L / ((tot - dms) / n * 1e-3)}


if __name__ == "__main__":
    main()
