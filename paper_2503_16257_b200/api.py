"""ctypes binding of libvidkv.so: same names and argument order as include/vidkv.h."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

VIDKV_F16, VIDKV_BF16, VIDKV_F32 = 0, 1, 2
VIDKV_TERNARY_SCALE_MEAN_ABS, VIDKV_TERNARY_SCALE_NONZERO_MEAN = 0, 1
VIDKV_KEY1BIT_FFT_SIGN, VIDKV_KEY1BIT_PLAIN_MINMAX = 0, 1
VIDKV_METRIC_VARIANCE, VIDKV_METRIC_OUTLIERS = 1, 2
STATUS_NAMES = {0: "OK", -1: "INVALID_ARG", -2: "UNSUPPORTED", -3: "ALIGNMENT", -4: "CAPACITY",
                -5: "STATE", -6: "CUDA", -7: "TIMEOUT"}

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class VidKVError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {STATUS_NAMES.get(status, status)} ({status})")


class _Config(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("H_kv", C.c_int32), ("H_q", C.c_int32),
                ("D", C.c_int32), ("G", C.c_int32), ("R", C.c_int32),
                ("k_ratio", C.c_float), ("p_ratio", C.c_float), ("gamma", C.c_float),
                ("in_dtype", C.c_int32), ("out_dtype", C.c_int32), ("key_1bit_mode", C.c_int32),
                ("ternary_scale", C.c_int32),
                ("max_prefill_tokens", C.c_int64), ("max_new_tokens", C.c_int64)]


class _Layout(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "header_bytes", "sel_offset", "sel_stride_b", "sel_words", "slab_offset", "slab_stride",
        "chunk_table_offset", "max_chunks", "kgroup_offset", "max_kgroups", "tern_offset",
        "max_supergroups", "prot_offset", "max_pgroups", "kres_offset", "vres_offset", "total_bytes")]


@dataclass
class VidKVConfig:
    B: int
    L: int
    max_prefill_tokens: int
    max_new_tokens: int
    H_kv: int = 4
    H_q: int = 28
    D: int = 128
    G: int = 32
    R: int = 128
    k_ratio: float = 0.5
    p_ratio: float = 0.0
    gamma: float = 0.7
    in_dtype: int = VIDKV_F16
    out_dtype: int = VIDKV_F32
    key_1bit_mode: int = 0
    ternary_scale: int = 0          # VIDKV_TERNARY_SCALE_MEAN_ABS | VIDKV_TERNARY_SCALE_NONZERO_MEAN

    def to_c(self) -> _Config:
        return _Config(self.B, self.L, self.H_kv, self.H_q, self.D, self.G, self.R, self.k_ratio,
                       self.p_ratio, self.gamma, self.in_dtype, self.out_dtype, self.key_1bit_mode, self.ternary_scale,
                       self.max_prefill_tokens, self.max_new_tokens)


_SIGNATURES = {
    "vidkv_version": (C.c_int32, []),
    "vidkv_launch_count": (C.c_uint64, []),
    "vidkv_attend_noalloc": (C.c_int32, [C.POINTER(_Config), C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int64,
                                         C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "vidkv_set_profile_events": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "vidkv_cache_bytes": (C.c_int32, [C.POINTER(_Config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "vidkv_cache_layout": (C.c_int32, [C.POINTER(_Config), C.POINTER(_Layout)]),
    "vidkv_cache_init": (C.c_int32, [C.POINTER(_Config), C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t,
                                     C.c_void_p, C.POINTER(C.c_void_p)]),
    "vidkv_cache_destroy": (C.c_int32, [C.c_void_p]),
    "vidkv_cache_reset": (C.c_int32, [C.c_void_p, C.c_void_p]),
    "vidkv_channel_metrics": (C.c_int32, [C.c_int32, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                          C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]),
    "vidkv_saliency_scores": (C.c_int32, [C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                          C.c_void_p, C.c_void_p, C.c_void_p]),
    "vidkv_select_tokens": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p]),
    "vidkv_set_token_mask": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p]),
    "vidkv_quantize_keys": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_int64, C.c_void_p]),
    "vidkv_quantize_values": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                          C.c_int64, C.c_void_p]),
    "vidkv_quantize_keys_layers": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                               C.c_int64, C.c_void_p]),
    "vidkv_quantize_values_layers": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                                 C.c_int64, C.c_void_p]),
    "vidkv_decode_attention": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_float, C.c_void_p]),
    "vidkv_decode_attention_partial": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                                   C.c_void_p, C.c_float, C.c_void_p]),
    "vidkv_merge_partials": (C.c_int32, [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int32, C.c_void_p]),
    "vidkv_layer_state": (C.c_int32, [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                      C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "vidkv_cache_status": (C.c_int32, [C.c_void_p, C.c_void_p]),
    "vidkv_debug_withhold_once": (C.c_int32, [C.c_int32]),
    "vidkv_debug_set_decode_plan": (C.c_int32, [C.c_void_p, C.c_int32]),
    "vidkv_debug_decode_plan": (C.c_int32, [C.POINTER(_Config), C.c_int64, C.c_int64, C.c_int32, C.c_int64, C.c_int32,
                                            C.c_int32, C.c_int32, C.POINTER(C.c_int64)]),
    "vidkv_export_codes": (C.c_int32, [C.c_void_p, C.c_int32] + [C.c_void_p] * 10 + [C.c_void_p]),
    "vidkv_get_selection": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "vidkv_dequantize_keys": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "vidkv_dequantize_values": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
}


def exported_symbols():
    """Names the binding expects libvidkv.so to export (all of include/vidkv.h)."""
    return sorted(_SIGNATURES)


def library_path() -> str:
    return os.path.join(_HERE, "libvidkv.so")


def load_library():
    """Load libvidkv.so (built in-tree by ``python -m paper_2503_16257_b200.build``).
    Fails loudly when the library is missing: there is no fallback path."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} not found: build it with `python -m paper_2503_16257_b200.build`")
        lib = C.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _LIB = lib
    return _LIB


def _check(fn: str, status: int):
    if status != 0:
        raise VidKVError(fn, status)


def vidkv_version() -> int:
    return load_library().vidkv_version()


def vidkv_launch_count() -> int:
    return load_library().vidkv_launch_count()


def vidkv_attend_noalloc(cfg: VidKVConfig, cache, n_prefill_quantized: int, n_flushed_chunks: int, n_residual: int,
                         n_protected: int, layer_begin: int, n_layers: int, q, out, softmax_scale: float = 0.0):
    """Attention of q over the packed cache tensor `cache` as it stands, for callers that cannot
    provide workspace memory: the scratch for partial results is a fixed array inside the library.  Same
    arguments as the C function; raises VidKVError (CAPACITY when the problem needs more than the
    array holds)."""
    c = cfg.to_c()
    _check("vidkv_attend_noalloc", load_library().vidkv_attend_noalloc(
        C.byref(c), C.c_void_p(cache.data_ptr()), n_prefill_quantized, n_flushed_chunks, n_residual, n_protected,
        layer_begin, n_layers, C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()), softmax_scale, _stream_ptr()))


def vidkv_channel_metrics(K, metric: int, M: float = 3.0):
    """Variance or outlier count of every key channel: K [B, H, T, 128] (float16 / bfloat16 device
    tensor, channel stride 1) -> float32 [B, H, 128]."""
    import torch
    B, H, T, D = K.shape
    assert D == 128 and K.stride(3) == 1
    dtype = VIDKV_F16 if K.dtype == torch.float16 else VIDKV_BF16
    scratch = torch.empty((B, H, 2, D), dtype=torch.float64, device=K.device)
    out = torch.empty((B, H, D), dtype=torch.float32, device=K.device)
    _check("vidkv_channel_metrics", load_library().vidkv_channel_metrics(
        dtype, C.c_void_p(K.data_ptr()), B, H, T, K.stride(0), K.stride(1), K.stride(2), metric, M,
        C.c_void_p(scratch.data_ptr()), C.c_void_p(out.data_ptr()), _stream_ptr()))
    return out


def vidkv_saliency_scores(x_v, x_t, text_sum=None, saliency=None):
    """Eq. 7 scores of the visual tokens: x_v [B, l_v, d], x_t [B, l_t, d] (float16 or bfloat16 device
    tensors) -> saliency [B, l_v] float32.  `text_sum` [B, d] float32 is scratch; both are
    allocated here when not given."""
    import torch
    B, l_v, d = x_v.shape
    l_t = x_t.shape[1]
    dtype = VIDKV_F16 if x_v.dtype == torch.float16 else VIDKV_BF16
    if text_sum is None:
        text_sum = torch.empty((B, d), dtype=torch.float32, device=x_v.device)
    if saliency is None:
        saliency = torch.empty((B, l_v), dtype=torch.float32, device=x_v.device)
    _check("vidkv_saliency_scores", load_library().vidkv_saliency_scores(
        dtype, C.c_void_p(x_v.data_ptr()), C.c_void_p(x_t.data_ptr()), B, l_v, l_t, d,
        C.c_void_p(text_sum.data_ptr()), C.c_void_p(saliency.data_ptr()), _stream_ptr()))
    return saliency


def vidkv_merge_partials(partials, out):
    """partials [n_parts, ..., 130] float32 (device) -> out [..., 128]: log-sum-exp merge of per-shard triples."""
    import torch
    assert partials.is_contiguous() and out.is_contiguous() and partials.dtype == torch.float32
    n_parts = partials.shape[0]
    n_rows = partials.numel() // (n_parts * 130)
    dt = {torch.float32: VIDKV_F32, torch.float16: VIDKV_F16, torch.bfloat16: VIDKV_BF16}[out.dtype]
    _check("vidkv_merge_partials", load_library().vidkv_merge_partials(
        C.c_void_p(partials.data_ptr()), n_parts, n_rows, C.c_void_p(out.data_ptr()), dt, _stream_ptr()))
    return out


def vidkv_debug_withhold_once(what: int):
    """Test hook: 1 = the next key quantization, 2 = the next decode call without protected tokens
    lets its bounded device-side wait run out (see include/vidkv.h)."""
    _check("vidkv_debug_withhold_once", load_library().vidkv_debug_withhold_once(what))


_PLAN_FIELDS = ("units_per_slab", "run_units", "n_runs", "parts_stride", "records", "records_capacity", "n_chunks",
                "n_units")


def vidkv_debug_decode_plan(cfg: VidKVConfig, n_prefill_quantized: int, n_flushed_chunks: int, n_residual: int,
                            n_protected: int, n_layers: int, sm_count: int = 148, run_units: int = 0) -> dict:
    """How a decode call with these token counts would be cut into work (host only, no device)."""
    out = (C.c_int64 * len(_PLAN_FIELDS))()
    c = cfg.to_c()
    _check("vidkv_debug_decode_plan", load_library().vidkv_debug_decode_plan(
        C.byref(c), n_prefill_quantized, n_flushed_chunks, n_residual, n_protected, n_layers, sm_count, run_units, out))
    return dict(zip(_PLAN_FIELDS, [int(v) for v in out]))


def vidkv_cache_bytes(cfg: VidKVConfig):
    cb, wb = C.c_size_t(0), C.c_size_t(0)
    c = cfg.to_c()
    _check("vidkv_cache_bytes", load_library().vidkv_cache_bytes(C.byref(c), C.byref(cb), C.byref(wb)))
    return cb.value, wb.value


def vidkv_cache_layout(cfg: VidKVConfig) -> dict:
    lay = _Layout()
    c = cfg.to_c()
    _check("vidkv_cache_layout", load_library().vidkv_cache_layout(C.byref(c), C.byref(lay)))
    return {n: getattr(lay, n) for n, _ in _Layout._fields_}


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _strides_bht(x):
    assert x.dim() == 4 and x.stride(3) == 1, "expected [B, H, T, D] with unit channel stride"
    return x.stride(0), x.stride(1), x.stride(2)


class VidKVCache:
    """Owns the two device buffers (torch uint8 tensors) and the library handle.  Methods carry
    the C ABI's names; tensors are passed as device pointers, work goes to the current stream."""

    def __init__(self, cfg: VidKVConfig, device="cuda"):
        import torch
        self.cfg = cfg
        self.lib = load_library()
        self.cache_bytes, self.workspace_bytes = vidkv_cache_bytes(cfg)
        self.layout = vidkv_cache_layout(cfg)
        self.cache = torch.empty(self.cache_bytes, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=device)
        self._c = cfg.to_c()
        h = C.c_void_p()
        _check("vidkv_cache_init", self.lib.vidkv_cache_init(
            C.byref(self._c), C.c_void_p(self.cache.data_ptr()), self.cache_bytes,
            C.c_void_p(self.workspace.data_ptr()), self.workspace.numel(), _stream_ptr(), C.byref(h)))
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self.lib.vidkv_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check("vidkv_cache_reset", self.lib.vidkv_cache_reset(self.handle, _stream_ptr()))

    def select_tokens(self, saliency, vis_begin: int, l_v: int, T: int):
        ptr = C.c_void_p(saliency.data_ptr()) if saliency is not None else C.c_void_p(0)
        if saliency is not None:
            assert saliency.is_contiguous() and saliency.dtype.is_floating_point and saliency.element_size() == 4
        _check("vidkv_select_tokens", self.lib.vidkv_select_tokens(self.handle, ptr, vis_begin, l_v, T, _stream_ptr()))

    def set_token_mask(self, E, T: int, n_protected: int = -1):
        """n_protected >= 0: asynchronous, a disagreeing row shows in status(); -1: counted by the
        library (one stream synchronisation)."""
        assert E.is_contiguous() and E.element_size() == 1
        _check("vidkv_set_token_mask", self.lib.vidkv_set_token_mask(self.handle, C.c_void_p(E.data_ptr()), T,
                                                                     n_protected, _stream_ptr()))

    def quantize_keys(self, layer: int, K):
        sb, sh, st = _strides_bht(K)
        _check("vidkv_quantize_keys", self.lib.vidkv_quantize_keys(
            self.handle, layer, C.c_void_p(K.data_ptr()), K.shape[2], sb, sh, st, _stream_ptr()))

    def quantize_values(self, layer: int, V):
        sb, sh, st = _strides_bht(V)
        _check("vidkv_quantize_values", self.lib.vidkv_quantize_values(
            self.handle, layer, C.c_void_p(V.data_ptr()), V.shape[2], sb, sh, st, _stream_ptr()))

    def _layers_args(self, X):
        assert X.dim() == 5 and X.stride(4) == 1, "expected [n_layers, B, H, T, D] with unit channel stride"
        assert X.stride(0) == X.shape[1] * X.stride(1), "layers must be stride_b * B elements apart"
        return X.shape[0], X.shape[3], X.stride(1), X.stride(2), X.stride(3)

    def quantize_keys_layers(self, layer_begin: int, K):
        n, T, sb, sh, st = self._layers_args(K)
        _check("vidkv_quantize_keys_layers", self.lib.vidkv_quantize_keys_layers(
            self.handle, layer_begin, n, C.c_void_p(K.data_ptr()), T, sb, sh, st, _stream_ptr()))

    def quantize_values_layers(self, layer_begin: int, V):
        n, T, sb, sh, st = self._layers_args(V)
        _check("vidkv_quantize_values_layers", self.lib.vidkv_quantize_values_layers(
            self.handle, layer_begin, n, C.c_void_p(V.data_ptr()), T, sb, sh, st, _stream_ptr()))

    def decode_attention(self, layer_begin: int, n_layers: int, q, k_new, v_new, out, softmax_scale: float = 0.0):
        for t in (q, k_new, v_new, out):
            assert t.is_contiguous()
        _check("vidkv_decode_attention", self.lib.vidkv_decode_attention(
            self.handle, layer_begin, n_layers, C.c_void_p(q.data_ptr()), C.c_void_p(k_new.data_ptr()),
            C.c_void_p(v_new.data_ptr()), C.c_void_p(out.data_ptr()), softmax_scale, _stream_ptr()))

    def decode_attention_partial(self, layer_begin: int, n_layers: int, q, k_new, v_new, partial, softmax_scale: float = 0.0):
        """One token shard's (maximum, sum, unnormalised out) triples; k_new = v_new = None: attend as it stands."""
        kp = C.c_void_p(k_new.data_ptr()) if k_new is not None else C.c_void_p(0)
        vp = C.c_void_p(v_new.data_ptr()) if v_new is not None else C.c_void_p(0)
        _check("vidkv_decode_attention_partial", self.lib.vidkv_decode_attention_partial(
            self.handle, layer_begin, n_layers, C.c_void_p(q.data_ptr()), kp, vp, C.c_void_p(partial.data_ptr()),
            softmax_scale, _stream_ptr()))

    def layer_state(self, layer: int) -> dict:
        a, b, c, d = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        _check("vidkv_layer_state", self.lib.vidkv_layer_state(self.handle, layer, C.byref(a), C.byref(b),
                                                              C.byref(c), C.byref(d)))
        return dict(n_quantized=a.value, n_residual=b.value, n_chunks=c.value, n_protected=d.value)

    def set_profile_events(self, ev_begin=None, ev_end=None):
        """torch.cuda.Event pair (created with enable_timing=True and recorded once) or None."""
        a = C.c_void_p(ev_begin.cuda_event) if ev_begin is not None else C.c_void_p(0)
        b = C.c_void_p(ev_end.cuda_event) if ev_end is not None else C.c_void_p(0)
        _check("vidkv_set_profile_events", self.lib.vidkv_set_profile_events(self.handle, a, b))

    def debug_set_decode_plan(self, run_units: int = 0):
        """Test hook: force the run length (160-token units per warp) of later decode calls; 0 = choose."""
        _check("vidkv_debug_set_decode_plan", self.lib.vidkv_debug_set_decode_plan(self.handle, run_units))

    def status(self) -> int:
        return self.lib.vidkv_cache_status(self.handle, _stream_ptr())

    def export_codes(self, layer: int, T: int) -> dict:
        """Plain arrays of every code and scale of one layer (torch tensors; see vidkv_export_codes);
        T is the prompt length given at prefill."""
        import torch
        st = self.layer_state(layer)
        B, H = self.cfg.B, self.cfg.H_kv
        ng = st["n_quantized"] // 32
        n_prefill_q = T - T % 32
        n_flush = (st["n_quantized"] - n_prefill_q) // 128
        nt = (n_prefill_q - st["n_protected"] + 31) // 32 + 4 * n_flush
        npg = (st["n_protected"] + 31) // 32
        dev = self.cache.device
        n2 = int(round(self.cfg.k_ratio * 128))
        n1 = 128 - n2
        plain = n1 > 0 and self.cfg.key_1bit_mode == VIDKV_KEY1BIT_PLAIN_MINMAX
        out = dict(
            k2=torch.zeros((B, H, 32 * ng, n2), dtype=torch.int8, device=dev),
            k1bits=torch.zeros((B, H, 32 * ng, n1), dtype=torch.uint8, device=dev),
            k_s2=torch.zeros((B, H, ng, n2), dtype=torch.float16, device=dev),
            k_z2=torch.zeros((B, H, ng, n2), dtype=torch.float16, device=dev),
            # plain min/max mode: per group the n1 scales, then the n1 zero points
            k_s1=torch.zeros((B, H, ng, 2, n1) if plain else (B, H, ng, n1), dtype=torch.float16, device=dev),
            v_trits=torch.zeros((B, H, 32 * nt, 128), dtype=torch.int8, device=dev),
            v_s=torch.zeros((B, H, nt, 128), dtype=torch.float16, device=dev),
            v2=torch.zeros((B, H, 32 * npg, 128), dtype=torch.int8, device=dev),
            v2_s=torch.zeros((B, H, npg, 128), dtype=torch.float16, device=dev),
            v2_z=torch.zeros((B, H, npg, 128), dtype=torch.float16, device=dev))
        ptr = [C.c_void_p(out[k].data_ptr() if out[k].numel() else 0)
               for k in ("k2", "k1bits", "k_s2", "k_z2", "k_s1", "v_trits", "v_s", "v2", "v2_s", "v2_z")]
        _check("vidkv_export_codes", self.lib.vidkv_export_codes(self.handle, layer, *ptr, _stream_ptr()))
        return out

    def get_selection(self, layer: int, T: int):
        """(dmask [B, H_kv, chunks, 128], E [B, T]) as uint8 tensors; see vidkv_get_selection."""
        import torch
        st = self.layer_state(layer)
        n_flush = (st["n_quantized"] - (T - T % 32)) // 128
        dev = self.cache.device
        dmask = torch.zeros((self.cfg.B, self.cfg.H_kv, 1 + n_flush, 128), dtype=torch.uint8, device=dev)
        E = torch.zeros((self.cfg.B, max(T, 1)), dtype=torch.uint8, device=dev)
        _check("vidkv_get_selection", self.lib.vidkv_get_selection(
            self.handle, layer, C.c_void_p(dmask.data_ptr()), C.c_void_p(E.data_ptr() if T else 0), _stream_ptr()))
        return dmask, E[:, :T]

    def dequantize_keys(self, layer: int):
        import torch
        st = self.layer_state(layer)
        out = torch.empty((self.cfg.B, self.cfg.H_kv, st["n_quantized"], self.cfg.D), dtype=torch.float32,
                          device=self.cache.device)
        _check("vidkv_dequantize_keys", self.lib.vidkv_dequantize_keys(self.handle, layer, C.c_void_p(out.data_ptr()),
                                                                       _stream_ptr()))
        return out

    def dequantize_values(self, layer: int):
        import torch
        st = self.layer_state(layer)
        out = torch.empty((self.cfg.B, self.cfg.H_kv, st["n_quantized"], self.cfg.D), dtype=torch.float32,
                          device=self.cache.device)
        _check("vidkv_dequantize_values", self.lib.vidkv_dequantize_values(self.handle, layer,
                                                                           C.c_void_p(out.data_ptr()), _stream_ptr()))
        return out
