"""VidKV 1.x-bit KV-cache hot path for B200 (sm_100a): thin Python binding over libvidkv.so.

The binding only marshals arguments (device pointers, sizes, the current CUDA stream);
every step of the method runs in the CUDA kernels behind the C ABI of ``include/vidkv.h``.
There is no CPU or PyTorch fallback: importing works without a GPU (so that the library's
symbols can be checked), but every compute call needs the compiled library and a device.
"""
from .api import (  # noqa: F401
    VidKVConfig, VidKVCache, VidKVError, load_library, library_path, exported_symbols,
    vidkv_cache_bytes, vidkv_cache_layout, vidkv_version, vidkv_launch_count, vidkv_attend_noalloc, vidkv_saliency_scores, vidkv_channel_metrics,
    vidkv_debug_decode_plan, vidkv_debug_withhold_once, vidkv_merge_partials,
    STATUS_NAMES,
    VIDKV_F16, VIDKV_BF16, VIDKV_F32, VIDKV_TERNARY_SCALE_MEAN_ABS, VIDKV_TERNARY_SCALE_NONZERO_MEAN, VIDKV_METRIC_VARIANCE, VIDKV_METRIC_OUTLIERS, VIDKV_KEY1BIT_FFT_SIGN, VIDKV_KEY1BIT_PLAIN_MINMAX,
)
