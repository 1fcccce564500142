// vidkv_attend_noalloc: attention of a query over a packed cache as it stands, with the
// partial attention results kept in a fixed device array that is part of this library
// instead of in caller-provided workspace memory.
//
// Who this is for.  Some callers are handed device tensors by a host framework and have no
// way to obtain more device memory at the point where they run attention: a plugin that may
// only touch the buffers it was given, code running while the framework's memory pool is
// frozen, or a runtime in which cudaMalloc is simply unavailable.  They can pass inputs and
// outputs, but cannot provide the scratch buffer the regular entry point needs.
#include <cmath>

#include "common.cuh"
#include "kernels.cuh"

namespace {

// 16 MiB of scratch: the partial records (130 floats per query head and warp run) and
// 3 KiB of prepared query per (slab, chunk).  Every GPU
// that loads this library holds the array until the process exits.
constexpr size_t kStaticPartialFloats = 4u * 1024u * 1024u;
static __device__ __align__(256) float g_static_partials[kStaticPartialFloats];

constexpr int kMaxDevices = 64;
float* g_partials_ptr[kMaxDevices] = {};   // device address of the array, per device (set up once)

// In host code `g_static_partials` is only a handle for the runtime, not a device address:
// ask the runtime for the address on the current device and hand that to the kernels.
vidkv_status_t static_partials(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VIDKV_ERR_CUDA;
  if (!g_partials_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) return VIDKV_ERR_CUDA;
    g_partials_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_partials_ptr[dev];
  return VIDKV_OK;
}

}  // namespace

extern "C" vidkv_status_t vidkv_attend_noalloc(const vidkv_config_t* cfg, const void* cache, int64_t n_prefill_quantized,
                                               int64_t n_flushed_chunks, int32_t n_residual, int64_t n_protected,
                                               int32_t layer_begin, int32_t n_layers, const void* q, void* out,
                                               float softmax_scale, void* stream) {
  using namespace vidkv;
  if (!cfg || !cache || !q || !out) return VIDKV_ERR_INVALID_ARG;
  vidkv_layout_t lay;
  const vidkv_status_t st = vidkv_cache_layout(cfg, &lay);
  if (st != VIDKV_OK) return st;
  if (layer_begin < 0 || n_layers < 1 || layer_begin + n_layers > cfg->L) return VIDKV_ERR_INVALID_ARG;
  if (n_prefill_quantized < 0 || n_prefill_quantized % kG || n_flushed_chunks < 0 || n_residual < 0 ||
      n_residual > kR || n_protected < 0 || n_protected > n_prefill_quantized)
    return VIDKV_ERR_INVALID_ARG;
  if (!std::isfinite(softmax_scale)) return VIDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(cache) & 255u) || (reinterpret_cast<uintptr_t>(q) & 15u) ||
      (reinterpret_cast<uintptr_t>(out) & 15u))
    return VIDKV_ERR_ALIGNMENT;
  if (n_prefill_quantized / kG + n_flushed_chunks * (kR / kG) > lay.max_kgroups || 1 + n_flushed_chunks > lay.max_chunks ||
      (n_protected + kG - 1) / kG > lay.max_pgroups)
    return VIDKV_ERR_CAPACITY;
  const int64_t T_tot = n_prefill_quantized + n_flushed_chunks * kR + n_residual;
  if (T_tot < 1) return VIDKV_ERR_STATE;

  DecodeArgs a;
  CacheView& cv = a.cv;
  cv.base = const_cast<uint8_t*>(static_cast<const uint8_t*>(cache));
  cv.kf = key_fmt_of_config(*cfg);
  cv.sel_offset = lay.sel_offset; cv.sel_stride_b = lay.sel_stride_b; cv.sel_words = lay.sel_words;
  cv.slab_offset = lay.slab_offset; cv.slab_stride = lay.slab_stride;
  cv.chunk_table_offset = lay.chunk_table_offset; cv.kgroup_offset = lay.kgroup_offset;
  cv.tern_offset = lay.tern_offset; cv.prot_offset = lay.prot_offset;
  cv.kres_offset = lay.kres_offset; cv.vres_offset = lay.vres_offset;
  cv.B = cfg->B; cv.H_kv = cfg->H_kv; cv.H_q = cfg->H_q; cv.rep = cfg->H_q / cfg->H_kv;
  a.q = q; a.k_new = nullptr; a.v_new = nullptr; a.out = out;
  a.layer0 = layer_begin; a.n_layers = n_layers;
  a.in_dtype = cfg->in_dtype; a.out_dtype = cfg->out_dtype;
  a.n_prot = n_protected;
  a.scale = softmax_scale > 0.0f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(kD));
  a.st.T_q0 = n_prefill_quantized; a.st.n_flush = n_flushed_chunks; a.st.n_res = n_residual;
  a.ev_begin = nullptr; a.ev_end = nullptr;
  a.withhold = 0;
  a.partial_out = nullptr;
  const int64_t n_slabs = static_cast<int64_t>(n_layers) * cfg->B * cfg->H_kv;
  a.append_row = -1;
  a.plan = plan_decode(a.st, n_slabs, n_protected > 0, device_sm_count(), 0);
  // the array holds the partial records, then (256-byte aligned) the per-chunk query images
  const int64_t prep_at = (a.plan.records * kRecordFloats * 4 + 255) / 256 * 256;
  const int64_t prep_bytes = static_cast<int64_t>(decode_prep_bytes(n_slabs, a.plan.n_chunks));
  if (prep_at + prep_bytes > static_cast<int64_t>(kStaticPartialFloats * sizeof(float))) return VIDKV_ERR_CAPACITY;
  const vidkv_status_t sp = static_partials(&a.partials);
  if (sp != VIDKV_OK) return sp;
  a.prep = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(a.partials) + prep_at);
  // Every record the merge reads is written by the attention kernel of this same call, so
  // nothing in the array has to be cleared between calls.
  if (launch_decode(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}
