// Host side of libvidkv: argument validation, sizing, per-layer token bookkeeping and the
// launch sequences of the C ABI declared in include/vidkv.h.
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "kernels.cuh"

using namespace vidkv;

namespace {

constexpr int64_t kAlign = 256;
inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

struct Layout {
  vidkv_layout_t lay;
  int64_t max_prot;          // protected tokens the cache can hold per slab
  int64_t max_total_tokens;  // prefill + new
};

vidkv_status_t check_config(const vidkv_config_t* c) {
  if (!c) return VIDKV_ERR_INVALID_ARG;
  if (c->B < 1 || c->L < 1 || c->H_kv < 1 || c->H_q < 1) return VIDKV_ERR_INVALID_ARG;
  if (c->max_prefill_tokens < 0 || c->max_new_tokens < 0) return VIDKV_ERR_INVALID_ARG;
  if (!(c->p_ratio >= 0.0f && c->p_ratio <= 1.0f)) return VIDKV_ERR_INVALID_ARG;
  if (!(c->gamma >= 0.0f) || !std::isfinite(c->gamma)) return VIDKV_ERR_INVALID_ARG;
  if (c->in_dtype != VIDKV_F16 && c->in_dtype != VIDKV_BF16) return VIDKV_ERR_INVALID_ARG;
  if (c->out_dtype != VIDKV_F16 && c->out_dtype != VIDKV_BF16 && c->out_dtype != VIDKV_F32) return VIDKV_ERR_INVALID_ARG;
  if (c->ternary_scale != VIDKV_TERNARY_SCALE_MEAN_ABS && c->ternary_scale != VIDKV_TERNARY_SCALE_NONZERO_MEAN)
    return VIDKV_ERR_INVALID_ARG;
  if (c->D != kD || c->G != kG || c->R != kR) return VIDKV_ERR_UNSUPPORTED;
  if (c->key_1bit_mode != VIDKV_KEY1BIT_FFT_SIGN && c->key_1bit_mode != VIDKV_KEY1BIT_PLAIN_MINMAX) return VIDKV_ERR_INVALID_ARG;
  if (c->k_ratio != 0.25f && c->k_ratio != 0.5f && c->k_ratio != 0.75f && c->k_ratio != 1.0f) return VIDKV_ERR_UNSUPPORTED;
  // Eq. 5 needs the transform over the normal channels; the paper applies it at k = 0.5 and 0.75 only
  if (c->key_1bit_mode == VIDKV_KEY1BIT_FFT_SIGN && c->k_ratio == 0.25f) return VIDKV_ERR_UNSUPPORTED;
  if (c->H_q % c->H_kv != 0 || c->H_q / c->H_kv > kMaxRep) return VIDKV_ERR_UNSUPPORTED;
  if (static_cast<int64_t>(c->L) * c->B * c->H_kv > 65535) return VIDKV_ERR_UNSUPPORTED;
  return VIDKV_OK;
}

void compute_layout(const vidkv_config_t& c, Layout* out) {
  vidkv_layout_t& l = out->lay;
  const int64_t Tp = c.max_prefill_tokens, Nn = c.max_new_tokens;
  const int64_t g0 = Tp / kG;
  const int64_t max_flush = (kG - 1 + Nn) / kR;
  out->max_prot = c.p_ratio > 0.0f ? static_cast<int64_t>(std::floor(static_cast<double>(c.p_ratio) * Tp)) : 0;
  out->max_total_tokens = Tp + Nn;
  l.header_bytes = kHeaderBytes;
  l.sel_offset = kHeaderBytes;
  l.sel_words = g0 + 1;
  l.sel_stride_b = round_up(2 * l.sel_words * 4, kAlign);
  l.slab_offset = round_up(l.sel_offset + l.sel_stride_b * c.B, kAlign);
  l.max_chunks = 1 + max_flush;
  l.max_kgroups = g0 + (kR / kG) * max_flush;
  l.max_supergroups = (g0 + 1 + (kR / kG) * max_flush + kSGGroups - 1) / kSGGroups;
  l.max_pgroups = (out->max_prot + kG - 1) / kG;
  int64_t off = 0;
  l.chunk_table_offset = off; off = round_up(off + l.max_chunks * kChunkBytes, kAlign);
  l.kgroup_offset = off;      off = round_up(off + l.max_kgroups * key_fmt_of_config(c).group_bytes, kAlign);
  l.tern_offset = off;        off = round_up(off + l.max_supergroups * kSGBytes, kAlign);
  l.prot_offset = off;        off = round_up(off + l.max_pgroups * kPGBytes, kAlign);
  l.kres_offset = off;        off += kResBytes;
  l.vres_offset = off;        off += kResBytes;
  l.slab_stride = round_up(off, kAlign);
  l.total_bytes = l.slab_offset + l.slab_stride * c.L * c.B * c.H_kv;
}

struct WsPlan {
  int64_t minmax_off, partials_off, prep_off, idx_prot_off, idx_rest_off, counts_off, total;
  int64_t partial_entries;
};

void plan_workspace(const vidkv_config_t& c, const Layout& L, WsPlan* w) {
  int64_t off = 0;
  w->minmax_off = off;
  off = round_up(off + 2 * static_cast<int64_t>(c.L) * c.B * c.H_kv * 2 * kD * 4, kAlign);   // two alternating buffers
  w->partial_entries = max_decode_records(static_cast<int64_t>(c.L) * c.B * c.H_kv, L.max_total_tokens);
  w->partials_off = off;
  off = round_up(off + w->partial_entries * kRecordFloats * 4, kAlign);
  w->prep_off = off;
  off = round_up(off + static_cast<int64_t>(decode_prep_bytes(static_cast<int64_t>(c.L) * c.B * c.H_kv, L.lay.max_chunks)),
                 kAlign);
  w->idx_prot_off = off;
  off = round_up(off + static_cast<int64_t>(c.B) * L.max_prot * 4, kAlign);
  w->idx_rest_off = off;
  off = round_up(off + (L.max_prot > 0 ? static_cast<int64_t>(c.B) * c.max_prefill_tokens * 4 : 0), kAlign);
  w->counts_off = off;
  off = round_up(off + static_cast<int64_t>(c.B) * 4, kAlign);
  w->total = off;
}

struct LayerInfo {
  bool k_done = false, v_done = false;
  int64_t T = 0, T_q0 = 0, n_flush = 0, new_tokens = 0;
  int n_res = 0;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

namespace vidkv { unsigned long long g_launch_count = 0; int g_debug_withhold = 0; }

struct vidkv_cache {
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
  vidkv_config_t cfg;
  Layout L;
  WsPlan ws;
  CacheView cv;
  uint8_t* cache;
  uint8_t* workspace;
  bool sel_set;
  int64_t sel_T, n_prot;
  int dbg_run_units = 0;        // test hook: forced run length of the stream kernels (0 = choose)
  int mm_parity = 0;            // which min / max buffer the next key quantization accumulates into
  int64_t mm_dirty[2] = {0, 0}; // words of each buffer written since it was last re-armed
  std::vector<LayerInfo> layers;
};

// The min / max buffers of the next key quantization over n_slabs slabs (see MinMaxBuffers).
static MinMaxBuffers next_minmax(vidkv_cache* h, int64_t n_slabs) {
  const int64_t words = static_cast<int64_t>(h->cfg.L) * h->cfg.B * h->cfg.H_kv * 2 * kD;
  uint32_t* base = reinterpret_cast<uint32_t*>(h->workspace + h->ws.minmax_off);
  const int p = h->mm_parity;
  MinMaxBuffers mm;
  mm.cur = base + p * words;
  mm.next = base + (1 - p) * words;
  mm.next_dirty_words = static_cast<int>(h->mm_dirty[1 - p]);
  h->mm_dirty[1 - p] = 0;
  h->mm_dirty[p] = n_slabs * 2 * kD;
  h->mm_parity = 1 - p;
  return mm;
}

extern "C" {

int32_t vidkv_version(void) { return 100; }

uint64_t vidkv_launch_count(void) { return g_launch_count; }

vidkv_status_t vidkv_set_profile_events(vidkv_cache_t* h, void* ev_begin, void* ev_end) {
  if (!h || ((ev_begin == nullptr) != (ev_end == nullptr))) return VIDKV_ERR_INVALID_ARG;
  h->ev_begin = static_cast<cudaEvent_t>(ev_begin);
  h->ev_end = static_cast<cudaEvent_t>(ev_end);
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_layout(const vidkv_config_t* cfg, vidkv_layout_t* layout) {
  if (!layout) return VIDKV_ERR_INVALID_ARG;
  const vidkv_status_t st = check_config(cfg);
  if (st != VIDKV_OK) return st;
  Layout L;
  compute_layout(*cfg, &L);
  *layout = L.lay;
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_bytes(const vidkv_config_t* cfg, size_t* cache_bytes, size_t* workspace_bytes) {
  if (!cache_bytes || !workspace_bytes) return VIDKV_ERR_INVALID_ARG;
  const vidkv_status_t st = check_config(cfg);
  if (st != VIDKV_OK) return st;
  Layout L;
  compute_layout(*cfg, &L);
  WsPlan w;
  plan_workspace(*cfg, L, &w);
  *cache_bytes = static_cast<size_t>(L.lay.total_bytes);
  *workspace_bytes = static_cast<size_t>(w.total);
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_init(const vidkv_config_t* cfg, void* cache, size_t cache_bytes, void* workspace,
                                size_t workspace_bytes, void* stream, vidkv_cache_t** handle) {
  if (!handle) return VIDKV_ERR_INVALID_ARG;
  *handle = nullptr;
  const vidkv_status_t st = check_config(cfg);
  if (st != VIDKV_OK) return st;
  if (!cache || !workspace) return VIDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(cache) % kAlign) || (reinterpret_cast<uintptr_t>(workspace) % kAlign))
    return VIDKV_ERR_ALIGNMENT;
  vidkv_cache* h = new (std::nothrow) vidkv_cache();
  if (!h) return VIDKV_ERR_INVALID_ARG;
  h->cfg = *cfg;
  compute_layout(*cfg, &h->L);
  plan_workspace(*cfg, h->L, &h->ws);
  if (cache_bytes < static_cast<size_t>(h->L.lay.total_bytes) || workspace_bytes < static_cast<size_t>(h->ws.total)) {
    delete h;
    return VIDKV_ERR_CAPACITY;
  }
  h->cache = static_cast<uint8_t*>(cache);
  h->workspace = static_cast<uint8_t*>(workspace);
  const vidkv_layout_t& l = h->L.lay;
  CacheView& cv = h->cv;
  cv.base = h->cache;
  cv.kf = key_fmt_of_config(*cfg);
  cv.sel_offset = l.sel_offset; cv.sel_stride_b = l.sel_stride_b; cv.sel_words = l.sel_words;
  cv.slab_offset = l.slab_offset; cv.slab_stride = l.slab_stride;
  cv.chunk_table_offset = l.chunk_table_offset; cv.kgroup_offset = l.kgroup_offset;
  cv.tern_offset = l.tern_offset; cv.prot_offset = l.prot_offset;
  cv.kres_offset = l.kres_offset; cv.vres_offset = l.vres_offset;
  cv.B = cfg->B; cv.H_kv = cfg->H_kv; cv.H_q = cfg->H_q; cv.rep = cfg->H_q / cfg->H_kv;
  h->sel_set = false; h->sel_T = 0; h->n_prot = 0;
  h->layers.assign(cfg->L, LayerInfo());
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(h->cache, 0, static_cast<size_t>(l.total_bytes), s) != cudaSuccess) { delete h; return VIDKV_ERR_CUDA; }
  // the kernel that arms the channel-range accumulators also writes the header words
  if (launch_init_minmax(reinterpret_cast<uint32_t*>(h->workspace + h->ws.minmax_off),
                         2 * static_cast<int64_t>(cfg->L) * cfg->B * cfg->H_kv * 2 * kD, reinterpret_cast<uint32_t*>(h->cache),
                         static_cast<uint32_t>(vidkv_version()), s) != cudaSuccess) {
    delete h;
    return VIDKV_ERR_CUDA;
  }
  *handle = h;
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_destroy(vidkv_cache_t* h) {
  if (!h) return VIDKV_ERR_INVALID_ARG;
  delete h;
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_reset(vidkv_cache_t* h, void* stream) {
  (void)stream;
  if (!h) return VIDKV_ERR_INVALID_ARG;
  h->sel_set = false; h->sel_T = 0; h->n_prot = 0;
  h->layers.assign(h->cfg.L, LayerInfo());
  return VIDKV_OK;
}

vidkv_status_t vidkv_channel_metrics(int32_t dtype, const void* K, int64_t B, int64_t H, int64_t T, int64_t stride_b,
                                     int64_t stride_h, int64_t stride_t, int32_t metric, float M, double* scratch,
                                     float* out, void* stream) {
  if (dtype != VIDKV_F16 && dtype != VIDKV_BF16) return VIDKV_ERR_INVALID_ARG;
  if (metric != VIDKV_METRIC_VARIANCE && metric != VIDKV_METRIC_OUTLIERS) return VIDKV_ERR_INVALID_ARG;
  if (B < 0 || H < 0 || T < 1 || !(M > 0.0f) || !std::isfinite(M)) return VIDKV_ERR_INVALID_ARG;
  if (B == 0 || H == 0) return VIDKV_OK;
  if (!K || !scratch || !out) return VIDKV_ERR_INVALID_ARG;
  if (B * H > 65535 || H > INT32_MAX) return VIDKV_ERR_UNSUPPORTED;
  if (stride_b % 8 || stride_h % 8 || stride_t % 8 || stride_t < kD) return VIDKV_ERR_ALIGNMENT;
  if (!aligned16(K) || !aligned16(scratch) || !aligned16(out)) return VIDKV_ERR_ALIGNMENT;
  const KSrc src{K, stride_b, stride_h, stride_t, static_cast<int32_t>(H)};
  if (launch_channel_metrics(dtype, src, B * H, T, metric, static_cast<double>(M), scratch, out,
                             static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_saliency_scores(int32_t dtype, const void* x_v, const void* x_t, int64_t B, int64_t l_v, int64_t l_t,
                                     int64_t d, float* text_sum, float* saliency, void* stream) {
  if (dtype != VIDKV_F16 && dtype != VIDKV_BF16) return VIDKV_ERR_INVALID_ARG;
  if (B < 0 || l_v < 0 || l_t < 0 || d < 1) return VIDKV_ERR_INVALID_ARG;
  if (B == 0 || l_v == 0) return VIDKV_OK;
  if (!x_v || !text_sum || !saliency || (l_t > 0 && !x_t)) return VIDKV_ERR_INVALID_ARG;
  if (d % 8 != 0 || d > 16384 || B > 65535) return VIDKV_ERR_UNSUPPORTED;
  if (!aligned16(x_v) || !aligned16(text_sum) || !aligned16(saliency) || (l_t > 0 && !aligned16(x_t))) return VIDKV_ERR_ALIGNMENT;
  if (launch_saliency(dtype, x_v, x_t, B, l_v, l_t, d, text_sum, saliency, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_select_tokens(vidkv_cache_t* h, const float* saliency, int64_t vis_begin, int64_t l_v, int64_t T,
                                   void* stream) {
  if (!h || T < 0) return VIDKV_ERR_INVALID_ARG;
  if (T > h->cfg.max_prefill_tokens) return VIDKV_ERR_CAPACITY;
  for (const LayerInfo& li : h->layers)
    if (li.v_done) return VIDKV_ERR_STATE;
  const int64_t T_q = T - T % kG;
  if (!saliency || h->cfg.p_ratio == 0.0f) {
    h->sel_set = true; h->sel_T = T; h->n_prot = 0;
    return VIDKV_OK;
  }
  if (vis_begin < 0 || l_v < 1 || vis_begin + l_v > T_q) return VIDKV_ERR_INVALID_ARG;
  if (!aligned16(saliency)) return VIDKV_ERR_ALIGNMENT;
  const int64_t n = static_cast<int64_t>(std::floor(static_cast<double>(h->cfg.p_ratio) * static_cast<double>(l_v)));
  if (n > h->L.max_prot) return VIDKV_ERR_CAPACITY;
  if (n > 0) {
    int32_t* ip = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_prot_off);
    int32_t* ir = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_rest_off);
    if (launch_select_tokens(saliency, vis_begin, l_v, n, T_q, h->cv, ip, ir, h->L.max_prot, h->cfg.max_prefill_tokens,
                             static_cast<cudaStream_t>(stream)) != cudaSuccess)
      return VIDKV_ERR_CUDA;
  }
  h->sel_set = true; h->sel_T = T; h->n_prot = n;
  return VIDKV_OK;
}

vidkv_status_t vidkv_set_token_mask(vidkv_cache_t* h, const uint8_t* E, int64_t T, int64_t n_protected, void* stream) {
  if (!h || !E || T < 0 || n_protected < -1) return VIDKV_ERR_INVALID_ARG;
  if (T > h->cfg.max_prefill_tokens) return VIDKV_ERR_CAPACITY;
  for (const LayerInfo& li : h->layers)
    if (li.v_done) return VIDKV_ERR_STATE;
  if (h->L.max_prot == 0 || n_protected > h->L.max_prot) return VIDKV_ERR_CAPACITY;
  const int64_t T_q = T - T % kG;
  if (n_protected > T_q) return VIDKV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* ip = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_prot_off);
  int32_t* ir = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_rest_off);
  int32_t* dc = reinterpret_cast<int32_t*>(h->workspace + h->ws.counts_off);
  if (launch_mask_to_selection(E, T, T_q, h->cv, ip, ir, h->L.max_prot, h->cfg.max_prefill_tokens, dc, n_protected, s) !=
      cudaSuccess)
    return VIDKV_ERR_CUDA;
  if (n_protected >= 0) {
    // the caller stated the count: nothing comes back to the host; a row that disagrees is
    // reported through the cache's status word
    h->sel_set = true; h->sel_T = T; h->n_prot = n_protected;
    return VIDKV_OK;
  }
  std::vector<int32_t> counts(h->cfg.B);
  if (cudaMemcpyAsync(counts.data(), dc, sizeof(int32_t) * h->cfg.B, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  for (int b = 1; b < h->cfg.B; ++b)
    if (counts[b] != counts[0]) return VIDKV_ERR_INVALID_ARG;
  if (counts[0] > h->L.max_prot) return VIDKV_ERR_CAPACITY;
  h->sel_set = true; h->sel_T = T; h->n_prot = counts[0];
  return VIDKV_OK;
}

static vidkv_status_t check_kv_args(vidkv_cache_t* h, int32_t layer, const void* X, int64_t T, int64_t sb, int64_t sh,
                                    int64_t st) {
  if (!h || T < 0 || (!X && T > 0)) return VIDKV_ERR_INVALID_ARG;   // an empty prompt may come with a null pointer
  if (layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  if (sb < 0 || sh < 0 || st < kD) return VIDKV_ERR_INVALID_ARG;
  if (!aligned16(X) || (sb % 8) || (sh % 8) || (st % 8)) return VIDKV_ERR_ALIGNMENT;
  if (T > h->cfg.max_prefill_tokens) return VIDKV_ERR_CAPACITY;
  return VIDKV_OK;
}

vidkv_status_t vidkv_quantize_keys_layers(vidkv_cache_t* h, int32_t layer_begin, int32_t n_layers, const void* K, int64_t T,
                                          int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream) {
  vidkv_status_t st = check_kv_args(h, layer_begin, K, T, stride_b, stride_h, stride_t);
  if (st != VIDKV_OK) return st;
  if (n_layers < 1 || layer_begin + n_layers > h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    const LayerInfo& li = h->layers[l];
    if (li.k_done) return VIDKV_ERR_STATE;
    if (li.v_done && li.T != T) return VIDKV_ERR_STATE;
  }
  const int64_t T_q = T - T % kG;
  const int r = static_cast<int>(T % kG);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  KSrc src{K, stride_b, stride_h, stride_t, h->cfg.H_kv};
  if (T_q > 0) {
    const MinMaxBuffers mm = next_minmax(h, static_cast<int64_t>(n_layers) * h->cfg.B * h->cfg.H_kv);
    if (launch_quantize_keys(h->cfg.in_dtype, src, T_q, h->cv, layer_begin, n_layers, 0, 0, mm, s) != cudaSuccess)
      return VIDKV_ERR_CUDA;
  }
  if (launch_copy_to_residual(h->cfg.in_dtype, src, T_q, r, h->cv, layer_begin, n_layers, false, 0, s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    LayerInfo& li = h->layers[l];
    li.k_done = true; li.T = T; li.T_q0 = T_q; li.n_res = r; li.n_flush = 0;
  }
  return VIDKV_OK;
}

vidkv_status_t vidkv_quantize_keys(vidkv_cache_t* h, int32_t layer, const void* K, int64_t T, int64_t stride_b,
                                   int64_t stride_h, int64_t stride_t, void* stream) {
  return vidkv_quantize_keys_layers(h, layer, 1, K, T, stride_b, stride_h, stride_t, stream);
}

vidkv_status_t vidkv_quantize_values_layers(vidkv_cache_t* h, int32_t layer_begin, int32_t n_layers, const void* V, int64_t T,
                                            int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream) {
  vidkv_status_t st = check_kv_args(h, layer_begin, V, T, stride_b, stride_h, stride_t);
  if (st != VIDKV_OK) return st;
  if (n_layers < 1 || layer_begin + n_layers > h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    const LayerInfo& li = h->layers[l];
    if (li.v_done) return VIDKV_ERR_STATE;
    if (li.k_done && li.T != T) return VIDKV_ERR_STATE;
  }
  if (h->cfg.p_ratio > 0.0f && !h->sel_set) return VIDKV_ERR_STATE;
  if (h->sel_set && h->n_prot > 0 && h->sel_T != T) return VIDKV_ERR_STATE;
  const int64_t T_q = T - T % kG;
  const int r = static_cast<int>(T % kG);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  KSrc src{V, stride_b, stride_h, stride_t, h->cfg.H_kv};
  SelView sel{nullptr, nullptr, 0, 0, 0};
  if (h->sel_set && h->n_prot > 0) {
    sel.idx_prot = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_prot_off);
    sel.idx_rest = reinterpret_cast<int32_t*>(h->workspace + h->ws.idx_rest_off);
    sel.stride_prot = h->L.max_prot;
    sel.stride_rest = h->cfg.max_prefill_tokens;
    sel.n_prot = h->n_prot;
  }
  if (T_q > 0 && launch_quantize_values(h->cfg.in_dtype, src, T_q, h->cv, layer_begin, n_layers, sel, h->cfg.gamma,
                                        h->cfg.ternary_scale == VIDKV_TERNARY_SCALE_NONZERO_MEAN, s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  if (launch_copy_to_residual(h->cfg.in_dtype, src, T_q, r, h->cv, layer_begin, n_layers, true, 0, s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    LayerInfo& li = h->layers[l];
    li.v_done = true; li.T = T; li.T_q0 = T_q; li.n_res = r; li.n_flush = 0;
  }
  return VIDKV_OK;
}

vidkv_status_t vidkv_quantize_values(vidkv_cache_t* h, int32_t layer, const void* V, int64_t T, int64_t stride_b,
                                     int64_t stride_h, int64_t stride_t, void* stream) {
  return vidkv_quantize_values_layers(h, layer, 1, V, T, stride_b, stride_h, stride_t, stream);
}

}  // extern "C"

// Algorithm 1 "Decoding" for a layer range.  append: k_new / v_new join the residual first (and a full
// residual is flushed afterwards); without it the cache is attended to as it stands.  partial: leave
// (maximum, sum, unnormalised out) per query head instead of the normalised output.
static vidkv_status_t decode_impl(vidkv_cache_t* h, int32_t layer_begin, int32_t n_layers, const void* q, const void* k_new,
                                  const void* v_new, void* out, float* partial, float softmax_scale, void* stream) {
  const bool append = k_new != nullptr;
  if (!h || !q || (k_new == nullptr) != (v_new == nullptr) || (!out && !partial)) return VIDKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || n_layers < 1 || layer_begin + n_layers > h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out) || !aligned16(partial)) return VIDKV_ERR_ALIGNMENT;
  if (!std::isfinite(softmax_scale)) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& first = h->layers[layer_begin];
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    const LayerInfo& li = h->layers[l];
    if (!li.k_done || !li.v_done) return VIDKV_ERR_STATE;
    if (li.T_q0 != first.T_q0 || li.n_flush != first.n_flush || li.n_res != first.n_res) return VIDKV_ERR_STATE;
    if (append && li.new_tokens + 1 > h->cfg.max_new_tokens) return VIDKV_ERR_CAPACITY;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int dt = h->cfg.in_dtype;
  // the append rides on the query-preparation kernel when there is one (some chunk is quantized)
  const bool has_chunks = first.T_q0 + first.n_flush * kR > 0;
  if (!append && !has_chunks && first.n_res == 0) return VIDKV_ERR_STATE;       // nothing to attend to
  if (append && !has_chunks && launch_append(dt, k_new, v_new, h->cv, layer_begin, n_layers, first.n_res, s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  DecodeArgs a;
  a.cv = h->cv;
  a.q = q; a.k_new = k_new; a.v_new = v_new; a.out = out;
  a.partials = reinterpret_cast<float*>(h->workspace + h->ws.partials_off);
  a.prep = reinterpret_cast<uint32_t*>(h->workspace + h->ws.prep_off);
  a.append_row = append && has_chunks ? first.n_res : -1;
  a.partial_out = partial;
  a.layer0 = layer_begin; a.n_layers = n_layers;
  a.in_dtype = dt; a.out_dtype = h->cfg.out_dtype;
  a.n_prot = h->n_prot;
  a.scale = softmax_scale > 0.0f ? softmax_scale : 1.0f / std::sqrt(static_cast<float>(kD));
  a.ev_begin = h->ev_begin; a.ev_end = h->ev_end;
  a.withhold = 0;
  a.st.T_q0 = first.T_q0; a.st.n_flush = first.n_flush; a.st.n_res = first.n_res + (append ? 1 : 0);
  const int64_t n_slabs = static_cast<int64_t>(n_layers) * h->cfg.B * h->cfg.H_kv;
  a.plan = plan_decode(a.st, n_slabs, h->n_prot > 0, device_sm_count(), h->dbg_run_units);
  if (a.plan.records > h->ws.partial_entries) return VIDKV_ERR_CAPACITY;
  if (launch_decode(a, s) != cudaSuccess) return VIDKV_ERR_CUDA;
  if (!append) return VIDKV_OK;
  const bool flush = a.st.n_res == kR;
  if (flush) {
    const int64_t es = h->cv.slab_stride / 2;    // slab stride in 16-bit elements
    const uint8_t* slab0 = h->cache + h->cv.slab_offset + static_cast<int64_t>(layer_begin) * h->cfg.B * h->cfg.H_kv * h->cv.slab_stride;
    KSrc ksrc{slab0 + h->cv.kres_offset, es * h->cfg.H_kv, es, kD, h->cfg.H_kv};
    KSrc vsrc{slab0 + h->cv.vres_offset, es * h->cfg.H_kv, es, kD, h->cfg.H_kv};
    const MinMaxBuffers mm = next_minmax(h, static_cast<int64_t>(n_layers) * h->cfg.B * h->cfg.H_kv);
    const int chunk = 1 + static_cast<int>(first.n_flush);
    const int64_t kgroup0 = first.T_q0 / kG + (kR / kG) * first.n_flush;
    if (launch_quantize_keys(dt, ksrc, kR, h->cv, layer_begin, n_layers, chunk, kgroup0, mm, s) != cudaSuccess)
      return VIDKV_ERR_CUDA;
    const int64_t n_rest = first.T_q0 - h->n_prot;
    const int64_t tgroup0 = (n_rest + kG - 1) / kG + (kR / kG) * first.n_flush;
    if (launch_flush_values(dt, vsrc, h->cv, layer_begin, n_layers, tgroup0, h->cfg.gamma,
                            h->cfg.ternary_scale == VIDKV_TERNARY_SCALE_NONZERO_MEAN, s) != cudaSuccess)
      return VIDKV_ERR_CUDA;
  }
  for (int l = layer_begin; l < layer_begin + n_layers; ++l) {
    LayerInfo& li = h->layers[l];
    li.new_tokens += 1;
    if (flush) { li.n_flush += 1; li.n_res = 0; }
    else li.n_res += 1;
  }
  return VIDKV_OK;
}

extern "C" {

vidkv_status_t vidkv_decode_attention(vidkv_cache_t* h, int32_t layer_begin, int32_t n_layers, const void* q,
                                      const void* k_new, const void* v_new, void* out, float softmax_scale,
                                      void* stream) {
  if (!k_new || !v_new || !out) return VIDKV_ERR_INVALID_ARG;
  return decode_impl(h, layer_begin, n_layers, q, k_new, v_new, out, nullptr, softmax_scale, stream);
}

vidkv_status_t vidkv_decode_attention_partial(vidkv_cache_t* h, int32_t layer_begin, int32_t n_layers, const void* q,
                                              const void* k_new, const void* v_new, float* partial, float softmax_scale,
                                              void* stream) {
  if (!partial) return VIDKV_ERR_INVALID_ARG;
  return decode_impl(h, layer_begin, n_layers, q, k_new, v_new, nullptr, partial, softmax_scale, stream);
}

vidkv_status_t vidkv_merge_partials(const float* partials, int64_t n_parts, int64_t n_rows, void* out, int32_t out_dtype,
                                    void* stream) {
  if (!partials || !out || n_parts < 1 || n_rows < 0) return VIDKV_ERR_INVALID_ARG;
  if (out_dtype != VIDKV_F16 && out_dtype != VIDKV_BF16 && out_dtype != VIDKV_F32) return VIDKV_ERR_INVALID_ARG;
  if (!aligned16(partials) || !aligned16(out)) return VIDKV_ERR_ALIGNMENT;
  if (n_rows == 0) return VIDKV_OK;
  if (n_rows > 0x7fffffff) return VIDKV_ERR_UNSUPPORTED;
  if (launch_merge_partials(partials, n_parts, n_rows, out, out_dtype, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_debug_withhold_once(int32_t what) {
  if (what < 0 || what > 2) return VIDKV_ERR_INVALID_ARG;
  g_debug_withhold = what;
  return VIDKV_OK;
}

vidkv_status_t vidkv_debug_set_decode_plan(vidkv_cache_t* h, int32_t run_units) {
  if (!h || run_units < 0) return VIDKV_ERR_INVALID_ARG;
  h->dbg_run_units = run_units;
  return VIDKV_OK;
}

vidkv_status_t vidkv_debug_decode_plan(const vidkv_config_t* cfg, int64_t n_prefill_quantized, int64_t n_flushed_chunks,
                                       int32_t n_residual, int64_t n_protected, int32_t n_layers, int32_t sm_count,
                                       int32_t run_units, int64_t* plan_out) {
  if (!plan_out) return VIDKV_ERR_INVALID_ARG;
  const vidkv_status_t st = check_config(cfg);
  if (st != VIDKV_OK) return st;
  if (n_layers < 1 || n_layers > cfg->L || n_prefill_quantized < 0 || n_prefill_quantized % kG || n_flushed_chunks < 0 ||
      n_residual < 0 || n_residual > kR || n_protected < 0 || sm_count < 1 || run_units < 0)
    return VIDKV_ERR_INVALID_ARG;
  Layout L;
  compute_layout(*cfg, &L);
  WsPlan w;
  plan_workspace(*cfg, L, &w);
  LayerState ls;
  ls.T_q0 = n_prefill_quantized; ls.n_flush = n_flushed_chunks; ls.n_res = n_residual;
  const DecodePlan p = plan_decode(ls, static_cast<int64_t>(n_layers) * cfg->B * cfg->H_kv, n_protected > 0, sm_count, run_units);
  plan_out[0] = p.units_per_slab; plan_out[1] = p.run_units; plan_out[2] = p.n_runs; plan_out[3] = p.parts_stride;
  plan_out[4] = p.records; plan_out[5] = w.partial_entries; plan_out[6] = p.n_chunks; plan_out[7] = p.n_units;
  return VIDKV_OK;
}

vidkv_status_t vidkv_layer_state(const vidkv_cache_t* h, int32_t layer, int64_t* n_quantized, int64_t* n_residual,
                                 int64_t* n_chunks, int64_t* n_protected) {
  if (!h || layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& li = h->layers[layer];
  if (n_quantized) *n_quantized = li.T_q0 + li.n_flush * kR;
  if (n_residual) *n_residual = li.n_res;
  if (n_chunks) *n_chunks = (li.T_q0 > 0 ? 1 : 0) + li.n_flush;
  if (n_protected) *n_protected = h->n_prot;
  return VIDKV_OK;
}

vidkv_status_t vidkv_cache_status(vidkv_cache_t* h, void* stream) {
  if (!h) return VIDKV_ERR_INVALID_ARG;
  int32_t word = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&word, h->cache + kHdrStatus, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return word;
}

vidkv_status_t vidkv_export_codes(vidkv_cache_t* h, int32_t layer, int8_t* k2, uint8_t* k1bits, void* k_s2, void* k_z2,
                                  void* k_s1, int8_t* v_trits, void* v_s, int8_t* v2, void* v2_s, void* v2_z,
                                  void* stream) {
  if (!h || layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& li = h->layers[layer];
  if (!li.k_done || !li.v_done) return VIDKV_ERR_STATE;
  const int64_t n_kgroups = li.T_q0 / kG + (kR / kG) * li.n_flush;
  const int64_t n_rest = li.T_q0 - h->n_prot;
  const int64_t n_tgroups = (n_rest + kG - 1) / kG + (kR / kG) * li.n_flush;
  const int64_t n_pgroups = (h->n_prot + kG - 1) / kG;
  if (launch_export_codes(h->cv, layer, n_kgroups, n_tgroups, n_pgroups, k2, k1bits, static_cast<uint16_t*>(k_s2),
                          static_cast<uint16_t*>(k_z2), static_cast<uint16_t*>(k_s1), v_trits, static_cast<uint16_t*>(v_s),
                          v2, static_cast<uint16_t*>(v2_s), static_cast<uint16_t*>(v2_z),
                          static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_get_selection(vidkv_cache_t* h, int32_t layer, uint8_t* dmask, uint8_t* E, void* stream) {
  if (!h || layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& li = h->layers[layer];
  if (dmask && !li.k_done) return VIDKV_ERR_STATE;
  const int n_chunks = static_cast<int>(1 + li.n_flush);
  const int64_t T = li.k_done || li.v_done ? li.T : h->sel_T;
  const int64_t T_sel = h->sel_set && h->n_prot > 0 ? h->sel_T - h->sel_T % kG : 0;
  if (launch_export_selection(h->cv, layer, n_chunks, dmask, T, T_sel, E, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_dequantize_keys(vidkv_cache_t* h, int32_t layer, float* out, void* stream) {
  if (!h || layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& li = h->layers[layer];
  if (!li.k_done) return VIDKV_ERR_STATE;
  if (li.T_q0 + li.n_flush * kR == 0) return VIDKV_OK;
  if (!out) return VIDKV_ERR_INVALID_ARG;
  if (launch_dequant_keys(h->cv, layer, li.T_q0, li.n_flush, out, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

vidkv_status_t vidkv_dequantize_values(vidkv_cache_t* h, int32_t layer, float* out, void* stream) {
  if (!h || layer < 0 || layer >= h->cfg.L) return VIDKV_ERR_INVALID_ARG;
  const LayerInfo& li = h->layers[layer];
  if (!li.v_done) return VIDKV_ERR_STATE;
  if (li.T_q0 + li.n_flush * kR == 0) return VIDKV_OK;
  if (!out) return VIDKV_ERR_INVALID_ARG;
  if (launch_dequant_values(h->cv, layer, li.T_q0, li.n_flush, h->n_prot, out, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return VIDKV_ERR_CUDA;
  return VIDKV_OK;
}

}  // extern "C"
