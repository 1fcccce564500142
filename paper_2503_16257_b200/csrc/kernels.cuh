// Internal launcher interface between the host API and the kernel files.
#pragma once

#include "common.cuh"

namespace vidkv {

// A [slabs, tokens, 128] source of keys or values.  Source slab i (= b * H + h, running
// over layers first when several layers are processed) starts at
// ptr + (i / H) * stride_b + (i % H) * stride_h elements; token t at + t * stride_t.
struct KSrc {
  const void* ptr;
  int64_t stride_b, stride_h, stride_t;
  int32_t H;
};

// Token-selection data handed to the value quantizer (NULL lists = no protection).
struct SelView {
  const int32_t* idx_prot;   // [B][n_prot]       ascending protected token ids
  const int32_t* idx_rest;   // [B][T - n_prot]   ascending unprotected token ids
  int64_t stride_prot, stride_rest;
  int64_t n_prot;
};

// Channel min / max accumulators of the range pass: 256 ordered-integer words per slab (128
// minima that start at all ones, 128 maxima that start at zero).  Two buffers alternate: a call
// accumulates into `cur`, which the call before it re-armed, and re-arms the first
// `next_dirty_words` words of `next` for the call after it, so no call spends a launch on it.
struct MinMaxBuffers {
  uint32_t* cur;
  uint32_t* next;
  int next_dirty_words;
};
// Also writes the cache header (magic, version, cleared status word) when `header` is not null.
cudaError_t launch_init_minmax(uint32_t* minmax, int64_t n_words, uint32_t* header, uint32_t version, cudaStream_t stream);

// Algorithm 3 on `T_tokens` tokens (a multiple of 32) of every slab of layers
// [layer0, layer0 + n_layers): writes chunk `chunk` of the chunk table and the key groups
// starting at group index kgroup0.
cudaError_t launch_quantize_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0,
                                 int n_layers, int chunk, int64_t kgroup0, const MinMaxBuffers& mm, cudaStream_t stream);

// Encode pass of Algorithm 3 for `n_slabs` slabs whose channel split (chunk table entry
// `chunk`) is already written.
cudaError_t launch_encode_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_slabs,
                               int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream);

// The same for the general key formats (other k, plain 1-bit code): one block per 32-token group.
cudaError_t launch_encode_keys_general(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0,
                                       int n_slabs, int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream);

// Device address of the 64-point DFT matrix in MMA B-fragment order: word
// ((ks * 8 + nt) * 32 + lane) * 4 + {0, 1} = leading binary16 pairs, + {2, 3} = remainders, for
// rows 16 ks + 2 r (+1; +8, +9) and column 16 (n / 2) + 2 nt + (n % 2), lane = 4 n + r; column f
// holds 1/8, (-1)^c / 8, cos(2 pi k c / 64) / 8 (f = 2k) or -sin(2 pi k c / 64) / 8 (f = 2k + 1).
// Filled on first use on each device by one small kernel; later calls order their stream after it with an event.
cudaError_t dft_fragments(const uint32_t** table, cudaStream_t stream);

// Algorithm 2 on the prefill tokens of n_layers layers (source slabs run over layers, then b, then h).  T_q (multiple of 32) tokens; the
// unprotected ones go to ternary stream positions 0.., the protected ones to 2-bit groups.
cudaError_t launch_quantize_values(int dtype, const KSrc& src, int64_t T_q, const CacheView& cv, int layer, int n_layers,
                                   const SelView& sel, float gamma, bool nonzero_mean_scale, cudaStream_t stream);

// 1.58Quant of a full 128-token residual of every slab of the given layers, appended at
// ternary stream group index tgroup0 (read-modify-write of shared supergroup bytes).
cudaError_t launch_flush_values(int dtype, const KSrc& src, const CacheView& cv, int layer0, int n_layers,
                                int64_t tgroup0, float gamma, bool nonzero_mean_scale, cudaStream_t stream);

// Copy `n_tok` tokens starting at token t_begin of every slab of one layer into the
// residual rings (rows r0 .. r0 + n_tok - 1); n_layers layers from `layer` on.
cudaError_t launch_copy_to_residual(int dtype, const KSrc& src, int64_t t_begin, int n_tok, const CacheView& cv,
                                    int layer, int n_layers, bool is_value, int r0, cudaStream_t stream);

// Token selection (Sec. 3.3(2)): top-n by saliency, E words + prefix counts into the cache,
// gather lists into the workspace.
cudaError_t launch_select_tokens(const float* saliency, int64_t vis_begin, int64_t l_v, int64_t n_prot, int64_t T_q,
                                 const CacheView& cv, int32_t* idx_prot, int32_t* idx_rest, int64_t stride_prot,
                                 int64_t stride_rest, cudaStream_t stream);
cudaError_t launch_mask_to_selection(const uint8_t* E, int64_t T, int64_t T_q, const CacheView& cv, int32_t* idx_prot,
                                     int32_t* idx_rest, int64_t stride_prot, int64_t stride_rest, int32_t* counts,
                                     int64_t expect_count, cudaStream_t stream);

// Token counts the decode kernels need (the same for every layer of one call).
struct LayerState {
  int64_t T_q0;        // prefill tokens quantized (multiple of 32)
  int64_t n_flush;     // flushed 128-token chunks
  int32_t n_res;       // residual tokens (after the append of this step)
};

constexpr int kStreamUnitTokens = 160;  // one unit of the stream kernel: 5 key groups = 1 ternary supergroup
constexpr int kStreamWarps = 4;         // warps per CTA of the stream kernel
constexpr int kStreamCtasPerSM = 3;     // its CTAs per multiprocessor (register bound)
constexpr int kStreamStpCtasPerSM = 2;  // the same for the variant with protected tokens (shared-memory bound)
constexpr int kPrepWords = 25;     // 32-bit words per lane per (slab, chunk) of prepared query
constexpr int kRecordFloats = 130; // one partial record: running maximum (base-2 logits), sum, out[128]

// How one attention call over n_slabs slabs is cut into work (host side, decode.cu): the
// quantized tokens of all slabs form one sequence of 160-token units (units_per_slab each); warp
// number w of the launch walks the units [w * run_units, (w + 1) * run_units) and leaves one
// partial record per slab it touches, record (slab, w - first warp of the slab).
// parts_stride = records reserved per slab; the partials buffer holds n_slabs * parts_stride * 8
// records of kRecordFloats floats.
struct DecodePlan {
  int32_t units_per_slab, run_units, n_runs;
  int64_t n_units;
  int32_t parts_stride;
  int32_t n_chunks;        // chunk-table entries the query preparation covers (0: nothing quantized)
  int64_t records;         // n_slabs * parts_stride * 8
};
// stp: the cache holds protected tokens (the kernel for them keeps fewer warps per multiprocessor).
// force_run_units: 0 = choose; otherwise the test hook's value.
DecodePlan plan_decode(const LayerState& st, int64_t n_slabs, bool stp, int sm_count, int force_run_units);
// Largest `records` any call on at most max_slabs slabs and max_tokens tokens can plan.
int64_t max_decode_records(int64_t max_slabs, int64_t max_tokens);
// Multiprocessors of the current device (cached per device); 0 on error.
int device_sm_count();

struct DecodeArgs {
  CacheView cv;
  const void* q;
  const void* k_new;
  const void* v_new;
  void* out;
  float* partials;     // [n_slabs][parts_stride][8 heads][kRecordFloats]
  uint32_t* prep;      // per (slab, chunk) query images of the tensor-core path (decode_prep_bytes)
  const uint32_t* dft; // DFT matrix fragments (dft_fragments), set by launch_decode_prep
  int32_t append_row;  // >= 0: the preparation kernel also writes k_new / v_new into this residual row
  int32_t layer0, n_layers;
  int32_t in_dtype, out_dtype;
  DecodePlan plan;
  int64_t n_prot;      // protected tokens per batch element (0 = no STP)
  float scale;
  LayerState st;
  cudaEvent_t ev_begin, ev_end;   // optional: recorded around the attention kernel (profiling)
  int32_t withhold;    // test hook: the stream kernel does not issue its first value copy
  float* partial_out;  // not null: leave [n_layers * B * H_q][kRecordFloats] (max, sum, unnormalised out) instead of `out`
};

// Eq. 7 scores from hidden states: text_sum [B, d] (scratch) and saliency [B, l_v], both float32.
cudaError_t launch_saliency(int dtype, const void* x_v, const void* x_t, int64_t B, int64_t l_v, int64_t l_t, int64_t d,
                            float* text_sum, float* saliency, cudaStream_t stream);

// Variance / outlier count per (slab, channel) of a key tensor; stats [n_slabs][2][128] float64 scratch.
cudaError_t launch_channel_metrics(int dtype, const KSrc& src, int64_t n_slabs, int64_t T_tokens, int metric, double M,
                                   double* stats, float* out, cudaStream_t stream);

// Test hook (vidkv_debug_withhold_once): 1 = the next key-encode launch withholds the tensor-core
// products of every block's first tile, 2 = the next stream-kernel launch withholds every warp's
// first value copy; the launch that honours it clears it.  0 = off.
extern int g_debug_withhold;

// Number of kernels launched by this library since it was loaded (host counter).
extern unsigned long long g_launch_count;
inline void count_launches(int n) { g_launch_count += static_cast<unsigned long long>(n); }

// Attention over the packed cache + residual: query preparation, the stream kernel, then the merge
// of the partial records, which also attends to the residual.
cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream);
// Log-sum-exp merge of n_parts partial sets [n_parts][n_rows][kRecordFloats] into out [n_rows][128].
cudaError_t launch_merge_partials(const float* parts, int64_t n_parts, int64_t n_rows, void* out, int out_dtype,
                                  cudaStream_t stream);
// Query preparation (and the step's append) for a.plan.n_chunks chunk-table entries per slab.
cudaError_t launch_decode_prep(DecodeArgs& a, cudaStream_t stream);
// Persistent warps over 160-token units: caches without / with protected tokens.
cudaError_t launch_decode_stream(const DecodeArgs& a, cudaStream_t stream);
cudaError_t launch_decode_stream_stp(const DecodeArgs& a, cudaStream_t stream);
size_t decode_prep_bytes(int64_t n_slabs, int64_t n_chunks);
// Write k_new / v_new [n_layers, B, H_kv, D] into row `row` of the residual rings.
cudaError_t launch_append(int dtype, const void* k_new, const void* v_new, const CacheView& cv, int layer0,
                          int n_layers, int row, cudaStream_t stream);

// Test-only dequantizers (float32 [B, H_kv, n_quantized, D]).
cudaError_t launch_dequant_keys(const CacheView& cv, int layer, int64_t T_q0, int64_t n_flush, float* out,
                                cudaStream_t stream);
cudaError_t launch_dequant_values(const CacheView& cv, int layer, int64_t T_q0, int64_t n_flush, int64_t n_prot,
                                  float* out, cudaStream_t stream);

// Test-only exports: undo the bit packing of one layer into plain arrays (any pointer may be null).
cudaError_t launch_export_codes(const CacheView& cv, int layer, int64_t n_kgroups, int64_t n_tgroups, int64_t n_pgroups,
                                int8_t* k2, uint8_t* k1, uint16_t* ks2, uint16_t* kz2, uint16_t* ks1, int8_t* trits,
                                uint16_t* vs, int8_t* v2, uint16_t* v2s, uint16_t* v2z, cudaStream_t stream);
cudaError_t launch_export_selection(const CacheView& cv, int layer, int n_chunks, uint8_t* dmask, int64_t T, int64_t T_sel,
                                    uint8_t* E, cudaStream_t stream);

}  // namespace vidkv
