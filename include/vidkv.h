/*
 * vidkv.h -- C ABI of libvidkv: the VidKV 1.x-bit KV-cache hot path on B200 (sm_100a).
 *
 * What the library computes (notation of the paper, arXiv 2503.16257):
 *   - keys    : MixQuant (Algorithm 3): per-chunk range-based channel split,
 *               2-bit GQuant (Eq. 4) on the anomalous half of the channels,
 *               FFT + 1-bit sign/mean-abs code (Eq. 5) on the normal half;
 *   - values  : 1.58Quant (Eq. 6, ternary, gamma) and STPQuant (Algorithm 2):
 *               the top n = floor(p * l_v) visual tokens by saliency (Eq. 7)
 *               are kept at 2 bits (Eq. 4), the rest ternary;
 *   - packing : codes, scales and zero points in one flat caller-owned buffer;
 *   - decode  : Algorithm 1 "Decoding" -- append the new token to the FP16
 *               residual, Softmax(q K^T / sqrt(D)) V over the packed cache plus
 *               the residual (Eq. 3) without materialising K or V, and the
 *               residual flush once it holds R = 128 tokens.
 *
 * Conventions
 *   - Every function returns a vidkv_status_t (0 = OK, negative = error); the
 *     library never throws, aborts or prints.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the
 *     argument is documented as a host pointer.  The library allocates no
 *     device memory: the caller asks vidkv_cache_bytes() for sizes, allocates,
 *     and passes the buffers in.  The handle is a small host object.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed
 *     as void*) and is asynchronous.  Argument errors are detected on the host
 *     before anything is launched.  No call synchronises the stream except
 *     vidkv_cache_status and vidkv_set_token_mask with n_protected == -1.  The first key
 *     quantization or decode call on each device fills the tables of DFT coefficients inside
 *     the library (56 KB) with one extra small kernel on the caller's stream and records an
 *     event that later calls make their streams wait for; make that first call outside any
 *     stream capture.
 *   - Fixed in this library: D = 128, G = 32, R = 128, H_q a multiple of H_kv with
 *     H_q / H_kv <= 8; k_ratio one of 0.25, 0.5, 0.75, 1 (32, 64, 96 or 128 two-bit key
 *     channels; Table 2's 1.25-, 1.5-, 1.75- and 2-bit key rows).  Other shapes return
 *     VIDKV_ERR_UNSUPPORTED.  k_ratio = 0.5 with VIDKV_KEY1BIT_FFT_SIGN (the default) has the
 *     key-group layout below and the fastest kernels; every other combination uses the
 *     general key-group layout described after it.
 *   - Element types: VIDKV_F16 / VIDKV_BF16 for K, V, q, k_new, v_new (in_dtype);
 *     VIDKV_F16 / VIDKV_BF16 / VIDKV_F32 for the attention output (out_dtype).
 *     Input values must be finite and representable in binary16.
 *   - One handle must not be used from two host threads at once, and calls on
 *     one handle must be issued on one stream (or on streams the caller orders).
 *     Different handles may be worked on from different streams at the same time.
 *     One exception on one handle: vidkv_quantize_keys and vidkv_quantize_values (and their _layers
 *     forms) write disjoint parts of the cache and workspace, so the values may be quantized on a
 *     second stream while the keys are, provided the token selection was enqueued before both and
 *     both streams are joined before the first decode call.
 *     The one-time set-up per device (tables, kernel attributes) is not guarded
 *     against concurrent host threads: make the first call on a device from one thread.
 *
 * Packed cache layout (little endian; all offsets are given by vidkv_layout_t)
 *   per slab = (layer, batch element, KV head):
 *     chunk table  : per chunk 128 bytes: 64 ascending anomalous channel ids,
 *                    then 64 ascending normal channel ids (uint8).  Chunk 0 is
 *                    the prefill; every residual flush appends a 128-token chunk.
 *     key groups   : per 32 tokens 1152 bytes (token t = 8 nt + tl of the group):
 *                    [0,512)    2-bit codes as 128 32-bit words: anomalous slot
 *                               j = 16 r + e of token t is in word ((4 tl + r) * 4 + nt)
 *                               at bits 2 (e / 2) + 16 (e % 2)  (even slots in the low
 *                               half-word, odd slots in the high one);
 *                    [512,768)  1-bit codes as 128 16-bit half-words: spectrum column
 *                               f = 16 r + e of token t is in half-word ((4 tl + r) * 4 + nt)
 *                               at bit 15 - e (1 = coefficient >= 0);
 *                    [768,896)  s  (binary16) of the 64 two-bit slots;
 *                    [896,1024) z  (binary16) of the 64 two-bit slots;
 *                    [1024,1152) s (binary16) of the 64 spectrum columns.
 *                    Spectrum columns of the orthonormal 64-point DFT of the
 *                    normal channels (ascending channel order), Hermitian half:
 *                    column 0 = Re X[0], 1 = Re X[32], 2k = Re X[k],
 *                    2k+1 = Im X[k] for k = 1..31.
 *     ternary supergroups : per 5 groups (160 stream tokens) 5376 bytes:
 *                    [0,4096)   one byte per (token j of the group, channel c), holding the
 *                               trits of channel c at token j of each of the 5 groups:
 *                               digit d_g = trit + 1, b = sum_g d_g * 3^(4-g),
 *                               stored byte = (256*b + 242) / 243.  With j = 2 m + parity,
 *                               m = 8 kt + 4 u + r and c = 32 w + 4 rho + e the byte is at
 *                               ((((kt*2 + u)*4 + w)*4 + r)*8 + rho)*8 + 2 e + parity;
 *                    [4096,5376) s (binary16) [5][128].
 *     protected groups (STP) : per 32 protected tokens 1536 bytes:
 *                    [0,1024) 2-bit codes as 256 32-bit words: with token
 *                    j = 16 kt + 8 u + 2 r + hf of the group and channel c = 32 w + 4 rho + e
 *                    the code is in word ((kt*4 + w)*4 + r)*8 + rho at bits
 *                    2 (4 u + e) + 16 hf; [1024,1280) s; [1280,1536) z.
 *     residual     : K_r and V_r, 128 x 128 elements each, in in_dtype.
 *   per batch element: the protection mask E as bit words plus, per word, the
 *   number of protected tokens before it.
 *
 * General key-group layout (every k_ratio / key_1bit_mode other than the default), with n2 two-bit
 * slots and n1 = 128 - n2 one-bit columns, both taken in blocks of 32:
 *     chunk table  : per chunk 128 bytes: n2 ascending anomalous channel ids, then the n1 normal ones.
 *     key groups   : per 32 tokens 8 n2 + 4 n1 + 4 n2 + 2 n1 (Eq. 5) or 4 n1 (plain) bytes
 *                    (token t = 8 nt + tl; lane = 4 tl + r, r = (index within the block) / 8):
 *                    2-bit codes : block b of 32 slots is 256 bytes; byte b * 256 + lane * 8 + nt * 2 + par
 *                               holds the slots 32 b + 8 r + e with e % 2 == par of token t, slot e at
 *                               bits 2 (e / 2);
 *                    1-bit codes : block b of 32 columns is 128 bytes; byte b * 128 + lane * 4 + nt holds
 *                               the columns 32 b + 8 r + e of token t, column e at bit 7 - e;
 *                    then s (binary16) [n2], z (binary16) [n2] of the two-bit slots;
 *                    then s (binary16) [n1] of the one-bit columns -- Eq. 5: columns of the orthonormal
 *                    n1-point DFT of the normal channels in the Hermitian order given above (column 1 =
 *                    Re X[n1 / 2]); plain mode: the normal channels in ascending order, code 0 / 1 with
 *                    value code * s + z -- and, in plain mode only, their z (binary16) [n1].
 */
#ifndef VIDKV_H_
#define VIDKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t vidkv_status_t;

enum {
  VIDKV_OK = 0,
  VIDKV_ERR_INVALID_ARG = -1,   /* null pointer, negative size, bad enum value, p outside [0,1] ... */
  VIDKV_ERR_UNSUPPORTED = -2,   /* a shape or mode this library does not implement */
  VIDKV_ERR_ALIGNMENT = -3,     /* a pointer or stride that is not 16-byte aligned */
  VIDKV_ERR_CAPACITY = -4,      /* more tokens than the cache was sized for, buffer too small */
  VIDKV_ERR_STATE = -5,         /* call order: decode before quantize, quantize twice, ... */
  VIDKV_ERR_CUDA = -6,          /* a CUDA runtime call or launch failed */
  VIDKV_ERR_TIMEOUT = -7        /* a bounded device-side wait ran out (reported via vidkv_cache_status) */
};

enum { VIDKV_F16 = 0, VIDKV_BF16 = 1, VIDKV_F32 = 2 };
/* Algorithm 3, 1BitQuant: how the normal (1-bit) key channels are coded.
 *   VIDKV_KEY1BIT_FFT_SIGN      Eq. 5: orthonormal DFT over the normal channels of a token, then sign bit and
 *                               per-(group, column) mean magnitude; k_ratio 0.5 or 0.75 (as in Sec. 4.1)
 *   VIDKV_KEY1BIT_PLAIN_MINMAX  the other branch: Eq. 4 with n = 1 on the channels as they are (levels
 *                               min and max of the group); k_ratio 0.25, 0.5 or 0.75
 * With k_ratio = 1 every channel is 2-bit and the mode has no effect. */
enum { VIDKV_KEY1BIT_FFT_SIGN = 0, VIDKV_KEY1BIT_PLAIN_MINMAX = 1 };
/* Channel metrics of Sec. 4.1(1) other than the range (which the method uses and computes itself). */
enum { VIDKV_METRIC_VARIANCE = 1, VIDKV_METRIC_OUTLIERS = 2 };
/* Scale stored with the ternary codes of Eq. 6 (the paper gives the codes only): the Mean |v|
 * that also sets the threshold, or the mean of |v| over the elements whose code is not 0
 * (the least-squares scale for those codes, as in ternary weight networks; 0 where every
 * code is 0).  The codes are the same in both modes. */
enum { VIDKV_TERNARY_SCALE_MEAN_ABS = 0, VIDKV_TERNARY_SCALE_NONZERO_MEAN = 1 };

/* Problem description (Algorithm 1 parameters G, R, p, k; Algorithm 2 gamma). */
typedef struct {
  int32_t B;                  /* batch elements */
  int32_t L;                  /* layers held by this cache */
  int32_t H_kv;               /* KV heads */
  int32_t H_q;                /* query heads (GQA: head h_q reads KV head h_q / (H_q/H_kv)) */
  int32_t D;                  /* head dimension (128) */
  int32_t G;                  /* group size (32) */
  int32_t R;                  /* residual length (128) */
  float k_ratio;              /* fraction of key channels kept at 2 bits: 0.25, 0.5 (default), 0.75 or 1 */
  float p_ratio;              /* fraction of visual tokens protected at 2 bits, in [0, 1] */
  float gamma;                /* ternary threshold factor (0.7) */
  int32_t in_dtype;           /* VIDKV_F16 | VIDKV_BF16 */
  int32_t out_dtype;          /* VIDKV_F16 | VIDKV_BF16 | VIDKV_F32 */
  int32_t key_1bit_mode;      /* VIDKV_KEY1BIT_FFT_SIGN | VIDKV_KEY1BIT_PLAIN_MINMAX */
  int32_t ternary_scale;      /* VIDKV_TERNARY_SCALE_MEAN_ABS (default) | VIDKV_TERNARY_SCALE_NONZERO_MEAN */
  int64_t max_prefill_tokens; /* largest T passed to vidkv_quantize_* */
  int64_t max_new_tokens;     /* decode steps the cache must be able to absorb */
} vidkv_config_t;

/* Byte offsets and strides of the packed cache (host struct; filled by vidkv_cache_layout). */
typedef struct {
  int64_t header_bytes;
  int64_t sel_offset;         /* start of the per-batch token-selection region */
  int64_t sel_stride_b;       /* bytes per batch element: E words, then prefix words */
  int64_t sel_words;          /* 32-bit words per batch element in each of the two arrays */
  int64_t slab_offset;        /* start of slab 0 */
  int64_t slab_stride;        /* bytes per slab; slab index = (layer*B + b)*H_kv + h */
  int64_t chunk_table_offset; /* within a slab */
  int64_t max_chunks;
  int64_t kgroup_offset;      /* within a slab */
  int64_t max_kgroups;
  int64_t tern_offset;        /* within a slab */
  int64_t max_supergroups;
  int64_t prot_offset;        /* within a slab */
  int64_t max_pgroups;
  int64_t kres_offset;        /* within a slab */
  int64_t vres_offset;        /* within a slab */
  int64_t total_bytes;
} vidkv_layout_t;

typedef struct vidkv_cache vidkv_cache_t;

/* Sizes (host only).  cache_bytes / workspace_bytes are what vidkv_cache_init wants.
 * The workspace holds partial attention results, prepared queries, channel ranges and
 * the gather lists of the token selection.  Between calls it carries the gather lists,
 * which vidkv_quantize_values reads, and the armed channel-range accumulators that
 * vidkv_cache_init sets up: it belongs to one handle and must not be overwritten while
 * that handle is in use. */
vidkv_status_t vidkv_cache_bytes(const vidkv_config_t* cfg, size_t* cache_bytes, size_t* workspace_bytes);

/* Offsets of every region of the packed cache for this configuration (host only). */
vidkv_status_t vidkv_cache_layout(const vidkv_config_t* cfg, vidkv_layout_t* layout);

/* Create a handle over caller-owned device buffers (256-byte aligned) and zero the
 * cache on `stream`.  The handle stays valid until vidkv_cache_destroy; the buffers
 * must outlive it.  Returns CAPACITY if a buffer is smaller than vidkv_cache_bytes says. */
vidkv_status_t vidkv_cache_init(const vidkv_config_t* cfg, void* cache, size_t cache_bytes,
                                void* workspace, size_t workspace_bytes, void* stream,
                                vidkv_cache_t** handle);
vidkv_status_t vidkv_cache_destroy(vidkv_cache_t* handle);

/* Forget all tokens (host state only; the next quantize calls overwrite the buffers). */
vidkv_status_t vidkv_cache_reset(vidkv_cache_t* handle, void* stream);

/* Sec. 3.3(2) / Eq. 7: the cross-modal scores I = X_v X_t^T from hidden states, summed over
 * the text tokens (the paper does not say how the text axis is reduced; a sum and a mean
 * rank alike):  saliency[b, i] = sum_j x_v[b, i, :] . x_t[b, j, :]  in float32.
 *   x_v      [B, l_v, d]  device, dtype VIDKV_F16 or VIDKV_BF16, contiguous
 *   x_t      [B, l_t, d]  device, same dtype, contiguous (l_t == 0: all scores are 0)
 *   text_sum [B, d]       device float32 scratch owned by the caller, overwritten
 *   saliency [B, l_v]     device float32, written; feed it to vidkv_select_tokens
 * d must be a multiple of 8 and at most 16384, B at most 65535 (else UNSUPPORTED); all
 * pointers 16-byte aligned.  Needs no cache handle.  Two launches on `stream`. */
vidkv_status_t vidkv_saliency_scores(int32_t dtype, const void* x_v, const void* x_t, int64_t B, int64_t l_v,
                                     int64_t l_t, int64_t d, float* text_sum, float* saliency, void* stream);

/* Sec. 4.1(1): the channel metrics the paper compares the range against, per (batch element,
 * head, channel) of a key tensor K [B, H, T, 128] (dtype VIDKV_F16 / VIDKV_BF16, element
 * strides as for vidkv_quantize_keys, T >= 1):
 *   VIDKV_METRIC_VARIANCE  population variance of the channel over the T tokens
 *   VIDKV_METRIC_OUTLIERS  number of tokens with |K_i| > M * mean_i |K_i|  (the paper sets M = 3
 *                          and writes the comparison without magnitudes; magnitudes are taken
 *                          here, or zero-centred channels would always count about T / 2)
 * out [B, H, 128] float32 device; scratch [B, H, 2, 128] float64 device, caller-owned,
 * overwritten.  Accumulation is in float64.  The cache is not involved: MixQuant's own channel
 * split stays range-based.  Three or four launches and one memset on `stream`. */
vidkv_status_t vidkv_channel_metrics(int32_t dtype, const void* K, int64_t B, int64_t H, int64_t T, int64_t stride_b,
                                     int64_t stride_h, int64_t stride_t, int32_t metric, float M, double* scratch,
                                     float* out, void* stream);

/* Sec. 3.3(2) / Eq. 7: choose the protected tokens.  saliency [B, l_v] float32 scores
 * the visual tokens vis_begin .. vis_begin + l_v - 1 of a prompt of T tokens; the top
 * n = floor(p_ratio * l_v) (ties: lower token index) are protected in every layer and
 * head.  Must precede vidkv_quantize_values when p_ratio > 0; with p_ratio == 0 or
 * saliency == NULL no token is protected.  Only tokens below T - T % G can be
 * protected (the rest stay FP16 in the residual). */
vidkv_status_t vidkv_select_tokens(vidkv_cache_t* handle, const float* saliency, int64_t vis_begin,
                                   int64_t l_v, int64_t T, void* stream);

/* Algorithm 2 takes the mask E as a parameter: the same, from a ready mask
 * E [B, T] (uint8, nonzero = protected; every batch element must protect the same
 * number of tokens, all below T - T % G).  n_protected >= 0 states that number: the call is
 * then asynchronous like the others, and a row of E that protects a different number sets
 * VIDKV_ERR_INVALID_ARG in the cache's status word (vidkv_cache_status).  n_protected == -1
 * lets the library count: it then reads the counts back and synchronises the stream once. */
vidkv_status_t vidkv_set_token_mask(vidkv_cache_t* handle, const uint8_t* E, int64_t T, int64_t n_protected,
                                    void* stream);

/* Algorithm 1 "Prefill", key half, for one layer: K [B, H_kv, T, D] (in_dtype) with
 * element strides stride_b / stride_h / stride_t (channel stride 1; strides multiples
 * of 8 elements).  The first T - T % G tokens are MixQuant-ed (Algorithm 3) into chunk
 * 0; the last T % G tokens are copied to the FP16 residual.  Once per layer per reset. */
vidkv_status_t vidkv_quantize_keys(vidkv_cache_t* handle, int32_t layer, const void* K, int64_t T,
                                   int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream);

/* Algorithm 1 "Prefill", value half: STPQuant (Algorithm 2) when tokens were selected,
 * else 1.58Quant (Eq. 6).  Same argument meaning as vidkv_quantize_keys; T must equal
 * the T given for the keys of this layer if those came first. */
vidkv_status_t vidkv_quantize_values(vidkv_cache_t* handle, int32_t layer, const void* V, int64_t T,
                                     int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream);

/* The same for n_layers consecutive layers in one call (fewer launches where a layer's tensors are
 * small): K / V [n_layers, B, H_kv, T, D] with the layers stride_b * B elements apart, i.e.
 * source slab (layer, b, h) starts at ((layer - layer_begin) * B + b) * stride_b + h * stride_h.
 * Every layer gets its own channel split and scales, exactly as with one call per layer. */
vidkv_status_t vidkv_quantize_keys_layers(vidkv_cache_t* handle, int32_t layer_begin, int32_t n_layers, const void* K,
                                          int64_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream);
vidkv_status_t vidkv_quantize_values_layers(vidkv_cache_t* handle, int32_t layer_begin, int32_t n_layers, const void* V,
                                            int64_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t, void* stream);

/* Algorithm 1 "Decoding" for n_layers independent layers in one call:
 *   q      [n_layers, B, H_q,  D]  (in_dtype)
 *   k_new  [n_layers, B, H_kv, D]  (in_dtype)    appended to the residual first
 *   v_new  [n_layers, B, H_kv, D]  (in_dtype)
 *   out    [n_layers, B, H_q,  D]  (out_dtype)   Softmax(q K^T * softmax_scale) V
 * softmax_scale <= 0 selects 1 / sqrt(D).  When a layer's residual reaches R tokens it
 * is quantized into a new 128-token chunk (own channel split; values by 1.58Quant) and
 * emptied.  All contiguous.  Returns CAPACITY when max_new_tokens would be exceeded.
 * Range: every query head is normalised by a power of two before it meets the stored
 * binary16 scales, so finite inputs give finite outputs as long as the Eq. 5 scales of the
 * spectrum stay below 16376 (normal-channel keys of magnitude up to a few thousand); the
 * Eq. 4 scales may take any binary16 value, and a bfloat16 query may exceed the binary16
 * range. */
vidkv_status_t vidkv_decode_attention(vidkv_cache_t* handle, int32_t layer_begin, int32_t n_layers,
                                      const void* q, const void* k_new, const void* v_new, void* out,
                                      float softmax_scale, void* stream);

/* Caches beyond one device (the 1000-frame case of Sec. 1): the token axis of Eq. 3 can be cut into
 * shards, each held by its own cache (its own device), because Softmax(q K^T) V over the whole
 * sequence follows from per-shard (maximum, sum, unnormalised output) triples.
 * vidkv_decode_attention_partial is vidkv_decode_attention for one shard:
 *   partial [n_layers, B, H_q, 130] float32 device: per query head the largest base-2 logit
 *           m = max_t (q . k_t) * softmax_scale * log2(e), l = sum_t 2^(logit_t - m) and
 *           o[128] = sum_t 2^(logit_t - m) v_t over the shard's tokens (packed cache + residual);
 *   k_new, v_new: the shard that owns the newest token passes them (appended first, residual
 *           flushed when full, exactly as in vidkv_decode_attention); the other shards pass NULL
 *           for both and are attended to as they stand (STATE if such a shard holds no token).
 * The caller moves the triples between devices (e.g. an all-gather of 130 floats per query head
 * and shard into its own memory) and vidkv_merge_partials combines them:
 *   partials [n_parts, n_rows, 130] float32 device, n_rows = n_layers * B * H_q;
 *   out [n_rows, 128] in out_dtype:  sum_p 2^(m_p - M) o_p / sum_p 2^(m_p - M) l_p, M = max_p m_p.
 * Every shard quantizes its own tokens (its own chunks and channel splits, Algorithm 3 applied to
 * the tokens it holds). */
vidkv_status_t vidkv_decode_attention_partial(vidkv_cache_t* handle, int32_t layer_begin, int32_t n_layers,
                                              const void* q, const void* k_new, const void* v_new, float* partial,
                                              float softmax_scale, void* stream);
vidkv_status_t vidkv_merge_partials(const float* partials, int64_t n_parts, int64_t n_rows, void* out,
                                    int32_t out_dtype, void* stream);

/* Host view of a layer's token counts (any pointer may be NULL). */
vidkv_status_t vidkv_layer_state(const vidkv_cache_t* handle, int32_t layer, int64_t* n_quantized,
                                 int64_t* n_residual, int64_t* n_chunks, int64_t* n_protected);

/* Device status word of the cache (synchronises `stream`): VIDKV_OK or the first
 * device-detected error. */
vidkv_status_t vidkv_cache_status(vidkv_cache_t* handle, void* stream);

/* Test and inspection only (never on the decode path): dequantize the quantized part of
 * one layer to float32, out [B, H_kv, n_quantized, D] contiguous.  DeQuant of Algorithm 1. */
vidkv_status_t vidkv_dequantize_keys(vidkv_cache_t* handle, int32_t layer, float* out, void* stream);
vidkv_status_t vidkv_dequantize_values(vidkv_cache_t* handle, int32_t layer, float* out, void* stream);

/* Test and inspection only: the packed codes and metadata of one layer as plain arrays, one
 * element per code, so that a test need not know the bit layout (Eq. 4, Eq. 5, Eq. 6 codes as
 * Algorithm 1 stores them).  With ng = n_quantized / 32 key groups, nt ternary stream groups
 * (ceil((n_prefill_quantized - n_protected) / 32) + 4 per flush) and np = ceil(n_protected / 32)
 * protected groups, per slab = (b, h) of the layer, all device pointers, any of them may be NULL
 * (n2 = 128 k_ratio two-bit channels, n1 = 128 - n2; 64 and 64 by default):
 *   k2      int8  [B, H_kv, 32 ng, n2]   Eq. 4 codes 0..3 of the 2-bit channels, slot order
 *                                        (slot j = j-th channel of the chunk's ascending 2-bit list)
 *   k1bits  uint8 [B, H_kv, 32 ng, n1]   Eq. 5 bits of the spectrum columns (column order of the layout),
 *                                        or the plain 1-bit codes of the normal channels (ascending)
 *   k_s2, k_z2  binary16 [B, H_kv, ng, n2]
 *   k_s1    binary16 [B, H_kv, ng, n1]; in plain min/max mode [B, H_kv, ng, 2, n1]: scales, then zero points
 *   v_trits int8  [B, H_kv, 32 nt, 128]  Eq. 6 codes -1, 0, +1 in ternary stream order
 *   v_s     binary16 [B, H_kv, nt, 128]
 *   v2      int8  [B, H_kv, 32 np, 128]  Eq. 4 codes of the protected tokens, stream order
 *   v2_s, v2_z        binary16 [B, H_kv, np, 128]
 * Positions past the end of a stream hold whatever the cache holds there (zeros after init). */
vidkv_status_t vidkv_export_codes(vidkv_cache_t* handle, int32_t layer, int8_t* k2, uint8_t* k1bits, void* k_s2,
                                  void* k_z2, void* k_s1, int8_t* v_trits, void* v_s, int8_t* v2, void* v2_s,
                                  void* v2_z, void* stream);

/* Test and inspection only: the selections of Algorithm 3 and Algorithm 2 as byte masks.
 *   dmask uint8 [B, H_kv, 1 + flushes, 128]  1 = 2-bit (anomalous) channel of that chunk (D-mask);
 *                                            chunk 0 is the prefill, all zero if it is empty
 *   E     uint8 [B, T]                       1 = protected token (T = the prompt length given at prefill)
 * Either pointer may be NULL. */
vidkv_status_t vidkv_get_selection(vidkv_cache_t* handle, int32_t layer, uint8_t* dmask, uint8_t* E, void* stream);

/* For callers that cannot obtain device memory.  (The paper has no counterpart to this
 * entry point; it exists for deployment reasons only.)  Some callers are handed their
 * device tensors by a host framework and cannot allocate more where attention runs -- a
 * plugin restricted to the buffers it was given, code running while the framework's memory
 * pool is frozen, a runtime without cudaMalloc -- so they cannot supply the workspace that
 * vidkv_cache_init wants.  This call needs no handle and no workspace: it computes
 *   out [n_layers, B, H_q, D] (out_dtype) = Softmax(q K^T * softmax_scale) V
 * for q [n_layers, B, H_q, D] (in_dtype) over the packed cache `cache` exactly as it stands
 * (no append, no flush), the cache having been filled through a handle built on the same
 * `cfg`.  The caller states the token counts that vidkv_layer_state reports for the layers:
 * n_prefill_quantized (a multiple of G), n_flushed_chunks, n_residual (0..R) and n_protected.
 * The scratch for partial results lives in a 16 MiB array inside the library, which every GPU
 * that loads the library keeps until the process exits.  It must hold 520 bytes per (query
 * head, partial record) -- about 8 * (warps resident on the device + 2 * n_layers * B * H_kv)
 * records at most -- plus 3200 bytes per (layer, batch element, KV head, chunk); larger
 * problems return VIDKV_ERR_CAPACITY (use fewer layers per call).
 * Nothing is allocated or freed.  The first call on each device looks up the array's device
 * address, so make that first call outside any stream capture.  All calls share the array:
 * two calls whose kernels may overlap on the GPU (different streams, no ordering) race on it;
 * calls ordered on one stream are fine, and nothing needs clearing between calls.
 * Errors as elsewhere: INVALID_ARG, UNSUPPORTED, ALIGNMENT (cache 256-byte, q/out 16-byte
 * aligned), CAPACITY, STATE (no tokens at all), CUDA. */
vidkv_status_t vidkv_attend_noalloc(const vidkv_config_t* cfg, const void* cache, int64_t n_prefill_quantized,
                                    int64_t n_flushed_chunks, int32_t n_residual, int64_t n_protected,
                                    int32_t layer_begin, int32_t n_layers, const void* q, void* out,
                                    float softmax_scale, void* stream);

/* Test hooks (no counterpart in the paper; the results of a decode call do not depend on them
 * beyond floating-point summation order).  Algorithm 1 "Decoding" leaves the evaluation order of
 * Eq. 3 open; the library cuts a decode call into work like this: the quantized tokens of all
 * slabs of the call form one sequence of 160-token units, and every warp of the launch walks a
 * run of `run_units` consecutive units (crossing slab boundaries where its run does) and leaves
 * one partial result per slab it touches.
 * vidkv_debug_set_decode_plan forces run_units (>= 1) for later vidkv_decode_attention calls on
 * this handle; 0 leaves the choice to the library.  A forced plan that needs more partial records
 * than the workspace holds makes the decode call return VIDKV_ERR_CAPACITY.
 * vidkv_debug_decode_plan (host only) reports the plan for given token counts on a device with
 * sm_count multiprocessors: plan_out[8] = { units per slab, run_units, runs (= warps),
 * records per slab, records needed, records the workspace of `cfg` holds, chunk-table entries,
 * units in all }. */
vidkv_status_t vidkv_debug_set_decode_plan(vidkv_cache_t* handle, int32_t run_units);
vidkv_status_t vidkv_debug_decode_plan(const vidkv_config_t* cfg, int64_t n_prefill_quantized, int64_t n_flushed_chunks,
                                       int32_t n_residual, int64_t n_protected, int32_t n_layers, int32_t sm_count,
                                       int32_t run_units, int64_t* plan_out);

/* Test hook for the two bounded device-side waits (no counterpart in the paper).  The key encoder
 * waits on the barrier its tensor-core products commit to, the stream kernel of the decode call
 * on the barriers of its bulk copies; both waits give up after a fixed number of polls, record
 * VIDKV_ERR_TIMEOUT in the cache's status word and leave in order (copies drained, tensor memory
 * freed).  what = 1 makes the next key quantization withhold the products of every block's first
 * tile, what = 2 makes the next decode call (on a cache without protected tokens) withhold every warp's first
 * value copy, so that the waits run out with nothing outstanding; the affected call's results
 * are garbage by design, the flag clears itself, and later calls are normal.  0 switches it off. */
vidkv_status_t vidkv_debug_withhold_once(int32_t what);

/* Profiling aid: record the two CUDA events (cudaEvent_t passed as void*) immediately before
 * and after the attention kernel (the stream kernel) of every later vidkv_decode_attention call on this
 * handle; NULL, NULL switches it off.  The events are the caller's. */
vidkv_status_t vidkv_set_profile_events(vidkv_cache_t* handle, void* ev_begin, void* ev_end);

/* Number of CUDA kernels this library has launched in this process (host counter). */
uint64_t vidkv_launch_count(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int32_t vidkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* VIDKV_H_ */
