// Key quantizer kernels: Algorithm 3 (MixQuant) of the paper.
//   k_range_kernel   per-channel min / max over the tokens of a chunk        (range)
//   k_select_kernel  top-64 channels by range -> D-mask / N-mask as id lists (TopK)
//   k_encode_kernel  2-bit GQuant (Eq. 4) on the anomalous channels and
//                    64-point real FFT + sign / mean-abs code (Eq. 5) on the rest
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

// ---------------------------------------------------------------------------------
// Range pass.  grid = (token splits, slabs); block = 256 threads = 16 rows x 16 lanes,
// each lane owns 8 consecutive channels (one 16-byte load per row).
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) k_range_kernel(KSrc src, int64_t T_tokens, int tokens_per_block,
                                                      uint32_t* __restrict__ minmax) {
  const int slab = blockIdx.y;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * tokens_per_block;
  const int64_t t1 = min(t0 + tokens_per_block, T_tokens);
  float mn[8], mx[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { mn[i] = INFINITY; mx[i] = -INFINITY; }
  for (int64_t t = t0 + row; t < t1; t += 16) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + t * src.stride_t) + lane16);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = Elem<T>::to_float2(w[i]);
      mn[2 * i] = fminf(mn[2 * i], f.x);      mx[2 * i] = fmaxf(mx[2 * i], f.x);
      mn[2 * i + 1] = fminf(mn[2 * i + 1], f.y); mx[2 * i + 1] = fmaxf(mx[2 * i + 1], f.y);
    }
  }
  __shared__ float s_mn[16][kD + 1], s_mx[16][kD + 1];
#pragma unroll
  for (int i = 0; i < 8; ++i) { s_mn[row][lane16 * 8 + i] = mn[i]; s_mx[row][lane16 * 8 + i] = mx[i]; }
  __syncthreads();
  if (threadIdx.x < kD) {
    float a = INFINITY, c = -INFINITY;
#pragma unroll
    for (int r = 0; r < 16; ++r) { a = fminf(a, s_mn[r][threadIdx.x]); c = fmaxf(c, s_mx[r][threadIdx.x]); }
    if (t0 < t1) {
      atomicMin(&minmax[slab * 2 * kD + threadIdx.x], float_ordered(a));
      atomicMax(&minmax[slab * 2 * kD + kD + threadIdx.x], float_ordered(c));
    }
  }
}

// ---------------------------------------------------------------------------------
// Channel selection.  One block of 128 threads per slab.  rank(c) = number of channels
// that come before c in (range descending, index ascending) order; the first 64 are
// the anomalous ones.  Writes the chunk-table entry: 64 anomalous ids ascending, then
// 64 normal ids ascending.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kD) k_select_kernel(const uint32_t* __restrict__ minmax, CacheView cv,
                                                      int layer0, int slabs_per_layer, int chunk) {
  const int slab = blockIdx.x;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  const int c = threadIdx.x;
  __shared__ float s_range[kD];
  __shared__ int s_abn[kD];
  const float mn = ordered_float(minmax[slab * 2 * kD + c]);
  const float mx = ordered_float(minmax[slab * 2 * kD + kD + c]);
  const float r = __fsub_rn(mx, mn);
  s_range[c] = r;
  __syncthreads();
  int rank = 0;
  for (int o = 0; o < kD; ++o) {
    const float ro = s_range[o];
    rank += (ro > r) || (ro == r && o < c);
  }
  const int is_abn = rank < kNA;
  s_abn[c] = is_abn;
  __syncthreads();
  int before = 0;
  for (int o = 0; o < c; ++o) before += s_abn[o];
  uint8_t* entry = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv) + cv.chunk_table_offset +
                   static_cast<int64_t>(chunk) * kChunkBytes;
  if (is_abn) entry[before] = static_cast<uint8_t>(c);
  else entry[kNA + (c - before)] = static_cast<uint8_t>(c);
}

// ---------------------------------------------------------------------------------
// 64-point real FFT in registers (one thread per token).
// z[n] = x[2n] + i x[2n+1]; Z = FFT32(z) by radix-2 decimation in frequency; then the
// usual split  X[k] = (Z[k] + conj Z[32-k]) / 2 - i e^{-2 pi i k / 64} (Z[k] - conj Z[32-k]) / 2.
// tw[m] = (cos, sin)(2 pi m / 64), m = 0..31, lives in shared memory.
// Output: the Hermitian half spectrum in storage order, scaled by 1/8 (orthonormal):
//   out[0] = Re X[0], out[1] = Re X[32], out[2k] = Re X[k], out[2k+1] = Im X[k].
// ---------------------------------------------------------------------------------
__device__ __forceinline__ constexpr int bitrev5(int v) {
  return ((v & 1) << 4) | ((v & 2) << 2) | (v & 4) | ((v & 8) >> 2) | ((v & 16) >> 4);
}

__device__ __forceinline__ void rfft64(float (&x)[64], const float2* __restrict__ tw) {
  // in place: x[2n] = Re z[n], x[2n+1] = Im z[n]
#pragma unroll
  for (int half = 16; half >= 1; half >>= 1) {         // 5 DIF stages, span = half
    const int step = 16 / half;                         // twiddle stride in units of 2 pi / 32
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      if ((i & half) == 0) {
        const int j = i + half;
        const int k = (i & (half - 1)) * step;          // exponent on W32
        const float ar = x[2 * i], ai = x[2 * i + 1], br = x[2 * j], bi = x[2 * j + 1];
        x[2 * i] = ar + br; x[2 * i + 1] = ai + bi;
        const float dr = ar - br, di = ai - bi;
        if (k == 0) { x[2 * j] = dr; x[2 * j + 1] = di; }
        else if (k == 8) { x[2 * j] = di; x[2 * j + 1] = -dr; }   // times -i
        else {
          const float2 w = tw[2 * k];                   // W32^k = e^{-2 pi i k / 32} = (cos, -sin)(2 pi 2k / 64)
          x[2 * j] = dr * w.x + di * w.y;
          x[2 * j + 1] = di * w.x - dr * w.y;
        }
      }
    }
  }
  // Z[k] sits at position bitrev5(k).  Split into the real-input spectrum.
  float out[64];
  {
    const float zr = x[0], zi = x[1];
    out[0] = (zr + zi) * 0.125f;                         // X[0]
    out[1] = (zr - zi) * 0.125f;                         // X[32]
  }
#pragma unroll
  for (int k = 1; k < 32; ++k) {
    const int p = bitrev5(k), q = bitrev5(32 - k);
    const float ar = x[2 * p], ai = x[2 * p + 1];        // Z[k]
    const float br = x[2 * q], bi = -x[2 * q + 1];       // conj Z[32-k]
    const float er = 0.5f * (ar + br), ei = 0.5f * (ai + bi);   // even part
    const float dr = 0.5f * (ar - br), di = 0.5f * (ai - bi);   // (Z[k] - conj Z[32-k]) / 2
    // odd part = -i * d ; times e^{-i th}, th = 2 pi k / 64: (-i d)(c - i s) = (di c - dr s) - i (dr c + di s)
    const float2 w = tw[k];
    const float orr = di * w.x - dr * w.y;
    const float oi = -(dr * w.x + di * w.y);
    out[2 * k] = (er + orr) * 0.125f;
    out[2 * k + 1] = (ei + oi) * 0.125f;
  }
#pragma unroll
  for (int i = 0; i < 64; ++i) x[i] = out[i];
}

// ---------------------------------------------------------------------------------
// Encode pass.  grid = (blocks of 128 tokens, slabs); block = 256 threads.
// The 128 x 128 tile is staged in shared memory as float (row stride 129).
// Warps 0-3: one thread per token, FFT of the 64 normal channels, sign bits, and the
//            per-group column means of |X| by a shuffle reduce-scatter.
// Warps 4-7: 2-bit GQuant of the 64 anomalous channels, 32-token groups.
// ---------------------------------------------------------------------------------
constexpr int kEncTokens = 128;
constexpr int kTileStride = kD + 1;

template <typename T>
__global__ void __launch_bounds__(256) k_encode_kernel(KSrc src, int64_t T_tokens, CacheView cv, int layer0,
                                                       int slabs_per_layer, int chunk, int64_t kgroup0) {
  extern __shared__ float smem[];
  float* tile = smem;                                       // [128][129]
  float2* tw = reinterpret_cast<float2*>(tile + kEncTokens * kTileStride);   // [32]
  uint16_t* s_s2 = reinterpret_cast<uint16_t*>(tw + 32);    // [4][64] binary16 bits
  uint16_t* s_z2 = s_s2 + 4 * kNA;                           // [4][64]
  uint8_t* s_perm = reinterpret_cast<uint8_t*>(s_z2 + 4 * kNA);   // [128]

  const int slab = blockIdx.y;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  const int b = bh / cv.H_kv, h = bh % cv.H_kv;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  uint8_t* slab_ptr = cv.slab(layer, b, h);
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * kEncTokens;
  const int n_tok = static_cast<int>(min(static_cast<int64_t>(kEncTokens), T_tokens - t0));   // multiple of 32
  const int n_groups = n_tok / kG;

  if (threadIdx.x < kD)
    s_perm[threadIdx.x] = slab_ptr[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + threadIdx.x];
  if (threadIdx.x < 32) {
    float sn, cs;
    sincospif(static_cast<float>(threadIdx.x) / 32.0f, &sn, &cs);   // angle 2 pi m / 64
    tw[threadIdx.x] = make_float2(cs, sn);
  }
  {
    const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
    for (int t = row; t < n_tok; t += 16) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (t0 + t) * src.stride_t) + lane16);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = Elem<T>::to_float2(w[i]);
        tile[t * kTileStride + lane16 * 8 + 2 * i] = f.x;
        tile[t * kTileStride + lane16 * 8 + 2 * i + 1] = f.y;
      }
    }
  }
  __syncthreads();

  uint8_t* kg_base = slab_ptr + cv.kgroup_offset + (kgroup0 + t0 / kG) * kKGroupBytes;

  if (threadIdx.x < 128) {
    // ---------------- FFT + 1-bit path: thread = token ----------------
    const int t = threadIdx.x, g = t >> 5, lane = t & 31;
    if (g < n_groups) {
      float x[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) x[i] = tile[t * kTileStride + s_perm[kNA + i]];
      rfft64(x, tw);
      uint32_t w0 = 0, w1 = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        w0 |= (x[i] >= 0.0f ? 1u : 0u) << i;
        w1 |= (x[32 + i] >= 0.0f ? 1u : 0u) << i;
      }
      uint8_t* kg = kg_base + g * kKGroupBytes;
      {
        // half-word r holds columns 16 r .. 16 r + 15, column e at bit 15 - e
        uint16_t* hw = reinterpret_cast<uint16_t*>(kg + kKG_Bits1);
        hw[k1_half_index(lane, 0)] = static_cast<uint16_t>(__brev(w0 & 0xffffu) >> 16);
        hw[k1_half_index(lane, 16)] = static_cast<uint16_t>(__brev(w0 >> 16) >> 16);
        hw[k1_half_index(lane, 32)] = static_cast<uint16_t>(__brev(w1 & 0xffffu) >> 16);
        hw[k1_half_index(lane, 48)] = static_cast<uint16_t>(__brev(w1 >> 16) >> 16);
      }
      // column sums of |x| over the 32 tokens (lanes): reduce-scatter by halves
#pragma unroll
      for (int i = 0; i < 64; ++i) x[i] = fabsf(x[i]);
#pragma unroll
      for (int width = 32; width >= 2; width >>= 1) {        // values held: 2*width -> width
        const int m = width >> 1;
        // lanes with bit m set keep the upper half, others the lower half
        const bool up = (lane & m) != 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i < width) {
            const float send = up ? x[i] : x[i + width];
            const float keep = up ? x[i + width] : x[i];
            x[i] = keep + __shfl_xor_sync(0xffffffffu, send, m);
          }
        }
      }
      // after widths 32,16,8,4,2 (masks 16,8,4,2,1) each lane holds 2 column sums: x[0], x[1].
      // Column index: bits chosen by the lane: col = 32*b16 + 16*b8 + 8*b4 + 4*b2 + 2*b1 + {0,1}
      const int col = ((lane & 16) ? 32 : 0) + ((lane & 8) ? 16 : 0) + ((lane & 4) ? 8 : 0) +
                      ((lane & 2) ? 4 : 0) + ((lane & 1) ? 2 : 0);
      uint16_t* s1 = reinterpret_cast<uint16_t*>(kg + kKG_S1);
      s1[col] = f2h_bits(x[0] * (1.0f / 32.0f));
      s1[col + 1] = f2h_bits(x[1] * (1.0f / 32.0f));
    }
  } else {
    // ---------------- 2-bit GQuant path ----------------
    const int u = threadIdx.x - 128;                          // 0..127
    // (a) statistics: (slot j, group g), two groups per thread
    for (int g = u >> 6; g < n_groups; g += 2) {
      const int j = u & 63;
      const int c = s_perm[j];
      float mn = INFINITY, mx = -INFINITY;
#pragma unroll 8
      for (int t = 0; t < kG; ++t) {
        const float v = tile[(g * kG + t) * kTileStride + c];
        mn = fminf(mn, v); mx = fmaxf(mx, v);
      }
      const uint16_t sh = f2h_bits(__fdiv_rn(__fsub_rn(mx, mn), 3.0f));
      const uint16_t zh = f2h_bits(mn);
      s_s2[g * kNA + j] = sh; s_z2[g * kNA + j] = zh;
      uint8_t* kg = kg_base + g * kKGroupBytes;
      reinterpret_cast<uint16_t*>(kg + kKG_S2)[j] = sh;
      reinterpret_cast<uint16_t*>(kg + kKG_Z2)[j] = zh;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    // (b) codes: item = (token, word); 16 slots per word
    for (int item = u; item < n_tok * 4; item += 128) {
      const int t = item >> 2, wi = item & 3, g = t >> 5;
      uint32_t word = 0;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int j = wi * 16 + i;
        const float s = h2f(s_s2[g * kNA + j]), z = h2f(s_z2[g * kNA + j]);
        const float v = tile[t * kTileStride + s_perm[j]];
        float q = rintf(__fdiv_rn(__fsub_rn(v, z), s));
        q = fminf(fmaxf(q, 0.0f), 3.0f);
        const uint32_t code = (s == 0.0f) ? 0u : static_cast<uint32_t>(q);
        word |= code << k2_bit(i);
      }
      uint8_t* kg = kg_base + g * kKGroupBytes;
      reinterpret_cast<uint32_t*>(kg + kKG_Codes2)[k2_word_index(t & 31, wi * 16)] = word;
    }
  }
}

// ---------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------
size_t k_encode_smem_bytes() {
  return kEncTokens * kTileStride * sizeof(float) + 32 * sizeof(float2) + 2 * 4 * kNA * sizeof(uint16_t) + kD;
}

template <typename T>
static cudaError_t launch_keys_t(const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_layers,
                                 int chunk, int64_t kgroup0, uint32_t* minmax, cudaStream_t stream) {
  const int slabs_per_layer = cv.B * cv.H_kv;
  const int n_slabs = slabs_per_layer * n_layers;
  if (T_tokens <= 0 || n_slabs <= 0) return cudaSuccess;
  cudaError_t e;
  // min array -> all ones (largest ordered key), max array -> zero, interleaved per slab
  if ((e = cudaMemsetAsync(minmax, 0, static_cast<size_t>(n_slabs) * 2 * kD * sizeof(uint32_t), stream))) return e;
  init_min_kernel<<<(n_slabs * kD + 255) / 256, 256, 0, stream>>>(minmax, n_slabs);
  int tokens_per_block = 512;
  const int64_t splits = (T_tokens + tokens_per_block - 1) / tokens_per_block;
  k_range_kernel<T><<<dim3(static_cast<unsigned>(splits), n_slabs), 256, 0, stream>>>(src, T_tokens, tokens_per_block,
                                                                                       minmax);
  k_select_kernel<<<n_slabs, kD, 0, stream>>>(minmax, cv, layer0, slabs_per_layer, chunk);
  static bool attr_set = false;
  const size_t smem = k_encode_smem_bytes();
  if (!attr_set) {
    if ((e = cudaFuncSetAttribute(k_encode_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    if ((e = cudaFuncSetAttribute(k_encode_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    attr_set = true;
  }
  const int64_t blocks = (T_tokens + kEncTokens - 1) / kEncTokens;
  k_encode_kernel<T><<<dim3(static_cast<unsigned>(blocks), n_slabs), 256, smem, stream>>>(
      src, T_tokens, cv, layer0, slabs_per_layer, chunk, kgroup0);
  count_launches(4);
  return cudaGetLastError();
}

__global__ void init_min_kernel(uint32_t* minmax, int n_slabs) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_slabs * kD) minmax[(i / kD) * 2 * kD + (i % kD)] = 0xffffffffu;
}

cudaError_t launch_quantize_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0,
                                 int n_layers, int chunk, int64_t kgroup0, uint32_t* minmax, cudaStream_t stream) {
  if (dtype == VIDKV_F16)
    return launch_keys_t<__half>(src, T_tokens, cv, layer0, n_layers, chunk, kgroup0, minmax, stream);
  return launch_keys_t<__nv_bfloat16>(src, T_tokens, cv, layer0, n_layers, chunk, kgroup0, minmax, stream);
}

}  // namespace vidkv
