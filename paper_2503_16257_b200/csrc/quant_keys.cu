// Key quantizer kernels: Algorithm 3 (MixQuant) of the paper.
//   k_range_kernel   per-channel min / max over the tokens of a chunk        (range)
//   k_select_kernel  top-64 channels by range -> D-mask / N-mask as id lists (TopK)
// The encode pass (Eq. 4 on the anomalous channels, DFT + sign / mean-abs code of Eq. 5 on
// the rest) lives in quant_keys_enc.cu.
#include <type_traits>

#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

// ---------------------------------------------------------------------------------
// Range pass.  grid = (token splits, slabs); block = 256 threads = 16 rows x 16 lanes,
// each lane owns 8 consecutive channels (one 16-byte load per row).
// ---------------------------------------------------------------------------------
template <typename T> struct Pair2;
template <> struct Pair2<__half> {
  using V = __half2;
  static __device__ __forceinline__ V mn(V a, V b) { return __hmin2(a, b); }
  static __device__ __forceinline__ V mx(V a, V b) { return __hmax2(a, b); }
  static __device__ __forceinline__ float2 f2(V a) { return __half22float2(a); }
};
template <> struct Pair2<__nv_bfloat16> {
  using V = __nv_bfloat162;
  static __device__ __forceinline__ V mn(V a, V b) { return __hmin2(a, b); }
  static __device__ __forceinline__ V mx(V a, V b) { return __hmax2(a, b); }
  static __device__ __forceinline__ float2 f2(V a) { return __bfloat1622float2(a); }
};

template <typename T>
__global__ void __launch_bounds__(256) k_range_kernel(KSrc src, int64_t T_tokens, int tokens_per_block,
                                                      uint32_t* __restrict__ minmax) {
  using P = Pair2<T>;
  using V = typename P::V;
  const int slab = blockIdx.y;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * tokens_per_block;
  const int64_t t1 = min(t0 + tokens_per_block, T_tokens);
  // element pairs stay in their 16-bit type: min / max need no conversion
  V mn[4], mx[4];
  bool any = false;
  int64_t t = t0 + row;
  if (t < t1) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + t * src.stride_t) + lane16);
    const V* pv = reinterpret_cast<const V*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { mn[i] = pv[i]; mx[i] = pv[i]; }
    any = true;
    t += 16;
  }
  for (; t + 48 < t1; t += 64) {                       // four rows in flight per thread
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = __ldg(reinterpret_cast<const uint4*>(base + (t + 16 * k) * src.stride_t) + lane16);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const V* pv = reinterpret_cast<const V*>(&v[k]);
#pragma unroll
      for (int i = 0; i < 4; ++i) { mn[i] = P::mn(mn[i], pv[i]); mx[i] = P::mx(mx[i], pv[i]); }
    }
  }
  for (; t < t1; t += 16) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + t * src.stride_t) + lane16);
    const V* pv = reinterpret_cast<const V*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { mn[i] = P::mn(mn[i], pv[i]); mx[i] = P::mx(mx[i], pv[i]); }
  }
  __shared__ float s_mn[16][kD + 1], s_mx[16][kD + 1];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 a = make_float2(INFINITY, INFINITY), c = make_float2(-INFINITY, -INFINITY);
    if (any) { a = P::f2(mn[i]); c = P::f2(mx[i]); }
    s_mn[row][lane16 * 8 + 2 * i] = a.x; s_mn[row][lane16 * 8 + 2 * i + 1] = a.y;
    s_mx[row][lane16 * 8 + 2 * i] = c.x; s_mx[row][lane16 * 8 + 2 * i + 1] = c.y;
  }
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
                                                      int layer0, int slabs_per_layer, int chunk,
                                                      uint32_t* __restrict__ rearm, int rearm_words) {
  // Re-arm the buffer the next call accumulates into (min half all ones, max half zero).  Nobody
  // reads it now: its last readers ran before this call's range pass in stream order.
  for (int i = blockIdx.x * kD + threadIdx.x; i < rearm_words; i += gridDim.x * kD)
    rearm[i] = (i & (2 * kD - 1)) < kD ? 0xffffffffu : 0u;
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
  const int n2 = cv.kf.n2;                 // Algorithm 3: D-mask = the top k D channels by range
  const int is_abn = rank < n2;
  s_abn[c] = is_abn;
  __syncthreads();
  int before = 0;
  for (int o = 0; o < c; ++o) before += s_abn[o];
  uint8_t* entry = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv) + cv.chunk_table_offset +
                   static_cast<int64_t>(chunk) * kChunkBytes;
  if (is_abn) entry[before] = static_cast<uint8_t>(c);
  else entry[n2 + (c - before)] = static_cast<uint8_t>(c);
}

// ---------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------
template <typename T>
static cudaError_t launch_keys_t(const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_layers,
                                 int chunk, int64_t kgroup0, const MinMaxBuffers& mm, cudaStream_t stream) {
  uint32_t* minmax = mm.cur;
  const int slabs_per_layer = cv.B * cv.H_kv;
  const int n_slabs = slabs_per_layer * n_layers;
  if (T_tokens <= 0 || n_slabs <= 0) return cudaSuccess;
  cudaError_t e;
  int tokens_per_block = 512;
  const int64_t splits = (T_tokens + tokens_per_block - 1) / tokens_per_block;
  k_range_kernel<T><<<dim3(static_cast<unsigned>(splits), n_slabs), 256, 0, stream>>>(src, T_tokens, tokens_per_block,
                                                                                       minmax);
  k_select_kernel<<<n_slabs, kD, 0, stream>>>(minmax, cv, layer0, slabs_per_layer, chunk, mm.next, mm.next_dirty_words);
  const int dt = std::is_same<T, __half>::value ? VIDKV_F16 : VIDKV_BF16;
  if ((e = cv.kf.general ? launch_encode_keys_general(dt, src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream)
                         : launch_encode_keys(dt, src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream)))
    return e;
  count_launches(2);
  return cudaGetLastError();
}

__global__ void init_min_kernel(uint32_t* minmax, int n_words, uint32_t* header, uint32_t version) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_words) minmax[i] = (i & (2 * kD - 1)) < kD ? 0xffffffffu : 0u;
  if (header && i == 0) { header[0] = kMagic; header[1] = version; header[2] = 0u; }
}

cudaError_t launch_init_minmax(uint32_t* minmax, int64_t n_words, uint32_t* header, uint32_t version, cudaStream_t stream) {
  init_min_kernel<<<static_cast<unsigned>((n_words + 255) / 256), 256, 0, stream>>>(minmax, static_cast<int>(n_words), header, version);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_quantize_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0,
                                 int n_layers, int chunk, int64_t kgroup0, const MinMaxBuffers& mm, cudaStream_t stream) {
  if (dtype == VIDKV_F16)
    return launch_keys_t<__half>(src, T_tokens, cv, layer0, n_layers, chunk, kgroup0, mm, stream);
  return launch_keys_t<__nv_bfloat16>(src, T_tokens, cv, layer0, n_layers, chunk, kgroup0, mm, stream);
}

}  // namespace vidkv
