// Cross-modal scores of Sec. 3.3(2) / Eq. 7 from hidden states: I = X_v X_t^T, reduced over the
// text tokens by summation, i.e. saliency[i] = X_v(i) . (sum_j X_t(j)).  Two streaming kernels:
// the column sums of the text block (small), then one dot product per visual token against
// that vector, which is one pass over X_v at memory speed (2 bytes per element read once).
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kSalThreads = 256;
constexpr int kSalRowsPerWarp = 8;
constexpr int kSalRowsPerBlock = (kSalThreads / 32) * kSalRowsPerWarp;

// text_sum[b, c] = sum_j x_t[b, j, c] in float32; one thread per pair of columns.
template <typename T>
__global__ void __launch_bounds__(kSalThreads) text_sum_kernel(const T* __restrict__ x_t, int64_t l_t, int64_t d,
                                                               float* __restrict__ text_sum) {
  const int64_t b = blockIdx.y;
  const int64_t c2 = static_cast<int64_t>(blockIdx.x) * kSalThreads + threadIdx.x;
  if (2 * c2 >= d) return;
  const uint32_t* p = reinterpret_cast<const uint32_t*>(x_t + b * l_t * d) + c2;
  float a0 = 0.0f, a1 = 0.0f;
  for (int64_t j = 0; j < l_t; ++j) {
    const float2 f = Elem<T>::to_float2(__ldg(p + j * (d / 2)));
    a0 += f.x; a1 += f.y;
  }
  *reinterpret_cast<float2*>(text_sum + b * d + 2 * c2) = make_float2(a0, a1);
}

// saliency[b, i] = x_v[b, i, :] . text_sum[b, :].  grid = (blocks of 64 rows, B); a warp owns 8
// consecutive rows and walks each in 16-byte pieces per lane, the vector sits in shared memory.
template <typename T>
__global__ void __launch_bounds__(kSalThreads) saliency_kernel(const T* __restrict__ x_v, int64_t l_v, int64_t d,
                                                               const float* __restrict__ text_sum,
                                                               float* __restrict__ saliency) {
  extern __shared__ __align__(16) float tsum[];
  const int64_t b = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t c = threadIdx.x * 4; c < d; c += kSalThreads * 4)
    *reinterpret_cast<float4*>(tsum + c) = __ldg(reinterpret_cast<const float4*>(text_sum + b * d + c));
  __syncthreads();
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kSalRowsPerBlock + warp * kSalRowsPerWarp;
  const int64_t pieces = d / 8;                 // 16-byte pieces per row
#pragma unroll 1
  for (int r = 0; r < kSalRowsPerWarp; r += 2) {
    // two rows at a time: their loads are independent
    const int64_t i0 = row0 + r, i1 = i0 + 1;
    if (i0 >= l_v) break;
    const bool two = i1 < l_v;
    const uint4* p0 = reinterpret_cast<const uint4*>(x_v + (b * l_v + i0) * d);
    const uint4* p1 = reinterpret_cast<const uint4*>(x_v + (b * l_v + (two ? i1 : i0)) * d);
    float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll 2
    for (int64_t k = lane; k < pieces; k += 32) {
      const uint4 u0 = __ldcs(p0 + k);
      const uint4 u1 = __ldcs(p1 + k);
      const float4 ta = *reinterpret_cast<const float4*>(tsum + 8 * k);
      const float4 tb = *reinterpret_cast<const float4*>(tsum + 8 * k + 4);
      const float2 a0 = Elem<T>::to_float2(u0.x), a1 = Elem<T>::to_float2(u0.y), a2 = Elem<T>::to_float2(u0.z), a3 = Elem<T>::to_float2(u0.w);
      const float2 b0 = Elem<T>::to_float2(u1.x), b1 = Elem<T>::to_float2(u1.y), b2 = Elem<T>::to_float2(u1.z), b3 = Elem<T>::to_float2(u1.w);
      acc0 = fmaf(a0.x, ta.x, acc0); acc0 = fmaf(a0.y, ta.y, acc0); acc0 = fmaf(a1.x, ta.z, acc0); acc0 = fmaf(a1.y, ta.w, acc0);
      acc0 = fmaf(a2.x, tb.x, acc0); acc0 = fmaf(a2.y, tb.y, acc0); acc0 = fmaf(a3.x, tb.z, acc0); acc0 = fmaf(a3.y, tb.w, acc0);
      acc1 = fmaf(b0.x, ta.x, acc1); acc1 = fmaf(b0.y, ta.y, acc1); acc1 = fmaf(b1.x, ta.z, acc1); acc1 = fmaf(b1.y, ta.w, acc1);
      acc1 = fmaf(b2.x, tb.x, acc1); acc1 = fmaf(b2.y, tb.y, acc1); acc1 = fmaf(b3.x, tb.z, acc1); acc1 = fmaf(b3.y, tb.w, acc1);
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) {
      acc0 += __shfl_xor_sync(0xffffffffu, acc0, m);
      acc1 += __shfl_xor_sync(0xffffffffu, acc1, m);
    }
    if (lane == 0) {
      saliency[b * l_v + i0] = acc0;
      if (two) saliency[b * l_v + i1] = acc1;
    }
  }
}

template <typename T>
cudaError_t launch_saliency_t(const void* x_v, const void* x_t, int64_t B, int64_t l_v, int64_t l_t, int64_t d,
                              float* text_sum, float* saliency, cudaStream_t stream) {
  cudaError_t e;
  const size_t smem = static_cast<size_t>(d) * sizeof(float);
  static size_t attr_smem[64] = {};
  int dev = 0;
  if ((e = cudaGetDevice(&dev))) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (smem > 48 * 1024 && smem > attr_smem[dev]) {
    if ((e = cudaFuncSetAttribute(saliency_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)))) return e;
    attr_smem[dev] = smem;
  }
  const dim3 g1(static_cast<unsigned>((d / 2 + kSalThreads - 1) / kSalThreads), static_cast<unsigned>(B));
  text_sum_kernel<T><<<g1, kSalThreads, 0, stream>>>(static_cast<const T*>(x_t), l_t, d, text_sum);
  if ((e = cudaGetLastError())) return e;
  const dim3 g2(static_cast<unsigned>((l_v + kSalRowsPerBlock - 1) / kSalRowsPerBlock), static_cast<unsigned>(B));
  saliency_kernel<T><<<g2, kSalThreads, smem, stream>>>(static_cast<const T*>(x_v), l_v, d, text_sum, saliency);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_saliency(int dtype, const void* x_v, const void* x_t, int64_t B, int64_t l_v, int64_t l_t, int64_t d,
                            float* text_sum, float* saliency, cudaStream_t stream) {
  if (dtype == VIDKV_F16) return launch_saliency_t<__half>(x_v, x_t, B, l_v, l_t, d, text_sum, saliency, stream);
  return launch_saliency_t<__nv_bfloat16>(x_v, x_t, B, l_v, l_t, d, text_sum, saliency, stream);
}

}  // namespace vidkv
