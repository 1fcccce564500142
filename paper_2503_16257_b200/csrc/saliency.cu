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
// consecutive rows and walks four of them at a time in 16-byte pieces per lane (four independent
// loads in flight per lane), the vector sits in shared memory.
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
  for (int r = 0; r < kSalRowsPerWarp; r += 4) {
    const int64_t i0 = row0 + r;
    if (i0 >= l_v) break;
    const uint4* p[4];
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int q = 0; q < 4; ++q) p[q] = reinterpret_cast<const uint4*>(x_v + (b * l_v + min(i0 + q, l_v - 1)) * d);
#pragma unroll 1
    for (int64_t k = lane; k < pieces; k += 32) {
      uint4 u[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) u[q] = __ldcs(p[q] + k);
      const float4 ta = *reinterpret_cast<const float4*>(tsum + 8 * k);
      const float4 tb = *reinterpret_cast<const float4*>(tsum + 8 * k + 4);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 a0 = Elem<T>::to_float2(u[q].x), a1 = Elem<T>::to_float2(u[q].y), a2 = Elem<T>::to_float2(u[q].z), a3 = Elem<T>::to_float2(u[q].w);
        float a = acc[q];
        a = fmaf(a0.x, ta.x, a); a = fmaf(a0.y, ta.y, a); a = fmaf(a1.x, ta.z, a); a = fmaf(a1.y, ta.w, a);
        a = fmaf(a2.x, tb.x, a); a = fmaf(a2.y, tb.y, a); a = fmaf(a3.x, tb.z, a); a = fmaf(a3.y, tb.w, a);
        acc[q] = a;
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], m);
      if (lane == 0 && i0 + q < l_v) saliency[b * l_v + i0 + q] = acc[q];
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
