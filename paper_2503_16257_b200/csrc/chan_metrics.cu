// The two channel metrics of Sec. 4.1(1) that the method does not use for its channel split
// (it uses the range): the Variance of a key channel over the tokens and its number of
// Outliers, N = sum_i 1[|K_i| > M * mean_i |K_i|].  Streaming passes over K with float64
// accumulators: a moments pass (sum and sum of squares, or sum of magnitudes), for the outliers
// a counting pass, and a small finishing kernel.  Upstream of the hot path; for inspection.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kCmThreads = 256;          // 16 rows x 16 lanes, a lane owns 8 consecutive channels
constexpr int kCmTokens = 512;           // tokens per block

template <typename T>
__device__ __forceinline__ void load8(const T* row, int lane16, float (&f)[8]) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(row) + lane16);
  const float2 a = Elem<T>::to_float2(v.x), b = Elem<T>::to_float2(v.y), c = Elem<T>::to_float2(v.z), d = Elem<T>::to_float2(v.w);
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

// Sum over the block's 16 rows of one statistic per channel, then one atomic add per channel.
__device__ __forceinline__ void block_add(double (&red)[16][kD + 1], const double (&acc)[8], double* dst) {
  const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 8; ++i) red[row][lane16 * 8 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < kD) {
    double s = 0.0;
#pragma unroll
    for (int r = 0; r < 16; ++r) s += red[r][threadIdx.x];
    atomicAdd(dst + threadIdx.x, s);
  }
  __syncthreads();
}

// VARIANCE: stats[slab][0] += sum x, stats[slab][1] += sum x^2.  Else: stats[slab][0] += sum |x|.
template <typename T, bool VARIANCE>
__global__ void __launch_bounds__(kCmThreads) chan_moments_kernel(KSrc src, int64_t T_tokens, double* __restrict__ stats) {
  __shared__ double red[16][kD + 1];
  const int slab = blockIdx.y;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * kCmTokens, t1 = min(t0 + kCmTokens, T_tokens);
  double a0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, a1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  auto add = [&](const float (&f)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const double x = static_cast<double>(f[i]);
      if (VARIANCE) { a0[i] += x; a1[i] = fma(x, x, a1[i]); }
      else a0[i] += fabs(x);
    }
  };
  int64_t t = t0 + row;
  for (; t + 48 < t1; t += 64) {                       // four rows in flight per thread
    float f[4][8];
#pragma unroll
    for (int k = 0; k < 4; ++k) load8<T>(base + (t + 16 * k) * src.stride_t, lane16, f[k]);
#pragma unroll
    for (int k = 0; k < 4; ++k) add(f[k]);
  }
  for (; t < t1; t += 16) {
    float f[8];
    load8<T>(base + t * src.stride_t, lane16, f);
    add(f);
  }
  block_add(red, a0, stats + static_cast<int64_t>(slab) * 2 * kD);
  if (VARIANCE) block_add(red, a1, stats + static_cast<int64_t>(slab) * 2 * kD + kD);
}

// stats[slab][1] += number of tokens with |x| > M * stats[slab][0] / T.
template <typename T>
__global__ void __launch_bounds__(kCmThreads) chan_outlier_kernel(KSrc src, int64_t T_tokens, double M, double* __restrict__ stats) {
  __shared__ double red[16][kD + 1];
  const int slab = blockIdx.y;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * kCmTokens, t1 = min(t0 + kCmTokens, T_tokens);
  double thr[8], cnt[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int i = 0; i < 8; ++i) thr[i] = M * (stats[static_cast<int64_t>(slab) * 2 * kD + lane16 * 8 + i] / static_cast<double>(T_tokens));
  int64_t t = t0 + row;
  for (; t + 48 < t1; t += 64) {                       // four rows in flight per thread
    float f[4][8];
#pragma unroll
    for (int k = 0; k < 4; ++k) load8<T>(base + (t + 16 * k) * src.stride_t, lane16, f[k]);
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int i = 0; i < 8; ++i) cnt[i] += fabs(static_cast<double>(f[k][i])) > thr[i] ? 1.0 : 0.0;
  }
  for (; t < t1; t += 16) {
    float f[8];
    load8<T>(base + t * src.stride_t, lane16, f);
#pragma unroll
    for (int i = 0; i < 8; ++i) cnt[i] += fabs(static_cast<double>(f[i])) > thr[i] ? 1.0 : 0.0;
  }
  block_add(red, cnt, stats + static_cast<int64_t>(slab) * 2 * kD + kD);
}

// out[slab][c]: population variance (sum x^2 - (sum x)^2 / T) / T, or the outlier count.
__global__ void chan_finish_kernel(const double* __restrict__ stats, int64_t T_tokens, int variance, float* __restrict__ out) {
  const int slab = blockIdx.x, c = threadIdx.x;
  const double s0 = stats[static_cast<int64_t>(slab) * 2 * kD + c], s1 = stats[static_cast<int64_t>(slab) * 2 * kD + kD + c];
  const double n = static_cast<double>(T_tokens);
  out[static_cast<int64_t>(slab) * kD + c] = static_cast<float>(variance ? fmax(0.0, (s1 - s0 * s0 / n) / n) : s1);
}

template <typename T>
cudaError_t launch_t(const KSrc& src, int64_t n_slabs, int64_t T_tokens, int metric, double M, double* stats, float* out,
                     cudaStream_t stream) {
  cudaError_t e;
  if ((e = cudaMemsetAsync(stats, 0, static_cast<size_t>(n_slabs) * 2 * kD * sizeof(double), stream))) return e;
  const dim3 grid(static_cast<unsigned>((T_tokens + kCmTokens - 1) / kCmTokens), static_cast<unsigned>(n_slabs));
  if (metric == VIDKV_METRIC_VARIANCE) {
    chan_moments_kernel<T, true><<<grid, kCmThreads, 0, stream>>>(src, T_tokens, stats);
    count_launches(2);
  } else {
    chan_moments_kernel<T, false><<<grid, kCmThreads, 0, stream>>>(src, T_tokens, stats);
    chan_outlier_kernel<T><<<grid, kCmThreads, 0, stream>>>(src, T_tokens, M, stats);
    count_launches(3);
  }
  chan_finish_kernel<<<static_cast<unsigned>(n_slabs), kD, 0, stream>>>(stats, T_tokens, metric == VIDKV_METRIC_VARIANCE, out);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_channel_metrics(int dtype, const KSrc& src, int64_t n_slabs, int64_t T_tokens, int metric, double M,
                                   double* stats, float* out, cudaStream_t stream) {
  if (dtype == VIDKV_F16) return launch_t<__half>(src, n_slabs, T_tokens, metric, M, stats, out, stream);
  return launch_t<__nv_bfloat16>(src, n_slabs, T_tokens, metric, M, stats, out, stream);
}

}  // namespace vidkv
