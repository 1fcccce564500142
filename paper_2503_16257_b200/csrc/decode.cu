// Decode attention over the packed cache (Algorithm 1 "Decoding", Eq. 3): the split-KV kernels
// live in decode_mma.cu; this file holds the merge of their partial results.  Each split emits
// (max, sum, unnormalised out[128]) per query head; decode_merge_kernel combines the splits.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

// One block of 128 threads per (layer, b, query head): log-sum-exp merge of the splits.
__global__ void __launch_bounds__(kD) decode_merge_kernel(const float* __restrict__ partials, int n_splits,
                                                          void* __restrict__ out, int out_dtype) {
  const int64_t qh = blockIdx.x;
  const int c = threadIdx.x;
  const float* pr = partials + qh * n_splits * 130;
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, pr[s * 130]);
  float num = 0.0f, den = 0.0f;
  for (int s = 0; s < n_splits; ++s) {
    const float w = expf(pr[s * 130] - M);
    num += w * pr[s * 130 + 2 + c];
    den += w * pr[s * 130 + 1];
  }
  const float o = num / den;
  if (out_dtype == VIDKV_F32) reinterpret_cast<float*>(out)[qh * kD + c] = o;
  else if (out_dtype == VIDKV_F16) reinterpret_cast<__half*>(out)[qh * kD + c] = __float2half_rn(o);
  else reinterpret_cast<__nv_bfloat16*>(out)[qh * kD + c] = __float2bfloat16_rn(o);
}

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream) {
  const cudaError_t e = launch_decode_mma(a, stream);
  if (e != cudaSuccess) return e;
  count_launches(1);
  decode_merge_kernel<<<a.n_layers * a.cv.B * a.cv.H_q, kD, 0, stream>>>(a.partials, a.n_parts, a.out, a.out_dtype);
  return cudaGetLastError();
}

}  // namespace vidkv
