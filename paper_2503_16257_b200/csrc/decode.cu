// Decode attention over the packed cache (Algorithm 1 "Decoding", Eq. 3): the split-KV kernels
// live in decode_mma.cu; this file holds the merge of their partial results.  Each split emits
// (max, sum, unnormalised out[128]) per query head; decode_merge_kernel combines the splits.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

// One block of 128 threads per (layer, b, query head): log-sum-exp merge of the splits, four
// records at a time with a running maximum so that a record's three loads (and those of its
// three neighbours) are in flight together.
__global__ void __launch_bounds__(kD) decode_merge_kernel(const float* __restrict__ partials, int n_splits,
                                                          void* __restrict__ out, int out_dtype) {
  const int64_t qh = blockIdx.x;
  const int c = threadIdx.x;
  const float* pr = partials + qh * n_splits * 130;
  float M = -INFINITY, num = 0.0f, den = 0.0f;
  for (int s0 = 0; s0 < n_splits; s0 += 4) {
    float m[4], l[4], v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bool ok = s0 + i < n_splits;
      const float* p = pr + (s0 + i) * 130;
      m[i] = ok ? p[0] : -INFINITY;
      l[i] = ok ? p[1] : 0.0f;
      v[i] = ok ? p[2 + c] : 0.0f;
    }
    const float Mn = fmaxf(fmaxf(M, fmaxf(m[0], m[1])), fmaxf(m[2], m[3]));
    if (Mn == -INFINITY) continue;
    const float so = expf(M - Mn);
    num *= so; den *= so;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float w = expf(m[i] - Mn);
      num += w * v[i];
      den += w * l[i];
    }
    M = Mn;
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
