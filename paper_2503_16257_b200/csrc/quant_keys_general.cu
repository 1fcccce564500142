// Key encode pass of Algorithm 3 (MixQuant) for the general key formats: k other than 0.5, and the
// plain min/max 1-bit code of 1BitQuant's other branch at any k.  One block per (slab, 32-token
// group), one thread per channel; the default format (k = 0.5 with Eq. 5) has its own tensor-core
// encoder and never comes here.
//   anomalous slot j   (Eq. 4, n = 2)  s = (max - min) / 3, z = min, both rounded to binary16;
//                      code = clamp(rint((x - z) / s), 0, 3) with the float32 division as written.
//   normal channel i, plain mode (Eq. 4, n = 1)  s = max - min, z = min; code in {0, 1}.
//   spectrum column f, Eq. 5  X = orthonormal n1-point DFT of the token's normal channels (ascending
//                      channel order), Hermitian half: column 0 = Re X[0], 1 = Re X[n1 / 2],
//                      2 k = Re X[k], 2 k + 1 = Im X[k]; bit = [X >= 0], s = mean |X| over the group.
//                      The sums run in float64 (the work is small and the scale then rounds once).
#include <math.h>

#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kMaxFftChannels = 32;   // Eq. 5 comes here for k = 0.75 only (k = 0.5 has the default format's encoder)

template <typename T>
__global__ void __launch_bounds__(kD) k_encode_general_kernel(KSrc src, CacheView cv, int layer0, int slabs_per_layer,
                                                              int chunk, int64_t kgroup0) {
  __shared__ __align__(16) float x[kG][kD + 4];   // the group's tile, token major
  __shared__ uint8_t code[kG][kD];           // one code per (token, slot / column), packed afterwards
  __shared__ uint8_t perm[kD];
  __shared__ double tw_cos[kD], tw_sin[kD];  // cos / sin of 2 pi m / n1
  __shared__ double mag[kG][kMaxFftChannels];   // |X| per (token, spectrum column)
  const int tid = threadIdx.x;
  const int slab = blockIdx.y;
  const int64_t g = blockIdx.x;
  const KeyFmt kf = cv.kf;
  const int n2 = kf.n2, n1 = kD - n2;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  uint8_t* slab_ptr = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv);
  perm[tid] = slab_ptr[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h +
                  g * kG * src.stride_t;
  // 16 bytes (8 channels) per thread and step: 16 threads per token row, 8 rows per step
  for (int t = tid >> 4; t < kG; t += kD / 16) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + t * src.stride_t) + (tid & 15));
    const float2 f0 = Elem<T>::to_float2(v.x), f1 = Elem<T>::to_float2(v.y), f2 = Elem<T>::to_float2(v.z), f3 = Elem<T>::to_float2(v.w);
    float4* dst = reinterpret_cast<float4*>(&x[t][(tid & 15) * 8]);
    dst[0] = make_float4(f0.x, f0.y, f1.x, f1.y);
    dst[1] = make_float4(f2.x, f2.y, f3.x, f3.y);
  }
  if (!kf.plain && tid < n1) sincospi(2.0 * static_cast<double>(tid) / static_cast<double>(n1), &tw_sin[tid], &tw_cos[tid]);
  __syncthreads();
  uint8_t* kg = slab_ptr + cv.kgroup_offset + (kgroup0 + g) * kf.group_bytes;

  if (tid < n2 || kf.plain) {
    // Eq. 4 on one channel of the group: two bits for an anomalous slot, one bit for a normal channel
    const bool two = tid < n2;
    const int c = perm[tid];
    float mn = x[0][c], mx = mn;
    for (int t = 1; t < kG; ++t) { mn = fminf(mn, x[t][c]); mx = fmaxf(mx, x[t][c]); }
    const float levels = two ? 3.0f : 1.0f;
    const uint16_t sh = f2h_bits(__fdiv_rn(__fsub_rn(mx, mn), levels));
    const uint16_t zh = f2h_bits(mn);
    const float s = h2f(sh), z = h2f(zh);
    for (int t = 0; t < kG; ++t) {
      float q = 0.0f;
      if (s != 0.0f) q = fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(x[t][c], z), s)), 0.0f), levels);
      code[t][tid] = static_cast<uint8_t>(q);
    }
    if (two) {
      reinterpret_cast<uint16_t*>(kg + kf.off_s2)[tid] = sh;
      reinterpret_cast<uint16_t*>(kg + kf.off_z2)[tid] = zh;
    } else {
      reinterpret_cast<uint16_t*>(kg + kf.off_s1)[tid - n2] = sh;
      reinterpret_cast<uint16_t*>(kg + kf.off_z1)[tid - n2] = zh;
    }
  }
  if (!kf.plain && n1 > 0) {
    // Eq. 5: the (token, spectrum column) pairs of the group are shared out over all threads; the
    // magnitudes wait in shared memory and one thread per column adds them up in token order
    const double norm = 1.0 / sqrt(static_cast<double>(n1));
    const int mask = n1 - 1;                  // Eq. 5 is offered for n1 = 32 (a power of two)
    for (int idx = tid; idx < n1 * kG; idx += kD) {
      const int f = idx & mask, t = idx / n1;
      const int k = f < 2 ? (f == 0 ? 0 : n1 / 2) : f >> 1;
      const bool imag = f >= 2 && (f & 1);
      double acc = 0.0;
      for (int i = 0; i < n1; ++i) {
        const int m = (k * i) & mask;
        acc += static_cast<double>(x[t][perm[n2 + i]]) * (imag ? -tw_sin[m] : tw_cos[m]);
      }
      acc *= norm;
      mag[t][f] = fabs(acc);
      code[t][n2 + f] = acc >= 0.0 ? 1 : 0;
    }
    __syncthreads();
    if (tid < n1) {
      double sum = 0.0;
      for (int t = 0; t < kG; ++t) sum += mag[t][tid];
      reinterpret_cast<uint16_t*>(kg + kf.off_s1)[tid] = __half_as_ushort(__double2half(sum / kG));
    }
  }
  __syncthreads();
  // pack: every output byte of the two code regions is put together by one thread
  for (int b = tid; b < n2 * 8; b += kD) {
    // byte b of the two-bit region: block, lane (tl, r), tile nt, parity of the slot
    const int blk = b >> 8, in = b & 255, lane = in >> 3, nt = (in >> 1) & 3, par = in & 1;
    const int t = 8 * nt + (lane >> 2), j0 = 32 * blk + 8 * (lane & 3) + par;
    uint32_t v = 0;
    for (int i = 0; i < 4; ++i) v |= static_cast<uint32_t>(code[t][j0 + 2 * i]) << (2 * i);
    kg[b] = static_cast<uint8_t>(v);
  }
  for (int b = tid; b < n1 * 4; b += kD) {
    const int blk = b >> 7, in = b & 127, lane = in >> 2, nt = in & 3;
    const int t = 8 * nt + (lane >> 2), f0 = 32 * blk + 8 * (lane & 3);
    uint32_t v = 0;
    for (int e = 0; e < 8; ++e) v |= static_cast<uint32_t>(code[t][n2 + f0 + e]) << (7 - e);
    kg[kf.off_bits1 + b] = static_cast<uint8_t>(v);
  }
}

}  // namespace

cudaError_t launch_encode_keys_general(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0,
                                       int n_slabs, int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream) {
  const int64_t groups = T_tokens / kG;
  if (groups <= 0 || n_slabs <= 0) return cudaSuccess;
  if (groups > INT32_MAX || n_slabs > 65535) return cudaErrorInvalidValue;
  const dim3 grid(static_cast<unsigned>(groups), static_cast<unsigned>(n_slabs));
  if (dtype == VIDKV_F16) k_encode_general_kernel<__half><<<grid, kD, 0, stream>>>(src, cv, layer0, slabs_per_layer, chunk, kgroup0);
  else k_encode_general_kernel<__nv_bfloat16><<<grid, kD, 0, stream>>>(src, cv, layer0, slabs_per_layer, chunk, kgroup0);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace vidkv
