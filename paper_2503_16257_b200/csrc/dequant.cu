// Test and inspection kernels: DeQuant of Algorithm 1 for a whole layer, to float32.
// Never used by the decode path (which reads the packed cache directly).
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

// grid = (key groups, slabs of one layer); block = 128 threads.
__global__ void __launch_bounds__(128) dequant_keys_kernel(CacheView cv, int layer, int64_t T_q0, int64_t T_qt,
                                                           float* __restrict__ out) {
  __shared__ __align__(16) uint8_t kg[kKGroupBytes];
  __shared__ uint8_t perm[kD];
  __shared__ float cs[64], sn[64];
  const int tid = threadIdx.x;
  const int slab = blockIdx.y;
  const int b = slab / cv.H_kv, h = slab % cv.H_kv;
  const int64_t gidx = blockIdx.x;
  const int64_t g0n = T_q0 / kG;
  const int chunk = gidx < g0n ? 0 : 1 + static_cast<int>((gidx - g0n) / (kR / kG));
  const uint8_t* sp = cv.slab(layer, b, h);
  perm[tid] = sp[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
  if (tid < kKGroupBytes / 16)
    reinterpret_cast<uint4*>(kg)[tid] = reinterpret_cast<const uint4*>(sp + cv.kgroup_offset + gidx * kKGroupBytes)[tid];
  if (tid < 64) {
    float s, c;
    sincospif(static_cast<float>(tid) / 32.0f, &s, &c);
    cs[tid] = c; sn[tid] = s;
  }
  __syncthreads();
  float* o = out + ((static_cast<int64_t>(slab) * T_qt) + gidx * kG) * kD;
  if (tid < 64) {
    const int j = tid, c = perm[j];
    const float s = h2f(reinterpret_cast<const uint16_t*>(kg + kKG_S2)[j]);
    const float z = h2f(reinterpret_cast<const uint16_t*>(kg + kKG_Z2)[j]);
    for (int t = 0; t < kG; ++t) {
      const uint32_t word = reinterpret_cast<const uint32_t*>(kg + kKG_Codes2)[k2_word_index(t, j)];
      o[t * kD + c] = static_cast<float>((word >> k2_bit(j)) & 3u) * s + z;
    }
  } else {
    const int i = tid - 64, c = perm[64 + i];
    const uint16_t* s1 = reinterpret_cast<const uint16_t*>(kg + kKG_S1);
    for (int t = 0; t < kG; ++t) {
      const uint16_t* hw = reinterpret_cast<const uint16_t*>(kg + kKG_Bits1);
      auto val = [&](int f) -> float {
        const uint32_t bit = (hw[k1_half_index(t, f)] >> k1_bit(f)) & 1u;
        const float s = h2f(s1[f]);
        return bit ? s : -s;
      };
      float acc = val(0) + ((i & 1) ? -val(1) : val(1));
      float acc2 = 0.0f;
      for (int k = 1; k < 32; ++k) {
        const int m = (k * i) & 63;
        acc2 += val(2 * k) * cs[m] - val(2 * k + 1) * sn[m];
      }
      o[t * kD + c] = 0.125f * acc + 0.25f * acc2;
    }
  }
}

// The same for the general key formats (see KeyFmt): thread = output channel position in the chunk's order.
__global__ void __launch_bounds__(128) dequant_keys_general_kernel(CacheView cv, int layer, int64_t T_q0, int64_t T_qt,
                                                                   float* __restrict__ out) {
  __shared__ __align__(16) uint8_t kg[kMaxKGroupBytes];
  __shared__ uint8_t perm[kD];
  __shared__ float cs[kD], sn[kD];
  const int tid = threadIdx.x;
  const int slab = blockIdx.y;
  const int b = slab / cv.H_kv, h = slab % cv.H_kv;
  const int64_t gidx = blockIdx.x;
  const int64_t g0n = T_q0 / kG;
  const KeyFmt kf = cv.kf;
  const int n2 = kf.n2, n1 = kD - n2;
  const int chunk = gidx < g0n ? 0 : 1 + static_cast<int>((gidx - g0n) / (kR / kG));
  const uint8_t* sp = cv.slab(layer, b, h);
  perm[tid] = sp[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
  if (tid < kf.group_bytes / 16)
    reinterpret_cast<uint4*>(kg)[tid] = reinterpret_cast<const uint4*>(sp + cv.kgroup_offset + gidx * kf.group_bytes)[tid];
  if (tid < n1) {
    float s, c;
    sincospif(2.0f * static_cast<float>(tid) / static_cast<float>(n1), &s, &c);
    cs[tid] = c; sn[tid] = s;
  }
  __syncthreads();
  float* o = out + ((static_cast<int64_t>(slab) * T_qt) + gidx * kG) * kD;
  const int c = perm[tid];
  if (tid < n2) {
    const int j = tid;
    const float s = h2f(reinterpret_cast<const uint16_t*>(kg + kf.off_s2)[j]);
    const float z = h2f(reinterpret_cast<const uint16_t*>(kg + kf.off_z2)[j]);
    for (int t = 0; t < kG; ++t) o[t * kD + c] = static_cast<float>((kg[gk2_byte(t, j)] >> gk2_bit(j)) & 3u) * s + z;
  } else if (kf.plain) {
    const int i = tid - n2;
    const float s = h2f(reinterpret_cast<const uint16_t*>(kg + kf.off_s1)[i]);
    const float z = h2f(reinterpret_cast<const uint16_t*>(kg + kf.off_z1)[i]);
    for (int t = 0; t < kG; ++t)
      o[t * kD + c] = static_cast<float>((kg[kf.off_bits1 + gk1_byte(t, i)] >> gk1_bit(i)) & 1u) * s + z;
  } else {
    // inverse orthonormal n1-point transform of the Hermitian half spectrum (+-s per column) at position i
    const int i = tid - n2;
    const uint16_t* s1 = reinterpret_cast<const uint16_t*>(kg + kf.off_s1);
    const float norm = rsqrtf(static_cast<float>(n1));
    for (int t = 0; t < kG; ++t) {
      auto val = [&](int f) -> float {
        const uint32_t bit = (kg[kf.off_bits1 + gk1_byte(t, f)] >> gk1_bit(f)) & 1u;
        const float s = h2f(s1[f]);
        return bit ? s : -s;
      };
      const float acc = val(0) + ((i & 1) ? -val(1) : val(1));
      float acc2 = 0.0f;
      for (int k = 1; k < n1 / 2; ++k) {
        const int m = (k * i) % n1;
        acc2 += val(2 * k) * cs[m] - val(2 * k + 1) * sn[m];
      }
      o[t * kD + c] = norm * (acc + 2.0f * acc2);
    }
  }
}

// grid = (32-token blocks of the quantized part, slabs of one layer); block = 128 threads.
__global__ void __launch_bounds__(128) dequant_values_kernel(CacheView cv, int layer, int64_t T_q0, int64_t T_qt,
                                                             int64_t n_prot, float* __restrict__ out) {
  const int c = threadIdx.x;
  const int slab = blockIdx.y;
  const int b = slab / cv.H_kv, h = slab % cv.H_kv;
  const uint8_t* sp = cv.slab(layer, b, h);
  float* o = out + (static_cast<int64_t>(slab) * T_qt + static_cast<int64_t>(blockIdx.x) * kG) * kD;
  for (int tt = 0; tt < kG; ++tt) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kG + tt;
    bool prot = false;
    int64_t pb = 0;
    if (n_prot > 0 && t < T_q0) {
      const uint32_t word = cv.e_words(b)[t / kG];
      pb = cv.e_prefix(b)[t / kG] + __popc(word & ((1u << (t & 31)) - 1u));
      prot = (word >> (t & 31)) & 1u;
    }
    float v;
    if (prot) {
      const uint8_t* pg = sp + cv.prot_offset + (pb / kG) * kPGBytes;
      const int j = static_cast<int>(pb % kG);
      const uint32_t word = reinterpret_cast<const uint32_t*>(pg)[prot_word_index(j, c)];
      v = static_cast<float>((word >> prot_bit(j, c)) & 3u) * h2f(reinterpret_cast<const uint16_t*>(pg + kPG_S)[c]) +
          h2f(reinterpret_cast<const uint16_t*>(pg + kPG_Z)[c]);
    } else {
      const int64_t n_rest = T_q0 - n_prot;
      const int64_t u = t < T_q0 ? t - pb : (n_rest + kG - 1) / kG * kG + (t - T_q0);
      const int64_t gi = u / kG;
      const uint8_t* sg = sp + cv.tern_offset + (gi / kSGGroups) * kSGBytes;
      const int slot = static_cast<int>(gi % kSGGroups);
      const int tr = trit_digit(trit_byte_decode(sg[tern_byte_offset(static_cast<int>(u % kG), c)]), slot) - 1;
      v = static_cast<float>(tr) * h2f(reinterpret_cast<const uint16_t*>(sg + kSG_Scales)[slot * kD + c]);
    }
    o[tt * kD + c] = v;
  }
}

cudaError_t launch_dequant_keys(const CacheView& cv, int layer, int64_t T_q0, int64_t n_flush, float* out,
                                cudaStream_t stream) {
  const int64_t T_qt = T_q0 + n_flush * kR;
  if (T_qt == 0) return cudaSuccess;
  if (cv.kf.general)
    dequant_keys_general_kernel<<<dim3(static_cast<unsigned>(T_qt / kG), cv.B * cv.H_kv), 128, 0, stream>>>(cv, layer, T_q0, T_qt, out);
  else
    dequant_keys_kernel<<<dim3(static_cast<unsigned>(T_qt / kG), cv.B * cv.H_kv), 128, 0, stream>>>(cv, layer, T_q0, T_qt, out);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_dequant_values(const CacheView& cv, int layer, int64_t T_q0, int64_t n_flush, int64_t n_prot,
                                  float* out, cudaStream_t stream) {
  const int64_t T_qt = T_q0 + n_flush * kR;
  if (T_qt == 0) return cudaSuccess;
  dequant_values_kernel<<<dim3(static_cast<unsigned>(T_qt / kG), cv.B * cv.H_kv), 128, 0, stream>>>(cv, layer, T_q0, T_qt,
                                                                                                     n_prot, out);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace vidkv
