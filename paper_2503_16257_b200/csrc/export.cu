// Test and inspection exports: the packed codes, metadata and selections of one layer as plain
// arrays (one element per code).  Never on the decode path.  The quantizer arithmetic is not
// repeated here: these kernels only undo the bit packing documented in include/vidkv.h.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

// grid = (key groups, slabs of the layer); 128 threads: thread = (slot or column j, half) over 32 tokens.
__global__ void __launch_bounds__(128) export_keys_kernel(CacheView cv, int layer, int64_t n_groups, int8_t* k2,
                                                          uint8_t* k1, uint16_t* ks2, uint16_t* kz2, uint16_t* ks1) {
  const int slab = blockIdx.y, tid = threadIdx.x;
  const int64_t g = blockIdx.x;
  const uint8_t* kg = cv.slab(layer, slab / cv.H_kv, slab % cv.H_kv) + cv.kgroup_offset + g * kKGroupBytes;
  const int j = tid & 63;
  const int64_t row0 = (static_cast<int64_t>(slab) * n_groups + g) * kG;
  if (tid < 64) {
    if (k2)
      for (int t = 0; t < kG; ++t) {
        const uint32_t word = reinterpret_cast<const uint32_t*>(kg + kKG_Codes2)[k2_word_index(t, j)];
        k2[(row0 + t) * 64 + j] = static_cast<int8_t>((word >> k2_bit(j)) & 3u);
      }
    const int64_t m = (static_cast<int64_t>(slab) * n_groups + g) * 64 + j;
    if (ks2) ks2[m] = reinterpret_cast<const uint16_t*>(kg + kKG_S2)[j];
    if (kz2) kz2[m] = reinterpret_cast<const uint16_t*>(kg + kKG_Z2)[j];
    if (ks1) ks1[m] = reinterpret_cast<const uint16_t*>(kg + kKG_S1)[j];
  } else if (k1) {
    for (int t = 0; t < kG; ++t) {
      const uint32_t hw = reinterpret_cast<const uint16_t*>(kg + kKG_Bits1)[k1_half_index(t, j)];
      k1[(row0 + t) * 64 + j] = static_cast<uint8_t>((hw >> k1_bit(j)) & 1u);
    }
  }
}

// The same for the general key formats: thread = slot (tid < n2) or one-bit column / channel.
// ks1 holds per group n1 scales, in plain mode followed by the n1 zero points.
__global__ void __launch_bounds__(128) export_keys_general_kernel(CacheView cv, int layer, int64_t n_groups, int8_t* k2,
                                                                  uint8_t* k1, uint16_t* ks2, uint16_t* kz2, uint16_t* ks1) {
  const int slab = blockIdx.y, tid = threadIdx.x;
  const int64_t g = blockIdx.x;
  const KeyFmt kf = cv.kf;
  const int n2 = kf.n2, n1 = kD - n2;
  const uint8_t* kg = cv.slab(layer, slab / cv.H_kv, slab % cv.H_kv) + cv.kgroup_offset + g * kf.group_bytes;
  const int64_t grp = static_cast<int64_t>(slab) * n_groups + g;
  if (tid < n2) {
    const int j = tid;
    if (k2)
      for (int t = 0; t < kG; ++t) k2[(grp * kG + t) * n2 + j] = static_cast<int8_t>((kg[gk2_byte(t, j)] >> gk2_bit(j)) & 3u);
    if (ks2) ks2[grp * n2 + j] = reinterpret_cast<const uint16_t*>(kg + kf.off_s2)[j];
    if (kz2) kz2[grp * n2 + j] = reinterpret_cast<const uint16_t*>(kg + kf.off_z2)[j];
  } else {
    const int f = tid - n2;
    if (k1)
      for (int t = 0; t < kG; ++t)
        k1[(grp * kG + t) * n1 + f] = static_cast<uint8_t>((kg[kf.off_bits1 + gk1_byte(t, f)] >> gk1_bit(f)) & 1u);
    if (ks1) {
      const int per = kf.plain ? 2 * n1 : n1;
      ks1[grp * per + f] = reinterpret_cast<const uint16_t*>(kg + kf.off_s1)[f];
      if (kf.plain) ks1[grp * per + n1 + f] = reinterpret_cast<const uint16_t*>(kg + kf.off_z1)[f];
    }
  }
}

// grid = (ternary stream groups, slabs); 128 threads = channels.
__global__ void __launch_bounds__(128) export_ternary_kernel(CacheView cv, int layer, int64_t n_groups, int8_t* trits,
                                                             uint16_t* vs) {
  const int slab = blockIdx.y, c = threadIdx.x;
  const int64_t g = blockIdx.x;
  const uint8_t* sg = cv.slab(layer, slab / cv.H_kv, slab % cv.H_kv) + cv.tern_offset + (g / kSGGroups) * kSGBytes;
  const int slot = static_cast<int>(g % kSGGroups);
  const int64_t row0 = (static_cast<int64_t>(slab) * n_groups + g) * kG;
  if (trits)
    for (int j = 0; j < kG; ++j)
      trits[(row0 + j) * kD + c] = static_cast<int8_t>(trit_digit(trit_byte_decode(sg[tern_byte_offset(j, c)]), slot) - 1);
  if (vs) vs[(static_cast<int64_t>(slab) * n_groups + g) * kD + c] = reinterpret_cast<const uint16_t*>(sg + kSG_Scales)[slot * kD + c];
}

// grid = (protected groups, slabs); 128 threads = channels.
__global__ void __launch_bounds__(128) export_protected_kernel(CacheView cv, int layer, int64_t n_groups, int8_t* v2,
                                                               uint16_t* s, uint16_t* z) {
  const int slab = blockIdx.y, c = threadIdx.x;
  const int64_t g = blockIdx.x;
  const uint8_t* pg = cv.slab(layer, slab / cv.H_kv, slab % cv.H_kv) + cv.prot_offset + g * kPGBytes;
  const int64_t row0 = (static_cast<int64_t>(slab) * n_groups + g) * kG;
  if (v2)
    for (int j = 0; j < kG; ++j) {
      const uint32_t word = reinterpret_cast<const uint32_t*>(pg)[prot_word_index(j, c)];
      v2[(row0 + j) * kD + c] = static_cast<int8_t>((word >> prot_bit(j, c)) & 3u);
    }
  const int64_t m = (static_cast<int64_t>(slab) * n_groups + g) * kD + c;
  if (s) s[m] = reinterpret_cast<const uint16_t*>(pg + kPG_S)[c];
  if (z) z[m] = reinterpret_cast<const uint16_t*>(pg + kPG_Z)[c];
}

// dmask [slabs of the layer][n_chunks][128]: 1 = the channel is one of the chunk's 2-bit channels.
__global__ void __launch_bounds__(128) export_dmask_kernel(CacheView cv, int layer, int n_chunks, uint8_t* dmask) {
  const int slab = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const uint8_t* perm = cv.slab(layer, slab / cv.H_kv, slab % cv.H_kv) + cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes;
  uint8_t* out = dmask + (static_cast<int64_t>(slab) * n_chunks + chunk) * kD;
  out[tid] = 0;
  __syncthreads();
  if (tid < cv.kf.n2) out[perm[tid]] = 1;
}

__global__ void export_mask_kernel(CacheView cv, int64_t T, int64_t T_sel, uint8_t* E) {
  const int b = blockIdx.y;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= T) return;
  E[b * T + t] = t < T_sel ? static_cast<uint8_t>((cv.e_words(b)[t / kG] >> (t & 31)) & 1u) : 0;
}

}  // namespace

cudaError_t launch_export_codes(const CacheView& cv, int layer, int64_t n_kgroups, int64_t n_tgroups, int64_t n_pgroups,
                                int8_t* k2, uint8_t* k1, uint16_t* ks2, uint16_t* kz2, uint16_t* ks1, int8_t* trits,
                                uint16_t* vs, int8_t* v2, uint16_t* v2s, uint16_t* v2z, cudaStream_t stream) {
  const int slabs = cv.B * cv.H_kv;
  if (n_kgroups > 0 && (k2 || k1 || ks2 || kz2 || ks1)) {
    if (cv.kf.general)
      export_keys_general_kernel<<<dim3(static_cast<unsigned>(n_kgroups), slabs), 128, 0, stream>>>(cv, layer, n_kgroups, k2, k1, ks2, kz2, ks1);
    else
      export_keys_kernel<<<dim3(static_cast<unsigned>(n_kgroups), slabs), 128, 0, stream>>>(cv, layer, n_kgroups, k2, k1, ks2, kz2, ks1);
    count_launches(1);
  }
  if (n_tgroups > 0 && (trits || vs)) {
    export_ternary_kernel<<<dim3(static_cast<unsigned>(n_tgroups), slabs), 128, 0, stream>>>(cv, layer, n_tgroups, trits, vs);
    count_launches(1);
  }
  if (n_pgroups > 0 && (v2 || v2s || v2z)) {
    export_protected_kernel<<<dim3(static_cast<unsigned>(n_pgroups), slabs), 128, 0, stream>>>(cv, layer, n_pgroups, v2, v2s, v2z);
    count_launches(1);
  }
  return cudaGetLastError();
}

cudaError_t launch_export_selection(const CacheView& cv, int layer, int n_chunks, uint8_t* dmask, int64_t T, int64_t T_sel,
                                    uint8_t* E, cudaStream_t stream) {
  if (dmask && n_chunks > 0) {
    export_dmask_kernel<<<dim3(n_chunks, cv.B * cv.H_kv), 128, 0, stream>>>(cv, layer, n_chunks, dmask);
    count_launches(1);
  }
  if (E && T > 0) {
    export_mask_kernel<<<dim3(static_cast<unsigned>((T + 255) / 256), cv.B), 256, 0, stream>>>(cv, T, T_sel, E);
    count_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace vidkv
