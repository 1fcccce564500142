// Query preparation of the decode attention (Algorithm 1 "Decoding", Eq. 3): per (slab, chunk)
// the register images of the query that the stream kernels (decode_stream.cu) multiply with the
// packed key codes.  Everything that depends on the query alone is done here, once per chunk:
//   anomalous channels  sum_j q_j (s_j code_j + z_j): the kernels need q at the chunk's 2-bit
//       channels, in the order of the MMA fragments;
//   normal channels     K' = IDFT(+-s), so q . K'_t = sum_f Q_f s_f (+-1) with Q the weighted
//       forward transform of the permuted query, computed here on the tensor cores against the
//       split-precision DFT matrix the encoder uses.
// The step's append of k_new / v_new to the residual rides on this kernel.
#include "decode_common.cuh"

namespace vidkv {

size_t decode_prep_bytes(int64_t n_slabs, int64_t n_chunks) {
  return static_cast<size_t>(n_slabs) * n_chunks * kPrepWords * 32 * sizeof(uint32_t);
}

// ---------------------------------------------------------------------------------
// Query preparation: one warp per (chunk, slab).  Writes, per lane, the 24 register images the
// attention kernel needs for this chunk's channel split:
//   words  0.. 7  binary16 pairs of q at the anomalous slots (16 r + 2 i, 16 r + 2 i + 1)
//   words  8..15  leading binary16 part of the transformed query Q at the spectrum
//                 columns (16 r + 2 i, 16 r + 2 i + 1)
//   words 16..23  binary16 remainder Q - leading part
//   word  24      float: softmax scale * log2 e * 2^(e + kQShift), which turns a score of this
//                 normalised query into a base-2 logit
// for head lane / 4 (zero when that head does not exist) and r = lane % 4, all of the query
// normalised by its head's power of two (head_exponent).
// Q_f = sum_c q_c W[c, f] with W the weights with which spectrum column f enters channel c of
// the inverse orthonormal 64-point transform of a Hermitian half spectrum: the forward DFT
// matrix, doubled for the columns f >= 2 that stand for a conjugate pair.  The product runs
// on the tensor cores against the same split-precision matrix fragments the encoder uses.
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) decode_prep_kernel(DecodeArgs a, int n_chunks, int n_items) {
  const CacheView& cv = a.cv;
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  pdl_release();                                           // the attention kernel may start its first copies now
  if (item >= n_items) return;
  const int chunk = item % n_chunks, slab = item / n_chunks;
  const int hd = lane >> 2, r = lane & 3;
  const int h = slab % cv.H_kv, lb = slab / cv.H_kv;
  const int rep = cv.rep;
  const uint8_t* perm = cv.slab(a.layer0 + lb / cv.B, lb % cv.B, h) + cv.chunk_table_offset +
                        static_cast<int64_t>(chunk) * kChunkBytes;
  const T* qrow = reinterpret_cast<const T*>(a.q) + (static_cast<int64_t>(lb) * cv.H_q + h * rep + hd) * kD;
  const bool live = hd < rep;
  const int qe = head_exponent<T, 4>(qrow, r, live);
  const float qf = pow2i(-qe - kQShift);                                   // normalised query, see head_exponent
  auto q_at = [&](int c) -> float { return live ? Elem<T>::to_float(qrow[c]) * qf : 0.0f; };
  if (chunk == 0 && a.append_row >= 0) {
    // Algorithm 1, Decoding: the step's new key / value row joins the residual (lanes 0-15 copy
    // the key row, 16-31 the value row); the attention kernel that follows reads it there.
    uint8_t* sp = cv.slab(a.layer0 + lb / cv.B, lb % cv.B, h);
    const uint4* srcp = reinterpret_cast<const uint4*>(lane < 16 ? a.k_new : a.v_new) + static_cast<int64_t>(slab) * 16 + (lane & 15);
    reinterpret_cast<uint4*>(sp + (lane < 16 ? cv.kres_offset : cv.vres_offset))[a.append_row * 16 + (lane & 15)] = __ldg(srcp);
  }
  uint32_t* out = a.prep + (static_cast<int64_t>(slab) * n_chunks + chunk) * (kPrepWords * 32) + lane;
  // anomalous slots
  {
    const uint4 p0 = __ldg(reinterpret_cast<const uint4*>(perm + 16 * r));
    const uint32_t pw[4] = {p0.x, p0.y, p0.z, p0.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t two = pw[i >> 1] >> (16 * (i & 1));
      out[i * 32] = pack_half2(q_at(two & 0xffu), q_at((two >> 8) & 0xffu));
    }
  }
  // transformed query: A = q at the normal channels (rows 8-15 unused), B = matrix fragments
  uint32_t af[4][2];
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
    const uint32_t pa = __ldg(reinterpret_cast<const uint16_t*>(perm + kNA + 16 * ks + 2 * r));
    const uint32_t pb = __ldg(reinterpret_cast<const uint16_t*>(perm + kNA + 16 * ks + 2 * r + 8));
    af[ks][0] = pack_half2(q_at(pa & 0xffu), q_at(pa >> 8));
    af[ks][1] = pack_half2(q_at(pb & 0xffu), q_at(pb >> 8));
  }
  float acc[8][4];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) { acc[nt][0] = 0.0f; acc[nt][1] = 0.0f; acc[nt][2] = 0.0f; acc[nt][3] = 0.0f; }
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const uint4 bw = __ldg(reinterpret_cast<const uint4*>(a.dft + ((ks * 8 + nt) * 32 + lane) * 4));
      mma_f16(acc[nt], af[ks][0], 0u, af[ks][1], 0u, bw.x, bw.y);
      mma_f16(acc[nt], af[ks][0], 0u, af[ks][1], 0u, bw.z, bw.w);
    }
  }
  // lane (hd, r) now holds Q of head hd at columns 16 r + 2 nt + {0, 1}
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const float w0 = (r == 0 && nt == 0) ? 1.0f : 2.0f;            // columns 0 and 1 are not doubled
    const float x0 = acc[nt][0] * w0, x1 = acc[nt][1] * w0;
    const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
    out[(8 + nt) * 32] = pack_half2(__half2float(h0), __half2float(h1));
    out[(16 + nt) * 32] = pack_half2(x0 - __half2float(h0), x1 - __half2float(h1));
  }
  // factor that turns a score in the normalised units into a base-2 logit
  out[24 * 32] = __float_as_uint(a.scale * 1.4426950408889634f * pow2i(qe + kQShift));
}

// ---------------------------------------------------------------------------------
// The same for the general key formats (KeyFmt): one warp per (chunk, slab); per lane (head hd = lane / 4,
// r = lane % 4), all of the normalised query:
//   words 0 .. n2/8 - 1         binary16 pairs of q at the two-bit slots 32 (w / 4) + 8 r + 2 (w % 4), + 1
//   then n1/8 words             plain mode: pairs of q at the one-bit channels with the same index rule;
//                               Eq. 5: leading binary16 part of the transformed query Q at those columns,
//   then (Eq. 5) n1/8 words     binary16 remainder Q - leading part
//   word 24                     the factor that turns a score into a base-2 logit
// Q_f = sum_c q_c W[c, f], W = the weights with which column f of the Hermitian half spectrum enters
// normal channel c under the inverse orthonormal n1-point transform (columns >= 2 count twice).
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) decode_prep_general_kernel(DecodeArgs a, int n_chunks, int n_items) {
  const CacheView& cv = a.cv;
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  pdl_release();                                           // the attention kernel may start its first copies now
  if (item >= n_items) return;
  const int chunk = item % n_chunks, slab = item / n_chunks;
  const int hd = lane >> 2, r = lane & 3;
  const int h = slab % cv.H_kv, lb = slab / cv.H_kv;
  const int rep = cv.rep;
  const int n2 = cv.kf.n2, n1 = kD - n2;
  const uint8_t* perm = cv.slab(a.layer0 + lb / cv.B, lb % cv.B, h) + cv.chunk_table_offset +
                        static_cast<int64_t>(chunk) * kChunkBytes;
  const T* qrow = reinterpret_cast<const T*>(a.q) + (static_cast<int64_t>(lb) * cv.H_q + h * rep + hd) * kD;
  const bool live = hd < rep;
  const int qe = head_exponent<T, 4>(qrow, r, live);
  const float qf = pow2i(-qe - kQShift);
  auto q_at = [&](int c) -> float { return live ? Elem<T>::to_float(qrow[c]) * qf : 0.0f; };
  if (chunk == 0 && a.append_row >= 0) {
    uint8_t* sp = cv.slab(a.layer0 + lb / cv.B, lb % cv.B, h);
    const uint4* srcp = reinterpret_cast<const uint4*>(lane < 16 ? a.k_new : a.v_new) + static_cast<int64_t>(slab) * 16 + (lane & 15);
    reinterpret_cast<uint4*>(sp + (lane < 16 ? cv.kres_offset : cv.vres_offset))[a.append_row * 16 + (lane & 15)] = __ldg(srcp);
  }
  uint32_t* out = a.prep + (static_cast<int64_t>(slab) * n_chunks + chunk) * (kPrepWords * 32) + lane;
  for (int w = 0; w < n2 / 8; ++w) {
    const int j = 32 * (w >> 2) + 8 * r + 2 * (w & 3);
    out[w * 32] = pack_half2(q_at(perm[j]), q_at(perm[j + 1]));
  }
  const int w1 = n2 / 8;
  if (cv.kf.plain) {
    for (int w = 0; w < n1 / 8; ++w) {
      const int i = 32 * (w >> 2) + 8 * r + 2 * (w & 3);
      out[(w1 + w) * 32] = pack_half2(q_at(perm[n2 + i]), q_at(perm[n2 + i + 1]));
    }
  } else {
    const float norm = rsqrtf(static_cast<float>(n1));
    for (int w = 0; w < n1 / 8; ++w) {
      float x[2];
      for (int e = 0; e < 2; ++e) {
        const int f = 32 * (w >> 2) + 8 * r + 2 * (w & 3) + e;
        const int k = f < 2 ? (f == 0 ? 0 : n1 / 2) : f >> 1;
        const bool imag = f >= 2 && (f & 1);
        float acc = 0.0f;
        for (int c = 0; c < n1; ++c) {
          float sn, cs;
          sincospif(2.0f * static_cast<float>((k * c) % n1) / static_cast<float>(n1), &sn, &cs);
          acc = fmaf(q_at(perm[n2 + c]), imag ? -sn : cs, acc);
        }
        x[e] = acc * norm * (f < 2 ? 1.0f : 2.0f);
      }
      const __half h0 = __float2half_rn(x[0]), h1 = __float2half_rn(x[1]);
      out[(w1 + w) * 32] = pack_half2(__half2float(h0), __half2float(h1));
      out[(w1 + n1 / 8 + w) * 32] = pack_half2(x[0] - __half2float(h0), x[1] - __half2float(h1));
    }
  }
  out[24 * 32] = __float_as_uint(a.scale * 1.4426950408889634f * pow2i(qe + kQShift));
}

cudaError_t launch_decode_prep(DecodeArgs& a, cudaStream_t stream) {
  a.dft = nullptr;
  const int n_slabs = a.n_layers * a.cv.B * a.cv.H_kv;
  const int n_chunks = a.plan.n_chunks;
  if (n_chunks < 1) return cudaSuccess;
  cudaError_t e;
  const int n_items = n_slabs * n_chunks;
  const int pgrid = (n_items + kThreads / 32 - 1) / (kThreads / 32);
  if (a.cv.kf.general) {
    if (a.in_dtype == VIDKV_F16) decode_prep_general_kernel<__half><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
    else decode_prep_general_kernel<__nv_bfloat16><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
    count_launches(1);
    return cudaGetLastError();
  }
  if ((e = dft_fragments(&a.dft, stream))) return e;
  if (a.in_dtype == VIDKV_F16) decode_prep_kernel<__half><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
  else decode_prep_kernel<__nv_bfloat16><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace vidkv
