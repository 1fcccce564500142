// Decode attention over the packed cache (Algorithm 1 "Decoding", Eq. 3), split-KV.
//
// One CTA = (split of the token axis, KV head of one (layer, batch element)).  It serves
// the `rep` query heads of that KV head.  Keys are never dequantized:
//   * anomalous channels: sum_j q_j (s_j code_j + z_j) = sum_j (q_j s_j) code_j + sum_j q_j z_j,
//     with q_j s_j and the constant formed once per 32-token group;
//   * normal channels: K' = IDFT(+-s), and the inverse transform is linear, so
//     q . K'_t = sum_f Q_f (+-s_f) with Q the (weighted) forward transform of the permuted
//     query, computed once per chunk.
// Phase 1 writes the scaled scores of the split to shared memory; phase 2 turns them into
// exp(score - max) and accumulates P V over the ternary stream, the protected 2-bit stream
// and the FP16 residual.  Each CTA emits (max, sum, unnormalised out[128]) per query head;
// decode_merge_kernel combines the splits.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

struct SplitSmem {
  float* S;          // [8][ST]
  float* q_raw;      // [8][128]
  float* q_abn;      // [8][64]
  float* q_hat;      // [8][64]
  float* cs;         // [64] cos(2 pi m / 64)
  float* sn;         // [64]
  float* qs2;        // [8][64]
  float* qs1;        // [8][64]
  float* qz;         // [8]
  float* red;        // [16]
  uint8_t* kg;       // [1152]
  uint8_t* perm;     // [128]
  uint16_t* tern_map;   // [ST]
  uint16_t* prot_map;   // [ST]
};

__host__ __device__ inline size_t split_smem_bytes(int ST) {
  return sizeof(float) * (8 * ST + 8 * 128 + 8 * 64 * 4 + 128 + 8 + 16) + kKGroupBytes + 128 + 4 * ST;
}

template <typename T>
__global__ void __launch_bounds__(256) decode_split_kernel(DecodeArgs a) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int ST = a.split_tokens;
  SplitSmem sm;
  {
    float* f = reinterpret_cast<float*>(smem_raw);
    sm.S = f; f += 8 * ST;
    sm.q_raw = f; f += 8 * 128;
    sm.q_abn = f; f += 8 * 64;
    sm.q_hat = f; f += 8 * 64;
    sm.qs2 = f; f += 8 * 64;
    sm.qs1 = f; f += 8 * 64;
    sm.cs = f; f += 64;
    sm.sn = f; f += 64;
    sm.qz = f; f += 8;
    sm.red = f; f += 16;
    sm.kg = reinterpret_cast<uint8_t*>(f);
    sm.perm = sm.kg + kKGroupBytes;
    sm.tern_map = reinterpret_cast<uint16_t*>(sm.perm + 128);
    sm.prot_map = sm.tern_map + ST;
  }
  const CacheView& cv = a.cv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x;
  const int slab = blockIdx.y;                       // (layer_idx * B + b) * H_kv + h
  const int h = slab % cv.H_kv;
  const int lb = slab / cv.H_kv;
  const int b = lb % cv.B, layer_idx = lb / cv.B;
  const int rep = cv.rep;
  uint8_t* slab_ptr = cv.slab(a.layer0 + layer_idx, b, h);

  const int64_t T_q0 = a.st.T_q0;
  const int64_t T_qt = T_q0 + a.st.n_flush * kR;      // quantized tokens
  const int64_t T_tot = T_qt + a.st.n_res;
  const int64_t t0 = static_cast<int64_t>(split) * ST;
  const int64_t t1 = min(t0 + ST, T_tot);
  const int64_t tq1 = min(t1, T_qt);                  // end of the quantized part of this split
  const int n_loc = static_cast<int>(t1 - t0);

  // ---- query rows, trig table
  {
    const T* qp = reinterpret_cast<const T*>(a.q) + (static_cast<int64_t>(lb) * cv.H_q + h * rep) * kD;
    for (int i = tid; i < 8 * kD; i += 256) {
      const int r = i >> 7, c = i & 127;
      sm.q_raw[i] = r < rep ? Elem<T>::to_float(qp[r * kD + c]) : 0.0f;
    }
    if (tid < 64) {
      float s, c;
      sincospif(static_cast<float>(tid) / 32.0f, &s, &c);
      sm.cs[tid] = c; sm.sn[tid] = s;
    }
  }
  __syncthreads();

  // ================= phase 1: scores =================
  int cur_chunk = -1;
  const int64_t g0n = T_q0 / kG;                      // key groups of the prefill chunk
  for (int64_t t = t0; t < tq1; t += kG) {
    const int64_t gidx = t / kG;
    const int chunk = gidx < g0n ? 0 : 1 + static_cast<int>((gidx - g0n) / (kR / kG));
    if (chunk != cur_chunk) {
      cur_chunk = chunk;
      if (tid < 128) sm.perm[tid] = slab_ptr[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
      __syncthreads();
      for (int i = tid; i < 8 * 64; i += 256) {
        const int r = i >> 6, j = i & 63;
        sm.q_abn[i] = sm.q_raw[r * kD + sm.perm[j]];
        // weighted forward transform of the permuted query at spectrum column f = j
        float acc = 0.0f;
        if (j < 2) {
          for (int c = 0; c < 64; ++c) {
            const float qv = sm.q_raw[r * kD + sm.perm[64 + c]];
            acc += (j == 1 && (c & 1)) ? -qv : qv;
          }
          acc *= 0.125f;
        } else {
          const int k = j >> 1;
          const bool im = j & 1;
          for (int c = 0; c < 64; ++c) {
            const float qv = sm.q_raw[r * kD + sm.perm[64 + c]];
            const int m = (k * c) & 63;
            acc += qv * (im ? -sm.sn[m] : sm.cs[m]);
          }
          acc *= 0.25f;
        }
        sm.q_hat[i] = acc;
      }
    }
    // stage the group record
    const uint8_t* kgp = slab_ptr + cv.kgroup_offset + gidx * kKGroupBytes;
    if (tid < kKGroupBytes / 16) reinterpret_cast<uint4*>(sm.kg)[tid] = __ldg(reinterpret_cast<const uint4*>(kgp) + tid);
    __syncthreads();
    {
      const uint16_t* s2 = reinterpret_cast<const uint16_t*>(sm.kg + kKG_S2);
      const uint16_t* z2 = reinterpret_cast<const uint16_t*>(sm.kg + kKG_Z2);
      const uint16_t* s1 = reinterpret_cast<const uint16_t*>(sm.kg + kKG_S1);
      for (int i = tid; i < 8 * 64; i += 256) {
        const int j = i & 63;
        sm.qs2[i] = sm.q_abn[i] * h2f(s2[j]);
        sm.qs1[i] = sm.q_hat[i] * h2f(s1[j]);
      }
      float zacc = sm.q_abn[warp * 64 + lane] * h2f(z2[lane]) + sm.q_abn[warp * 64 + 32 + lane] * h2f(z2[32 + lane]);
#pragma unroll
      for (int o = 16; o; o >>= 1) zacc += __shfl_xor_sync(0xffffffffu, zacc, o);
      if (lane == 0) sm.qz[warp] = zacc;
    }
    __syncthreads();
    {
      const float* qs2 = sm.qs2 + warp * 64;
      const float* qs1 = sm.qs1 + warp * 64;
      float acc = sm.qz[warp];
      // token = lane
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint32_t w2 = reinterpret_cast<const uint32_t*>(sm.kg + kKG_Codes2)[k2_word_index(lane, 16 * w)];
        const uint32_t w1 = reinterpret_cast<const uint16_t*>(sm.kg + kKG_Bits1)[k1_half_index(lane, 16 * w)];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          acc += qs2[w * 16 + i] * static_cast<float>((w2 >> k2_bit(i)) & 3u);
          const float v = qs1[w * 16 + i];
          acc += ((w1 >> k1_bit(i)) & 1u) ? v : -v;
        }
      }
      sm.S[warp * ST + static_cast<int>(t - t0) + lane] = acc * a.scale;
    }
    __syncthreads();
  }
  // residual tokens of this split: plain dot products with the FP16 rows
  if (t1 > T_qt) {
    const int64_t r_begin = max(t0, T_qt) - T_qt, r_end = t1 - T_qt;
    const T* kres = reinterpret_cast<const T*>(slab_ptr + cv.kres_offset);
    for (int64_t r = r_begin + lane; r < r_end; r += 32) {
      const uint4* row = reinterpret_cast<const uint4*>(kres + r * kD);
      const float* qr = sm.q_raw + warp * kD;
      float acc = 0.0f;
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const uint4 v = row[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = Elem<T>::to_float2(w[k]);
          acc += qr[i * 8 + 2 * k] * f.x + qr[i * 8 + 2 * k + 1] * f.y;
        }
      }
      sm.S[warp * ST + static_cast<int>(T_qt + r - t0)] = acc * a.scale;
    }
  }
  __syncthreads();

  // ================= softmax numerators =================
  float m_h, l_h;
  {
    float m = -INFINITY;
    for (int i = lane; i < n_loc; i += 32) m = fmaxf(m, sm.S[warp * ST + i]);
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.0f;
    for (int i = lane; i < n_loc; i += 32) {
      const float p = expf(sm.S[warp * ST + i] - m);
      sm.S[warp * ST + i] = p;
      l += p;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    m_h = m; l_h = l;
  }
  // ================= stream maps (only with protected tokens) =================
  const bool stp = a.n_prot > 0;
  const int64_t tp0 = min(t0, T_q0), tp1 = min(tq1, T_q0);          // prefill part of the split
  int64_t pp0 = 0, pp1 = 0;
  if (stp) {
    const uint32_t* ep = cv.e_prefix(b);
    pp0 = ep[tp0 / kG]; pp1 = ep[tp1 / kG];
  }
  // Ternary stream positions.  Prefill tokens: position = token - (protected tokens before it).
  // Flushed tokens start at the next group boundary after the prefill stream.
  const int64_t n_rest = T_q0 - a.n_prot;
  const int64_t u_fl0 = (n_rest + kG - 1) / kG * kG;
  const int64_t ua0 = tp0 - pp0, ua1 = max(tp1 - pp1, ua0);          // prefill part
  const int64_t tf0 = max(t0, T_q0), tf1 = max(tq1, tf0);           // flushed part (tokens)
  if (stp) {
    const uint32_t* ew = cv.e_words(b);
    const uint32_t* ep = cv.e_prefix(b);
    for (int i = tid; i < static_cast<int>(tp1 - t0); i += 256) {
      const int64_t t = t0 + i;
      const uint32_t word = ew[t / kG];
      const int64_t pb = ep[t / kG] + __popc(word & ((1u << (t & 31)) - 1u));
      if (word & (1u << (t & 31))) sm.prot_map[pb - pp0] = static_cast<uint16_t>(i);
      else sm.tern_map[(t - pb) - ua0] = static_cast<uint16_t>(i);
    }
  }
  __syncthreads();

  // ================= phase 2: P V =================
  {
    const int c = tid & 127, hh = tid >> 7;
    const float* P0 = sm.S + (hh * 4 + 0) * ST;
    const float* P1 = sm.S + (hh * 4 + 1) * ST;
    const float* P2 = sm.S + (hh * 4 + 2) * ST;
    const float* P3 = sm.S + (hh * 4 + 3) * ST;
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    // ternary stream: mode 0 = prefill part (through the map when tokens are protected),
    // mode 1 = flushed part (positions follow the tokens)
    const uint8_t* tern = slab_ptr + cv.tern_offset;
    for (int mode = 0; mode < 2; ++mode) {
      const int64_t u0 = mode == 0 ? ua0 : u_fl0 + (tf0 - T_q0);
      const int64_t u1 = mode == 0 ? ua1 : u_fl0 + (tf1 - T_q0);
      if (u1 <= u0) continue;
      for (int64_t gi = u0 / kG; gi <= (u1 - 1) / kG; ++gi) {
        const uint8_t* sg = tern + (gi / kSGGroups) * kSGBytes;
        const int slot = static_cast<int>(gi % kSGGroups);
        const float s = h2f(reinterpret_cast<const uint16_t*>(sg + kSG_Scales)[slot * kD + c]);
        const int j0 = static_cast<int>(max(gi * kG, u0) - gi * kG);
        const int j1 = static_cast<int>(min(gi * kG + kG, u1) - gi * kG);
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
        for (int j = j0; j < j1; ++j) {
          const float tr = static_cast<float>(trit_digit(trit_byte_decode(sg[tern_byte_offset(j, c)]), slot) - 1);
          const int64_t u = gi * kG + j;
          const int li = mode == 1 ? static_cast<int>(u - u_fl0 + T_q0 - t0)
                                   : (stp ? static_cast<int>(sm.tern_map[u - ua0]) : static_cast<int>(u - t0));
          g0 += P0[li] * tr; g1 += P1[li] * tr; g2 += P2[li] * tr; g3 += P3[li] * tr;
        }
        acc0 += s * g0; acc1 += s * g1; acc2 += s * g2; acc3 += s * g3;
      }
    }
    // protected 2-bit stream
    if (pp1 > pp0) {
      const uint8_t* prot = slab_ptr + cv.prot_offset;
      for (int64_t gi = pp0 / kG; gi <= (pp1 - 1) / kG; ++gi) {
        const uint8_t* pg = prot + gi * kPGBytes;
        const float s = h2f(reinterpret_cast<const uint16_t*>(pg + kPG_S)[c]);
        const float z = h2f(reinterpret_cast<const uint16_t*>(pg + kPG_Z)[c]);
        const int j0 = static_cast<int>(max(gi * kG, pp0) - gi * kG);
        const int j1 = static_cast<int>(min(gi * kG + kG, pp1) - gi * kG);
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f, z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
        for (int j = j0; j < j1; ++j) {
          const uint32_t word = reinterpret_cast<const uint32_t*>(pg)[j * 8 + (c >> 4)];
          const float code = static_cast<float>((word >> (2 * (c & 15))) & 3u);
          const int li = sm.prot_map[gi * kG + j - pp0];
          const float p0 = P0[li], p1 = P1[li], p2 = P2[li], p3 = P3[li];
          g0 += p0 * code; g1 += p1 * code; g2 += p2 * code; g3 += p3 * code;
          z0 += p0; z1 += p1; z2 += p2; z3 += p3;
        }
        acc0 += s * g0 + z * z0; acc1 += s * g1 + z * z1; acc2 += s * g2 + z * z2; acc3 += s * g3 + z * z3;
      }
    }
    // residual
    if (t1 > T_qt) {
      const int64_t r_begin = max(t0, T_qt) - T_qt, r_end = t1 - T_qt;
      const T* vres = reinterpret_cast<const T*>(slab_ptr + cv.vres_offset);
      for (int64_t r = r_begin; r < r_end; ++r) {
        const float v = Elem<T>::to_float(vres[r * kD + c]);
        const int li = static_cast<int>(T_qt + r - t0);
        acc0 += P0[li] * v; acc1 += P1[li] * v; acc2 += P2[li] * v; acc3 += P3[li] * v;
      }
    }
    const float accs[4] = {acc0, acc1, acc2, acc3};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r = hh * 4 + k;
      if (r < rep) {
        const int64_t qh = static_cast<int64_t>(lb) * cv.H_q + h * rep + r;
        a.partials[(qh * a.n_splits + split) * 130 + 2 + c] = accs[k];
      }
    }
  }
  if (lane == 0 && warp < rep) {
    const int64_t qh = static_cast<int64_t>(lb) * cv.H_q + h * rep + warp;
    float* pr = a.partials + (qh * a.n_splits + split) * 130;
    pr[0] = m_h; pr[1] = l_h;
  }
}

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

static cudaError_t launch_decode_cc(const DecodeArgs& a, cudaStream_t stream) {
  const int n_slabs = a.n_layers * a.cv.B * a.cv.H_kv;
  const size_t smem = split_smem_bytes(a.split_tokens);
  static size_t attr_smem = 0;
  if (smem > 48 * 1024 && smem > attr_smem) {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(decode_split_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    if ((e = cudaFuncSetAttribute(decode_split_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    attr_smem = smem;
  }
  const dim3 grid(a.n_splits, n_slabs);
  if (a.ev_begin) cudaEventRecord(a.ev_begin, stream);
  if (a.in_dtype == VIDKV_F16) decode_split_kernel<__half><<<grid, 256, smem, stream>>>(a);
  else decode_split_kernel<__nv_bfloat16><<<grid, 256, smem, stream>>>(a);
  if (a.ev_end) cudaEventRecord(a.ev_end, stream);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream) {
  // Protected tokens permute the value streams: those caches take the CUDA-core kernel.
  const cudaError_t e = a.n_prot > 0 ? launch_decode_cc(a, stream) : launch_decode_mma(a, stream);
  if (e != cudaSuccess) return e;
  count_launches(1);
  decode_merge_kernel<<<a.n_layers * a.cv.B * a.cv.H_q, kD, 0, stream>>>(a.partials, a.n_splits, a.out, a.out_dtype);
  return cudaGetLastError();
}

}  // namespace vidkv
