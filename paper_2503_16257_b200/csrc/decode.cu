// Decode attention over the packed cache (Algorithm 1 "Decoding", Eq. 3): how a call is cut into
// work (plan_decode), the launch sequence, and the last kernel of a step, which merges the
// partial records of the attention kernels by log-sum-exp and, for caches without protected
// tokens, attends to the FP16 / BF16 residual itself.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kMaxSMs = 256;        // multiprocessor count the sizing formulas assume at most
constexpr int kMinRunUnits = 2;     // a warp's run is never shorter (one record per 320 tokens at worst)

// Tokens per split of the split kernel: the largest of {640, 320, 160} that still gives
// >= 4 CTAs per SM on a 148-SM part, else 160.
int choose_split_tokens(int64_t T_tot, int64_t n_slabs) {
  const int cand[3] = {640, 320, 160};
  for (int s : cand)
    if (n_slabs * ((T_tot + s - 1) / s) >= 592) return s;
  return 160;
}

}  // namespace

int device_sm_count() {
  static int sm_of_device[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (sm_of_device[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
    sm_of_device[dev] = n;
  }
  return sm_of_device[dev];
}

DecodePlan plan_decode(const LayerState& st, int64_t n_slabs, int64_t n_prot, int sm_count, int force_split_tokens,
                       int force_run_units) {
  DecodePlan p = {};
  const int64_t T_qt = st.T_q0 + st.n_flush * kR;
  p.n_chunks = T_qt > 0 ? 1 + static_cast<int32_t>(st.n_flush) : 0;
  if (n_prot > 0) {
    const int64_t T_tot = T_qt + st.n_res;
    p.stream = 0;
    p.split_tokens = force_split_tokens > 0 ? force_split_tokens : choose_split_tokens(T_tot, n_slabs);
    p.n_splits = static_cast<int32_t>((T_tot + p.split_tokens - 1) / p.split_tokens);
    p.parts_stride = p.n_splits;
  } else {
    p.stream = 1;
    p.units_per_slab = static_cast<int32_t>((T_qt + kStreamUnitTokens - 1) / kStreamUnitTokens);
    p.n_units = n_slabs * p.units_per_slab;
    const int sms = sm_count < 1 ? 1 : (sm_count > kMaxSMs ? kMaxSMs : sm_count);
    const int64_t warps = static_cast<int64_t>(sms) * kStreamCtasPerSM * kStreamWarps;
    int64_t run = (p.n_units + warps - 1) / warps;
    if (run < kMinRunUnits) run = kMinRunUnits;
    if (force_run_units > 0) run = force_run_units;
    p.run_units = static_cast<int32_t>(run);
    p.n_runs = static_cast<int32_t>((p.n_units + run - 1) / run);
    p.parts_stride = p.units_per_slab > 0 ? static_cast<int32_t>((p.units_per_slab + run - 1) / run) + 1 : 1;
  }
  p.records = n_slabs * p.parts_stride * kMaxRep;
  return p;
}

int64_t max_decode_records(int64_t max_slabs, int64_t max_tokens, bool stp) {
  if (max_tokens < 1) max_tokens = 1;
  // Stream kernel: parts per slab = ceil(S / run) + 1 with run >= max(1, n_units / warps) (the
  // chooser never goes below kMinRunUnits, the test hook may force 1), so
  // slabs * parts <= min(slabs * S, warps + slabs) + slabs for every S.
  const int64_t S = (max_tokens + kStreamUnitTokens - 1) / kStreamUnitTokens;
  const int64_t warps = static_cast<int64_t>(kMaxSMs) * kStreamCtasPerSM * kStreamWarps;
  int64_t parts = max_slabs * S;
  if (parts > warps + max_slabs) parts = warps + max_slabs;
  parts += max_slabs;
  if (stp) {
    // Split kernel: 640-token splits give slabs * ceil(T / 640) records; 320- and 160-token splits
    // are only chosen while the coarser size yields fewer than 592 CTAs, i.e. below 1184 of them.
    int64_t sp = max_slabs * ((max_tokens + 639) / 640);
    if (sp < 1184) sp = 1184;
    if (sp > parts) parts = sp;
  }
  return parts * kMaxRep;
}

// ---------------------------------------------------------------------------------
// One block of 128 threads per slab = (layer, batch element, KV head), serving its query heads.
// Residual tokens (stream plan): thread t scores token t against every head, a warp per head
// finds the maximum over the residual scores and the records' maxima and turns the scores into
// probabilities, thread c accumulates channel c of P V_r; then the records join with their
// weights 2^(m_record - M).  Scores and maxima are base-2 logits (score * scale * log2 e).
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kD) decode_merge_kernel(DecodeArgs a, int with_residual) {
  __shared__ float qs[kMaxRep][kD];
  __shared__ float P[kMaxRep][kR];
  __shared__ float Mh[kMaxRep], Lh[kMaxRep];
  const CacheView& cv = a.cv;
  const int slab = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = slab % cv.H_kv, lb = slab / cv.H_kv, rep = cv.rep;
  const uint8_t* slab_ptr = cv.base + cv.slab_offset + (static_cast<int64_t>(a.layer0) * cv.B * cv.H_kv + slab) * cv.slab_stride;
  const int n_res = with_residual ? a.st.n_res : 0;
  int n_parts;
  {
    const DecodePlan& pl = a.plan;
    if (!pl.stream) n_parts = pl.n_splits;
    else if (pl.units_per_slab == 0) n_parts = 0;
    else {
      const int64_t u0 = static_cast<int64_t>(slab) * pl.units_per_slab;
      n_parts = static_cast<int>((u0 + pl.units_per_slab - 1) / pl.run_units - u0 / pl.run_units) + 1;
    }
  }
  const float* rec = a.partials + static_cast<int64_t>(slab) * a.plan.parts_stride * (kMaxRep * kRecordFloats);
  const int64_t q0 = (static_cast<int64_t>(lb) * cv.H_q + h * rep) * kD;
  if (n_res > 0) {
    const T* qp = reinterpret_cast<const T*>(a.q) + q0;
    for (int k = 0; k < rep; ++k) qs[k][tid] = Elem<T>::to_float(qp[k * kD + tid]);
    __syncthreads();
    if (tid < n_res) {
      const uint4* kr = reinterpret_cast<const uint4*>(slab_ptr + cv.kres_offset) + tid * (kD / 8);
      float acc[kMaxRep];
#pragma unroll
      for (int k = 0; k < kMaxRep; ++k) acc[k] = 0.0f;
      for (int c8 = 0; c8 < kD / 8; ++c8) {
        const uint4 v = __ldg(kr + c8);
        const float2 x0 = Elem<T>::to_float2(v.x), x1 = Elem<T>::to_float2(v.y);
        const float2 x2 = Elem<T>::to_float2(v.z), x3 = Elem<T>::to_float2(v.w);
#pragma unroll
        for (int k = 0; k < kMaxRep; ++k) {
          if (k < rep) {
            const float4 qa = *reinterpret_cast<const float4*>(&qs[k][c8 * 8]);
            const float4 qb = *reinterpret_cast<const float4*>(&qs[k][c8 * 8 + 4]);
            acc[k] += qa.x * x0.x + qa.y * x0.y + qa.z * x1.x + qa.w * x1.y + qb.x * x2.x + qb.y * x2.y + qb.z * x3.x +
                      qb.w * x3.y;
          }
        }
      }
      const float sl2 = a.scale * 1.4426950408889634f;
#pragma unroll
      for (int k = 0; k < kMaxRep; ++k)
        if (k < rep) P[k][tid] = acc[k] * sl2;
    }
    __syncthreads();
  }
  // maxima and denominators: warp w takes heads w and w + 4
  for (int k = warp; k < rep; k += kD / 32) {
    float m = -INFINITY;
    for (int t = lane; t < n_res; t += 32) m = fmaxf(m, P[k][t]);
    for (int j = lane; j < n_parts; j += 32) m = fmaxf(m, rec[(j * kMaxRep + k) * kRecordFloats]);
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.0f;
    for (int t = lane; t < n_res; t += 32) {
      const float p = exp2f(P[k][t] - m);
      P[k][t] = p;
      l += p;
    }
    for (int j = lane; j < n_parts; j += 32) {
      const float* pr = rec + (j * kMaxRep + k) * kRecordFloats;
      l += pr[1] * exp2f(pr[0] - m);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) { Mh[k] = m; Lh[k] = l; }
  }
  __syncthreads();
  float o[kMaxRep];
#pragma unroll
  for (int k = 0; k < kMaxRep; ++k) o[k] = 0.0f;
  if (n_res > 0) {
    const T* vres = reinterpret_cast<const T*>(slab_ptr + cv.vres_offset) + tid;
    for (int t = 0; t < n_res; ++t) {
      const float v = Elem<T>::to_float(vres[t * kD]);
#pragma unroll
      for (int k = 0; k < kMaxRep; ++k)
        if (k < rep) o[k] += P[k][t] * v;
    }
  }
  for (int j = 0; j < n_parts; ++j) {
#pragma unroll
    for (int k = 0; k < kMaxRep; ++k) {
      if (k < rep) {
        const float* pr = rec + (j * kMaxRep + k) * kRecordFloats;
        o[k] += exp2f(pr[0] - Mh[k]) * pr[2 + tid];
      }
    }
  }
#pragma unroll
  for (int k = 0; k < kMaxRep; ++k) {
    if (k < rep) {
      const float v = o[k] / Lh[k];
      const int64_t i = q0 + k * kD + tid;
      if (a.out_dtype == VIDKV_F32) reinterpret_cast<float*>(a.out)[i] = v;
      else if (a.out_dtype == VIDKV_F16) reinterpret_cast<__half*>(a.out)[i] = __float2half_rn(v);
      else reinterpret_cast<__nv_bfloat16*>(a.out)[i] = __float2bfloat16_rn(v);
    }
  }
}

cudaError_t launch_decode(const DecodeArgs& a_in, cudaStream_t stream) {
  DecodeArgs a = a_in;
  cudaError_t e;
  const int n_slabs = a.n_layers * a.cv.B * a.cv.H_kv;
  if (a.plan.n_chunks > 0) {
    if ((e = launch_decode_prep(a, stream)) != cudaSuccess) return e;
    if (a.ev_begin) cudaEventRecord(a.ev_begin, stream);
    e = a.plan.stream ? launch_decode_stream(a, stream) : launch_decode_stp(a, stream);
    if (a.ev_end) cudaEventRecord(a.ev_end, stream);
    if (e != cudaSuccess) return e;
  }
  count_launches(1);
  const int with_residual = a.plan.stream;
  if (a.in_dtype == VIDKV_F16) decode_merge_kernel<__half><<<n_slabs, kD, 0, stream>>>(a, with_residual);
  else decode_merge_kernel<__nv_bfloat16><<<n_slabs, kD, 0, stream>>>(a, with_residual);
  return cudaGetLastError();
}

}  // namespace vidkv
