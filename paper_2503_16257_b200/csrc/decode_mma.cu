// Decode attention over the packed cache on the tensor cores (Algorithm 1 "Decoding",
// Eq. 3), split-KV: decode_mma_kernel for caches without protected tokens, decode_stp_kernel
// for caches with them (STPQuant), decode_prep_kernel for the per-chunk query images.
//
// The packed codes never become FP16 K or V in memory.  They are expanded in registers to
// small exact binary16 numbers and fed to mma.sync.m16n8k16 as one operand; everything that
// depends on the query or on the per-group metadata goes into the other operand:
//
//   scores (transposed: rows = query heads, columns = tokens)
//     anomalous channels  sum_j q_j (s_j code_j + z_j)
//                         = sum_j (q_j s_j) (4 + code_j) + sum_j q_j z_j - 4 sum_j q_j s_j
//       codes come out of the 2-bit words with one shift and one mask as 4 + code in binary16;
//       q_j s_j is formed per 32-token group as an exact pair hi + lo of binary16 numbers
//       (rows 0-7 of the A operand carry hi, rows 8-15 lo, the two halves of the accumulator
//       are added afterwards); the two constants come from one more MMA whose B operand is the
//       raw z and s metadata;
//     normal channels     K' = IDFT(+-s), so q . K'_t = sum_f Q_f s_f (+-1) with Q the
//       weighted forward transform of the permuted query (decode_prep_kernel, once per chunk);
//       the sign bits become +-1.0 with one shift and one mask.
//   P V (rows = channels, columns = query heads)
//     each byte of the ternary plane holds the digits of five groups; they are peeled with a
//     multiply by 3 per digit on two bytes at a time (16-bit lanes) and leave 4 + digit =
//     5 + trit in binary16; the 5 is removed through the accumulator's initial value
//     -5 sum_t p_t, and the per-(group, channel) scale multiplies the group's accumulator.
//
// One CTA (4 warps) walks one or more consecutive splits of the token axis of one (layer, batch
// element, KV head).  A split's key groups, then its ternary supergroups, are copied into the same
// shared-memory buffer with cp.async; phase 1 (warps split the 32-token groups) writes scores, a
// softmax pass turns them into binary16 probabilities in place, phase 2 (warps split the channels)
// accumulates P V.  With protected tokens the probabilities are scattered into stream order and
// the protected 2-bit groups are read from global memory as they are consumed.
#include "decode_common.cuh"

namespace vidkv {

namespace {
}  // namespace

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
// Per-thread view of one split: which tokens it covers and where its slab lives.
// ---------------------------------------------------------------------------------
struct Split {
  int tid, lane, warp, hd, r;             // hd = lane / 4 (MMA row group), r = lane % 4
  uint32_t m_field, c_four, m_sign, c_neg1;
  int split, slab, h, lb, rep;
  const uint8_t* slab_ptr;
  int64_t T_q0, T_qt, t0, t1, tq1, gk0;   // prefill-quantized / all quantized tokens; split range; first key group
  int n_loc, nq, n_kg;                    // tokens, quantized tokens, key groups in the split
};

__device__ __forceinline__ Split make_split(const DecodeArgs& a, int split) {
  Split c;
  c.tid = threadIdx.x; c.lane = c.tid & 31; c.warp = c.tid >> 5; c.hd = c.lane >> 2; c.r = c.lane & 3;
  c.m_field = kExpand[0]; c.c_four = kExpand[1]; c.m_sign = kExpand[2]; c.c_neg1 = kExpand[3];
  c.split = split; c.slab = blockIdx.y;
  const CacheView& cv = a.cv;
  c.h = c.slab % cv.H_kv; c.lb = c.slab / cv.H_kv; c.rep = cv.rep;
  c.slab_ptr = cv.slab(a.layer0 + c.lb / cv.B, c.lb % cv.B, c.h);
  c.T_q0 = a.st.T_q0;
  c.T_qt = c.T_q0 + a.st.n_flush * kR;
  const int64_t T_tot = c.T_qt + a.st.n_res;
  c.t0 = static_cast<int64_t>(c.split) * a.plan.split_tokens;
  c.t1 = min(c.t0 + a.plan.split_tokens, T_tot);
  c.tq1 = max(min(c.t1, c.T_qt), c.t0);
  c.n_loc = static_cast<int>(c.t1 - c.t0);
  c.nq = static_cast<int>(c.tq1 - c.t0);
  c.n_kg = c.nq / kG;
  c.gk0 = c.t0 / kG;
  return c;
}

// qexp[k] = head_exponent of query head k of the CTA's slab (0 for a head that does not exist);
// warp w fills entries 2 w and 2 w + 1.
template <typename T>
__device__ __forceinline__ void query_exponents(const DecodeArgs& a, const Split& c, int* qexp) {
  const T* qp = reinterpret_cast<const T*>(a.q) + (static_cast<int64_t>(c.lb) * a.cv.H_q + c.h * c.rep) * kD;
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    const int k = 2 * c.warp + hh;
    const int e = head_exponent<T, 32>(qp + k * kD, c.lane, k < c.rep);
    if (c.lane == 0) qexp[k] = e;
  }
}

// Phase 1: raw scores q . k (before the softmax scale, in units of the head's query normalisation
// 2^(-qexp[head] - kQShift)) of every token of the split into S[head][token - t0]: the packed key
// groups staged in kbuf, then the FP16 / BF16 residual rows.
template <typename T>
__device__ __forceinline__ void score_phase(const DecodeArgs& a, int n_chunks, const Split& c, const uint8_t* kbuf,
                                            float* S, int SS, const int* qexp) {
  const CacheView& cv = a.cv;
  const int lane = c.lane, warp = c.warp, hd = c.hd, r = c.r, slab = c.slab, h = c.h, lb = c.lb, rep = c.rep;
  const uint32_t m_field = c.m_field, c_four = c.c_four, m_sign = c.m_sign, c_neg1 = c.c_neg1;
  const uint8_t* slab_ptr = c.slab_ptr;
  const int64_t T_q0 = c.T_q0, T_qt = c.T_qt, t0 = c.t0, t1 = c.t1, gk0 = c.gk0;
  const int n_kg = c.n_kg;
  {
    const int64_t g0n = T_q0 / kG;                        // key groups of the prefill chunk
    int cur_chunk = -1;
    uint32_t qa[8], qha[8], qhb[8];
    for (int g = warp; g < n_kg; g += 4) {
      const int64_t gidx = gk0 + g;
      const int chunk = gidx < g0n ? 0 : 1 + static_cast<int>((gidx - g0n) / (kR / kG));
      if (chunk != cur_chunk) {
        cur_chunk = chunk;
        const uint32_t* pp = a.prep + (static_cast<int64_t>(slab) * n_chunks + chunk) * (kPrepWords * 32) + lane;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          qa[i] = __ldg(pp + i * 32);
          qha[i] = __ldg(pp + (8 + i) * 32);
          qhb[i] = __ldg(pp + (16 + i) * 32);
        }
      }
      const uint8_t* kg = kbuf + g * kKGroupBytes;
      uint32_t s2[8], z2[8], s1[8];
      {
        const uint4 x0 = *reinterpret_cast<const uint4*>(kg + kKG_S2 + 32 * r);
        const uint4 x1 = *reinterpret_cast<const uint4*>(kg + kKG_S2 + 32 * r + 16);
        s2[0] = x0.x; s2[1] = x0.y; s2[2] = x0.z; s2[3] = x0.w; s2[4] = x1.x; s2[5] = x1.y; s2[6] = x1.z; s2[7] = x1.w;
        const uint8_t* zs = kg + ((hd & 1) ? kKG_S2 : kKG_Z2) + 32 * r;   // B operand of the constants: z for even columns, s for odd
        const uint4 y0 = *reinterpret_cast<const uint4*>(zs);
        const uint4 y1 = *reinterpret_cast<const uint4*>(zs + 16);
        z2[0] = y0.x; z2[1] = y0.y; z2[2] = y0.z; z2[3] = y0.w; z2[4] = y1.x; z2[5] = y1.y; z2[6] = y1.z; z2[7] = y1.w;
        const uint4 w0 = *reinterpret_cast<const uint4*>(kg + kKG_S1 + 32 * r);
        const uint4 w1 = *reinterpret_cast<const uint4*>(kg + kKG_S1 + 32 * r + 16);
        s1[0] = w0.x; s1[1] = w0.y; s1[2] = w0.z; s1[3] = w0.w; s1[4] = w1.x; s1[5] = w1.y; s1[6] = w1.z; s1[7] = w1.w;
      }
      // constants of the group: column 2 r of the result = sum q z, column 2 r + 1 = sum q s
      float cst;
      {
        float cz[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) mma_f16(cz, qa[2 * ks], 0u, qa[2 * ks + 1], 0u, z2[2 * ks], z2[2 * ks + 1]);
        cst = cz[0] - 4.0f * cz[1];
      }
      // q s as exact binary16 pairs hi + lo
      uint32_t hi2[8], lo2[8], hi1[8], lo1[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        hi2[i] = hmul2_u(qa[i], s2[i]);
        lo2[i] = hfms2_u(qa[i], s2[i], hi2[i]);
        hi1[i] = hmul2_u(qha[i], s1[i]);
        lo1[i] = hfma2_u(qhb[i], s1[i], hfms2_u(qha[i], s1[i], hi1[i]));
      }
      const uint4 c2 = *reinterpret_cast<const uint4*>(kg + kKG_Codes2 + lane * 16);
      const uint2 c1 = *reinterpret_cast<const uint2*>(kg + kKG_Bits1 + lane * 8);
      const uint32_t w2[4] = {c2.x, c2.y, c2.z, c2.w};
      const uint32_t h1[4] = {c1.x & 0xffffu, c1.x >> 16, c1.y & 0xffffu, c1.y >> 16};
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        float acc[4];
        const uint32_t w = w2[nt];
        uint32_t x[8];
        x[0] = and_or(w << 8, m_field, c_four);
        x[1] = and_or(w << 6, m_field, c_four);
        x[2] = and_or(w << 4, m_field, c_four);
        x[3] = and_or(w << 2, m_field, c_four);
        x[4] = and_or(w, m_field, c_four);
        x[5] = and_or(w >> 2, m_field, c_four);
        x[6] = and_or(w >> 4, m_field, c_four);
        x[7] = and_or(w >> 6, m_field, c_four);
        mma_f16_c(acc, hi2[0], lo2[0], hi2[1], lo2[1], x[0], x[1], cst, cst, 0.0f, 0.0f);
#pragma unroll
        for (int ks = 1; ks < 4; ++ks)
          mma_f16(acc, hi2[2 * ks], lo2[2 * ks], hi2[2 * ks + 1], lo2[2 * ks + 1], x[2 * ks], x[2 * ks + 1]);
        // sign bits: low lane <- bit 15 - 2 m, high lane <- bit 14 - 2 m of the half-word
        const uint32_t X = h1[nt] * 0x00020001u;
        uint32_t y[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) y[m] = and_xor(X << (2 * m), m_sign, c_neg1);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_f16(acc, hi1[2 * ks], lo1[2 * ks], hi1[2 * ks + 1], lo1[2 * ks + 1], y[2 * ks], y[2 * ks + 1]);
        *reinterpret_cast<float2*>(S + hd * SS + g * kG + nt * 8 + 2 * r) = make_float2(acc[0] + acc[2], acc[1] + acc[3]);
      }
    }
  }
  // residual tokens of this split: q . k on the tensor cores straight from the FP16 / BF16 rows
  if (t1 > T_qt) {
    const int r_begin = static_cast<int>(max(t0, T_qt) - T_qt), r_end = static_cast<int>(t1 - T_qt);
    const T* kres = reinterpret_cast<const T*>(slab_ptr + cv.kres_offset);
    const T* qp = reinterpret_cast<const T*>(a.q) + (static_cast<int64_t>(lb) * cv.H_q + h * rep) * kD;
    uint32_t qn[16];
#pragma unroll
    for (int i = 0; i < 16; ++i)
      qn[i] = hd < rep ? __ldg(reinterpret_cast<const uint32_t*>(qp + hd * kD + 8 * i + 2 * r)) : 0u;
    const float qf = pow2i(-qexp[hd] - kQShift);                         // the raw query is used here: same units as above
    const int n_tiles = (r_end - r_begin + 7) / 8;
    for (int tile = warp; tile < n_tiles; tile += 4) {
      const int row = min(r_begin + tile * 8 + hd, r_end - 1);          // clamped: extra columns are dropped
      const uint32_t* kr = reinterpret_cast<const uint32_t*>(kres + static_cast<int64_t>(row) * kD) + r;
      float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) mma_in<T>(acc, qn[2 * ks], qn[2 * ks + 1], kr[ks * 8], kr[ks * 8 + 4]);
      const int c0 = r_begin + tile * 8 + 2 * r;
      float* srow = S + hd * SS + static_cast<int>(T_qt - t0);
      if (c0 < r_end) srow[c0] = acc[0] * qf;
      if (c0 + 1 < r_end) srow[c0 + 1] = acc[1] * qf;
    }
  }
}

// Phase 2, ternary stream: tot[i][.] += sum over n_sg staged supergroups of s * (P V) for the
// warp's 32 channels.  prow = this lane's probability row (binary16), its entry 0 matching
// token 0 of the first staged supergroup; psum = -5 * group sums of those probabilities,
// [group][8 heads]; groups from n_grp on do not exist (zero scale).
// With MASKED, groups before g_first hold no token of this split either: their MMAs, loads and
// scale steps are skipped (the digit peel still has to pass over them).
template <bool MASKED>
__device__ __forceinline__ void ternary_phase(const Split& c, const uint8_t* vbuf, int n_sg, int g_first, int n_grp,
                                              const uint8_t* prow, const float* psum, float (&tot)[2][4]) {
  const int warp = c.warp, hd = c.hd, r = c.r;
  const uint32_t m_field = c.m_field, c_four = c.c_four;
  {
    for (int sg = 0; sg < n_sg; ++sg) {
      const uint8_t* sgp = vbuf + sg * kSGBytes;
      const int n_valid = min(kSGGroups, n_grp - sg * kSGGroups);
      const int g_lo = MASKED ? g_first - sg * kSGGroups : 0;
      float acc[kSGGroups][2][4];
      float2 ps[kSGGroups];
#pragma unroll
      for (int g = 0; g < kSGGroups; ++g)
        ps[g] = *reinterpret_cast<const float2*>(psum + (sg * kSGGroups + g) * 8 + 2 * r);
#pragma unroll
      for (int kt = 0; kt < 2; ++kt) {
        const uint2 wa = *reinterpret_cast<const uint2*>(sgp + ((((kt * 2 + 0) * 4 + warp) * 4 + r) * 8 + hd) * 8);
        const uint2 wb = *reinterpret_cast<const uint2*>(sgp + ((((kt * 2 + 1) * 4 + warp) * 4 + r) * 8 + hd) * 8);
        uint32_t W[8];
        W[0] = prmt(wa.x, 0u, 0x4140u); W[1] = prmt(wa.x, 0u, 0x4342u);
        W[2] = prmt(wb.x, 0u, 0x4140u); W[3] = prmt(wb.x, 0u, 0x4342u);
        W[4] = prmt(wa.y, 0u, 0x4140u); W[5] = prmt(wa.y, 0u, 0x4342u);
        W[6] = prmt(wb.y, 0u, 0x4140u); W[7] = prmt(wb.y, 0u, 0x4342u);
#pragma unroll
        for (int k = 0; k < 8; ++k) W[k] = mad_u32(W[k], 3u, 0u);          // 3 * byte per 16-bit lane
#pragma unroll
        for (int g = 0; g < kSGGroups; ++g) {
          if (MASKED && g >= n_valid) continue;
          uint32_t A[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            // W holds 3 * (remaining byte) per 16-bit lane; the digit sits at bits 8-9.
            // Next W = 3 * (W - digit << 8) = 3 W - 3 A + 3 * 0x4400 (no lane ever borrows).
            // Half of the lanes take that route (two multiply-adds), the other half mask the digit
            // away and multiply (one logic, one multiply-add): the two pipes share the work evenly.
            A[k] = and_or(W[k], m_field, c_four);
            if (k & 1) W[k] = mad_u32(A[k], 0xfffffffdu, mad_u32(W[k], 3u, 0xcc00cc00u));
            else W[k] = mad_u32(W[k] & 0x00ff00ffu, 3u, 0u);
          }
          if (MASKED && g < g_lo) continue;
          // groups past the end of the cache meet zero probabilities (and a zero scale below)
          const uint8_t* pb = prow + (sg * (kSGGroups * kG) + g * kG + kt * 16 + 2 * r) * 2;
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(pb);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(pb + 16);
          if (kt == 0) {
            mma_f16_c(acc[g][0], A[0], A[1], A[2], A[3], b0, b1, ps[g].x, ps[g].y, ps[g].x, ps[g].y);
            mma_f16_c(acc[g][1], A[4], A[5], A[6], A[7], b0, b1, ps[g].x, ps[g].y, ps[g].x, ps[g].y);
          } else {
            mma_f16(acc[g][0], A[0], A[1], A[2], A[3], b0, b1);
            mma_f16(acc[g][1], A[4], A[5], A[6], A[7], b0, b1);
          }
        }
      }
#pragma unroll
      for (int g = 0; g < kSGGroups; ++g) {
        if (!MASKED || (g >= g_lo && g < n_valid)) {
          uint2 sc = *reinterpret_cast<const uint2*>(sgp + kSG_Scales + g * (kD * 2) + (32 * warp + 4 * hd) * 2);
          if (g >= n_valid) sc = make_uint2(0u, 0u);
          const float2 sa = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));
          const float2 sb = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));
          tot[0][0] += sa.x * acc[g][0][0]; tot[0][1] += sa.x * acc[g][0][1];
          tot[0][2] += sa.y * acc[g][0][2]; tot[0][3] += sa.y * acc[g][0][3];
          tot[1][0] += sb.x * acc[g][1][0]; tot[1][1] += sb.x * acc[g][1][1];
          tot[1][2] += sb.y * acc[g][1][2]; tot[1][3] += sb.y * acc[g][1][3];
        }
      }
    }
  }
}

// P V of the FP16 / BF16 residual rows of the split, added to tot.  The probability of
// residual row rr and head k is pres[k * pres_stride + pres_index0 + rr] (binary16).  Thread =
// channel computes the eight heads' sums into O[head][channel] (the staging buffer, which must
// be free), then every thread picks up the entries of its accumulator layout.  All threads
// call it or none.
template <typename T>
__device__ __forceinline__ void residual_pv(const DecodeArgs& a, const Split& c, float* O, const __half* pres,
                                            int pres_stride, int pres_index0, float (&tot)[2][4]) {
  const CacheView& cv = a.cv;
  const int ch = c.tid;
  const int r_begin = static_cast<int>(max(c.t0, c.T_qt) - c.T_qt), r_end = static_cast<int>(c.t1 - c.T_qt);
  const T* vres = reinterpret_cast<const T*>(c.slab_ptr + cv.vres_offset);
  float o[kMaxRep];
#pragma unroll
  for (int k = 0; k < kMaxRep; ++k) o[k] = 0.0f;
  for (int rr = r_begin; rr < r_end; ++rr) {
    const float v = Elem<T>::to_float(vres[rr * kD + ch]);
#pragma unroll
    for (int k = 0; k < kMaxRep; ++k) o[k] += __half2float(pres[k * pres_stride + pres_index0 + rr]) * v;
  }
#pragma unroll
  for (int k = 0; k < kMaxRep; ++k) O[k * kD + ch] = o[k];
  __syncthreads();
  const int c0 = 32 * c.warp + 4 * c.hd, r = c.r;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    tot[i][0] += O[(2 * r) * kD + c0 + 2 * i];
    tot[i][1] += O[(2 * r + 1) * kD + c0 + 2 * i];
    tot[i][2] += O[(2 * r) * kD + c0 + 2 * i + 1];
    tot[i][3] += O[(2 * r + 1) * kD + c0 + 2 * i + 1];
  }
  __syncthreads();
}

// Write one partial record per query head: (max, sum, unnormalised out[128]).  ml[h] = maximum
// (base-2 logit), ml[8 + h] = sum of the probabilities; O is the staging buffer (free, 4 KB).
__device__ __forceinline__ void write_partial(const DecodeArgs& a, const Split& c, int part, float* O, const float* ml,
                                              const float (&tot)[2][4]) {
  const int c0 = 32 * c.warp + 4 * c.hd, r = c.r;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    O[(2 * r) * kD + c0 + 2 * i] = tot[i][0];
    O[(2 * r + 1) * kD + c0 + 2 * i] = tot[i][1];
    O[(2 * r) * kD + c0 + 2 * i + 1] = tot[i][2];
    O[(2 * r + 1) * kD + c0 + 2 * i + 1] = tot[i][3];
  }
  __syncthreads();
  const int ch = c.tid;
#pragma unroll
  for (int k = 0; k < kMaxRep; ++k) {
    if (k < c.rep) {
      float* pr = a.partials + ((static_cast<int64_t>(c.slab) * a.plan.parts_stride + part) * kMaxRep + k) * kRecordFloats;
      pr[2 + ch] = O[k * kD + ch];
      if (ch == 0) { pr[0] = ml[k]; pr[1] = ml[8 + k]; }
    }
  }
}

// Softmax numerators of the 8 score rows (warp w owns rows 2 w and 2 w + 1): p = exp(scale *
// (score - row max)), rounded to binary16.  Without protected tokens the probabilities
// replace the scores in place (entry i of the row, as binary16).  With them (STP) the row is
// cleared once its scores are in registers and becomes the ternary-stream row: quantized
// tokens [0, nq) go to their stream position through `map` (bit 15 = protected stream, row of
// Pprot), residual tokens [nq, n_loc) to Pres[row][i - nq].
// red[row] = row maximum as a base-2 logit (score * scale * log2 e), red[8 + row] = sum of the probabilities.  The scores arrive in
// units of the head's query normalisation; the inverse power of two joins the softmax scale.
template <bool STP, bool FULL = false>     // FULL: the split holds exactly 640 tokens, no bound checks
__device__ __forceinline__ void softmax_phase(const DecodeArgs& a, const Split& c, float* S, int SS, float* red,
                                              int n_pad, const uint16_t* map, __half* Pprot, int PP, __half* Pres,
                                              int PRS, const int* qexp) {
  const int lane = c.lane, n_loc = c.n_loc;
  constexpr int kMaxPairs = 10;                                          // ST <= 640: 320 pairs per row
#pragma unroll 1
  for (int hh = 0; hh < 2; ++hh) {
    const int row_h = c.warp * 2 + hh;
    const float scale_h = a.scale * pow2i(qexp[row_h] + kQShift);
    const float sl2 = scale_h * 1.4426950408889634f;
    float* row = S + row_h * SS;
    float2 v[kMaxPairs];
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < kMaxPairs; ++k) {
      const int i = 2 * lane + 64 * k;
      if (FULL) {
        v[k] = *reinterpret_cast<const float2*>(row + i);
      } else {
        v[k] = i < n_loc ? *reinterpret_cast<const float2*>(row + i) : make_float2(-INFINITY, -INFINITY);
        if (i + 1 >= n_loc) v[k].y = -INFINITY;
      }
      m = fmaxf(m, fmaxf(v[k].x, v[k].y));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    __syncwarp();
    if (STP) {
      for (int i = lane; i < SS / 4; i += 32) reinterpret_cast<uint4*>(row)[i] = make_uint4(0u, 0u, 0u, 0u);
      __syncwarp();
    }
    const float ms = m * sl2;
    float l = 0.0f;
    uint32_t* prow = reinterpret_cast<uint32_t*>(row);
    __half* trow = reinterpret_cast<__half*>(row);
#pragma unroll
    for (int k = 0; k < kMaxPairs; ++k) {
      const int i = 2 * lane + 64 * k;
      const float p0 = ex2_approx(fmaf(v[k].x, sl2, -ms)), p1 = ex2_approx(fmaf(v[k].y, sl2, -ms));
      l += p0 + p1;
      if (STP) {
        if (i < c.nq) {
          const uint32_t d = *reinterpret_cast<const uint32_t*>(map + i);
          const uint32_t d0 = d & 0xffffu, d1 = d >> 16;
          __half* q0 = (d0 & 0x8000u) ? Pprot + row_h * PP + (d0 & 0x7fffu) : trow + d0;
          __half* q1 = (d1 & 0x8000u) ? Pprot + row_h * PP + (d1 & 0x7fffu) : trow + d1;
          *q0 = __float2half_rn(p0);
          *q1 = __float2half_rn(p1);
        } else if (i < n_loc) {
          *reinterpret_cast<uint32_t*>(Pres + row_h * PRS + (i - c.nq)) = pack_half2(p0, p1);
        }
      } else if (FULL || i < n_pad) {
        prow[i >> 1] = pack_half2(p0, p1);
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) { red[row_h] = m * sl2; red[8 + row_h] = l; }
  }
}

// out[g * 8 + head] = factor * sum of the 32 binary16 entries of group g of every row
__device__ __forceinline__ void group_sums(const Split& c, const __half* P, int row_stride, int n_groups, float factor,
                                           float* out) {
  for (int i = c.tid; i < n_groups * 8; i += kThreads) {
    const int g = i >> 3, hh = i & 7;
    const uint4* pr = reinterpret_cast<const uint4*>(P + hh * row_stride + g * kG);   // 64 bytes, 16-byte aligned
    float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 v = pr[k];
      const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
      const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
      const float2 f2 = __half22float2(*reinterpret_cast<const __half2*>(&v.z));
      const float2 f3 = __half22float2(*reinterpret_cast<const __half2*>(&v.w));
      s0 += (f0.x + f0.y) + (f1.x + f1.y);
      s1 += (f2.x + f2.y) + (f3.x + f3.y);
    }
    out[i] = factor * (s0 + s1);
  }
}

// ---------------------------------------------------------------------------------
// Caches with protected tokens (STPQuant, Algorithm 2).  The values of the split's tokens sit
// in two streams whose order differs from the key order: unprotected tokens in the ternary
// stream (position = token - protected tokens before it; flushed tokens follow from the next
// group boundary), protected ones in 2-bit groups.  The probabilities are therefore scattered
// into stream-ordered rows, zero wherever a staged stream position belongs to another split.
// Shared memory for a split of ST tokens (160, 320 or 640):
//   buf   ST/32 key groups, then ST/160 + 2 ternary supergroups, at the end the output staging
//   S     8 rows of SSP floats: scores, then the row's probabilities as binary16 in three pieces:
//         [0, 160 n_sg) the staged ternary stream, then 32 n_pg entries of the protected stream,
//         then the residual tokens.  The pieces hold the split's tokens plus the slack of their
//         group alignment: at most ST + 349 + 62 + 2 entries.
//   map   ST destinations                            psum_t, psum_p, red, qexp
// The protected groups are read from global memory as they are consumed.
// ---------------------------------------------------------------------------------
__host__ __device__ inline int stp_sg_max(int ST) { return ST / 160 + 2; }
__host__ __device__ inline int stp_pg_max(int ST) { return ST / 32 + 1; }
__host__ __device__ inline int stp_row_floats(int ST) {       // a row must hold the scores and, later, the streams
  const int scores = ST + 4;
  const int streams = ((ST + 349 + 62 + 2 + 1) / 2 + 7) / 8 * 8 + 4;   // = 4 mod 8 floats: the 8 rows start in different banks
  return scores > streams ? scores : streams;
}

size_t decode_stp_smem_bytes(int ST) {
  const size_t buf = static_cast<size_t>(stp_sg_max(ST)) * kSGBytes;        // >= ST/32 key groups
  return buf + sizeof(float) * 8 * stp_row_floats(ST) + 2 * ST +
         sizeof(float) * (8 * stp_sg_max(ST) * kSGGroups + 8 * stp_pg_max(ST) + 16 + 8);
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 4) decode_stp_kernel(DecodeArgs a, int n_chunks) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int ST = a.plan.split_tokens;
  const int SS = stp_row_floats(ST);
  const int PT = 2 * SS;                                   // row stride in binary16 entries
  uint8_t* buf = smem_raw;
  float* S = reinterpret_cast<float*>(buf + stp_sg_max(ST) * kSGBytes);
  uint16_t* map = reinterpret_cast<uint16_t*>(S + 8 * SS);
  float* psum_t = reinterpret_cast<float*>(map + ST);
  float* psum_p = psum_t + 8 * stp_sg_max(ST) * kSGGroups;
  float* red = psum_p + 8 * stp_pg_max(ST);
  int* qexp = reinterpret_cast<int*>(red + 16);
  const Split c = make_split(a, blockIdx.x);
  query_exponents<T>(a, c, qexp);                          // visible after the barrier before the scores
  const CacheView& cv = a.cv;
  const int b = c.lb % cv.B;
  const uint32_t* ew = cv.e_words(b);
  const uint32_t* ep = cv.e_prefix(b);

  // ---- keys first
  {
    const uint8_t* ksrc = c.slab_ptr + cv.kgroup_offset + c.gk0 * kKGroupBytes;
    stage_async(buf, ksrc, c.n_kg * (kKGroupBytes / 16), c.tid);
    cp_async_commit();
  }
  // ---- where the split's tokens sit in the two value streams
  const int64_t tp0 = min(c.t0, c.T_q0), tp1 = min(c.tq1, c.T_q0);              // prefill part
  const int64_t pp0 = ep[tp0 / kG], pp1 = ep[tp1 / kG];                         // protected positions
  const int64_t n_rest = c.T_q0 - a.n_prot;
  const int64_t u_fl0 = (n_rest + kG - 1) / kG * kG;                            // flushed tokens start here
  const int64_t ua0 = tp0 - pp0, ua1 = tp1 - pp1;
  const int64_t tf0 = max(c.t0, c.T_q0), tf1 = max(c.tq1, tf0);                 // flushed part
  const int64_t ub0 = u_fl0 + (tf0 - c.T_q0), ub1 = u_fl0 + (tf1 - c.T_q0);
  const bool has_a = ua1 > ua0, has_b = tf1 > tf0;
  const int64_t U0 = has_a ? ua0 : (has_b ? ub0 : 0), U1 = has_b ? ub1 : (has_a ? ua1 : 0);
  const int64_t sgA = U0 / (kG * kSGGroups);
  const int n_sg = U1 > U0 ? static_cast<int>((U1 - 1) / (kG * kSGGroups) - sgA + 1) : 0;
  const int64_t Ubase = sgA * (kG * kSGGroups);
  const int64_t pgA = pp0 / kG;
  const int n_pg = pp1 > pp0 ? static_cast<int>((pp1 - 1) / kG - pgA + 1) : 0;
  const int64_t Pbase = pgA * kG;
  const int64_t tg_total = (n_rest + kG - 1) / kG + (kR / kG) * a.st.n_flush;   // ternary groups that exist
  // the protected and the residual probabilities follow the staged ternary stream in each row of S
  __half* Pprot = reinterpret_cast<__half*>(S) + n_sg * (kSGGroups * kG);
  __half* Pres = Pprot + n_pg * kG;

  // ---- destinations of the quantized tokens
  for (int i = c.tid; i < c.nq; i += kThreads) {
    const int64_t t = c.t0 + i;
    uint32_t d;
    if (t < c.T_q0) {
      const uint32_t word = ew[t / kG];
      const int64_t pb = ep[t / kG] + __popc(word & ((1u << (t & 31)) - 1u));
      d = (word >> (t & 31)) & 1u ? 0x8000u | static_cast<uint32_t>(pb - Pbase) : static_cast<uint32_t>((t - pb) - Ubase);
    } else {
      d = static_cast<uint32_t>(u_fl0 + (t - c.T_q0) - Ubase);
    }
    map[i] = static_cast<uint16_t>(d);
  }

  cp_async_wait<0>();
  __syncthreads();
  score_phase<T>(a, n_chunks, c, buf, S, SS, qexp);
  __syncthreads();
  {
    // the key groups are spent: the ternary supergroups take their place while the softmax runs
    const uint8_t* vsrc = c.slab_ptr + cv.tern_offset + sgA * kSGBytes;
    stage_async(buf, vsrc, n_sg * (kSGBytes / 16), c.tid);
    cp_async_commit();
  }
  softmax_phase<true>(a, c, S, SS, red, 0, map, Pprot, PT, Pres, PT, qexp);
  __syncthreads();
  group_sums(c, reinterpret_cast<const __half*>(S), PT, n_sg * kSGGroups, -5.0f, psum_t);
  group_sums(c, Pprot, PT, n_pg, 1.0f, psum_p);
  cp_async_wait<0>();
  __syncthreads();

  float tot[2][4] = {{0.0f, 0.0f, 0.0f, 0.0f}, {0.0f, 0.0f, 0.0f, 0.0f}};
  // groups of the staged supergroups that hold tokens of this split: [U0 / 32, ceil(U1 / 32)), and no group past the stream's end
  const int g_first = static_cast<int>(U0 / kG - sgA * kSGGroups);
  const int g_end = static_cast<int>(min(tg_total, (U1 + kG - 1) / kG) - sgA * kSGGroups);
  ternary_phase<true>(c, buf, n_sg, g_first, g_end, reinterpret_cast<const uint8_t*>(S + c.hd * SS), psum_t, tot);
  // ---- protected stream: 2-bit codes (Eq. 4) as 4 + code, then s * (acc - 4 sum p) + z * sum p
  if (n_pg > 0) {
    const int warp = c.warp, hd = c.hd, r = c.r;
    const uint8_t* prow = reinterpret_cast<const uint8_t*>(Pprot + hd * PT);
    const uint8_t* gbase = c.slab_ptr + cv.prot_offset + pgA * kPGBytes;
    const int w_off = (((warp * 4) + r) * 8 + hd) * 4, m_off = (32 * warp + 4 * hd) * 2;
    // operands of the group being consumed are loaded one group ahead
    uint32_t w0 = __ldg(reinterpret_cast<const uint32_t*>(gbase + w_off));
    uint32_t w1 = __ldg(reinterpret_cast<const uint32_t*>(gbase + 512 + w_off));
    uint2 sc = __ldg(reinterpret_cast<const uint2*>(gbase + kPG_S + m_off));
    uint2 zc = __ldg(reinterpret_cast<const uint2*>(gbase + kPG_Z + m_off));
    for (int pg = 0; pg < n_pg; ++pg) {
      const uint32_t wk[2] = {w0, w1};
      const uint2 scc = sc, zcc = zc;
      if (pg + 1 < n_pg) {
        const uint8_t* gp = gbase + (pg + 1) * kPGBytes;
        w0 = __ldg(reinterpret_cast<const uint32_t*>(gp + w_off));
        w1 = __ldg(reinterpret_cast<const uint32_t*>(gp + 512 + w_off));
        sc = __ldg(reinterpret_cast<const uint2*>(gp + kPG_S + m_off));
        zc = __ldg(reinterpret_cast<const uint2*>(gp + kPG_Z + m_off));
      }
      const float2 sp = *reinterpret_cast<const float2*>(psum_p + pg * 8 + 2 * r);
      float acc[2][4];
#pragma unroll
      for (int kt = 0; kt < 2; ++kt) {
        const uint32_t w = wk[kt];
        uint32_t x[8];
        x[0] = and_or(w << 8, c.m_field, c.c_four);
        x[1] = and_or(w << 6, c.m_field, c.c_four);
        x[2] = and_or(w << 4, c.m_field, c.c_four);
        x[3] = and_or(w << 2, c.m_field, c.c_four);
        x[4] = and_or(w, c.m_field, c.c_four);
        x[5] = and_or(w >> 2, c.m_field, c.c_four);
        x[6] = and_or(w >> 4, c.m_field, c.c_four);
        x[7] = and_or(w >> 6, c.m_field, c.c_four);
        const uint8_t* pb = prow + (pg * kG + kt * 16 + 2 * r) * 2;
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(pb);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(pb + 16);
        if (kt == 0) {
          mma_f16_c(acc[0], x[0], x[1], x[4], x[5], b0, b1, -4.0f * sp.x, -4.0f * sp.y, -4.0f * sp.x, -4.0f * sp.y);
          mma_f16_c(acc[1], x[2], x[3], x[6], x[7], b0, b1, -4.0f * sp.x, -4.0f * sp.y, -4.0f * sp.x, -4.0f * sp.y);
        } else {
          mma_f16(acc[0], x[0], x[1], x[4], x[5], b0, b1);
          mma_f16(acc[1], x[2], x[3], x[6], x[7], b0, b1);
        }
      }
      const float2 sa = __half22float2(*reinterpret_cast<const __half2*>(&scc.x));
      const float2 sb = __half22float2(*reinterpret_cast<const __half2*>(&scc.y));
      const float2 za = __half22float2(*reinterpret_cast<const __half2*>(&zcc.x));
      const float2 zb = __half22float2(*reinterpret_cast<const __half2*>(&zcc.y));
      tot[0][0] += sa.x * acc[0][0] + za.x * sp.x; tot[0][1] += sa.x * acc[0][1] + za.x * sp.y;
      tot[0][2] += sa.y * acc[0][2] + za.y * sp.x; tot[0][3] += sa.y * acc[0][3] + za.y * sp.y;
      tot[1][0] += sb.x * acc[1][0] + zb.x * sp.x; tot[1][1] += sb.x * acc[1][1] + zb.x * sp.y;
      tot[1][2] += sb.y * acc[1][2] + zb.y * sp.x; tot[1][3] += sb.y * acc[1][3] + zb.y * sp.y;
    }
  }
  __syncthreads();                                       // the output staging reuses buf
  if (c.t1 > c.T_qt)
    residual_pv<T>(a, c, reinterpret_cast<float*>(buf), Pres, PT,
                   -static_cast<int>(max(c.t0, c.T_qt) - c.T_qt), tot);
  write_partial(a, c, blockIdx.x, reinterpret_cast<float*>(buf), red, tot);
}

cudaError_t launch_decode_prep(DecodeArgs& a, cudaStream_t stream) {
  a.dft = nullptr;
  const int n_slabs = a.n_layers * a.cv.B * a.cv.H_kv;
  const int n_chunks = a.plan.n_chunks;
  if (n_chunks < 1) return cudaSuccess;
  cudaError_t e;
  if ((e = dft_fragments(&a.dft, stream))) return e;
  const int n_items = n_slabs * n_chunks;
  const int pgrid = (n_items + kThreads / 32 - 1) / (kThreads / 32);
  if (a.in_dtype == VIDKV_F16) decode_prep_kernel<__half><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
  else decode_prep_kernel<__nv_bfloat16><<<pgrid, kThreads, 0, stream>>>(a, n_chunks, n_items);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_decode_stp(const DecodeArgs& a, cudaStream_t stream) {
  const int n_slabs = a.n_layers * a.cv.B * a.cv.H_kv;
  const size_t smem = decode_stp_smem_bytes(a.plan.split_tokens);
  static size_t attr_smem_dev[64] = {};   // function attributes are per device
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (smem > attr_smem_dev[dev]) {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(decode_stp_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    if ((e = cudaFuncSetAttribute(decode_stp_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    attr_smem_dev[dev] = smem;
  }
  const dim3 grid(a.plan.n_splits, n_slabs);
  if (a.in_dtype == VIDKV_F16) decode_stp_kernel<__half><<<grid, kThreads, smem, stream>>>(a, a.plan.n_chunks);
  else decode_stp_kernel<__nv_bfloat16><<<grid, kThreads, smem, stream>>>(a, a.plan.n_chunks);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace vidkv
