// Decode attention over the packed cache for caches without protected tokens (Algorithm 1
// "Decoding", Eq. 3): the stream kernel.
//
// The quantized tokens of all slabs of a call form one sequence of 160-token units (five
// 32-token key groups and the ternary supergroup that holds the same tokens' values).  Every
// warp of the launch owns a contiguous run of units and works through it alone, the way a
// streaming softmax does:
//   1. the unit's key groups arrive in the warp's key buffer by one bulk copy
//      (cp.async.bulk + mbarrier); the scores q . K' of its 160 tokens come out of
//      mma.sync.m16n8k16 with rows = query heads (exact binary16 pair hi + lo of q_j s_j),
//      columns = tokens, the codes expanded in registers as the B operand:
//      shifts and masks are all they need;
//   2. the accumulator fragment of that product (head = lane / 4, tokens 2 r, 2 r + 1) is
//      exactly the B fragment of the next one, so the probabilities 2^(logit - running maximum)
//      stay in registers as binary16 pairs; the running maximum only moves (and the
//      accumulated output is only rescaled) when a unit's maximum exceeds it by more than
//      kStaleLog2, so probabilities reach 2^kStaleLog2 at most;
//   3. the unit's ternary supergroup (second bulk copy, in flight during step 1) is peeled digit
//      by digit into 5 + trit, multiplied with the probabilities into per-group accumulators
//      that start at -5 sum p (the sums come from a product with a constant matrix, which also
//      yields the softmax denominator), and the per-(group, channel) scales fold the group
//      accumulators into the warp's running output for all 128 channels x 8 heads.
// While a unit is being worked on, the next unit's keys and values are already on their way
// into the two buffers (a buffer is refilled as soon as its reader is done).  A warp leaves one
// partial record (maximum, sum, out[128]) per query head for every slab its run touches; the
// merge kernel combines them and attends to the FP16 / BF16 residual.
//
// Nothing is shared between warps: no block-wide barrier, no shared score matrix.
#include "decode_common.cuh"

namespace vidkv {

namespace {

constexpr int kKBufBytes = kSGGroups * kKGroupBytes;   // 5760: the key groups of one unit
constexpr int kVBufBytes = kSGBytes;                   // 5376: its ternary supergroup
constexpr int kTotBytes = 4 * 2 * 32 * 16;             // 4096: the warp's running output (128 channels x 8 heads, float)
constexpr int kWarpBufBytes = kKBufBytes + kVBufBytes + kTotBytes;   // 15232 per warp
constexpr int kGenKBufBytes = kSGGroups * kMaxKGroupBytes;           // key buffer of the general key formats
constexpr uint32_t kWaitLimit = 1u << 19;              // mbarrier polls before a warp gives up (about a second)
constexpr float kStaleLog2 = 6.0f;                     // the running maximum may lag a unit's maximum by this much
constexpr uint32_t kMinus5 = 0xc500c500u;              // binary16 pair (-5.0, -5.0)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// One bulk copy global -> shared of `bytes` (multiple of 16, both addresses 16-byte aligned),
// completion counted on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  const uint32_t b = smem_u32(bar), d = smem_u32(dst);
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(d),
               "l"(src), "r"(bytes), "r"(b)
               : "memory");
}
// Bounded wait for the phase with the given parity; false if it never completed.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t b = smem_u32(bar);
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(b), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}

// Per-lane state of the running softmax of one slab (the running output itself is in shared memory).
struct Running {
  float l[2];           // sums of the probabilities of heads 2 r, 2 r + 1
  float m;              // running maximum (base-2 logit) of head hd
};

// Raw scores of one 32-token key group: sc[nt][0..1] = q . K' of head hd and tokens 8 nt + 2 r, + 1
// without the group's constant, which is returned in cst (the same for the 32 tokens), all in the
// units of the normalised query.  Consecutive products go to different accumulators (the four
// 8-token tiles, and the chain of the constants in between), so that no product waits for the
// one issued just before it.
__device__ __forceinline__ void score_group(const uint8_t* kg, int lane, int hd, int r, const uint32_t (&qa)[8],
                                            const uint32_t (&qha)[8], const uint32_t (&qhb)[8], uint32_t m_field,
                                            uint32_t c_four, uint32_t m_sign, uint32_t c_neg1, float (&sc)[4][2],
                                            float& cst) {
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
  const uint4 c2 = *reinterpret_cast<const uint4*>(kg + kKG_Codes2 + lane * 16);
  const uint2 c1 = *reinterpret_cast<const uint2*>(kg + kKG_Bits1 + lane * 8);
  const uint32_t w2[4] = {c2.x, c2.y, c2.z, c2.w};
  const uint32_t wh[4] = {c2.x >> 6, c2.y >> 6, c2.z >> 6, c2.w >> 6};   // fields 5-7 come from one right shift
  // sign bits: low lane <- bit 15 - 2 m, high lane <- bit 14 - 2 m of the token's half-word
  const uint32_t X[4] = {(c1.x & 0xffffu) * 0x00020001u, (c1.x >> 16) * 0x00020001u, (c1.y & 0xffffu) * 0x00020001u,
                         (c1.y >> 16) * 0x00020001u};
  float acc[4][4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) { acc[nt][0] = 0.0f; acc[nt][1] = 0.0f; acc[nt][2] = 0.0f; acc[nt][3] = 0.0f; }
  // constants of the group: column 2 r of the result = sum q z, column 2 r + 1 = sum q s
  float cz[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  // anomalous channels: q s as exact binary16 pairs hi + lo against 4 + code
  {
    uint32_t hi2[8], lo2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      hi2[i] = hmul2_u(qa[i], s2[i]);
      lo2[i] = hfms2_u(qa[i], s2[i], hi2[i]);
    }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      mma_f16(cz, qa[2 * ks], 0u, qa[2 * ks + 1], 0u, z2[2 * ks], z2[2 * ks + 1]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        // fields 2 ks and 2 ks + 1 of the word: shifts by 8 - 4 ks and 6 - 4 ks bits
        const uint32_t f0 = ks == 0 ? w2[nt] << 8 : ks == 1 ? w2[nt] << 4 : ks == 2 ? w2[nt] : wh[nt] << 2;
        const uint32_t f1 = ks == 0 ? w2[nt] << 6 : ks == 1 ? w2[nt] << 2 : ks == 2 ? wh[nt] << 4 : wh[nt];
        mma_f16(acc[nt], hi2[2 * ks], lo2[2 * ks], hi2[2 * ks + 1], lo2[2 * ks + 1], and_or(f0, m_field, c_four),
                and_or(f1, m_field, c_four));
      }
    }
  }
  // normal channels in the frequency domain: Q (leading part + remainder, rows hd and hd + 8) against
  // +-s: the scale takes the sign inside the one logic instruction that used to make +-1, and the
  // products Q s are formed exactly by the tensor core
  {
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        mma_f16(acc[nt], qha[2 * ks], qhb[2 * ks], qha[2 * ks + 1], qhb[2 * ks + 1],
                nand_xor(X[nt] << (4 * ks), m_sign, s1[2 * ks]), nand_xor(X[nt] << (4 * ks + 2), m_sign, s1[2 * ks + 1]));
    }
  }
  cst = cz[0] - 4.0f * cz[1];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    sc[nt][0] = acc[nt][0] + acc[nt][2];
    sc[nt][1] = acc[nt][1] + acc[nt][3];
  }
}

// The same for a key group in the general layout (KeyFmt): blocks of 32 two-bit slots, then blocks of
// 32 one-bit columns.  pp points at this lane's prepared query words of the group's chunk (32 words
// apart).  Two-bit slots as above (q s as hi + lo against 4 + code).  One-bit columns: Eq. 5 as above
// with the transformed query; in plain mode the value is code s + z = (+-1) s / 2 + (z + s / 2), so q s
// (hi + lo) meets +-1, the products are halved at the end and the constant takes sum q z + sum q s / 2.
__device__ __forceinline__ void score_group_general(const uint8_t* kg, const KeyFmt& kf, int lane, int hd, int r,
                                                    const uint32_t* pp, uint32_t m_field, uint32_t c_four, uint32_t m_sign,
                                                    uint32_t c_neg1, float (&sc)[4][2], float& cst) {
  float acc[4][4], acc1[4][4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
    for (int i = 0; i < 4; ++i) { acc[nt][i] = 0.0f; acc1[nt][i] = 0.0f; }
  }
  float cz[4] = {0.0f, 0.0f, 0.0f, 0.0f}, cz1[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  const int n2b = kf.n2 >> 5, n1b = (kD - kf.n2) >> 5;
#pragma unroll 1
  for (int b = 0; b < n2b; ++b) {
    uint32_t qa[4], hi[4], lo[4];
    const uint4 sv = *reinterpret_cast<const uint4*>(kg + kf.off_s2 + 64 * b + 16 * r);
    const uint4 zv = *reinterpret_cast<const uint4*>(kg + ((hd & 1) ? kf.off_s2 : kf.off_z2) + 64 * b + 16 * r);
    const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w}, zw[4] = {zv.x, zv.y, zv.z, zv.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      qa[j] = __ldg(pp + (4 * b + j) * 32);
      hi[j] = hmul2_u(qa[j], sw[j]);
      lo[j] = hfms2_u(qa[j], sw[j], hi[j]);
    }
    const uint2 cw = *reinterpret_cast<const uint2*>(kg + 256 * b + lane * 8);
    uint32_t W[4];
    W[0] = prmt(cw.x, 0u, 0x1404u); W[1] = prmt(cw.x, 0u, 0x3424u);
    W[2] = prmt(cw.y, 0u, 0x1404u); W[3] = prmt(cw.y, 0u, 0x3424u);
#pragma unroll
    for (int kp = 0; kp < 2; ++kp) {
      mma_f16(cz, qa[2 * kp], 0u, qa[2 * kp + 1], 0u, zw[2 * kp], zw[2 * kp + 1]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        mma_f16(acc[nt], hi[2 * kp], lo[2 * kp], hi[2 * kp + 1], lo[2 * kp + 1], and_or(W[nt] >> (4 * kp), m_field, c_four),
                and_or(W[nt] >> (4 * kp + 2), m_field, c_four));
    }
  }
  const int w1 = kf.n2 >> 3, nw1 = (kD - kf.n2) >> 3;
#pragma unroll 1
  for (int b = 0; b < n1b; ++b) {
    // the stored scale takes the sign of the code bit and goes to the tensor core as it is; the other
    // operand is the transformed query as hi + lo (Eq. 5) or the query itself (plain mode, exact in one piece)
    uint32_t ah[4], al[4];
    const uint4 sv = *reinterpret_cast<const uint4*>(kg + kf.off_s1 + 64 * b + 16 * r);
    const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
    if (kf.plain) {
      const uint4 zv = *reinterpret_cast<const uint4*>(kg + ((hd & 1) ? kf.off_s1 : kf.off_z1) + 64 * b + 16 * r);
      const uint32_t zw[4] = {zv.x, zv.y, zv.z, zv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        ah[j] = __ldg(pp + (w1 + 4 * b + j) * 32);
        al[j] = 0u;
      }
      mma_f16(cz1, ah[0], 0u, ah[1], 0u, zw[0], zw[1]);
      mma_f16(cz1, ah[2], 0u, ah[3], 0u, zw[2], zw[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        ah[j] = __ldg(pp + (w1 + 4 * b + j) * 32);
        al[j] = __ldg(pp + (w1 + nw1 + 4 * b + j) * 32);
      }
    }
    const uint32_t cw = *reinterpret_cast<const uint32_t*>(kg + kf.off_bits1 + 128 * b + lane * 4);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const uint32_t X = ((cw >> (8 * nt)) & 0xffu) * 0x02000100u;   // low lane: bit 7 at the sign, high lane: bit 6
#pragma unroll
      for (int kp = 0; kp < 2; ++kp)
        mma_f16(acc1[nt], ah[2 * kp], al[2 * kp], ah[2 * kp + 1], al[2 * kp + 1], nand_xor(X << (4 * kp), m_sign, sw[2 * kp]),
                nand_xor(X << (4 * kp + 2), m_sign, sw[2 * kp + 1]));
    }
  }
  const float f1 = kf.plain ? 0.5f : 1.0f;
  cst = cz[0] - 4.0f * cz[1] + (kf.plain ? cz1[0] + 0.5f * cz1[1] : 0.0f);
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    sc[nt][0] = acc[nt][0] + acc[nt][2] + f1 * (acc1[nt][0] + acc1[nt][2]);
    sc[nt][1] = acc[nt][1] + acc[nt][3] + f1 * (acc1[nt][1] + acc1[nt][3]);
  }
}

// Running output of the warp, kept in shared memory: float4 tot[j][lane], j = 2 w + i, holds the
// accumulator fragment of channels 32 w + 4 hd + 2 i + (e >> 1) and heads 2 r + (e & 1), e = 0..3.

// P V of one staged ternary supergroup: for NG of its groups, P[g][nt] holds the probabilities of
// head hd at stream tokens 32 g + 8 nt + 2 r, + 1 (binary16 pairs) and ps[g] the accumulator
// fragment -5 * (sum of those probabilities) of heads 2 r, 2 r + 1.  32 channels (two MMA row
// blocks) at a time: fragment i of block w covers channels 32 w + 4 hd + 2 i + {0, 1} in rows hd,
// hd + 8.  Adds into the warp's running output.
template <int NG>
__device__ __forceinline__ void pv_ternary(const uint8_t* vbuf, float* totbuf, const uint32_t (&P)[NG][4],
                                           const float (&ps)[NG][4], int lane, int hd, int r, uint32_t m_field,
                                           uint32_t c_four) {
#pragma unroll 1
  for (int w = 0; w < 4; ++w) {
    float acc[NG][2][4];
#pragma unroll
    for (int kt = 0; kt < 2; ++kt) {
      const uint2 wa = *reinterpret_cast<const uint2*>(vbuf + ((((kt * 2 + 0) * 4 + w) * 4 + r) * 8 + hd) * 8);
      const uint2 wb = *reinterpret_cast<const uint2*>(vbuf + ((((kt * 2 + 1) * 4 + w) * 4 + r) * 8 + hd) * 8);
      uint32_t W[8];
      W[0] = prmt(wa.x, 0u, 0x4140u); W[1] = prmt(wa.x, 0u, 0x4342u);
      W[2] = prmt(wb.x, 0u, 0x4140u); W[3] = prmt(wb.x, 0u, 0x4342u);
      W[4] = prmt(wa.y, 0u, 0x4140u); W[5] = prmt(wa.y, 0u, 0x4342u);
      W[6] = prmt(wb.y, 0u, 0x4140u); W[7] = prmt(wb.y, 0u, 0x4342u);
#pragma unroll
      for (int k = 0; k < 8; ++k) W[k] = mad_u32(W[k], 3u, 0u);          // 3 * byte per 16-bit lane
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        uint32_t A[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          // W holds 3 * (remaining byte) per 16-bit lane; the digit sits at bits 8-9.
          // Next W = 3 * (W - digit << 8) = 3 W - 3 A + 3 * 0x4400 (no lane ever borrows).
          // Half of the lanes take that route (two multiply-adds), the other half mask the digit
          // away and multiply (one logic, one multiply-add): the two pipes share the work.
          A[k] = and_or(W[k], m_field, c_four);
          if (g + 1 < NG) {
            if (k & 1) W[k] = mad_u32(A[k], 0xfffffffdu, mad_u32(W[k], 3u, 0xcc00cc00u));
            else W[k] = mad_u32(W[k] & 0x00ff00ffu, 3u, 0u);
          }
        }
        const uint32_t b0 = P[g][2 * kt], b1 = P[g][2 * kt + 1];
        if (kt == 0) {
          mma_f16_c(acc[g][0], A[0], A[1], A[2], A[3], b0, b1, ps[g][0], ps[g][1], ps[g][2], ps[g][3]);
          mma_f16_c(acc[g][1], A[4], A[5], A[6], A[7], b0, b1, ps[g][0], ps[g][1], ps[g][2], ps[g][3]);
        } else {
          mma_f16(acc[g][0], A[0], A[1], A[2], A[3], b0, b1);
          mma_f16(acc[g][1], A[4], A[5], A[6], A[7], b0, b1);
        }
      }
    }
    float4* tp = reinterpret_cast<float4*>(totbuf) + (2 * w) * 32 + lane;
    float4 t0 = tp[0], t1 = tp[32];
#pragma unroll
    for (int g = 0; g < NG; ++g) {
      const uint2 sc2 = *reinterpret_cast<const uint2*>(vbuf + kSG_Scales + g * (kD * 2) + (32 * w + 4 * hd) * 2);
      const float2 sa = __half22float2(*reinterpret_cast<const __half2*>(&sc2.x));
      const float2 sb = __half22float2(*reinterpret_cast<const __half2*>(&sc2.y));
      t0.x += sa.x * acc[g][0][0]; t0.y += sa.x * acc[g][0][1];
      t0.z += sa.y * acc[g][0][2]; t0.w += sa.y * acc[g][0][3];
      t1.x += sb.x * acc[g][1][0]; t1.y += sb.x * acc[g][1][1];
      t1.z += sb.y * acc[g][1][2]; t1.w += sb.y * acc[g][1][3];
    }
    tp[0] = t0;
    tp[32] = t1;
  }
}

// One unit of NG (1..5) groups: scores, probabilities, P V into the running state.
// Returns false if a copy never arrived.
template <int NG, bool GEN>
__device__ __forceinline__ bool process_unit(const KeyFmt& kf, const uint32_t*& ppc, uint8_t* kbuf, uint8_t* vbuf, float* totbuf, uint64_t* kbar, uint64_t* vbar,
                                             uint32_t& kpar, uint32_t& vpar, int lane, int hd, int r,
                                             const uint32_t* prep_slab, int64_t g_first, int64_t g0n, int& cur_chunk,
                                             uint32_t (&qa)[8], uint32_t (&qha)[8], uint32_t (&qhb)[8], float sl2,
                                             Running& run, bool more, const uint8_t* next_k, uint32_t next_k_bytes,
                                             const uint8_t* next_v) {
  const uint32_t m_field = kExpand[0], c_four = kExpand[1], m_sign = kExpand[2], c_neg1 = kExpand[3];
  const int kgb = GEN ? kf.group_bytes : kKGroupBytes;      // bytes of one key group
  if (!mbar_wait(kbar, kpar)) return false;
  kpar ^= 1u;
  // ---- scores, group by group; a group's scores replace its (spent) bytes in the key buffer:
  // float2 (tokens 8 nt + 2 r, + 1 of head hd) at word pair (nt * 32 + lane) of the group, the
  // group's additive constant at word 256 + lane
  float mx = -INFINITY;
#pragma unroll 1
  for (int g = 0; g < NG; ++g) {
    const int64_t gidx = g_first + g;
    const int chunk = gidx < g0n ? 0 : 1 + static_cast<int>((gidx - g0n) / (kR / kG));
    if (chunk != cur_chunk) {
      cur_chunk = chunk;
      const uint32_t* pp = prep_slab + static_cast<int64_t>(chunk) * (kPrepWords * 32);
      ppc = pp;
      if (!GEN) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          qa[i] = __ldg(pp + i * 32);
          qha[i] = __ldg(pp + (8 + i) * 32);
          qhb[i] = __ldg(pp + (16 + i) * 32);
        }
      }
    }
    float sc[4][2], cst;
    uint8_t* kg = kbuf + g * kgb;
    if (GEN) score_group_general(kg, kf, lane, hd, r, ppc, m_field, c_four, m_sign, c_neg1, sc, cst);
    else score_group(kg, lane, hd, r, qa, qha, qhb, m_field, c_four, m_sign, c_neg1, sc, cst);
    __syncwarp();                                           // every lane has read the group's bytes
    float gm = fmaxf(sc[0][0], sc[0][1]);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      reinterpret_cast<float2*>(kg)[nt * 32 + lane] = make_float2(sc[nt][0], sc[nt][1]);
      gm = fmaxf(gm, fmaxf(sc[nt][0], sc[nt][1]));
    }
    reinterpret_cast<float*>(kg)[256 + lane] = cst;         // the group's constant joins in the exponent
    mx = fmaxf(mx, gm + cst);
  }
  // ---- probabilities against the running maximum
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
  {
    const float mu = mx * sl2;                              // sl2 > 0
    const bool up = mu > run.m + kStaleLog2;                // always true for the first unit (run.m = -inf)
    if (__any_sync(0xffffffffu, up)) {
      const float m_new = up ? mu : run.m;
      const float f = ex2_approx(run.m - m_new);            // 1 for heads whose maximum stays
      run.m = m_new;
      const float fa = __shfl_sync(0xffffffffu, f, 8 * r), fb = __shfl_sync(0xffffffffu, f, 8 * r + 4);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4* t = reinterpret_cast<float4*>(totbuf) + j * 32 + lane;
        float4 v = *t;
        v.x *= fa; v.y *= fb; v.z *= fa; v.w *= fb;
        *t = v;
      }
      run.l[0] *= fa; run.l[1] *= fb;
    }
  }
  uint32_t P[NG][4];
  float ps[NG][4];
#pragma unroll
  for (int g = 0; g < NG; ++g) {
    const float off = fmaf(reinterpret_cast<const float*>(kbuf + g * kgb)[256 + lane], sl2, -run.m);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const float2 v = reinterpret_cast<const float2*>(kbuf + g * kgb)[nt * 32 + lane];
      P[g][nt] = pack_half2(ex2_approx(fmaf(v.x, sl2, off)), ex2_approx(fmaf(v.y, sl2, off)));
    }
    // -5 * (sums of the rounded probabilities) of heads 2 r, 2 r + 1, for rows hd and hd + 8 alike:
    // a product with a matrix of -5, whose accumulator fragment is the initial value of every
    // P V accumulator of the group as it stands
    ps[g][0] = 0.0f; ps[g][1] = 0.0f; ps[g][2] = 0.0f; ps[g][3] = 0.0f;
    mma_f16(ps[g], kMinus5, kMinus5, kMinus5, kMinus5, P[g][0], P[g][1]);
    mma_f16(ps[g], kMinus5, kMinus5, kMinus5, kMinus5, P[g][2], P[g][3]);
    run.l[0] = fmaf(-0.2f, ps[g][0], run.l[0]);
    run.l[1] = fmaf(-0.2f, ps[g][1], run.l[1]);
  }
  __syncwarp();                                             // the scores are in registers: the key buffer is free
  if (more && lane == 0) {
    // the buffer was used through ordinary loads and stores; order them before the bulk copy's writes
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    bulk_load(kbuf, next_k, next_k_bytes, kbar);
  }
  // ---- P V over the ternary supergroup
  if (!mbar_wait(vbar, vpar)) {
    if (more) mbar_wait(kbar, kpar);                        // let the key copy issued above land before leaving
    return false;
  }
  vpar ^= 1u;
  pv_ternary<NG>(vbuf, totbuf, P, ps, lane, hd, r, m_field, c_four);
  __syncwarp();
  if (more && lane == 0) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    bulk_load(vbuf, next_v, kVBufBytes, vbar);
  }
  return true;
}

__device__ __forceinline__ void write_record(const DecodeArgs& a, int slab, int run_id, int lane, int hd, int r,
                                             const Running& run, const float* totbuf) {
  const DecodePlan& pl = a.plan;
  const int rep = a.cv.rep;
  const int first = static_cast<int>(static_cast<int64_t>(slab) * pl.units_per_slab / pl.run_units);
  float* rec = a.partials + (static_cast<int64_t>(slab) * pl.parts_stride + (run_id - first)) * (kMaxRep * kRecordFloats);
#pragma unroll
  for (int w = 0; w < 4; ++w)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float4 t = reinterpret_cast<const float4*>(totbuf)[(w * 2 + i) * 32 + lane];
      const int c = 32 * w + 4 * hd + 2 * i;
      if (2 * r < rep) {
        rec[(2 * r) * kRecordFloats + 2 + c] = t.x;
        rec[(2 * r) * kRecordFloats + 2 + c + 1] = t.z;
      }
      if (2 * r + 1 < rep) {
        rec[(2 * r + 1) * kRecordFloats + 2 + c] = t.y;
        rec[(2 * r + 1) * kRecordFloats + 2 + c + 1] = t.w;
      }
    }
  if (hd == 0) {
    if (2 * r < rep) rec[(2 * r) * kRecordFloats + 1] = run.l[0];
    if (2 * r + 1 < rep) rec[(2 * r + 1) * kRecordFloats + 1] = run.l[1];
  }
  if (r == 0 && hd < rep) rec[hd * kRecordFloats] = run.m;
}

}  // namespace

template <bool GEN>
__global__ void __launch_bounds__(kStreamWarps * 32, kStreamCtasPerSM) decode_stream_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[kStreamWarps][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, hd = lane >> 2, r = lane & 3;
  const DecodePlan& pl = a.plan;
  const CacheView& cv = a.cv;
  const int run_id = blockIdx.x * kStreamWarps + warp;
  const int64_t u_begin = static_cast<int64_t>(run_id) * pl.run_units;
  const int64_t u_end = min(u_begin + pl.run_units, pl.n_units);
  if (u_begin >= u_end) return;                            // warps do not wait on one another
  const KeyFmt& kf = a.cv.kf;
  const int kgb = GEN ? kf.group_bytes : kKGroupBytes;
  constexpr int kbuf_bytes = GEN ? kGenKBufBytes : kKBufBytes;
  uint8_t* kbuf = smem_raw + warp * (kbuf_bytes + kVBufBytes + kTotBytes);
  uint8_t* vbuf = kbuf + kbuf_bytes;
  float* totbuf = reinterpret_cast<float*>(vbuf + kVBufBytes);
  uint64_t* kbar = &bars[warp][0];
  uint64_t* vbar = &bars[warp][1];
  if (lane == 0) {
    mbar_init(kbar, 1);
    mbar_init(vbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const int S = pl.units_per_slab;
  const int64_t n_groups = (a.st.T_q0 + a.st.n_flush * kR) / kG;   // key groups = ternary groups per slab
  const int64_t g0n = a.st.T_q0 / kG;
  const uint8_t* slab0 = cv.base + cv.slab_offset + static_cast<int64_t>(a.layer0) * cv.B * cv.H_kv * cv.slab_stride;
  int slab = static_cast<int>(u_begin / S);
  int k = static_cast<int>(u_begin - static_cast<int64_t>(slab) * S);
  auto groups_of = [&](int kk) -> int {
    const int64_t left = n_groups - static_cast<int64_t>(kk) * kSGGroups;
    return left < kSGGroups ? static_cast<int>(left) : kSGGroups;
  };
  auto key_src = [&](int sl, int kk) -> const uint8_t* {
    return slab0 + static_cast<int64_t>(sl) * cv.slab_stride + cv.kgroup_offset + static_cast<int64_t>(kk) * (kSGGroups * kgb);
  };
  auto val_src = [&](int sl, int kk) -> const uint8_t* {
    return slab0 + static_cast<int64_t>(sl) * cv.slab_stride + cv.tern_offset + static_cast<int64_t>(kk) * kVBufBytes;
  };
  if (lane == 0) {
    bulk_load(kbuf, key_src(slab, k), groups_of(k) * kgb, kbar);
    if (!a.withhold) bulk_load(vbuf, val_src(slab, k), kVBufBytes, vbar);   // (test hook: see DecodeArgs::withhold)
  }
  // the packed cache is not written by the query preparation, so the copies above may start while
  // it still runs; the prepared query is read from here on
  pdl_wait();
  pdl_release();
  uint32_t kpar = 0u, vpar = 0u;
  Running run;
  run.l[0] = 0.0f; run.l[1] = 0.0f; run.m = -INFINITY;
  uint32_t qa[8], qha[8], qhb[8];
  const uint32_t* ppc = nullptr;
  int cur_chunk = -1, cur_slab = -1;
  const uint32_t* prep_slab = nullptr;
  float sl2 = 0.0f;
  bool ok = true;
#pragma unroll 1
  for (int64_t u = u_begin; u < u_end; ++u) {
    if (slab != cur_slab) {
      if (cur_slab >= 0) write_record(a, cur_slab, run_id, lane, hd, r, run, totbuf);
      cur_slab = slab;
      cur_chunk = -1;
#pragma unroll
      for (int j = 0; j < 8; ++j) reinterpret_cast<float4*>(totbuf)[j * 32 + lane] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      run.l[0] = 0.0f; run.l[1] = 0.0f;
      run.m = -INFINITY;
      prep_slab = a.prep + static_cast<int64_t>(slab) * pl.n_chunks * (kPrepWords * 32) + lane;
      sl2 = __uint_as_float(__ldg(prep_slab + 24 * 32));
    }
    const int ng = groups_of(k);
    int nslab = slab, nk = k + 1;
    if (nk == S) { nk = 0; ++nslab; }
    const bool more = u + 1 < u_end;
    const uint8_t* next_k = more ? key_src(nslab, nk) : nullptr;
    const uint32_t next_k_bytes = more ? static_cast<uint32_t>(groups_of(nk) * kgb) : 0u;
    const uint8_t* next_v = more ? val_src(nslab, nk) : nullptr;
#define VIDKV_UNIT(N)                                                                                                \
  ok = process_unit<N, GEN>(kf, ppc, kbuf, vbuf, totbuf, kbar, vbar, kpar, vpar, lane, hd, r, prep_slab,                           \
                       static_cast<int64_t>(k) * kSGGroups, g0n, cur_chunk, qa, qha, qhb, sl2, run, more, next_k,      \
                       next_k_bytes, next_v)
    if (ng == 5) VIDKV_UNIT(5);
    else if (ng == 4) VIDKV_UNIT(4);
    else if (ng == 3) VIDKV_UNIT(3);
    else if (ng == 2) VIDKV_UNIT(2);
    else VIDKV_UNIT(1);
#undef VIDKV_UNIT
    if (!ok) break;
    slab = nslab; k = nk;
  }
  if (!ok) {
    // a copy never arrived: report it and leave (the wait already ran its full course, so nothing
    // this warp issued can still be expected)
    if (lane == 0) atomicCAS(reinterpret_cast<int*>(cv.base + kHdrStatus), VIDKV_OK, VIDKV_ERR_TIMEOUT);
    return;
  }
  write_record(a, cur_slab, run_id, lane, hd, r, run, totbuf);
}

// ---------------------------------------------------------------------------------
// Caches with protected tokens (STPQuant, Algorithm 2): the same walk over 160-token key units,
// but the values of a unit's tokens sit in two streams whose order differs from the key order:
// unprotected tokens in the ternary stream (position = token - protected tokens before it;
// flushed tokens follow from the next group boundary), protected ones in 2-bit groups of 32.
// The probabilities of a unit are therefore scattered (as binary16) into two per-warp rings in
// stream order, one row per head, and a ternary supergroup (160 stream positions) or protected
// group (32) is multiplied as soon as all of its positions have been written.  Positions of a
// supergroup or group that belong to a neighbouring run stay zero; the neighbour multiplies the
// same bytes with its own probabilities.  The running maximum is kept integral (base-2), so that
// probabilities waiting in the rings are rescaled exactly when it moves.
// Per-warp shared memory: key buffer, ternary supergroup buffer, protected group buffer, running
// output, and the rings: one row per head with 320 ternary and 192 protected positions.
// ---------------------------------------------------------------------------------
namespace {

constexpr int kTRing = 2 * kStreamUnitTokens;          // ternary ring: an unfinished supergroup plus one unit
constexpr int kPRing = 6 * kG;                         // protected ring: an unfinished group plus one unit
constexpr int kPRingAt = kTRing * 2;                   // a head's row: 320 ternary entries, then 192 protected ones,
constexpr int kRingRow = (kTRing + kPRing) * 2 + 48;   // then padding: 1072 bytes, rows start in different banks
constexpr int kStpWarpBytes = kKBufBytes + kVBufBytes + kPGBytes + kTotBytes + 8 * kRingRow;
constexpr uint32_t kMinus4 = 0xc400c400u;              // binary16 pair (-4.0, -4.0)

// P V of one protected group (Eq. 4 codes as 4 + code): P4[nt] = probabilities of head hd at
// the group's tokens 8 nt + 2 r, + 1.  out += s * (sum (4 + code) p - 4 sum p) + z * sum p.
__device__ __forceinline__ void pv_protected(const uint8_t* pg, float* totbuf, const uint32_t (&P4)[4], float (&l)[2],
                                             int lane, int hd, int r, uint32_t m_field, uint32_t c_four) {
  float cq[4] = {0.0f, 0.0f, 0.0f, 0.0f};               // -4 * (sum of the probabilities) of heads 2 r, 2 r + 1
  mma_f16(cq, kMinus4, kMinus4, kMinus4, kMinus4, P4[0], P4[1]);
  mma_f16(cq, kMinus4, kMinus4, kMinus4, kMinus4, P4[2], P4[3]);
  const float sp0 = -0.25f * cq[0], sp1 = -0.25f * cq[1];
  l[0] += sp0; l[1] += sp1;
#pragma unroll 1
  for (int w = 0; w < 4; ++w) {
    const int w_off = (((w * 4) + r) * 8 + hd) * 4, m_off = (32 * w + 4 * hd) * 2;
    const uint32_t wk[2] = {*reinterpret_cast<const uint32_t*>(pg + w_off), *reinterpret_cast<const uint32_t*>(pg + 512 + w_off)};
    const uint2 sc = *reinterpret_cast<const uint2*>(pg + kPG_S + m_off);
    const uint2 zc = *reinterpret_cast<const uint2*>(pg + kPG_Z + m_off);
    float acc[2][4];
#pragma unroll
    for (int kt = 0; kt < 2; ++kt) {
      const uint32_t wd = wk[kt], wh = wd >> 6;
      uint32_t x[8];
      x[0] = and_or(wd << 8, m_field, c_four);
      x[1] = and_or(wd << 6, m_field, c_four);
      x[2] = and_or(wd << 4, m_field, c_four);
      x[3] = and_or(wd << 2, m_field, c_four);
      x[4] = and_or(wd, m_field, c_four);
      x[5] = and_or(wh << 4, m_field, c_four);
      x[6] = and_or(wh << 2, m_field, c_four);
      x[7] = and_or(wh, m_field, c_four);
      const uint32_t b0 = P4[2 * kt], b1 = P4[2 * kt + 1];
      if (kt == 0) {
        mma_f16_c(acc[0], x[0], x[1], x[4], x[5], b0, b1, cq[0], cq[1], cq[2], cq[3]);
        mma_f16_c(acc[1], x[2], x[3], x[6], x[7], b0, b1, cq[0], cq[1], cq[2], cq[3]);
      } else {
        mma_f16(acc[0], x[0], x[1], x[4], x[5], b0, b1);
        mma_f16(acc[1], x[2], x[3], x[6], x[7], b0, b1);
      }
    }
    const float2 sa = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));
    const float2 sb = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));
    const float2 za = __half22float2(*reinterpret_cast<const __half2*>(&zc.x));
    const float2 zb = __half22float2(*reinterpret_cast<const __half2*>(&zc.y));
    float4* tp = reinterpret_cast<float4*>(totbuf) + (2 * w) * 32 + lane;
    float4 t0 = tp[0], t1 = tp[32];
    t0.x += sa.x * acc[0][0] + za.x * sp0; t0.y += sa.x * acc[0][1] + za.x * sp1;
    t0.z += sa.y * acc[0][2] + za.y * sp0; t0.w += sa.y * acc[0][3] + za.y * sp1;
    t1.x += sb.x * acc[1][0] + zb.x * sp0; t1.y += sb.x * acc[1][1] + zb.x * sp1;
    t1.z += sb.y * acc[1][2] + zb.y * sp0; t1.w += sb.y * acc[1][3] + zb.y * sp1;
    tp[0] = t0;
    tp[32] = t1;
  }
}

// Zero the entries of stream positions [pos_begin, pos_end) in every head's row; `ring` points at
// entry 0 of the stream's part of row 0, ring_len is the stream's ring length.
__device__ __forceinline__ void zero_ring_range(uint8_t* ring, int ring_len, int pos_begin, int pos_end, int lane) {
  for (int pos = pos_begin + lane; pos < pos_end; pos += 32) {
    const int idx = pos % ring_len;
#pragma unroll
    for (int k = 0; k < 8; ++k) *reinterpret_cast<uint16_t*>(ring + k * kRingRow + idx * 2) = 0;
  }
}

}  // namespace

template <bool GEN>
__global__ void __launch_bounds__(kStreamWarps * 32, kStreamStpCtasPerSM) decode_stream_stp_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[kStreamWarps][3];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, hd = lane >> 2, r = lane & 3;
  const DecodePlan& pl = a.plan;
  const CacheView& cv = a.cv;
  const int run_id = blockIdx.x * kStreamWarps + warp;
  const int64_t u_begin = static_cast<int64_t>(run_id) * pl.run_units;
  const int64_t u_end = min(u_begin + pl.run_units, pl.n_units);
  if (u_begin >= u_end) return;
  const KeyFmt& kf = a.cv.kf;
  const int kgb = GEN ? kf.group_bytes : kKGroupBytes;
  constexpr int kbuf_bytes = GEN ? kGenKBufBytes : kKBufBytes;
  uint8_t* kbuf = smem_raw + warp * (kStpWarpBytes - kKBufBytes + kbuf_bytes);
  uint8_t* vbuf = kbuf + kbuf_bytes;
  uint8_t* pbuf = vbuf + kVBufBytes;
  float* totbuf = reinterpret_cast<float*>(pbuf + kPGBytes);
  uint8_t* rings = reinterpret_cast<uint8_t*>(totbuf) + kTotBytes;
  uint8_t* myrow = rings + hd * kRingRow;                  // the row of this lane's head
  uint64_t* kbar = &bars[warp][0];
  uint64_t* vbar = &bars[warp][1];
  uint64_t* pbar = &bars[warp][2];
  if (lane == 0) {
    mbar_init(kbar, 1);
    mbar_init(vbar, 1);
    mbar_init(pbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const uint32_t m_field = kExpand[0], c_four = kExpand[1], m_sign = kExpand[2], c_neg1 = kExpand[3];
  const int S = pl.units_per_slab;
  // token and stream positions fit 32 bits (the layout's group counts do)
  const int T_q0 = static_cast<int>(a.st.T_q0), T_qt = T_q0 + static_cast<int>(a.st.n_flush) * kR;
  const int n_groups = T_qt / kG, g0n = T_q0 / kG;
  const int n_prot = static_cast<int>(a.n_prot), n_rest = T_q0 - n_prot;
  const int u_fl0 = (n_rest + kG - 1) / kG * kG;                                          // flushed tokens start here
  const int tg_total = (n_rest + kG - 1) / kG + (kR / kG) * static_cast<int>(a.st.n_flush);   // ternary groups that exist
  const int sg_total = (tg_total + kSGGroups - 1) / kSGGroups;
  const int pg_total = (n_prot + kG - 1) / kG;
  const uint8_t* slab0 = cv.base + cv.slab_offset + static_cast<int64_t>(a.layer0) * cv.B * cv.H_kv * cv.slab_stride;
  int slab = static_cast<int>(u_begin / S);
  int k = static_cast<int>(u_begin - static_cast<int64_t>(slab) * S);
  auto groups_of = [&](int kk) -> int {
    const int left = n_groups - kk * kSGGroups;
    return left < kSGGroups ? left : kSGGroups;
  };
  auto key_src = [&](int sl, int kk) -> const uint8_t* {
    return slab0 + static_cast<int64_t>(sl) * cv.slab_stride + cv.kgroup_offset + static_cast<int64_t>(kk) * (kSGGroups * kgb);
  };
  if (lane == 0) bulk_load(kbuf, key_src(slab, k), groups_of(k) * kgb, kbar);
  pdl_wait();                                              // the prepared query (and nothing else so far) comes from the kernel before
  pdl_release();
  const uint32_t lt_mask = (1u << lane) - 1u;              // lanes (= tokens of a group) before this one
  uint32_t kpar = 0u, vpar = 0u, ppar = 0u;
  bool v_pending = false, p_pending = false;               // a copy into vbuf / pbuf has been issued and not yet waited for
  Running run;
  run.l[0] = 0.0f; run.l[1] = 0.0f; run.m = -INFINITY;
  uint32_t qa[8], qha[8], qhb[8];
  const uint32_t* ppc = nullptr;
  int cur_chunk = -1, cur_slab = -1;
  const uint32_t* prep_slab = nullptr;
  const uint32_t* ew = nullptr;
  const uint32_t* ep = nullptr;
  const uint8_t* slab_ptr = nullptr;
  int sg_next = 0, pg_next = 0;
  float sl2 = 0.0f;
  bool ok = true;
#pragma unroll 1
  for (int64_t u = u_begin; u < u_end && ok; ++u) {
    const int t_unit = k * kStreamUnitTokens;
    if (slab != cur_slab) {
      if (cur_slab >= 0) write_record(a, cur_slab, run_id, lane, hd, r, run, totbuf);
      cur_slab = slab;
      cur_chunk = -1;
      slab_ptr = slab0 + static_cast<int64_t>(slab) * cv.slab_stride;
      const int b = (slab / cv.H_kv) % cv.B;
      ew = cv.e_words(b);
      ep = cv.e_prefix(b);
      // zero the running output and both rings
      for (int i = lane; i < (kTotBytes + 8 * kRingRow) / 16; i += 32)
        reinterpret_cast<uint4*>(totbuf)[i] = make_uint4(0u, 0u, 0u, 0u);
      run.l[0] = 0.0f; run.l[1] = 0.0f;
      run.m = -INFINITY;
      prep_slab = a.prep + static_cast<int64_t>(slab) * pl.n_chunks * (kPrepWords * 32) + lane;
      sl2 = __uint_as_float(__ldg(prep_slab + 24 * 32));
      // where the run enters the two value streams
      int pp0, uu0;
      if (t_unit <= T_q0) { pp0 = static_cast<int>(__ldg(ep + t_unit / kG)); uu0 = t_unit - pp0; }
      else { pp0 = n_prot; uu0 = u_fl0 + (t_unit - T_q0); }
      sg_next = uu0 / kStreamUnitTokens;
      pg_next = pp0 / kG;
      __syncwarp();
      if (lane == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (sg_next < sg_total) bulk_load(vbuf, slab_ptr + cv.tern_offset + static_cast<int64_t>(sg_next) * kVBufBytes, kVBufBytes, vbar);
        if (pg_next < pg_total) bulk_load(pbuf, slab_ptr + cv.prot_offset + static_cast<int64_t>(pg_next) * kPGBytes, kPGBytes, pbar);
      }
      v_pending = sg_next < sg_total;
      p_pending = pg_next < pg_total;
    }
    const int ng = groups_of(k);
    int nslab = slab, nk = k + 1;
    if (nk == S) { nk = 0; ++nslab; }
    const bool more = u + 1 < u_end;
    const bool last_of_slab = !more || nslab != slab;      // the run leaves this slab after this unit
    // the E words and prefix counts of the unit's groups (lane g: group g; lane ng: the prefix count at the
    // unit's end) are fetched now and picked up with shuffles after the scores, their latency hidden behind them
    uint32_t e_word_l = 0u;
    int e_base_l = 0;
    {
      const int gl = t_unit / kG + lane;
      if (lane <= ng && gl * kG <= T_q0) {
        e_base_l = static_cast<int>(__ldg(ep + gl));
        if (lane < ng && gl * kG < T_q0) e_word_l = __ldg(ew + gl);
      }
    }
    // ---- scores of the unit's groups into the key buffer (raw scores, then the group's constant)
    if (!mbar_wait(kbar, kpar)) { ok = false; break; }
    kpar ^= 1u;
    float mx = -INFINITY;
#pragma unroll 1
    for (int g = 0; g < ng; ++g) {
      const int gidx = k * kSGGroups + g;
      const int chunk = gidx < g0n ? 0 : 1 + (gidx - g0n) / (kR / kG);
      if (chunk != cur_chunk) {
        cur_chunk = chunk;
        const uint32_t* pp = prep_slab + static_cast<int64_t>(chunk) * (kPrepWords * 32);
        ppc = pp;
        if (!GEN) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            qa[i] = __ldg(pp + i * 32);
            qha[i] = __ldg(pp + (8 + i) * 32);
            qhb[i] = __ldg(pp + (16 + i) * 32);
          }
        }
      }
      float sc[4][2], cst;
      uint8_t* kg = kbuf + g * kgb;
      if (GEN) score_group_general(kg, kf, lane, hd, r, ppc, m_field, c_four, m_sign, c_neg1, sc, cst);
      else score_group(kg, lane, hd, r, qa, qha, qhb, m_field, c_four, m_sign, c_neg1, sc, cst);
      __syncwarp();
      float gm = fmaxf(sc[0][0], sc[0][1]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        reinterpret_cast<float2*>(kg)[nt * 32 + lane] = make_float2(sc[nt][0], sc[nt][1]);
        gm = fmaxf(gm, fmaxf(sc[nt][0], sc[nt][1]));
      }
      reinterpret_cast<float*>(kg)[256 + lane] = cst;
      mx = fmaxf(mx, gm + cst);
    }
    // ---- running maximum (integral), exact rescale of everything that is kept in its units
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    {
      const float mu = mx * sl2;
      const bool up = mu > run.m + kStaleLog2;
      if (__any_sync(0xffffffffu, up)) {
        const float m_new = up ? ceilf(mu) : run.m;
        const float f = ex2_approx(run.m - m_new);          // a power of two (0 on the first unit)
        run.m = m_new;
        const float fa = __shfl_sync(0xffffffffu, f, 8 * r), fb = __shfl_sync(0xffffffffu, f, 8 * r + 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float4* t = reinterpret_cast<float4*>(totbuf) + j * 32 + lane;
          float4 v = *t;
          v.x *= fa; v.y *= fb; v.z *= fa; v.w *= fb;
          *t = v;
        }
        run.l[0] *= fa; run.l[1] *= fb;
        // probabilities waiting in the rings: row hd belongs to this lane's head, its four lanes share the row
        const __half2 f2 = __float2half2_rn(f);
        for (int i = r; i < kRingRow / 4; i += 4) {
          __half2* q = reinterpret_cast<__half2*>(myrow) + i;
          *q = __hmul2(*q, f2);
        }
        __syncwarp();
      }
    }
    // ---- probabilities, scattered into stream order.  Where a token goes depends on the token
    // alone, so lane j works out the destination of the group's token j (byte offset inside a
    // head's row: 2 * ternary ring index, or kPRingAt + 2 * protected ring index) and the lanes
    // pick up the destinations of their own four token pairs with shuffles.
#pragma unroll 1
    for (int g = 0; g < ng; ++g) {
      const uint8_t* kg = kbuf + g * kgb;
      const float off = fmaf(reinterpret_cast<const float*>(kg)[256 + lane], sl2, -run.m);
      const int tg = t_unit + g * kG;
      const uint32_t word = __shfl_sync(0xffffffffu, e_word_l, g);
      const int base = __shfl_sync(0xffffffffu, e_base_l, g);   // protected tokens before the group
      if (tg < T_q0) {
        const int below = __popc(word & lt_mask);
        const bool prot = (word >> lane) & 1u;
        int idx = prot ? (base + below) % kPRing : (tg - base + lane - below) % kTRing;
        uint32_t dst = static_cast<uint32_t>(prot ? kPRingAt + 2 * idx : 2 * idx);
        dst |= __shfl_down_sync(0xffffffffu, dst, 1) << 16;   // even lanes: this token and the next
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const float2 v = reinterpret_cast<const float2*>(kg)[nt * 32 + lane];
          const __half2 ph = __floats2half2_rn(ex2_approx(fmaf(v.x, sl2, off)), ex2_approx(fmaf(v.y, sl2, off)));
          const uint32_t d = __shfl_sync(0xffffffffu, dst, 8 * nt + 2 * r);
          *reinterpret_cast<__half*>(myrow + (d & 0xffffu)) = __low2half(ph);
          *reinterpret_cast<__half*>(myrow + (d >> 16)) = __high2half(ph);
        }
      } else {
        if (tg == T_q0 && u_fl0 > n_rest) zero_ring_range(rings, kTRing, n_rest, u_fl0, lane);   // the gap before the flushed tokens
        const int tmod = (u_fl0 + (tg - T_q0)) % kTRing;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const float2 v = reinterpret_cast<const float2*>(kg)[nt * 32 + lane];
          *reinterpret_cast<__half2*>(myrow + (tmod + 8 * nt + 2 * r) * 2) =
              __floats2half2_rn(ex2_approx(fmaf(v.x, sl2, off)), ex2_approx(fmaf(v.y, sl2, off)));
        }
      }
    }
    __syncwarp();
    if (more && lane == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      bulk_load(kbuf, key_src(nslab, nk), groups_of(nk) * kgb, kbar);
    }
    // ---- how far the two streams are complete now
    const int t_end = t_unit + ng * kG;
    int pp_hi, u_hi;
    if (t_end <= T_q0) { pp_hi = __shfl_sync(0xffffffffu, e_base_l, ng); u_hi = t_end - pp_hi; }
    else { pp_hi = n_prot; u_hi = u_fl0 + (t_end - T_q0); }
    if (last_of_slab) {
      // what is left of the last supergroup / group belongs to a neighbour (or to nobody): zeros
      const int sg_end = (u_hi + kStreamUnitTokens - 1) / kStreamUnitTokens * kStreamUnitTokens;
      zero_ring_range(rings, kTRing, u_hi, sg_end, lane);
      zero_ring_range(rings + kPRingAt, kPRing, pp_hi, (pp_hi + kG - 1) / kG * kG, lane);
      __syncwarp();
    }
    // ---- ternary supergroups whose positions are all written
    while (ok && (last_of_slab ? sg_next * kStreamUnitTokens < u_hi : (sg_next + 1) * kStreamUnitTokens <= u_hi)) {
      if (!mbar_wait(vbar, vpar)) { ok = false; break; }
      vpar ^= 1u;
      v_pending = false;
      uint32_t P[kSGGroups][4];
      float ps[kSGGroups][4];
      const uint8_t* rp = myrow + ((sg_next & 1) * kStreamUnitTokens + 2 * r) * 2;
#pragma unroll
      for (int g = 0; g < kSGGroups; ++g) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) P[g][nt] = *reinterpret_cast<const uint32_t*>(rp + (g * kG + 8 * nt) * 2);
        ps[g][0] = 0.0f; ps[g][1] = 0.0f; ps[g][2] = 0.0f; ps[g][3] = 0.0f;
        mma_f16(ps[g], kMinus5, kMinus5, kMinus5, kMinus5, P[g][0], P[g][1]);
        mma_f16(ps[g], kMinus5, kMinus5, kMinus5, kMinus5, P[g][2], P[g][3]);
        run.l[0] = fmaf(-0.2f, ps[g][0], run.l[0]);
        run.l[1] = fmaf(-0.2f, ps[g][1], run.l[1]);
      }
      pv_ternary<kSGGroups>(vbuf, totbuf, P, ps, lane, hd, r, m_field, c_four);
      ++sg_next;
      __syncwarp();
      if (sg_next < sg_total) {
        if (lane == 0) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          bulk_load(vbuf, slab_ptr + cv.tern_offset + static_cast<int64_t>(sg_next) * kVBufBytes, kVBufBytes, vbar);
        }
        v_pending = true;
      }
    }
    // ---- protected groups whose positions are all written
    while (ok && (last_of_slab ? pg_next * kG < pp_hi : (pg_next + 1) * kG <= pp_hi)) {
      if (!mbar_wait(pbar, ppar)) { ok = false; break; }
      ppar ^= 1u;
      p_pending = false;
      uint32_t P4[4];
      const uint8_t* rp = myrow + kPRingAt + ((pg_next % 6) * kG + 2 * r) * 2;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) P4[nt] = *reinterpret_cast<const uint32_t*>(rp + 8 * nt * 2);
      pv_protected(pbuf, totbuf, P4, run.l, lane, hd, r, m_field, c_four);
      ++pg_next;
      __syncwarp();
      if (pg_next < pg_total) {
        if (lane == 0) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          bulk_load(pbuf, slab_ptr + cv.prot_offset + static_cast<int64_t>(pg_next) * kPGBytes, kPGBytes, pbar);
        }
        p_pending = true;
      }
    }
    if (last_of_slab && ok) {
      // copies fetched ahead for a neighbour's part of the streams: let them land, the buffers are reused
      if (v_pending) { ok = mbar_wait(vbar, vpar); vpar ^= 1u; v_pending = false; }
      if (ok && p_pending) { ok = mbar_wait(pbar, ppar); ppar ^= 1u; p_pending = false; }
    }
    slab = nslab; k = nk;
  }
  if (!ok) {
    if (lane == 0) atomicCAS(reinterpret_cast<int*>(cv.base + kHdrStatus), VIDKV_OK, VIDKV_ERR_TIMEOUT);
    return;
  }
  write_record(a, cur_slab, run_id, lane, hd, r, run, totbuf);
}

cudaError_t launch_decode_stream_stp(const DecodeArgs& a, cudaStream_t stream) {
  const bool gen = a.cv.kf.general != 0;
  const size_t smem = static_cast<size_t>(kStreamWarps) * (kStpWarpBytes + (gen ? kGenKBufBytes - kKBufBytes : 0));
  static bool attr_set[64][2] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[dev][gen]) {
    const cudaError_t e = gen ? cudaFuncSetAttribute(decode_stream_stp_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                              : cudaFuncSetAttribute(decode_stream_stp_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set[dev][gen] = true;
  }
  const int grid = (a.plan.n_runs + kStreamWarps - 1) / kStreamWarps;
  if (grid < 1) return cudaSuccess;
  // with profiling events around the launch the kernel starts after the event, as an ordinary launch
  cudaError_t le;
  if (a.ev_begin) {
    if (gen) decode_stream_stp_kernel<true><<<grid, kStreamWarps * 32, smem, stream>>>(a);
    else decode_stream_stp_kernel<false><<<grid, kStreamWarps * 32, smem, stream>>>(a);
    le = cudaGetLastError();
  } else {
    le = gen ? launch_dependent(decode_stream_stp_kernel<true>, dim3(grid), dim3(kStreamWarps * 32), smem, stream, a)
             : launch_dependent(decode_stream_stp_kernel<false>, dim3(grid), dim3(kStreamWarps * 32), smem, stream, a);
  }
  count_launches(1);
  return le;
}

cudaError_t launch_decode_stream(const DecodeArgs& a_in, cudaStream_t stream) {
  DecodeArgs a = a_in;
  if (g_debug_withhold == 2) { a.withhold = 1; g_debug_withhold = 0; }
  const bool gen = a.cv.kf.general != 0;
  const size_t smem = static_cast<size_t>(kStreamWarps) * (kWarpBufBytes + (gen ? kGenKBufBytes - kKBufBytes : 0));
  static bool attr_set[64][2] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[dev][gen]) {
    const cudaError_t e = gen ? cudaFuncSetAttribute(decode_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                              : cudaFuncSetAttribute(decode_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set[dev][gen] = true;
  }
  const int grid = (a.plan.n_runs + kStreamWarps - 1) / kStreamWarps;
  if (grid < 1) return cudaSuccess;
  cudaError_t le;
  if (a.ev_begin) {
    if (gen) decode_stream_kernel<true><<<grid, kStreamWarps * 32, smem, stream>>>(a);
    else decode_stream_kernel<false><<<grid, kStreamWarps * 32, smem, stream>>>(a);
    le = cudaGetLastError();
  } else {
    le = gen ? launch_dependent(decode_stream_kernel<true>, dim3(grid), dim3(kStreamWarps * 32), smem, stream, a)
             : launch_dependent(decode_stream_kernel<false>, dim3(grid), dim3(kStreamWarps * 32), smem, stream, a);
  }
  count_launches(1);
  return le;
}

}  // namespace vidkv
