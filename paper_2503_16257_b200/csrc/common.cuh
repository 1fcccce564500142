// Shared constants and small device helpers of libvidkv (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/vidkv.h"

namespace vidkv {

constexpr int kD = 128;            // head dimension
constexpr int kG = 32;             // group size (tokens per scale group)
constexpr int kR = 128;            // residual length
constexpr int kNA = 64;            // anomalous (2-bit) channels at k = 0.5
constexpr int kNF = 64;            // normal channels = spectrum columns (1-bit)
constexpr int kMaxRep = 8;         // query heads per KV head handled by one CTA

constexpr int kChunkBytes = 128;   // channel permutation of one chunk
constexpr int kKGroupBytes = 1152; // one 32-token key group
constexpr int kKG_Codes2 = 0, kKG_Bits1 = 512, kKG_S2 = 768, kKG_Z2 = 896, kKG_S1 = 1024;
constexpr int kSGGroups = 5;       // groups per ternary supergroup (5 trits per byte)
constexpr int kSGBytes = 5376;
constexpr int kSG_Scales = 4096;
constexpr int kPGBytes = 1536;     // one 32-token protected (2-bit) value group
constexpr int kPG_S = 1024, kPG_Z = 1280;
constexpr int kResBytes = kR * kD * 2;
constexpr int kHeaderBytes = 256;
constexpr int kHdrStatus = 8;      // byte offset of the device status word

constexpr uint32_t kMagic = 0x564b4456u;  // "VDKV"

// Key-group format of a cache (Algorithm 3 with its parameter k and the 1-bit mode).  The default
// (64 two-bit channels, Eq. 5 on the other 64) has the fixed layout above and its own kernels; every
// other combination uses the general layout, built from blocks of 32 channels:
//   [0, 256 n2b)            2-bit codes, block by block: lane l = 4 tl + r of a warp owns the 8 bytes
//                           8 l .. 8 l + 7 of a block = four 16-bit half-words, one per 8-token tile
//                           nt; the half-word of token t = 8 nt + tl holds the block's slots
//                           8 r + e: even e in the low byte, odd e in the high byte, at bits 2 (e / 2);
//   then 128 n1b bytes      1-bit codes, block by block: lane l owns the 32-bit word l of a block,
//                           byte nt of it holds columns 8 r + e of token 8 nt + tl at bit 7 - e;
//   then s (binary16) and z (binary16) of the n2 two-bit slots;
//   then s of the n1 one-bit columns (Eq. 5: spectrum columns of the orthonormal n1-point DFT of the
//   normal channels in Hermitian order; plain mode: the normal channels), and in plain mode their z.
struct KeyFmt {
  int32_t n2;            // two-bit (anomalous) channels: 32, 64, 96 or 128
  int32_t plain;         // 1: the one-bit channels carry the plain min/max code (Eq. 4 with n = 1), 0: Eq. 5
  int32_t general;       // 0: the default format with its fixed layout
  int32_t group_bytes;   // bytes of one 32-token key group
  int32_t off_bits1, off_s2, off_z2, off_s1, off_z1;   // general layout: byte offsets inside a group
  __host__ __device__ int n1() const { return kD - n2; }
};
inline KeyFmt make_key_fmt(int n2, int plain) {
  KeyFmt f;
  f.n2 = n2; f.plain = plain;
  f.general = !(n2 == kNA && !plain);
  if (!f.general) {
    f.group_bytes = kKGroupBytes;
    f.off_bits1 = kKG_Bits1; f.off_s2 = kKG_S2; f.off_z2 = kKG_Z2; f.off_s1 = kKG_S1; f.off_z1 = kKGroupBytes;
    return f;
  }
  const int n1 = kD - n2;
  f.off_bits1 = n2 * 8;
  f.off_s2 = f.off_bits1 + n1 * 4;
  f.off_z2 = f.off_s2 + n2 * 2;
  f.off_s1 = f.off_z2 + n2 * 2;
  f.off_z1 = f.off_s1 + n1 * 2;
  f.group_bytes = f.off_z1 + (plain ? n1 * 2 : 0);
  return f;
}
// The key format a configuration asks for (k_ratio and key_1bit_mode already validated).
inline KeyFmt key_fmt_of_config(const vidkv_config_t& c) {
  const int n2 = static_cast<int>(c.k_ratio * kD + 0.5f);
  return make_key_fmt(n2, (n2 < kD && c.key_1bit_mode == VIDKV_KEY1BIT_PLAIN_MINMAX) ? 1 : 0);
}
constexpr int kMaxKGroupBytes = 1536;   // the largest general key group (all channels at two bits)
// General layout: where slot j (of the n2 two-bit slots) / column f (of the n1 one-bit columns) of token t sits.
__host__ __device__ __forceinline__ int gk2_byte(int t, int j) {
  return (j >> 5) * 256 + ((t & 7) * 4 + ((j >> 3) & 3)) * 8 + (t >> 3) * 2 + (j & 1);
}
__host__ __device__ __forceinline__ int gk2_bit(int j) { return 2 * ((j & 7) >> 1); }
__host__ __device__ __forceinline__ int gk1_byte(int t, int f) {
  return (f >> 5) * 128 + ((t & 7) * 4 + ((f >> 3) & 3)) * 4 + (t >> 3);
}
__host__ __device__ __forceinline__ int gk1_bit(int f) { return 7 - (f & 7); }

// Device-side view of one cache: everything a kernel needs to find a slab region.
struct CacheView {
  uint8_t* base;
  KeyFmt kf;
  int64_t sel_offset, sel_stride_b, sel_words;
  int64_t slab_offset, slab_stride;
  int64_t chunk_table_offset, kgroup_offset, tern_offset, prot_offset, kres_offset, vres_offset;
  int32_t B, H_kv, H_q, rep;

  __host__ __device__ uint8_t* slab(int64_t layer, int64_t b, int64_t h) const {
    return base + slab_offset + ((layer * B + b) * H_kv + h) * slab_stride;
  }
  __host__ __device__ const uint32_t* e_words(int64_t b) const {
    return reinterpret_cast<const uint32_t*>(base + sel_offset + b * sel_stride_b);
  }
  __host__ __device__ const uint32_t* e_prefix(int64_t b) const {
    return e_words(b) + sel_words;
  }
};

template <typename T> struct Elem;
template <> struct Elem<__half> {
  static __device__ __forceinline__ float to_float(__half v) { return __half2float(v); }
  static __device__ __forceinline__ float2 to_float2(uint32_t v) {
    return __half22float2(*reinterpret_cast<__half2*>(&v));
  }
};
template <> struct Elem<__nv_bfloat16> {
  static __device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ float2 to_float2(uint32_t v) {
    return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v));
  }
};

__device__ __forceinline__ float h2f(uint16_t bits) {
  return __half2float(__ushort_as_half(bits));
}
__device__ __forceinline__ uint16_t f2h_bits(float v) {
  return __half_as_ushort(__float2half_rn(v));
}

// Monotone map float -> uint32 (for atomic min / max on floats).
__device__ __forceinline__ uint32_t float_ordered(float f) {
  uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ordered_float(uint32_t u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// Ternary byte code: five digits d in {0,1,2} (d = trit + 1), most significant first,
// b = sum d_g * 3^(4-g); the stored byte is ceil(256 * b / 243), which lets a decoder
// peel digits with multiply / shift and no division.
__host__ __device__ __forceinline__ uint32_t trit_byte_encode(uint32_t b) { return (256u * b + 242u) / 243u; }
__host__ __device__ __forceinline__ uint32_t trit_byte_decode(uint32_t q) { return (q * 243u) >> 8; }
// Byte plane of a ternary supergroup (4096 bytes = 32 stream tokens x 128 channels), laid out
// for the tensor-core decoder: token j = 2 m + parity, pair m = 8 kt + 4 u + r; channel
// c = 32 w + 4 rho + e.  The 8 bytes (e, parity) of one (m, w, rho) are contiguous, and the
// 32 (r, rho) combinations of one (kt, u, w) form one 256-byte run, so that a warp reads the
// operands of one 16-token MMA step with one conflict-free 64-bit load per lane.
__host__ __device__ __forceinline__ int tern_byte_offset(int j, int c) {
  const int m = j >> 1, kt = m >> 3, u = (m >> 2) & 1, r = m & 3;
  const int w = c >> 5, rho = (c >> 2) & 7, e = c & 3;
  return (((((kt * 2 + u) * 4 + w) * 4 + r) * 8 + rho) * 8) + 2 * e + (j & 1);
}
// 2-bit key codes of one 32-token group (512 bytes): token t = 8 nt + tl, anomalous slot
// j = 16 r + e.  Lane l = 4 tl + r of a warp owns the four 32-bit words 4 l .. 4 l + 3 (one per
// nt); inside a word, slot e sits at bit 2 (e / 2) + 16 (e % 2), i.e. even slots fill the low
// half-word and odd slots the high one (a binary16 pair comes out of one mask).
__host__ __device__ __forceinline__ int k2_word_index(int t, int j) { return ((t & 7) * 4 + (j >> 4)) * 4 + (t >> 3); }
__host__ __device__ __forceinline__ int k2_bit(int j) { return 2 * ((j & 15) >> 1) + 16 * (j & 1); }
// 1-bit key codes of one group (256 bytes): spectrum column f = 16 r + e of token t lives in
// the 16-bit half-word with the same index as the 2-bit word above, at bit 15 - e.
__host__ __device__ __forceinline__ int k1_half_index(int t, int f) { return ((t & 7) * 4 + (f >> 4)) * 4 + (t >> 3); }
__host__ __device__ __forceinline__ int k1_bit(int f) { return 15 - (f & 15); }
// 2-bit codes of one protected (STP) value group (1024 bytes = 256 words): protected token
// j = 16 kt + 8 u + 2 r + hf of the group, channel c = 32 w + 4 rho + e.  Word
// ((kt * 4 + w) * 4 + r) * 8 + rho holds 4 channels x 4 tokens: the code sits at bit
// 2 (4 u + e) + 16 hf, so the low half-word belongs to an even token, the high one to the
// next token, and one word yields the eight operand registers of one 16-token MMA step.
__host__ __device__ __forceinline__ int prot_word_index(int j, int c) {
  return ((((j >> 4) * 4 + (c >> 5)) * 4 + ((j >> 1) & 3)) * 8) + ((c >> 2) & 7);
}
__host__ __device__ __forceinline__ int prot_bit(int j, int c) { return 2 * (4 * ((j >> 3) & 1) + (c & 3)) + 16 * (j & 1); }
__host__ __device__ __forceinline__ int trit_digit(uint32_t b, int slot) {
  const uint32_t p3[5] = {81u, 27u, 9u, 3u, 1u};
  return static_cast<int>((b / p3[slot]) % 3u);
}

}  // namespace vidkv
