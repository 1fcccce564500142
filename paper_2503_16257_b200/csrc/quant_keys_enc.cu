// Key encode pass of Algorithm 3 (MixQuant) for one tile of 128 tokens x 128 channels:
//   normal channels   (Eq. 5) orthonormal 64-point DFT over the channel axis as one 128 x 64 x 64
//                     matrix product on the fifth-generation tensor cores (tcgen05.mma, operands
//                     in shared memory in the 128-byte-swizzled K-major layout, accumulator in
//                     tensor memory).  A = the tile's values, binary16, exact; B = the DFT matrix
//                     split into a binary16 leading part and a binary16 remainder, so that
//                     products carry 22 bits; float32 accumulation.  Then the sign bit and the
//                     per-group mean |.| of every spectrum column, one thread per token;
//   anomalous channels (Eq. 4) min / max per (32-token group, channel), s = (max - min) / 3,
//                     z = min rounded to binary16, code = clamp(rint((x - z) / s), 0, 3).
//                     The division is not done per element: code >= k is a monotone predicate
//                     of x, so per (group, channel) the three smallest element values X_k with
//                     code(X_k) >= k are found once with the defining float32 arithmetic, and
//                     the elements are compared against them two at a time.
// grid = (tiles of 128 tokens, slabs); block = 256 threads = 8 warps.
#include <math.h>

#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kEncTokens = 128;
constexpr int kRowBytes = 272;                 // 256 bytes of data + 16 of padding per staged token
constexpr int kDftWords = 4 * 8 * 32 * 4;      // [k step][column tile][lane][hi0, hi1, lo0, lo1]

// B fragments of the DFT matrix in the order the MMA wants them (see dft_table_kernel).
__device__ __align__(16) uint32_t g_dft_frag[kDftWords];

// The same matrix as the B operand of tcgen05.mma: two blocks (leading part, remainder) of
// [64 spectrum columns][64 channel positions] binary16, K-major with the 128-byte swizzle.
constexpr int kUmmaBlockBytes = 64 * 128;
__device__ __align__(1024) uint8_t g_dft_umma[2 * kUmmaBlockBytes];

// Byte offset of element (row, k) of a K-major operand with 64 binary16 per row under the
// 128-byte swizzle: 8-row atoms of 1024 bytes, 16-byte pieces XORed with the row within the atom.
__host__ __device__ constexpr int sw128_offset(int row, int k) {
  return (row >> 3) * 1024 + (row & 7) * 128 + ((((k >> 3) ^ row) & 7) << 4) + (k & 7) * 2;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<const __half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<const uint32_t*>(&v); }

// Element-type helpers: raw 16-bit patterns in, binary16 1.0 / 0.0 pairs out of the comparison.
template <typename T> struct Ops;
template <> struct Ops<__half> {
  static __device__ __forceinline__ float to_float(uint16_t b) { return __half2float(__ushort_as_half(b)); }
  static __device__ __forceinline__ uint16_t from_float_rn(float f) { return __half_as_ushort(__float2half_rn(f)); }
  static __device__ __forceinline__ uint16_t vmin(uint16_t a, uint16_t b) { return __half_as_ushort(__hmin(__ushort_as_half(a), __ushort_as_half(b))); }
  static __device__ __forceinline__ uint16_t vmax(uint16_t a, uint16_t b) { return __half_as_ushort(__hmax(__ushort_as_half(a), __ushort_as_half(b))); }
  static __device__ __forceinline__ uint32_t ge(uint32_t a, uint32_t b) { return as_u32(__hge2(as_h2(a), as_h2(b))); }
  static __device__ __forceinline__ uint32_t to_half_pair(uint32_t raw) { return raw; }
  static constexpr uint16_t kInf = 0x7c00u;
};
template <> struct Ops<__nv_bfloat16> {
  static __device__ __forceinline__ float to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
  static __device__ __forceinline__ uint16_t from_float_rn(float f) { return __bfloat16_as_ushort(__float2bfloat16_rn(f)); }
  static __device__ __forceinline__ uint16_t vmin(uint16_t a, uint16_t b) { return to_float(a) <= to_float(b) ? a : b; }
  static __device__ __forceinline__ uint16_t vmax(uint16_t a, uint16_t b) { return to_float(a) >= to_float(b) ? a : b; }
  static __device__ __forceinline__ uint32_t ge(uint32_t a, uint32_t b) {
    const __nv_bfloat162 r = __hge2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r) & 0x3c003c00u;   // bfloat16 1.0 -> binary16 1.0
  }
  static __device__ __forceinline__ uint32_t to_half_pair(uint32_t raw) {
    const __half2 h = __floats2half2_rn(__uint_as_float(raw << 16), __uint_as_float(raw & 0xffff0000u));
    return as_u32(h);
  }
  static constexpr uint16_t kInf = 0x7f80u;
};

// Value order of 16-bit sign-magnitude patterns as integers (both zeros map to 0).
__device__ __forceinline__ int ord_of(uint16_t b) { return (b & 0x8000u) ? -static_cast<int>(b & 0x7fffu) : static_cast<int>(b); }
__device__ __forceinline__ uint16_t bits_of(int o) { return o >= 0 ? static_cast<uint16_t>(o) : static_cast<uint16_t>(0x8000u | static_cast<uint32_t>(-o)); }

// Eq. 4 for one element, in the defining arithmetic (float32, IEEE division, round half to even):
// is the code of the element with value order o at least k?  (k = 1..3, so the clamp to [0, 3]
// does not change the answer.)
template <typename T>
__device__ __forceinline__ bool code_at_least(int o, float z, float s, float k) {
  const float d = __fsub_rn(Ops<T>::to_float(bits_of(o)), z);
  return rintf(__fdiv_rn(d, s)) >= k;
}

}  // namespace

// Column f of the DFT matrix at channel position c: f = 0: 1/8; f = 1: (-1)^c / 8;
// f = 2k: cos(2 pi k c / 64) / 8; f = 2k + 1: -sin(2 pi k c / 64) / 8.
__device__ double dft_weight(int f, int c) {
  if (f == 0) return 0.125;
  if (f == 1) return (c & 1) ? -0.125 : 0.125;
  double sn, cs;
  sincospi(static_cast<double>(((f >> 1) * c) & 63) / 32.0, &sn, &cs);
  return ((f & 1) ? -sn : cs) * 0.125;
}

// One block of 256 threads.  mma.sync fragments (used by the decode path for the query): word
// layout for k step ks, column tile nt and lane (n = lane / 4, r = lane % 4): rows
// k0 = 16 ks + 2 r (and k0 + 1; k0 + 8, k0 + 9) of column f = 16 (n / 2) + 2 nt + (n % 2), so
// that after the product lane (., r) holds the spectrum columns 16 r .. 16 r + 15 of its two rows.
__global__ void dft_table_kernel() {
  for (int i = threadIdx.x; i < kDftWords / 4; i += blockDim.x) {
    const int lane = i & 31, nt = (i >> 5) & 7, ks = i >> 8;
    const int n = lane >> 2, r = lane & 3;
    const int f = 16 * (n >> 1) + 2 * nt + (n & 1);
    float w[4];
    const int rows[4] = {16 * ks + 2 * r, 16 * ks + 2 * r + 1, 16 * ks + 2 * r + 8, 16 * ks + 2 * r + 9};
    for (int j = 0; j < 4; ++j) w[j] = static_cast<float>(dft_weight(f, rows[j]));
    const __half h0 = __float2half_rn(w[0]), h1 = __float2half_rn(w[1]), h2 = __float2half_rn(w[2]), h3 = __float2half_rn(w[3]);
    g_dft_frag[i * 4 + 0] = as_u32(__halves2half2(h0, h1));
    g_dft_frag[i * 4 + 1] = as_u32(__halves2half2(h2, h3));
    g_dft_frag[i * 4 + 2] = as_u32(__floats2half2_rn(w[0] - __half2float(h0), w[1] - __half2float(h1)));
    g_dft_frag[i * 4 + 3] = as_u32(__floats2half2_rn(w[2] - __half2float(h2), w[3] - __half2float(h3)));
  }
  // tcgen05 operand: row = spectrum column f, k = position c among the normal channels
  for (int i = threadIdx.x; i < 64 * 64; i += blockDim.x) {
    const int f = i >> 6, c = i & 63;
    const float w = static_cast<float>(dft_weight(f, c));
    const __half hi = __float2half_rn(w);
    const __half lo = __float2half_rn(w - __half2float(hi));
    *reinterpret_cast<__half*>(g_dft_umma + sw128_offset(f, c)) = hi;
    *reinterpret_cast<__half*>(g_dft_umma + kUmmaBlockBytes + sw128_offset(f, c)) = lo;
  }
}

// ---- tcgen05 helpers -------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// Shared-memory matrix descriptor of a K-major operand with one 128-byte swizzle atom along K:
// start address / 16, 8-row groups 1024 bytes apart, descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  return static_cast<uint64_t>((smem_addr >> 4) & 0x3fffu) | (static_cast<uint64_t>(1u) << 16) |
         (static_cast<uint64_t>(1024u >> 4) << 32) | (static_cast<uint64_t>(1u) << 46) | (static_cast<uint64_t>(2u) << 61);
}
// Instruction descriptor: float32 accumulator, binary16 A and B, both K-major, N = 64, M = 128.
constexpr uint32_t kUmmaIdesc = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr int kTmemCols = 64;
constexpr int kWaitLimit = 1 << 14;

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(kUmmaIdesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// 32 consecutive accumulator columns of the calling warp's 32 lanes of tensor memory.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared memory of one block, from a 1024-byte boundary:
//   [0, 16384)       A operand: the normal channels of the tile, [128 tokens][64 positions]
//   [16384, 51200)   the staged tile, [128][272] raw elements; once the tile has been sorted into
//                    the A operand and the gathered anomalous values, its first 16 KB take the B operand
//   [51200, 67584)   anomalous values gathered per code word
//   then thresholds [4][3][32] pairs, the channel order [128], the mbarrier, the tensor-memory address
constexpr int kSmAop = 0, kSmTile = 16384, kSmGath = kSmTile + kEncTokens * kRowBytes, kSmThr = kSmGath + 4 * 128 * 32,
              kSmPerm = kSmThr + 4 * 3 * 32 * 4, kSmBar = kSmPerm + kD, kSmEnd = kSmBar + 16;

size_t k_encode_smem_bytes() { return kSmEnd + 1024; }

template <typename T>
__global__ void __launch_bounds__(256, 3) k_encode_kernel(KSrc src, int64_t T_tokens, CacheView cv, int layer0,
                                                          int slabs_per_layer, int chunk, int64_t kgroup0) {
  extern __shared__ uint8_t esm_raw[];
  uint8_t* esm = esm_raw + ((1024u - (smem_u32(esm_raw) & 1023u)) & 1023u);
  uint8_t* aop = esm + kSmAop;
  uint8_t* tile = esm + kSmTile;
  uint16_t* gath = reinterpret_cast<uint16_t*>(esm + kSmGath);   // [group][word of the group's 2-bit block][16 slots]
  uint32_t* thr = reinterpret_cast<uint32_t*>(esm + kSmThr);
  uint8_t* perm = esm + kSmPerm;
  uint64_t* mbar = reinterpret_cast<uint64_t*>(esm + kSmBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(esm + kSmBar + 8);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int slab = blockIdx.y;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  uint8_t* slab_ptr = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv);
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * kEncTokens;
  const int n_tok = static_cast<int>(min(static_cast<int64_t>(kEncTokens), T_tokens - t0));   // multiple of 32
  const int n_groups = n_tok / kG;
  uint8_t* kg_base = slab_ptr + cv.kgroup_offset + (kgroup0 + t0 / kG) * kKGroupBytes;

  // ---- stage the tile; meanwhile set up the barrier and 64 columns of tensor memory
  {
    const int row0 = tid >> 4, piece = tid & 15;   // 16 threads per token row, 16 rows per sweep
    const uint8_t* srow = reinterpret_cast<const uint8_t*>(base + (t0 + row0) * src.stride_t) + piece * 16;
    uint8_t* drow = tile + row0 * kRowBytes + piece * 16;
    const int64_t sstep = 16 * src.stride_t * static_cast<int64_t>(sizeof(T));
#pragma unroll
    for (int it = 0; it < kEncTokens / 16; ++it)
      if (row0 + 16 * it < n_tok) cp_async16(drow + it * 16 * kRowBytes, srow + it * sstep);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  if (tid < kD) perm[tid] = slab_ptr[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(mbar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  // ---- A: Eq. 4 metadata and thresholds, thread = (anomalous slot j, group g)
  {
    const int j = tid & 63, g = tid >> 6;
    if (g < n_groups) {
      const uint8_t* p = tile + (g * kG) * kRowBytes + perm[j] * 2;
      // token t of the group goes to word ((t % 8) * 4 + j / 16) * 4 + t / 8, slot j % 16
      uint16_t* gp = gath + (g * 128 + (j >> 4) * 4) * 16 + (j & 15);
      uint16_t mn = *reinterpret_cast<const uint16_t*>(p), mx = mn;
      gp[0] = mn;
#pragma unroll
      for (int t = 1; t < kG; ++t) {
        const uint16_t v = *reinterpret_cast<const uint16_t*>(p + t * kRowBytes);
        mn = Ops<T>::vmin(mn, v); mx = Ops<T>::vmax(mx, v);
        gp[((t & 7) * 16 + (t >> 3)) * 16] = v;
      }
      const float fmn = Ops<T>::to_float(mn), fmx = Ops<T>::to_float(mx);
      const uint16_t sh = f2h_bits(__fdiv_rn(__fsub_rn(fmx, fmn), 3.0f));
      const uint16_t zh = f2h_bits(fmn);
      uint8_t* kg = kg_base + g * kKGroupBytes;
      reinterpret_cast<uint16_t*>(kg + kKG_S2)[j] = sh;
      reinterpret_cast<uint16_t*>(kg + kKG_Z2)[j] = zh;
      const float s = h2f(sh), z = h2f(zh);
      uint16_t* th = reinterpret_cast<uint16_t*>(thr + g * 3 * 32);
#pragma unroll 1
      for (int k = 1; k <= 3; ++k) {
        uint16_t X = Ops<T>::kInf;                     // s == 0: every code is 0
        if (s != 0.0f) {
          int o = ord_of(Ops<T>::from_float_rn(fmaf(static_cast<float>(k) - 0.5f, s, z)));
          // the threshold is almost always the candidate or its upper neighbour: two evaluations
          const float kf = static_cast<float>(k);
          const bool p0 = code_at_least<T>(o, z, s, kf);
          const bool p1 = code_at_least<T>(p0 ? o - 1 : o + 1, z, s, kf);
          if (p0 != p1) {
            o += p0 ? 0 : 1;
          } else if (p0) {
            o -= 1;
#pragma unroll 1
            for (int it = 0; it < 4 && code_at_least<T>(o - 1, z, s, kf); ++it) --o;
          } else {
            o += 2;
#pragma unroll 1
            for (int it = 0; it < 4 && !code_at_least<T>(o, z, s, kf); ++it) ++o;
          }
          X = bits_of(o);
        }
        th[(k - 1) * 64 + j] = X;
      }
    }
  }

  // ---- B: the normal channels as the A operand; warp = 16 tokens, lane = two channel positions
  if (warp * 16 < n_tok) {
    const uint32_t pc = *reinterpret_cast<const uint16_t*>(perm + kNA + 2 * lane);
    const int c0 = (pc & 0xffu) * 2, c1 = (pc >> 8) * 2;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int row = warp * 16 + i;
      const uint8_t* rp = tile + row * kRowBytes;
      const uint32_t raw = *reinterpret_cast<const uint16_t*>(rp + c0) | (static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(rp + c1)) << 16);
      *reinterpret_cast<uint32_t*>(aop + sw128_offset(row, 2 * lane)) = Ops<T>::to_half_pair(raw);
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  // ---- the tile is no longer needed: fetch the B operand (both parts of the matrix) over it
  {
    uint8_t* wdst = tile;
#pragma unroll
    for (int i = 0; i < 2 * kUmmaBlockBytes / (256 * 16); ++i) cp_async16(wdst + (i * 256 + tid) * 16, g_dft_umma + (i * 256 + tid) * 16);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  // ---- D: 2-bit codes, thread = one 32-bit word = (token, 16 slots), two words per thread
  {
    const int widx = tid & 127;
    const int r4 = (widx >> 2) & 3;
    const uint32_t k1024 = 0x64006400u;
    const uint32_t wgt[4] = {0x3c003c00u, 0x44004400u, 0x4c004c00u, 0x54005400u};   // 1, 4, 16, 64
#pragma unroll 1
    for (int g = tid >> 7; g < n_groups; g += 2) {
      const uint4* gv = reinterpret_cast<const uint4*>(gath + (g * 128 + widx) * 16);
      const uint4 v0 = gv[0], v1 = gv[1];
      const uint32_t v[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      const uint4* th = reinterpret_cast<const uint4*>(thr + g * 3 * 32 + 8 * r4);
      uint32_t x1[8], x2[8], x3[8];
      { const uint4 a0 = th[0], a1 = th[1]; x1[0] = a0.x; x1[1] = a0.y; x1[2] = a0.z; x1[3] = a0.w; x1[4] = a1.x; x1[5] = a1.y; x1[6] = a1.z; x1[7] = a1.w; }
      { const uint4 a0 = th[8], a1 = th[9]; x2[0] = a0.x; x2[1] = a0.y; x2[2] = a0.z; x2[3] = a0.w; x2[4] = a1.x; x2[5] = a1.y; x2[6] = a1.z; x2[7] = a1.w; }
      { const uint4 a0 = th[16], a1 = th[17]; x3[0] = a0.x; x3[1] = a0.y; x3[2] = a0.z; x3[3] = a0.w; x3[4] = a1.x; x3[5] = a1.y; x3[6] = a1.z; x3[7] = a1.w; }
      __half2 lo = as_h2(k1024), hi = as_h2(k1024);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const __half2 code = __hadd2(__hadd2(as_h2(Ops<T>::ge(v[i], x1[i])), as_h2(Ops<T>::ge(v[i], x2[i]))),
                                     as_h2(Ops<T>::ge(v[i], x3[i])));
        if (i < 4) lo = __hfma2(code, as_h2(wgt[i & 3]), lo);
        else hi = __hfma2(code, as_h2(wgt[i & 3]), hi);
      }
      // 1024 + n keeps n in the low byte of each lane: fields 0-3 and 4-7 of both half-words
      uint32_t word;
      asm("prmt.b32 %0, %1, %2, 0x6240;" : "=r"(word) : "r"(as_u32(lo)), "r"(as_u32(hi)));
      reinterpret_cast<uint32_t*>(kg_base + g * kKGroupBytes + kKG_Codes2)[widx] = word;
    }
  }

  // ---- the product: X[128 x 64] = A (leading part of the matrix) + A (remainder), K = 64 in four steps each
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint64_t da = umma_desc_sw128(smem_u32(aop));
    const uint64_t db = umma_desc_sw128(smem_u32(tile));
#pragma unroll
    for (int part = 0; part < 2; ++part) {
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)   // 16 binary16 = 32 bytes along K per step: the start address field counts 16 bytes
        umma_f16(tmem, da + static_cast<uint64_t>(2 * ks), db + static_cast<uint64_t>(part * (kUmmaBlockBytes >> 4) + 2 * ks),
                 (part | ks) != 0 ? 1u : 0u);
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(mbar)) : "memory");
  }
  // every thread waits for the accumulator; the wait is bounded, a timeout is reported in the status word
  uint32_t done = 0;
  for (int it = 0; it < kWaitLimit && !done; ++it) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(mbar)), "r"(0u) : "memory");
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  done = __all_sync(0xffffffffu, done != 0);

  // ---- sign bits and s = Mean |X| (Eq. 5): warp = (group g, 32 spectrum columns), lane = token
  const int g = warp & 3, half = warp >> 2;
  if (!done) {
    if (tid == 0) atomicCAS(reinterpret_cast<int*>(cv.base + kHdrStatus), 0, static_cast<int>(VIDKV_ERR_TIMEOUT));
  } else if (g < n_groups) {
    uint32_t x[32];
    tmem_ld32(tmem + (static_cast<uint32_t>(g * 32) << 16) + static_cast<uint32_t>(half * 32), x);
    // column e of a 16-column block goes to bit 15 - e of the block's half-word; 1 = coefficient >= 0
    uint32_t w = 0u;
#pragma unroll
    for (int c = 0; c < 32; ++c) w = __funnelshift_l(x[c], w, 1);
    w = ~w;
    uint16_t* hw = reinterpret_cast<uint16_t*>(kg_base + g * kKGroupBytes + kKG_Bits1);
    const int hidx = ((lane & 7) * 4 + 2 * half) * 4 + (lane >> 3);
    hw[hidx] = static_cast<uint16_t>(w >> 16);
    hw[hidx + 4] = static_cast<uint16_t>(w);
    // column sums of |X| over the group's 32 tokens: reduce-scatter over the lanes, lane l ends with column l
    float p[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) p[c] = fabsf(__uint_as_float(x[c]));
#pragma unroll
    for (int width = 16; width >= 1; width >>= 1) {
      const bool up = (lane & width) != 0;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (i < width) {
          const float send = up ? p[i] : p[i + width];
          const float keep = up ? p[i + width] : p[i];
          p[i] = keep + __shfl_xor_sync(0xffffffffu, send, width);
        }
      }
    }
    reinterpret_cast<uint16_t*>(kg_base + g * kKGroupBytes + kKG_S1)[half * 32 + lane] = f2h_bits(p[0] * (1.0f / 32.0f));
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------
// Host launcher of the encode pass
// ---------------------------------------------------------------------------------
// The DFT fragments are written once per device, ordered before their first use on `stream`
// (and, through the synchronisation, before any later use on another stream).
cudaError_t dft_fragments(const uint32_t** table, cudaStream_t stream) {
  static bool done[64] = {};
  static const uint32_t* addr[64] = {};
  cudaError_t e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev))) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!done[dev]) {
    void* p = nullptr;
    if ((e = cudaGetSymbolAddress(&p, g_dft_frag))) return e;
    dft_table_kernel<<<1, 256, 0, stream>>>();
    if ((e = cudaGetLastError())) return e;
    if ((e = cudaStreamSynchronize(stream))) return e;
    addr[dev] = static_cast<const uint32_t*>(p);
    done[dev] = true;
    count_launches(1);
  }
  *table = addr[dev];
  return cudaSuccess;
}

template <typename T>
static cudaError_t launch_encode_t(const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_slabs,
                                   int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream) {
  cudaError_t e;
  const uint32_t* table = nullptr;
  if ((e = dft_fragments(&table, stream))) return e;
  static bool attr_set = false;
  const size_t smem = k_encode_smem_bytes();
  if (!attr_set) {
    if ((e = cudaFuncSetAttribute(k_encode_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    if ((e = cudaFuncSetAttribute(k_encode_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    attr_set = true;
  }
  const int64_t blocks = (T_tokens + kEncTokens - 1) / kEncTokens;
  k_encode_kernel<T><<<dim3(static_cast<unsigned>(blocks), n_slabs), 256, smem, stream>>>(src, T_tokens, cv, layer0,
                                                                                         slabs_per_layer, chunk, kgroup0);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_encode_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_slabs,
                               int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream) {
  if (dtype == VIDKV_F16) return launch_encode_t<__half>(src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream);
  return launch_encode_t<__nv_bfloat16>(src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream);
}

}  // namespace vidkv
