// Key encode pass of Algorithm 3 (MixQuant), one tile of 128 tokens x 128 channels at a time.
// The tile is the B operand of one product on the fifth-generation tensor cores (tcgen05.mma,
// operands in shared memory in the 128-byte-swizzled K-major layout, accumulators in tensor
// memory); the A operand has one row per output of the channel sort:
//   anomalous channels (Eq. 4) 64 selector rows (a single 1.0) copy the 64 anomalous channels
//                     exactly, so that accumulator row = slot, columns = tokens.  Per (slot,
//                     32-token group): min / max, s = (max - min) / 3, z = min rounded to
//                     binary16, code = clamp(rint((x - z) / s), 0, 3).  No division: code >= k
//                     is a monotone predicate of x, so the three smallest element values X_k
//                     with code(X_k) >= k are found once, with an exact test (code_at_least),
//                     and the elements are compared against them two at a time; the 2-bit
//                     fields are assembled into the cache's code words across lanes.
//   normal channels   (Eq. 5) 64 rows hold the columns of the orthonormal 64-point DFT over the
//                     channel axis, spread over the slab's normal channels and split into
//                     parts (binary16: 2, bfloat16: 3) so that products carry 22 - 24 bits;
//                     float32 accumulation.  Accumulator row = spectrum column: the sign bits
//                     and the per-group mean |.| are per-thread work, a warp-wide bit
//                     transpose gives the cache's (token, 16 columns) half-words.
// Persistent grid of two blocks per SM; block = 256 threads = 8 warps.
#include <math.h>

#include <algorithm>
#include <cstdint>

#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

namespace {

constexpr int kEncTokens = 128;
constexpr int kDftWords = 4 * 8 * 32 * 4;      // [k step][column tile][lane][hi0, hi1, lo0, lo1]

// B fragments of the DFT matrix in the order the MMA wants them (see dft_table_kernel).
__device__ __align__(16) uint32_t g_dft_frag[kDftWords];

// The same matrix as plain 16-bit patterns [part][spectrum column f][channel position c]:
// parts 0, 1: binary16 leading part and remainder; parts 2, 3, 4: bfloat16 leading, middle and
// last part (w = sum of the parts to 22 resp. 24 bits).
constexpr int kWParts = 5;
__device__ __align__(16) uint16_t g_dft_w[kWParts * 64 * 64];

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

// Eq. 4 for one element: is clamp(rint(RN(RN(x - z) / s)), 0, 3) >= k for the element with value
// order o (k = 1..3, s > 0)?  Decided without the division.  rint(q) >= k holds from q = 0.5 + 2^-24,
// 1.5 and 2.5 + 2^-22 on (round half to even), and the rounded quotient reaches that float exactly
// when the real quotient passes the midpoint below it: d / s > 0.5 + 2^-25, >= 1.5 - 2^-24,
// > 2.5 + 2^-23 (ties go to the even neighbour 0.5, 1.5, 2.5).  With c = k - 0.5 the sign of
// d - (c + delta) s is that of u - delta s, u = fma(-c, s, d): c s is exact, u is exact whenever
// d is within a factor two of c s (the only case where delta matters), delta s is a power of two times s.
template <typename T>
__device__ __forceinline__ bool code_at_least(int o, float z, float s, int k) {
  const float d = __fsub_rn(Ops<T>::to_float(bits_of(o)), z);
  const float u = fmaf(0.5f - static_cast<float>(k), s, d);
  if (k == 1) return u > 0x1p-25f * s;
  if (k == 2) return u >= -0x1p-24f * s;
  return u > 0x1p-23f * s;
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
  for (int i = threadIdx.x; i < 64 * 64; i += blockDim.x) {
    const int f = i >> 6, c = i & 63;
    const float w = static_cast<float>(dft_weight(f, c));
    const __half hi = __float2half_rn(w);
    g_dft_w[i] = __half_as_ushort(hi);
    g_dft_w[4096 + i] = __half_as_ushort(__float2half_rn(w - __half2float(hi)));
    const __nv_bfloat16 b0 = __float2bfloat16_rn(w);
    const float r1 = w - __bfloat162float(b0);
    const __nv_bfloat16 b1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(b1);
    g_dft_w[2 * 4096 + i] = __bfloat16_as_ushort(b0);
    g_dft_w[3 * 4096 + i] = __bfloat16_as_ushort(b1);
    g_dft_w[4 * 4096 + i] = __bfloat16_as_ushort(__float2bfloat16_rn(r2));
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
constexpr int kTmemCols = 256;        // two float32 accumulators of 128 x 128
constexpr int kWaitLimit = 1 << 14;

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
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
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// Per element type: how the DFT matrix is split (binary16: 2 parts, bfloat16: 3 parts), the
// operand format code of the instruction descriptor, and 1.0.
template <typename T> struct Enc;
template <> struct Enc<__half> {
  static constexpr int kParts = 2, kFmt = 0, kTab = 0;
  static constexpr uint16_t kOne = 0x3c00u;
  static __device__ __forceinline__ uint32_t pack(float a, float b) { return as_u32(__floats2half2_rn(a, b)); }
};
template <> struct Enc<__nv_bfloat16> {
  static constexpr int kParts = 3, kFmt = 1, kTab = 2;
  static constexpr uint16_t kOne = 0x3f80u;
  static __device__ __forceinline__ uint32_t pack(float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
  }
};

// Shared memory of one block, from a 1024-byte boundary.  All operands are K-major with the
// 128-byte swizzle, one 64-channel block of K after the other.
//   [0, 32768)     the tile as the B operand: [2 K blocks][128 tokens][64 channels]
//   then           X: the remaining parts of the DFT rows, per part [2 K blocks][64 rows][64 channels]
//                  A: the leading part, [2 K blocks][128 rows][64 channels].  Arrangement 0: row
//                  m < 64 selects the anomalous channel of slot m, row 64 + f holds column f of the
//                  DFT matrix spread over the normal channels (zero elsewhere); arrangement 1 swaps
//                  the two halves.
//                  The products of X use M = 128 too: in arrangement 0 the descriptor starts 64
//                  rows early, in arrangement 1 it runs 64 rows long; the extra rows read
//                  neighbouring shared memory and land in accumulator rows that nobody reads.
//   then the channel order [128], the mbarrier, the tensor-memory address, the fault flag
constexpr int kSmTile = 0, kSmAex = 32768;
template <typename T> __host__ __device__ constexpr int enc_sm_ahi() { return kSmAex + 16384 * (Enc<T>::kParts - 1); }
template <typename T> __host__ __device__ constexpr int enc_sm_perm() { return enc_sm_ahi<T>() + 32768; }
template <typename T> __host__ __device__ constexpr int enc_sm_bytes() { return enc_sm_perm<T>() + kD + 32 + 1024; }

size_t k_encode_smem_bytes(int dtype) { return dtype == VIDKV_F16 ? enc_sm_bytes<__half>() : enc_sm_bytes<__nv_bfloat16>(); }

// Persistent blocks, two per SM: block b encodes the tiles [n b / G, n (b + 1) / G) of the
// launch's n = slabs x tiles-per-slab tiles.  Warp w works on tensor-memory lanes 32 (w % 4):
// warps with w % 4 < 2 own 32 anomalous slots each, the others 32 spectrum columns each (and
// issue the tile loads); w / 4 picks two of the tile's four 32-token groups.
template <typename T>
__global__ void __launch_bounds__(256, 2) k_encode_kernel(KSrc src, int64_t T_tokens, CacheView cv, int layer0,
                                                          int slabs_per_layer, int chunk, int64_t kgroup0,
                                                          int tiles_per_slab, int total_tiles, int withhold_first) {
  extern __shared__ uint8_t esm_raw[];
  uint8_t* esm = esm_raw + ((1024u - (smem_u32(esm_raw) & 1023u)) & 1023u);
  uint8_t* tile = esm + kSmTile;
  uint8_t* a_hi = esm + enc_sm_ahi<T>();
  uint8_t* a_ex = esm + kSmAex;
  uint8_t* perm = esm + enc_sm_perm<T>();
  uint64_t* mbar = reinterpret_cast<uint64_t*>(perm + kD);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(perm + kD + 8);
  volatile uint32_t* fault = reinterpret_cast<volatile uint32_t*>(perm + kD + 12);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int quad = warp & 3, half = warp >> 2;
  // Row arrangement of the A operand: 0 puts the anomalous slots in rows 0 .. 63 and the DFT
  // columns in rows 64 .. 127, 1 the other way round.  The two blocks that share an SM (b and
  // b + G / 2 when blocks are handed out breadth first) take different arrangements so that the
  // heavier anomalous warps of one block sit on the schedulers of the lighter warps of the other.
  const int arr = (2 * blockIdx.x >= gridDim.x) ? 1 : 0;
  const bool loader = (quad >= 2) != (arr == 1);        // the spectrum warps also move the tiles
  const int lt = half * 64 + (quad & 1) * 32 + lane;    // 0 .. 127 among the loading threads

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(mbar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    *fault = 0u;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  const int tile_begin = static_cast<int>(static_cast<int64_t>(total_tiles) * blockIdx.x / gridDim.x);
  const int tile_end = static_cast<int>(static_cast<int64_t>(total_tiles) * (blockIdx.x + 1) / gridDim.x);

  // Tiles are walked as (slab, tile of the slab) pairs so that divisions happen once per block,
  // once for the tile being encoded and once for the tile being fetched.
  int slab = tile_begin / tiles_per_slab, ti = tile_begin - slab * tiles_per_slab;
  int lslab = slab, lti = ti, lbase_slab = -1;
  const T* lbase = nullptr;

  // 16-byte pieces of a tile: thread lt moves piece lt % 16 of the rows lt / 16 + 8 i
  auto load_next_tile = [&]() {
    if (lslab != lbase_slab) {
      lbase_slab = lslab;
      lbase = reinterpret_cast<const T*>(src.ptr) + (lslab / src.H) * src.stride_b + (lslab % src.H) * src.stride_h;
    }
    const int64_t t0 = static_cast<int64_t>(lti) * kEncTokens;
    const int n_tok = static_cast<int>(min(static_cast<int64_t>(kEncTokens), T_tokens - t0));
    const int row0 = lt >> 4, piece = lt & 15;
    const uint8_t* srow = reinterpret_cast<const uint8_t*>(lbase + (t0 + row0) * src.stride_t) + piece * 16;
    uint8_t* drow = tile + (piece >> 3) * 16384 + row0 * 128 + (((piece & 7) ^ row0) << 4);
    const int64_t sstep = 8 * src.stride_t * static_cast<int64_t>(sizeof(T));
#pragma unroll
    for (int i = 0; i < kEncTokens / 8; ++i)
      if (row0 + 8 * i < n_tok) cp_async16(drow + i * 1024, srow + i * sstep);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (++lti == tiles_per_slab) { lti = 0; ++lslab; }
  };

  int cur_slab = -1;
  uint32_t phase = 0;
  uint8_t* slab_ptr = nullptr;
  if (loader && tile_begin < tile_end) load_next_tile();
  for (int t = tile_begin; t < tile_end; ++t, ti = (ti + 1 == tiles_per_slab) ? 0 : ti + 1, slab += (ti == 0) ? 1 : 0) {
    if (slab != cur_slab) {
      const int layer = layer0 + slab / slabs_per_layer;
      const int bh = slab % slabs_per_layer;
      slab_ptr = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv);
    }
    const int64_t t0 = static_cast<int64_t>(ti) * kEncTokens;
    const int n_tok = static_cast<int>(min(static_cast<int64_t>(kEncTokens), T_tokens - t0));   // multiple of 32
    const int n_groups = n_tok / kG;
    uint8_t* kg_base = slab_ptr + cv.kgroup_offset + (kgroup0 + t0 / kG) * kKGroupBytes;

    // ---- a new slab: its channel order and the A operand built from it
    if (slab != cur_slab) {
      cur_slab = slab;
      if (tid < kD) perm[tid] = slab_ptr[cv.chunk_table_offset + static_cast<int64_t>(chunk) * kChunkBytes + tid];
      constexpr int kAVec = (32768 + 16384 * (Enc<T>::kParts - 1)) / 16;
      for (int i = tid; i < kAVec; i += 256) reinterpret_cast<uint4*>(a_ex)[i] = make_uint4(0u, 0u, 0u, 0u);
      __syncthreads();
      if (tid < kNA) {
        const int c = perm[tid];
        *reinterpret_cast<uint16_t*>(a_hi + (c >> 6) * 16384 + sw128_offset(64 * arr + tid, c & 63)) = Enc<T>::kOne;
      }
      for (int i = tid; i < 64 * 64; i += 256) {
        const int f = i >> 6, c = perm[kNA + (i & 63)];
        *reinterpret_cast<uint16_t*>(a_hi + (c >> 6) * 16384 + sw128_offset(64 - 64 * arr + f, c & 63)) = g_dft_w[Enc<T>::kTab * 4096 + i];
#pragma unroll
        for (int part = 1; part < Enc<T>::kParts; ++part)
          *reinterpret_cast<uint16_t*>(a_ex + (part - 1) * 16384 + (c >> 6) * 8192 + sw128_offset(f, c & 63)) =
              g_dft_w[(Enc<T>::kTab + part) * 4096 + i];
      }
    }

    // ---- the tile has landed; the accumulators of the previous tile have been read
    if (loader) asm volatile("cp.async.wait_group 0;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (*fault) break;

    // ---- D[128 rows x 128 tokens] = A (leading) x tile^T; D'[.. x ..] = A (remaining parts) x tile^T
    // (withhold_first, a test hook: the block's first tile gets neither products nor a commit, so the
    // wait below runs out with nothing outstanding)
    if (tid == 0 && !(withhold_first && t == tile_begin)) {
      constexpr uint32_t idesc = (1u << 4) | (static_cast<uint32_t>(Enc<T>::kFmt) << 7) | (static_cast<uint32_t>(Enc<T>::kFmt) << 10) |
                                 ((128u >> 3) << 17) | ((128u >> 4) << 24);
#pragma unroll
      for (int kb = 0; kb < 2; ++kb) {
        const uint64_t da = umma_desc_sw128(smem_u32(a_hi + kb * 16384)), db = umma_desc_sw128(smem_u32(tile + kb * 16384));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)   // 16 elements = 32 bytes along K per step; the address field counts 16 bytes
          umma_f16(tmem, da + static_cast<uint64_t>(2 * ks), db + static_cast<uint64_t>(2 * ks), idesc, (kb | ks) != 0 ? 1u : 0u);
      }
#pragma unroll
      for (int part = 1; part < Enc<T>::kParts; ++part) {
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          // the part's 64 rows are rows 64 .. 127 of arrangement 0 (start 8192 bytes early), rows 0 .. 63 of arrangement 1
          const uint64_t da = umma_desc_sw128(smem_u32(a_ex + (part - 1) * 16384 + kb * 8192 - (arr ? 0 : 8192)));
          const uint64_t db = umma_desc_sw128(smem_u32(tile + kb * 16384));
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            umma_f16(tmem + 128u, da + static_cast<uint64_t>(2 * ks), db + static_cast<uint64_t>(2 * ks), idesc,
                     (part - 1) | kb | ks ? 1u : 0u);
        }
      }
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(mbar)) : "memory");
    }
    // every thread waits for the accumulators; the wait is bounded, a timeout is reported in the status word
    uint32_t done = 0;
    for (int it = 0; it < kWaitLimit && !done; ++it) {
      asm volatile(
          "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(done) : "r"(smem_u32(mbar)), "r"(phase) : "memory");
    }
    phase ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    done = __all_sync(0xffffffffu, done != 0);
    if (!done) {
      if (lane == 0) {
        *fault = 1u;
        atomicCAS(reinterpret_cast<int*>(cv.base + kHdrStatus), 0, static_cast<int>(VIDKV_ERR_TIMEOUT));
      }
      continue;
    }
    // the products are done with shared memory: fetch the next tile behind the epilogue
    if (loader && t + 1 < tile_end) load_next_tile();

    if (!loader) {
      // ---- Eq. 4: lane = anomalous slot j, the accumulator row holds its 128 tokens (exact values)
      const int j = (quad & 1) * 32 + lane, wg = j >> 4;
      const int pos = (lane >> 1) & 3;                            // field of the slot inside its code byte
      const bool pb0 = (lane & 2) != 0, pb1 = (lane & 4) != 0;    // bits of pos
      const bool bb0 = (lane & 8) != 0, bb1 = (lane & 1) != 0;    // bits of the slot's byte index 2 (e % 2) + e / 8
      const uint32_t wgt = pos == 0 ? 0x3c003c00u : pos == 1 ? 0x44004400u : pos == 2 ? 0x4c004c00u : 0x54005400u;   // 4^pos
#pragma unroll 1
      for (int g = 2 * half; g < 2 * half + 2 && g < n_groups; ++g) {
        uint32_t x[32];
        tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(g * 32), x);
        float fmn = __uint_as_float(x[0]), fmx = fmn;
#pragma unroll
        for (int i = 1; i < 32; ++i) { fmn = fminf(fmn, __uint_as_float(x[i])); fmx = fmaxf(fmx, __uint_as_float(x[i])); }
        const uint16_t sh = f2h_bits(__fdiv_rn(__fsub_rn(fmx, fmn), 3.0f));
        const uint16_t zh = f2h_bits(fmn);
        uint8_t* kg = kg_base + g * kKGroupBytes;
        reinterpret_cast<uint16_t*>(kg + kKG_S2)[j] = sh;
        reinterpret_cast<uint16_t*>(kg + kKG_Z2)[j] = zh;
        const float sc = h2f(sh), z = h2f(zh);
        uint32_t thr[3];
#pragma unroll
        for (int k = 1; k <= 3; ++k) {
          uint16_t X = Ops<T>::kInf;                     // s == 0: every code is 0
          if (sc != 0.0f) {
            int o = ord_of(Ops<T>::from_float_rn(fmaf(static_cast<float>(k) - 0.5f, sc, z)));
            // the threshold is almost always the candidate or its upper neighbour: two evaluations
            const bool p0 = code_at_least<T>(o, z, sc, k);
            const bool p1 = code_at_least<T>(p0 ? o - 1 : o + 1, z, sc, k);
            if (p0 != p1) {
              o += p0 ? 0 : 1;
            } else if (p0) {
              o -= 1;
#pragma unroll 1
              for (int it = 0; it < 4 && code_at_least<T>(o - 1, z, sc, k); ++it) --o;
            } else {
              o += 2;
#pragma unroll 1
              for (int it = 0; it < 4 && !code_at_least<T>(o, z, sc, k); ++it) ++o;
            }
            X = bits_of(o);
          }
          thr[k - 1] = static_cast<uint32_t>(X) * 0x10001u;
        }
        // codes of token pairs as 1024 + code * 4^pos per 16-bit lane: the low byte of a lane is the
        // slot's contribution to the code byte of that token
        uint32_t w[8];   // w[tl]: bytes nt = 0..3 for the tokens tl + 8 nt
#pragma unroll
        for (int sp = 0; sp < 4; ++sp) {
          uint32_t h[4];
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            const int tp = sp + 4 * nt;   // tokens 2 sp + 8 nt and the next one
            const uint32_t v = Enc<T>::pack(__uint_as_float(x[2 * tp]), __uint_as_float(x[2 * tp + 1]));
            __half2 acc = __hfma2(as_h2(Ops<T>::ge(v, thr[0])), as_h2(wgt), as_h2(0x64006400u));
            acc = __hfma2(as_h2(Ops<T>::ge(v, thr[1])), as_h2(wgt), acc);
            acc = __hfma2(as_h2(Ops<T>::ge(v, thr[2])), as_h2(wgt), acc);
            h[nt] = as_u32(acc);
          }
          const uint32_t p01 = prmt(h[0], h[1], 0x6240u), p23 = prmt(h[2], h[3], 0x6240u);
          w[2 * sp] = prmt(p01, p23, 0x5410u);
          w[2 * sp + 1] = prmt(p01, p23, 0x7632u);
        }
        // OR over the four slots of a byte (lanes ^ 4, ^ 2), each lane keeping the token sets tl = 2 pos, 2 pos + 1
        uint32_t w1[4], w2[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t keep = pb1 ? w[4 + i] : w[i], send = pb1 ? w[i] : w[4 + i];
          w1[i] = keep | __shfl_xor_sync(0xffffffffu, send, 4);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const uint32_t keep = pb0 ? w1[2 + i] : w1[i], send = pb0 ? w1[i] : w1[2 + i];
          w2[i] = keep | __shfl_xor_sync(0xffffffffu, send, 2);
        }
        // gather the four bytes of a word from the four lanes that hold them (lanes ^ 8, ^ 1); the
        // lane ends with the words of token nt = 2 bb0 + bb1 of both of its token sets
        uint32_t u0, u1;
        {
          const uint32_t lo = prmt(w2[0], w2[1], 0x5410u), hi = prmt(w2[0], w2[1], 0x7632u);
          const uint32_t keep = bb0 ? hi : lo, recv = __shfl_xor_sync(0xffffffffu, bb0 ? lo : hi, 8);
          const uint32_t a = bb0 ? recv : keep, b = bb0 ? keep : recv;   // a: even byte of the pair, b: odd byte
          u0 = prmt(a, b, 0x5140u);
          u1 = prmt(a, b, 0x7362u);
        }
        {
          const uint32_t first = prmt(u0, u1, 0x5410u), second = prmt(u0, u1, 0x7632u);
          const uint32_t keep = bb1 ? second : first, recv = __shfl_xor_sync(0xffffffffu, bb1 ? first : second, 1);
          const uint32_t lowpair = bb1 ? recv : keep, highpair = bb1 ? keep : recv;
          const int nt = (bb0 ? 2 : 0) + (bb1 ? 1 : 0);
          uint32_t* codes = reinterpret_cast<uint32_t*>(kg + kKG_Codes2);
          codes[((2 * pos) * 4 + wg) * 4 + nt] = prmt(lowpair, highpair, 0x5410u);
          codes[((2 * pos + 1) * 4 + wg) * 4 + nt] = prmt(lowpair, highpair, 0x7632u);
        }
      }
    } else {
      // ---- Eq. 5: lane = spectrum column f, the two accumulators' rows 64 + f hold its 128 tokens
      const int hq = quad & 1, f = hq * 32 + lane;
#pragma unroll 1
      for (int g = 2 * half; g < 2 * half + 2 && g < n_groups; ++g) {
        uint32_t xa[32], xb[32];
        tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(g * 32), xa);
        tmem_ld32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(128 + g * 32), xb);
        float sum = 0.0f;
        uint32_t bits = 0u;   // bit i = sign bit of the column's coefficient of token i
#pragma unroll
        for (int i = 31; i >= 0; --i) {
          const float X = __uint_as_float(xa[i]) + __uint_as_float(xb[i]);
          sum += fabsf(X);
          bits = __funnelshift_l(__float_as_uint(X), bits, 1);
        }
        uint8_t* kg = kg_base + g * kKGroupBytes;
        reinterpret_cast<uint16_t*>(kg + kKG_S1)[f] = f2h_bits(sum * (1.0f / 32.0f));
        // 32 x 32 bit transpose over the warp: afterwards lane = token, bit l = column 32 hq + l
#pragma unroll
        for (int jb = 4; jb >= 0; --jb) {
          const int js = 1 << jb;
          const uint32_t m = jb == 4 ? 0x0000ffffu : jb == 3 ? 0x00ff00ffu : jb == 2 ? 0x0f0f0f0fu : jb == 1 ? 0x33333333u : 0x55555555u;
          const uint32_t y = __shfl_xor_sync(0xffffffffu, bits, js);
          const bool up = (lane & js) != 0;
          const uint32_t keep = up ? ~m : m;
          const uint32_t ysh = up ? (y >> js) : (y << js);
          bits = (bits & keep) | (ysh & ~keep);
        }
        // column e of a 16-column block goes to bit 15 - e of the block's half-word, 1 = coefficient >= 0
        const uint32_t mine = ~__brev(bits);
        uint16_t* hw = reinterpret_cast<uint16_t*>(kg + kKG_Bits1);
        const int hidx = ((lane & 7) * 4 + 2 * hq) * 4 + (lane >> 3);
        hw[hidx] = static_cast<uint16_t>(mine >> 16);
        hw[hidx + 4] = static_cast<uint16_t>(mine);
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  if (loader) asm volatile("cp.async.wait_group 0;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------
// Host launcher of the encode pass
// ---------------------------------------------------------------------------------
// The DFT fragments are written once per device by a small kernel on the stream of the first
// call that needs them, followed by an event; every call makes its stream wait for that event
// (free once it has completed), so uses on other streams are ordered after the fill without a
// host-side synchronisation.
cudaError_t dft_fragments(const uint32_t** table, cudaStream_t stream) {
  static bool done[64] = {};
  static const uint32_t* addr[64] = {};
  static cudaEvent_t ready[64] = {};
  cudaError_t e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev))) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!done[dev]) {
    void* p = nullptr;
    if ((e = cudaGetSymbolAddress(&p, g_dft_frag))) return e;
    if ((e = cudaEventCreateWithFlags(&ready[dev], cudaEventDisableTiming))) return e;
    dft_table_kernel<<<1, 256, 0, stream>>>();
    if ((e = cudaGetLastError())) return e;
    if ((e = cudaEventRecord(ready[dev], stream))) return e;
    addr[dev] = static_cast<const uint32_t*>(p);
    done[dev] = true;
    count_launches(1);
  } else if ((e = cudaStreamWaitEvent(stream, ready[dev], 0))) {
    return e;
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
  static int n_sms[64] = {};   // per device; 0 = the kernel's attributes are not set there yet
  constexpr int smem = enc_sm_bytes<T>();
  int dev = 0;
  if ((e = cudaGetDevice(&dev))) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (n_sms[dev] == 0) {
    if ((e = cudaFuncSetAttribute(k_encode_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem))) return e;
    if ((e = cudaDeviceGetAttribute(&n_sms[dev], cudaDevAttrMultiProcessorCount, dev))) return e;
  }
  const int64_t tiles_per_slab = (T_tokens + kEncTokens - 1) / kEncTokens;
  const int64_t total = tiles_per_slab * n_slabs;
  if (total <= 0) return cudaSuccess;
  if (total > INT32_MAX) return cudaErrorInvalidValue;
  const int blocks = static_cast<int>(std::min<int64_t>(total, 2 * n_sms[dev]));
  const int withhold = (g_debug_withhold == 1) ? 1 : 0;
  if (withhold) g_debug_withhold = 0;
  k_encode_kernel<T><<<blocks, 256, smem, stream>>>(src, T_tokens, cv, layer0, slabs_per_layer, chunk, kgroup0,
                                                    static_cast<int>(tiles_per_slab), static_cast<int>(total), withhold);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_encode_keys(int dtype, const KSrc& src, int64_t T_tokens, const CacheView& cv, int layer0, int n_slabs,
                               int slabs_per_layer, int chunk, int64_t kgroup0, cudaStream_t stream) {
  if (dtype == VIDKV_F16) return launch_encode_t<__half>(src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream);
  return launch_encode_t<__nv_bfloat16>(src, T_tokens, cv, layer0, n_slabs, slabs_per_layer, chunk, kgroup0, stream);
}

}  // namespace vidkv
