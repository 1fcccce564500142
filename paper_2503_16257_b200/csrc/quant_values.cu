// Value quantizer kernels: Algorithm 2 of the paper (1.58Quant, STPQuant), the token
// selection of Sec. 3.3(2), and the residual copies of Algorithm 1.
#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {

__device__ __forceinline__ __half2 as_half2(uint32_t v) { return *reinterpret_cast<const __half2*>(&v); }

// ---------------------------------------------------------------------------------
// 1.58Quant (Eq. 6) of one supergroup = 5 groups x 32 stream tokens x 128 channels.
// grid = (supergroups, slabs of one layer); block = 256 threads.
// Stream position u of the unprotected tokens maps to token idx_rest[u] (identity when
// no token is protected).
//   stage   the 160 x 128 tile is copied to shared memory as it is (cp.async, 16 bytes a piece);
//   pass 1  s = Mean |v| per (group, channel): thread = (channel pair, quarter of the group's
//           tokens), float32 partial sums combined in a fixed order;
//   pass 2  thread = one 32-bit word of the byte plane = (token pair, channel pair): the
//           comparisons |v| > alpha run on two channels at a time against the smallest
//           representable number above alpha = gamma * s, the five digits of a byte are
//           chained in binary16 (exact, <= 242), and the byte code comes from a 243-entry table.
// ---------------------------------------------------------------------------------
constexpr int kSGTokens = kSGGroups * kG;   // 160
constexpr int kVRowBytes = 272;             // 256 bytes of data + padding: rows four apart land 16 banks apart

template <typename T> struct Simd2;
template <> struct Simd2<__half> {
  // 1.0 / 0.0 in binary16 per lane
  static __device__ __forceinline__ uint32_t ge(uint32_t a, uint32_t b) {
    const __half2 r = __hge2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r);
  }
  static __device__ __forceinline__ uint32_t gt(uint32_t a, uint32_t b) {
    const __half2 r = __hgt2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r);
  }
  // smallest element value strictly above x >= 0
  static __device__ __forceinline__ uint16_t above(float x) {
    return static_cast<uint16_t>(__half_as_ushort(__float2half_rd(x)) + 1u);
  }
};
template <> struct Simd2<__nv_bfloat16> {
  // the comparison yields 1.0 in bfloat16 (0x3f80); keeping bits 10-13 turns it into binary16 1.0
  static __device__ __forceinline__ uint32_t ge(uint32_t a, uint32_t b) {
    const __nv_bfloat162 r = __hge2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r) & 0x3c003c00u;
  }
  static __device__ __forceinline__ uint32_t gt(uint32_t a, uint32_t b) {
    const __nv_bfloat162 r = __hgt2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r) & 0x3c003c00u;
  }
  static __device__ __forceinline__ uint16_t above(float x) {
    return static_cast<uint16_t>(__bfloat16_as_ushort(__float2bfloat16_rd(x)) + 1u);
  }
};

__device__ __forceinline__ void cp_async16_v(void* smem_dst, const void* gmem_src) {
  const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}

// NZ: the stored scale is the mean of |v| over the non-zero codes instead of Mean |v| (one more
// sweep over the staged tile; needs kSGGroups * 4 * kD more floats of shared memory).
template <typename T, bool NZ>
__global__ void __launch_bounds__(256) v_ternary_kernel(KSrc src, int64_t n_rest, CacheView cv, int layer0,
                                                        SelView sel, float gamma) {
  extern __shared__ __align__(16) uint8_t vsm[];
  uint8_t* tile = vsm;                                                         // [160][288]
  float* part = reinterpret_cast<float*>(tile + kSGTokens * kVRowBytes);       // [5][4][128]
  uint32_t* thr = reinterpret_cast<uint32_t*>(part + kSGGroups * 4 * kD);      // [5][64] threshold pairs
  uint8_t* lut = reinterpret_cast<uint8_t*>(thr + kSGGroups * 64);             // [256]
  float* cnt = reinterpret_cast<float*>(lut + 256);                            // [5][4][128], NZ only
  const int tid = threadIdx.x;
  const int slab = blockIdx.y;                              // over the layers of the call, then b, then h
  const int lb = slab / cv.H_kv, h = slab % cv.H_kv;
  const int b = lb % cv.B, layer = layer0 + lb / cv.B;
  const T* base = reinterpret_cast<const T*>(src.ptr) + static_cast<int64_t>(lb) * src.stride_b + h * src.stride_h;
  const int64_t u0 = static_cast<int64_t>(blockIdx.x) * kSGTokens;
  const int n_rows = static_cast<int>(min(static_cast<int64_t>(kSGTokens), n_rest - u0));
  const int32_t* idx = sel.idx_rest ? sel.idx_rest + b * sel.stride_rest : nullptr;
  // ---- stage (rows past the end of the stream are zero: their trits come out 0)
  {
    // thread = 16-byte piece (tid % 16) of rows tid / 16 + 16 k.  The stream positions of all its
    // rows are fetched first, so that the gather list costs one memory latency, not one per row.
    constexpr int kRowsPerThread = kSGTokens * 16 / 256;
    const int row0 = tid >> 4, piece = tid & 15;
    int64_t tok[kRowsPerThread];
#pragma unroll
    for (int k = 0; k < kRowsPerThread; ++k) {
      const int row = row0 + 16 * k;
      tok[k] = row < n_rows ? (idx ? static_cast<int64_t>(__ldg(idx + u0 + row)) : (u0 + row)) : -1;
    }
#pragma unroll
    for (int k = 0; k < kRowsPerThread; ++k) {
      uint8_t* dst = tile + (row0 + 16 * k) * kVRowBytes + piece * 16;
      if (tok[k] >= 0) cp_async16_v(dst, reinterpret_cast<const uint8_t*>(base + tok[k] * src.stride_t) + piece * 16);
      else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  if (tid < 243) lut[tid] = static_cast<uint8_t>(trit_byte_encode(tid));
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  uint8_t* sg = cv.slab(layer, b, h) + cv.tern_offset + static_cast<int64_t>(blockIdx.x) * kSGBytes;
  // ---- pass 1: partial sums of |v| over 8 tokens
  {
    const int cp = tid & 63, q = tid >> 6;
#pragma unroll
    for (int g = 0; g < kSGGroups; ++g) {
      float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(tile + (g * kG + q * 8 + j) * kVRowBytes + cp * 4);
        const float2 f = Elem<T>::to_float2(w);
        a0 += fabsf(f.x); a1 += fabsf(f.y);
      }
      *reinterpret_cast<float2*>(part + (g * 4 + q) * kD + 2 * cp) = make_float2(a0, a1);
    }
  }
  __syncthreads();
  for (int item = tid; item < kSGGroups * kD; item += 256) {
    const int c = item & (kD - 1), g = item >> 7;
    const int n = max(0, min(kG, n_rows - g * kG));
    uint16_t a = 1u;                                   // empty group: every v is 0, nothing exceeds it
    if (n > 0) {
      const float* pp = part + g * 4 * kD + c;
      const float sum = ((pp[0] + pp[kD]) + pp[2 * kD]) + pp[3 * kD];
      const uint16_t sh = f2h_bits(__fdiv_rn(sum, static_cast<float>(n)));
      if (!NZ) reinterpret_cast<uint16_t*>(sg + kSG_Scales)[g * kD + c] = sh;
      a = Simd2<T>::above(__fmul_rn(gamma, h2f(sh)));
    }
    reinterpret_cast<uint16_t*>(thr)[item] = a;
  }
  __syncthreads();
  if (NZ) {
    // ---- sums and counts of |v| over the elements whose code is not 0 (v >= A or v <= -A)
    const int cp = tid & 63, q = tid >> 6;
    const uint32_t one = 0x3c003c00u;
#pragma unroll
    for (int g = 0; g < kSGGroups; ++g) {
      const uint32_t A = thr[g * 64 + cp], nA = A ^ 0x80008000u;
      float a0 = 0.0f, a1 = 0.0f, c0 = 0.0f, c1 = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(tile + (g * kG + q * 8 + j) * kVRowBytes + cp * 4);
        const __half2 nz = __hsub2(__hadd2(as_half2(Simd2<T>::ge(w, A)), as_half2(one)), as_half2(Simd2<T>::gt(w, nA)));
        const float2 m = __half22float2(nz), f = Elem<T>::to_float2(w);
        a0 = fmaf(m.x, fabsf(f.x), a0); a1 = fmaf(m.y, fabsf(f.y), a1);
        c0 += m.x; c1 += m.y;
      }
      *reinterpret_cast<float2*>(part + (g * 4 + q) * kD + 2 * cp) = make_float2(a0, a1);
      *reinterpret_cast<float2*>(cnt + (g * 4 + q) * kD + 2 * cp) = make_float2(c0, c1);
    }
    __syncthreads();
    for (int item = tid; item < kSGGroups * kD; item += 256) {
      const int c = item & (kD - 1), g = item >> 7;
      if (n_rows - g * kG > 0) {
        const float* pp = part + g * 4 * kD + c;
        const float* pc = cnt + g * 4 * kD + c;
        const float sum = ((pp[0] + pp[kD]) + pp[2 * kD]) + pp[3 * kD];
        const float n_nz = ((pc[0] + pc[kD]) + pc[2 * kD]) + pc[3 * kD];
        reinterpret_cast<uint16_t*>(sg + kSG_Scales)[g * kD + c] = n_nz > 0.0f ? f2h_bits(__fdiv_rn(sum, n_nz)) : static_cast<uint16_t>(0);
      }
    }
  }
  // ---- pass 2: one word of the plane per thread and step
#pragma unroll
  for (int wi = 0; wi < kG * kD / 4 / 256; ++wi) {
    // bits 4 and 5 of the word index trade places: a warp then reads 16 words of each of two rows
    // that lie four rows apart (conflict-free with the 272-byte row stride) and still writes
    // whole 64-byte pieces of the plane
    const int w0 = tid + 256 * wi;
    const int wd = (w0 & ~0x30) | ((w0 & 0x10) << 1) | ((w0 & 0x20) >> 1);
    const int cp = 16 * ((wd >> 6) & 3) + 2 * ((wd >> 1) & 7) + (wd & 1);
    const int m = 8 * ((wd >> 9) & 1) + 4 * ((wd >> 8) & 1) + ((wd >> 4) & 3);
    uint32_t b0 = 0u, b1 = 0u;                        // binary16 pairs (even channel, odd channel) of tokens 2m, 2m+1
    const uint32_t three = 0x42004200u;
    const uint8_t* rp0 = tile + (2 * m) * kVRowBytes + cp * 4;
    const uint32_t* thp = thr + cp;
#pragma unroll
    for (int g = 0; g < kSGGroups; ++g) {
      const uint32_t A = thp[g * 64], nA = A ^ 0x80008000u;
      const uint8_t* rp = rp0 + g * (kG * kVRowBytes);
      const uint32_t v0 = *reinterpret_cast<const uint32_t*>(rp);
      const uint32_t v1 = *reinterpret_cast<const uint32_t*>(rp + kVRowBytes);
      // digit = [v > alpha] + [v >= -alpha] = [v >= A] + [v > -A]
      const __half2 d0 = __hadd2(as_half2(Simd2<T>::ge(v0, A)), as_half2(Simd2<T>::gt(v0, nA)));
      const __half2 d1 = __hadd2(as_half2(Simd2<T>::ge(v1, A)), as_half2(Simd2<T>::gt(v1, nA)));
      const __half2 t0 = __hfma2(as_half2(b0), *reinterpret_cast<const __half2*>(&three), d0);
      const __half2 t1 = __hfma2(as_half2(b1), *reinterpret_cast<const __half2*>(&three), d1);
      b0 = *reinterpret_cast<const uint32_t*>(&t0);
      b1 = *reinterpret_cast<const uint32_t*>(&t1);
    }
    // 1024 + b puts the integer b into the low mantissa bits
    const uint32_t k1024 = 0x64006400u;
    const __half2 e0 = __hadd2(as_half2(b0), *reinterpret_cast<const __half2*>(&k1024));
    const __half2 e1 = __hadd2(as_half2(b1), *reinterpret_cast<const __half2*>(&k1024));
    const uint32_t x0 = *reinterpret_cast<const uint32_t*>(&e0), x1 = *reinterpret_cast<const uint32_t*>(&e1);
    // word bytes: (even ch, tok 2m), (even ch, tok 2m+1), (odd ch, tok 2m), (odd ch, tok 2m+1)
    const uint32_t word = static_cast<uint32_t>(lut[x0 & 0xffu]) | (static_cast<uint32_t>(lut[x1 & 0xffu]) << 8) |
                          (static_cast<uint32_t>(lut[(x0 >> 16) & 0xffu]) << 16) |
                          (static_cast<uint32_t>(lut[(x1 >> 16) & 0xffu]) << 24);
    reinterpret_cast<uint32_t*>(sg)[wd] = word;
  }
}

// ---------------------------------------------------------------------------------
// 2-bit GQuant (Eq. 4) of one group of up to 32 protected tokens.  grid = (groups, slabs).
//
// code(v) = clamp(rint((v - z) / s), 0, 3) does not decrease with v, so it equals the number of
// k in {1, 2, 3} with v >= t_k, t_k the smallest value of the input type whose code reaches k.
// One thread per channel finds the three t_k with the literal formula (IEEE division included)
// evaluated on a handful of candidates around z + (k - 1/2) s; the elements are then coded with
// three comparisons each instead of a division each.
// ---------------------------------------------------------------------------------
template <typename T> struct Ordered16;     // 16-bit patterns of T <-> integers in value order
template <> struct Ordered16<__half> {
  static constexpr int kMin = 0x0400, kMax = 0xfbff;          // keys of -65504 and +65504
  static __device__ __forceinline__ float value(int key) {
    const uint16_t b = static_cast<uint16_t>(key ^ ((key & 0x8000) ? 0x8000 : 0xffff));
    return __half2float(__ushort_as_half(b));
  }
  static __device__ __forceinline__ int key(float x) {
    const uint16_t b = __half_as_ushort(__float2half_rn(x));
    return b ^ ((b & 0x8000u) ? 0xffffu : 0x8000u);
  }
};
template <> struct Ordered16<__nv_bfloat16> {
  static constexpr int kMin = 0x0080, kMax = 0xff7f;          // keys of the largest finite magnitudes
  static __device__ __forceinline__ float value(int key) {
    const uint32_t b = static_cast<uint32_t>(key ^ ((key & 0x8000) ? 0x8000 : 0xffff));
    return __uint_as_float(b << 16);
  }
  static __device__ __forceinline__ int key(float x) {
    const uint16_t b = __bfloat16_as_ushort(__float2bfloat16_rn(x));
    return b ^ ((b & 0x8000u) ? 0xffffu : 0x8000u);
  }
};

// Smallest value of type T (as a float) whose Eq. 4 code with (s, z) is >= k; +infinity if none.
template <typename T>
__device__ __forceinline__ float code_threshold(float s, float z, int k) {
  using O = Ordered16<T>;
  if (!(s > 0.0f)) return INFINITY;                            // zero range: every code is 0
  const float kf = static_cast<float>(k);
  auto reaches = [&](int key) -> bool {
    float q = rintf(__fdiv_rn(__fsub_rn(O::value(key), z), s));
    q = fminf(fmaxf(q, 0.0f), 3.0f);
    return q >= kf;
  };
  const int ck = min(max(O::key(fmaf(kf - 0.5f, s, z)), O::kMin), O::kMax);
  int lo = max(ck - 4, O::kMin - 1), hi = min(ck + 4, O::kMax);   // invariant: code(lo) < k <= code(hi)
  if (!reaches(hi)) {
    lo = hi; hi = O::kMax;
    if (!reaches(hi)) return INFINITY;
  }
  if (lo >= O::kMin && reaches(lo)) { hi = lo; lo = O::kMin - 1; }
  while (hi - lo > 1) {                                        // at most 16 rounds
    const int mid = (lo + hi) >> 1;
    if (reaches(mid)) hi = mid; else lo = mid;
  }
  return O::value(hi);
}

template <typename T>
__global__ void __launch_bounds__(128) v_protect_kernel(KSrc src, CacheView cv, int layer0, SelView sel) {
  __shared__ __align__(16) uint16_t tile[kG * kD];
  __shared__ float s_thr[3][kD];
  const int slab = blockIdx.y;
  const int lb = slab / cv.H_kv, h = slab % cv.H_kv;
  const int b = lb % cv.B, layer = layer0 + lb / cv.B;
  const T* base = reinterpret_cast<const T*>(src.ptr) + static_cast<int64_t>(lb) * src.stride_b + h * src.stride_h;
  const int64_t p0 = static_cast<int64_t>(blockIdx.x) * kG;
  const int n_rows = static_cast<int>(min(static_cast<int64_t>(kG), sel.n_prot - p0));
  const int32_t* idx = sel.idx_prot + b * sel.stride_prot;
  {
    const int lane16 = threadIdx.x & 15, row = threadIdx.x >> 4;
    for (int r = row; r < kG; r += 8) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < n_rows) v = __ldg(reinterpret_cast<const uint4*>(base + static_cast<int64_t>(idx[p0 + r]) * src.stride_t) + lane16);
      reinterpret_cast<uint4*>(tile + r * kD)[lane16] = v;
    }
  }
  __syncthreads();
  uint8_t* pg = cv.slab(layer, b, h) + cv.prot_offset + static_cast<int64_t>(blockIdx.x) * kPGBytes;
  {
    const int c = threadIdx.x;
    float mn = INFINITY, mx = -INFINITY;
    for (int j = 0; j < n_rows; ++j) {
      const float v = Elem<T>::to_float(reinterpret_cast<const T*>(tile)[j * kD + c]);
      mn = fminf(mn, v); mx = fmaxf(mx, v);
    }
    const uint16_t sh = f2h_bits(__fdiv_rn(__fsub_rn(mx, mn), 3.0f)), zh = f2h_bits(mn);
    reinterpret_cast<uint16_t*>(pg + kPG_S)[c] = sh;
    reinterpret_cast<uint16_t*>(pg + kPG_Z)[c] = zh;
    const float s = h2f(sh), z = h2f(zh);
#pragma unroll
    for (int k = 1; k <= 3; ++k) s_thr[k - 1][c] = code_threshold<T>(s, z, k);
  }
  __syncthreads();
  for (int item = threadIdx.x; item < kG * 8; item += 128) {
    // item = word index ((kt * 4 + w) * 4 + r) * 8 + rho: 4 channels x 4 tokens
    const int rho = item & 7, r = (item >> 3) & 3, w = (item >> 5) & 3, kt = item >> 7;
    const int c0 = 32 * w + 4 * rho;
    float t1[4], t2[4], t3[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { t1[e] = s_thr[0][c0 + e]; t2[e] = s_thr[1][c0 + e]; t3[e] = s_thr[2][c0 + e]; }
    uint32_t word = 0;
#pragma unroll
    for (int f = 0; f < 16; ++f) {
      const int e = f & 3, u = (f >> 2) & 1, hf = f >> 3;
      const int j = 16 * kt + 8 * u + 2 * r + hf;
      if (j < n_rows) {
        const float v = Elem<T>::to_float(reinterpret_cast<const T*>(tile)[j * kD + c0 + e]);
        const uint32_t code = static_cast<uint32_t>(v >= t1[e]) + static_cast<uint32_t>(v >= t2[e]) + static_cast<uint32_t>(v >= t3[e]);
        word |= code << (2 * (4 * u + e) + 16 * hf);
      }
    }
    reinterpret_cast<uint32_t*>(pg)[item] = word;
  }
}

// ---------------------------------------------------------------------------------
// Residual flush, value half (Algorithm 1, Decoding): 1.58Quant of the 128 residual tokens
// of every slab, appended as 4 groups at ternary stream group index tgroup0.  The groups
// may land in a supergroup that already holds earlier groups, so bytes are updated digit
// by digit.  grid = slabs (over layers); block = 128 threads (thread = channel).
// ---------------------------------------------------------------------------------
template <typename T, bool NZ>
__global__ void __launch_bounds__(kD) v_flush_kernel(KSrc src, CacheView cv, int layer0, int slabs_per_layer,
                                                     int64_t tgroup0, float gamma) {
  const int slab = blockIdx.x;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  const T* base = reinterpret_cast<const T*>(src.ptr) + (slab / src.H) * src.stride_b + (slab % src.H) * src.stride_h;
  uint8_t* tern = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv) + cv.tern_offset;
  const int c = threadIdx.x;
  const uint32_t p3[5] = {81u, 27u, 9u, 3u, 1u};
  for (int g4 = 0; g4 < kR / kG; ++g4) {
    const int64_t gi = tgroup0 + g4;
    uint8_t* sg = tern + (gi / kSGGroups) * kSGBytes;
    const int slot = static_cast<int>(gi % kSGGroups);
    float sum = 0.0f;
    for (int j = 0; j < kG; ++j) sum += fabsf(Elem<T>::to_float(base[(g4 * kG + j) * src.stride_t + c]));
    const uint16_t sh = f2h_bits(__fdiv_rn(sum, static_cast<float>(kG)));
    const float a = __fmul_rn(gamma, h2f(sh));
    float nz_sum = 0.0f, nz_cnt = 0.0f;
    for (int j = 0; j < kG; ++j) {
      const float v = Elem<T>::to_float(base[(g4 * kG + j) * src.stride_t + c]);
      const uint32_t d = v > a ? 2u : (v < -a ? 0u : 1u);
      if (NZ && d != 1u) { nz_sum += fabsf(v); nz_cnt += 1.0f; }
      const uint32_t bold = trit_byte_decode(sg[tern_byte_offset(j, c)]);
      const uint32_t dold = (bold / p3[slot]) % 3u;
      sg[tern_byte_offset(j, c)] = static_cast<uint8_t>(trit_byte_encode(bold - dold * p3[slot] + d * p3[slot]));
    }
    // the stored scale: Mean |v|, or the mean of |v| over the non-zero codes (0 where there is none)
    reinterpret_cast<uint16_t*>(sg + kSG_Scales)[slot * kD + c] =
        !NZ ? sh : (nz_cnt > 0.0f ? f2h_bits(__fdiv_rn(nz_sum, nz_cnt)) : static_cast<uint16_t>(0));
  }
}

// ---------------------------------------------------------------------------------
// Residual copies (Algorithm 1: X_r = X[l - r:], and the per-step append).
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void copy_to_residual_kernel(KSrc src, int64_t t_begin, int n_tok, CacheView cv, int layer0,
                                        int64_t res_offset, int r0) {
  const int slab = blockIdx.x;
  const int lb = slab / cv.H_kv, h = slab % cv.H_kv;
  const int b = lb % cv.B, layer = layer0 + lb / cv.B;
  const T* base = reinterpret_cast<const T*>(src.ptr) + static_cast<int64_t>(lb) * src.stride_b + h * src.stride_h;
  uint4* dst = reinterpret_cast<uint4*>(cv.slab(layer, b, h) + res_offset);
  for (int i = threadIdx.x; i < n_tok * 16; i += blockDim.x) {
    const int r = i >> 4, l = i & 15;
    dst[(r0 + r) * 16 + l] = __ldg(reinterpret_cast<const uint4*>(base + (t_begin + r) * src.stride_t) + l);
  }
}

// One block of 32 threads per (layer, b, h): lanes 0-15 copy the key row, 16-31 the value row.
__global__ void append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, CacheView cv,
                              int layer0, int slabs_per_layer, int row) {
  const int slab = blockIdx.x;
  const int layer = layer0 + slab / slabs_per_layer;
  const int bh = slab % slabs_per_layer;
  uint8_t* sp = cv.slab(layer, bh / cv.H_kv, bh % cv.H_kv);
  const int l = threadIdx.x & 15;
  if (threadIdx.x < 16)
    reinterpret_cast<uint4*>(sp + cv.kres_offset)[row * 16 + l] = __ldg(k_new + static_cast<int64_t>(slab) * 16 + l);
  else
    reinterpret_cast<uint4*>(sp + cv.vres_offset)[row * 16 + l] = __ldg(v_new + static_cast<int64_t>(slab) * 16 + l);
}

// ---------------------------------------------------------------------------------
// Token selection: top n of l_v saliency scores per batch element (ties: lower index).
// One block of 1024 threads per batch element.  Phase 1: 4-pass radix select of the n-th
// largest key.  Phase 2: E words, per-word prefix counts and the two gather lists.
// ---------------------------------------------------------------------------------
__device__ __forceinline__ int block_exclusive_scan_1024(int v, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += y;
    }
    s_warp[lane] = w;
  }
  __syncthreads();
  const int warp_off = warp ? s_warp[warp - 1] : 0;
  *total = s_warp[31];
  __syncthreads();
  return warp_off + x - v;
}

// mode 0: from saliency (radix select); mode 1: from a byte mask E [B][T].
__global__ void __launch_bounds__(1024) select_tokens_kernel(const float* __restrict__ saliency,
                                                             const uint8_t* __restrict__ mask, int64_t mask_stride,
                                                             int64_t vis_begin, int64_t l_v, int64_t n_prot,
                                                             int64_t T_q, CacheView cv, int32_t* idx_prot,
                                                             int32_t* idx_rest, int64_t stride_prot,
                                                             int64_t stride_rest, int32_t* counts,
                                                             int64_t expect_count) {
  __shared__ int hist[256];
  __shared__ int s_warp[32];
  __shared__ uint32_t s_prefix, s_need;
  const int b = blockIdx.x;
  const float* sal = saliency ? saliency + b * l_v : nullptr;
  uint32_t thr = 0, need = 0;
  if (sal && n_prot > 0) {
    uint32_t prefix = 0, pmask = 0;
    need = static_cast<uint32_t>(n_prot);
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (threadIdx.x < 256) hist[threadIdx.x] = 0;
      __syncthreads();
      for (int64_t i = threadIdx.x; i < l_v; i += 1024) {
        const uint32_t key = float_ordered(sal[i]);
        if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        uint32_t cum = 0;
        int d = 255;
        for (; d > 0; --d) {
          if (cum + hist[d] >= need) break;
          cum += hist[d];
        }
        s_prefix = prefix | (static_cast<uint32_t>(d) << shift);
        s_need = need - cum;
      }
      __syncthreads();
      prefix = s_prefix; need = s_need;
      pmask |= 255u << shift;
      __syncthreads();
    }
    thr = prefix;       // key of the n-th largest; `need` of the keys equal to it are taken
  }
  uint32_t* e_words = const_cast<uint32_t*>(cv.e_words(b));
  uint32_t* e_prefix = const_cast<uint32_t*>(cv.e_prefix(b));
  const int64_t W = T_q / kG;
  int eq_carry = 0, prot_carry = 0;
  for (int64_t wbase = 0; wbase < W; wbase += 1024) {
    const int64_t w = wbase + threadIdx.x;
    uint32_t word_gt = 0, word_eq = 0;
    if (w < W) {
      for (int i = 0; i < 32; ++i) {
        const int64_t t = w * 32 + i;
        if (mask) {
          if (mask[b * mask_stride + t]) word_gt |= 1u << i;
        } else if (sal && n_prot > 0 && t >= vis_begin && t < vis_begin + l_v) {
          const uint32_t key = float_ordered(sal[t - vis_begin]);
          if (key > thr) word_gt |= 1u << i;
          else if (key == thr) word_eq |= 1u << i;
        }
      }
    }
    int total;
    int eq_before = block_exclusive_scan_1024(__popc(word_eq), s_warp, &total) + eq_carry;
    eq_carry += total;
    uint32_t word = word_gt;
    int take = static_cast<int>(need) - eq_before;
    for (uint32_t rem = word_eq; rem && take > 0; rem &= rem - 1, --take) word |= rem & (0u - rem);
    int prot_before = block_exclusive_scan_1024(__popc(word), s_warp, &total) + prot_carry;
    prot_carry += total;
    if (w < W) {
      e_words[w] = word;
      e_prefix[w] = static_cast<uint32_t>(prot_before);
      int pk = prot_before;
      for (int i = 0; i < 32; ++i) {
        const int64_t t = w * 32 + i;
        if (word & (1u << i)) { if (idx_prot && pk < stride_prot) idx_prot[b * stride_prot + pk] = static_cast<int32_t>(t); ++pk; }
        else if (idx_rest) idx_rest[b * stride_rest + (t - pk)] = static_cast<int32_t>(t);
      }
    }
  }
  if (threadIdx.x == 0) {
    e_prefix[W] = static_cast<uint32_t>(prot_carry);
    e_words[W] = 0;
    if (counts) counts[b] = prot_carry;
    // a mask whose row does not protect the number of tokens the caller stated
    if (expect_count >= 0 && prot_carry != expect_count)
      atomicCAS(reinterpret_cast<int*>(cv.base + kHdrStatus), VIDKV_OK, VIDKV_ERR_INVALID_ARG);
  }
}

// ---------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------
template <typename T, bool NZ>
static cudaError_t quantize_values_t(const KSrc& src, int64_t T_q, const CacheView& cv, int layer, int n_layers,
                                     const SelView& sel, float gamma, cudaStream_t stream) {
  const int n_slabs = n_layers * cv.B * cv.H_kv;
  const int64_t n_rest = T_q - sel.n_prot;
  if (n_rest > 0) {
    const int64_t sgs = (n_rest + kSGTokens - 1) / kSGTokens;
    const size_t smem = kSGTokens * kVRowBytes + sizeof(float) * kSGGroups * 4 * kD + sizeof(uint32_t) * kSGGroups * 64 + 256 +
                        (NZ ? sizeof(float) * kSGGroups * 4 * kD : 0);
    static bool attr_set_dev[64] = {};   // function attributes are per device (and per instantiation)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    bool& attr_set = attr_set_dev[dev];
    if (!attr_set) {
      cudaError_t e;
      if ((e = cudaFuncSetAttribute(v_ternary_kernel<T, NZ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
      attr_set = true;
    }
    v_ternary_kernel<T, NZ><<<dim3(static_cast<unsigned>(sgs), n_slabs), 256, smem, stream>>>(src, n_rest, cv, layer, sel, gamma);
    count_launches(1);
  }
  if (sel.n_prot > 0) {
    const int64_t pgs = (sel.n_prot + kG - 1) / kG;
    v_protect_kernel<T><<<dim3(static_cast<unsigned>(pgs), n_slabs), 128, 0, stream>>>(src, cv, layer, sel);
    count_launches(1);
  }
  return cudaGetLastError();
}

cudaError_t launch_quantize_values(int dtype, const KSrc& src, int64_t T_q, const CacheView& cv, int layer, int n_layers,
                                   const SelView& sel, float gamma, bool nonzero_mean_scale, cudaStream_t stream) {
  if (dtype == VIDKV_F16)
    return nonzero_mean_scale ? quantize_values_t<__half, true>(src, T_q, cv, layer, n_layers, sel, gamma, stream)
                              : quantize_values_t<__half, false>(src, T_q, cv, layer, n_layers, sel, gamma, stream);
  return nonzero_mean_scale ? quantize_values_t<__nv_bfloat16, true>(src, T_q, cv, layer, n_layers, sel, gamma, stream)
                            : quantize_values_t<__nv_bfloat16, false>(src, T_q, cv, layer, n_layers, sel, gamma, stream);
}

template <typename T, bool NZ>
static void flush_values_t(const KSrc& src, const CacheView& cv, int layer0, int n_layers, int64_t tgroup0, float gamma,
                           cudaStream_t stream) {
  const int spl = cv.B * cv.H_kv;
  v_flush_kernel<T, NZ><<<spl * n_layers, kD, 0, stream>>>(src, cv, layer0, spl, tgroup0, gamma);
}

cudaError_t launch_flush_values(int dtype, const KSrc& src, const CacheView& cv, int layer0, int n_layers,
                                int64_t tgroup0, float gamma, bool nonzero_mean_scale, cudaStream_t stream) {
  if (dtype == VIDKV_F16) {
    if (nonzero_mean_scale) flush_values_t<__half, true>(src, cv, layer0, n_layers, tgroup0, gamma, stream);
    else flush_values_t<__half, false>(src, cv, layer0, n_layers, tgroup0, gamma, stream);
  } else {
    if (nonzero_mean_scale) flush_values_t<__nv_bfloat16, true>(src, cv, layer0, n_layers, tgroup0, gamma, stream);
    else flush_values_t<__nv_bfloat16, false>(src, cv, layer0, n_layers, tgroup0, gamma, stream);
  }
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_copy_to_residual(int dtype, const KSrc& src, int64_t t_begin, int n_tok, const CacheView& cv,
                                    int layer, int n_layers, bool is_value, int r0, cudaStream_t stream) {
  if (n_tok <= 0) return cudaSuccess;
  const int64_t off = is_value ? cv.vres_offset : cv.kres_offset;
  // 16-bit elements either way: the copy is type-agnostic
  (void)dtype;
  copy_to_residual_kernel<__half><<<n_layers * cv.B * cv.H_kv, 256, 0, stream>>>(src, t_begin, n_tok, cv, layer, off, r0);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_append(int dtype, const void* k_new, const void* v_new, const CacheView& cv, int layer0,
                          int n_layers, int row, cudaStream_t stream) {
  (void)dtype;
  const int spl = cv.B * cv.H_kv;
  append_kernel<<<spl * n_layers, 32, 0, stream>>>(static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                                   cv, layer0, spl, row);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_select_tokens(const float* saliency, int64_t vis_begin, int64_t l_v, int64_t n_prot, int64_t T_q,
                                 const CacheView& cv, int32_t* idx_prot, int32_t* idx_rest, int64_t stride_prot,
                                 int64_t stride_rest, cudaStream_t stream) {
  select_tokens_kernel<<<cv.B, 1024, 0, stream>>>(saliency, nullptr, 0, vis_begin, l_v, n_prot, T_q, cv, idx_prot,
                                                  idx_rest, stride_prot, stride_rest, nullptr, -1);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_mask_to_selection(const uint8_t* E, int64_t T, int64_t T_q, const CacheView& cv, int32_t* idx_prot,
                                     int32_t* idx_rest, int64_t stride_prot, int64_t stride_rest, int32_t* counts,
                                     int64_t expect_count, cudaStream_t stream) {
  select_tokens_kernel<<<cv.B, 1024, 0, stream>>>(nullptr, E, T, 0, 0, 0, T_q, cv, idx_prot, idx_rest, stride_prot,
                                                  stride_rest, counts, expect_count);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace vidkv
