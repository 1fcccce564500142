// Device helpers shared by the decode attention kernels (decode_prep.cu, decode_stream.cu, decode.cu):
// mma.sync wrappers, the logic / multiply-add forms of the code expansion, and the query
// normalisation.
#pragma once

#include "common.cuh"
#include "kernels.cuh"

namespace vidkv {
namespace {

constexpr int kThreads = 128;

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// d = a b + c with c given separately (no copy into the accumulator beforehand)
__device__ __forceinline__ void mma_f16_c(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1, float c0, float c1, float c2, float c3) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c0), "f"(c1), "f"(c2), "f"(c3));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// q . k with the operands in the cache's element type (rows 8-15 of A unused)
template <typename T> __device__ __forceinline__ void mma_in(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1);
template <> __device__ __forceinline__ void mma_in<__half>(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  mma_f16(d, a0, 0u, a2, 0u, b0, b1);
}
template <> __device__ __forceinline__ void mma_in<__nv_bfloat16>(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0,
                                                                  uint32_t b1) {
  mma_bf16(d, a0, 0u, a2, 0u, b0, b1);
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
// Copy n16 16-byte pieces from global to shared memory, pieces interleaved over the CTA's threads;
// unrolled by four so that the offsets are immediates.
__device__ __forceinline__ void stage_async(uint8_t* dst, const uint8_t* src, int n16, int tid) {
  constexpr int kStep = 128 * 16;
  uint8_t* d = dst + tid * 16;
  const uint8_t* s = src + tid * 16;
  int i = tid;
  for (; i + 3 * 128 < n16; i += 4 * 128, d += 4 * kStep, s += 4 * kStep) {
    cp_async16(d, s);
    cp_async16(d + kStep, s + kStep);
    cp_async16(d + 2 * kStep, s + 2 * kStep);
    cp_async16(d + 3 * kStep, s + 3 * kStep);
  }
  for (; i < n16; i += 128, d += kStep, s += kStep) cp_async16(d, s);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint32_t hmul2_u(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// a * b + c on two binary16 lanes (one rounding)
__device__ __forceinline__ uint32_t hfma2_u(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// a * b - c on two binary16 lanes (one rounding)
__device__ __forceinline__ uint32_t hfms2_u(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  const __half2 x = __hfma2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b),
                            __hneg2(*reinterpret_cast<const __half2*>(&c)));
  d = *reinterpret_cast<const uint32_t*>(&x);
  return d;
}
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// (x & m) | c and (x & m) ^ c as one three-input logic instruction
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t m, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "r"(m), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t and_xor(uint32_t x, uint32_t m, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(x), "r"(m), "r"(c));
  return d;
}
// (~x & m) ^ c: with m the sign bits, c comes out negated where x has a 0 bit
__device__ __forceinline__ uint32_t nand_xor(uint32_t x, uint32_t m, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xA6;" : "=r"(d) : "r"(x), "r"(m), "r"(c));
  return d;
}
// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start
// while the kernel before it still runs; pdl_wait() returns once that kernel has completed and its
// writes are visible (a no-op for an ordinary launch), pdl_release() lets the kernel after this one start.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Launch `kernel` so that it may overlap the tail of the previous kernel on `stream` (it must call pdl_wait()
// before touching anything that kernel writes).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// Bit patterns of the code expansion.  They live in constant memory rather than in the
// instruction stream so that mask and pattern both reach the logic instruction as register
// operands (an instruction encodes one immediate at most).
static __constant__ uint32_t kExpand[4] = {0x03000300u,   // two-bit field at mantissa bits 8-9 of each binary16 lane
                                    0x44004400u,   // 4.0 in each lane
                                    0x80008000u,   // the sign bits
                                    0xbc00bc00u};  // -1.0 in each lane

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// 2^k as a float, |k| <= 126
__device__ __forceinline__ float pow2i(int k) { return __uint_as_float(static_cast<uint32_t>(127 + k) << 23); }

// Query normalisation.  The score operands q_j s_j and Q_f s_f are binary16 numbers, so a large
// query entry times a large key scale would overflow although the score itself is an ordinary
// float.  Every query head is therefore multiplied by the power of two 2^(-e - kQShift), e =
// floor(log2(max_c |q_c|)), which puts its largest entry into [1/8, 1/4): no product of a scaled
// entry (or of a spectrum coefficient, at most 16 times the largest entry) with a binary16 scale
// below 16376 leaves the binary16 range.  Scores are linear in q, so the softmax multiplies by the
// inverse power of two; both factors are exact.  head_exponent returns e (0 for a head that is all
// zero or holds no finite maximum); the NSUB lanes sub = 0..NSUB-1 share the 128 entries of the row,
// and all 32 lanes of the warp must call it.
constexpr int kQShift = 3;
template <typename T, int NSUB>
__device__ __forceinline__ int head_exponent(const T* qrow, int sub, bool live) {
  float m = 0.0f;
  if (live) {
    const uint2* p = reinterpret_cast<const uint2*>(qrow + sub * (kD / NSUB));
#pragma unroll
    for (int i = 0; i < kD / NSUB / 4; ++i) {
      const uint2 v = __ldg(p + i);
      const float2 a = Elem<T>::to_float2(v.x), b = Elem<T>::to_float2(v.y);
      m = fmaxf(m, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(b.x), fabsf(b.y))));
    }
  }
#pragma unroll
  for (int o = NSUB / 2; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (!(m > 0.0f) || m > 3.0e38f) return 0;
  const int e = static_cast<int>(__float_as_uint(m) >> 23) - 127;
  return max(-100, min(100, e));
}


}  // namespace
}  // namespace vidkv
