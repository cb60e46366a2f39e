// Shared device/host helpers for the libxconv kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace xconv {

typedef __nv_bfloat16 bf16;
typedef __half f16;

// Workspace header (two 32-bit words).  Every API call draws a fresh non-zero tag; word 1 holds the
// tag of the last call that ran a pipelined kernel, word 0 the tag of a call in which a bounded wait
// ran out.  The last call timed out iff the two are equal and non-zero -- so the header never has to
// be cleared, whatever the scratch memory held before.
enum : unsigned int { WS_OK = 0u };

// Programmatic dependent launch: a kernel launched with launch_pdl may start while the kernel before
// it in the stream is still draining; it must call pdl_wait() before it reads or overwrites anything
// that kernel touches.  pdl_trigger() lets the kernel after this one start its own preamble early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f(f16 v) { return __half2float(v); }

template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ f16 from_f<f16>(float v) { return __float2half_rn(v); }

// Four consecutive elements as floats; the pointer must be aligned to 4 elements.
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 ld4(const bf16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  float4 f;
  f.x = __uint_as_float(u.x << 16);
  f.y = __uint_as_float(u.x & 0xffff0000u);
  f.z = __uint_as_float(u.y << 16);
  f.w = __uint_as_float(u.y & 0xffff0000u);
  return f;
}
__device__ __forceinline__ float4 ld4(const f16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
  const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4(f16* p, float4 v) {
  __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ void st4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// Elements idx..idx+3 of p, zero beyond `limit`; vector access when `vec` says rows are 4-aligned.
template <typename T>
__device__ __forceinline__ float4 ld4_guard(const T* p, long idx, long limit, bool vec) {
  if (vec && idx + 3 < limit) return ld4(p + idx);
  float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
  if (idx + 0 < limit) f.x = to_f(p[idx + 0]);
  if (idx + 1 < limit) f.y = to_f(p[idx + 1]);
  if (idx + 2 < limit) f.z = to_f(p[idx + 2]);
  if (idx + 3 < limit) f.w = to_f(p[idx + 3]);
  return f;
}
template <typename T>
__device__ __forceinline__ void st4_guard(T* p, long idx, long limit, bool vec, float4 v) {
  if (vec && idx + 3 < limit) { st4(p + idx, v); return; }
  if (idx + 0 < limit) p[idx + 0] = from_f<T>(v.x);
  if (idx + 1 < limit) p[idx + 1] = from_f<T>(v.y);
  if (idx + 2 < limit) p[idx + 2] = from_f<T>(v.z);
  if (idx + 3 < limit) p[idx + 3] = from_f<T>(v.w);
}

// Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11): counter (c0, c1, c2, 0), key = the seed.
// One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2, c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0), then
// the key moves on by the Weyl constants.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1, uint32_t c2 = 0u) {
  uint32_t c3 = 0u;
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Standard normal probing vectors from Philox words (xconv_gaussian_probes_from_seed).  Every step below is one
// correctly rounded IEEE float operation (the _rn intrinsics are never contracted into fused multiply-adds), in a
// fixed order, so that a host program following the same steps in float gets the same bits.

// ln(t * 2^-24) for an odd t below 2^24: t = 2^k f, f in [1, 2), halved when above sqrt(2); ln f = 2 artanh(s),
// s = (f - 1) / (f + 1), by the odd series up to s^11.
__device__ __forceinline__ float ln_u24(uint32_t t) {
  const int k = 31 - __clz((int)t);
  float f = __uint_as_float(((t << (23 - k)) & 0x007FFFFFu) | 0x3F800000u);
  const int big = f > 1.41421354f ? 1 : 0;
  if (big) f = __fmul_rn(f, 0.5f);
  const float e = (float)(k - 24 + big);
  const float s = __fdiv_rn(__fsub_rn(f, 1.0f), __fadd_rn(f, 1.0f));
  const float s2 = __fmul_rn(s, s);
  float p = (float)(1.0 / 11.0);
  p = __fadd_rn(__fmul_rn(p, s2), (float)(1.0 / 9.0));
  p = __fadd_rn(__fmul_rn(p, s2), (float)(1.0 / 7.0));
  p = __fadd_rn(__fmul_rn(p, s2), (float)(1.0 / 5.0));
  p = __fadd_rn(__fmul_rn(p, s2), (float)(1.0 / 3.0));
  p = __fadd_rn(__fmul_rn(p, s2), 1.0f);
  const float lnf = __fmul_rn(__fmul_rn(2.0f, s), p);
  return __fadd_rn(__fmul_rn(e, (float)0.693147182), lnf);
}

// (cos, sin) of 2 pi t / 2^24 for an odd t below 2^24: the top three bits are the octant, the rest an angle in
// (0, pi/4) measured from the nearer end of the octant, where the Taylor polynomials up to x^9 and x^10 serve.
__device__ __forceinline__ float2 sincos_u24(uint32_t t) {
  const uint32_t octant = t >> 21;
  uint32_t frac = t & 0x1FFFFFu;
  if (octant & 1u) frac = 0x200000u - frac;
  const float x = __fmul_rn((float)frac, (float)3.74507039e-07);      // 2 pi / 2^24
  const float x2 = __fmul_rn(x, x);
  float ps = (float)(1.0 / 362880.0);
  ps = __fadd_rn(__fmul_rn(ps, x2), (float)(-1.0 / 5040.0));
  ps = __fadd_rn(__fmul_rn(ps, x2), (float)(1.0 / 120.0));
  ps = __fadd_rn(__fmul_rn(ps, x2), (float)(-1.0 / 6.0));
  ps = __fadd_rn(__fmul_rn(ps, x2), 1.0f);
  const float sn = __fmul_rn(ps, x);
  float pc = (float)(-1.0 / 3628800.0);
  pc = __fadd_rn(__fmul_rn(pc, x2), (float)(1.0 / 40320.0));
  pc = __fadd_rn(__fmul_rn(pc, x2), (float)(-1.0 / 720.0));
  pc = __fadd_rn(__fmul_rn(pc, x2), (float)(1.0 / 24.0));
  pc = __fadd_rn(__fmul_rn(pc, x2), -0.5f);
  pc = __fadd_rn(__fmul_rn(pc, x2), 1.0f);
  const bool swap = ((octant + 1u) >> 1) & 1u;           // octants 1, 2, 5, 6: sine and cosine trade places
  float c = swap ? sn : pc, s = swap ? pc : sn;
  if (((octant + 2u) >> 2) & 1u) c = -c;                 // cos < 0 in octants 2..5
  if (octant >> 2) s = -s;                               // sin < 0 in octants 4..7
  return make_float2(c, s);
}

// The two normals of one pair of Philox words: uniforms (2 (w >> 9) + 1) / 2^24, Box-Muller.
__device__ __forceinline__ float2 box_muller_u24(uint32_t wa, uint32_t wb) {
  const float rad = __fsqrt_rn(__fmul_rn(-2.0f, ln_u24(((wa >> 9) << 1) | 1u)));
  const float2 cs = sincos_u24(((wb >> 9) << 1) | 1u);
  return make_float2(__fmul_rn(rad, cs.x), __fmul_rn(rad, cs.y));
}

}  // namespace xconv
