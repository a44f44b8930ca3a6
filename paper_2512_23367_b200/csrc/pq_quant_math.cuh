// Arithmetic of the symmetric INT8 quantizer (Eq. 1-2 of the paper), shared by the quantizer kernels and by the
// kernels that quantize their own activations: every one of them must produce the same codes.
#pragma once
#include <cuda_fp16.h>

#include <cstdint>

namespace pq {

// Largest magnitude of the eight FP16 values of a 16-byte chunk (exact: taken in FP16).
__device__ __forceinline__ float absmax8(const uint4& v) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
  __half2 m = __hmax2(__hmax2(__habs2(h[0]), __habs2(h[1])), __hmax2(__habs2(h[2]), __habs2(h[3])));
  return fmaxf(__low2float(m), __high2float(m));
}

// Eq. 1 for four values at a time.
// Four scaled values -> four INT8 codes in one word (code i in byte i): round to nearest even, then two
// packing conversions that saturate to [-128, 127].
template <bool kDivide>
__device__ __forceinline__ uint32_t codes4(float x0, float x1, float x2, float x3, float f) {
  const int a0 = __float2int_rn(kDivide ? __fdiv_rn(x0, f) : __fmul_rn(x0, f));
  const int a1 = __float2int_rn(kDivide ? __fdiv_rn(x1, f) : __fmul_rn(x1, f));
  const int a2 = __float2int_rn(kDivide ? __fdiv_rn(x2, f) : __fmul_rn(x2, f));
  const int a3 = __float2int_rn(kDivide ? __fdiv_rn(x3, f) : __fmul_rn(x3, f));
  uint32_t hi, out;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(a3), "r"(a2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(a1), "r"(a0), "r"(hi));
  return out;
}

// Scale and multiplier of a row with largest magnitude a:  s = a / 127.5,  code = rne(x * (127.5 / a)).
__device__ __forceinline__ void act_scale(float a, float* s, float* f) {
  *s = __fdiv_rn(a, 127.5f);
  *f = (a == 0.0f) ? 0.0f : __fdiv_rn(127.5f, a);
}

}  // namespace pq
