// The arithmetic of the token-wise E4M3 activation quantizer (Section 3, Appendix A; Eq. 1 with Z = 0) on
// 16-byte pieces of a row, shared by the stand-alone quantizer kernels and by the GEMM kernel that
// quantizes its activations itself, so that both produce the same bits.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace zq {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Two FP32 values -> two E4M3 bytes (round to nearest even, saturate to +-448); `lo` lands in bits 0..7.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ float absmax8(uint4 v, float a) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a = fmaxf(a, fabsf(bf16_lo(w[i])));  // fmaxf drops a NaN operand
    a = fmaxf(a, fabsf(bf16_hi(w[i])));
  }
  return a;
}

__device__ __forceinline__ uint2 cast8(uint4 v, float inv) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t p[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    p[i] = cvt_e4m3x2(__fmul_rn(bf16_lo(w[i]), inv), __fmul_rn(bf16_hi(w[i]), inv));
  return make_uint2(p[0] | (p[1] << 16), p[2] | (p[3] << 16));
}

// acc + sum over 8 elements of x (bf16 pairs in xv) times V (fp16 pairs in vv)
__device__ __forceinline__ float dot8(uint4 xv, uint4 vv, float acc) {
  const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
  const uint32_t vw[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __half2 h;
    *reinterpret_cast<uint32_t*>(&h) = vw[i];
    const float2 vf = __half22float2(h);
    acc = fmaf(bf16_lo(xw[i]), vf.x, acc);
    acc = fmaf(bf16_hi(xw[i]), vf.y, acc);
  }
  return acc;
}

}  // namespace zq
