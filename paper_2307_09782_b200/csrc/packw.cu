// Fine-grained FP4-E2M1 weight quantizer and packer with the scale constraints none / M1 / M2.
// Section 3 (FGQ; "Casting the FP4 to FP8", items M1 and M2), Appendix A (group size).  Variants: FP8-E4M3
// codes (the W8A8 FP-FP rows of Table 2) for the block-scaled kernel, and a shift clamp of 13 for E5M2 as the
// cast target (footnote to "Casting the FP4 to FP8").
//
// One CTA per output row (rows of the last, partial tile beyond N are written as zeros).  A lane
// owns 8 consecutive elements, i.e. one 32-bit word of packed codes.  Pass 1 reduces the absmax of
// every group (segmented warp shuffle; shared-memory atomics for the group size 320, which does not divide
// a warp's 256 elements) and leaves the group scales in shared memory; then the
// row-wide quantity of the constrained modes (largest exponent for M1, largest scale for M2) is
// reduced; pass 2 re-reads the row (still in L2), divides, rounds to E2M1 and writes the codes in
// one of the two tiled layouts the GEMM kernels stream (MX = true: plain nibbles plus E8M0 block scales for
// the tensor core's own FP4 operand).  All scale decisions use the bits of the FP32 scale, never a
// logarithm.
#include <limits.h>

#include "zq_common.cuh"

namespace zq {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// floor(log2 s) and the 23-bit fraction field of a positive finite FP32 (subnormals normalised first)
__device__ __forceinline__ void exp_frac(float s, int* e, uint32_t* f) {
  int adj = 0;
  if (s < 1.17549435e-38f) {  // subnormal: scale by 2^24, exactly
    s *= 16777216.0f;
    adj = -24;
  }
  const uint32_t b = __float_as_uint(s);
  *e = static_cast<int>((b >> 23) & 0xFF) - 127 + adj;
  *f = b & 0x7FFFFFu;
}

// Two FP32 values -> two E4M3 bytes (round to nearest even, saturate to +-448); `lo` lands in bits 0..7.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

// Round to nearest E2M1 magnitude, ties to the code with mantissa bit 0, saturating at 6.
// Returns the 3 magnitude bits; the sign is taken from the quotient separately.
__device__ __forceinline__ uint32_t e2m1_magnitude(float v) {
  const float a = fabsf(v);
  return (a > 0.25f) + (a >= 0.75f) + (a > 1.25f) + (a >= 1.75f) + (a > 2.5f) + (a >= 3.5f) + (a > 5.0f);
}

// LAYOUT: 0 tiles for the kernel that casts (E2M1), 1 tiles for the block-scaled kernel (E2M1),
//         2 tiles for the block-scaled kernel with FP8-E4M3 codes.
template <int GROUP, int LAYOUT>
__global__ void __launch_bounds__(kThreads)
pack_weight_kernel(const float* __restrict__ W, int N, int K, int mode, int max_shift, uint8_t* __restrict__ tiles,
                   uint8_t* __restrict__ shift, float* __restrict__ scale) {
  constexpr bool MX = LAYOUT != 0;
  constexpr bool W8 = LAYOUT == 2;
  constexpr float kQmax = W8 ? 448.0f : 6.0f;     // largest magnitude of the code format
  constexpr int kCodeBytes = W8 ? 2 * kTileCodeBytes : kTileCodeBytes;
  extern __shared__ float s_S[];  // [G] unconstrained group scales (0 = all-zero group)
  __shared__ int s_red_i[kWarps];
  __shared__ float s_red_f[kWarps];
  constexpr int LPG = GROUP / 8;  // lanes per group
  const int n = blockIdx.x;
  const int G = K / GROUP;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kblocks = K / kTileK;
  constexpr int kTB = W8 ? kMx8TileBytes : (MX ? kMxTileBytes : kTileBytes);
  uint8_t* tile_row = tiles + static_cast<int64_t>(n / kTileRows) * kblocks * kTB;
  const int r = n % kTileRows;

  if (n >= N) {  // padding row of the last tile: zero codes and shifts
    for (int k = threadIdx.x * 8; k < K; k += kThreads * 8) {
      uint8_t* blk = tile_row + static_cast<int64_t>(k / kTileK) * kTB;
      const int within = k % kTileK;
      if (MX) {
        const int kb = k / kTileK;
        uint8_t* codes_kb = tile_row + static_cast<int64_t>(kb) * kCodeBytes;
        if (W8) *reinterpret_cast<uint2*>(codes_kb + r * 128 + within) = make_uint2(0u, 0u);
        else *reinterpret_cast<uint32_t*>(codes_kb + r * 64 + within / 2) = 0u;
        if (within % 32 == 0)
          tile_row[static_cast<int64_t>(kblocks) * kCodeBytes + kb * kMxTileScaleBytes + 16 * (r % 32) + 4 * (r / 32) +
                   within / 32] = 127;
      } else {
        *reinterpret_cast<uint32_t*>(blk + ((within / 32) * kTileRows + r) * 16 + ((within % 32) / 8) * 4) = 0u;
        if (within % 64 == 0) blk[kTileCodeBytes + 2 * r + within / 64] = 0;
      }
    }
    return;
  }
  const float* row = W + static_cast<int64_t>(n) * K;
  constexpr bool kShuffle = LPG <= 32 && (LPG & (LPG - 1)) == 0;  // groups that tile a warp's 256 elements
  if (!kShuffle) {
    for (int j = threadIdx.x; j < G; j += kThreads) s_S[j] = 0.0f;
    __syncthreads();
  }

  for (int kbase = warp * 256; kbase < K; kbase += kThreads * 8) {  // warp-uniform trip count
    const int k = kbase + lane * 8;
    const bool in = k < K;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 v0 = in ? __ldg(reinterpret_cast<const float4*>(row + k)) : zero4;
    const float4 v1 = in ? __ldg(reinterpret_cast<const float4*>(row + k + 4)) : zero4;
    float a = fmaxf(fmaxf(fmaxf(fabsf(v0.x), fabsf(v0.y)), fmaxf(fabsf(v0.z), fabsf(v0.w))),
                    fmaxf(fmaxf(fabsf(v1.x), fabsf(v1.y)), fmaxf(fabsf(v1.z), fabsf(v1.w))));
    if (kShuffle) {
#pragma unroll
      for (int o = 1; o < LPG; o <<= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, o));
      if (in && (lane % LPG) == 0) s_S[k / GROUP] = (a == 0.0f) ? 0.0f : __fdiv_rn(a, kQmax);
    } else if (in) {
      // non-negative floats order like their bit patterns
      atomicMax(reinterpret_cast<int*>(s_S) + k / GROUP, __float_as_int(a));
    }
  }
  __syncthreads();
  if (!kShuffle) {
    for (int j = threadIdx.x; j < G; j += kThreads) {
      const float a = s_S[j];
      s_S[j] = (a == 0.0f) ? 0.0f : __fdiv_rn(a, kQmax);
    }
    __syncthreads();
  }

  // row-wide reduction for the constrained modes
  int P = 0;          // M1: largest ceil(log2 S_j)
  float Smax = 1.0f;  // M2: largest S_j
  if (mode != ZQ_SCALE_NONE) {
    int p_loc = INT_MIN;
    float s_loc = 0.0f;
    for (int j = threadIdx.x; j < G; j += kThreads) {
      const float s = s_S[j];
      if (s != 0.0f) {
        int e;
        uint32_t f;
        exp_frac(s, &e, &f);
        p_loc = max(p_loc, e + (f != 0 ? 1 : 0));
        s_loc = fmaxf(s_loc, s);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      p_loc = max(p_loc, __shfl_xor_sync(0xFFFFFFFFu, p_loc, o));
      s_loc = fmaxf(s_loc, __shfl_xor_sync(0xFFFFFFFFu, s_loc, o));
    }
    if (lane == 0) {
      s_red_i[warp] = p_loc;
      s_red_f[warp] = s_loc;
    }
    __syncthreads();
    p_loc = s_red_i[0];
    s_loc = s_red_f[0];
    for (int w = 1; w < kWarps; ++w) {
      p_loc = max(p_loc, s_red_i[w]);
      s_loc = fmaxf(s_loc, s_red_f[w]);
    }
    P = (p_loc == INT_MIN) ? 0 : p_loc;
    Smax = (s_loc == 0.0f) ? 1.0f : s_loc;
    if (threadIdx.x == 0) scale[n] = (mode == ZQ_SCALE_M1) ? ldexpf(1.0f, P) : Smax;
  }

  int e_max = 0;
  uint32_t f_max = 0;
  if (mode == ZQ_SCALE_M2) exp_frac(Smax, &e_max, &f_max);

  for (int k = (warp * 32 + lane) * 8; k < K; k += kThreads * 8) {
    const int j = k / GROUP;
    const float s = s_S[j];
    float shat;
    int d = 0;
    if (mode == ZQ_SCALE_NONE) {
      shat = (s == 0.0f) ? 1.0f : s;
      if ((k % GROUP) == 0) scale[static_cast<int64_t>(n) * G + j] = shat;
    } else {
      if (s != 0.0f) {
        int e;
        uint32_t f;
        exp_frac(s, &e, &f);
        // M1: P - ceil(log2 s).   M2: ceil(log2(Smax / s)) from the two exponent / fraction fields.
        d = (mode == ZQ_SCALE_M1) ? P - (e + (f != 0 ? 1 : 0)) : (e_max - e) + (f_max > f ? 1 : 0);
      }
      d = min(d, max_shift);
      shat = (mode == ZQ_SCALE_M1) ? ldexpf(1.0f, P - d) : ldexpf(Smax, -d);
      if ((k % GROUP) == 0) shift[static_cast<int64_t>(n) * G + j] = static_cast<uint8_t>(d);
    }
    const float4 v0 = __ldg(reinterpret_cast<const float4*>(row + k));
    const float4 v1 = __ldg(reinterpret_cast<const float4*>(row + k + 4));
    const float q[8] = {__fdiv_rn(v0.x, shat), __fdiv_rn(v0.y, shat), __fdiv_rn(v0.z, shat), __fdiv_rn(v0.w, shat),
                        __fdiv_rn(v1.x, shat), __fdiv_rn(v1.y, shat), __fdiv_rn(v1.z, shat), __fdiv_rn(v1.w, shat)};
    uint32_t w = 0;
    if (!W8) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        w |= e2m1_magnitude(q[i]) << (4 * i);
        const uint32_t sgn = __float_as_uint(q[i]) >> 31;
        w |= sgn << (MX ? 4 * i + 3 : (i < 4 ? 8 * i + 7 : 8 * (i - 4) + 3));
      }
    }
    uint8_t* blk = tile_row + static_cast<int64_t>(k / kTileK) * kTB;
    const int within = k % kTileK;
    if (MX) {
      const int kb = k / kTileK;
      uint8_t* codes_kb = tile_row + static_cast<int64_t>(kb) * kCodeBytes;
      if (W8) {
        // E4M3 codes, round to nearest even, saturating at +-448: the conversion the activation quantizer uses
        const uint32_t c0 = cvt_e4m3x2(q[0], q[1]) | (cvt_e4m3x2(q[2], q[3]) << 16);
        const uint32_t c1 = cvt_e4m3x2(q[4], q[5]) | (cvt_e4m3x2(q[6], q[7]) << 16);
        *reinterpret_cast<uint2*>(codes_kb + r * 128 + within) = make_uint2(c0, c1);
      } else {
        *reinterpret_cast<uint32_t*>(codes_kb + r * 64 + within / 2) = w;
      }
      if (within % 32 == 0)
        tile_row[static_cast<int64_t>(kblocks) * kCodeBytes + kb * kMxTileScaleBytes + 16 * (r % 32) + 4 * (r / 32) +
                 within / 32] = static_cast<uint8_t>(127 - d);
    } else {
      *reinterpret_cast<uint32_t*>(blk + ((within / 32) * kTileRows + r) * 16 + ((within % 32) / 8) * 4) = w;
      if (within % 64 == 0) blk[kTileCodeBytes + 2 * r + within / 64] = static_cast<uint8_t>(d);
    }
  }
}

}  // namespace

int launch_pack_weight(const float* W, int64_t N, int64_t K, int group, int mode, int layout, uint8_t* codes,
                       uint8_t* shift, float* scale, cudaStream_t st) {
  if (N == 0) return ZQ_OK;
  const int G = static_cast<int>(K / group);
  const size_t smem = static_cast<size_t>(G) * sizeof(float);
  const int rows = static_cast<int>((N + kTileRows - 1) / kTileRows) * kTileRows;
  dim3 grid(static_cast<unsigned>(rows));
  // stored shifts: up to 5 while E4M3 is the cast target (Section 3), 13 for E5M2, and as far as an E8M0
  // block scale reaches for FP8 codes
  const int max_shift = layout == ZQ_WEIGHTS_CAST_E5M2 ? 13 : (layout == ZQ_WEIGHTS_MX_FP8 ? 127 : 5);
  const int lay = layout == ZQ_WEIGHTS_MX ? 1 : (layout == ZQ_WEIGHTS_MX_FP8 ? 2 : 0);
#define ZQ_PACK(GROUP)                                                                                                     \
  if (lay == 1)                                                                                                            \
    pack_weight_kernel<GROUP, 1><<<grid, kThreads, smem, st>>>(W, int(N), int(K), mode, max_shift, codes, shift, scale);   \
  else if (lay == 2)                                                                                                       \
    pack_weight_kernel<GROUP, 2><<<grid, kThreads, smem, st>>>(W, int(N), int(K), mode, max_shift, codes, shift, scale);   \
  else                                                                                                                     \
    pack_weight_kernel<GROUP, 0><<<grid, kThreads, smem, st>>>(W, int(N), int(K), mode, max_shift, codes, shift, scale)
  switch (group) {
    case 64: ZQ_PACK(64); break;
    case 128: ZQ_PACK(128); break;
    case 256: ZQ_PACK(256); break;
    case 320: ZQ_PACK(320); break;
    default: return ZQ_ERR_SHAPE;
  }
#undef ZQ_PACK
  count_launch();
  return cudaGetLastError() == cudaSuccess ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // namespace zq
