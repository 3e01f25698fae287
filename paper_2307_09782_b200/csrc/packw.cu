// Fine-grained FP4-E2M1 weight quantizer and packer with the scale constraints none / M1 / M2.
// Section 3 (FGQ; "Casting the FP4 to FP8", items M1 and M2), Appendix A (group size).
//
// One CTA per output row.  Pass 1: each warp reduces the absmax of its groups and leaves the group
// scale in shared memory.  Then the row-wide quantity of the constrained modes (largest exponent for
// M1, largest scale for M2) is reduced.  Pass 2 re-reads the row (it is still in L2), divides,
// rounds to E2M1 and writes two codes per byte.  All scale decisions use the bits of the FP32 scale,
// never a logarithm.
#include <limits.h>

#include "zq_common.cuh"

namespace zq {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kShiftMax = 5;

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

// Round to nearest E2M1 magnitude, ties to the code with mantissa bit 0, saturating at 6; sign kept.
__device__ __forceinline__ uint32_t encode_e2m1(float v) {
  const float a = fabsf(v);
  const uint32_t m = (a > 0.25f) + (a >= 0.75f) + (a > 1.25f) + (a >= 1.75f) + (a > 2.5f) + (a >= 3.5f) + (a > 5.0f);
  return m | ((__float_as_uint(v) >> 31) << 3);
}

template <int EPL>  // elements per lane = group / 32
__global__ void __launch_bounds__(kThreads)
pack_weight_kernel(const float* __restrict__ W, int K, int G, int mode, uint8_t* __restrict__ codes,
                   uint8_t* __restrict__ shift, float* __restrict__ scale) {
  extern __shared__ float s_S[];  // [G] unconstrained group scales (0 = all-zero group)
  __shared__ int s_red_i[kWarps];
  __shared__ float s_red_f[kWarps];
  const int64_t n = blockIdx.x;
  const float* row = W + n * static_cast<int64_t>(K);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int group = EPL * 32;

  for (int j = warp; j < G; j += kWarps) {
    const float* p = row + static_cast<int64_t>(j) * group + lane * EPL;
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < EPL; i += 2) {
      const float2 v = __ldg(reinterpret_cast<const float2*>(p + i));
      a = fmaxf(a, fmaxf(fabsf(v.x), fabsf(v.y)));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, o));
    if (lane == 0) s_S[j] = (a == 0.0f) ? 0.0f : __fdiv_rn(a, 6.0f);
  }
  __syncthreads();

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

  for (int j = warp; j < G; j += kWarps) {
    const float s = s_S[j];
    float shat;
    if (mode == ZQ_SCALE_NONE) {
      shat = (s == 0.0f) ? 1.0f : s;
      if (lane == 0) scale[n * G + j] = shat;
    } else {
      int d = 0;
      if (s != 0.0f) {
        int e;
        uint32_t f;
        exp_frac(s, &e, &f);
        // M1: P - ceil(log2 s).   M2: ceil(log2(Smax / s)) from the two exponent / fraction fields.
        d = (mode == ZQ_SCALE_M1) ? P - (e + (f != 0 ? 1 : 0)) : (e_max - e) + (f_max > f ? 1 : 0);
      }
      d = min(d, kShiftMax);
      shat = (mode == ZQ_SCALE_M1) ? ldexpf(1.0f, P - d) : ldexpf(Smax, -d);
      if (lane == 0) shift[n * G + j] = static_cast<uint8_t>(d);
    }
    const float* p = row + static_cast<int64_t>(j) * group + lane * EPL;
    uint32_t packed = 0;
#pragma unroll
    for (int i = 0; i < EPL; i += 2) {
      const float2 v = __ldg(reinterpret_cast<const float2*>(p + i));
      packed |= encode_e2m1(__fdiv_rn(v.x, shat)) << (4 * i);
      packed |= encode_e2m1(__fdiv_rn(v.y, shat)) << (4 * i + 4);
    }
    uint8_t* out = codes + n * static_cast<int64_t>(K / 2) + static_cast<int64_t>(j) * (group / 2) + lane * (EPL / 2);
    if (EPL == 2) *out = static_cast<uint8_t>(packed);
    else if (EPL == 4) *reinterpret_cast<uint16_t*>(out) = static_cast<uint16_t>(packed);
    else *reinterpret_cast<uint32_t*>(out) = packed;
  }
}

}  // namespace

int launch_pack_weight(const float* W, int64_t N, int64_t K, int group, int mode, uint8_t* codes,
                       uint8_t* shift, float* scale, cudaStream_t st) {
  if (N == 0) return ZQ_OK;
  const int G = static_cast<int>(K / group);
  const size_t smem = static_cast<size_t>(G) * sizeof(float);
  dim3 grid(static_cast<unsigned>(N));
  switch (group) {
    case 64: pack_weight_kernel<2><<<grid, kThreads, smem, st>>>(W, int(K), G, mode, codes, shift, scale); break;
    case 128: pack_weight_kernel<4><<<grid, kThreads, smem, st>>>(W, int(K), G, mode, codes, shift, scale); break;
    case 256: pack_weight_kernel<8><<<grid, kThreads, smem, st>>>(W, int(K), G, mode, codes, shift, scale); break;
    default: return ZQ_ERR_SHAPE;
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // namespace zq
