// Token-wise FP8-E4M3 activation quantizer with the optional LoRC down-projection t = V x.
// Section 3 (token-wise activation quantization; LoRC), Appendix A, Eq. 1 with Z = 0.
//
// One CTA per token.  The row is read once from HBM with 16-byte loads and kept in registers
// between the absmax reduction and the cast (rows longer than the register budget are re-read).
// A thread's unit is 16 consecutive elements: two 16-byte loads in, one 16-byte store out.
#include <cooperative_groups.h>
#include <cuda_fp16.h>

#include <mutex>

#include "act_cast.cuh"
#include "zq_common.cuh"

namespace zq {
namespace {

constexpr int kUnit = 16;   // elements per thread-unit
constexpr int kVpt = 8;     // units a thread keeps in registers
constexpr int kMaxThreads = 256;
constexpr int kRChunk = 8;  // LoRC rows of V handled per pass over the registers

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// amax_in != nullptr: the caller knows the tokens' absolute maxima (the epilogue of the layer before collected
// them): no reduction; the row is still kept in registers for the LoRC product.
template <bool CACHED>
__global__ void __launch_bounds__(kMaxThreads)
act_quant_kernel(const uint4* __restrict__ x, int K, int64_t ldx_vec, uint8_t* __restrict__ q,
                 float* __restrict__ sx, const uint4* __restrict__ V, int r, float* __restrict__ t,
                 const float* __restrict__ amax_in) {
  pdl_launch_dependents();
  pdl_wait();  // x may be the output of the kernel before this one
  const int64_t m = blockIdx.x;
  const int nunits = K / kUnit;
  const uint4* row = x + m * ldx_vec;  // 8 bf16 per uint4
  uint4* qrow = reinterpret_cast<uint4*>(q + m * static_cast<int64_t>(K));
  const int T = blockDim.x, tid = threadIdx.x;
  __shared__ float red[kMaxThreads / 32];
  __shared__ float red_t[kMaxThreads / 32][kRChunk];

  uint4 c0[kVpt], c1[kVpt];
  float a = 0.0f;
  if (CACHED) {
#pragma unroll
    for (int i = 0; i < kVpt; ++i) {
      const int u = tid + i * T;
      if (u < nunits) {
        c0[i] = __ldg(row + 2 * u);
        c1[i] = __ldg(row + 2 * u + 1);
      } else {
        c0[i] = make_uint4(0, 0, 0, 0);
        c1[i] = make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int i = 0; i < kVpt; ++i) a = absmax8(c1[i], absmax8(c0[i], a));
  } else {
    for (int u = tid; u < nunits; u += T) a = absmax8(__ldg(row + 2 * u + 1), absmax8(__ldg(row + 2 * u), a));
  }
  a = warp_max(a);
  if ((tid & 31) == 0) red[tid >> 5] = a;
  __syncthreads();
  a = red[0];
  for (int w = 1; w < (T >> 5); ++w) a = fmaxf(a, red[w]);
  if (amax_in != nullptr) a = __ldg(amax_in + m);

  float s = 1.0f, inv = 1.0f;
  if (a != 0.0f) {
    s = __fdiv_rn(a, 448.0f);
    inv = __fdiv_rn(448.0f, a);
  }
  if (tid == 0) sx[m] = s;

  if (CACHED) {
#pragma unroll
    for (int i = 0; i < kVpt; ++i) {
      const int u = tid + i * T;
      if (u < nunits) {
        const uint2 lo = cast8(c0[i], inv), hi = cast8(c1[i], inv);
        qrow[u] = make_uint4(lo.x, lo.y, hi.x, hi.y);
      }
    }
  } else {
    for (int u = tid; u < nunits; u += T) {
      const uint2 lo = cast8(__ldg(row + 2 * u), inv), hi = cast8(__ldg(row + 2 * u + 1), inv);
      qrow[u] = make_uint4(lo.x, lo.y, hi.x, hi.y);
    }
  }

  // LoRC down-projection with the raw row (Section 3): t[m, j] = sum_k V[j, k] x[m, k]
  if (V != nullptr) {
    const int kvec = K / 8;  // uint4 per row of V
    for (int j0 = 0; j0 < r; j0 += kRChunk) {
      float acc[kRChunk];
#pragma unroll
      for (int j = 0; j < kRChunk; ++j) acc[j] = 0.0f;
      if (CACHED) {
#pragma unroll
        for (int i = 0; i < kVpt; ++i) {
          const int u = tid + i * T;
          if (u < nunits) {
#pragma unroll
            for (int j = 0; j < kRChunk; ++j)
              if (j0 + j < r) {
                const uint4* vr = V + static_cast<int64_t>(j0 + j) * kvec;
                acc[j] = dot8(c1[i], __ldg(vr + 2 * u + 1), dot8(c0[i], __ldg(vr + 2 * u), acc[j]));
              }
          }
        }
      } else {
        for (int u = tid; u < nunits; u += T) {
          const uint4 a0 = __ldg(row + 2 * u), a1 = __ldg(row + 2 * u + 1);
#pragma unroll
          for (int j = 0; j < kRChunk; ++j)
            if (j0 + j < r) {
              const uint4* vr = V + static_cast<int64_t>(j0 + j) * kvec;
              acc[j] = dot8(a1, __ldg(vr + 2 * u + 1), dot8(a0, __ldg(vr + 2 * u), acc[j]));
            }
        }
      }
#pragma unroll
      for (int j = 0; j < kRChunk; ++j) {
        const float v = warp_sum(acc[j]);
        if ((tid & 31) == 0) red_t[tid >> 5][j] = v;
      }
      __syncthreads();
      if (tid < kRChunk && j0 + tid < r) {
        float v = 0.0f;
        for (int w = 0; w < (T >> 5); ++w) v += red_t[w][tid];
        t[m * r + j0 + tid] = v;
      }
      __syncthreads();
    }
  }
}

// ---- many tokens: eight rows per CTA -------------------------------------------------------------
// With one row per CTA every row re-reads all of V (r x K fp16) from L2, eight times the bytes of the
// row itself at rank 8, and spends eight FMAs per element on t = V x.  Here a CTA takes eight rows and
// the LoRC product goes to the tensor cores: bf16 and fp16 values are exact TF32 numbers, so
// mma.m16n8k8 (TF32 in, FP32 accumulate) computes exact products.  The MMA's A operand is V (its eight
// rows in the upper half of the 16, the lower half zero), its B operand eight token rows; a lane loads
// 16 bytes of "its" token row and 16 bytes of "its" V row at the same K offset and feeds them to four
// MMAs, so no value is moved between lanes.  Pass 1 streams the rows once from HBM for absmax and t;
// pass 2 reads them again (they are still in L2: 148 CTAs x 8 rows) for the cast.
constexpr int kRows = 8;
constexpr int kRowsThreads = 1024;
constexpr int kRowsWarps = kRowsThreads / 32;
constexpr int kRowsUnroll = 4;  // 32-element K slices a warp has in flight
constexpr int kRowsMinTokens = 384;

__device__ __forceinline__ void mma_tf32_16x8x8(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (registers a1, a3) are zero
  asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// SCALED: the tokens' absolute maxima are given (amax_in), so the codes are written in the one pass that also
// forms t, and nothing is read twice.
template <bool HAS_V, bool SCALED>
__global__ void __launch_bounds__(kRowsThreads, 1)
act_quant_rows_kernel(const uint4* __restrict__ x, int M, int K, int64_t ldx_vec, uint8_t* __restrict__ q,
                      float* __restrict__ sx, const uint4* __restrict__ V, float* __restrict__ t,
                      const float* __restrict__ amax_in) {
  __shared__ float s_amax[kRowsWarps][kRows];
  __shared__ float s_acc[kRowsWarps][kRows * 8];
  __shared__ float s_inv[kRows];
  pdl_launch_dependents();
  pdl_wait();  // x (and amax_in) may be the output of the kernel before this one
  const int m0 = blockIdx.x * kRows;
  const int nrows = min(kRows, M - m0);
  const int nvec = K / 8;  // 16-byte vectors per row
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;  // g: token row of this lane, and its row of V
  const uint4* xr = x + static_cast<int64_t>(m0) * ldx_vec;
  const uint4* xrow = xr + static_cast<int64_t>(g) * ldx_vec;
  const uint4* vrow = V + static_cast<int64_t>(g) * nvec;
  const bool row_ok = g < nrows;
  float inv_g = 1.0f;
  if (SCALED) {
    if (tid < kRows) {
      const float a = tid < nrows ? __ldg(amax_in + m0 + tid) : 0.0f;
      float s = 1.0f, inv = 1.0f;
      if (a != 0.0f) {
        s = __fdiv_rn(a, 448.0f);
        inv = __fdiv_rn(448.0f, a);
      }
      s_inv[tid] = inv;
      if (tid < nrows) sx[m0 + tid] = s;
    }
    __syncthreads();
    inv_g = s_inv[g];
  }
  uint2* qrow8 = reinterpret_cast<uint2*>(q + static_cast<int64_t>(m0 + (row_ok ? g : 0)) * K);

  float amax = 0.0f;
  float d[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // d[0], d[1]: t[token 2 tig, 2 tig + 1][j = g], partial over this warp's K
  // a warp takes 32-element slices of K: slice index = (it * warps + warp) * unroll + i
  for (int base = warp * kRowsUnroll * 4; base < nvec; base += kRowsWarps * kRowsUnroll * 4) {
    uint4 xv[kRowsUnroll], vv[kRowsUnroll];
#pragma unroll
    for (int i = 0; i < kRowsUnroll; ++i) {
      const int u = base + i * 4 + tig;
      const bool in = u < nvec;
      xv[i] = (in && row_ok) ? __ldg(xrow + u) : make_uint4(0, 0, 0, 0);
      if (HAS_V) vv[i] = in ? __ldg(vrow + u) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < kRowsUnroll; ++i) {
      if (SCALED) {
        const int u = base + i * 4 + tig;
        if (u < nvec && row_ok) qrow8[u] = cast8(xv[i], inv_g);
      } else {
        amax = absmax8(xv[i], amax);
      }
      if (HAS_V) {
        const uint32_t xw[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
        const uint32_t vw[4] = {vv[i].x, vv[i].y, vv[i].z, vv[i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __half2 h;
          *reinterpret_cast<uint32_t*>(&h) = vw[e];
          const float2 vf = __half22float2(h);
          // elements 2e and 2e+1 of both 8-element pieces stand at MMA-K positions tig and tig + 4
          mma_tf32_16x8x8(d, __float_as_uint(vf.x), __float_as_uint(vf.y), xw[e] << 16, xw[e] & 0xFFFF0000u);
        }
      }
    }
  }
  // the four lanes of a token row
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  if (tig == 0) s_amax[warp][g] = amax;
  if (HAS_V) {
    s_acc[warp][(2 * tig) * 8 + g] = d[0];      // [token][j]
    s_acc[warp][(2 * tig + 1) * 8 + g] = d[1];
  }
  __syncthreads();
  if (!SCALED && tid < kRows) {
    float a = s_amax[0][tid];
    for (int w = 1; w < kRowsWarps; ++w) a = fmaxf(a, s_amax[w][tid]);
    float s = 1.0f, inv = 1.0f;
    if (a != 0.0f) {
      s = __fdiv_rn(a, 448.0f);
      inv = __fdiv_rn(448.0f, a);
    }
    s_inv[tid] = inv;
    if (tid < nrows) sx[m0 + tid] = s;
  }
  if (HAS_V && tid >= 64 && tid < 64 + kRows * 8 && ((tid - 64) >> 3) < nrows) {
    float v = 0.0f;
    for (int w = 0; w < kRowsWarps; ++w) v += s_acc[w][tid - 64];
    t[static_cast<int64_t>(m0) * 8 + (tid - 64)] = v;
  }
  if (SCALED) return;  // the codes were written in the pass above
  __syncthreads();
  const int nunits = K / kUnit;
  for (int idx = tid; idx < nrows * nunits; idx += kRowsThreads) {
    const int r = idx / nunits, u = idx - r * nunits;
    const float inv = s_inv[r];
    const uint4* row = xr + r * ldx_vec;
    const uint2 lo = cast8(__ldg(row + 2 * u), inv), hi = cast8(__ldg(row + 2 * u + 1), inv);
    reinterpret_cast<uint4*>(q + static_cast<int64_t>(m0 + r) * K)[u] = make_uint4(lo.x, lo.y, hi.x, hi.y);
  }
}

// ---- a few hundred tokens: eight rows per cluster, the rows held in shared memory --------------------
// Between the two kernels around it: too few tokens for the eight-row CTAs above to fill the device, too many
// for a cluster per row below, whose every cluster reads all of V.  Here a cluster of C CTAs takes eight rows
// and each CTA a slice of at most 4096 columns of them, which one thread fetches into shared memory with
// eight bulk copies: the rows are read from HBM exactly once, V once per eight rows, absmax and the LoRC sums
// meet through distributed shared memory, and the cast reads shared memory.
// The wait for the copies is bounded like every wait of this library; the quantizer has no status word, so a
// wait that ran out shows as sx = +inf (and no codes written) for the rows concerned.
constexpr int kTileThreads = 384;
constexpr int kTileWarps = kTileThreads / 32;
constexpr int kTileMaxVec = 512;  // 16-byte vectors (8 elements) of a row one CTA holds
constexpr int kTilePadVec = 4;    // row pitch = slice + 64 bytes: the two rows of a quarter-warp hit disjoint banks
constexpr int kTileMaxCluster = 8;
constexpr int kTileMinTokens = 32;

template <bool HAS_V, int C>
__global__ void __cluster_dims__(C, 1, 1) __launch_bounds__(kTileThreads, 3)
act_quant_tile_kernel(const uint4* __restrict__ x, int M, int K, int64_t ldx_vec, int vec_per_cta,
                      uint8_t* __restrict__ q, float* __restrict__ sx, const uint4* __restrict__ V,
                      float* __restrict__ t) {
  namespace cg = cooperative_groups;
  extern __shared__ uint4 s_x[];  // [kRows][vec_per_cta + kTilePadVec]
  __shared__ float s_amax[kTileWarps][kRows];
  __shared__ float s_acc[kTileWarps][kRows * 8];
  __shared__ float s_part_amax[kRows];   // this CTA's partial absmax per row (read by the whole cluster)
  __shared__ float s_part_t[kRows * 8];  // this CTA's partial LoRC sums [token][j] (read by rank 0)
  __shared__ float s_inv[kRows];
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_abort;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = C == 1 ? 0 : static_cast<int>(cluster.block_rank());
  const int m0 = blockIdx.y * kRows;
  const int nrows = min(kRows, M - m0);
  const int nvec = K / 8;
  const int v_begin = rank * vec_per_cta;
  const int nv = max(0, min(nvec, v_begin + vec_per_cta) - v_begin);  // vectors of this CTA's slice
  const int pitch = vec_per_cta + kTilePadVec;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;  // g: token row of this lane, and its row of V
  const uint4* xr = x + static_cast<int64_t>(m0) * ldx_vec + v_begin;
  if (tid == 0) {
    mbar_init(&s_bar, 1);
    s_abort = 0;
    fence_mbar_init();
  }
  pdl_launch_dependents();
  __syncthreads();
  if (tid == 0 && nv > 0) {
    pdl_wait();  // x may be the output of the kernel before this one
    mbar_arrive_expect_tx(&s_bar, static_cast<uint32_t>(nrows) * nv * 16u);
    for (int r = 0; r < nrows; ++r)
      bulk_load(s_x + r * pitch, xr + static_cast<int64_t>(r) * ldx_vec, nv * 16u, &s_bar);
  }
  const uint4* vrow = V + static_cast<int64_t>(g) * nvec + v_begin;
  const uint4* srow = s_x + g * pitch;
  const bool row_ok = g < nrows;

  float amax = 0.0f;
  float d[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // d[0], d[1]: t[token 2 tig, 2 tig + 1][j = g] over this warp's columns
  bool arrived = false;
  for (int base = warp * kRowsUnroll * 4; base < nv; base += kTileWarps * kRowsUnroll * 4) {
    uint4 vv[kRowsUnroll];
    if (HAS_V) {  // V does not depend on the copies: its loads go out before the wait
#pragma unroll
      for (int i = 0; i < kRowsUnroll; ++i) {
        const int u = base + i * 4 + tig;
        vv[i] = u < nv ? __ldg(vrow + u) : make_uint4(0, 0, 0, 0);
      }
    }
    if (!arrived) {
      if (!mbar_wait(&s_bar, 0, &s_abort)) s_abort = 1;
      arrived = true;
    }
#pragma unroll
    for (int i = 0; i < kRowsUnroll; ++i) {
      const int u = base + i * 4 + tig;
      const uint4 xv = (u < nv && row_ok) ? srow[u] : make_uint4(0, 0, 0, 0);
      amax = absmax8(xv, amax);
      if (HAS_V) {
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
        const uint32_t vw[4] = {vv[i].x, vv[i].y, vv[i].z, vv[i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __half2 h;
          *reinterpret_cast<uint32_t*>(&h) = vw[e];
          const float2 vf = __half22float2(h);
          // elements 2e and 2e+1 of both 8-element pieces stand at MMA-K positions tig and tig + 4
          mma_tf32_16x8x8(d, __float_as_uint(vf.x), __float_as_uint(vf.y), xw[e] << 16, xw[e] & 0xFFFF0000u);
        }
      }
    }
  }
  if (!arrived && nv > 0 && !mbar_wait(&s_bar, 0, &s_abort)) s_abort = 1;  // the cast below reads the slice too
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  if (tig == 0) s_amax[warp][g] = amax;
  if (HAS_V) {
    s_acc[warp][(2 * tig) * 8 + g] = d[0];  // [token][j]
    s_acc[warp][(2 * tig + 1) * 8 + g] = d[1];
  }
  __syncthreads();
  const bool failed = s_abort != 0;
  if (tid < kRows) {
    float a = s_amax[0][tid];
    for (int w = 1; w < kTileWarps; ++w) a = fmaxf(a, s_amax[w][tid]);
    s_part_amax[tid] = failed ? __int_as_float(0x7F800000) : a;
  }
  if (HAS_V && tid >= 64 && tid < 64 + kRows * 8) {
    float v = 0.0f;
    for (int w = 0; w < kTileWarps; ++w) v += s_acc[w][tid - 64];
    s_part_t[tid - 64] = v;
  }
  if (C > 1) cluster.sync(); else __syncthreads();  // every CTA's partial results are written and visible
  if (tid < kRows) {
    float a = 0.0f;
    if (C == 1) {
      a = s_part_amax[tid];
    } else {
      for (int k = 0; k < C; ++k) a = fmaxf(a, cluster.map_shared_rank(s_part_amax, k)[tid]);
    }
    float s = 1.0f, inv = 1.0f;
    if (a != 0.0f) {
      s = __fdiv_rn(a, 448.0f);
      inv = __fdiv_rn(448.0f, a);
    }
    s_inv[tid] = inv;
    if (rank == 0 && tid < nrows) sx[m0 + tid] = s;
  }
  if (HAS_V && rank == 0 && tid >= 64 && tid < 64 + kRows * 8 && ((tid - 64) >> 3) < nrows) {
    float v = 0.0f;
    if (C == 1) {
      v = s_part_t[tid - 64];
    } else {
      for (int k = 0; k < C; ++k) v += cluster.map_shared_rank(s_part_t, k)[tid - 64];
    }
    t[static_cast<int64_t>(m0) * 8 + (tid - 64)] = v;
  }
  __syncthreads();
  // cast from shared memory: a thread's unit is one 16-byte vector in, eight bytes out
  if (!failed) {
    uint2* qv = reinterpret_cast<uint2*>(q);
    for (int idx = tid; idx < nrows * nv; idx += kTileThreads) {
      const int r = idx / nv, u = idx - r * nv;
      qv[static_cast<int64_t>(m0 + r) * nvec + v_begin + u] = cast8(s_x[r * pitch + u], s_inv[r]);
    }
  }
  if (C > 1) cluster.sync();  // no CTA may exit while a peer can still read its shared memory
}

template <bool HAS_V, int C>
cudaError_t launch_tile(const void* x, int64_t M, int64_t K, int64_t ldx, int vec_per_cta, uint8_t* q, float* sx,
                        const void* V, float* t, cudaStream_t st) {
  auto kernel = act_quant_tile_kernel<HAS_V, C>;
  const size_t smem = static_cast<size_t>(kRows) * (vec_per_cta + kTilePadVec) * sizeof(uint4);
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(once, [&] {
    attr_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kRows * (kTileMaxVec + kTilePadVec) * static_cast<int>(sizeof(uint4)));
  });
  if (attr_err != cudaSuccess) return attr_err;
  dim3 grid(C, static_cast<unsigned>((M + kRows - 1) / kRows));
  return launch_chained(kernel, grid, dim3(kTileThreads), smem, st, false, static_cast<const uint4*>(x),
                        static_cast<int>(M), static_cast<int>(K), ldx / 8, vec_per_cta, q, sx,
                        static_cast<const uint4*>(V), t);
}

template <bool HAS_V>
cudaError_t launch_tile_c(int c, const void* x, int64_t M, int64_t K, int64_t ldx, int vec_per_cta, uint8_t* q,
                          float* sx, const void* V, float* t, cudaStream_t st) {
  switch (c) {
    case 1: return launch_tile<HAS_V, 1>(x, M, K, ldx, vec_per_cta, q, sx, V, t, st);
    case 2: return launch_tile<HAS_V, 2>(x, M, K, ldx, vec_per_cta, q, sx, V, t, st);
    case 4: return launch_tile<HAS_V, 4>(x, M, K, ldx, vec_per_cta, q, sx, V, t, st);
    default: return launch_tile<HAS_V, 8>(x, M, K, ldx, vec_per_cta, q, sx, V, t, st);
  }
}

// ---- few tokens: a cluster of eight CTAs per row -------------------------------------------------
// With one CTA per token a decode-size call (1-64 tokens) leaves most SMs idle and its latency is one
// CTA walking a whole row and all of V.  Here eight CTAs of a thread-block cluster share a row: each
// takes an eighth of K, the partial absmax and LoRC sums meet through distributed shared memory, and
// every CTA casts its own part.
constexpr int kClusterSize = 8;
constexpr int kClusterThreads = 256;
constexpr int kClusterVpt = 2;  // 16-element units a thread keeps in registers

__global__ void __cluster_dims__(kClusterSize, 1, 1) __launch_bounds__(kClusterThreads)
act_quant_cluster_kernel(const uint4* __restrict__ x, int K, int64_t ldx_vec, uint8_t* __restrict__ q,
                         float* __restrict__ sx, const uint4* __restrict__ V, int r, float* __restrict__ t) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  pdl_launch_dependents();
  pdl_wait();  // x may be the output of the kernel before this one
  const int rank = static_cast<int>(cluster.block_rank());
  const int64_t m = blockIdx.y;
  const int nunits = K / kUnit;
  const int per = (nunits + kClusterSize - 1) / kClusterSize;
  const int u_begin = rank * per, u_end = min(nunits, u_begin + per);
  const uint4* row = x + m * ldx_vec;
  uint4* qrow = reinterpret_cast<uint4*>(q + m * static_cast<int64_t>(K));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  __shared__ float s_warp[kClusterThreads / 32];
  __shared__ float s_warp_t[kClusterThreads / 32][kRChunk];
  __shared__ float s_amax;        // this CTA's partial absmax (read by the whole cluster)
  __shared__ float s_tpart[64];   // this CTA's partial LoRC sums (read by rank 0)

  uint4 c0[kClusterVpt], c1[kClusterVpt];
  float a = 0.0f;
#pragma unroll
  for (int i = 0; i < kClusterVpt; ++i) {
    const int u = u_begin + tid + i * kClusterThreads;
    if (u < u_end) {
      c0[i] = __ldg(row + 2 * u);
      c1[i] = __ldg(row + 2 * u + 1);
    } else {
      c0[i] = make_uint4(0, 0, 0, 0);
      c1[i] = make_uint4(0, 0, 0, 0);
    }
    a = absmax8(c1[i], absmax8(c0[i], a));
  }
  a = warp_max(a);
  if (lane == 0) s_warp[warp] = a;

  if (V != nullptr) {
    const int kvec = K / 8;
    for (int j0 = 0; j0 < r; j0 += kRChunk) {
      float acc[kRChunk];
#pragma unroll
      for (int j = 0; j < kRChunk; ++j) acc[j] = 0.0f;
#pragma unroll
      for (int i = 0; i < kClusterVpt; ++i) {
        const int u = u_begin + tid + i * kClusterThreads;
        if (u < u_end) {
#pragma unroll
          for (int j = 0; j < kRChunk; ++j)
            if (j0 + j < r) {
              const uint4* vr = V + static_cast<int64_t>(j0 + j) * kvec;
              acc[j] = dot8(c1[i], __ldg(vr + 2 * u + 1), dot8(c0[i], __ldg(vr + 2 * u), acc[j]));
            }
        }
      }
#pragma unroll
      for (int j = 0; j < kRChunk; ++j) {
        const float v = warp_sum(acc[j]);
        if (lane == 0) s_warp_t[warp][j] = v;
      }
      __syncthreads();
      if (tid < kRChunk && j0 + tid < r) {
        float v = 0.0f;
        for (int w = 0; w < kClusterThreads / 32; ++w) v += s_warp_t[w][tid];
        s_tpart[j0 + tid] = v;
      }
      __syncthreads();
    }
  } else {
    __syncthreads();
  }
  if (tid == 0) {
    float v = s_warp[0];
    for (int w = 1; w < kClusterThreads / 32; ++w) v = fmaxf(v, s_warp[w]);
    s_amax = v;
  }
  cluster.sync();  // every CTA's s_amax and s_tpart are written and visible cluster-wide

  float amax = 0.0f;
  for (int k = 0; k < kClusterSize; ++k) amax = fmaxf(amax, *cluster.map_shared_rank(&s_amax, k));
  float s = 1.0f, inv = 1.0f;
  if (amax != 0.0f) {
    s = __fdiv_rn(amax, 448.0f);
    inv = __fdiv_rn(448.0f, amax);
  }
  if (rank == 0) {
    if (tid == 0) sx[m] = s;
    if (V != nullptr && tid < r) {
      float v = 0.0f;
      for (int k = 0; k < kClusterSize; ++k) v += cluster.map_shared_rank(s_tpart, k)[tid];
      t[m * r + tid] = v;
    }
  }
#pragma unroll
  for (int i = 0; i < kClusterVpt; ++i) {
    const int u = u_begin + tid + i * kClusterThreads;
    if (u < u_end) {
      const uint2 lo = cast8(c0[i], inv), hi = cast8(c1[i], inv);
      qrow[u] = make_uint4(lo.x, lo.y, hi.x, hi.y);
    }
  }
  cluster.sync();  // no CTA may exit while a peer can still read its shared memory
}

}  // namespace

int launch_act_quant(const void* x, int64_t M, int64_t K, int64_t ldx, uint8_t* q, float* sx,
                     const void* V, int r, float* t, cudaStream_t st, const float* amax_in) {
  if (M == 0) return ZQ_OK;
  cudaError_t err = cudaSuccess;
  const uint4* xv = static_cast<const uint4*>(x);
  const uint4* Vv = static_cast<const uint4*>(V);
  if (amax_in != nullptr && (V == nullptr || r == 8)) {
    // the absolute maxima are known: one streaming pass, eight rows per CTA whatever the token count
    dim3 grid(static_cast<unsigned>((M + kRows - 1) / kRows));
    if (V)
      err = launch_chained(act_quant_rows_kernel<true, true>, grid, dim3(kRowsThreads), 0, st, false, xv,
                           static_cast<int>(M), static_cast<int>(K), ldx / 8, q, sx, Vv, t, amax_in);
    else
      err = launch_chained(act_quant_rows_kernel<false, true>, grid, dim3(kRowsThreads), 0, st, false, xv,
                           static_cast<int>(M), static_cast<int>(K), ldx / 8, q, sx, Vv, t, amax_in);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
  }
  // enough rows for the eight-row CTAs to beat one row per CTA (measured: from about 50 CTAs on), and the
  // rank the row kernel is written for
  if (amax_in == nullptr && M >= kRowsMinTokens && (V == nullptr || r == 8)) {
    dim3 grid(static_cast<unsigned>((M + kRows - 1) / kRows));
    if (V)
      err = launch_chained(act_quant_rows_kernel<true, false>, grid, dim3(kRowsThreads), 0, st, false, xv,
                           static_cast<int>(M), static_cast<int>(K), ldx / 8, q, sx, Vv, t, amax_in);
    else
      err = launch_chained(act_quant_rows_kernel<false, false>, grid, dim3(kRowsThreads), 0, st, false, xv,
                           static_cast<int>(M), static_cast<int>(K), ldx / 8, q, sx, Vv, t, amax_in);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
  }
  // a few hundred tokens: eight rows per cluster of as many CTAs as make slices of at most 2048 columns (as long
  // as the cluster allows), so that even 32 tokens spread over dozens of SMs
  if (amax_in == nullptr && M >= kTileMinTokens && M < kRowsMinTokens && (V == nullptr || r == 8) && K >= 1024 &&
      K / 8 <= kTileMaxCluster * kTileMaxVec) {
    const int nvec = static_cast<int>(K / 8);
    int c = 1;
    while (c < kTileMaxCluster && (nvec + c - 1) / c > kTileMaxVec / 2) c *= 2;
    const int vec_per_cta = ((nvec + c - 1) / c + 3) / 4 * 4;
    err = V ? launch_tile_c<true>(c, x, M, K, ldx, vec_per_cta, q, sx, V, t, st)
            : launch_tile_c<false>(c, x, M, K, ldx, vec_per_cta, q, sx, nullptr, t, st);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
  }
  // fewer tokens than that, rows long enough to be worth sharing: a cluster of eight CTAs per row
  if (amax_in == nullptr && M < kRowsMinTokens && (M <= 256 || K >= 16384) && K >= 2048 &&
      K / kUnit <= kClusterSize * kClusterThreads * kClusterVpt) {
    dim3 grid(kClusterSize, static_cast<unsigned>(M));
    err = launch_chained(act_quant_cluster_kernel, grid, dim3(kClusterThreads), 0, st, false, xv, static_cast<int>(K),
                         ldx / 8, q, sx, Vv, r, t);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
  }
  const int nunits = static_cast<int>(K / kUnit);
  int threads = ((nunits + 31) / 32) * 32;
  if (threads > kMaxThreads) threads = kMaxThreads;
  const bool cached = nunits <= threads * kVpt;
  dim3 grid(static_cast<unsigned>(M));
  if (cached)
    err = launch_chained(act_quant_kernel<true>, grid, dim3(threads), 0, st, false, xv, static_cast<int>(K), ldx / 8, q,
                         sx, Vv, r, t, amax_in);
  else
    err = launch_chained(act_quant_kernel<false>, grid, dim3(threads), 0, st, false, xv, static_cast<int>(K), ldx / 8,
                         q, sx, Vv, r, t, amax_in);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // namespace zq
