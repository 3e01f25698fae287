// Construction of the LoRC factors on the device (Section 3, first paragraph: the singular value decomposition
// of the error matrix E = W - W^ between the original and the quantized weight, truncated to rank r, its
// singular values split evenly between the two factors; Appendix A: ranks 8 .. 56).
//
// The paper takes a full SVD (an offline step on the host).  Here the rank-r part is found by randomized
// subspace iteration (Halko, Martinsson, Tropp 2011), which only needs products with E and E^T:
//   Y = E Omega                      Omega [K, l] Gaussian, l = r + 8, drawn by the caller
//   repeat `iters` times:  Q = orth(Y);  Z = E^T Q;  P = orth(Z);  Y = E P
//   Q = orth(Y);  Z = E^T Q  (= B^T for the small matrix B = Q^T E [l, K])
//   B B^T = Z^T Z = S diag(sigma^2) S^T   (Jacobi eigen-decomposition of an l x l matrix)
//   U^ = Q S_r diag(sigma_r)^(1/2),   V^ = diag(sigma_r)^(-1/2) S_r^T B
// orth() is a Cholesky QR applied twice.  Everything is FP32; the factors are stored as FP16, the type the
// linear layer reads them in.  All kernels are plain CUDA-core code: the step is offline and small next to
// the layer itself (six passes over E at two power iterations).
#include <cuda_fp16.h>

#include <type_traits>

#include "zq_common.cuh"

namespace zq {
namespace {

constexpr int kLMax = 72;  // r + oversampling, r <= 64
constexpr int kOver = 8;

// Round to nearest E2M1 value, ties to the code with mantissa bit 0, saturating at 6 (as the packer does).
__device__ __forceinline__ float e2m1_round(float v) {
  const float a = fabsf(v);
  const int c = (a > 0.25f) + (a >= 0.75f) + (a > 1.25f) + (a >= 1.75f) + (a > 2.5f) + (a >= 3.5f) + (a > 5.0f);
  const float mag = c == 0 ? 0.0f : (c == 1 ? 0.5f : (c == 2 ? 1.0f : (c == 3 ? 1.5f : (c == 4 ? 2.0f : (c == 5 ? 3.0f : (c == 6 ? 4.0f : 6.0f))))));
  return copysignf(mag, v);
}

// E[n, k] = W[n, k] - dec(RNE_E2M1(fl32(W / S^))) * S^, with S^ from the packer's shift / scale arrays.
__global__ void lorc_error_kernel(const float* __restrict__ W, int64_t K, int group, int mode,
                                  const uint8_t* __restrict__ shift, const float* __restrict__ scale,
                                  float* __restrict__ E) {
  const int64_t n = blockIdx.x;
  const int64_t G = K / group;
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
    const int64_t g = k / group;
    const float shat = mode == ZQ_SCALE_NONE ? scale[n * G + g] : ldexpf(scale[n], -static_cast<int>(shift[n * G + g]));
    const float w = W[n * K + k];
    E[n * K + k] = w - e2m1_round(__fdiv_rn(w, shat)) * shat;
  }
}

// C[n, 0..l) = sum_k A[n, k] * B[k, 0..l)   (A [rows, cols] row-major, B [cols, l]); one warp per row.
template <int L4>  // ceil(l / 4) accumulators of 4: l <= 4 * L4
__global__ void lorc_mul_kernel(const float* __restrict__ A, int64_t rows, int64_t cols, const float* __restrict__ B,
                                int l, float* __restrict__ C) {
  const int64_t n = static_cast<int64_t>(blockIdx.x) * (blockDim.x / 32) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (n >= rows) return;
  float acc[4 * L4];
#pragma unroll
  for (int j = 0; j < 4 * L4; ++j) acc[j] = 0.0f;
  for (int64_t k = lane; k < cols; k += 32) {
    const float a = __ldg(A + n * cols + k);
    const float* b = B + k * l;
#pragma unroll
    for (int j = 0; j < 4 * L4; ++j)
      if (j < l) acc[j] = fmaf(a, __ldg(b + j), acc[j]);
  }
#pragma unroll
  for (int j = 0; j < 4 * L4; ++j) {
    float v = acc[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    if (lane == 0 && j < l) C[n * l + j] = v;
  }
}

// C[k, 0..l) += sum_{n in chunk} A[n, k] * Y[n, 0..l)   (A [rows, cols] row-major: the product with A^T);
// a thread owns one column k, a CTA 128 columns and one chunk of rows whose part of Y sits in shared memory.
template <int L4>
__global__ void lorc_mul_t_kernel(const float* __restrict__ A, int64_t rows, int64_t cols, const float* __restrict__ Y,
                                  int l, int rows_per_cta, float* __restrict__ C) {
  extern __shared__ float s_y[];  // [chunk rows][l]
  const int64_t k = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t n0 = static_cast<int64_t>(blockIdx.y) * rows_per_cta;
  const int64_t n1 = n0 + rows_per_cta < rows ? n0 + rows_per_cta : rows;
  float acc[4 * L4];
#pragma unroll
  for (int j = 0; j < 4 * L4; ++j) acc[j] = 0.0f;
  for (int64_t nb = n0; nb < n1; nb += 32) {
    const int cnt = static_cast<int>(n1 - nb < 32 ? n1 - nb : 32);
    __syncthreads();
    for (int i = threadIdx.x; i < cnt * l; i += blockDim.x) s_y[i] = Y[nb * l + i];
    __syncthreads();
    if (k < cols) {
      for (int i = 0; i < cnt; ++i) {
        const float a = __ldg(A + (nb + i) * cols + k);
#pragma unroll
        for (int j = 0; j < 4 * L4; ++j)
          if (j < l) acc[j] = fmaf(a, s_y[i * l + j], acc[j]);
      }
    }
  }
  if (k < cols) {
#pragma unroll
    for (int j = 0; j < 4 * L4; ++j)
      if (j < l) atomicAdd(C + k * l + j, acc[j]);
  }
}

// G[l, l] += Y^T Y over a chunk of the rows of Y [rows, l].
__global__ void lorc_gram_kernel(const float* __restrict__ Y, int64_t rows, int l, int rows_per_cta, float* __restrict__ G) {
  const int64_t n0 = static_cast<int64_t>(blockIdx.x) * rows_per_cta;
  const int64_t n1 = n0 + rows_per_cta < rows ? n0 + rows_per_cta : rows;
  for (int e = threadIdx.x; e < l * l; e += blockDim.x) {
    const int i = e / l, j = e % l;
    if (j < i) continue;  // the upper triangle; mirrored below
    float acc = 0.0f;
    for (int64_t n = n0; n < n1; ++n) acc = fmaf(Y[n * l + i], Y[n * l + j], acc);
    atomicAdd(G + i * l + j, acc);
    if (j != i) atomicAdd(G + j * l + i, acc);
  }
}

// One CTA: Cholesky G = R^T R (R upper triangular) and Rinv = R^-1, both [l, l].  The diagonal is lifted by
// 1e-6 of its largest entry first: when Y has fewer independent columns than l (an error matrix of low rank)
// the dependent directions then come out as columns of small norm instead of divisions by zero; they add
// nothing to the leading Ritz pairs.
__global__ void lorc_chol_inv_kernel(float* __restrict__ G, int l, float* __restrict__ Rinv) {
  __shared__ float R[kLMax * kLMax];
  __shared__ float Ri[kLMax * kLMax];
  const int t = threadIdx.x;
  for (int e = t; e < l * l; e += blockDim.x) {
    R[e] = G[e];
    Ri[e] = 0.0f;
  }
  __syncthreads();
  const float tiny = 1e-30f;
  if (t == 0) {
    float dmax = 0.0f;
    for (int i = 0; i < l; ++i) dmax = fmaxf(dmax, R[i * l + i]);
    const float lift = 1e-6f * dmax + tiny;
    for (int i = 0; i < l; ++i) R[i * l + i] += lift;
  }
  __syncthreads();
  for (int c = 0; c < l; ++c) {
    if (t == 0) {
      float d = R[c * l + c];
      R[c * l + c] = sqrtf(d > tiny ? d : tiny);
    }
    __syncthreads();
    const float piv = R[c * l + c];
    for (int j = c + 1 + t; j < l; j += blockDim.x) R[c * l + j] /= piv;  // row c of R
    __syncthreads();
    for (int e = t; e < (l - c - 1) * (l - c - 1); e += blockDim.x) {     // trailing update
      const int i = c + 1 + e / (l - c - 1), j = c + 1 + e % (l - c - 1);
      if (j >= i) R[i * l + j] -= R[c * l + i] * R[c * l + j];
    }
    __syncthreads();
  }
  // Rinv by back substitution, one column per thread: R * x = e_j
  for (int j = t; j < l; j += blockDim.x) {
    for (int i = j; i >= 0; --i) {
      float v = (i == j) ? 1.0f : 0.0f;
      for (int m = i + 1; m <= j; ++m) v -= R[i * l + m] * Ri[m * l + j];
      Ri[i * l + j] = v / R[i * l + i];
    }
  }
  __syncthreads();
  for (int e = t; e < l * l; e += blockDim.x) Rinv[e] = Ri[e];
}

// Y[n, :] <- Y[n, :] * M   (M [l, l]); one thread per row.
__global__ void lorc_right_mul_kernel(float* __restrict__ Y, int64_t rows, int l, const float* __restrict__ Mx) {
  __shared__ float s_m[kLMax * kLMax];
  for (int e = threadIdx.x; e < l * l; e += blockDim.x) s_m[e] = Mx[e];
  __syncthreads();
  const int64_t n = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (n >= rows) return;
  float y[kLMax];
  for (int i = 0; i < l; ++i) y[i] = Y[n * l + i];
  for (int j = 0; j < l; ++j) {
    float v = 0.0f;
    for (int i = 0; i < l; ++i) v = fmaf(y[i], s_m[i * l + j], v);
    Y[n * l + j] = v;
  }
}

// One CTA: cyclic Jacobi eigen-decomposition of the symmetric T [l, l]: T = S diag(lambda) S^T.  Writes the
// eigenvectors as the columns of S, sorted by descending eigenvalue, and the eigenvalues.
__global__ void lorc_eig_kernel(const float* __restrict__ T, int l, float* __restrict__ S, float* __restrict__ lambda) {
  __shared__ float A[kLMax * kLMax];
  __shared__ float V[kLMax * kLMax];
  __shared__ float s_c, s_s;
  __shared__ int order[kLMax];
  const int t = threadIdx.x;
  for (int e = t; e < l * l; e += blockDim.x) {
    A[e] = T[e];
    V[e] = (e / l == e % l) ? 1.0f : 0.0f;
  }
  __syncthreads();
  for (int sweep = 0; sweep < 12; ++sweep) {  // FP32 Jacobi has converged long before
    for (int p = 0; p < l - 1; ++p)
      for (int q = p + 1; q < l; ++q) {
        if (t == 0) {
          const float apq = A[p * l + q], app = A[p * l + p], aqq = A[q * l + q];
          float c = 1.0f, s = 0.0f;
          if (fabsf(apq) > 1e-12f * sqrtf(fabsf(app * aqq)) && apq != 0.0f) {
            const float zeta = (aqq - app) / (2.0f * apq);
            const float tt = (zeta >= 0.0f ? 1.0f : -1.0f) / (fabsf(zeta) + sqrtf(1.0f + zeta * zeta));
            c = rsqrtf(1.0f + tt * tt);
            s = c * tt;
          }
          s_c = c;
          s_s = s;
        }
        __syncthreads();
        const float c = s_c, s = s_s;
        if (s != 0.0f) {
          for (int i = t; i < l; i += blockDim.x) {  // columns p and q of A and V
            const float aip = A[i * l + p], aiq = A[i * l + q];
            A[i * l + p] = c * aip - s * aiq;
            A[i * l + q] = s * aip + c * aiq;
            const float vip = V[i * l + p], viq = V[i * l + q];
            V[i * l + p] = c * vip - s * viq;
            V[i * l + q] = s * vip + c * viq;
          }
          __syncthreads();
          for (int i = t; i < l; i += blockDim.x) {  // rows p and q of A
            const float api = A[p * l + i], aqi = A[q * l + i];
            A[p * l + i] = c * api - s * aqi;
            A[q * l + i] = s * api + c * aqi;
          }
        }
        __syncthreads();
      }
  }
  if (t == 0) {
    for (int i = 0; i < l; ++i) order[i] = i;
    for (int a = 0; a < l; ++a)
      for (int b = a + 1; b < l; ++b)
        if (A[order[b] * l + order[b]] > A[order[a] * l + order[a]]) {
          const int x = order[a];
          order[a] = order[b];
          order[b] = x;
        }
  }
  __syncthreads();
  for (int e = t; e < l * l; e += blockDim.x) S[e] = V[(e / l) * l + order[e % l]];
  for (int j = t; j < l; j += blockDim.x) lambda[j] = A[order[j] * l + order[j]];
}

// out[n, c] = f16( sum_j X[n, j] * S[j, c] * g(lambda_c) ),  c < r;  g = sigma^(1/2) (U^) or sigma^(-1/2) (V^),
// sigma = sqrt(lambda).  U^ is stored [rows, r]; V^ transposed, [r, rows].
__global__ void lorc_finish_kernel(const float* __restrict__ X, int64_t rows, int l, int r, const float* __restrict__ S,
                                   const float* __restrict__ lambda, int inverse, int transpose_out,
                                   __half* __restrict__ out) {
  const int64_t n = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (n >= rows) return;
  for (int c = 0; c < r; ++c) {
    float v = 0.0f;
    for (int j = 0; j < l; ++j) v = fmaf(X[n * l + j], S[j * l + c], v);
    const float sigma = sqrtf(fmaxf(lambda[c], 0.0f));
    const float g = inverse ? (sigma > 0.0f ? rsqrtf(sigma) : 0.0f) : sqrtf(sigma);
    v *= g;
    if (transpose_out) out[static_cast<int64_t>(c) * rows + n] = __float2half_rn(v);
    else out[n * r + c] = __float2half_rn(v);
  }
}

struct LorcWs {
  size_t off_E, off_Y, off_Z, off_G, off_Rinv, off_S, off_lambda, total;
};
LorcWs lorc_ws(int64_t N, int64_t K, int l) {
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  LorcWs w{};
  size_t off = 0;
  w.off_E = off;
  off += up(static_cast<size_t>(N) * K * 4);
  w.off_Y = off;
  off += up(static_cast<size_t>(N) * l * 4);
  w.off_Z = off;
  off += up(static_cast<size_t>(K) * l * 4);
  w.off_G = off;
  off += up(static_cast<size_t>(l) * l * 4);
  w.off_Rinv = off;
  off += up(static_cast<size_t>(l) * l * 4);
  w.off_S = off;
  off += up(static_cast<size_t>(l) * l * 4);
  w.off_lambda = off;
  off += up(static_cast<size_t>(l) * 4);
  w.total = off;
  return w;
}

template <typename F>
bool by_width(int l, F&& f) {  // the accumulator count of the product kernels is a template parameter
  if (l <= 16) return f(std::integral_constant<int, 4>{});
  if (l <= 32) return f(std::integral_constant<int, 8>{});
  if (l <= 48) return f(std::integral_constant<int, 12>{});
  return f(std::integral_constant<int, 18>{});
}

}  // namespace
}  // namespace zq

using namespace zq;

extern "C" {

size_t zq_lorc_workspace_bytes(int64_t N, int64_t K, int r) {
  if (N <= 0 || K <= 0 || r <= 0 || r > 64 || r % 8) return 0;
  return lorc_ws(N, K, r + kOver).total;
}

int zq_lorc_factors(const float* W, int64_t N, int64_t K, int group, zq_scale_mode mode, const uint8_t* shift,
                    const float* scale, int r, const float* omega, int iters, void* U_f16, void* V_f16,
                    float* sigma2, void* workspace, size_t workspace_bytes, void* stream) {
  if (mode != ZQ_SCALE_NONE && mode != ZQ_SCALE_M1 && mode != ZQ_SCALE_M2) return ZQ_ERR_MODE;
  if (N <= 0 || K <= 0 || group <= 0 || K % group || r <= 0 || r > 64 || r % 8 || iters < 0 || iters > 8 ||
      N > 0x7FFFFFFF || K > (int64_t(1) << 30))
    return ZQ_ERR_SHAPE;
  const int l = r + kOver;
  if (l > N || l > K) return ZQ_ERR_SHAPE;
  if (!W || !scale || !omega || !U_f16 || !V_f16 || (mode != ZQ_SCALE_NONE && !shift)) return ZQ_ERR_NULL;
  if (!workspace) return ZQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ZQ_ERR_ALIGN;
  const LorcWs w = lorc_ws(N, K, l);
  if (workspace_bytes < w.total) return ZQ_ERR_WORKSPACE;
  if (int e = check_device_sm100()) return e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* E = reinterpret_cast<float*>(ws + w.off_E);
  float* Y = reinterpret_cast<float*>(ws + w.off_Y);
  float* Z = reinterpret_cast<float*>(ws + w.off_Z);
  float* G = reinterpret_cast<float*>(ws + w.off_G);
  float* Rinv = reinterpret_cast<float*>(ws + w.off_Rinv);
  float* S = reinterpret_cast<float*>(ws + w.off_S);
  float* lambda = reinterpret_cast<float*>(ws + w.off_lambda);
  bool ok = true;
  int launches = 0;

  lorc_error_kernel<<<static_cast<unsigned>(N), 256, 0, st>>>(W, K, group, mode, shift, scale, E);
  ++launches;
  // C [rows, l] = A B  and  C [cols, l] = A^T Y  with A = E [N, K]
  auto mul = [&](const float* B, float* C) {
    by_width(l, [&](auto L4) {
      lorc_mul_kernel<decltype(L4)::value><<<static_cast<unsigned>((N + 7) / 8), 256, 0, st>>>(E, N, K, B, l, C);
      return true;
    });
    ++launches;
  };
  auto mul_t = [&](const float* Yin, float* C) {
    ok = ok && cudaMemsetAsync(C, 0, static_cast<size_t>(K) * l * 4, st) == cudaSuccess;
    const int rows_per_cta = 256;
    dim3 grid(static_cast<unsigned>((K + 127) / 128), static_cast<unsigned>((N + rows_per_cta - 1) / rows_per_cta));
    by_width(l, [&](auto L4) {
      lorc_mul_t_kernel<decltype(L4)::value><<<grid, 128, 32 * l * sizeof(float), st>>>(E, N, K, Yin, l, rows_per_cta, C);
      return true;
    });
    ++launches;
  };
  // X [rows, l] <- an orthonormal basis of its columns (Cholesky QR, twice)
  auto orth = [&](float* X, int64_t rows) {
    for (int pass = 0; pass < 2; ++pass) {
      ok = ok && cudaMemsetAsync(G, 0, static_cast<size_t>(l) * l * 4, st) == cudaSuccess;
      lorc_gram_kernel<<<static_cast<unsigned>((rows + 255) / 256), 256, 0, st>>>(X, rows, l, 256, G);
      lorc_chol_inv_kernel<<<1, 256, 0, st>>>(G, l, Rinv);
      lorc_right_mul_kernel<<<static_cast<unsigned>((rows + 127) / 128), 128, 0, st>>>(X, rows, l, Rinv);
      launches += 3;
    }
  };

  mul(omega, Y);
  for (int it = 0; it < iters; ++it) {
    orth(Y, N);
    mul_t(Y, Z);
    orth(Z, K);
    mul(Z, Y);
  }
  orth(Y, N);    // Q
  mul_t(Y, Z);   // B^T = E^T Q
  ok = ok && cudaMemsetAsync(G, 0, static_cast<size_t>(l) * l * 4, st) == cudaSuccess;
  lorc_gram_kernel<<<static_cast<unsigned>((K + 255) / 256), 256, 0, st>>>(Z, K, l, 256, G);   // B B^T
  lorc_eig_kernel<<<1, 128, 0, st>>>(G, l, S, lambda);
  lorc_finish_kernel<<<static_cast<unsigned>((N + 127) / 128), 128, 0, st>>>(Y, N, l, r, S, lambda, 0, 0,
                                                                            static_cast<__half*>(U_f16));
  lorc_finish_kernel<<<static_cast<unsigned>((K + 127) / 128), 128, 0, st>>>(Z, K, l, r, S, lambda, 1, 1,
                                                                            static_cast<__half*>(V_f16));
  launches += 4;
  if (sigma2)  // the eigenvalues of B B^T are the squares of the singular values
    ok = ok && cudaMemcpyAsync(sigma2, lambda, static_cast<size_t>(r) * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  count_launch(launches);
  return (ok && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // extern "C"
