// zq_w4a8_linear_noalloc: the quantized linear layer for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off the table: code inside a real-time or
// safety-reviewed serving loop whose memory plan is frozen at start-up, plug-ins that are handed
// tensors by a host framework but own no allocator, and processes whose memory pool has already
// claimed the whole device.  The regular entry point needs a caller-provided workspace for the
// split-K counters and partial sums; this variant keeps that scratch in a fixed array that is part of
// the library image, so the caller passes only inputs and outputs.
//
// The array lives in every device context that loads the library until the process exits.  All
// calls on a device share it, so two calls that overlap on the GPU (different streams, or different
// host threads) race on it: serialize them.
#include <mutex>

#include "zq_common.cuh"

namespace zq {
namespace {

// status words + tile counters, then split-K partial sums
constexpr size_t kScratchBytes = size_t(32) << 20;  // 32 MiB
constexpr size_t kScratchPartialFloats = (kScratchBytes - kWsHeadBytes) / 4;

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// The device address of g_scratch on the current device.  In host code the symbol's name is only a
// handle; the address the kernels need comes from cudaGetSymbolAddress, once per device.
int scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ZQ_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return ZQ_ERR_SHAPE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) return ZQ_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return ZQ_OK;
}

}  // namespace
}  // namespace zq

using namespace zq;

extern "C" {

size_t zq_w4a8_linear_noalloc_max_scratch_bytes(void) { return kScratchBytes; }

int zq_w4a8_linear_noalloc(const uint8_t* q, const float* sx, int64_t M, int64_t N, int64_t K, int group,
                           zq_scale_mode mode, const uint8_t* codes, const uint8_t* shift, const float* scale,
                           const void* U, const float* t, int r, void* y, zq_out_dtype ydt, int64_t ldy,
                           void* stream) {
  if (mode != ZQ_SCALE_NONE && mode != ZQ_SCALE_M1 && mode != ZQ_SCALE_M2) return ZQ_ERR_MODE;
  if (ydt != ZQ_OUT_F32 && ydt != ZQ_OUT_BF16) return ZQ_ERR_MODE;
  if (M < 0 || N < 0 || K <= 0 || K % 128 || (group != 64 && group != 128 && group != 256) || K % group || r < 0 ||
      r > 64 || r % 8 || ldy < N || M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > (int64_t(1) << 30))
    return ZQ_ERR_SHAPE;
  if (M == 0 || N == 0) return ZQ_OK;
  if (!q || !sx || !codes || !scale || !y || (r > 0 && (!U || !t)))
    return ZQ_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(codes) | reinterpret_cast<uintptr_t>(U) |
       reinterpret_cast<uintptr_t>(t)) & 15u)
    return ZQ_ERR_ALIGN;
  // the fixed scratch bounds the split-K partial sums this problem may need
  const GemmPlan pl = plan_gemm(M, N, K, mode, ZQ_WEIGHTS_CAST);
  if (pl.partial_floats > kScratchPartialFloats || pl.ctas <= 0) return ZQ_ERR_WORKSPACE;

  if (int e = check_device_sm100()) return e;
  void* scratch = nullptr;
  if (int e = scratch_address(&scratch)) return e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* base = static_cast<unsigned char*>(scratch);
  // The array keeps whatever the last call left: the tile counters must start at zero.  The status words
  // are left alone, so that an error recorded by an earlier call stays readable until
  // zq_w4a8_linear_noalloc_status fetches (and clears) it.
  if (cudaMemsetAsync(base + kWsStatusBytes, 0, kWsCounterBytes, st) != cudaSuccess) return ZQ_ERR_CUDA;

  GemmArgs a{};
  a.q = q;
  a.sx = sx;
  a.M = M;
  a.N = N;
  a.K = K;
  a.group = group;
  a.mode = mode;
  a.codes = codes;
  a.shift = shift;
  a.scale = scale;
  a.U = r > 0 ? U : nullptr;
  a.t = r > 0 ? t : nullptr;
  a.r = r;
  a.y = y;
  a.ydt = ydt;
  a.ldy = ldy;
  a.status = reinterpret_cast<int*>(base);
  a.counters = reinterpret_cast<int*>(base + kWsStatusBytes);
  a.partials = reinterpret_cast<float*>(base + kWsHeadBytes);
  a.partial_floats = kScratchPartialFloats;
  return launch_w4a8_gemm(a, st);
}

int zq_w4a8_linear_noalloc_status(int* detail, void* stream) {
  void* scratch = nullptr;
  if (int e = scratch_address(&scratch)) return e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int words[2] = {0, 0};
  if (cudaMemcpyAsync(words, scratch, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ZQ_ERR_CUDA;
  if (detail) *detail = words[1];
  if (words[0] == 0) return ZQ_OK;
  if (cudaMemsetAsync(scratch, 0, 8, st) != cudaSuccess) return ZQ_ERR_CUDA;
  return ZQ_ERR_DEVICE_TIMEOUT;
}

}  // extern "C"
