// C-ABI entry points of libzqfp: argument validation, workspace carving, kernel dispatch.
// The operations themselves are defined in include/zqfp.h next to their citations.
#include <atomic>
#include <mutex>

#include "zq_common.cuh"

namespace zq {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
static std::atomic<int> g_exclusive{0};
bool exclusive_device() { return g_exclusive.load(std::memory_order_relaxed) != 0; }

int check_device_sm100() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ZQ_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ZQ_ERR_CUDA;
  return major == 10 ? ZQ_OK : ZQ_ERR_ARCH;
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool valid_mode(int mode) { return mode == ZQ_SCALE_NONE || mode == ZQ_SCALE_M1 || mode == ZQ_SCALE_M2; }
// 320 does not divide the 128-element K block: the per-group promotion of mode none is not written for it
bool valid_group(int g, int mode) { return g == 64 || g == 128 || g == 256 || (g == 320 && mode != ZQ_SCALE_NONE); }
// the tensor core's block scales are powers of two, and E5M2 as the cast target is about the shifts: only
// the constrained modes can use those layouts
bool valid_layout(int layout, int mode) {
  return layout == ZQ_WEIGHTS_CAST || layout == ZQ_WEIGHTS_MX ||
         ((layout == ZQ_WEIGHTS_MX_FP8 || layout == ZQ_WEIGHTS_CAST_E5M2) && mode != ZQ_SCALE_NONE);
}
inline bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }
// the sizes every linear entry point and size query accepts (the group size is checked where it is known)
bool valid_linear_shape(int64_t M, int64_t N, int64_t K, int r) {
  return M >= 0 && N >= 0 && K > 0 && K % 128 == 0 && r >= 0 && r <= 64 && r % 8 == 0 && M <= 0x7FFFFFFF &&
         N <= 0x7FFFFFFF && K <= (int64_t(1) << 30);
}

// Largest split-K scratch any token count up to M can need at this (N, K), over both kernel families.
// The plan depends on the token count only through the tile width and the number of token tiles, i.e.
// through ceil(m / 192), ceil(m / 224), ceil(m / 256) and a few thresholds up to 256: it is evaluated on
// both sides of every such breakpoint up to 65536 tokens; beyond that an upper bound of every plan is
// taken as well (no plan has more than 4 x SMs contributors of a 256 x 128 tile).
size_t max_partial_floats(int64_t M, int64_t N, int64_t K) {
  size_t best = 0;
  if (M <= 0 || N <= 0) return 0;
  auto probe = [&](int64_t m) {
    if (m <= 0 || m > M) return;
    for (int variant = 0; variant < 4; ++variant) {  // (none, cast), (M1, cast), (M1, block-scaled), (none, block-scaled)
      const GemmPlan pl = plan_gemm(m, N, K, (variant == 0 || variant == 3) ? ZQ_SCALE_NONE : ZQ_SCALE_M1,
                                    variant >= 2 ? ZQ_WEIGHTS_MX : ZQ_WEIGHTS_CAST);
      if (pl.partial_floats > best) best = pl.partial_floats;
      if (pl.pair) {  // a bf16 y takes the single-CTA plan
        const GemmPlan ps = plan_gemm(m, N, K, ZQ_SCALE_M1, ZQ_WEIGHTS_MX, false);
        if (ps.partial_floats > best) best = ps.partial_floats;
      }
    }
  };
  const int64_t small[10] = {16, 32, 64, 128, 129, 192, 193, 224, 256, M};
  for (int i = 0; i < 10; ++i) probe(small[i]);
  const int64_t top = M < 65536 ? M : 65536;
  const int widths[3] = {192, 224, 256};
  for (int w = 0; w < 3; ++w)
    for (int64_t m = widths[w]; m <= top; m += widths[w]) {
      probe(m);
      probe(m + 1);
    }
  if (M > 65536) {
    const size_t bound = 4 * static_cast<size_t>(sm_count()) * 256 * 128;
    if (bound > best) best = bound;
  }
  return best;
}

struct WsLayout {
  size_t off_partials, partial_floats, off_q, off_sx, off_t, off_x, off_y, total;
};
WsLayout ws_layout(int64_t M, int64_t N, int64_t K, int r, bool host_io) {
  WsLayout w{};
  size_t off = kWsHeadBytes;
  w.off_partials = off;
  w.partial_floats = max_partial_floats(M, N, K);
  off += round_up(w.partial_floats * 4, 256);
  w.off_q = off;
  off += round_up(static_cast<size_t>(M) * K, 256);
  w.off_sx = off;
  off += round_up(static_cast<size_t>(M) * 4, 256);
  w.off_t = off;
  off += round_up(static_cast<size_t>(M) * (r > 0 ? r : 1) * 4, 256);
  w.off_x = w.off_y = off;
  if (host_io) {
    w.off_x = off;
    off += round_up(static_cast<size_t>(M) * K * 2, 256);
    w.off_y = off;
    off += round_up(static_cast<size_t>(M) * N * 4, 256);
  }
  w.total = off;
  return w;
}

}  // namespace
}  // namespace zq

using namespace zq;

extern "C" {

const char* zq_status_string(int status) {
  switch (status) {
    case ZQ_OK: return "ok";
    case ZQ_ERR_NULL: return "a required pointer is NULL";
    case ZQ_ERR_SHAPE: return "unsupported shape";
    case ZQ_ERR_ALIGN: return "pointer or leading dimension not aligned";
    case ZQ_ERR_MODE: return "unknown scale mode or output type";
    case ZQ_ERR_WORKSPACE: return "workspace missing or too small";
    case ZQ_ERR_ARCH: return "device is not compute capability 10.x";
    case ZQ_ERR_CUDA: return "CUDA call failed";
    case ZQ_ERR_DEVICE_TIMEOUT: return "a kernel gave up on a bounded wait";
  }
  return "unknown status";
}

int64_t zq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int zq_set_exclusive_device(int on) { return g_exclusive.exchange(on ? 1 : 0, std::memory_order_relaxed); }

namespace {
int quantize_act(const void* x, int64_t M, int64_t K, int64_t ldx, const float* absmax, bool scaled, uint8_t* q,
                 float* sx, const void* V, int r, float* t, void* stream) {
  if (M < 0 || K < 16 || K % 16 || ldx < K || K > (int64_t(1) << 30) || M > 0x7FFFFFFF) return ZQ_ERR_SHAPE;
  if (V && (r <= 0 || r > 64)) return ZQ_ERR_SHAPE;
  if (M == 0) return ZQ_OK;
  if (!x || !q || !sx || (V && !t) || (scaled && !absmax)) return ZQ_ERR_NULL;
  if (!aligned16(x) || !aligned16(q) || ldx % 8 || (V && !aligned16(V))) return ZQ_ERR_ALIGN;
  if (int e = check_device_sm100()) return e;
  return launch_act_quant(x, M, K, ldx, q, sx, V, V ? r : 0, t, static_cast<cudaStream_t>(stream),
                          scaled ? absmax : nullptr);
}
}  // namespace

int zq_quantize_act_fp8(const void* x, int64_t M, int64_t K, int64_t ldx, uint8_t* q, float* sx,
                        const void* V, int r, float* t, void* stream) {
  return quantize_act(x, M, K, ldx, nullptr, false, q, sx, V, r, t, stream);
}

int zq_quantize_act_fp8_scaled(const void* x, int64_t M, int64_t K, int64_t ldx, const float* absmax, uint8_t* q,
                               float* sx, const void* V, int r, float* t, void* stream) {
  return quantize_act(x, M, K, ldx, absmax, true, q, sx, V, r, t, stream);
}

int zq_packed_weight_sizes(int64_t N, int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout,
                           size_t* codes_bytes, size_t* shift_bytes, size_t* scale_bytes) {
  if (!valid_mode(mode) || !valid_layout(layout, mode)) return ZQ_ERR_MODE;
  if (N < 0 || K <= 0 || !valid_group(group, mode) || K % group || K % kTileK) return ZQ_ERR_SHAPE;
  const size_t G = static_cast<size_t>(K / group);
  if (codes_bytes)
    *codes_bytes = static_cast<size_t>((N + kTileRows - 1) / kTileRows) * static_cast<size_t>(K / kTileK) * tile_bytes(layout);
  if (shift_bytes) *shift_bytes = mode == ZQ_SCALE_NONE ? 0 : static_cast<size_t>(N) * G;
  if (scale_bytes) *scale_bytes = mode == ZQ_SCALE_NONE ? static_cast<size_t>(N) * G * 4 : static_cast<size_t>(N) * 4;
  return ZQ_OK;
}

int zq_pack_weight_fp4(const float* W, int64_t N, int64_t K, int group, zq_scale_mode mode,
                       zq_weight_layout layout, uint8_t* codes, uint8_t* shift, float* scale, void* stream) {
  if (!valid_mode(mode) || !valid_layout(layout, mode)) return ZQ_ERR_MODE;
  if (N < 0 || K <= 0 || !valid_group(group, mode) || K % group || K % kTileK || N > 0x7FFFFFFF - kTileRows ||
      K > (int64_t(1) << 30))
    return ZQ_ERR_SHAPE;
  if (N == 0) return ZQ_OK;
  if (!W || !codes || !scale || (mode != ZQ_SCALE_NONE && !shift)) return ZQ_ERR_NULL;
  if (!aligned16(W) || !aligned16(codes)) return ZQ_ERR_ALIGN;
  if (int e = check_device_sm100()) return e;
  return launch_pack_weight(W, N, K, group, mode, layout, codes, shift, scale, static_cast<cudaStream_t>(stream));
}

size_t zq_w4a8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int r) {
  if (!valid_linear_shape(M, N, K, r)) return 0;
  return ws_layout(M, N, K, r, false).total;
}

size_t zq_w4a8_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int r) {
  if (!valid_linear_shape(M, N, K, r)) return 0;
  return ws_layout(M, N, K, r, true).total;
}

int zq_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return ZQ_ERR_NULL;
  if (workspace_bytes < kWsHeadBytes) return ZQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ZQ_ERR_ALIGN;
  return cudaMemsetAsync(workspace, 0, kWsHeadBytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? ZQ_OK
                                                                                                       : ZQ_ERR_CUDA;
}

namespace {
int linear_impl(const uint8_t* q, const float* sx, const void* x_bf16, int64_t ldx, int64_t M, int64_t N,
                int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout, const uint8_t* codes,
                const uint8_t* shift, const float* scale, const void* U, const void* V, const float* t, int r,
                void* y, zq_out_dtype ydt, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream,
                int relu, float* y_absmax) {
  if (!valid_mode(mode) || !valid_layout(layout, mode) || (ydt != ZQ_OUT_F32 && ydt != ZQ_OUT_BF16))
    return ZQ_ERR_MODE;
  if (!valid_linear_shape(M, N, K, r) || !valid_group(group, mode) || K % group || ldy < N) return ZQ_ERR_SHAPE;
  if (M == 0 || N == 0) return ZQ_OK;
  if (!codes || !scale || !y || (r > 0 && !U)) return ZQ_ERR_NULL;
  if (x_bf16) {
    if (r > 0 && !V) return ZQ_ERR_NULL;
    if (ldx < K) return ZQ_ERR_SHAPE;
  } else if (!q || !sx || (r > 0 && !t)) {
    return ZQ_ERR_NULL;
  }
  if (!aligned16(codes) || (q && !aligned16(q)) || (U && !aligned16(U)) || (t && !aligned16(t)) ||
      (x_bf16 && (!aligned16(x_bf16) || ldx % 8 || (V && !aligned16(V)))) ||
      (layout_is_mx(layout) && !aligned32(codes)))
    return ZQ_ERR_ALIGN;
  if (!workspace) return ZQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ZQ_ERR_ALIGN;
  const WsLayout w = ws_layout(M, N, K, r, false);
  const size_t need = x_bf16 ? w.total : w.off_q;
  if (workspace_bytes < need) return ZQ_ERR_WORKSPACE;
  const GemmPlan pl = plan_gemm(M, N, K, mode, layout);
  if (pl.ctas <= 0) return ZQ_ERR_SHAPE;
  if (int e = check_device_sm100()) return e;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // the epilogues add the tokens' maxima in with atomic max: start from zero
  if (y_absmax && cudaMemsetAsync(y_absmax, 0, static_cast<size_t>(M) * sizeof(float), st) != cudaSuccess)
    return ZQ_ERR_CUDA;
  if (x_bf16 && layout_is_mx(layout) && mode != ZQ_SCALE_NONE && M <= kFusedMaxTokens) {
    // Few tokens (decode): the block-scaled kernel quantizes the activations itself, so the layer is one
    // launch.  If that launch is refused, the two-kernel path below runs instead.
    GemmArgs f{};
    f.q = ws + w.off_q;  // where the kernel leaves the codes
    f.M = M;
    f.N = N;
    f.K = K;
    f.group = group;
    f.mode = mode;
    f.layout = layout;
    f.codes = codes;
    f.shift = shift;
    f.scale = scale;
    f.U = r > 0 ? U : nullptr;
    f.r = r;
    f.y = y;
    f.ydt = ydt;
    f.ldy = ldy;
    f.status = reinterpret_cast<int*>(ws);
    f.counters = reinterpret_cast<int*>(ws + kWsStatusBytes);
    f.partials = reinterpret_cast<float*>(ws + w.off_partials);
    f.partial_floats = w.partial_floats;
    f.x = x_bf16;
    f.ldx = ldx;
    f.V = r > 0 ? V : nullptr;
    f.fused_scratch = ws + kWsStatusBytes + kWsCounterBytes;
    f.relu = relu;
    f.y_amax = y_absmax;
    const int e = launch_w4a8_mx_gemm(f, st);
    if (e != kFusedLaunchRefused) return e;
  }
  if (x_bf16) {
    uint8_t* q_ws = ws + w.off_q;
    float* sx_ws = reinterpret_cast<float*>(ws + w.off_sx);
    float* t_ws = reinterpret_cast<float*>(ws + w.off_t);
    const int e = launch_act_quant(x_bf16, M, K, ldx, q_ws, sx_ws, r > 0 ? V : nullptr, r, t_ws, st);
    if (e) return e;
    q = q_ws;
    sx = sx_ws;
    t = t_ws;
  }
  GemmArgs a{};
  a.q = q;
  a.sx = sx;
  a.M = M;
  a.N = N;
  a.K = K;
  a.group = group;
  a.mode = mode;
  a.layout = layout;
  a.codes = codes;
  a.shift = shift;
  a.scale = scale;
  a.U = r > 0 ? U : nullptr;
  a.t = r > 0 ? t : nullptr;
  a.r = r;
  a.y = y;
  a.ydt = ydt;
  a.ldy = ldy;
  a.status = reinterpret_cast<int*>(ws);
  a.counters = reinterpret_cast<int*>(ws + kWsStatusBytes);
  a.partials = reinterpret_cast<float*>(ws + w.off_partials);
  a.partial_floats = w.partial_floats;
  a.relu = relu;
  a.y_amax = y_absmax;
  return layout_is_mx(layout) ? launch_w4a8_mx_gemm(a, st) : launch_w4a8_gemm(a, st);
}
}  // namespace

int zq_w4a8_linear(const uint8_t* q, const float* sx, const void* x_bf16, int64_t ldx, int64_t M, int64_t N,
                   int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout, const uint8_t* codes,
                   const uint8_t* shift, const float* scale, const void* U, const void* V, const float* t, int r,
                   void* y, zq_out_dtype ydt, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
  return linear_impl(q, sx, x_bf16, ldx, M, N, K, group, mode, layout, codes, shift, scale, U, V, t, r, y, ydt, ldy,
                     workspace, workspace_bytes, stream, 0, nullptr);
}

int zq_w4a8_linear_fused_out(const uint8_t* q, const float* sx, const void* x_bf16, int64_t ldx, int64_t M,
                             int64_t N, int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout,
                             const uint8_t* codes, const uint8_t* shift, const float* scale, const void* U,
                             const void* V, const float* t, int r, void* y, zq_out_dtype ydt, int64_t ldy,
                             void* workspace, size_t workspace_bytes, void* stream, int relu, float* y_absmax) {
  return linear_impl(q, sx, x_bf16, ldx, M, N, K, group, mode, layout, codes, shift, scale, U, V, t, r, y, ydt, ldy,
                     workspace, workspace_bytes, stream, relu ? 1 : 0, y_absmax);
}

int zq_w4a8_linear_plan(int64_t M, int64_t N, int64_t K, zq_scale_mode mode, zq_weight_layout layout,
                        int64_t* plan) {
  if (!plan) return ZQ_ERR_NULL;
  if (!valid_mode(mode) || !valid_layout(layout, mode)) return ZQ_ERR_MODE;
  if (M <= 0 || N <= 0 || K <= 0 || K % 128 || M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > (int64_t(1) << 30))
    return ZQ_ERR_SHAPE;
  const GemmPlan pl = plan_gemm(M, N, K, mode, layout);
  const int64_t v[ZQ_PLAN_WORDS] = {pl.bm,   pl.m_tiles,     pl.n_tiles, pl.ctas, pl.stream,    pl.persist,
                                    pl.splits, pl.kb_per_split, pl.base,  pl.rem,  pl.tail_pos0, pl.m_group,
                                    static_cast<int64_t>(pl.partial_floats), sm_count(), pl.pair};
  for (int i = 0; i < ZQ_PLAN_WORDS; ++i) plan[i] = v[i];
  return ZQ_OK;
}

namespace {

// Copy streams and events of the host-buffer entry point, one set per device, created on first use and
// kept until the process exits.  Large calls are cut into row chunks so that the upload of chunk i + 1,
// the kernels of chunk i and the download of chunk i - 1 overlap (token rows are independent).
constexpr int kHostMaxChunks = 32;
constexpr int64_t kHostChunkRows = 1024;
struct HostPipe {
  bool ok = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t entry = nullptr, up[kHostMaxChunks] = {}, done[kHostMaxChunks] = {};
};
HostPipe* host_pipe() {
  static HostPipe pipes[64];
  static std::once_flag once[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::call_once(once[dev], [dev] {
    HostPipe& p = pipes[dev];
    bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.entry, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kHostMaxChunks; ++i)
      ok = cudaEventCreateWithFlags(&p.up[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.done[i], cudaEventDisableTiming) == cudaSuccess;
    p.ok = ok;
  });
  return pipes[dev].ok ? &pipes[dev] : nullptr;
}

}  // namespace

int zq_w4a8_linear_host(const void* x_host, int64_t M, int64_t N, int64_t K, int group, zq_scale_mode mode,
                        zq_weight_layout layout, const uint8_t* codes, const uint8_t* shift, const float* scale,
                        const void* U, const void* V, int r, float* y_host, void* workspace, size_t workspace_bytes,
                        void* stream) {
  if (!valid_mode(mode) || !valid_layout(layout, mode)) return ZQ_ERR_MODE;
  if (!valid_linear_shape(M, N, K, r) || !valid_group(group, mode) || K % group) return ZQ_ERR_SHAPE;
  if (M == 0 || N == 0) return ZQ_OK;
  if (!x_host || !y_host) return ZQ_ERR_NULL;
  if (!workspace) return ZQ_ERR_WORKSPACE;
  const WsLayout w = ws_layout(M, N, K, r, true);
  if (workspace_bytes < w.total) return ZQ_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* x_dev = ws + w.off_x;
  float* y_dev = reinterpret_cast<float*>(ws + w.off_y);
  const uint8_t* xh = static_cast<const uint8_t*>(x_host);

  // chunks of at least kHostChunkRows rows, at most kHostMaxChunks of them
  int64_t rows = kHostChunkRows;
  if ((M + rows - 1) / rows > kHostMaxChunks) rows = (M + kHostMaxChunks - 1) / kHostMaxChunks;
  rows = (rows + 63) / 64 * 64;
  HostPipe* hp = M > rows ? host_pipe() : nullptr;
  if (!hp) {
    // one piece, everything on the caller's stream
    if (cudaMemcpyAsync(x_dev, xh, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return ZQ_ERR_CUDA;
    const int e = zq_w4a8_linear(nullptr, nullptr, x_dev, K, M, N, K, group, mode, layout, codes, shift, scale, U, V,
                                 nullptr, r, y_dev, ZQ_OUT_F32, N, workspace, w.off_x, stream);
    if (e) return e;
    if (cudaMemcpyAsync(y_host, y_dev, static_cast<size_t>(M) * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
      return ZQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? ZQ_OK : ZQ_ERR_CUDA;
  }

  // uploads wait for whatever the caller queued before this call
  if (cudaEventRecord(hp->entry, st) != cudaSuccess || cudaStreamWaitEvent(hp->in, hp->entry, 0) != cudaSuccess)
    return ZQ_ERR_CUDA;
  int rc = ZQ_OK;
  int c = 0;
  for (int64_t m0 = 0; m0 < M && rc == ZQ_OK; m0 += rows, ++c) {
    const int64_t mc = M - m0 < rows ? M - m0 : rows;
    uint8_t* xd = x_dev + static_cast<size_t>(m0) * K * 2;
    float* yd = y_dev + static_cast<size_t>(m0) * N;
    if (cudaMemcpyAsync(xd, xh + static_cast<size_t>(m0) * K * 2, static_cast<size_t>(mc) * K * 2,
                        cudaMemcpyHostToDevice, hp->in) != cudaSuccess ||
        cudaEventRecord(hp->up[c], hp->in) != cudaSuccess || cudaStreamWaitEvent(st, hp->up[c], 0) != cudaSuccess) {
      rc = ZQ_ERR_CUDA;
      break;
    }
    rc = zq_w4a8_linear(nullptr, nullptr, xd, K, mc, N, K, group, mode, layout, codes, shift, scale, U, V, nullptr, r, yd,
                        ZQ_OUT_F32, N, workspace, w.off_x, stream);
    if (rc) break;
    if (cudaEventRecord(hp->done[c], st) != cudaSuccess || cudaStreamWaitEvent(hp->out, hp->done[c], 0) != cudaSuccess ||
        cudaMemcpyAsync(y_host + static_cast<size_t>(m0) * N, yd, static_cast<size_t>(mc) * N * 4,
                        cudaMemcpyDeviceToHost, hp->out) != cudaSuccess)
      rc = ZQ_ERR_CUDA;
  }
  // the call is synchronous: nothing of it is left in flight, also after an error
  const bool s1 = cudaStreamSynchronize(hp->in) == cudaSuccess;
  const bool s2 = cudaStreamSynchronize(st) == cudaSuccess;
  const bool s3 = cudaStreamSynchronize(hp->out) == cudaSuccess;
  if (rc) return rc;
  return (s1 && s2 && s3) ? ZQ_OK : ZQ_ERR_CUDA;
}

int zq_device_status(void* workspace, int* detail, void* stream) {
  if (!workspace) return ZQ_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int words[2] = {0, 0};
  if (cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ZQ_ERR_CUDA;
  if (detail) *detail = words[1];
  if (words[0] != 0) {
    if (cudaMemsetAsync(workspace, 0, 8, st) != cudaSuccess) return ZQ_ERR_CUDA;
    return ZQ_ERR_DEVICE_TIMEOUT;
  }
  return ZQ_OK;
}

}  // extern "C"
