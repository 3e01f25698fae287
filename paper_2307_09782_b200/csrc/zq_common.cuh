// Shared helpers for the zqfp kernels: thin wrappers over the sm_100a PTX this library uses
// (mbarrier, TMA bulk tensor loads, tcgen05 MMA / TMEM) and the host-side launch bookkeeping.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/zqfp.h"

namespace zq {

// ---- host-side bookkeeping ---------------------------------------------------------------------
void count_launch(int n = 1);  // adds to the process-wide launch counter
int check_device_sm100();      // ZQ_OK when the current device is compute capability 10.x

// Workspace head: status words the kernels may write (256 bytes), then the split-K tile counters.
constexpr size_t kWsStatusBytes = 256;
// status[0] error code, status[1] detail
constexpr int kWsMaxTiles = 16384;  // counters: one int per output tile
constexpr size_t kWsCounterBytes = size_t(kWsMaxTiles) * 4;
// ... then the scratch in which the CTAs of the block-scaled kernel meet when it quantizes the activations itself
constexpr int kFusedMaxTokens = 16;
constexpr int kFusedMaxRank = 64;
constexpr int kFusedSlots = 8;           // copies of the absmax / LoRC sums the atomics are spread over
constexpr size_t kWsFusedBytes = 37632;  // 16 bytes of counters + 8 x (16 absmax words + 16 x 64 LoRC sums) + the sums' total, rounded up
constexpr size_t kWsHeadBytes = kWsStatusBytes + kWsCounterBytes + kWsFusedBytes;

// ---- packed weight format (written by the packer, streamed by the GEMM) --------------------------
// The weight is stored as tiles of 128 output rows x 128 input features, tile (nt, kb) at byte offset
// (nt * (K / 128) + kb) * kTileBytes, so that a CTA walking along K reads one contiguous stream.
// A tile holds
//   [0, 8192)    codes: 16-byte chunk c (elements 32c .. 32c+31 of the K block) of row r at (c * 128 + r) * 16;
//                inside a chunk, 32-bit word j holds elements 8j .. 8j+7: nibble i (bits 4i .. 4i+2) = the
//                E2M1 magnitude bits of element i, bit 8b+7 = sign of element b, bit 8b+3 = sign of element
//                4+b (b < 4).  That order lets the cast to E4M3 take signs with one AND per four elements.
//   [8192, 8448) shifts: byte 2r + h = exponent shift of row r for elements 64h .. 64h+63 (zero in mode none)
// Rows beyond N in the last tile are zero.
constexpr int kTileRows = 128;
constexpr int kTileK = 128;
constexpr int kTileCodeBytes = kTileRows * kTileK / 2;
constexpr int kTileShiftBytes = 2 * kTileRows;
constexpr int kTileBytes = kTileCodeBytes + kTileShiftBytes;

// Layout ZQ_WEIGHTS_MX (modes M1 / M2), for the tensor core's own FP4 operand.  The same 128 x 128 tiles, 8704
// bytes each, but a block of 128 output rows keeps the codes of all its K blocks first and their scales after:
// block nt starts at nt * (K / 128) * 8704 and holds
//   [kb * 8192, +8192)                codes of K block kb, row-major: row r at r * 64, element k of the K block
//                                     in byte k / 2 (even k in the low nibble), a nibble being the plain E2M1
//                                     code (sign in bit 3)
//   [(K / 128) * 8192 + kb * 512, +512)  its block scales, one E8M0 byte 127 - shift per row and 32 elements, in
//                                     the order the tensor-memory copy wants: byte 16 * (r % 32) + 4 * (r / 32) + s
//                                     for row r, elements 32s .. 32s+31
// so that the codes (and the scales) of consecutive K blocks are contiguous and one copy brings several.
constexpr int kMxTileScaleBytes = 4 * kTileRows;
constexpr int kMxTileBytes = kTileCodeBytes + kMxTileScaleBytes;
__host__ __device__ inline int64_t mx_code_offset(int kb) { return static_cast<int64_t>(kb) * kTileCodeBytes; }
__host__ __device__ inline int64_t mx_scale_offset(int kblocks, int kb) {
  return static_cast<int64_t>(kblocks) * kTileCodeBytes + static_cast<int64_t>(kb) * kMxTileScaleBytes;
}

// Layout ZQ_WEIGHTS_MX_FP8: the same arrangement with one E4M3 byte per element (a tile's codes are 16384 bytes,
// row r at r * 128), for FP8 weights.
constexpr int kMx8TileBytes = 2 * kTileCodeBytes + kMxTileScaleBytes;

inline size_t tile_bytes(int layout) {
  return layout == ZQ_WEIGHTS_MX ? kMxTileBytes : (layout == ZQ_WEIGHTS_MX_FP8 ? kMx8TileBytes : kTileBytes);
}
inline bool layout_is_mx(int layout) { return layout == ZQ_WEIGHTS_MX || layout == ZQ_WEIGHTS_MX_FP8; }

// ---- launchers implemented in the .cu files ------------------------------------------------------
// amax_in: the tokens' absolute maxima when the caller already has them (one pass: no reduction, no second read)
int launch_act_quant(const void* x, int64_t M, int64_t K, int64_t ldx, uint8_t* q, float* sx,
                     const void* V, int r, float* t, cudaStream_t st, const float* amax_in = nullptr);
int launch_pack_weight(const float* W, int64_t N, int64_t K, int group, int mode, int layout, uint8_t* codes,
                       uint8_t* shift, float* scale, cudaStream_t st);

struct GemmArgs {
  const uint8_t* q;      // [M, K] E4M3
  const float* sx;       // [M]
  int64_t M, N, K;
  int group, mode;
  int layout;            // ZQ_WEIGHTS_CAST or ZQ_WEIGHTS_MX
  const uint8_t* codes;  // tiled, see above
  const uint8_t* shift;  // [N, G] or NULL (not read by the GEMM: the tiles carry the shifts)
  const float* scale;    // [N] or [N, G]
  const void* U;         // fp16 [N, r] or NULL
  const float* t;        // [M, r] or NULL
  int r;
  void* y;
  int ydt;
  int64_t ldy;
  int* status;           // workspace status words
  int* counters;         // split-K tile counters
  float* partials;       // split-K partial sums
  size_t partial_floats; // capacity of `partials`
  // set only when the block-scaled kernel is to quantize the activations itself (at most kFusedMaxTokens tokens;
  // q then names the buffer the kernel writes the codes to, sx and t are unused):
  const void* x;         // bf16 [M, ldx]
  int64_t ldx;
  const void* V;         // fp16 [r, K] or NULL
  void* fused_scratch;   // kWsFusedBytes of the workspace head
  // fusion on the output side: y = max(y, 0) before the store, and / or the per-token max |y| (of the values as
  // stored) added with atomic max into y_amax [M] for the next layer's quantizer.  Either one keeps shared output
  // tiles off the paths that add into y (their final values are known to no CTA): partial sums go through the
  // workspace instead, as for a bf16 y.
  int relu;
  float* y_amax;
};
// Returned by launch_w4a8_mx_gemm when that launch was refused (the grid cannot be resident at once): nothing
// ran; the caller quantizes with the separate kernel and launches the plain GEMM.
constexpr int kFusedLaunchRefused = 1;
// Tile shape chosen for a problem (shared by the workspace-size query and the launcher).
struct GemmPlan {
  int bm;      // tokens per tile (the MMA's N extent)
  int m_tiles, n_tiles;
  int stream;  // 1: the (tile, K block) units are dealt out evenly to `ctas` CTAs; 0: tiles x splits CTAs
  int persist; // 1: `ctas` CTAs walk whole tiles, every ctas-th one, up to position tail_pos0 of the launch
               //    order; the rest (less than one round) is dealt out as unit ranges (base, rem)
  int tail_pos0;
  int ctas;
  int splits;        // stream == 0: split-K factor
  int kb_per_split;  // stream == 0: 128-element K blocks per split
  int base, rem;     // stream == 1: units per CTA (the first `rem` CTAs take one more)
  int m_group;       // the launch order runs through groups of this many token tiles (0 or 1: along N only)
  int pair;          // 1: CTA pairs (CTAs 2c, 2c + 1 = pair c).  Positions, tail_pos0 and the units of base / rem then
                     //    count pair positions (token tile x two neighbouring channel tiles) and pairs, not tiles and CTAs
  size_t partial_floats;
};
// allow_pair = false: the plan for single CTAs (shared output tiles of a bf16 y go through the workspace, which
// the pair kernel does not do).
GemmPlan plan_gemm(int64_t M, int64_t N, int64_t K, int mode, int layout, bool allow_pair = true);
int launch_w4a8_gemm(const GemmArgs& a, cudaStream_t st);           // ZQ_WEIGHTS_CAST
int launch_w4a8_mx_gemm(const GemmArgs& a, cudaStream_t st);        // ZQ_WEIGHTS_MX
int sm_count();
bool exclusive_device();  // see zq_set_exclusive_device
constexpr int kErrDetailSelfTest = 100;  // status detail written by zq_selftest_bounded_wait

#ifdef __CUDACC__
// ---- programmatic dependent launch ---------------------------------------------------------------
// The kernels of one layer (quantizer, then GEMM) and of consecutive layers are chained with programmatic
// stream serialization: a kernel lets its successor start early (launch_dependents), and every kernel waits
// for its predecessor's completion (pdl_wait) before it touches anything the predecessor may have written.
// What runs before that wait is setup, and in the GEMM the first weight copies (weights are read-only data
// of the layer).  A kernel launched without such a predecessor passes the wait at once.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with the programmatic-serialization attribute (and, if asked, as a cooperative launch).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  bool cooperative, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  unsigned n = 0;
  at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cooperative) {
    at[n].id = cudaLaunchAttributeCooperative;
    at[n].val.cooperative = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- device: bounded waits -----------------------------------------------------------------------
// Every wait in this library is bounded (a poll count and, for the parked waits, two seconds of
// wall time); when one runs out the kernel records an error in the workspace status word and
// unwinds instead of hanging.
constexpr uint32_t kSpinLimit = 1u << 24;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same test, but the hardware may park the thread for up to `hint_ns` while the phase is pending
// (it resumes as soon as the phase completes), so a waiting warp costs almost no issue slots.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when kWaitLimitNs passed or another thread of the CTA already raised
// `abort_flag`; the caller then records the error and unwinds.
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    if (mbar_try_wait_parked(bar, parity, 50000u)) return true;
    if (*abort_flag) return false;
    if (((spin & 7u) == 7u || limit_ns < kWaitLimitNs) && global_timer_ns() - t0 > limit_ns) return false;
  }
  return false;
}

// Warp-uniform wait: lane 0 polls, the result is broadcast, and the warp leaves converged (the
// tcgen05 .sync.aligned instructions that follow such a wait need every lane to arrive together).
// All 32 lanes must call it.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  int ok = 0;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
  ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
  return ok != 0;
}

// One lane of a converged warp (the same lane every time).  Code that feeds tcgen05 / TMA instructions
// is kept warp-uniform and only the issuing instruction is predicated on this, so that addresses and
// descriptors stay in uniform registers.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xFFFFFFFF;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- device: proxies, TMA ------------------------------------------------------------------------
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled load global -> shared, completion counted in bytes on `bar`.  c0 is the innermost
// coordinate; c0 * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* m, int c0, int c1,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

// The same for a 3-D tensor map (c0 innermost).
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, int c0, int c1, int c2,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// The same for a 4-D tensor map.
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* m, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
      : "memory");
}

// Contiguous global -> shared copy of `bytes` (multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// ---- device: tcgen05 / TMEM ----------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {  // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // one full warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], 8-bit float operands (E4M3 x E4M3), FP32 accumulate.
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with the A operand taken from tensor memory (row i of A in lane i, 4 bytes of K per column).
__device__ __forceinline__ void umma_f8_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Block-scaled form: A and B are MX operands (here E2M1 x E4M3) whose 32-element blocks along K are
// multiplied by the power-of-two (E8M0) scales found in tensor memory at sfa / sfb.
__device__ __forceinline__ void umma_mxf8f6f4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}
// Shared memory -> tensor memory: 32 rows of 16 bytes (described by `sdesc`) land in lanes 0..31 of four
// consecutive columns and are repeated in the other three lane quarters.  Runs in order with the MMAs
// issued by the same thread.
__device__ __forceinline__ void tmem_cp_32x128b_x4(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// Arrive once on `bar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// ---- CTA pairs (cta_group::2): two CTAs of a cluster work on one MMA of 256 rows ---------------------
// Each CTA holds its own 128 rows of A, half of the rows of B and its own 128 lanes of D; the leader (cluster
// rank 0) issues the MMAs for both.  Allocation and release of tensor memory are executed by one warp of
// each CTA; copies, MMAs and commits by one thread of the leader.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// The address, in the cluster's shared window, of the same shared-memory location in CTA `rank`.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {  // every thread of every CTA of the cluster
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {  // a barrier of any CTA of the cluster
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {  // one full warp of each CTA
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {  // one full warp of each CTA
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Tiled loads whose completion is counted on a barrier of either CTA of the pair (`bar_cluster_addr`: an
// address in the cluster's shared window); the destination is this CTA's shared memory.
__device__ __forceinline__ void tma_load_3d_pair(void* smem_dst, const CUtensorMap* m, int c0, int c1, int c2,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(void* smem_dst, const CUtensorMap* m, int c0, int c1, int c2, int c3,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
      : "memory");
}
__device__ __forceinline__ void umma_mxf8f6f4_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                   uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}
// Each CTA's 32 x 16 bytes of its own shared memory (same offset in both) to its own tensor memory.
__device__ __forceinline__ void tmem_cp_32x128b_x4_pair(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// Arrive once on the barrier at this shared-memory offset in both CTAs of the pair when every MMA issued so
// far by this thread has completed.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(smem_u32(bar)), "h"(static_cast<uint16_t>(3))
      : "memory");
}
// 16 consecutive FP32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// 4 consecutive FP32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
// 8 consecutive FP32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
// Store 16 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// The same wait, tied to the registers of a load issued earlier: their later uses cannot be scheduled
// ahead of the wait.
template <int NC>
__device__ __forceinline__ void tmem_ld_wait_regs(float* v) {
  static_assert(NC == 4 || NC == 8 || NC == 16, "4, 8 or 16 columns");
  if (NC == 16)
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]),
                   "+f"(v[8]), "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]),
                   "+f"(v[15])
                 :
                 : "memory");
  else if (NC == 8)
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7])
                 :
                 : "memory");
  else
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]) : : "memory");
}

// ---- packed pairs of FP32 (one 64-bit register; both halves computed by one instruction) ----------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes, stored as 8-row x 128-byte
// atoms (1024 bytes apart) with the 128-byte swizzle.  Adding (bytes >> 4) to the low word moves the
// start along K inside the 128-byte row.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr >> 4) & 0x3FFF);  // start address, 16-byte units
  d |= uint64_t(1) << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= uint64_t(1024 >> 4) << 32;            // stride byte offset: next 8-row atom
  d |= uint64_t(1) << 46;                    // descriptor version of this architecture
  d |= uint64_t(2) << 61;                    // 128-byte swizzle
  return d;
}
// Shared-memory descriptor without swizzle: rows of 16 bytes, 8-row groups `group_stride` bytes apart.
__device__ __forceinline__ uint64_t umma_desc_rows16(uint32_t smem_addr, uint32_t group_stride) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr >> 4) & 0x3FFF);
  d |= uint64_t(group_stride >> 4) << 32;
  d |= uint64_t(1) << 46;
  return d;
}
// Instruction descriptor of the block-scaled MMA: A = E2M1, B = E4M3, E8M0 scales, both operands K-major,
// D is 128 x n; sf_id selects which of the four scale bytes of a tensor-memory column this MMA uses.
__device__ __forceinline__ uint32_t umma_idesc_mx_e2m1_e4m3(uint32_t n, uint32_t a_sf_id, uint32_t b_sf_id) {
  return (b_sf_id << 4) | (5u << 7) | (0u << 10) | ((n >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) |
         (a_sf_id << 29);
}
// The same with an E4M3 A operand (FP8 weights).
__device__ __forceinline__ uint32_t umma_idesc_mx_e4m3_e4m3(uint32_t n, uint32_t a_sf_id, uint32_t b_sf_id) {
  return (b_sf_id << 4) | (0u << 7) | (0u << 10) | ((n >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) |
         (a_sf_id << 29);
}
// Instruction descriptor: E4M3 x E4M3 -> FP32, both operands K-major, D is 128 x n.
__device__ __forceinline__ uint32_t umma_idesc_e4m3(uint32_t n) {
  return (1u << 4) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
#endif  // __CUDACC__

}  // namespace zq
