// Pieces shared by the two W4A8 GEMM kernel families (the one that casts FP4 to FP8 on the CUDA cores and
// the one that hands FP4 tiles and power-of-two block scales to the tensor core): work partition, the
// split-K hand-over, the epilogue arithmetic of Section 3 (token scale x channel scale x accumulator plus
// the LoRC term) and the tensor-map helper.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "zq_common.cuh"

namespace zq {
namespace gemm {

constexpr int kTileN = 128;   // output channels per CTA (MMA M extent)
constexpr int kBlockK = 128;  // K elements per pipeline step
constexpr int kAStageCols = kBlockK / 4;  // TMEM columns of one widened 128 x 128 tile (4 bytes per column)

// error detail codes written to status[1]
enum {
  kErrProducer = 1, kErrWiden = 2, kErrMma = 3, kErrEpilogue = 4, kErrPromote = 5, kErrAlign = 6, kErrHandover = 7,
  kErrGridWait = 8  // the quantizer inside the block-scaled kernel gave up waiting for the other CTAs' shares
};

// Scratch of the quantizer that runs inside the block-scaled kernel, part of the workspace head.  Every launch
// finds it zero and leaves it zero.
struct FusedScratch {
  unsigned int arrived_absmax;  // CTAs whose share of the tokens' absmax / LoRC sums is in
  unsigned int arrived_codes;   // CTAs whose share of the E4M3 codes is written
  unsigned int departed;        // CTAs that have finished; the last one clears the scratch
  unsigned int pad;
  // Atomics of many CTAs on one address are served one after the other (224 K blocks on one word took about
  // 10 us), so K block kb adds into copy kb % kFusedSlots and the readers combine the copies.
  unsigned int amax_bits[kFusedSlots][kFusedMaxTokens];   // per token: max |x| as FP32 bits (non-negative floats order like integers)
  float t[kFusedSlots][kFusedMaxTokens * kFusedMaxRank];  // per token: t = V x, [m][r] token-major, accumulated with atomics
  float t_sum[kFusedMaxTokens * kFusedMaxRank];           // the copies of t added up (by CTA 0, between the two meetings)
};
static_assert(sizeof(FusedScratch) <= kWsFusedBytes, "the scratch must fit its part of the workspace head");

struct Params {
  int M, N, K;
  int G;             // groups per row
  int group;
  int kblocks;       // K blocks per output tile
  int n_tiles, tiles;  // output tiles along N, and in total (tile index = m_tile * n_tiles + n_tile)
  // Work is counted in units of one K block of one output tile, unit u = tile * kblocks + kb.  A CTA
  // owns the contiguous units [u0, u1) and walks them as segments (one per output tile it touches):
  //   stream == 0: CTA c = z * tiles + tile owns K blocks [z * kb_per_split, ...) of that tile
  //   stream == 1: the units of all tiles are dealt out evenly, base (+1 for the first rem CTAs) each
  int stream;
  int persist;   // CTAs walk whole tiles, every gridDim.x-th position of the launch order (block-scaled kernel),
                 // up to position tail_pos0; the tiles from there on are dealt out as unit ranges like stream == 1
  int tail_pos0;
  int dealt0;    // first unit of the units that are dealt out as ranges (0 when stream == 1)
  int m_group;   // the launch order runs through groups of this many token tiles (see raster_tile)
  int atomic_y;  // streaming launch with FP32 y: CTAs that share a tile add their share into a zeroed y
  int handover;  // cooperative launch: shared FP32 tiles are handed over through per-tile flags (one CTA stores,
                 // the others wait for its flag and add), so y needs no clearing
  int splits, kb_per_split;
  int base, rem;
  const uint8_t* codes;  // tiled weight
  const float* scale;
  const float* sx;
  const __half* U;
  const float* t;
  int r;
  void* y;
  int ydt;
  int64_t ldy;
  int* status;
  int* counters;
  float* partials;
  int cast_e5m2;  // the kernel that casts: E5M2 instead of E4M3 as the cast target
  // the block-scaled kernel with the quantizer inside: raw activations, LoRC down-projection matrix, where the
  // codes go (the buffer the token tensor map reads), and the scratch the CTAs meet in
  const __nv_bfloat16* x;
  int64_t ldx;
  const __half* V;
  uint8_t* q_out;
  FusedScratch* fq;
  // fusion on the output side (see GemmArgs)
  int relu;
  float* y_amax;
};

constexpr int cmin(int a, int b) { return a < b ? a : b; }

#ifdef __CUDACC__
__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

__device__ __forceinline__ void raise_error(const Params& p, volatile int* abort_flag, int detail) {
  *abort_flag = 1;
  if (atomicCAS(p.status, 0, ZQ_ERR_DEVICE_TIMEOUT) == 0) p.status[1] = detail;
}

// Launch order -> output tile.  CTAs that run at the same time should share operands in L2: numbering
// them along N alone makes one wave read 148 different weight tiles against one token tile, and the whole
// weight streams from HBM once per token tile.  Numbering through groups of m_group token tiles (N
// outer, the group's token tiles inner) lets a wave share m_group token tiles and 1 / m_group as many
// weight tiles, so the weight streams once per group.
__device__ __forceinline__ int raster_tile(const Params& p, int idx) {
  if (p.m_group <= 1) return idx;
  const int per_group = p.m_group * p.n_tiles;
  const int g = idx / per_group, within = idx - g * per_group;
  const int gm = min(p.m_group, p.tiles / p.n_tiles - g * p.m_group);  // the last group may be smaller
  return (g * p.m_group + within % gm) * p.n_tiles + within / gm;
}

__device__ __forceinline__ int range_start(const Params& p, int c) { return c * p.base + min(c, p.rem); }
__device__ __forceinline__ int cta_of_unit(const Params& p, int u) {
  const int big = p.rem * (p.base + 1);
  return (u < big || p.base == 0) ? u / (p.base + 1) : p.rem + (u - big) / p.base;
}
// The CTAs that contribute partial sums to `tile`: first CTA and their number.
__device__ __forceinline__ void contributors(const Params& p, int tile, int* first, int* count) {
  if (p.stream || p.persist) {
    const int u = tile * p.kblocks - p.dealt0;
    *first = cta_of_unit(p, u);
    *count = cta_of_unit(p, u + p.kblocks - 1) - *first + 1;
  } else {
    *first = 0;
    *count = p.splits;
  }
}
// Workspace slot of the partial sum that contributor j (CTA first + j) leaves for `tile`.  A CTA with a
// dealt-out range can leave two (for the tile its range starts in and for the one it ends in).
__device__ __forceinline__ size_t partial_slot(const Params& p, int tile, int first, int j) {
  if (!(p.stream || p.persist)) return static_cast<size_t>(tile) * p.splits + j;
  const int c = first + j;
  return 2 * static_cast<size_t>(c) + ((p.dealt0 + range_start(p, c)) / p.kblocks == tile ? 0 : 1);
}

// Final arithmetic of NC consecutive tokens (tile columns c0 .. c0+NC-1) of one output channel, and the store.
//   y[m, n] = sx[m] * cs * acc + sum_j t[m, j] * U[n, j]
// s_sx holds the tile's token scales and s_tT its rank-8 LoRC rows, transposed ([j][BM]) so that two
// neighbouring tokens' t values sit side by side: tokens are finished in pairs with packed FP32
// instructions.  u2 holds the channel's U row, each value in both halves, when r == 8 (the common rank);
// other ranks read t and U through the cache.
// `add`: y was zeroed by the launcher and this CTA holds only part of the K range, so it adds (FP32 atomics,
// order-dependent in the last bit); `lorc`: this CTA is the one that contributes the LoRC term.
// `store_ok` == false: the channel lies beyond N; the thread is here only for the warp-wide maximum of p.y_amax.
template <int NC, int BM>
__device__ __forceinline__ void finalize(const Params& p, const float* v, int m0, int c0, int n, float cs,
                                         const uint64_t* u2, const float* __restrict__ s_sx,
                                         const float* __restrict__ s_tT, bool add = false, bool lorc = true,
                                         bool store_ok = true) {
  // All NC results are computed before the first store, so that the columns' loads and FMA chains
  // interleave instead of running one column at a time behind each store.
  static_assert(NC % 4 == 0, "columns are taken four at a time");
  uint64_t o2[NC / 2];
  const uint64_t cs2 = pack2(cs, cs);
#pragma unroll
  for (int c = 0; c < NC; c += 4) {
    const float4 s4 = *reinterpret_cast<const float4*>(s_sx + c0 + c);
    o2[c / 2] = mul2(mul2(pack2(s4.x, s4.y), cs2), pack2(v[c], v[c + 1]));
    o2[c / 2 + 1] = mul2(mul2(pack2(s4.z, s4.w), cs2), pack2(v[c + 2], v[c + 3]));
  }
  if (lorc && p.r == 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int c = 0; c < NC; c += 4) {
        const float4 t4 = *reinterpret_cast<const float4*>(s_tT + j * BM + c0 + c);
        o2[c / 2] = fma2(pack2(t4.x, t4.y), u2[j], o2[c / 2]);
        o2[c / 2 + 1] = fma2(pack2(t4.z, t4.w), u2[j], o2[c / 2 + 1]);
      }
    }
  }
  float out[NC];
#pragma unroll
  for (int c = 0; c < NC; c += 2) unpack2(o2[c / 2], out[c], out[c + 1]);
  if (lorc && p.r > 0 && p.r != 8) {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const int m = m0 + c0 + c;
      if (m < p.M) {
        const float* tr = p.t + static_cast<int64_t>(m) * p.r;
        const __half* ur = p.U + static_cast<int64_t>(n) * p.r;
        // t may have been accumulated by this very launch (quantizer inside the kernel): read it through L2
        for (int j = 0; j < p.r; ++j) out[c] = fmaf(__ldcg(tr + j), __half2float(__ldg(ur + j)), out[c]);
      }
    }
  }
  if (p.relu && !add) {
#pragma unroll
    for (int c = 0; c < NC; ++c) out[c] = fmaxf(out[c], 0.0f);
  }
  if (p.y_amax != nullptr && !add) {
    // Per-token max |y| over this warp's 32 channels, of the values as they are stored (rounding to bf16 is
    // monotone, so it commutes with the maximum).  Non-negative floats order like their bit patterns: one
    // warp-wide integer maximum per token; lane c keeps token c's.  The running maxima settle after the first few
    // channel tiles, so each lane first looks at what is there (a stale value only costs a redundant atomic) and
    // adds its token's maximum in only if it is larger.  Every lane of the warp is here (a channel beyond N comes
    // with store_ok == false and counts as zero).
    static_assert(NC <= 32, "one lane per token of the step");
    const int lane = threadIdx.x & 31;
    const int m_mine = m0 + c0 + lane;
    unsigned int* slot = reinterpret_cast<unsigned int*>(p.y_amax) + m_mine;
    const bool mine_ok = lane < NC && m_mine < p.M;
    const unsigned int seen = mine_ok ? __ldcg(slot) : 0xFFFFFFFFu;
    unsigned int mine = 0u;
    if (p.ydt == ZQ_OUT_F32) {
      const unsigned int keep = store_ok ? 0x7FFFFFFFu : 0u;  // drops the sign
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const unsigned int bits = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(out[c]) & keep);
        if (lane == c) mine = bits;
      }
    } else {
      // the bf16 value's magnitude is the upper half of its FP32 pattern
      const unsigned int keep = store_ok ? 0x7FFFu : 0u;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const unsigned int h = __bfloat16_as_ushort(__float2bfloat16_rn(out[c]));
        const unsigned int bits = __reduce_max_sync(0xFFFFFFFFu, h & keep);
        if (lane == c) mine = bits << 16;
      }
    }
    if (mine_ok && mine > seen) atomicMax(slot, mine);
  }
  if (!store_ok) return;
  const int64_t base = static_cast<int64_t>(m0 + c0) * p.ldy + n;
  if (add) {
    float* y = static_cast<float*>(p.y) + base;
#pragma unroll
    for (int c = 0; c < NC; ++c)
      if (m0 + c0 + c < p.M) atomicAdd(y + c * p.ldy, out[c]);
  } else if (p.ydt == ZQ_OUT_F32) {
    float* y = static_cast<float*>(p.y) + base;
#pragma unroll
    for (int c = 0; c < NC; ++c)
      if (m0 + c0 + c < p.M) y[c * p.ldy] = out[c];
  } else {
    __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.y) + base;
#pragma unroll
    for (int c = 0; c < NC; ++c)
      if (m0 + c0 + c < p.M) y[c * p.ldy] = __float2bfloat16_rn(out[c]);
  }
}

template <int NC>
__device__ __forceinline__ void tmem_ld_issue(uint32_t taddr, float* v) {
  if (NC == 16) tmem_ld16(taddr, v);
  else if (NC == 8) tmem_ld8(taddr, v);
  else tmem_ld4(taddr, v);
}
template <int NC>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float* v) {
  tmem_ld_issue<NC>(taddr, v);
  tmem_ld_wait();
}

#endif  // __CUDACC__

// ---- host ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  });
  return fn;
}

// 2-D u8 tensor [rows, row_bytes] -> tiles of box_rows x box_bytes, written to shared memory swizzled.
inline bool make_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_bytes,
              uint32_t box_rows, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {box_bytes, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline Params make_params(const GemmArgs& a, const GemmPlan& plan) {
  Params p{};
  p.M = static_cast<int>(a.M);
  p.N = static_cast<int>(a.N);
  p.K = static_cast<int>(a.K);
  p.group = a.group;
  p.G = static_cast<int>(a.K / a.group);
  p.kblocks = static_cast<int>(a.K / kBlockK);
  p.n_tiles = plan.n_tiles;
  p.tiles = plan.n_tiles * plan.m_tiles;
  p.stream = plan.stream;
  p.persist = plan.persist;
  p.tail_pos0 = plan.tail_pos0;
  p.dealt0 = plan.persist ? plan.tail_pos0 * p.kblocks : 0;
  p.m_group = plan.m_group;
  p.relu = a.relu;
  p.y_amax = a.y_amax;
  p.atomic_y = (plan.stream && a.ydt == ZQ_OUT_F32 && plan.partial_floats > 0 && !a.relu && !a.y_amax) ? 1 : 0;
  p.splits = plan.splits;
  p.kb_per_split = plan.kb_per_split;
  p.base = plan.base;
  p.rem = plan.rem;
  p.codes = a.codes;
  p.scale = a.scale;
  p.sx = a.sx;
  p.U = static_cast<const __half*>(a.U);
  p.t = a.t;
  p.r = a.U ? a.r : 0;
  p.y = a.y;
  p.ydt = a.ydt;
  p.ldy = a.ldy;
  p.status = a.status;
  p.counters = a.counters;
  p.partials = a.partials;
  p.x = static_cast<const __nv_bfloat16*>(a.x);
  p.ldx = a.ldx;
  p.V = static_cast<const __half*>(a.V);
  p.q_out = const_cast<uint8_t*>(a.q);
  p.fq = static_cast<FusedScratch*>(a.fused_scratch);
  return p;
}

}  // namespace gemm
}  // namespace zq
