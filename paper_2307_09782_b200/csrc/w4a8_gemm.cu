// W4A8 GEMM: y = sx * scale * (Q_fp8(x) . cast_fp8(W_fp4)^T) + t U^T        (Section 3)
//
// The cast FP4 -> FP8 (Section 3, "Casting the FP4 to FP8") runs inside the kernel as an exponent
// shift.  One bulk copy per K block stages a packed E2M1 tile (codes + its shift bytes, contiguous in
// HBM) in shared memory; CUDA cores expand each nibble to an E4M3 byte through an 8-entry
// byte-permute table whose entries already carry the group's shift and write the widened row
// straight into TENSOR MEMORY, from where tcgen05 MMAs (kind::f8f6f4, E4M3 x E4M3, FP32
// accumulators, also in TMEM) take it as their A operand.  Token tiles arrive by TMA and are the
// shared-memory B operand.  The widened weights never touch shared memory.
//
// Orientation: the weight tile is the MMA's 128-row operand (D rows = output channels n, one TMEM
// lane each), the token tile is the N-extent operand (D columns = tokens m, BM of them).  That keeps
// the widening work per tile fixed at 128 x 128 codes per K block whatever the token count, lets one
// kernel serve decode (BM = 16) and prefill (BM = 256), makes "thread = output channel" the natural
// mapping for widening (a thread writes its own TMEM lane) and turns every per-channel quantity
// (scale, shift, U row, group scale) into a per-thread scalar in the epilogue.
//
// Three rings, each as deep as its own resource allows, because the copy -> widen -> MMA -> release
// chain is several K blocks long and each resource is held for a different part of it:
//   P  packed weight tiles in shared memory   producer -> widen warps     (released by the widen warps)
//   T  token tiles in shared memory           producer -> MMA             (released by tcgen05.commit)
//   A  widened weight tiles in tensor memory  widen warps -> MMA          (released by tcgen05.commit)
//
// Warp roles (NG widen groups):
//   0 .. 4NG-1   widen groups of four warps (one warp per TMEM lane quarter); group g widens the K
//                blocks i with i % NG == g, so NG K blocks are in flight and the hand-off latencies
//                overlap.  M1/M2: the same warps run the epilogue (group g takes 1/NG of the columns).
//   4NG          packed-weight producer (bulk copies, one lane)
//   4NG+1        token producer (TMA, one lane)
//   4NG+2        TMEM allocation, MMA issue (one lane)
//   4NG+3 .. +6  mode none only: per-group promotion (TMEM -> registers, times the FP32 group scale)
//                and the epilogue
// Ring depths NP and NA are multiples of NG, so a P or A stage is always handled by the same widen
// group; that group then sees every round of the stage's barriers, which a parity wait needs.
#include "w4a8_gemm_shared.cuh"

namespace zq {
namespace {

using namespace gemm;

template <int BM, bool NONE>
struct Cfg {
  // CTAs per SM this configuration is sized for.  Decode tiles run three small CTAs per SM, so that one
  // CTA's start-up and per-tile epilogue overlap the others' main loops.
  static constexpr int kMinBlocks = (NONE || BM > 128) ? 1 : (BM <= 16 ? 3 : 2);
  static constexpr int NG = kMinBlocks == 3 ? 1 : 2;  // widen groups
  static constexpr int kWidenWarps = 4 * NG;
  static constexpr int kWeightWarp = kWidenWarps;
  static constexpr int kTokenWarp = kWidenWarps + 1;
  static constexpr int kMmaWarp = kWidenWarps + 2;
  static constexpr int kPromoteWarp0 = kWidenWarps + 3;  // mode none: four promotion / epilogue warps
  static constexpr int kThreads = 32 * (kWidenWarps + 3 + (NONE ? 4 : 0));
  static constexpr int kTokBytes = BM * kBlockK;
  static constexpr int kDCols = NONE ? 2 * BM : BM;                 // accumulator columns (two buffers in mode none)
  static constexpr int kDColsPad = kDCols < 32 ? 32 : kDCols;
  static constexpr int kTmemCols = kMinBlocks == 1 ? 512 : (kMinBlocks == 2 ? 256 : 128);
  // Small token tiles (decode) tie the three rings into one: a stage holds the packed tile, the
  // 2-8 KB token tile and the TMEM stage, is filled by one producer and released by one tcgen05.commit,
  // so the MMA warp waits once and commits once per K block (its loop is what bounds a decode CTA).
  static constexpr bool kTied = !NONE && BM >= 32 && BM <= 64;
  static constexpr int NA = cmin(8, (kTmemCols - kDColsPad) / kAStageCols) / NG * NG;  // widened stages in TMEM
  // shared memory: token stages first (as many as the chain needs, at most 10), the rest to packed stages
  static constexpr int kBudget = (kMinBlocks == 1 ? 220 : (kMinBlocks == 2 ? 104 : 70)) * 1024 - BM * 36 - 512;
  static constexpr int kBoth = cmin(10, kBudget / (kTileBytes + kTokBytes));
  static constexpr int NT = kTied ? cmin(NA, kBoth / NG * NG) : kBoth;
  static constexpr int NP = kTied ? NT : cmin(12, (kBudget - NT * kTokBytes) / kTileBytes) / NG * NG;
  static_assert(!kTied || (NT == NA && NP == NA), "tied rings share one depth");
  static constexpr int kEpiThreads = NONE ? 128 : 128 * NG;
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr int offTok = 0;
  static constexpr int offPacked = offTok + NT * kTokBytes;
  static constexpr int offSx = offPacked + NP * kTileBytes;   // [BM] token scales
  static constexpr int offT = offSx + BM * 4;                 // [BM][8] LoRC down-projection (rank 8)
  static constexpr int offBars = offT + BM * 32;
  static constexpr int kNumBars = 2 * NP + 2 * NT + 2 * NA + 6;
  static constexpr int offMisc = offBars + kNumBars * 8;
  static constexpr int kSmemBytes = offMisc + 32;
  static_assert(NA >= NG && NP >= NG && NT >= 3 && NA % NG == 0 && NP % NG == 0, "ring depths");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory");
};

// Expand 8 packed E2M1 codes (one 32-bit word of the tile format: magnitude of element i in bits
// 4i .. 4i+2, sign of element b < 4 in bit 8b+7, sign of element 4+b in bit 8b+3) to 8 E4M3 bytes.
// lut_lo / lut_hi hold the E4M3 magnitudes of the 8 E2M1 magnitudes with the group's shift already
// subtracted from their exponent fields.
__device__ __forceinline__ void widen8(uint32_t w, uint32_t lut_lo, uint32_t lut_hi, uint32_t& o0, uint32_t& o1) {
  const uint32_t wm = w & 0x77777777u;
  uint32_t m0, m1;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(m0) : "r"(lut_lo), "r"(lut_hi), "r"(wm));        // selector: low 16 bits
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(m1) : "r"(lut_lo), "r"(lut_hi), "r"(wm >> 16));
  o0 = m0 | (w & 0x80808080u);
  o1 = m1 | ((w << 4) & 0x80808080u);
}

template <int BM, bool NONE>
__global__ void __launch_bounds__(Cfg<BM, NONE>::kThreads, Cfg<BM, NONE>::kMinBlocks)
w4a8_gemm_kernel(const __grid_constant__ CUtensorMap tm_q, const Params p) {
  using C = Cfg<BM, NONE>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* s_tok = smem + C::offTok;
  uint8_t* s_packed = smem + C::offPacked;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offBars);
  uint64_t* p_full = bars;                     // [NP] packed tile landed            (widen warps wait)
  uint64_t* p_empty = p_full + C::NP;          // [NP] packed tile read (4 warps)    (weight producer waits)
  uint64_t* t_full = p_empty + C::NP;          // [NT] token tile landed             (MMA waits)
  uint64_t* t_empty = t_full + C::NT;          // [NT] MMAs that read it done        (token producer waits)
  uint64_t* a_full = t_empty + C::NT;          // [NA] widened tile in TMEM (4 warps) (MMA waits)
  uint64_t* a_empty = a_full + C::NA;          // [NA] MMAs that read it done        (widen warps wait)
  uint64_t* acc_full = a_empty + C::NA;        // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint64_t* drain_bar = acc_full + 4;          // [1]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::offMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::offMisc + 4);
  int* s_last = reinterpret_cast<int*>(smem + C::offMisc + 8);
  float* s_sx = reinterpret_cast<float*>(smem + C::offSx);
  float* s_t = reinterpret_cast<float*>(smem + C::offT);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's units [u0, u1)
  int u0, u1;
  if (p.stream) {
    u0 = range_start(p, blockIdx.x);
    u1 = range_start(p, blockIdx.x + 1);
  } else {
    const int z = blockIdx.x / p.tiles, tile = raster_tile(p, blockIdx.x % p.tiles);
    u0 = tile * p.kblocks + z * p.kb_per_split;
    u1 = min(u0 + p.kb_per_split, (tile + 1) * p.kblocks);
  }
  const int nunits = u1 - u0;
  // all of a CTA's tiles share one token tile (streaming is only used with a single row of tiles)
  const int m0 = ((u0 / p.kblocks) / p.n_tiles) * BM;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::NP; ++i) {
      mbar_init(&p_full[i], 1);
      mbar_init(&p_empty[i], 4);
    }
    for (int i = 0; i < C::NT; ++i) {
      mbar_init(&t_full[i], 1);
      mbar_init(&t_empty[i], 1);
    }
    for (int i = 0; i < C::NA; ++i) {
      mbar_init(&a_full[i], 4);
      mbar_init(&a_empty[i], 1);
    }
    mbar_init(&acc_full[0], 1);
    mbar_init(&acc_full[1], 1);
    // mode none: two buffers, released by the 128 promotion threads; otherwise one accumulator,
    // handed back once per segment by the widen warps (one arrival per warp)
    mbar_init(&acc_empty[0], NONE ? 128 : C::kWidenWarps);
    mbar_init(&acc_empty[1], 128);
    mbar_init(drain_bar, 1);
    *s_abort = 0;
    *s_last = 0;
    fence_mbar_init();
    if ((smem_u32(smem) & 1023u) != 0) raise_error(p, s_abort, kErrAlign);
  }
  if (warp == C::kTokenWarp && lane == 0) prefetch_tensormap(&tm_q);
  if (warp < C::kWidenWarps) {
    // token scales and (rank 8) LoRC rows of this CTA's tokens, for the epilogue
    for (int c = threadIdx.x; c < BM; c += 32 * C::kWidenWarps) s_sx[c] = (m0 + c < p.M) ? __ldg(p.sx + m0 + c) : 0.0f;
    if (p.r == 8)
      for (int c = threadIdx.x; c < BM * 8; c += 32 * C::kWidenWarps)  // transposed: [j][BM]
        s_t[(c & 7) * BM + (c >> 3)] = (m0 + (c >> 3) < p.M) ? __ldg(p.t + static_cast<int64_t>(m0) * 8 + c) : 0.0f;
  }
  if (warp == C::kMmaWarp) tmem_alloc(s_tmem, C::kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_a = tmem_base + C::kDColsPad;  // widened-weight stages follow the accumulators
  const bool ok_start = (*s_abort == 0);

  if (warp == C::kWeightWarp) {
    // ------------------------------------------------------------------ packed-weight producer
    if (ok_start) {  // warp-uniform loop, one elected lane issues the copies
      const bool issuer = elect_one();
      int s = 0, issued = 0;
      uint32_t ph = 0;
      int tile = u0 / p.kblocks, kb = u0 % p.kblocks;
      for (int i = 0; i < nunits; ++i) {
        // tied rings: the stage (packed tile, token tile, TMEM stage) is free once the MMAs of the K block
        // that used it last have completed
        if (!mbar_wait(C::kTied ? &a_empty[s] : &p_empty[s], ph ^ 1, s_abort)) {
          if (issuer) raise_error(p, s_abort, kErrProducer);
          break;
        }
        if (issuer) {
          const uint8_t* src =
              p.codes + (static_cast<int64_t>(tile % p.n_tiles) * p.kblocks + kb) * kTileBytes;
          mbar_arrive_expect_tx(&p_full[s], C::kTied ? kTileBytes + C::kTokBytes : kTileBytes);
          bulk_load(s_packed + s * kTileBytes, src, kTileBytes, &p_full[s]);
          if (C::kTied) tma_load_2d(s_tok + s * C::kTokBytes, &tm_q, kb * kBlockK, m0, &p_full[s]);
        }
        __syncwarp();
        issued = i + 1;
        if (++kb == p.kblocks) {
          kb = 0;
          ++tile;
        }
        if (++s == C::NP) {
          s = 0;
          ph ^= 1;
        }
      }
      // never leave with copies still in flight: wait (bounded) for the last phase issued per stage
      for (int i = max(0, issued - C::NP); i < issued; ++i) {
        uint32_t spin = 0;
        while (!mbar_try_wait(&p_full[i % C::NP], (i / C::NP) & 1) && ++spin < kSpinLimit) {
        }
      }
    }
  } else if (warp == C::kTokenWarp) {
    // ------------------------------------------------------------------ token producer
    if (ok_start && !C::kTied) {  // warp-uniform loop, one elected lane issues the copies
      const bool issuer = elect_one();
      int s = 0, issued = 0;
      uint32_t ph = 0;
      int kb = u0 % p.kblocks;
      for (int i = 0; i < nunits; ++i) {
        if (!mbar_wait(&t_empty[s], ph ^ 1, s_abort)) {
          if (issuer) raise_error(p, s_abort, kErrProducer);
          break;
        }
        if (issuer) {
          mbar_arrive_expect_tx(&t_full[s], C::kTokBytes);
          tma_load_2d(s_tok + s * C::kTokBytes, &tm_q, kb * kBlockK, m0, &t_full[s]);
        }
        __syncwarp();
        issued = i + 1;
        if (++kb == p.kblocks) kb = 0;
        if (++s == C::NT) {
          s = 0;
          ph ^= 1;
        }
      }
      for (int i = max(0, issued - C::NT); i < issued; ++i) {
        uint32_t spin = 0;
        while (!mbar_try_wait(&t_full[i % C::NT], (i / C::NT) & 1) && ++spin < kSpinLimit) {
        }
      }
    }
  } else if (warp == C::kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the loop (uniform control flow and addresses); one elected lane issues.
    if (ok_start) {
      const bool issuer = elect_one();
      const uint32_t idesc = umma_idesc_e4m3(BM) | (p.cast_e5m2 ? (1u << 7) : 0u);  // A operand E4M3 or E5M2
      const uint64_t bdesc0 = umma_desc_k128(smem_u32(s_tok));
      const int mpg = p.group / 32;  // MMAs per weight group (mode none)
      int mma_count = 0;
      int st = 0, sa = 0;
      uint32_t pht = 0, pha = 0;
      int kb = u0 % p.kblocks, seg = 0;
      bool seg_first = true;  // the next K block starts a segment (a new accumulation)
      bool failed = false;
      for (int i = 0; i < nunits && !failed; ++i) {
        // tied rings: the widen warps saw the stage's barrier (which counts both copies) complete before
        // they arrived on a_full, so this one wait also orders the token tile before the MMAs
        if (!mbar_wait(&a_full[sa], pha, s_abort) || (!C::kTied && !mbar_wait(&t_full[st], pht, s_abort))) {
          failed = true;
          break;
        }
        if (!NONE && seg_first && seg > 0) {
          // the epilogue of the previous segment must have read the accumulator
          if (!mbar_wait(&acc_empty[0], (seg - 1) & 1, s_abort)) {
            failed = true;
            break;
          }
        }
        tc_fence_after_sync();
        const uint32_t a_addr = tmem_a + sa * kAStageCols;
        const uint64_t bdesc = bdesc0 + static_cast<uint64_t>((st * C::kTokBytes) >> 4);
#pragma unroll
        for (int k = 0; k < kBlockK / 32; ++k) {
          uint32_t d_tmem = tmem_base;
          uint32_t accumulate = (!seg_first || k > 0) ? 1u : 0u;
          if (NONE) {
            const int grp = mma_count / mpg, within = mma_count % mpg, b = grp & 1;
            if (within == 0) {
              if (!mbar_wait(&acc_empty[b], ((grp >> 1) & 1) ^ 1, s_abort)) {
                failed = true;
                break;
              }
              tc_fence_after_sync();
            }
            d_tmem = tmem_base + b * BM;
            accumulate = within > 0 ? 1u : 0u;
          }
          if (issuer) umma_f8_tmem_a(d_tmem, a_addr + 8 * k, bdesc + 2 * k, idesc, accumulate);
          ++mma_count;
          if (NONE && (mma_count % mpg) == 0 && issuer) umma_commit(&acc_full[((mma_count / mpg) - 1) & 1]);
        }
        if (failed) break;
        const bool seg_last = (kb + 1 == p.kblocks) || (i + 1 == nunits);
        if (issuer) {
          if (!C::kTied) umma_commit(&t_empty[st]);
          umma_commit(&a_empty[sa]);
          if (!NONE && seg_last) umma_commit(&acc_full[seg & 1]);
        }
        __syncwarp();
        seg_first = seg_last;
        if (seg_last) ++seg;
        if (++kb == p.kblocks) kb = 0;
        if (++st == C::NT) {
          st = 0;
          pht ^= 1;
        }
        if (++sa == C::NA) {
          sa = 0;
          pha ^= 1;
        }
      }
      if (failed) {
        if (issuer) {
          raise_error(p, s_abort, kErrMma);
          umma_commit(drain_bar);  // let the MMAs already issued finish before TMEM is released
        }
        uint32_t spin = 0;
        while (!mbar_try_wait(drain_bar, 0) && ++spin < kSpinLimit) {
        }
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ widen / promote / epilogue
    const int q4 = warp & 3;         // TMEM lane quarter of this warp
    const int row = q4 * 32 + lane;  // output channel within the tile = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const bool widen_role = warp < C::kWidenWarps;
    const bool epi_role = NONE ? (warp >= C::kPromoteWarp0) : true;
    const int grp = warp >> 2;  // widen group (widen warps only)
    bool failed = !ok_start;

    // ring positions of this widen group: stages grp, grp + NG, ... (NP and NA are multiples of NG)
    int wi = grp, sp = grp, sa = grp;
    uint32_t php = 0, pha = 0;

    const int part = NONE ? 0 : grp;  // which share of the columns this widen group finishes
    constexpr int kMyCols = NONE ? BM : (BM / C::NG >= 16 ? BM / C::NG : 16);
    // Mode none keeps its running sums in a register array, which needs the column loop unrolled; the
    // other modes keep the loop rolled so that its body stays resident in the instruction cache.
    constexpr int kEpiUnroll = NONE ? kMyCols / 16 : 1;
    // Columns per epilogue step.  A decode CTA runs its epilogue once or twice, on code that is cold in the
    // instruction cache, so there the body is kept to four columns; larger tiles reuse the body many times
    // (eight columns where two CTAs share an SM and registers are scarcer).
    constexpr int EC = NONE ? 16 : (BM <= 32 ? 4 : (BM <= 128 ? 8 : 16));
    const int col0 = NONE ? 0 : part * kMyCols;
    const bool has_cols = NONE ? true : (col0 < BM);
    const uint32_t t_lane = tmem_base + lane_base;

    // Every thread walks every segment and executes the same named-barrier sequence whether or not it
    // has failed, so a bounded wait that ran out can never leave others stuck at a hardware barrier.
    int seg = 0;
    for (int us = u0; us < u1; ++seg) {
      const int tile = us / p.kblocks;
      const int ue = min(u1, (tile + 1) * p.kblocks);
      const int n0 = (tile % p.n_tiles) * kTileN;
      const int n = n0 + row;
      const bool n_ok = n < p.N;

      if (widen_role) {
        // A lane widens whole rows: 64 packed bytes -> 128 E4M3 bytes = 32 TMEM columns of its own lane.
        for (; wi < ue - u0 && !failed; wi += C::NG) {
          // tied rings: the producer refilled the stage only after the MMAs that read its TMEM half were done
          if (!mbar_wait_warp(&p_full[sp], php, s_abort) ||
              (!C::kTied && !mbar_wait_warp(&a_empty[sa], pha ^ 1, s_abort))) {
            raise_error(p, s_abort, kErrWiden);
            failed = true;
            break;
          }
          tc_fence_after_sync();
          const uint8_t* tile_s = s_packed + sp * kTileBytes;
          uint4 pk[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) pk[c] = *reinterpret_cast<const uint4*>(tile_s + (c * kTileRows + row) * 16);
          // the tile carries its shift bytes (zero in mode none): one per row and 64-element half
          const uint32_t d2 = NONE ? 0u : *reinterpret_cast<const uint16_t*>(tile_s + kTileCodeBytes + 2 * row);
          uint32_t w[32];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t d = (d2 >> (8 * h)) & 0xFFu;
            // the magnitudes 0, 0.5, 1, 1.5 | 2, 3, 4, 6 as E4M3 bytes (exponent field from bit 3) or as E5M2
            // bytes (from bit 2), the shift subtracted from the exponent field of every non-zero entry
            const uint32_t lut_lo = p.cast_e5m2 ? 0x3E3C3800u - d * 0x04040400u : 0x3C383000u - d * 0x08080800u;
            const uint32_t lut_hi = p.cast_e5m2 ? 0x46444240u - d * 0x04040404u : 0x4C484440u - d * 0x08080808u;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              const uint4 v = pk[2 * h + c];
              uint32_t* o = w + (2 * h + c) * 8;
              widen8(v.x, lut_lo, lut_hi, o[0], o[1]);
              widen8(v.y, lut_lo, lut_hi, o[2], o[3]);
              widen8(v.z, lut_lo, lut_hi, o[4], o[5]);
              widen8(v.w, lut_lo, lut_hi, o[6], o[7]);
            }
          }
          // every lane's loads of the packed tile have been consumed: hand the stage back
          __syncwarp();
          if (!C::kTied && lane == 0) mbar_arrive(&p_empty[sp]);
          const uint32_t dst = tmem_a + sa * kAStageCols + lane_base;
          tmem_st16(dst, w);
          tmem_st16(dst + 16, w + 16);
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&a_full[sa]);
          sp += C::NG;
          if (sp >= C::NP) {
            sp -= C::NP;
            php ^= 1;
          }
          sa += C::NG;
          if (sa >= C::NA) {
            sa -= C::NA;
            pha ^= 1;
          }
        }
      }

      // ---- accumulators -> registers -> y (or -> workspace, when other CTAs share the tile)
      if (epi_role) {
        float cs = 1.0f;
        uint64_t u[8];  // the channel's U row, each value in both halves of a packed pair
#pragma unroll
        for (int e = 0; e < 8; ++e) u[e] = 0ull;
        if (!NONE && n_ok) cs = __ldg(p.scale + n);
        if (p.r == 8 && n_ok) {
          const uint4 h = __ldg(reinterpret_cast<const uint4*>(p.U + static_cast<int64_t>(n) * 8));
          const uint32_t hw[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __half2 h2;
            *reinterpret_cast<uint32_t*>(&h2) = hw[e];
            const float2 f = __half22float2(h2);
            u[2 * e] = pack2(f.x, f.x);
            u[2 * e + 1] = pack2(f.y, f.y);
          }
        }

        float run[NONE ? BM : 1];
        if (NONE) {
          // per-group promotion: run += S[n, g] * (this group's FP32 partial sum)
#pragma unroll
          for (int c = 0; c < BM; ++c) run[c] = 0.0f;
          const int kb_first = us % p.kblocks;
          const int groups = ((ue - us) * kBlockK) / p.group;
          const int g0 = (kb_first * kBlockK) / p.group;
          const float* srow = n_ok ? p.scale + static_cast<int64_t>(n) * p.G : nullptr;
          float S_next = (srow && groups > 0) ? __ldg(srow + g0) : 0.0f;
          for (int g = 0; g < groups && !failed; ++g) {
            const int b = g & 1;
            const float S = S_next;
            if (srow && g + 1 < groups) S_next = __ldg(srow + g0 + g + 1);
            if (!mbar_wait_warp(&acc_full[b], (g >> 1) & 1, s_abort)) {
              raise_error(p, s_abort, kErrPromote);
              failed = true;
              break;
            }
            tc_fence_after_sync();
#pragma unroll
            for (int c = 0; c < BM; c += 16) {
              float v[16];
              tmem_ld16(t_lane + b * BM + c, v);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 16; ++e) run[c + e] = fmaf(S, v[e], run[c + e]);
            }
            tc_fence_before_sync();
            mbar_arrive(&acc_empty[b]);
          }
        } else if (!failed) {
          if (!mbar_wait_warp(&acc_full[seg & 1], (seg >> 1) & 1, s_abort)) {
            raise_error(p, s_abort, kErrEpilogue);
            failed = true;
          }
          tc_fence_after_sync();
        }

        const bool whole_tile = (ue - us) == p.kblocks;
        if (whole_tile) {
          if (NONE) {
            if (!failed) {
#pragma unroll
              for (int c = 0; c < BM; c += EC)
                if (n_ok || p.y_amax) finalize<EC, BM>(p, run + c, m0, c, n, cs, u, s_sx, s_t, false, true, n_ok);
            }
          } else if (!failed && has_cols) {
            // the next step's accumulator columns are in flight while this step's are finished
            float nxt[EC];
            tmem_ld_issue<EC>(t_lane + col0, nxt);
#pragma unroll 1
            for (int c = 0; c < kMyCols; c += EC) {
              float v[EC];
              tmem_ld_wait_regs<EC>(nxt);
#pragma unroll
              for (int e = 0; e < EC; ++e) v[e] = nxt[e];
              if (c + EC < kMyCols) tmem_ld_issue<EC>(t_lane + col0 + c + EC, nxt);
              if (n_ok || p.y_amax) finalize<EC, BM>(p, v, m0, col0 + c, n, cs, u, s_sx, s_t, false, true, n_ok);
            }
          }
        } else if (!NONE && p.atomic_y) {
          // Several CTAs share this tile and y was zeroed before the launch: every CTA scales its share
          // and adds it; the first contributor also adds the LoRC term.  No fence, ticket or second pass.
          int first, count;
          contributors(p, tile, &first, &count);
          const bool lorc = static_cast<int>(blockIdx.x) == first;
          if (!failed && has_cols) {
#pragma unroll 1
            for (int c = 0; c < kMyCols; c += EC) {
              float v[EC];
              tmem_ld_cols<EC>(t_lane + col0 + c, v);
              if (n_ok) finalize<EC, BM>(p, v, m0, col0 + c, n, cs, u, s_sx, s_t, true, lorc);
            }
          }
        } else {
          // Several CTAs share this tile: leave the raw partial sums in the workspace; the CTA that
          // arrives last adds all of them in contributor order (deterministic) and finishes the tile.
          int first, count;
          contributors(p, tile, &first, &count);
          const int my_j = p.stream ? static_cast<int>(blockIdx.x) - first : static_cast<int>(blockIdx.x) / p.tiles;
          float* my_partial = p.partials + partial_slot(p, tile, first, my_j) * (BM * kTileN);
          if (!failed && has_cols) {
#pragma unroll(kEpiUnroll)
            for (int c = 0; c < kMyCols; c += EC) {
              float v[EC];
              if (NONE) {
#pragma unroll
                for (int e = 0; e < EC; ++e) v[e] = run[c + e];
              } else {
                tmem_ld_cols<EC>(t_lane + col0 + c, v);
              }
#pragma unroll
              for (int e = 0; e < EC; ++e) my_partial[(col0 + c + e) * kTileN + row] = v[e];
            }
          }
          __threadfence();
          named_bar_sync(1, C::kEpiThreads);
          const bool leader = NONE ? (threadIdx.x == 32 * C::kPromoteWarp0) : (threadIdx.x == 0);
          if (leader) {
            const int ticket = (*s_abort) ? -1 : atomicAdd(p.counters + tile, 1);
            *s_last = (ticket == count - 1) ? 1 : 0;
            if (ticket == count - 1) p.counters[tile] = 0;  // ready for the next call
          }
          named_bar_sync(1, C::kEpiThreads);
          if (*s_last && has_cols) {
            __threadfence();
#pragma unroll 1
            for (int c = 0; c < kMyCols; c += EC) {
              float v[EC];
#pragma unroll
              for (int e = 0; e < EC; ++e) v[e] = 0.0f;
              for (int j = 0; j < count; ++j) {
                const float* src =
                    p.partials + partial_slot(p, tile, first, j) * (BM * kTileN) + (col0 + c) * kTileN + row;
#pragma unroll
                for (int e = 0; e < EC; ++e) v[e] += __ldcg(src + e * kTileN);
              }
              if (n_ok || p.y_amax) finalize<EC, BM>(p, v, m0, col0 + c, n, cs, u, s_sx, s_t, false, true, n_ok);
            }
          }
          named_bar_sync(1, C::kEpiThreads);  // s_last is reused by the next segment
        }
        if (!NONE) {
          // the accumulator has been read: the MMA warp may start the next segment
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[0]);
        }
      }
      us = ue;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == C::kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::kTmemCols);
  }
}

// ---- host ------------------------------------------------------------------------------------------

template <int BM, bool NONE>
int launch_cfg(const GemmArgs& a, const GemmPlan& plan, const Params& p, cudaStream_t st) {
  using C = Cfg<BM, NONE>;
  CUtensorMap tm_q;
  if (!make_map(&tm_q, a.q, static_cast<uint64_t>(a.K), static_cast<uint64_t>(a.M), kBlockK, BM,
                CU_TENSOR_MAP_SWIZZLE_128B))
    return ZQ_ERR_CUDA;
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(once, [] {
    attr_err = cudaFuncSetAttribute(w4a8_gemm_kernel<BM, NONE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    C::kSmemBytes);
  });
  if (attr_err != cudaSuccess) return ZQ_ERR_CUDA;
  if (p.atomic_y &&
      cudaMemset2DAsync(a.y, static_cast<size_t>(a.ldy) * 4, 0, static_cast<size_t>(a.N) * 4, static_cast<size_t>(a.M),
                        st) != cudaSuccess)
    return ZQ_ERR_CUDA;
  dim3 grid(static_cast<unsigned>(plan.ctas));
  w4a8_gemm_kernel<BM, NONE><<<grid, C::kThreads, C::kSmemBytes, st>>>(tm_q, p);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // namespace

// SMs of the current device (148 when no device can be asked, e.g. for a host-only size query).
int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      return 148;
  }
  return n;
}

GemmPlan plan_gemm(int64_t M, int64_t N, int64_t K, int mode, int layout, bool allow_pair) {
  GemmPlan pl{};
  const bool mx = layout_is_mx(layout);
  // mode none keeps a tile's running sums in registers: 64 tokens in the kernel that casts, 128 in the block-scaled one
  const int bm_max = (mode == ZQ_SCALE_NONE) ? (mx ? 128 : 64) : 256;
  int bm = 16;
  while (bm < bm_max && bm < M) bm *= 2;
  // the block-scaled kernel also has a 192-token tile, the widest that leaves room for two accumulators:
  // it serves every token count beyond one 256-token tile
  const bool wide = mx && mode != ZQ_SCALE_NONE;  // token tiles beyond 128
  if (wide && (M > 256 || (M > 128 && M <= 192))) bm = 192;
  // 224 tokens still leave room for two accumulators and move fewer shared-memory bytes per flop (the
  // bound of this kernel); taken when the padding of the last tile does not eat the gain
  if (wide && M > 256 && ((M + 223) / 224) * 224 * 20 < ((M + 191) / 192) * 192 * 21 &&
      ((M + 223) / 224) * ((N + kTileN - 1) / kTileN) >= 4 * static_cast<int64_t>(sm_count()))
    bm = 224;
  // long rows: the epilogue is a small share of a tile, and a 256-token tile (one accumulator, no overlap)
  // moves fewer shared-memory bytes per flop
  if (wide && M > 256 && K >= 16384 &&
      ((M + 255) / 256) * ((N + kTileN - 1) / kTileN) >= 4 * static_cast<int64_t>(sm_count()))
    bm = 256;
  pl.bm = bm;
  pl.m_tiles = static_cast<int>((M + bm - 1) / bm);
  pl.n_tiles = static_cast<int>((N + kTileN - 1) / kTileN);
  const int64_t tiles = static_cast<int64_t>(pl.m_tiles) * pl.n_tiles;
  const int kblocks = static_cast<int>(K / kBlockK);
  if (tiles <= 0 || kblocks <= 0) return pl;  // nothing to do: an empty plan (ctas == 0)
  if (wide && allow_pair && bm >= 128 && pl.n_tiles % 2 == 0 && sm_count() >= 2 && tiles <= kWsMaxTiles) {
    // CTA pairs: the two CTAs of a cluster share each token tile (128 or 176 ... 224 tokens, two accumulators) and
    // take two neighbouring channel tiles.  Work is counted in units of one K block of one pair position
    // (token tile x channel-tile pair) and partitioned among the pairs like the single CTAs' below: whole
    // positions in whole rounds where there are at least four rounds, the rest (or everything) dealt out as
    // contiguous unit ranges.  Taken when its padded token columns are at most 15 % more than the single
    // CTAs' (the pairs run about 20 % faster).
    const int64_t pairs = sm_count() / 2, np = pl.n_tiles / 2;
    // The token tile: the width with the least estimated time = rounds the pairs need (whole rounds count in
    // full when the last one is left uneven) x what a round costs (16 KB of codes per K block and CTA plus 64
    // bytes per token: shared-memory bytes, the bound of this kernel).
    GemmPlan best{};
    double best_cost = 0.0;
    for (const int cand : {224, 208, 192, 176, 128}) {
      if (cand == 128 && M > 128) continue;  // 128-token tiles: one row of them only
      GemmPlan pp{};
      pp.pair = 1;
      pp.bm = cand;
      pp.m_tiles = static_cast<int>((M + cand - 1) / cand);
      pp.n_tiles = pl.n_tiles;
      pp.splits = 1;
      pp.kb_per_split = kblocks;
      const int64_t positions = pp.m_tiles * np, punits = positions * kblocks;
      if (pp.m_tiles > 1) {
        const int64_t fit = (int64_t(32) << 20) / (static_cast<int64_t>(cand) * K);
        pp.m_group = static_cast<int>(fit < 1 ? 1 : (fit > 8 ? 8 : fit));
      }
      double rounds;
      if (positions >= 4 * pairs) {
        pp.persist = 1;
        pp.ctas = static_cast<int>(2 * pairs);
        int64_t tail = positions % pairs;
        if ((pairs - tail) * kblocks < 60 * pairs) tail = 0;  // too little to gain: leave the last round uneven
        pp.tail_pos0 = static_cast<int>(positions - tail);
        pp.base = static_cast<int>(tail * kblocks / pairs);
        pp.rem = static_cast<int>(tail * kblocks % pairs);
        rounds = tail > 0 || positions % pairs == 0 ? static_cast<double>(positions) / pairs
                                                    : static_cast<double>((positions + pairs - 1) / pairs);
      } else if (punits >= 8 && punits < (int64_t(1) << 30)) {
        int64_t g = pairs < punits / 4 ? pairs : punits / 4;
        if (g < 1) g = 1;
        pp.stream = 1;
        pp.ctas = static_cast<int>(2 * g);
        pp.base = static_cast<int>(punits / g);
        pp.rem = static_cast<int>(punits % g);
        rounds = static_cast<double>(positions) / g;
      } else {
        continue;
      }
      const double cost = rounds * (256 + cand);
      if (best.pair == 0 || cost < best_cost) {
        best = pp;
        best_cost = cost;
      }
    }
    // taken when its padded token columns are at most 15 % more than the single CTAs' (the pairs run about 20 % faster)
    if (best.pair && static_cast<int64_t>(best.m_tiles) * best.bm * 100 <= static_cast<int64_t>(pl.m_tiles) * bm * 115)
      return best;
  }
  // CTAs per SM the kernel family is sized for at this tile
  // (the block-scaled kernel: always one; its launches with shared tiles are cooperative, and a cooperative
  // launch of a kernel that allocates tensor memory is given one CTA per SM)
  const int ctas_per_sm = mx ? 1 : ((mode == ZQ_SCALE_NONE || bm > 128) ? 1 : (bm <= 16 ? 3 : 2));
  const int64_t resident = static_cast<int64_t>(ctas_per_sm) * sm_count();
  const int64_t units = tiles * kblocks;
  // as many token tiles per group of the launch order as keep the group's tokens around 32 MB (they must
  // stay in L2 while the group walks all of N), at most 8
  if (pl.m_tiles > 1) {
    const int64_t fit = (int64_t(32) << 20) / (static_cast<int64_t>(bm) * K);
    pl.m_group = static_cast<int>(fit < 1 ? 1 : (fit > 8 ? 8 : fit));
  }
  if (mx && ((pl.m_tiles > 1 && (tiles >= 4 * resident || tiles > kWsMaxTiles)) ||
             (pl.m_tiles == 1 && bm >= 128 && tiles >= resident))) {
    // many tokens: one resident wave of CTAs walks whole tiles (with fewer than four tiles per CTA the
    // uneven last round would cost too much: those shapes take the contiguous unit ranges below).  Also one
    // row of wide tiles that fills a resident wave.  (One row of narrow tiles always takes the unit ranges:
    // with one CTA per SM whole tiles would leave a second, half-empty round.)
    pl.persist = 1;
    const int64_t g = tiles < resident ? tiles : resident;
    pl.ctas = static_cast<int>(g);
    pl.splits = 1;
    pl.kb_per_split = kblocks;
    // whole rounds as whole tiles; the tiles of the last, incomplete round as unit ranges over all CTAs
    // (they hand partial sums over through the workspace)
    // ... when that saves more than the shared tiles' extra epilogues cost (about 60 K blocks' time)
    int64_t tail_tiles = tiles <= kWsMaxTiles ? tiles % g : 0;
    if ((g - tail_tiles) * kblocks < 60 * g) tail_tiles = 0;
    pl.tail_pos0 = static_cast<int>(tiles - tail_tiles);
    pl.base = static_cast<int>(tail_tiles * kblocks / g);
    pl.rem = static_cast<int>(tail_tiles * kblocks % g);
    pl.partial_floats = tail_tiles > 0 ? 2 * static_cast<size_t>(g) * bm * kTileN : 0;
    return pl;
  }
  if ((mx || (mode != ZQ_SCALE_NONE && bm == 16 && pl.m_tiles == 1)) && tiles <= kWsMaxTiles && units >= 8 &&
      units < (int64_t(1) << 30)) {
    // At most 16 tokens (decode): the weight streams exactly once and the per-tile epilogue is tiny, so deal
    // the (tile, K block) units out evenly to one resident wave of CTAs, at least 4 units each.  (In the casting
    // kernel wider token tiles measured slower this way: their shared tiles cost more atomics than the wave
    // balance saves.  The block-scaled kernel finishes one tile while it accumulates the next and does this
    // for every single row of tiles.)
    int64_t g = resident < units / 4 ? resident : units / 4;
    if (g < 1) g = 1;
    pl.stream = 1;
    pl.ctas = static_cast<int>(g);
    pl.base = static_cast<int>(units / g);
    pl.rem = static_cast<int>(units % g);
    pl.splits = 1;
    pl.kb_per_split = kblocks;
    // a CTA leaves at most two partial sums (the tile its range starts in and the one it ends in)
    pl.partial_floats = (g == tiles && pl.rem == 0 && pl.base == kblocks) ? 0 : 2 * static_cast<size_t>(g) * bm * kTileN;
    return pl;
  }
  // split K until about one resident wave of CTAs exists, keeping at least 4 K blocks per CTA and (for
  // 256-wide groups) whole groups per CTA
  int splits = 1;
  const int64_t target = static_cast<int64_t>(ctas_per_sm < 2 ? 2 : ctas_per_sm) * sm_count();
  if (tiles < target && tiles <= kWsMaxTiles) {
    splits = static_cast<int>((target + tiles - 1) / tiles);
    const int max_splits = kblocks / 4 > 0 ? kblocks / 4 : 1;
    if (splits > max_splits) splits = max_splits;
  }
  int kbps = (kblocks + splits - 1) / splits;
  if (kbps % 2) ++kbps;  // whole 256-element groups per split
  if (kbps > kblocks) kbps = kblocks;
  splits = (kblocks + kbps - 1) / kbps;
  pl.stream = 0;
  pl.splits = splits;
  pl.kb_per_split = kbps;
  pl.ctas = static_cast<int>(tiles * splits);
  pl.partial_floats = splits > 1 ? static_cast<size_t>(tiles) * splits * bm * kTileN : 0;
  return pl;
}

int launch_w4a8_gemm(const GemmArgs& a, cudaStream_t st) {
  const GemmPlan plan = plan_gemm(a.M, a.N, a.K, a.mode, ZQ_WEIGHTS_CAST);
  if (plan.partial_floats > a.partial_floats) return ZQ_ERR_WORKSPACE;
  Params p = make_params(a, plan);
  p.cast_e5m2 = a.layout == ZQ_WEIGHTS_CAST_E5M2 ? 1 : 0;
  const bool none = a.mode == ZQ_SCALE_NONE;
  switch (plan.bm) {
    case 16: return none ? launch_cfg<16, true>(a, plan, p, st) : launch_cfg<16, false>(a, plan, p, st);
    case 32: return none ? launch_cfg<32, true>(a, plan, p, st) : launch_cfg<32, false>(a, plan, p, st);
    case 64: return none ? launch_cfg<64, true>(a, plan, p, st) : launch_cfg<64, false>(a, plan, p, st);
    case 128: return none ? ZQ_ERR_SHAPE : launch_cfg<128, false>(a, plan, p, st);
    case 256: return none ? ZQ_ERR_SHAPE : launch_cfg<256, false>(a, plan, p, st);
  }
  return ZQ_ERR_SHAPE;
}

}  // namespace zq
