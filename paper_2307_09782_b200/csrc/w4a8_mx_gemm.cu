// W4A8 GEMM with the cast FP4 -> FP8 left to the tensor core:
//   y = sx * scale * (Q_fp8(x) . (E2M1 codes * 2^-shift)^T) + t U^T                      (Section 3)
//
// Section 3 ("Casting the FP4 to FP8") constrains the group scales to powers of two (M1) or to
// power-of-two fractions of a per-channel scale (M2) so that FP4 weights reach the FP8 tensor core
// with a bit shift instead of a multiplication.  This architecture's tensor core takes that step itself: its
// block-scaled MMA (kind::mxf8f6f4) multiplies an E2M1 operand by an E4M3 operand and applies one
// power-of-two (E8M0) scale per row and 32 elements of K, which is exactly the constrained group
// scale 2^-shift.  The kernel therefore moves bytes and issues MMAs; no CUDA core touches a weight.
//
//   weights  one TMA load per pipeline stage brings one (wide token tiles) or two (up to 64 tokens) 128 x 128
//            tiles of packed nibbles (8 KB each, contiguous in HBM) into shared memory, expanded by the copy
//            engine to the tensor core's 16-byte-aligned FP4 form (8 bytes of nibbles, 8 bytes of padding).
//            With few tokens a CTA's rate is bound by the number of copies it issues, not by their bytes
//            (a CTA got through one 8.7 KB copy per 0.3 us whatever the ring depth), hence two K blocks per
//            copy there;
//   scales   the tiles' 512 E8M0 bytes each (contiguous for consecutive K blocks) arrive by one bulk copy
//            and go to tensor memory with tcgen05.cp, issued by the MMA thread right before a tile's four MMAs;
//   tokens   E4M3 tiles by TMA, the shared-memory B operand, with a block scale of one;
//   D        FP32 in tensor memory, two buffers where they fit, so that the epilogue of one output tile
//            overlaps the main loop of the next.
//
// Orientation, the split-K hand-over and the epilogue are those of the casting kernel.  Work partition
// (plan_gemm): few tokens or few tiles: the (tile, K block) units are dealt out evenly as contiguous
// ranges to one resident wave of CTAs; many tokens: one CTA per SM walks whole output tiles of 128
// channels x 192 / 224 tokens (two accumulator buffers in use) or x 256 tokens (long rows, one buffer),
// every gridDim.x-th one of the launch order, and the tiles of the last, incomplete round are dealt out
// as unit ranges again.  Where tiles are shared and y is FP32 the launch is cooperative and a shared tile
// is handed over through a flag: its last contributor stores, the others wait for the flag and add.
//
// What bounds it: with many tokens, shared-memory bandwidth (the copy engine writes, and the tensor core
// reads back, 16 KB of padded codes plus 128 bytes per token per K block); with few tokens, HBM
// latency and the fixed cost of a short kernel, not instruction issue.
//
// Warp roles: 0..3 epilogue (one TMEM lane quarter each), 4 producer (one lane issues all copies of a
// stage onto one barrier), 5 TMEM allocation and MMA issue.
#include "act_cast.cuh"
#include "w4a8_gemm_shared.cuh"

namespace zq {
namespace {

using namespace gemm;

constexpr int kSfbCols = 16;  // token-side block scales (all one): room for 256 tokens, written once

// W8: the weight codes are FP8-E4M3 bytes (layout ZQ_WEIGHTS_MX_FP8) instead of packed E2M1 nibbles: 16 KB per
// tile in HBM, copied as they are (they fill the same 16 KB of shared memory as the padded FP4 form).
// NONE (unconstrained FP32 group scales, Section 3: what M1 / M2 remove): the block scales are all 2^0, the two
// accumulator buffers hold one weight group's partial sum each, the epilogue warps multiply it by the group's
// FP32 scale and add it up in registers while the MMAs of the next group run, and the finished tile goes back to a
// third tensor-memory region, from which the usual epilogue takes it.
template <int BM, bool W8, bool NONE = false>
struct MxCfg {
  static_assert(!NONE || (BM <= 128 && !W8), "mode none: the running sums are BM registers per thread");
  // One CTA per SM: launches whose CTAs share output tiles are cooperative, and a cooperative launch of a
  // kernel that allocates tensor memory is given one CTA per SM (the occupancy query answers 1 whatever the
  // registers and shared memory; with two CTAs per SM planned, grids beyond the SM count were refused).
  static constexpr int kMinBlocks = 1;
  static constexpr int kKps = BM <= 64 ? 2 : 1;  // K blocks per pipeline stage
  static constexpr int kCodeBytes = W8 ? 2 * kTileCodeBytes : kTileCodeBytes;  // a tile's codes in HBM
  static constexpr int kTileBytesHbm = kCodeBytes + kMxTileScaleBytes;
  static constexpr int kProducerWarp = 4;
  static constexpr int kMmaWarp = 5;
  static constexpr int kThreads = 192;
  static constexpr int kEpiThreads = 128;
  static constexpr int kABytes1 = kTileRows * kTileK;  // shared-memory footprint of one code tile (padded FP4)
  static constexpr int kTokBytes1 = BM * kBlockK;
  static constexpr int kABytes = kKps * kABytes1;      // per stage
  static constexpr int kTokBytes = kKps * kTokBytes1;
  static constexpr int kSfBytes = kKps * kMxTileScaleBytes;
  // bytes a stage's barrier counts besides the scales (whole boxes: what lies beyond the tensor is filled
  // with zeros and counted too)
  static constexpr int kStageTxBoxes = kKps * kCodeBytes + kTokBytes;
  static constexpr int kBudget = (kMinBlocks == 1 ? 220 : 110) * 1024 - BM * 36 - 512;
  static constexpr int NS = cmin(12, kBudget / (kABytes + kSfBytes + kTokBytes));
  static constexpr int NB = BM <= 224 ? 2 : 1;  // accumulator buffers
  static constexpr int kDColsPad = BM < 32 ? 32 : BM;
  static constexpr int kResultCol0 = NB * kDColsPad;  // NONE: the finished tile
  static constexpr int kSfaCol0 = (NONE ? NB + 1 : NB) * kDColsPad;
  static constexpr int kSfbCol0 = kSfaCol0 + 4 * kKps * NS;
  static constexpr int kColsUsed = kSfbCol0 + kSfbCols;
  static constexpr int kTmemCols = kColsUsed <= 128 ? 128 : (kColsUsed <= 256 ? 256 : 512);
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr int offA = 0;
  static constexpr int offTok = offA + NS * kABytes;
  static constexpr int offSf = offTok + NS * kTokBytes;
  static constexpr int offSx = offSf + NS * kSfBytes;  // [BM] token scales
  static constexpr int offT = offSx + BM * 4;                   // [8][BM] LoRC down-projection (rank 8)
  static constexpr int offBars = offT + BM * 32;
  static constexpr int kNumBars = 2 * NS + 2 * NB + 1;
  static constexpr int offMisc = offBars + kNumBars * 8;
  static constexpr int kSmemBytes = offMisc + 32;
  static_assert(NS >= 3, "pipeline depth");
  static_assert(kTokBytes1 % 1024 == 0 || kKps == 1, "the second token tile of a stage must start on a swizzle atom");
  static_assert(kTmemCols * kMinBlocks <= 512, "tensor memory");
  static_assert(kSmemBytes * kMinBlocks <= 226 * 1024, "shared memory");
};

// The output-tile segments of one CTA, in the order all three roles walk them.
//   persist: whole tiles, every gridDim.x-th position of the launch order (see raster_tile), so that the CTAs
//            running at one time work on neighbouring tiles; the positions of the last, incomplete round
//            are then dealt out as unit ranges, so that no SM idles through a whole tile's time;
//   stream / split K: the contiguous unit range [us, u1), cut at tile boundaries.
struct Segments {
  int us, u1;
  int idx, step;
  bool persist, pairs;
  // `worker` of `workers`: a CTA of the grid, or (CTA-pair kernel) a pair of the grid's pairs, whose positions
  // are pair positions (see pair_tile) and are handed back as they are
  __device__ __forceinline__ explicit Segments(const Params& p, int worker = static_cast<int>(blockIdx.x),
                                               int workers = static_cast<int>(gridDim.x), bool pair_positions = false) {
    persist = p.persist != 0;
    pairs = pair_positions;
    idx = worker;
    step = workers;
    us = u1 = 0;
    if (p.stream || persist) {
      us = p.dealt0 + range_start(p, worker);
      u1 = p.dealt0 + range_start(p, worker + 1);
    } else {
      const int z = blockIdx.x / p.tiles, pos = blockIdx.x % p.tiles;
      us = pos * p.kblocks + z * p.kb_per_split;
      u1 = min(us + p.kb_per_split, (pos + 1) * p.kblocks);
    }
  }
  // next segment: K blocks [kb0, kb0 + nkb) of the output tile at position `pos` of the launch order,
  // which is tile `tile` (m_tile * n_tiles + n_tile); split-K bookkeeping goes by position
  __device__ __forceinline__ bool next(const Params& p, int& pos, int& tile, int& kb0, int& nkb) {
    if (persist && idx < p.tail_pos0) {
      pos = idx;
      idx += step;
      kb0 = 0;
      nkb = p.kblocks;
    } else {
      // unit range: all of a streaming CTA's work, or its share of the last, incomplete round of a
      // persistent launch
      if (us >= u1) return false;
      pos = us / p.kblocks;
      kb0 = us - pos * p.kblocks;
      const int ue = min(u1, (pos + 1) * p.kblocks);
      nkb = ue - us;
      us = ue;
    }
    tile = pairs ? pos : raster_tile(p, pos);
    return true;
  }
};

// One pipeline stage at a time through a CTA's segments, in the order the MMAs take them: the stage holds
// the K blocks kb .. kb + nk - 1 (nk <= KPS) of the output tile `tile`.
template <int KPS>
struct StageWalker {
  Segments sg;
  int tile = 0, kb = 0, left = 0;
  __device__ __forceinline__ explicit StageWalker(const Segments& s) : sg(s) {}
  __device__ __forceinline__ bool next(const Params& p, int& o_tile, int& o_kb) {
    if (left == 0) {
      int pos, kb0, nkb;
      if (!sg.next(p, pos, tile, kb0, nkb)) return false;
      kb = kb0;
      left = nkb;
    }
    o_tile = tile;
    o_kb = kb;
    const int nk = min(KPS, left);
    kb += nk;
    left -= nk;
    return true;
  }
};

// Thread 0 of a CTA: count this CTA in (if it had a share of the work) and wait, bounded, until `expected`
// CTAs have.  The launch is cooperative, so all of them are running.
__device__ __forceinline__ bool grid_meet(unsigned int* counter, unsigned int expected, bool counts,
                                          volatile int* abort_flag) {
  __threadfence();
  if (counts) atomicAdd(counter, 1u);
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    if (*reinterpret_cast<volatile unsigned int*>(counter) >= expected) {
      __threadfence();
      return true;
    }
    if (*abort_flag) return false;
    if ((spin & 63u) == 63u && global_timer_ns() - t0 > kWaitLimitNs) return false;
  }
  return false;
}

// FUSEQ: the kernel quantizes the activations itself (one tile of at most 16 tokens), so that the layer is one
// launch.  While the producer's first weight copies are on their way, the epilogue warps (idle until the first
// accumulator is due) (1) add their CTA's share of every token's absmax and of the LoRC down-projection
// t = V x into a scratch in which all CTAs meet, (2) once all shares are in, cast their share of x to E4M3
// into the workspace's q buffer, and (3) once all codes are written, release the producer, which loads the
// token tiles from q exactly as it would after a separate quantizer kernel.  The main loop is untouched.
// (Casting the tokens straight into the pipeline stages, by extra warps or by the producer warp, was tried in
// several forms first: each ran the main loop at 0.7 us or more per stage against the 0.39 us of the copies
// alone.)  The two meetings cost about 3 us during which only the ring's first stages stream.
template <int BM, bool W8, bool FUSEQ, bool NONE>
__global__ void __launch_bounds__(MxCfg<BM, W8, NONE>::kThreads, MxCfg<BM, W8, NONE>::kMinBlocks)
w4a8_mx_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_q,
                    const Params p) {
  using C = MxCfg<BM, W8, NONE>;
  static_assert(!NONE || C::NB == 2, "mode none alternates two group accumulators");
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* s_a = smem + C::offA;
  uint8_t* s_tok = smem + C::offTok;
  uint8_t* s_sf = smem + C::offSf;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offBars);
  uint64_t* full = bars;                  // [NS] all three copies of the stage landed   (MMA waits)
  uint64_t* empty = full + C::NS;         // [NS] the MMAs that read the stage are done   (producer waits)
  uint64_t* acc_full = empty + C::NS;     // [NB] a segment's accumulation is complete    (epilogue waits)
  uint64_t* acc_empty = acc_full + C::NB; // [NB] the epilogue has read the buffer        (MMA waits)
  uint64_t* drain_bar = acc_empty + C::NB;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::offMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::offMisc + 4);
  int* s_last = reinterpret_cast<int*>(smem + C::offMisc + 8);
  float* s_sx = reinterpret_cast<float*>(smem + C::offSx);
  float* s_t = reinterpret_cast<float*>(smem + C::offT);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::NS; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < C::NB; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 4);  // one arrival per epilogue warp
    }
    mbar_init(drain_bar, 1);
    *s_abort = 0;
    *s_last = 0;
    fence_mbar_init();
    if ((smem_u32(smem) & 1023u) != 0) raise_error(p, s_abort, kErrAlign);
  }
  if (warp == C::kProducerWarp && lane == 0) {
    prefetch_tensormap(&tm_w);
    prefetch_tensormap(&tm_q);
  }
  if (warp == C::kMmaWarp) tmem_alloc(s_tmem, C::kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_sfa = tmem_base + C::kSfaCol0;
  const uint32_t tmem_sfb = tmem_base + C::kSfbCol0;
  const bool ok_start = (*s_abort == 0);
  if (warp < 4) {
    // the tokens' block scales are all 2^0: fill their columns once (every lane quarter holds a copy)
    uint32_t ones[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) ones[i] = 0x7F7F7F7Fu;
    tmem_st16(tmem_sfb + (static_cast<uint32_t>(warp * 32) << 16), ones);
    tmem_st_wait();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  Segments sg(p);
  int pos, tile, kb0, nkb;
  if (threadIdx.x == 0) pdl_launch_dependents();  // the next kernel of the stream may begin its own setup

  if (warp == C::kProducerWarp) {
    // ------------------------------------------------------------------ producer
    if (ok_start) {  // warp-uniform loops, one elected lane issues the copies
      const bool issuer = elect_one();
      // The copies of one stage.  The boxes always span kKps K blocks (beyond the row's last K block the copy
      // engine fills in zeros; a K block past the end of this CTA's range is read but not used); the scales
      // are copied for the K blocks that exist only, never past the row's end.
      auto issue_weights = [&](int s, int tile_, int kb) {
        if (issuer) {
          const int nt = tile_ % p.n_tiles;
          const uint8_t* sf_row = p.codes + static_cast<int64_t>(nt) * p.kblocks * C::kTileBytesHbm +
                                  static_cast<int64_t>(p.kblocks) * C::kCodeBytes;  // the row block's scales
          const int nsf = min(C::kKps, p.kblocks - kb);
          mbar_arrive_expect_tx(&full[s], C::kStageTxBoxes + nsf * kMxTileScaleBytes);  // the tokens' bytes too
          tma_load_4d(s_a + s * C::kABytes, &tm_w, 0, 0, kb, nt, &full[s]);
          bulk_load(s_sf + s * C::kSfBytes, sf_row + static_cast<int64_t>(kb) * kMxTileScaleBytes,
                    nsf * kMxTileScaleBytes, &full[s]);
        }
      };
      auto issue_tokens = [&](int s, int tile_, int kb) {
        if (issuer) tma_load_3d(s_tok + s * C::kTokBytes, &tm_q, 0, (tile_ / p.n_tiles) * BM, kb, &full[s]);
      };
      int s = 0, issued = 0;
      uint32_t ph = 0;
      bool ok = true;
      StageWalker<C::kKps> w(sg), w_tok(sg);
      int w_tile, w_kb;
      // The weights are the layer's own read-only data: the copies of the first NS stages (all free at the
      // start) go out before the wait for the kernel ahead in the stream, whose output the tokens may be.
      while (issued < C::NS && w.next(p, w_tile, w_kb)) {
        issue_weights(issued, w_tile, w_kb);
        ++issued;
      }
      __syncwarp();
      if (FUSEQ) {
        named_bar_sync(3, C::kEpiThreads + 32);  // every CTA's codes are in q
        asm volatile("fence.proxy.async.global;" ::: "memory");  // written by ordinary stores, read by the copy engine
      } else {
        pdl_wait();
      }
      for (int i = 0; i < issued; ++i) {
        w_tok.next(p, w_tile, w_kb);
        issue_tokens(i, w_tile, w_kb);
      }
      __syncwarp();
      if (issued == C::NS) ph = 1;  // the ring has wrapped once
      while (ok && w.next(p, w_tile, w_kb)) {
        if (!mbar_wait(&empty[s], ph ^ 1, s_abort)) {
          if (issuer) raise_error(p, s_abort, kErrProducer);
          ok = false;
          break;
        }
        issue_weights(s, w_tile, w_kb);
        issue_tokens(s, w_tile, w_kb);
        __syncwarp();
        ++issued;
        if (++s == C::NS) {
          s = 0;
          ph ^= 1;
        }
      }
      // never leave with copies still in flight: wait (bounded) for the last phase issued per stage
      for (int i = max(0, issued - C::NS); i < issued; ++i) {
        uint32_t spin = 0;
        while (!mbar_try_wait(&full[i % C::NS], (i / C::NS) & 1) && ++spin < kSpinLimit) {
        }
      }
    } else if (FUSEQ) {
      named_bar_sync(3, C::kEpiThreads + 32);
    }
  } else if (warp == C::kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the loops (uniform control flow and addresses); one elected lane issues.
    if (ok_start) {
      const bool issuer = elect_one();
      const uint64_t adesc0 = umma_desc_k128(smem_u32(s_a));
      const uint64_t bdesc0 = umma_desc_k128(smem_u32(s_tok));
      const uint64_t sfdesc0 = umma_desc_rows16(smem_u32(s_sf), 128);
      int s = 0, seg = 0;
      uint32_t ph = 0;
      bool failed = false;
      int gcount = 0;  // NONE: weight groups started so far (group g accumulates in buffer g % 2)
      const int mpg = NONE ? p.group / 32 : 1;  // NONE: MMAs (32 elements of K each) per weight group
      while (!failed && sg.next(p, pos, tile, kb0, nkb)) {
        const int buf = seg % C::NB;
        // the epilogue of the segment that used this accumulator buffer last must have read it
        if (!NONE && seg >= C::NB && !mbar_wait(&acc_empty[buf], ((seg / C::NB) - 1) & 1, s_abort)) {
          failed = true;
          break;
        }
        uint32_t d_tmem = tmem_base + buf * C::kDColsPad;
        int gid_prev = -1, gbuf = 0;
        for (int i = 0; i < nkb && !failed; i += C::kKps) {
          const int nk = min(C::kKps, nkb - i);  // K blocks of this stage that belong to the segment
          if (!mbar_wait(&full[s], ph, s_abort)) {
            failed = true;
            break;
          }
          tc_fence_after_sync();
#pragma unroll
          for (int j = 0; j < C::kKps; ++j) {
            if (j < nk && !failed) {
              const uint32_t sfa = tmem_sfa + 4 * (s * C::kKps + j);
              const uint64_t adesc = adesc0 + static_cast<uint64_t>((s * C::kABytes + j * C::kABytes1) >> 4);
              const uint64_t bdesc = bdesc0 + static_cast<uint64_t>((s * C::kTokBytes + j * C::kTokBytes1) >> 4);
              if (issuer)
                tmem_cp_32x128b_x4(sfa, sfdesc0 + static_cast<uint64_t>((s * C::kSfBytes + j * kMxTileScaleBytes) >> 4));
#pragma unroll
              for (int k = 0; k < kBlockK / 32; ++k) {
                uint32_t accumulate = (i > 0 || j > 0 || k > 0) ? 1u : 0u;
                if (NONE) {
                  // a new weight group (by its absolute position in the row) starts a fresh partial sum in the
                  // other buffer, once the epilogue warps have read what that buffer held
                  const int gid = ((kb0 + i + j) * (kBlockK / 32) + k) / mpg;
                  if (gid != gid_prev) {
                    if (gid_prev >= 0 && issuer) umma_commit(&acc_full[gbuf]);
                    gbuf = gcount & 1;
                    if (gcount >= 2 && !mbar_wait(&acc_empty[gbuf], ((gcount >> 1) - 1) & 1, s_abort)) failed = true;
                    tc_fence_after_sync();
                    ++gcount;
                    gid_prev = gid;
                    accumulate = 0u;
                    d_tmem = tmem_base + gbuf * C::kDColsPad;
                  }
                }
                // scale byte k of the K block's four columns belongs to elements 32k .. 32k+31
                if (issuer && !failed)
                  umma_mxf8f6f4(d_tmem, adesc + 2 * k, bdesc + 2 * k,
                                W8 ? umma_idesc_mx_e4m3_e4m3(BM, k, 0) : umma_idesc_mx_e2m1_e4m3(BM, k, 0),
                                sfa + (static_cast<uint32_t>(k) << 30), tmem_sfb, accumulate);
              }
            }
          }
          if (issuer) {
            umma_commit(&empty[s]);
            if (i + C::kKps >= nkb) umma_commit(&acc_full[NONE ? gbuf : buf]);
          }
          __syncwarp();
          if (++s == C::NS) {
            s = 0;
            ph ^= 1;
          }
        }
        ++seg;
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
    // ------------------------------------------------------------------ epilogue
    const int row = warp * 32 + lane;  // output channel within the tile = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    constexpr int EC = BM <= 32 ? 4 : (BM <= 128 ? 8 : 16);  // columns per step
    bool failed = !ok_start;
    int m0_loaded = -1;
    int gcount = 0;  // NONE: weight groups promoted so far
    pdl_wait();  // x, sx, t, the hand-over flags and y may still be in use by the kernel ahead in the stream
    if (FUSEQ) {
      // Section 3 / Appendix A, token-wise: a_m = max_k |x[m,k]|, q = RNE_E4M3(fl32(x * fl32(448 / a_m))), and
      // t = V x with the raw x.  This CTA's share: K blocks blockIdx.x, + gridDim.x, ...; a thread takes 16
      // consecutive elements of token row threadIdx.x / 8 (eight neighbouring lanes share a row).
      FusedScratch* fq = p.fq;
      const int chunk = threadIdx.x & 7, m = threadIdx.x >> 3;
      const bool m_ok = m < p.M;
      const unsigned int sharers = static_cast<unsigned int>(min(static_cast<int>(gridDim.x), p.kblocks));
      const bool has_share = static_cast<int>(blockIdx.x) < p.kblocks;
      // the first two K blocks of the share stay in registers between the two passes
      constexpr int kKeep = 2;
      uint4 xk[kKeep][2];
#pragma unroll
      for (int i = 0; i < kKeep; ++i) {
        const int kb = blockIdx.x + i * gridDim.x;
        xk[i][0] = xk[i][1] = make_uint4(0, 0, 0, 0);
        if (ok_start && m_ok && kb < p.kblocks) {
          const uint4* xp = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(m) * p.ldx + kb * kBlockK) + 2 * chunk;
          xk[i][0] = __ldg(xp);
          xk[i][1] = __ldg(xp + 1);
        }
      }
      if (ok_start) {
        int i = 0;
        for (int kb = blockIdx.x; kb < p.kblocks; kb += gridDim.x, ++i) {
          uint4 x0 = make_uint4(0, 0, 0, 0), x1 = x0;
          if (i == 0) {
            x0 = xk[0][0];
            x1 = xk[0][1];
          } else if (i == 1) {
            x0 = xk[1][0];
            x1 = xk[1][1];
          } else if (m_ok) {
            const uint4* xp = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(m) * p.ldx + kb * kBlockK) + 2 * chunk;
            x0 = __ldg(xp);
            x1 = __ldg(xp + 1);
          }
          const int slot = kb % kFusedSlots;
          float a = absmax8(x1, absmax8(x0, 0.0f));
          a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, 1));
          a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, 2));
          a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, 4));
          if (m_ok && chunk == 0 && a != 0.0f) atomicMax(&fq->amax_bits[slot][m], __float_as_uint(a));
          for (int j0 = 0; j0 < p.r; j0 += 8) {  // p.r is a multiple of 8 (0 without LoRC)
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint4* vp = reinterpret_cast<const uint4*>(p.V + static_cast<int64_t>(j0 + j) * p.K + kb * kBlockK) + 2 * chunk;
              acc[j] = dot8(x1, __ldg(vp + 1), dot8(x0, __ldg(vp), 0.0f));
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], 1);
              acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], 2);
              acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], 4);
            }
            if (m_ok && chunk == 0) {
#pragma unroll
              for (int j = 0; j < 8; ++j) atomicAdd(&fq->t[slot][m * p.r + j0 + j], acc[j]);
            }
          }
        }
      }
      __threadfence();
      named_bar_sync(2, C::kEpiThreads);
      if (threadIdx.x == 0 && !grid_meet(&fq->arrived_absmax, sharers, has_share && ok_start, s_abort))
        raise_error(p, s_abort, kErrGridWait);
      named_bar_sync(2, C::kEpiThreads);
      if (ok_start && *s_abort == 0) {
        if (blockIdx.x == 0)  // one CTA adds the copies of t up for everybody's epilogue
          for (int e = threadIdx.x; e < p.M * p.r; e += C::kEpiThreads) {
            float v = 0.0f;
#pragma unroll
            for (int sl = 0; sl < kFusedSlots; ++sl) v += __ldcg(&fq->t[sl][e]);
            fq->t_sum[e] = v;
          }
        float a = 0.0f;
        if (m_ok) {
#pragma unroll
          for (int sl = 0; sl < kFusedSlots; ++sl) a = fmaxf(a, __uint_as_float(__ldcg(&fq->amax_bits[sl][m])));
        }
        const float inv = a != 0.0f ? __fdiv_rn(448.0f, a) : 1.0f;
        int i = 0;
        for (int kb = blockIdx.x; kb < p.kblocks; kb += gridDim.x, ++i) {
          if (m_ok) {
            uint4 x0, x1;
            if (i == 0) {
              x0 = xk[0][0];
              x1 = xk[0][1];
            } else if (i == 1) {
              x0 = xk[1][0];
              x1 = xk[1][1];
            } else {
              const uint4* xp = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(m) * p.ldx + kb * kBlockK) + 2 * chunk;
              x0 = __ldg(xp);
              x1 = __ldg(xp + 1);
            }
            const uint2 lo = cast8(x0, inv), hi = cast8(x1, inv);
            *reinterpret_cast<uint4*>(p.q_out + static_cast<int64_t>(m) * p.K + kb * kBlockK + 16 * chunk) =
                make_uint4(lo.x, lo.y, hi.x, hi.y);
          }
        }
        asm volatile("fence.proxy.async.global;" ::: "memory");  // the copy engine will read these stores
      }
      __threadfence();
      named_bar_sync(2, C::kEpiThreads);
      if (threadIdx.x == 0 && !grid_meet(&fq->arrived_codes, sharers, has_share && ok_start, s_abort))
        raise_error(p, s_abort, kErrGridWait);
      named_bar_sync(3, C::kEpiThreads + 32);  // releases the producer's token loads
      if (*s_abort) failed = true;
    }

    // Every thread walks every segment and executes the same named-barrier sequence whether or not it
    // has failed, so a bounded wait that ran out can never leave others stuck at a hardware barrier.
    for (int seg = 0; sg.next(p, pos, tile, kb0, nkb); ++seg) {
      const int m0 = (tile / p.n_tiles) * BM;
      const int n = (tile % p.n_tiles) * kTileN + row;
      const bool n_ok = n < p.N;
      const int buf = seg % C::NB;
      // where the finished tile is read from: the segment's accumulator, or (NONE) the region the promoted sums go to
      const uint32_t t_lane = tmem_base + (NONE ? C::kResultCol0 : buf * C::kDColsPad) + lane_base;

      if (m0 != m0_loaded) {
        // token scales and (rank 8) LoRC rows of this tile's tokens
        named_bar_sync(2, C::kEpiThreads);  // the previous tile's reads are done
        if (FUSEQ) {
          // token scales from the absmax the CTAs agreed on: sx = fl32(a / 448), 1 for an all-zero token
          for (int c = threadIdx.x; c < BM; c += C::kEpiThreads) {
            float a = 0.0f;
            if (c < p.M)
              for (int sl = 0; sl < kFusedSlots; ++sl) a = fmaxf(a, __uint_as_float(__ldcg(&p.fq->amax_bits[sl][c])));
            s_sx[c] = c < p.M ? (a != 0.0f ? __fdiv_rn(a, 448.0f) : 1.0f) : 0.0f;
          }
          if (p.r == 8)
            for (int c = threadIdx.x; c < BM * 8; c += C::kEpiThreads)
              s_t[(c & 7) * BM + (c >> 3)] = ((c >> 3) < p.M) ? __ldcg(&p.fq->t_sum[c]) : 0.0f;
        } else {
          for (int c = threadIdx.x; c < BM; c += C::kEpiThreads) s_sx[c] = (m0 + c < p.M) ? __ldg(p.sx + m0 + c) : 0.0f;
          if (p.r == 8)
            for (int c = threadIdx.x; c < BM * 8; c += C::kEpiThreads)  // transposed: [j][BM]
              s_t[(c & 7) * BM + (c >> 3)] =
                  (m0 + (c >> 3) < p.M) ? __ldg(p.t + static_cast<int64_t>(m0) * 8 + c) : 0.0f;
        }
        named_bar_sync(2, C::kEpiThreads);
        m0_loaded = m0;
      }

      float cs = 1.0f;
      uint64_t u[8];  // the channel's U row, each value in both halves of a packed pair
#pragma unroll
      for (int e = 0; e < 8; ++e) u[e] = 0ull;
      if (n_ok && !NONE) cs = __ldg(p.scale + n);
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
      if (NONE) {
        // Per-group promotion (Section 3, the unconstrained scales that M1 / M2 do away with): every weight
        // group's FP32 partial sum is multiplied by the group's scale S[n, g] and added to the running sums in
        // registers, while the MMAs of the next group fill the other buffer.
        const int mpg = p.group / 32;
        const int g_first = (kb0 * (kBlockK / 32)) / mpg, g_last = ((kb0 + nkb) * (kBlockK / 32) - 1) / mpg;
        const float* srow = p.scale + static_cast<int64_t>(n_ok ? n : 0) * p.G;
        float run[BM];
#pragma unroll
        for (int c = 0; c < BM; ++c) run[c] = 0.0f;
        float S_next = n_ok ? __ldg(srow + g_first) : 0.0f;
        for (int g = g_first; g <= g_last; ++g) {
          const float S = S_next;
          if (n_ok && g < g_last) S_next = __ldg(srow + g + 1);
          const int gb = gcount & 1;
          if (!failed && !mbar_wait_warp(&acc_full[gb], (gcount >> 1) & 1, s_abort)) {
            raise_error(p, s_abort, kErrEpilogue);
            failed = true;
          }
          tc_fence_after_sync();
          if (!failed) {
            const uint32_t g_lane = tmem_base + gb * C::kDColsPad + lane_base;
            // the next 16 columns are in flight while these are added up
            float nxt[16];
            tmem_ld_issue<16>(g_lane, nxt);
#pragma unroll
            for (int c = 0; c < BM; c += 16) {
              float v[16];
              tmem_ld_wait_regs<16>(nxt);
#pragma unroll
              for (int e = 0; e < 16; ++e) v[e] = nxt[e];
              if (c + 16 < BM) tmem_ld_issue<16>(g_lane + c + 16, nxt);
#pragma unroll
              for (int e = 0; e < 16; ++e) run[c + e] = fmaf(S, v[e], run[c + e]);
            }
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[gb]);  // the MMA warp may start a new group in this buffer
          ++gcount;
        }
        // the finished tile goes to the result region, where the common code below finds it
#pragma unroll
        for (int c = 0; c < BM; c += 16) tmem_st16(t_lane + c, reinterpret_cast<const uint32_t*>(run + c));
        tmem_st_wait();
      } else if (!failed) {
        if (!mbar_wait_warp(&acc_full[buf], (seg / C::NB) & 1, s_abort)) {
          raise_error(p, s_abort, kErrEpilogue);
          failed = true;
        }
        tc_fence_after_sync();
      }
      if (nkb == p.kblocks) {
        if (!failed) {
          // the next step's accumulator columns are in flight while this step's are finished
          float nxt[EC];
          tmem_ld_issue<EC>(t_lane, nxt);
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_wait_regs<EC>(nxt);
#pragma unroll
            for (int e = 0; e < EC; ++e) v[e] = nxt[e];
            if (c + EC < BM) tmem_ld_issue<EC>(t_lane + c + EC, nxt);
            if (n_ok || p.y_amax) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, false, true, n_ok);
          }
        }
      } else if (p.atomic_y && p.handover) {
        // Several CTAs share this tile (FP32 y, cooperative launch: all CTAs are resident).  The tile's last
        // contributor in K order meets it as the first segment of its range, i.e. early: it STORES its
        // share (with the LoRC term) and raises the tile's flag.  The others meet the tile at the end of
        // their ranges: they wait for the flag (long set by then) and ADD their shares.  Nothing has to
        // clear y first.  The adder that finds all others done leaves the flag at zero for the next call.
        int first, count;
        contributors(p, pos, &first, &count);
        const bool storer = static_cast<int>(blockIdx.x) == first + count - 1;
        int* flag = p.counters + pos;
        if (!storer) {
          if (threadIdx.x == 0) {
            const uint64_t t0 = global_timer_ns();
            bool ok = false;
            for (uint32_t spin = 0; spin < kSpinLimit && !ok; ++spin) {
              ok = *reinterpret_cast<volatile int*>(flag) != 0 || *s_abort != 0;
              if (!ok && (spin & 63u) == 63u && global_timer_ns() - t0 > kWaitLimitNs) break;
            }
            if (!ok) raise_error(p, s_abort, kErrHandover);
            __threadfence();
          }
          named_bar_sync(2, C::kEpiThreads);
          if (*s_abort) failed = true;
        }
        if (!failed) {
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_cols<EC>(t_lane + c, v);
            if (n_ok) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, !storer, storer);
          }
        }
        __threadfence();  // this thread's stores / adds are performed before the flag moves
        named_bar_sync(2, C::kEpiThreads);
        if (threadIdx.x == 0 && !*s_abort) {
          if (storer) {
            atomicExch(flag, 1);
          } else if (atomicAdd(flag, 1) == count - 1) {
            atomicExch(flag, 0);  // storer + all other adders were counted before this one
          }
        }
      } else if (p.atomic_y) {
        // Several CTAs share this tile and y was zeroed before the launch: every CTA scales its share
        // and adds it; the first contributor also adds the LoRC term.  No fence, ticket or second pass.
        int first, count;
        contributors(p, pos, &first, &count);
        const bool lorc = static_cast<int>(blockIdx.x) == first;
        if (!failed) {
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_cols<EC>(t_lane + c, v);
            if (n_ok) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, true, lorc);
          }
        }
      } else {
        // Several CTAs share this tile: leave the raw partial sums in the workspace; the CTA that
        // arrives last adds all of them in contributor order (deterministic) and finishes the tile.
        int first, count;
        contributors(p, pos, &first, &count);
        const int my_j = (p.stream || p.persist) ? static_cast<int>(blockIdx.x) - first : static_cast<int>(blockIdx.x) / p.tiles;
        float* my_partial = p.partials + partial_slot(p, pos, first, my_j) * (BM * kTileN);
        if (!failed) {
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_cols<EC>(t_lane + c, v);
#pragma unroll
            for (int e = 0; e < EC; ++e) my_partial[(c + e) * kTileN + row] = v[e];
          }
        }
        __threadfence();
        named_bar_sync(1, C::kEpiThreads);
        if (threadIdx.x == 0) {
          const int ticket = (*s_abort) ? -1 : atomicAdd(p.counters + pos, 1);
          *s_last = (ticket == count - 1) ? 1 : 0;
          if (ticket == count - 1) p.counters[pos] = 0;  // ready for the next call
        }
        named_bar_sync(1, C::kEpiThreads);
        if (*s_last) {
          __threadfence();
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
#pragma unroll
            for (int e = 0; e < EC; ++e) v[e] = 0.0f;
            for (int j = 0; j < count; ++j) {
              const float* src = p.partials + partial_slot(p, pos, first, j) * (BM * kTileN) + c * kTileN + row;
#pragma unroll
              for (int e = 0; e < EC; ++e) v[e] += __ldcg(src + e * kTileN);
            }
            if (n_ok || p.y_amax) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, false, true, n_ok);
          }
        }
        named_bar_sync(1, C::kEpiThreads);  // s_last is reused by the next segment
      }
      // the accumulator buffer has been read: the MMA warp may reuse it
      tc_fence_before_sync();
      __syncwarp();
      if (!NONE && lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == C::kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::kTmemCols);
  }
  if (FUSEQ) {
    // The CTA that leaves last clears the scratch for the next launch (every other CTA has read what it
    // needs before it counts itself out).  After a wait that ran out the scratch is left as it is: the
    // workspace has to be re-initialized anyway.
    if (threadIdx.x == 0)
      *s_last = (*s_abort == 0 && atomicAdd(&p.fq->departed, 1u) == gridDim.x - 1) ? 1 : 0;
    __syncthreads();
    if (*s_last) {
      for (int i = threadIdx.x; i < kFusedSlots * kFusedMaxTokens; i += C::kThreads) (&p.fq->amax_bits[0][0])[i] = 0u;
      for (int sl = 0; sl < kFusedSlots; ++sl)
        for (int i = threadIdx.x; i < kFusedMaxTokens * p.r; i += C::kThreads) p.fq->t[sl][i] = 0.0f;
      if (threadIdx.x == 0) {
        p.fq->arrived_absmax = 0u;
        p.fq->arrived_codes = 0u;
        p.fq->departed = 0u;
      }
    }
  }
}

// ---- many tokens: CTA pairs ---------------------------------------------------------------------------
// With wide token tiles the kernel above is bound by the bytes that reach shared memory: per K block 16 KB of
// codes and 128 bytes per token.  Here the two CTAs of a cluster share one token tile: one MMA of 256 channels x
// BM tokens (cta_group::2) reads channels 0..127 and tokens 0..BM/2-1 from the leader's shared memory, channels
// 128..255 and the other half of the tokens from its peer's, and accumulates each CTA's 128 channels in that
// CTA's own tensor memory.  Each CTA loads its own weight tile, scales and half of the tokens (all counted on
// the leader's barrier), the leader's MMA thread issues for both, its commits release the stages and publish
// the accumulators in both CTAs, and each CTA's epilogue warps finish their own 128 channels.  The token bytes
// per CTA and K block are halved.
// Work partition: as above with pairs in place of CTAs and pair positions (token tile x two neighbouring channel
// tiles) in place of tiles: whole positions in whole rounds, the rest dealt out as contiguous unit ranges; a
// position shared by several pairs is handed over through per-CTA flags (FP32 y only): the last contributor in K
// order stores, the others wait for its flag and add.  All pairs of the grid fit the device at once.
template <int BM, bool W8>
struct PairCfg {
  static constexpr int kThreads = 192;
  static constexpr int kEpiThreads = 128;
  static constexpr int kProducerWarp = 4;
  static constexpr int kMmaWarp = 5;
  static constexpr int kHalf = BM / 2;  // token rows in each CTA's shared memory
  static constexpr int kCodeBytes = W8 ? 2 * kTileCodeBytes : kTileCodeBytes;  // a tile's codes in HBM
  static constexpr int kABytes = kTileRows * kTileK;  // in shared memory (padded FP4, or FP8)
  static constexpr int kTokBytes = kHalf * kBlockK;
  static constexpr int kSfBytes = kMxTileScaleBytes;
  static constexpr int kStageTx = kCodeBytes + kTokBytes + kSfBytes;  // bytes one CTA's copies of a stage count
  static constexpr int kStageBytes = kABytes + kTokBytes + kSfBytes;
  static constexpr int NS = cmin(8, (218 * 1024 - BM * 36 - 512) / kStageBytes);
  static constexpr int NB = 2;  // accumulator buffers
  static constexpr int kSfaCol0 = NB * BM;
  static constexpr int kSfbCol0 = kSfaCol0 + 4 * NS;
  static constexpr int kColsUsed = kSfbCol0 + kSfbCols;
  static constexpr int kTmemCols = 512;
  static constexpr int offA = 0;
  static constexpr int offTok = offA + NS * kABytes;
  static constexpr int offSf = offTok + NS * kTokBytes;
  static constexpr int offSx = offSf + NS * kSfBytes;
  static constexpr int offT = offSx + BM * 4;
  static constexpr int offBars = offT + BM * 32;
  static constexpr int kNumBars = 2 * NS + 2 * NB + 1;
  static constexpr int offMisc = offBars + kNumBars * 8;
  static constexpr int kSmemBytes = offMisc + 32;
  static_assert(BM % 16 == 0 && BM >= 64 && BM <= 224, "token tile of the pair: two accumulators");
  static_assert(kTokBytes % 1024 == 0, "token stages must start on a swizzle atom");
  static_assert(NS >= 4, "pipeline depth");
  static_assert(kColsUsed <= kTmemCols, "tensor memory");
  static_assert(kSmemBytes <= 226 * 1024, "shared memory");
};

// Pair position -> (token tile, pair of channel tiles).  Like raster_tile: through groups of m_group token
// tiles, the group's token tiles inner, so that the pairs running at one time share operands in L2.
__device__ __forceinline__ void pair_tile(const Params& p, int pos, int& m_tile, int& n_pair) {
  const int np = p.n_tiles / 2, m_tiles = p.tiles / p.n_tiles;
  const int mg = p.m_group < 1 ? 1 : p.m_group;
  const int per_group = mg * np;
  const int g = pos / per_group, within = pos - g * per_group;
  const int gm = min(mg, m_tiles - g * mg);
  m_tile = g * mg + within % gm;
  n_pair = within / gm;
}

template <int BM, bool W8>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairCfg<BM, W8>::kThreads, 1)
w4a8_mx_pair_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_q,
                         const __grid_constant__ CUtensorMap tm_sf, const Params p) {
  using C = PairCfg<BM, W8>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* s_a = smem + C::offA;
  uint8_t* s_tok = smem + C::offTok;
  uint8_t* s_sf = smem + C::offSf;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offBars);
  uint64_t* full = bars;                  // [NS] leader's: both CTAs' copies of the stage landed   (MMA waits)
  uint64_t* empty = full + C::NS;         // [NS] each CTA's: the MMAs that read the stage are done  (producers wait)
  uint64_t* acc_full = empty + C::NS;     // [NB] each CTA's: a tile's accumulation is complete      (epilogues wait)
  uint64_t* acc_empty = acc_full + C::NB; // [NB] leader's: both CTAs' epilogues have read the buffer (MMA waits)
  uint64_t* drain_bar = acc_empty + C::NB;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::offMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::offMisc + 4);
  float* s_sx = reinterpret_cast<float*>(smem + C::offSx);
  float* s_t = reinterpret_cast<float*>(smem + C::offT);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pairs = static_cast<int>(gridDim.x) / 2, pair = static_cast<int>(blockIdx.x) / 2;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::NS; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < C::NB; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 8);  // one arrival per epilogue warp of either CTA
    }
    mbar_init(drain_bar, 1);
    *s_abort = 0;
    fence_mbar_init();
    if ((smem_u32(smem) & 1023u) != 0) raise_error(p, s_abort, kErrAlign);
  }
  if (warp == C::kProducerWarp && lane == 0) {
    prefetch_tensormap(&tm_w);
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_sf);
  }
  if (warp == C::kMmaWarp) tmem_alloc_pair(s_tmem, C::kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_sfa = tmem_base + C::kSfaCol0;
  const uint32_t tmem_sfb = tmem_base + C::kSfbCol0;
  if (warp < 4) {
    // the tokens' block scales are all 2^0: each CTA fills its copy once
    uint32_t ones[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) ones[i] = 0x7F7F7F7Fu;
    tmem_st16(tmem_sfb + (static_cast<uint32_t>(warp * 32) << 16), ones);
    tmem_st_wait();
  }
  tc_fence_before_sync();
  cluster_sync_all();  // both CTAs' barriers are initialized, their tensor memory allocated and the scales of one written
  tc_fence_after_sync();
  const bool ok_start = (*s_abort == 0);
  if (threadIdx.x == 0) pdl_launch_dependents();

  if (warp == C::kProducerWarp) {
    // ------------------------------------------------------------------ producer (both CTAs)
    if (ok_start) {
      const bool issuer = elect_one();
      pdl_wait();  // the tokens may be the output of the kernel ahead in the stream
      int s = 0, issued = 0;
      uint32_t ph = 0;
      bool ok = true;
      Segments sg(p, pair, pairs, true);
      int pos, tile_unused, kb0, nkb;
      while (ok && sg.next(p, pos, tile_unused, kb0, nkb)) {
        int m_tile, n_pair;
        pair_tile(p, pos, m_tile, n_pair);
        const int nt = 2 * n_pair + static_cast<int>(rank);
        const int row0 = m_tile * BM + static_cast<int>(rank) * C::kHalf;
        for (int kb = kb0; kb < kb0 + nkb; ++kb) {
          if (issued >= C::NS && !mbar_wait(&empty[s], ph ^ 1, s_abort)) {
            if (issuer) raise_error(p, s_abort, kErrProducer);
            ok = false;
            break;
          }
          if (issuer) {
            const uint32_t bar = map_to_rank(smem_u32(&full[s]), 0);
            if (leader) mbar_arrive_expect_tx(&full[s], 2 * C::kStageTx);
            tma_load_4d_pair(s_a + s * C::kABytes, &tm_w, 0, 0, kb, nt, bar);
            tma_load_3d_pair(s_sf + s * C::kSfBytes, &tm_sf, 0, 4 * kb, nt, bar);
            tma_load_3d_pair(s_tok + s * C::kTokBytes, &tm_q, 0, row0, kb, bar);
          }
          __syncwarp();
          ++issued;
          if (++s == C::NS) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      // never leave with copies still in flight: the stages this CTA filled last are released by the MMAs that
      // read them, which run only after the copies landed
      for (int i = max(0, issued - C::NS); i < issued; ++i) {
        uint32_t spin = 0;
        while (!mbar_try_wait(&empty[i % C::NS], (i / C::NS) & 1) && ++spin < kSpinLimit && !*s_abort) {
        }
      }
    }
  } else if (warp == C::kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (ok_start && leader) {
      const bool issuer = elect_one();
      const uint64_t adesc0 = umma_desc_k128(smem_u32(s_a));
      const uint64_t bdesc0 = umma_desc_k128(smem_u32(s_tok));
      const uint64_t sfdesc0 = umma_desc_rows16(smem_u32(s_sf), 128);
      int s = 0, seg = 0;
      uint32_t ph = 0;
      bool failed = false;
      Segments sg(p, pair, pairs, true);
      int pos, tile_unused, kb0, nkb;
      for (; !failed && sg.next(p, pos, tile_unused, kb0, nkb); ++seg) {
        const int buf = seg % C::NB;
        if (seg >= C::NB && !mbar_wait(&acc_empty[buf], ((seg / C::NB) - 1) & 1, s_abort)) {
          failed = true;
          break;
        }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + buf * BM;
        for (int kb = 0; kb < nkb && !failed; ++kb) {
          if (!mbar_wait(&full[s], ph, s_abort)) {
            failed = true;
            break;
          }
          tc_fence_after_sync();
          if (issuer) {
            const uint32_t sfa = tmem_sfa + 4 * s;
            const uint64_t adesc = adesc0 + static_cast<uint64_t>((s * C::kABytes) >> 4);
            const uint64_t bdesc = bdesc0 + static_cast<uint64_t>((s * C::kTokBytes) >> 4);
            tmem_cp_32x128b_x4_pair(sfa, sfdesc0 + static_cast<uint64_t>((s * C::kSfBytes) >> 4));
#pragma unroll
            for (int k = 0; k < kBlockK / 32; ++k) {
              const uint32_t idesc = (W8 ? umma_idesc_mx_e4m3_e4m3(BM, k, 0) : umma_idesc_mx_e2m1_e4m3(BM, k, 0)) +
                                     ((128u >> 4) << 24);  // 256 rows: 128 in each CTA
              umma_mxf8f6f4_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, sfa + (static_cast<uint32_t>(k) << 30),
                                 tmem_sfb, (kb > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_pair(&empty[s]);
            if (kb + 1 == nkb) umma_commit_pair(&acc_full[buf]);
          }
          __syncwarp();
          if (++s == C::NS) {
            s = 0;
            ph ^= 1;
          }
        }
      }
      if (failed) {
        if (issuer) {
          raise_error(p, s_abort, kErrMma);
          umma_commit_pair(drain_bar);  // let the MMAs already issued finish before tensor memory is released
        }
        uint32_t spin = 0;
        while (!mbar_try_wait(drain_bar, 0) && ++spin < kSpinLimit) {
        }
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs, own 128 channels)
    const int row = warp * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    constexpr int EC = 16;
    bool failed = !ok_start;
    int m0_loaded = -1;
    pdl_wait();  // sx, t and y may still be in use by the kernel ahead in the stream
    int seg = 0;
    Segments sg(p, pair, pairs, true);
    int pos, tile_unused, kb0, nkb;
    for (; sg.next(p, pos, tile_unused, kb0, nkb); ++seg) {
      int m_tile, n_pair;
      pair_tile(p, pos, m_tile, n_pair);
      const int m0 = m_tile * BM;
      const int n = (2 * n_pair + static_cast<int>(rank)) * kTileN + row;
      const bool n_ok = n < p.N;
      const int buf = seg % C::NB;
      const uint32_t t_lane = tmem_base + buf * BM + lane_base;
      if (m0 != m0_loaded) {
        named_bar_sync(2, C::kEpiThreads);  // the previous tile's reads are done
        for (int c = threadIdx.x; c < BM; c += C::kEpiThreads) s_sx[c] = (m0 + c < p.M) ? __ldg(p.sx + m0 + c) : 0.0f;
        if (p.r == 8)
          for (int c = threadIdx.x; c < BM * 8; c += C::kEpiThreads)  // transposed: [j][BM]
            s_t[(c & 7) * BM + (c >> 3)] = (m0 + (c >> 3) < p.M) ? __ldg(p.t + static_cast<int64_t>(m0) * 8 + c) : 0.0f;
        named_bar_sync(2, C::kEpiThreads);
        m0_loaded = m0;
      }
      float cs = 1.0f;
      uint64_t u[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) u[e] = 0ull;
      if (n_ok) cs = __ldg(p.scale + n);
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
      if (!failed && !mbar_wait_warp(&acc_full[buf], (seg / C::NB) & 1, s_abort)) {
        raise_error(p, s_abort, kErrEpilogue);
        failed = true;
      }
      tc_fence_after_sync();
      if (nkb == p.kblocks) {
        if (!failed) {
          float nxt[EC];
          tmem_ld_issue<EC>(t_lane, nxt);
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_wait_regs<EC>(nxt);
#pragma unroll
            for (int e = 0; e < EC; ++e) v[e] = nxt[e];
            if (c + EC < BM) tmem_ld_issue<EC>(t_lane + c + EC, nxt);
            if (n_ok || p.y_amax) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, false, true, n_ok);
          }
        }
      } else {
        // Several pairs share this position (FP32 y).  Its last contributor in K order meets it as the first
        // segment of its range, i.e. early: it STORES its share (with the LoRC term) and raises this CTA's flag of
        // the position.  The others meet it at the end of their ranges: they wait for the flag and ADD their
        // shares.  The adder that finds all others done leaves the flag at zero for the next call.
        int first, count;
        contributors(p, pos, &first, &count);
        const bool storer = pair == first + count - 1;
        int* flag = p.counters + 2 * pos + static_cast<int>(rank);
        if (!storer) {
          if (threadIdx.x == 0) {
            const uint64_t t0 = global_timer_ns();
            bool ok = false;
            for (uint32_t spin = 0; spin < kSpinLimit && !ok; ++spin) {
              ok = *reinterpret_cast<volatile int*>(flag) != 0 || *s_abort != 0;
              if (!ok && (spin & 63u) == 63u && global_timer_ns() - t0 > kWaitLimitNs) break;
            }
            if (!ok) raise_error(p, s_abort, kErrHandover);
            __threadfence();
          }
          named_bar_sync(2, C::kEpiThreads);
          if (*s_abort) failed = true;
        }
        if (!failed) {
#pragma unroll 1
          for (int c = 0; c < BM; c += EC) {
            float v[EC];
            tmem_ld_cols<EC>(t_lane + c, v);
            if (n_ok) finalize<EC, BM>(p, v, m0, c, n, cs, u, s_sx, s_t, !storer, storer);
          }
        }
        __threadfence();  // this thread's stores / adds are performed before the flag moves
        named_bar_sync(2, C::kEpiThreads);
        if (threadIdx.x == 0 && !*s_abort) {
          if (storer) {
            atomicExch(flag, 1);
          } else if (atomicAdd(flag, 1) == count - 1) {
            atomicExch(flag, 0);  // storer + all other adders were counted before this one
          }
        }
      }
      // this warp has read the buffer: tell the leader's MMA thread
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&acc_empty[buf]), 0));
    }
  }

  tc_fence_before_sync();
  cluster_sync_all();  // both CTAs are done with both CTAs' tensor memory and barriers
  if (warp == C::kMmaWarp) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, C::kTmemCols);
  }
}

// ---- host ------------------------------------------------------------------------------------------
// The packed weight as a 4-D tensor of 4-bit elements [row blocks][K blocks][128 rows][128 elements]; the copy
// engine expands a box of `kps` 128 x 128 tiles to the 16-byte-aligned FP4 form in shared memory, 128-byte
// swizzled, one tile after the other.
// (FP8 weights: the same tensor of bytes, copied as it is.)
bool make_weight_map(CUtensorMap* m, const void* base, uint64_t n_tiles, uint64_t kblocks, uint32_t kps, bool w8) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const uint64_t code_bytes = w8 ? 2 * kTileCodeBytes : kTileCodeBytes;
  const cuuint64_t dims[4] = {kTileK, kTileRows, kblocks, n_tiles};
  const cuuint64_t strides[3] = {code_bytes / kTileRows, code_bytes, kblocks * (code_bytes + kMxTileScaleBytes)};
  const cuuint32_t box[4] = {kTileK, kTileRows, kps, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, w8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The E4M3 activations q [M, K] as a 3-D tensor [K blocks][M rows][128 bytes]: a box of `kps` K blocks x bm
// rows lands in shared memory as `kps` token tiles of bm x 128 bytes, one after the other, 128-byte swizzled.
bool make_token_map(CUtensorMap* m, const void* base, uint64_t K, uint64_t M, uint32_t bm, uint32_t kps) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {kBlockK, M, K / kBlockK};
  const cuuint64_t strides[2] = {K, kBlockK};
  const cuuint32_t box[3] = {kBlockK, bm, kps};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BM, bool W8, bool FUSEQ, bool NONE>
int launch_mx_cfg(const GemmArgs& a, const GemmPlan& plan, const Params& p, cudaStream_t st) {
  using C = MxCfg<BM, W8, NONE>;
  CUtensorMap tm_w, tm_q;
  if (!make_weight_map(&tm_w, a.codes, static_cast<uint64_t>(plan.n_tiles), static_cast<uint64_t>(p.kblocks), C::kKps, W8) ||
      !make_token_map(&tm_q, a.q, static_cast<uint64_t>(a.K), static_cast<uint64_t>(a.M), BM, C::kKps))
    return ZQ_ERR_CUDA;
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(once, [] {
    attr_err = cudaFuncSetAttribute(w4a8_mx_gemm_kernel<BM, W8, FUSEQ, NONE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    C::kSmemBytes);
  });
  if (attr_err != cudaSuccess) return ZQ_ERR_CUDA;
  dim3 grid(static_cast<unsigned>(plan.ctas));
  const bool fused_out = a.relu || a.y_amax;  // final values must be known to one CTA: no adding into y
  const bool shared_f32 =
      a.ydt == ZQ_OUT_F32 && !fused_out && (p.atomic_y || (plan.persist && plan.tail_pos0 < p.tiles));
  if (shared_f32 || FUSEQ) {
    // Output tiles are shared by CTAs that accumulate into FP32 y.  In a cooperative launch (all CTAs
    // resident, which the plan's grid is sized for) they hand over through per-tile flags: one stores,
    // the others wait for it and add.  If the device cannot hold the grid at once: unit ranges -> clear
    // y with a memset and let every CTA add; persistent launch -> partial sums through the workspace.
    // (The kernel with the quantizer inside has its CTAs meet in a scratch as well, so its launch is always
    // cooperative; if that is refused nothing has run and the caller takes the two-kernel path.)
    Params pc = p;
    if (shared_f32) {
      pc.atomic_y = 1;
      pc.handover = 1;
    }
    void* args[3] = {&tm_w, &tm_q, &pc};
    // chained to the kernel ahead (see pdl_wait); if the two launch attributes are refused together, cooperative alone.
    // The cooperative attribute is what guarantees that all CTAs of the grid (one per SM at most) run at the same
    // time; it costs about 3.5 us per launch (the launch waits for the whole device to be free).  A caller that
    // has promised the device to this library alone (zq_set_exclusive_device) gets a plain launch: with nothing
    // else running, a grid of at most one CTA per SM is resident as soon as the kernel ahead has drained.
    if (launch_chained(w4a8_mx_gemm_kernel<BM, W8, FUSEQ, NONE>, grid, dim3(C::kThreads), C::kSmemBytes, st, !exclusive_device(), tm_w, tm_q, pc) ==
        cudaSuccess) {
      count_launch();
      return ZQ_OK;
    }
    (void)cudaGetLastError();
    if (cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(w4a8_mx_gemm_kernel<BM, W8, FUSEQ, NONE>), grid, dim3(C::kThreads),
                                    args, C::kSmemBytes, st) == cudaSuccess) {
      count_launch();
      return ZQ_OK;
    }
    (void)cudaGetLastError();  // not launched; fall back
    if (FUSEQ) return kFusedLaunchRefused;
    if (p.atomic_y && cudaMemset2DAsync(a.y, static_cast<size_t>(a.ldy) * 4, 0, static_cast<size_t>(a.N) * 4,
                                        static_cast<size_t>(a.M), st) != cudaSuccess)
      return ZQ_ERR_CUDA;
  }
  const cudaError_t err = launch_chained(w4a8_mx_gemm_kernel<BM, W8, FUSEQ, NONE>, grid, dim3(C::kThreads), C::kSmemBytes, st, false,
                                         tm_w, tm_q, p);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
}

// The tiles' E8M0 scales (512 bytes per tile, behind the row block's codes) as a 3-D tensor
// [row blocks][4 * K blocks][128 bytes]: a box of 4 rows is one tile's scales.
bool make_scale_map(CUtensorMap* m, const void* codes, uint64_t n_tiles, uint64_t kblocks, bool w8) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const uint64_t code_bytes = w8 ? 2 * kTileCodeBytes : kTileCodeBytes;
  const cuuint64_t dims[3] = {128, 4 * kblocks, n_tiles};
  const cuuint64_t strides[2] = {128, kblocks * (code_bytes + kMxTileScaleBytes)};
  const cuuint32_t box[3] = {128, 4, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const uint8_t* base = static_cast<const uint8_t*>(codes) + kblocks * code_bytes;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Returns kPairNotTaken when the device grants no CTA pair for this kernel; nothing has run then.
constexpr int kPairNotTaken = -1001;
template <int BM, bool W8>
int launch_pair_cfg(const GemmArgs& a, const GemmPlan& plan, Params p, cudaStream_t st) {
  using C = PairCfg<BM, W8>;
  auto kernel = w4a8_mx_pair_gemm_kernel<BM, W8>;
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  static int max_pairs = 0;
  std::call_once(once, [&] {
    attr_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (attr_err == cudaSuccess) {
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3(2 * sm_count());
      cfg.blockDim = dim3(C::kThreads);
      cfg.dynamicSmemBytes = C::kSmemBytes;
      if (cudaOccupancyMaxActiveClusters(&max_pairs, kernel, &cfg) != cudaSuccess) max_pairs = 0;
      (void)cudaGetLastError();
    }
  });
  if (attr_err != cudaSuccess || max_pairs < 1) return kPairNotTaken;
  CUtensorMap tm_w, tm_q, tm_sf;
  if (!make_weight_map(&tm_w, a.codes, static_cast<uint64_t>(plan.n_tiles), static_cast<uint64_t>(p.kblocks), 1, W8) ||
      !make_token_map(&tm_q, a.q, static_cast<uint64_t>(a.K), static_cast<uint64_t>(a.M), C::kHalf, 1) ||
      !make_scale_map(&tm_sf, a.codes, static_cast<uint64_t>(plan.n_tiles), static_cast<uint64_t>(p.kblocks), W8))
    return ZQ_ERR_CUDA;
  // shared positions are handed over by flags between pairs that must all be running: the plan's grid has to fit
  if (plan.ctas / 2 > max_pairs) return kPairNotTaken;
  const cudaError_t err = launch_chained(kernel, dim3(plan.ctas), dim3(C::kThreads), C::kSmemBytes, st, false, tm_w,
                                         tm_q, tm_sf, p);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ZQ_OK : ZQ_ERR_CUDA;
}

}  // namespace

int launch_w4a8_mx_gemm(const GemmArgs& a, cudaStream_t st) {
  GemmPlan plan = plan_gemm(a.M, a.N, a.K, a.mode, ZQ_WEIGHTS_MX);
  if (plan.pair) {
    // positions shared between pairs are added into an FP32 y; a bf16 y (or one with ReLU / the tokens' maxima
    // fused in) takes the single CTAs, and so does a device that grants the pair kernel fewer pairs than planned
    const bool shared = plan.stream || plan.tail_pos0 < plan.m_tiles * (plan.n_tiles / 2);
    int e = kPairNotTaken;
    if (!(shared && (a.ydt != ZQ_OUT_F32 || a.relu || a.y_amax))) {
      Params pp = make_params(a, plan);
      const bool w8p = a.layout == ZQ_WEIGHTS_MX_FP8;
      switch (plan.bm) {
        case 128: e = w8p ? launch_pair_cfg<128, true>(a, plan, pp, st) : launch_pair_cfg<128, false>(a, plan, pp, st); break;
        case 176: e = w8p ? launch_pair_cfg<176, true>(a, plan, pp, st) : launch_pair_cfg<176, false>(a, plan, pp, st); break;
        case 192: e = w8p ? launch_pair_cfg<192, true>(a, plan, pp, st) : launch_pair_cfg<192, false>(a, plan, pp, st); break;
        case 208: e = w8p ? launch_pair_cfg<208, true>(a, plan, pp, st) : launch_pair_cfg<208, false>(a, plan, pp, st); break;
        case 224: e = w8p ? launch_pair_cfg<224, true>(a, plan, pp, st) : launch_pair_cfg<224, false>(a, plan, pp, st); break;
      }
    }
    if (e != kPairNotTaken) return e;
    plan = plan_gemm(a.M, a.N, a.K, a.mode, ZQ_WEIGHTS_MX, false);
  }
  if (plan.partial_floats > a.partial_floats) return ZQ_ERR_WORKSPACE;
  Params p = make_params(a, plan);
  const bool w8 = a.layout == ZQ_WEIGHTS_MX_FP8;
  if (a.x) {
    // the kernel quantizes the activations itself: one tile of at most kFusedMaxTokens tokens
    if (a.M > kFusedMaxTokens || plan.bm != 16 || plan.m_tiles != 1 || a.r > kFusedMaxRank || !a.fused_scratch || !a.q)
      return ZQ_ERR_SHAPE;
    p.sx = nullptr;
    p.t = p.fq->t_sum;  // token-major [M, r], as the separate quantizer writes it
    if (a.mode == ZQ_SCALE_NONE) return ZQ_ERR_MODE;
    return w8 ? launch_mx_cfg<16, true, true, false>(a, plan, p, st) : launch_mx_cfg<16, false, true, false>(a, plan, p, st);
  }
  if (a.mode == ZQ_SCALE_NONE) {  // unconstrained FP32 group scales: per-group promotion, token tiles up to 128
    if (w8) return ZQ_ERR_MODE;
    switch (plan.bm) {
      case 16: return launch_mx_cfg<16, false, false, true>(a, plan, p, st);
      case 32: return launch_mx_cfg<32, false, false, true>(a, plan, p, st);
      case 64: return launch_mx_cfg<64, false, false, true>(a, plan, p, st);
      case 128: return launch_mx_cfg<128, false, false, true>(a, plan, p, st);
    }
    return ZQ_ERR_SHAPE;
  }
#define ZQ_MX_CASE(BM_) \
  case BM_: return w8 ? launch_mx_cfg<BM_, true, false, false>(a, plan, p, st) : launch_mx_cfg<BM_, false, false, false>(a, plan, p, st)
  switch (plan.bm) {
    ZQ_MX_CASE(16);
    ZQ_MX_CASE(32);
    ZQ_MX_CASE(64);
    ZQ_MX_CASE(128);
    ZQ_MX_CASE(192);
    ZQ_MX_CASE(224);
    ZQ_MX_CASE(256);
  }
#undef ZQ_MX_CASE
  return ZQ_ERR_SHAPE;
}

}  // namespace zq
