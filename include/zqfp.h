/*
 * zqfp — W4A8 quantized linear layer (FP4-E2M1 weights, FP8-E4M3 activations, LoRC) for sm_100a.
 *
 * C ABI.  Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller;
 * the library never allocates or frees device memory.  Every call enqueues its work on `stream`
 * (a cudaStream_t passed as void*, NULL = the default stream) and returns without synchronizing,
 * except where stated.  Return value: ZQ_OK, or a negative ZQ_ERR_* found by host-side validation
 * before anything was launched.  No exception crosses the boundary.  Calls on distinct streams with
 * distinct workspaces are independent; two calls that share a workspace must not overlap on the GPU.
 *
 * Notation (follows the paper): x[M,K] activations (tokens x input features), W[N,K] weight
 * (output x input features, as nn.Linear stores it), group = number of consecutive input features
 * of one output row that share a weight scale, G = K / group, r = LoRC rank.
 */
#ifndef ZQFP_H_
#define ZQFP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ZQ_OK 0
#define ZQ_ERR_NULL (-1)           /* a required pointer is NULL */
#define ZQ_ERR_SHAPE (-2)          /* a size is negative, not a supported multiple, or too large */
#define ZQ_ERR_ALIGN (-3)          /* a pointer or a leading dimension breaks its alignment rule */
#define ZQ_ERR_MODE (-4)           /* unknown scale mode or output type */
#define ZQ_ERR_WORKSPACE (-5)      /* workspace missing or smaller than *_workspace_bytes() says */
#define ZQ_ERR_ARCH (-6)           /* the current device is not compute capability 10.x */
#define ZQ_ERR_CUDA (-7)           /* a CUDA runtime / driver call failed (launch, tensor map) */
#define ZQ_ERR_DEVICE_TIMEOUT (-8) /* a kernel gave up on a bounded wait; see zq_device_status */

/* Weight-scale constraint, Section 3 "Casting the FP4 to FP8". */
typedef enum {
  ZQ_SCALE_NONE = 0, /* unconstrained FP32 scale per group */
  ZQ_SCALE_M1 = 1,   /* (M1) every group scale is rounded up to a power of two */
  ZQ_SCALE_M2 = 2    /* (M2) group scale = per-channel S_max divided by a power of two */
} zq_scale_mode;

typedef enum { ZQ_OUT_F32 = 0, ZQ_OUT_BF16 = 1 } zq_out_dtype;

/* How the packed weight is laid out, which decides who performs the cast FP4 -> FP8 of Section 3
 * ("Casting the FP4 to FP8") during the GEMM.  Codes, shifts and scales are the same either way. */
typedef enum {
  ZQ_WEIGHTS_CAST = 0, /* the kernel casts each code to E4M3 itself, as an exponent-field subtraction */
  ZQ_WEIGHTS_MX = 1,   /* modes M1 / M2 only: the tensor core reads the E2M1 codes directly and applies the
                          power-of-two shift of each group as an E8M0 block scale (exact, being a power of two) */
  ZQ_WEIGHTS_MX_FP8 = 2,    /* modes M1 / M2 only: FP8-E4M3 weight codes instead of FP4 (the W8A8 FP - FP rows of
                               Table 2; group scale absmax / 448), in the block-scaled arrangement: the same GEMM
                               without the cast */
  ZQ_WEIGHTS_CAST_E5M2 = 3  /* modes M1 / M2 only: as ZQ_WEIGHTS_CAST, but the kernel casts each code to E5M2 (Section
                               3, footnote to "Casting the FP4 to FP8"), whose five exponent bits keep the cast a
                               subtraction in the exponent field down to a shift of 13; shifts are stored clamped
                               to [0, 13] */
} zq_weight_layout;

const char* zq_status_string(int status);

/*
 * Token-wise FP8 activation quantization (Section 3, the activation quantizer of the W4A8 scheme;
 * Appendix A; symmetric, i.e. Eq. 1 with Z = 0, in the E4M3 format of Section 2 / 4).
 *
 *   a_m = max_k |x[m,k]| ;  sx[m] = a_m / 448 ;  q[m,k] = RNE_E4M3( fl32( x[m,k] * fl32(448 / a_m) ) )
 *   saturating at +-448; a token whose elements are all zero gets sx = 1 and codes 0.
 * If V != NULL it also computes the LoRC down-projection (Section 3, LoRC) with the raw x:
 *   t[m,j] = sum_k V[j,k] * x[m,k],  j < r, accumulated in FP32.
 *
 * x    : bf16 [M, ldx] row-major, ldx >= K in elements; 16-byte aligned, ldx % 8 == 0
 * q    : out, E4M3 bytes [M, K] dense; 16-byte aligned
 * sx   : out, FP32 [M]
 * V    : fp16 [r, K] dense or NULL; 16-byte aligned;  t: out, FP32 [M, r] (required iff V != NULL)
 * K % 16 == 0, 16 <= K; 0 <= M; 0 < r <= 64 when V is given.  M == 0 is a no-op.
 */
int zq_quantize_act_fp8(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q,
                        float* sx, const void* V_f16, int r, float* t, void* stream);

/*
 * Sizes in bytes of the three buffers zq_pack_weight_fp4 writes:
 *   codes: ceil(N/128) * (K/128) * 8448 (ZQ_WEIGHTS_CAST, ZQ_WEIGHTS_CAST_E5M2), * 8704 (ZQ_WEIGHTS_MX) or
 *          * 16896 (ZQ_WEIGHTS_MX_FP8), tiled, see below ;
 *   shift: N*G (M1, M2) or 0 (none) ;
 *   scale: 4*N (M1, M2) or 4*N*G (none).
 */
int zq_packed_weight_sizes(int64_t N, int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout,
                           size_t* codes_bytes, size_t* shift_bytes, size_t* scale_bytes);

/*
 * Fine-grained FP4 weight quantization (Section 3: FGQ; Appendix A: group size) with the scale
 * constraints of Section 3 "Casting the FP4 to FP8".
 *
 *   per (n, group j):  S_j = max|W| / 6  (FP32 division);
 *   none: S^_j = S_j                                  -> scale[n,j] = S_j
 *   M1  : S^_j = 2^ceil(log2 S_j)                     -> scale[n] = 2^P, P = max_j ceil(log2 S_j),
 *                                                        shift[n,j] = P - ceil(log2 S_j)
 *   M2  : S^_j = S_max / 2^ceil(log2(S_max / S_j))    -> scale[n] = S_max = max_j S_j,
 *                                                        shift[n,j] = ceil(log2(S_max / S_j))
 *   code = RNE_E2M1( fl32( W[n,k] / S^_j ) ), saturating at +-6.
 * Shifts are stored clamped to [0, 5] (the range in which the cast to E4M3 is a subtraction in the
 * exponent field); a clamped group is quantized with scale[n] * 2^-5.  A group of all zeros takes no
 * part in the row maximum, gets shift 0 (and scale 1 in mode none).
 *
 * W     : FP32 [N, K] dense row-major; 16-byte aligned
 * codes : out, 16-byte aligned, in the layout the GEMM streams (the paper does not fix one): tiles of
 *         128 output rows x 128 input features, tile (nt, kb) at byte offset (nt * (K/128) + kb) * 8448.
 *         A tile is 8192 bytes of codes followed by 256 shift bytes:
 *           - the 16-byte chunk c (elements 32c .. 32c+31 of the K block) of row r sits at (c*128 + r)*16;
 *             its 32-bit word j holds elements 8j .. 8j+7: bits 4i .. 4i+2 = the three E2M1 magnitude
 *             bits (e1 e0 m) of element i, bit 8b+7 = sign of element b, bit 8b+3 = sign of element 4+b
 *             (b = 0..3);
 *           - byte 8192 + 2r + h = the shift of row r for elements 64h .. 64h+63 (0 in mode none).
 *         Rows of the last tile beyond N are zero.
 *         With ZQ_WEIGHTS_MX (M1 / M2 only; ZQ_ERR_MODE otherwise; 32-byte aligned) a block of 128 output rows
 *         takes (K/128) * 8704 bytes, the codes of all its K blocks first and their scales after:
 *           - [kb*8192, +8192): K block kb; row r at r*64, element k of the K block in byte k/2, even k in
 *             the low nibble, a nibble being the E2M1 code s e1 e0 m;
 *           - byte (K/128)*8192 + kb*512 + 16*(r % 32) + 4*(r / 32) + s = 127 - shift of row r for elements
 *             32s .. 32s+31 of K block kb (the E8M0 encoding of 2^-shift), the order in which the tensor
 *             core's scale copy reads them.
 *         Rows beyond N have zero codes and scale bytes 127.
 *         With ZQ_WEIGHTS_MX_FP8 the codes are E4M3 bytes, code = RNE_E4M3(fl32(W / S^)) saturating at +-448
 *         with S_j = max|W| / 448, one byte per element: a block of 128 output rows takes (K/128) * 16896
 *         bytes, [kb*16384, +16384) holding K block kb with row r at r*128, then the scale bytes as above
 *         from (K/128)*16384 on; shifts are stored clamped to [0, 127].
 * shift : out, u8 [N, G] (M1, M2), the same shifts in plain form; ignored (may be NULL) in mode none
 * scale : out, FP32 [N] (M1, M2) or [N, G] (none)
 * group in {64, 128, 256, 320} (320, the paper's choice for a hidden size of 3200, with M1 / M2 only);
 * K % group == 0 and K % 128 == 0; N >= 0.
 */
int zq_pack_weight_fp4(const float* W, int64_t N, int64_t K, int group, zq_scale_mode mode,
                       zq_weight_layout layout, uint8_t* codes, uint8_t* shift, float* scale, void* stream);

/*
 * Workspace for zq_w4a8_linear: a status word, split-K tile counters and partial sums, and (when the
 * call quantizes x itself) q, sx and t.  Zero it ONCE with zq_workspace_init before its first use;
 * the kernels leave the counters zero again.  The size depends only on (M, N, K, r); a workspace
 * sized for M tokens serves every smaller token count at the same (N, K, r).
 */
size_t zq_w4a8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int r);
int zq_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * The quantized linear layer (Section 3):
 *   y[m,n] = sx[m] * sum_k dec_E4M3(q[m,k]) * ( dec_E2M1(code[n,k]) * S^[n, k/group] )
 *            + sum_{j<r} U[n,j] * t[m,j]
 * For M1 / M2 the weight is cast to E4M3 inside the kernel by subtracting shift[n, k/group] from the
 * exponent field (Section 3, "Casting the FP4 to FP8"), the FP8 x FP8 products are accumulated in
 * FP32 over all of K, and sx[m] * scale[n] multiplies the sum once.  With ZQ_WEIGHTS_MX the tensor core
 * performs that cast: it multiplies the E2M1 codes by the E4M3 activations and by 2^-shift as a block
 * scale; the products and their sum are the same numbers.  In mode none the FP32 group scale multiplies
 * each group's partial sum.
 *
 * Activations come either pre-quantized (q, sx, and t when r > 0; x_bf16 = NULL) or raw
 * (x_bf16 [M, ldx] given, q = sx = t = NULL): then the call first runs zq_quantize_act_fp8 into the
 * workspace (with V when r > 0).
 *
 * codes / scale : as written by zq_pack_weight_fp4 for the same (N, K, group, mode, layout); shift is not read
 *                 (the tiles carry the shifts) and may be NULL
 * U : fp16 [N, r] dense or NULL (r = 0);  V : fp16 [r, K], only read when x_bf16 is given and r > 0
 * y : out, [M, ldy] FP32 or bf16 (ydt), ldy >= N in elements
 * K % 128 == 0; group in {64, 128, 256, 320}; r in {0, 8, 16, ..., 64}; q, codes 16-byte aligned (codes 32-byte
 * aligned with ZQ_WEIGHTS_MX).
 * M == 0 or N == 0 is a no-op.  Summation order over K depends on the launch shape, so FP32 results are
 * not bit-identical across token counts.  Where the K range of an output tile is shared by several CTAs
 * and y is FP32 (ZQ_WEIGHTS_CAST: M <= 16; ZQ_WEIGHTS_MX: up to 256 tokens, and larger token counts
 * with fewer than about 600 output tiles of 128 x 192, and the last round of larger ones) the CTAs add
 * their shares into y with FP32 atomics: the last bit can then differ from run to run; other shapes, and
 * bf16 y, are reproducible.
 */
int zq_w4a8_linear(const uint8_t* q, const float* sx, const void* x_bf16, int64_t ldx, int64_t M,
                   int64_t N, int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout,
                   const uint8_t* codes, const uint8_t* shift, const float* scale, const void* U_f16, const void* V_f16,
                   const float* t, int r, void* y, zq_out_dtype ydt, int64_t ldy, void* workspace,
                   size_t workspace_bytes, void* stream);

/*
 * Not an operation of the paper: a promise about how the library is used.  Launches whose CTAs hand shared output
 * tiles over to one another (few tokens: the K range of a tile is split between CTAs; the kernel that quantizes
 * its activations itself) need every CTA of the grid running at the same time.  By default they are cooperative
 * launches, which guarantee it and cost about 3.5 us each.  After zq_set_exclusive_device(1) the caller promises
 * that no other kernel (of any stream or process) runs on the device while such a call executes; the launches
 * are then plain ones, whose grids of at most one CTA per SM are resident as soon as the kernel ahead in the
 * stream has drained.  If the promise is broken, CTAs may wait for CTAs that cannot start: the waits are bounded
 * and the call ends with ZQ_ERR_DEVICE_TIMEOUT in the workspace status, not with a hang.
 * Process-wide; returns the previous setting.
 */
int zq_set_exclusive_device(int on);

/*
 * Fusion on the output side of the layer (Section 3: the next layer quantizes this layer's output token-wise
 * to FP8, Appendix A): zq_w4a8_linear with two additions.
 *   relu      non-zero: y = max(y, 0) before the store (the MLP non-linearity of the OPT family).
 *   y_absmax  device float [M] or NULL: receives, per token, the maximum of |y| over all N outputs, of the
 *             values as they are stored (after relu; after the rounding to bf16 when ydt is bf16).  The call
 *             clears the array first (on the stream) and the epilogues add in with atomic maxima.
 * With these maxima the next layer's quantizer needs no reduction: zq_quantize_act_fp8_scaled below.  (The
 * ReLU costs nothing; the maxima cost a warp reduction and an atomic per token, warp and tile, which pays only
 * for narrow outputs of long rows.)
 * Output tiles shared by several CTAs take the partial-sum route through the workspace here (as for a bf16 y):
 * nobody adds into y, because the final value must be known to the CTA that forms the maximum.
 * Everything else (arguments, workspace, errors) as zq_w4a8_linear.
 */
int zq_w4a8_linear_fused_out(const uint8_t* q, const float* sx, const void* x_bf16, int64_t ldx, int64_t M,
                             int64_t N, int64_t K, int group, zq_scale_mode mode, zq_weight_layout layout,
                             const uint8_t* codes, const uint8_t* shift, const float* scale, const void* U_f16,
                             const void* V_f16, const float* t, int r, void* y, zq_out_dtype ydt, int64_t ldy,
                             void* workspace, size_t workspace_bytes, void* stream, int relu, float* y_absmax);

/*
 * zq_quantize_act_fp8 for a caller that already has the tokens' absolute maxima (Section 3, Appendix A, Eq. 1 with
 * Z = 0: s_x = absmax / 448, q = RNE_E4M3(x * (448 / absmax))): one pass over x, no reduction.
 *   absmax  device float [M]: max_k |x[m, k]| exactly (e.g. from zq_w4a8_linear_fused_out of the layer before);
 *           a value that is not the row's maximum gives codes that differ from zq_quantize_act_fp8's.
 * Other arguments, outputs and errors as zq_quantize_act_fp8.
 */
int zq_quantize_act_fp8_scaled(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* absmax,
                               uint8_t* q, float* sx, const void* V_f16, int r, float* t, void* stream);

/*
 * How zq_w4a8_linear would partition a problem on the current device (no launch; host only).  Not an
 * operation of the paper: it exposes the launch plan so that its arithmetic can be checked without a GPU.
 * Work is counted in units of one 128-element K block of one output tile (128 channels x bm tokens);
 * positions of the launch order map to tiles through groups of m_group token tiles (N outer, the group's
 * token tiles inner; m_group <= 1: along N only).
 *   plan[0] bm, [1] m_tiles, [2] n_tiles, [3] ctas,
 *   [4] stream  (1: the units are dealt out as contiguous ranges, base each, the first rem CTAs one more),
 *   [5] persist (1: CTA c walks whole tiles at positions c, c + ctas, ... below tail_pos0; the units of the
 *                tiles from tail_pos0 on are dealt out as ranges like stream),
 *   [6] splits, [7] kb_per_split (neither stream nor persist: CTA z * tiles + pos takes K blocks
 *                [z * kb_per_split, ...) of the tile at position pos),
 *   [8] base, [9] rem, [10] tail_pos0, [11] m_group, [12] floats of partial-sum scratch, [13] SMs assumed,
 *   [14] pair   (1, with persist: the CTAs work in pairs, CTAs 2c and 2c + 1 on one token tile and two
 *                neighbouring channel tiles; pair c walks the pair positions c, c + ctas / 2, ... of
 *                m_tiles x n_tiles / 2, whole tiles only; a pair position maps to (token tile, channel-tile
 *                pair) through the same groups of m_group token tiles, and CTA 2c + h takes channel tile
 *                2 * pair + h).
 */
#define ZQ_PLAN_WORDS 15
int zq_w4a8_linear_plan(int64_t M, int64_t N, int64_t K, zq_scale_mode mode, zq_weight_layout layout,
                        int64_t* plan);

/*
 * The same layer for callers whose activations live in HOST memory: copies x (bf16 [M, K] dense,
 * host, ideally pinned) to the device, runs quantizer + linear, copies y (FP32 [M, N] dense, host)
 * back and synchronizes the stream before returning.  Weights, U, V and the workspace stay on the
 * device.  The workspace must have zq_w4a8_linear_host_workspace_bytes(M, N, K, r) bytes and must
 * have been zeroed once with zq_workspace_init.  Calls with more than 1024 tokens are cut into row chunks
 * (token rows are independent) whose upload, kernels and download overlap on two copy streams that the
 * library creates on first use, per device, and keeps; the kernels still run on `stream`, and everything
 * has completed when the call returns.
 */
size_t zq_w4a8_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int r);
int zq_w4a8_linear_host(const void* x_bf16_host, int64_t M, int64_t N, int64_t K, int group,
                        zq_scale_mode mode, zq_weight_layout layout, const uint8_t* codes,
                        const uint8_t* shift, const float* scale, const void* U_f16, const void* V_f16, int r,
                        float* y_host, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronizes `stream`, reads the workspace's status word and clears it.  Returns ZQ_OK or
 * ZQ_ERR_DEVICE_TIMEOUT (a kernel's bounded wait on a barrier ran out; its output is invalid and the
 * workspace must be re-initialized).  `detail` (host, may be NULL) receives a code naming the wait.
 */
int zq_device_status(void* workspace, int* detail, void* stream);

/*
 * Construction of the LoRC factors (Section 3, first paragraph; Appendix A: ranks 8 .. 56): the rank-r part of
 * the singular value decomposition of the error matrix E = W - W^ between the original weight and its
 * quantized form (FP4-E2M1 codes with the scales of zq_pack_weight_fp4), the singular values split evenly:
 *   U^ = P_r diag(sigma_r)^(1/2) [N, r],  V^ = diag(sigma_r)^(1/2) Q_r^T [r, K],  E ~ U^ V^.
 * The paper takes a full SVD on the host; here the leading subspace is found by randomized subspace
 * iteration, which needs only products with E and its transpose: `omega` is the caller's draw of a Gaussian
 * test matrix and `iters` the number of power iterations (2 is plenty when E has a spectral gap; the error
 * of a plain quantized weight has a nearly flat spectrum, where more iterations buy little).  Any orthogonal
 * re-mixing of the factors is an equally valid answer: compare U^ V^ or the spanned subspace, not elements.
 *
 * W      : FP32 [N, K] dense, the original weight
 * shift / scale : as written by zq_pack_weight_fp4 for (N, K, group, mode) with ZQ_WEIGHTS_CAST or ZQ_WEIGHTS_MX
 * omega  : FP32 [K, r + 8] dense, independent standard normal draws
 * U_f16  : out, fp16 [N, r];  V_f16 : out, fp16 [r, K];  sigma2 : out, optional, FP32 [r], squares of the r
 *          leading singular values of E
 * workspace : zq_lorc_workspace_bytes(N, K, r) bytes, 256-byte aligned (holds E in FP32 and the iterates)
 * r in {8, 16, ..., 64}; r + 8 <= min(N, K); 0 <= iters <= 8; K % group == 0.
 */
size_t zq_lorc_workspace_bytes(int64_t N, int64_t K, int r);
int zq_lorc_factors(const float* W, int64_t N, int64_t K, int group, zq_scale_mode mode, const uint8_t* shift,
                    const float* scale, int r, const float* omega, int iters, void* U_f16, void* V_f16,
                    float* sigma2, void* workspace, size_t workspace_bytes, void* stream);

/*
 * (No operation of the paper: a check of the library's own failure reporting.)  Launches one CTA that waits,
 * with the wait routine the GEMM kernels use and a limit of `limit_us` microseconds (1 .. 1000000), on a
 * barrier that nothing ever completes.  The wait gives up, the kernel writes ZQ_ERR_DEVICE_TIMEOUT and the
 * detail code 100 into the workspace status words and returns by itself: no trap, no fault, nothing left
 * spinning.  zq_device_status(workspace) then returns ZQ_ERR_DEVICE_TIMEOUT and clears the words; the same
 * workspace is usable again after zq_workspace_init.
 */
int zq_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t limit_us, void* stream);

/*
 * (The paper has no counterpart for this entry point; it exists for deployment reasons only.)
 *
 * zq_w4a8_linear for callers that cannot allocate device memory and therefore have no workspace to
 * hand over: a serving loop whose memory plan is fixed at start-up, a plug-in that receives tensors
 * from a host framework but owns no allocator, a process whose pool already holds the whole device.
 * The split-K counters and partial sums live in a fixed 32 MiB array inside the library
 * (zq_w4a8_linear_noalloc_max_scratch_bytes), resident on every GPU that loads the library until the
 * process exits.  The call allocates and frees nothing.
 *
 * Same operation, arguments and limits as zq_w4a8_linear with weights in the ZQ_WEIGHTS_CAST layout and
 * pre-quantized activations (q, sx, and
 * t when r > 0; there is no raw-x path, since that would need scratch for q).  The fixed array bounds
 * the split-K partial sums (4 bytes x splits x padded M x padded N).  A problem that needs more
 * returns ZQ_ERR_WORKSPACE and launches nothing.  Problems with about 300 or more 128 x 256 output
 * tiles are not split and always fit; so do the M <= 128 cases of layers up to 28672 x 28672.
 * The first call on a device looks up the array's device address (once per device, with that device
 * current); make that first call outside any stream capture.
 * Every call on a device shares the one array: the call clears the counters it needs at zero, but two
 * calls that overlap on the GPU race on it, so issue them on one stream or serialize them yourself.
 * The workspace of zq_device_status does not exist here; zq_w4a8_linear_noalloc_status is its counterpart:
 * it synchronizes `stream`, reads the status words at the head of the array on the current device and
 * clears them; ZQ_OK, or ZQ_ERR_DEVICE_TIMEOUT with `detail` (host, may be NULL) naming the wait that ran
 * out in some call since the last query (that call's y is invalid).  It allocates nothing either.
 */
size_t zq_w4a8_linear_noalloc_max_scratch_bytes(void);
int zq_w4a8_linear_noalloc(const uint8_t* q, const float* sx, int64_t M, int64_t N, int64_t K, int group,
                           zq_scale_mode mode, const uint8_t* codes, const uint8_t* shift,
                           const float* scale, const void* U_f16, const float* t, int r, void* y,
                           zq_out_dtype ydt, int64_t ldy, void* stream);
int zq_w4a8_linear_noalloc_status(int* detail, void* stream);

/* Number of kernels of this library launched by the calling process so far (all entry points). */
int64_t zq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ZQFP_H_ */
