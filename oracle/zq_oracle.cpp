// CPU oracle for the W4A8 quantized linear layer of ZeroQuant-FP.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
// checked against.  It shares no code with the CUDA path and nothing in the product may call it.
//
// What it states, and where the paper defines it:
//   * ExMy minifloat formats (Section 2, "ExMy notation": x exponent bits, y mantissa bits,
//     7 bits in total for FP8 and 3 for FP4; Section 4 picks E4M3 and E2M1).
//   * token-wise activation quantization and fine-grained (group-wise) weight quantization
//     (Section 3, first paragraph; Appendix A), symmetric, i.e. Eq. 1 with Z = 0.
//   * the two power-of-two scale constraints (Section 3, "Casting the FP4 to FP8", items M1, M2)
//     and the cast FP4 -> FP8 as an exponent shift that they make possible.
//   * LoRC: a rank-r product added to the quantized weight (Section 3, first paragraph).
//
// Arithmetic: single FP32 operations where the method fixes the precision of a decision
// (scales, the value handed to a rounding), FP64 everywhere else.  No blocking, no fusion,
// no reordering; OpenMP only splits loops over independent rows.
//
// Beyond the hot path, for the variants and comparisons of Sections 2-4 and the appendix: the E5M2 and E3M0
// formats, FP8 weights (W8A8), any shift range (E5M2 as the cast target reaches 13), the uniform integer
// quantizer of Eq. 1, and the construction of the LoRC factors by SVD.  Those live in the second extern "C"
// block at the end of the file and leave the functions above them untouched.
//
// Parity status: every function below is pinned by the CPU tests (format tables typed from the
// format definitions, closed forms of M1/M2, brute force in Python on tiny inputs).  The
// paper-level quantities (perplexities) are "parity unpinned": they need models and corpora.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// storage-type helpers (exact conversions, no rounding involved)
// ---------------------------------------------------------------------------------------------
inline float bf16_bits_to_float(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// IEEE binary16 -> double, by the definition of the format.
inline double f16_bits_to_double(uint16_t h) {
  int s = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
  double v;
  if (e == 0) v = std::ldexp(static_cast<double>(m), -24);
  else if (e == 31) v = m ? std::numeric_limits<double>::quiet_NaN()
                          : std::numeric_limits<double>::infinity();
  else v = std::ldexp(1.0 + m / 1024.0, e - 15);
  return s ? -v : v;
}

// ---------------------------------------------------------------------------------------------
// ExMy minifloat (Section 2).  E exponent bits, Mn mantissa bits, IEEE-style bias 2^(E-1)-1,
// gradual underflow.  `vmax` is the largest finite magnitude of the format as used here:
//   E2M1: all 16 codes are finite numbers, largest 6.
//   E4M3: the hardware variant, where exponent 15 / mantissa 7 is NaN and nothing is infinite,
//         largest 448 (Section 2 footnote: the paper's simulator did not reserve that pattern).
// ---------------------------------------------------------------------------------------------
struct MiniFloat {
  int E, Mn, bias;
  double vmax;
  int nan_code;  // magnitude bits of the NaN pattern, or -1 when the format has none
  bool ieee_top = false;  // the largest exponent field encodes infinity (mantissa 0) and NaN, as in IEEE 754
};
const MiniFloat kE2M1{2, 1, 1, 6.0, -1};
const MiniFloat kE4M3{4, 3, 7, 448.0, 0x7F};

double mf_decode(const MiniFloat& f, unsigned code) {
  const unsigned mag_bits = f.E + f.Mn;
  unsigned s = (code >> mag_bits) & 1u;
  unsigned mag = code & ((1u << mag_bits) - 1u);
  if (f.nan_code >= 0 && static_cast<int>(mag) == f.nan_code)
    return std::numeric_limits<double>::quiet_NaN();
  unsigned e = mag >> f.Mn, m = mag & ((1u << f.Mn) - 1u);
  if (f.ieee_top && e == (1u << f.E) - 1u) {
    if (m) return std::numeric_limits<double>::quiet_NaN();
    return s ? -std::numeric_limits<double>::infinity() : std::numeric_limits<double>::infinity();
  }
  double frac = static_cast<double>(m) / static_cast<double>(1u << f.Mn);
  double v = (e == 0) ? std::ldexp(frac, 1 - f.bias)          // subnormal: 0.m * 2^(1-bias)
                      : std::ldexp(1.0 + frac, static_cast<int>(e) - f.bias);
  return s ? -v : v;
}

// Round-to-nearest, ties to the even mantissa, saturating to +-vmax (no infinities).
unsigned mf_encode(const MiniFloat& f, float vin) {
  const unsigned mag_bits = f.E + f.Mn;
  uint32_t vb;
  std::memcpy(&vb, &vin, 4);
  const unsigned sign = (vb >> 31) << mag_bits;
  if (std::isnan(vin)) {
    if (f.ieee_top) return sign | (((1u << f.E) - 1u) << f.Mn) | 1u;
    return sign | static_cast<unsigned>(f.nan_code >= 0 ? f.nan_code : 0);
  }
  double a = std::fabs(static_cast<double>(vin));
  const int emin = 1 - f.bias;
  double r;  // the rounded magnitude
  if (std::isinf(a)) {
    r = f.vmax;
  } else if (a == 0.0) {
    r = 0.0;
  } else {
    int ex;
    std::frexp(a, &ex);          // a = frac * 2^ex, frac in [0.5, 1)  =>  floor(log2 a) = ex - 1
    int e = ex - 1;
    if (e < emin) e = emin;      // below the smallest normal the spacing stays that of emin
    double quantum = std::ldexp(1.0, e - f.Mn);
    // a / quantum is exact (power of two); nearbyint rounds ties to even in the default mode,
    // and an even multiple of the quantum is an even mantissa field.
    r = std::nearbyint(a / quantum) * quantum;
    if (r > f.vmax) r = f.vmax;
  }
  // write r (exactly representable now) into its fields
  unsigned mag;
  if (r == 0.0) {
    mag = 0;
  } else {
    int ex;
    double frac = std::frexp(r, &ex);  // r = frac * 2^ex
    int e = ex - 1;
    if (e < emin) {                    // subnormal: r = m * 2^(emin - Mn)
      mag = static_cast<unsigned>(std::ldexp(r, f.Mn - emin));
    } else {
      unsigned m = static_cast<unsigned>(std::ldexp(frac * 2.0 - 1.0, f.Mn));
      mag = (static_cast<unsigned>(e + f.bias) << f.Mn) | m;
    }
  }
  return sign | mag;
}

// floor(log2 v) and whether v is an exact power of two, for finite v > 0 (subnormals included).
inline void log2_parts(float v, int* floor_log2, bool* is_pow2) {
  int ex;
  double frac = std::frexp(static_cast<double>(v), &ex);
  *floor_log2 = ex - 1;
  *is_pow2 = (frac == 0.5);
}

inline int ceil_log2(float v) {
  int fl;
  bool p2;
  log2_parts(v, &fl, &p2);
  return p2 ? fl : fl + 1;
}

// E5M2 keeps the IEEE top exponent for infinities and NaNs (largest finite value 57344); mf_decode and
// mf_encode treat it through `ieee_top`.  E3M0 (Appendix A, Table A.1) has no mantissa bit: powers of two
// 2^-2 .. 2^4 and zero.
const MiniFloat kE5M2{5, 2, 15, 57344.0, -1, true};
const MiniFloat kE3M0{3, 0, 3, 16.0, -1, false};

const int kShiftMax = 5;  // largest exponent shift for which every non-zero E2M1 value stays a normal E4M3 number

}  // namespace

extern "C" {

enum { ORC_SCALE_NONE = 0, ORC_SCALE_M1 = 1, ORC_SCALE_M2 = 2 };

// ---- formats (Section 2) --------------------------------------------------------------------
double orc_e2m1_decode(unsigned code) { return mf_decode(kE2M1, code & 0xFu); }
unsigned orc_e2m1_encode(float v) { return mf_encode(kE2M1, v); }
double orc_e4m3_decode(unsigned code) { return mf_decode(kE4M3, code & 0xFFu); }
unsigned orc_e4m3_encode(float v) { return mf_encode(kE4M3, v); }

// ---- the cast FP4 -> FP8 as an exponent shift (Section 3, "Casting the FP4 to FP8") ----------
// Returns the E4M3 byte whose value is decode_e2m1(code) * 2^-shift.  Stated here through the
// value (decode, scale by a power of two, encode); the tests check that this never rounds for
// 0 <= shift <= 5, which is what makes the cast a pure shift of the exponent field.
unsigned orc_widen_e2m1_to_e4m3(unsigned code, int shift) {
  double v = std::ldexp(mf_decode(kE2M1, code & 0xFu), -shift);
  return mf_encode(kE4M3, static_cast<float>(v));
}

// ---- token-wise FP8 activation quantization (Section 3; Appendix A) --------------------------
// x: bf16 bit patterns [M, ldx]; q: E4M3 bytes [M, K]; sx: [M]; optional LoRC down-projection
// t[m, j] = sum_k V[j, k] * x[m, k] with the raw x (V: fp16 bits [r, K]; t: double [M, r]).
int orc_quantize_act_fp8(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, uint8_t* q,
                         float* sx, const uint16_t* V, int r, double* t) {
  if (!x || !q || !sx || M < 0 || K <= 0 || ldx < K) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    const uint16_t* row = x + m * ldx;
    float a = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      float v = std::fabs(bf16_bits_to_float(row[k]));
      if (v > a) a = v;  // NaN never wins the comparison
    }
    float s, inv;
    if (a == 0.0f) {
      s = 1.0f;
      inv = 1.0f;
    } else {
      s = a / 448.0f;    // one FP32 division each
      inv = 448.0f / a;
    }
    sx[m] = s;
    for (int64_t k = 0; k < K; ++k) {
      volatile float scaled = bf16_bits_to_float(row[k]) * inv;  // one FP32 multiply, then one rounding to E4M3
      q[m * K + k] = static_cast<uint8_t>(mf_encode(kE4M3, scaled));
    }
    if (V && t && r > 0) {
      for (int j = 0; j < r; ++j) {
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
          acc += f16_bits_to_double(V[j * K + k]) * static_cast<double>(bf16_bits_to_float(row[k]));
        t[m * r + j] = acc;
      }
    }
  }
  return 0;
}

// ---- fine-grained FP4 weight quantization with scale constraints (Section 3, M1 / M2) --------
// W: fp32 [N, K]; group: elements of one row sharing a scale; codes: [N, K/2], element 2b in the
// low nibble of byte b and element 2b+1 in the high nibble.
// mode none : scale[n, j] = S = absmax / 6                                   (shift unused)
// mode M1   : S^ = 2^ceil(log2 S); stored as scale[n] = 2^P, P = max_j ceil(log2 S_j), and
//             shift[n, j] = P - ceil(log2 S_j)
// mode M2   : S^_j = S_max / 2^ceil(log2(S_max / S_j)); stored as scale[n] = S_max and
//             shift[n, j] = ceil(log2(S_max / S_j)); codes saturate at +-6
// A shift larger than 5 is stored as 5 and the group is quantized with the scale that the stored
// shift stands for.  A group whose elements are all zero takes no part in the row maximum and
// gets shift 0.
int orc_pack_weight_fp4(const float* W, int64_t N, int64_t K, int group, int mode, uint8_t* codes,
                        uint8_t* shift, float* scale) {
  if (!W || !codes || !scale || N < 0 || K <= 0 || group <= 0 || K % group || (K & 1)) return -1;
  if (mode != ORC_SCALE_NONE && !shift) return -1;
  const int64_t G = K / group;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    const float* row = W + n * K;
    std::vector<float> S(G);       // the unconstrained scale of each group; 0 marks an all-zero group
    for (int64_t j = 0; j < G; ++j) {
      float a = 0.0f;
      for (int k = 0; k < group; ++k) {
        float v = std::fabs(row[j * group + k]);
        if (v > a) a = v;
      }
      S[j] = (a == 0.0f) ? 0.0f : a / 6.0f;  // FP32 division
    }
    std::vector<float> Shat(G);    // the scale each group is actually quantized with
    if (mode == ORC_SCALE_NONE) {
      for (int64_t j = 0; j < G; ++j) {
        Shat[j] = (S[j] == 0.0f) ? 1.0f : S[j];
        scale[n * G + j] = Shat[j];
      }
    } else if (mode == ORC_SCALE_M1) {
      bool any = false;
      int P = 0;
      for (int64_t j = 0; j < G; ++j)
        if (S[j] != 0.0f) {
          int p = ceil_log2(S[j]);
          if (!any || p > P) P = p;
          any = true;
        }
      scale[n] = static_cast<float>(std::ldexp(1.0, P));
      for (int64_t j = 0; j < G; ++j) {
        int d = 0;
        if (S[j] != 0.0f) d = P - ceil_log2(S[j]);
        if (d > kShiftMax) d = kShiftMax;
        shift[n * G + j] = static_cast<uint8_t>(d);
        Shat[j] = static_cast<float>(std::ldexp(1.0, P - d));
      }
    } else {  // M2
      float Smax = 0.0f;
      for (int64_t j = 0; j < G; ++j)
        if (S[j] > Smax) Smax = S[j];
      if (Smax == 0.0f) Smax = 1.0f;
      scale[n] = Smax;
      for (int64_t j = 0; j < G; ++j) {
        int d = 0;
        if (S[j] != 0.0f) {
          // ceil(log2(Smax / S_j)) = the smallest d >= 0 with S_j * 2^d >= Smax (exact in double)
          while (d < 400 && std::ldexp(static_cast<double>(S[j]), d) < static_cast<double>(Smax)) ++d;
        }
        if (d > kShiftMax) d = kShiftMax;
        shift[n * G + j] = static_cast<uint8_t>(d);
        Shat[j] = static_cast<float>(std::ldexp(static_cast<double>(Smax), -d));
      }
    }
    for (int64_t b = 0; b < K / 2; ++b) {
      unsigned byte = 0;
      for (int h = 0; h < 2; ++h) {
        int64_t k = 2 * b + h;
        volatile float ratio = row[k] / Shat[k / group];  // FP32 division, then one rounding to E2M1
        byte |= (mf_encode(kE2M1, ratio) & 0xFu) << (4 * h);
      }
      codes[n * (K / 2) + b] = static_cast<uint8_t>(byte);
    }
  }
  return 0;
}

// The scale that group (n, j) was quantized with, as a double, from the stored fields.
double orc_group_scale(int mode, const uint8_t* shift, const float* scale, int64_t n, int64_t j,
                       int64_t G) {
  if (mode == ORC_SCALE_NONE) return static_cast<double>(scale[n * G + j]);
  return std::ldexp(static_cast<double>(scale[n]), -static_cast<int>(shift[n * G + j]));
}

// ---- the quantized linear layer with LoRC (Section 3) ----------------------------------------
// y[m, n] = sum_k (dec_e4m3(q[m,k]) * sx[m]) * (dec_e2m1(code[n,k]) * S^[n, k/group])
//           + sum_j U[n, j] * t[m, j]
// in FP64.  `rows` (may be NULL = all) lists the token rows m to evaluate; y is [nrows, N].
int orc_w4a8_linear(const uint8_t* q, const float* sx, int64_t M, int64_t N, int64_t K, int group,
                    int mode, const uint8_t* codes, const uint8_t* shift, const float* scale,
                    const uint16_t* U, const double* t, int r, const int64_t* rows, int64_t nrows,
                    double* y) {
  if (!q || !sx || !codes || !scale || !y || K <= 0 || group <= 0 || K % group) return -1;
  if (mode != ORC_SCALE_NONE && !shift) return -1;
  const int64_t G = K / group;
  if (!rows) nrows = M;
#pragma omp parallel for schedule(dynamic, 16) collapse(2)
  for (int64_t i = 0; i < nrows; ++i) {
    for (int64_t n = 0; n < N; ++n) {
      const int64_t m = rows ? rows[i] : i;
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double xhat = mf_decode(kE4M3, q[m * K + k]) * static_cast<double>(sx[m]);
        unsigned byte = codes[n * (K / 2) + k / 2];
        unsigned code = (k & 1) ? (byte >> 4) : (byte & 0xFu);
        double what = mf_decode(kE2M1, code) * orc_group_scale(mode, shift, scale, n, k / group, G);
        acc += xhat * what;
      }
      if (U && t && r > 0)
        for (int j = 0; j < r; ++j) acc += f16_bits_to_double(U[n * r + j]) * t[m * r + j];
      y[i * N + n] = acc;
    }
  }
  return 0;
}

// The same layer written the way the constrained modes are meant to be executed: the weight is
// first cast to E4M3 by the exponent shift, the contraction runs over the two 8-bit operands, and
// the token scale and the channel scale multiply the sum once.  Used by the tests to show that the
// shift form equals the scale form above (M1 / M2 only).
int orc_w4a8_linear_shift_form(const uint8_t* q, const float* sx, int64_t M, int64_t N, int64_t K,
                               int group, const uint8_t* codes, const uint8_t* shift,
                               const float* chan_scale, double* y) {
  if (!q || !sx || !codes || !shift || !chan_scale || !y || K % group) return -1;
  const int64_t G = K / group;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        unsigned byte = codes[n * (K / 2) + k / 2];
        unsigned code = (k & 1) ? (byte >> 4) : (byte & 0xFu);
        unsigned w8 = orc_widen_e2m1_to_e4m3(code, shift[n * G + k / group]);
        acc += mf_decode(kE4M3, q[m * K + k]) * mf_decode(kE4M3, w8);
      }
      y[m * N + n] = acc * static_cast<double>(sx[m]) * static_cast<double>(chan_scale[n]);
    }
  return 0;
}

int orc_num_threads(void) {
  int n = 1;
#pragma omp parallel
  {
#pragma omp master
    {
#ifdef _OPENMP
      n = omp_get_num_threads();
#endif
    }
  }
  return n;
}

}  // extern "C"

// =============================================================================================
// Variants and comparisons (additions; nothing above depends on them)
// =============================================================================================
namespace {

const MiniFloat* weight_format(int wfmt) {
  switch (wfmt) {
    case 0: return &kE2M1;
    case 1: return &kE4M3;
    case 2: return &kE3M0;
  }
  return nullptr;
}

// One-sided (Hestenes) Jacobi SVD of A [m x n], m >= n, in FP64: rotates pairs of columns of A until all are
// mutually orthogonal, accumulating the rotations in Vt.  On return the columns of A are U * diag(sigma).
void jacobi_svd(std::vector<double>& A, int64_t m, int64_t n, std::vector<double>& V) {
  V.assign(static_cast<size_t>(n) * n, 0.0);
  for (int64_t i = 0; i < n; ++i) V[i * n + i] = 1.0;
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0.0;
    for (int64_t p = 0; p < n - 1; ++p)
      for (int64_t q = p + 1; q < n; ++q) {
        double alpha = 0.0, beta = 0.0, gamma = 0.0;
        for (int64_t i = 0; i < m; ++i) {
          alpha += A[i * n + p] * A[i * n + p];
          beta += A[i * n + q] * A[i * n + q];
          gamma += A[i * n + p] * A[i * n + q];
        }
        if (gamma == 0.0 || alpha == 0.0 || beta == 0.0) continue;
        const double rel = std::fabs(gamma) / std::sqrt(alpha * beta);
        if (rel > off) off = rel;
        if (rel < 1e-15) continue;
        const double zeta = (beta - alpha) / (2.0 * gamma);
        const double tt = (zeta >= 0.0 ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
        const double c = 1.0 / std::sqrt(1.0 + tt * tt), sn = c * tt;
        for (int64_t i = 0; i < m; ++i) {
          const double ap = A[i * n + p], aq = A[i * n + q];
          A[i * n + p] = c * ap - sn * aq;
          A[i * n + q] = sn * ap + c * aq;
        }
        for (int64_t i = 0; i < n; ++i) {
          const double vp = V[i * n + p], vq = V[i * n + q];
          V[i * n + p] = c * vp - sn * vq;
          V[i * n + q] = sn * vp + c * vq;
        }
      }
    if (off < 1e-14) break;
  }
}

}  // namespace

extern "C" {

double orc_e5m2_decode(unsigned code) { return mf_decode(kE5M2, code & 0xFFu); }
unsigned orc_e5m2_encode(float v) { return mf_encode(kE5M2, v); }
double orc_e3m0_decode(unsigned code) { return mf_decode(kE3M0, code & 0xFu); }
unsigned orc_e3m0_encode(float v) { return mf_encode(kE3M0, v); }

// The cast FP4 -> FP8 with E5M2 as the target (Section 3, footnote to "Casting the FP4 to FP8"): the E5M2
// byte whose value is decode_e2m1(code) * 2^-shift.  With five exponent bits every non-zero E2M1 value stays
// a normal number down to shift 13, so there the cast is a subtraction of the shift from the exponent field.
unsigned orc_widen_e2m1_to_e5m2(unsigned code, int shift) {
  double v = std::ldexp(mf_decode(kE2M1, code & 0xFu), -shift);
  return mf_encode(kE5M2, static_cast<float>(v));
}

// Fine-grained weight quantization as orc_pack_weight_fp4, for any of the weight formats of the paper's
// tables (wfmt 0: FP4-E2M1, 1: FP8-E4M3 as in the W8A8 rows of Table 2, 2: FP4-E3M0 as in Table A.1) and any
// clamp of the stored shift (5 for the E4M3 cast target, 13 for E5M2, 127 for a power-of-two block scale).
// The unconstrained scale of a group is absmax / vmax(format).  codes: one byte per element, [N, K].
int orc_pack_weight(const float* W, int64_t N, int64_t K, int group, int mode, int wfmt, int max_shift,
                    uint8_t* codes, uint8_t* shift, float* scale) {
  const MiniFloat* fmt = weight_format(wfmt);
  if (!fmt || !W || !codes || !scale || N < 0 || K <= 0 || group <= 0 || K % group || max_shift < 0) return -1;
  if (mode != ORC_SCALE_NONE && !shift) return -1;
  const int64_t G = K / group;
  const float vmax = static_cast<float>(fmt->vmax);
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    const float* row = W + n * K;
    std::vector<float> S(G), Shat(G);
    for (int64_t j = 0; j < G; ++j) {
      float a = 0.0f;
      for (int k = 0; k < group; ++k) {
        float v = std::fabs(row[j * group + k]);
        if (v > a) a = v;
      }
      S[j] = (a == 0.0f) ? 0.0f : a / vmax;  // FP32 division
    }
    if (mode == ORC_SCALE_NONE) {
      for (int64_t j = 0; j < G; ++j) {
        Shat[j] = (S[j] == 0.0f) ? 1.0f : S[j];
        scale[n * G + j] = Shat[j];
      }
    } else if (mode == ORC_SCALE_M1) {
      bool any = false;
      int P = 0;
      for (int64_t j = 0; j < G; ++j)
        if (S[j] != 0.0f) {
          int p = ceil_log2(S[j]);
          if (!any || p > P) P = p;
          any = true;
        }
      scale[n] = static_cast<float>(std::ldexp(1.0, P));
      for (int64_t j = 0; j < G; ++j) {
        int d = 0;
        if (S[j] != 0.0f) d = P - ceil_log2(S[j]);
        if (d > max_shift) d = max_shift;
        shift[n * G + j] = static_cast<uint8_t>(d);
        Shat[j] = static_cast<float>(std::ldexp(1.0, P - d));
      }
    } else {
      float Smax = 0.0f;
      for (int64_t j = 0; j < G; ++j)
        if (S[j] > Smax) Smax = S[j];
      if (Smax == 0.0f) Smax = 1.0f;
      scale[n] = Smax;
      for (int64_t j = 0; j < G; ++j) {
        int d = 0;
        if (S[j] != 0.0f)
          while (d < 400 && std::ldexp(static_cast<double>(S[j]), d) < static_cast<double>(Smax)) ++d;
        if (d > max_shift) d = max_shift;
        shift[n * G + j] = static_cast<uint8_t>(d);
        Shat[j] = static_cast<float>(std::ldexp(static_cast<double>(Smax), -d));
      }
    }
    for (int64_t k = 0; k < K; ++k) {
      volatile float ratio = row[k] / Shat[k / group];  // FP32 division, then one rounding to the format
      codes[n * K + k] = static_cast<uint8_t>(mf_encode(*fmt, ratio));
    }
  }
  return 0;
}

// The quantized linear layer as orc_w4a8_linear, for weights from orc_pack_weight (one code byte per element).
int orc_linear_general(const uint8_t* q, const float* sx, int64_t M, int64_t N, int64_t K, int group, int mode,
                       int wfmt, const uint8_t* codes, const uint8_t* shift, const float* scale,
                       const uint16_t* U, const double* t, int r, const int64_t* rows, int64_t nrows, double* y) {
  const MiniFloat* fmt = weight_format(wfmt);
  if (!fmt || !q || !sx || !codes || !scale || !y || K <= 0 || group <= 0 || K % group) return -1;
  if (mode != ORC_SCALE_NONE && !shift) return -1;
  const int64_t G = K / group;
  if (!rows) nrows = M;
#pragma omp parallel for schedule(dynamic, 16) collapse(2)
  for (int64_t i = 0; i < nrows; ++i) {
    for (int64_t n = 0; n < N; ++n) {
      const int64_t m = rows ? rows[i] : i;
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double xhat = mf_decode(kE4M3, q[m * K + k]) * static_cast<double>(sx[m]);
        double what = mf_decode(*fmt, codes[n * K + k]) * orc_group_scale(mode, shift, scale, n, k / group, G);
        acc += xhat * what;
      }
      if (U && t && r > 0)
        for (int j = 0; j < r; ++j) acc += f16_bits_to_double(U[n * r + j]) * t[m * r + j];
      y[i * N + n] = acc;
    }
  }
  return 0;
}

// The uniform integer quantizer of Eq. 1 (Section 2, "The Uniform Quantization of INT8") on one vector, with
// its dequantized values as the result.  Symmetric (Z = 0): S = absmax / (2^(bits-1) - 1), levels
// -(2^(bits-1) - 1) .. 2^(bits-1) - 1.  Asymmetric: the zero point is the vector's minimum,
// S = (max - min) / (2^bits - 1), levels 0 .. 2^bits - 1.  Rounding to nearest, ties to even; FP64.
int orc_int_fake_quant(const double* x, int64_t n, int bits, int symmetric, double* out) {
  if (!x || !out || n < 0 || bits < 2 || bits > 16) return -1;
  if (n == 0) return 0;
  double lo = x[0], hi = x[0], amax = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    if (x[i] < lo) lo = x[i];
    if (x[i] > hi) hi = x[i];
    if (std::fabs(x[i]) > amax) amax = std::fabs(x[i]);
  }
  if (symmetric) {
    const double qmax = std::ldexp(1.0, bits - 1) - 1.0;
    const double S = amax == 0.0 ? 1.0 : amax / qmax;
    for (int64_t i = 0; i < n; ++i) {
      double lv = std::nearbyint(x[i] / S);
      if (lv > qmax) lv = qmax;
      if (lv < -qmax) lv = -qmax;
      out[i] = lv * S;
    }
  } else {
    const double qmax = std::ldexp(1.0, bits) - 1.0;
    const double S = hi == lo ? 1.0 : (hi - lo) / qmax;
    for (int64_t i = 0; i < n; ++i) {
      double lv = std::nearbyint((x[i] - lo) / S);
      if (lv > qmax) lv = qmax;
      if (lv < 0.0) lv = 0.0;
      out[i] = lv * S + lo;
    }
  }
  return 0;
}

// Dequantized value of every element of a vector quantized to a minifloat format with one scale
// absmax / vmax (symmetric, Eq. 1's FP counterpart): fmt 0 E2M1, 1 E4M3, 2 E3M0, 3 E5M2.
int orc_fp_fake_quant(const double* x, int64_t n, int fmt_id, double* out) {
  const MiniFloat* fmt = fmt_id == 3 ? &kE5M2 : weight_format(fmt_id);
  if (!fmt || !x || !out || n < 0) return -1;
  double amax = 0.0;
  for (int64_t i = 0; i < n; ++i)
    if (std::fabs(x[i]) > amax) amax = std::fabs(x[i]);
  const double S = amax == 0.0 ? 1.0 : amax / fmt->vmax;
  for (int64_t i = 0; i < n; ++i) out[i] = mf_decode(*fmt, mf_encode(*fmt, static_cast<float>(x[i] / S))) * S;
  return 0;
}

// LoRC factors (Section 3, first paragraph): the singular value decomposition E = P diag(sigma) Q^T of the
// error matrix E = W - W^ [N x K], truncated to rank r and split evenly between the two factors:
//   U^ = P_r diag(sigma_r)^(1/2)  [N x r],   V^ = diag(sigma_r)^(1/2) Q_r^T  [r x K],   so that U^ V^ is the
// best rank-r approximation of E.  sigma (all min(N, K) values, descending) is returned too.
int orc_lorc_factors(const double* E, int64_t N, int64_t K, int r, double* U, double* V, double* sigma) {
  if (!E || !U || !V || N <= 0 || K <= 0 || r <= 0 || r > N || r > K) return -1;
  const bool tall = N >= K;
  const int64_t m = tall ? N : K, n = tall ? K : N;
  std::vector<double> A(static_cast<size_t>(m) * n), Vr;
  for (int64_t i = 0; i < m; ++i)
    for (int64_t j = 0; j < n; ++j) A[i * n + j] = tall ? E[i * K + j] : E[j * K + i];  // A = E or E^T
  jacobi_svd(A, m, n, Vr);
  std::vector<double> sg(n);
  std::vector<int64_t> order(n);
  for (int64_t j = 0; j < n; ++j) {
    double ss = 0.0;
    for (int64_t i = 0; i < m; ++i) ss += A[i * n + j] * A[i * n + j];
    sg[j] = std::sqrt(ss);
    order[j] = j;
  }
  for (int64_t a = 0; a < n; ++a)  // selection sort, descending
    for (int64_t b = a + 1; b < n; ++b)
      if (sg[order[b]] > sg[order[a]]) std::swap(order[a], order[b]);
  if (sigma)
    for (int64_t j = 0; j < n; ++j) sigma[j] = sg[order[j]];
  for (int c = 0; c < r; ++c) {
    const int64_t j = order[c];
    const double s = sg[j], rs = std::sqrt(s);
    // left vector of A: column j of A / s (length m); right vector of A: column j of Vr (length n)
    for (int64_t i = 0; i < m; ++i) {
      const double left = s > 0.0 ? A[i * n + j] / s : 0.0;
      if (tall) U[i * r + c] = left * rs;   // A = E: left vectors are E's
      else V[c * K + i] = left * rs;        // A = E^T: left vectors of A are E's right vectors
    }
    for (int64_t i = 0; i < n; ++i) {
      const double right = Vr[i * n + j];
      if (tall) V[c * K + i] = right * rs;
      else U[i * r + c] = right * rs;
    }
  }
  return 0;
}

}  // extern "C"
