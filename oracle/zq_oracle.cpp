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
  if (std::isnan(vin)) return sign | static_cast<unsigned>(f.nan_code >= 0 ? f.nan_code : 0);
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
