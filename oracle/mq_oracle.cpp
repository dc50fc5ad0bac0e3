// mq_oracle.cpp -- CPU oracle for the MicroQonv hot path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct restatement of what the path computes, written from the
// paper's equations and the OCP MX element definitions it cites.  It shares no code, header,
// table or constant generator with the CUDA library and is used only by the tests, by the
// smoke check and by the benchmark's CPU-baseline leg.  Nothing here is tuned; OpenMP is
// applied to outermost loops only so the big parity cases finish in seconds.
//
// Parity pins (tests marked "not gpu"): every function below is pinned -- element decode/encode
// against closed forms and library casts, the scale against 2^(floor(log2 amax) - emax), the
// quantizer against hand-derived block vectors and invariants, the im2col against a second
// index derivation, the three convolutions against a float64 library convolution, the GEMM
// formulation of Sec. II-C and the adjoint identities.
//
// Notation follows the paper: X in R^{N.Cin.Hin.Win}, W in R^{Cout.Cin.Kh.Kw},
// G_Y in R^{N.Cout.Hout.Wout} (Sec. II-A); X_{Cin,N}, X'_{Cin,N}, W_{f Cout,Cin},
// G_{Yf Cout,N} (Sec. IV-A, IV-B).
//
// Readings of the paper taken here (the paper is silent or uses another variant):
//  * block scale is E8M0 (the "original microscaling format", Sec. II-D) with the OCP floor
//    rule, no per-tensor scale; elements E2M1 / E4M3 / E5M2 / E3M2 / E2M3, round-to-nearest-even, saturating;
//  * a quantization block is a br x bc rectangle over the two axes Sec. IV-B names for each
//    tensor (X: N x Cin, W: Cout x Cin, G_Y: N x Cout) at one spatial / tap position;
//    32 x 32 is the square of Sec. IV-B with sqrt(B) = 32, 1 x 32 is the line block of Sec. III-A;
//  * stored order inside a spatial position is [n][c] with c fastest ("channel-batch-first");
//  * the paper's own number format (Sec. III-A, Eq. 4-6: an fp32 scale per tensor, an E4M3 scale per block, E2M1
//    elements) is provided beside the E8M0 one (orc_quantize_ts and friends).  The paper does not say in which precision
//    Eq. 4-6 are evaluated; since their roundings decide integer codes, they are evaluated here in IEEE single precision,
//    one rounding per written operation, in the order the equations are written - the precision of the tensors they act on.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <cstdlib>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// Problem statement of Sec. II-A, with the stride / padding the evaluation uses (Sec. IV-C).
struct Conv {
  int N, Cin, H, W, Cout, Kh, Kw, sh, sw, ph, pw;
  int Ho() const { return (H + 2 * ph - Kh) / sh + 1; }
  int Wo() const { return (W + 2 * pw - Kw) / sw + 1; }
};
Conv conv_from(const int* d) {
  Conv c{d[0], d[1], d[2], d[3], d[4], d[5], d[6], d[7], d[8], d[9], d[10]};
  return c;
}

enum Fmt { E4M3 = 0, E5M2 = 1, E2M1 = 2, E3M2 = 3, E2M3 = 4 };
enum Role { ROLE_X = 0, ROLE_W = 1, ROLE_DY = 2 };

// ---- element formats (OCP MX v1.0 / OFP8 definitions cited in Sec. II-D) -------------------
// bits: width of a code, sign included; store_bits: bits a code occupies in the stored tensor (the 6-bit formats of
// MicroQonv+ / "-6", Sec. V, are kept one code per byte, value in the low six bits)
struct FmtInfo { int ebits, mbits, bias, emax, max_code, bits, store_bits; };
FmtInfo fmt_info(int fmt) {
  switch (fmt) {
    case E4M3: return {4, 3, 7, 8, 0x7E, 8, 8};    // no Inf; S.1111.111 is NaN; max 448
    case E5M2: return {5, 2, 15, 15, 0x7B, 8, 8};  // IEEE-like: 0x7C Inf, 0x7D..0x7F NaN; max 57344
    case E3M2: return {3, 2, 3, 4, 0x1F, 6, 8};    // no Inf/NaN; max 1.75 * 2^4 = 28
    case E2M3: return {2, 3, 1, 2, 0x1F, 6, 8};    // no Inf/NaN; max 1.875 * 2^2 = 7.5
    default:   return {2, 1, 1, 2, 0x7, 4, 4};     // E2M1: no Inf/NaN; max 6
  }
}

// value of the magnitude bits `m` (sign stripped) of a finite code, from the field definition:
// exponent field 0 -> subnormal  mant * 2^(1-bias-mbits);  else (2^mbits + mant) * 2^(e-bias-mbits)
double decode_mag(int fmt, int m) {
  FmtInfo f = fmt_info(fmt);
  int e = m >> f.mbits;
  int mant = m & ((1 << f.mbits) - 1);
  if (e == 0) return std::ldexp((double)mant, 1 - f.bias - f.mbits);
  return std::ldexp((double)((1 << f.mbits) + mant), e - f.bias - f.mbits);
}

double decode_elem(int fmt, int code) {
  FmtInfo f = fmt_info(fmt);
  int sign = (code >> (f.bits - 1)) & 1;
  int m = code & ((1 << (f.bits - 1)) - 1);
  double v;
  if (m > f.max_code) v = (fmt == E5M2 && m == 0x7C) ? INFINITY : NAN;
  else v = decode_mag(fmt, m);
  return sign ? -v : v;
}

// Round(.) of Eq. 6, round-to-nearest, ties to the even code, saturating at the largest finite
// magnitude.  Done as a search over the decode table, not with bit manipulation.
int encode_elem(int fmt, double v) {
  FmtInfo f = fmt_info(fmt);
  int sign = std::signbit(v) ? 1 : 0;
  double a = std::fabs(v);
  if (a >= decode_mag(fmt, f.max_code)) return (sign << (f.bits - 1)) | f.max_code;  // saturation
  int best = 0;
  double best_err = INFINITY;
  for (int m = 0; m <= f.max_code; ++m) {
    double err = std::fabs(decode_mag(fmt, m) - a);
    if (err < best_err || (err == best_err && (m & 1) == 0)) {
      best_err = err;
      best = m;
    }
  }
  return (sign << (f.bits - 1)) | best;
}

// ---- stochastic Round(.) of Eq. 6 (Sec. III-A: used for the gradient) ----------------------------
// The paper names the rounding but no generator.  Reading taken: one draw per element from a counter-based
// generator keyed by (seed, index of the element in the logical NCHW / OIHW tensor), so the result does not
// depend on the order in which elements are visited; u = (top 23 bits + 1/2) / 2^23 lies strictly inside
// (0, 1).  With lo <= |v| < hi the neighbouring grid magnitudes, the element becomes hi when
// u < (|v| - lo) / (hi - lo) and lo otherwise: the expectation is |v| up to 2^-24 of a grid step, grid
// values never move, and magnitudes at or beyond the largest finite one saturate as in round-to-nearest.
uint32_t mix32(uint32_t x) {  // an invertible 32-bit finalizer: xor-shift, odd multiply, twice, xor-shift
  x ^= x >> 16;
  x *= 0x7FEB352Du;
  x ^= x >> 15;
  x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x;
}
uint32_t sr_bits(uint64_t seed, uint64_t index) {
  uint32_t key = mix32((uint32_t)seed ^ mix32((uint32_t)(seed >> 32) ^ mix32((uint32_t)(index >> 32))));
  return mix32((uint32_t)index ^ key);
}
int encode_elem_sr(int fmt, double v, uint32_t bits) {
  FmtInfo f = fmt_info(fmt);
  int sign = std::signbit(v) ? 1 : 0;
  double a = std::fabs(v);
  if (a >= decode_mag(fmt, f.max_code)) return (sign << (f.bits - 1)) | f.max_code;  // saturation
  int lo = 0;  // magnitudes grow with the code: the last code whose value does not exceed a
  for (int m = 0; m <= f.max_code; ++m)
    if (decode_mag(fmt, m) <= a) lo = m;
  double vlo = decode_mag(fmt, lo), vhi = decode_mag(fmt, lo + 1);
  double frac = (a - vlo) / (vhi - vlo);
  double u = ((double)(bits >> 9) + 0.5) / 8388608.0;
  return (sign << (f.bits - 1)) | (u < frac ? lo + 1 : lo);
}

// E8M0 code of a block: the role of Eq. 5 in the power-of-two form of the original MX format,
// shared exponent = floor(log2(amax)) - emax_elem, biased by 127 and clamped to [0, 254].
int scale_code(int fmt, double amax) {
  if (!(amax > 0.0)) return 0;
  int e;
  std::frexp(amax, &e);  // amax = f * 2^e with f in [0.5, 1)  =>  floor(log2 amax) = e - 1
  int code = (e - 1) - fmt_info(fmt).emax + 127;
  if (code < 0) code = 0;
  if (code > 254) code = 254;
  return code;
}

double scale_value(int code) { return std::ldexp(1.0, code - 127); }

// ---- the paper's own number format: per-tensor scale + E4M3 block scale + E2M1 elements (Sec. III-A, Eq. 4-6) ------
// Eq. 4:  T_scale = max|X| / (max B_sf * max B_ef)                with max B_sf = 448 (E4M3), max B_ef = 6 (E2M1)
// Eq. 5:  B_scale = CastE4M3( max|X_i| / (T_scale * max B_ef) )   round to nearest E4M3 value
// Eq. 6:  X_i^q   = Round( X_i / (B_scale * T_scale) )            round to nearest E2M1 value
// Each written operation is one IEEE single-precision operation (see the header).  Readings where the paper is silent:
// ties go to the even code and magnitudes beyond the largest finite value saturate, in both roundings (as for the E8M0
// format); a block or tensor of zeros has scale 0 and codes +-0 (no division takes place); when the tensor's maximum
// is supplied from outside (statistics of earlier batches, Sec. VII-B) values may exceed it and saturate likewise.
float tensor_scale_of(float amax) { return amax / (448.0f * 6.0f); }                       // Eq. 4
int block_scale_code(float block_amax, float tscale) {                                     // Eq. 5
  if (!(block_amax > 0.0f) || !(tscale > 0.0f)) return 0;
  float arg = block_amax / (tscale * 6.0f);
  return encode_elem(E4M3, (double)arg) & 0x7F;
}
int ts_elem_code(float x, float bscale, float tscale, bool stochastic, uint32_t bits) {    // Eq. 6
  int sign = std::signbit(x) ? 8 : 0;
  if (!(bscale > 0.0f) || !(tscale > 0.0f)) return sign;
  float scaled = x / (bscale * tscale);
  return stochastic ? encode_elem_sr(E2M1, (double)scaled, bits) : encode_elem(E2M1, (double)scaled);
}


// ---- the 2-D views of Sec. IV-B -------------------------------------------------------------
// Each tensor is seen, at every position p (a pixel (h,w) for X, (ho,wo) for G_Y, a tap (kh,kw)
// for W), as an R x C matrix whose two axes are the ones the squares cover:
//   X  : R = N,    C = Cin     W : R = Cout, C = Cin     G_Y : R = N, C = Cout
struct View {
  int P, R, C, Cp, role;
  int d1, d2;  // logical dims for the source index
};
View view_of(const Conv& c, int role) {
  View v{};
  v.role = role;
  if (role == ROLE_X)       { v.P = c.H * c.W;       v.R = c.N;    v.C = c.Cin;  }
  else if (role == ROLE_W)  { v.P = c.Kh * c.Kw;     v.R = c.Cout; v.C = c.Cin;  }
  else                      { v.P = c.Ho() * c.Wo(); v.R = c.N;    v.C = c.Cout; }
  v.Cp = (v.C + 31) / 32 * 32;
  return v;
}
// index into the logical tensor (NCHW for X and G_Y, OIHW for W): position is the fastest axis
inline size_t src_index(const View& v, int p, int r, int c) { return ((size_t)r * v.C + c) * v.P + p; }
// index of an element in the stored order: X, G_Y -> [p][r][c];  W -> [r][p][c]   (c fastest)
inline size_t code_index(const View& v, int p, int r, int c) {
  if (v.role == ROLE_W) return ((size_t)r * v.P + p) * v.Cp + c;
  return ((size_t)p * v.R + r) * v.Cp + c;
}
inline size_t scale_index(const View& v, int br, int bc, int p, int rb, int cb) {
  int Rb = (v.R + br - 1) / br, Cb = v.Cp / bc;
  if (v.role == ROLE_W) return ((size_t)rb * v.P + p) * Cb + cb;
  return ((size_t)p * Rb + rb) * Cb + cb;
}

inline int get_code(const uint8_t* codes, int fmt, size_t idx) {
  if (fmt == E2M1) return (codes[idx >> 1] >> ((idx & 1) * 4)) & 0xF;  // lower index -> low nibble
  return codes[idx];
}
inline void put_code(uint8_t* codes, int fmt, size_t idx, int code) {
  if (fmt == E2M1) {
    int sh = (idx & 1) * 4;
    codes[idx >> 1] = (uint8_t)((codes[idx >> 1] & ~(0xF << sh)) | ((code & 0xF) << sh));
  } else {
    codes[idx] = (uint8_t)code;
  }
}

}  // namespace

extern "C" {

int orc_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

double orc_decode_elem(int fmt, int code) { return decode_elem(fmt, code); }
int orc_encode_elem(int fmt, double v) { return encode_elem(fmt, v); }
int orc_scale_code(int fmt, double amax) { return scale_code(fmt, amax); }
int orc_encode_elem_sr(int fmt, double v, uint32_t bits) { return encode_elem_sr(fmt, v, bits); }
uint32_t orc_sr_bits(uint64_t seed, uint64_t index) { return sr_bits(seed, index); }

int orc_out_hw(const int* d, int* ho, int* wo) {
  Conv c = conv_from(d);
  *ho = c.Ho();
  *wo = c.Wo();
  return 0;
}

// sizes of the stored MX tensor (bytes) for a role / element format / block shape
int orc_qtensor_sizes(const int* d, int role, int fmt, int br, int bc, int64_t* codes_bytes, int64_t* scales_bytes) {
  Conv c = conv_from(d);
  View v = view_of(c, role);
  int64_t elems = (int64_t)v.P * v.R * v.Cp;
  *codes_bytes = elems * fmt_info(fmt).store_bits / 8;
  *scales_bytes = (int64_t)v.P * ((v.R + br - 1) / br) * (v.Cp / bc);
  return 0;
}

// Microscaling quantization (Sec. III-A, Eq. 5-6 in the E8M0 form), applied once to a tensor in
// the 2-D view of Sec. IV-B.  src: fp32, NCHW (X, G_Y) or OIHW (W).  Padded channels get code 0.
static int quantize_impl(const int* d, int role, int fmt, int br, int bc, const float* src, uint8_t* codes, uint8_t* scales, bool stochastic,
                         uint64_t seed) {
  Conv cv = conv_from(d);
  View v = view_of(cv, role);
  if (bc <= 0 || br <= 0 || v.Cp % bc != 0) return 1;
  int64_t cb_bytes, sb_bytes;
  orc_qtensor_sizes(d, role, fmt, br, bc, &cb_bytes, &sb_bytes);
  std::memset(codes, 0, (size_t)cb_bytes);
  std::memset(scales, 0, (size_t)sb_bytes);
  int Rb = (v.R + br - 1) / br, Cb = v.Cp / bc;
  // a byte of packed E2M1 codes never straddles two blocks (bc even), and blocks of one position
  // touch disjoint bytes, so positions can be processed independently
#pragma omp parallel for schedule(static)
  for (int p = 0; p < v.P; ++p) {
    for (int rb = 0; rb < Rb; ++rb) {
      for (int cb = 0; cb < Cb; ++cb) {
        double amax = 0.0;
        for (int r = rb * br; r < (rb + 1) * br && r < v.R; ++r)
          for (int c = cb * bc; c < (cb + 1) * bc && c < v.C; ++c) {
            double a = std::fabs((double)src[src_index(v, p, r, c)]);
            if (a > amax) amax = a;
          }
        int sc = scale_code(fmt, amax);
        scales[scale_index(v, br, bc, p, rb, cb)] = (uint8_t)sc;
        for (int r = rb * br; r < (rb + 1) * br && r < v.R; ++r)
          for (int c = cb * bc; c < (cb + 1) * bc && c < v.C; ++c) {
            double x = (double)src[src_index(v, p, r, c)];
            double scaled = std::ldexp(x, 127 - sc);  // X_i / B_scale of Eq. 6, exact
            int code = stochastic ? encode_elem_sr(fmt, scaled, sr_bits(seed, (uint64_t)src_index(v, p, r, c))) : encode_elem(fmt, scaled);
            put_code(codes, fmt, code_index(v, p, r, c), code);
          }
      }
    }
  }
  return 0;
}
int orc_quantize(const int* d, int role, int fmt, int br, int bc, const float* src, uint8_t* codes, uint8_t* scales) {
  return quantize_impl(d, role, fmt, br, bc, src, codes, scales, false, 0);
}
// The same with the stochastic Round(.) of Eq. 6; block scales are those of the deterministic quantizer.
int orc_quantize_sr(const int* d, int role, int fmt, int br, int bc, const float* src, uint64_t seed, uint8_t* codes, uint8_t* scales) {
  return quantize_impl(d, role, fmt, br, bc, src, codes, scales, true, seed);
}

// Fake quantization of Sec. III-A: element value times its block scale.  out: double, logical order.
int orc_dequant(const int* d, int role, int fmt, int br, int bc, const uint8_t* codes, const uint8_t* scales, double* out) {
  Conv cv = conv_from(d);
  View v = view_of(cv, role);
#pragma omp parallel for schedule(static)
  for (int p = 0; p < v.P; ++p)
    for (int r = 0; r < v.R; ++r)
      for (int c = 0; c < v.C; ++c) {
        int code = get_code(codes, fmt, code_index(v, p, r, c));
        int sc = scales[scale_index(v, br, bc, p, r / br, c / bc)];
        out[src_index(v, p, r, c)] = decode_elem(fmt, code) * scale_value(sc);
      }
  return 0;
}


// ---- the paper's own format (Eq. 4-6) on br x bc blocks --------------------------------------------------------------
// codes: E2M1, packed as in orc_quantize; scales: one E4M3 byte per block, in the order of orc_quantize's scales;
// tensor_scale: T_scale; tensor_amax: max|X| of this tensor.  amax_in < 0: T_scale from this tensor's own maximum
// (two passes over the data); amax_in >= 0: T_scale from that value instead (statistics of earlier batches).
int orc_quantize_ts(const int* d, int role, int br, int bc, const float* src, float amax_in, int stochastic, uint64_t seed, uint8_t* codes,
                    uint8_t* scales, float* tensor_scale, float* tensor_amax) {
  Conv cv = conv_from(d);
  View v = view_of(cv, role);
  if (bc <= 0 || br <= 0 || v.Cp % bc != 0 || (bc & 1)) return 1;
  int64_t cb_bytes, sb_bytes;
  orc_qtensor_sizes(d, role, E2M1, br, bc, &cb_bytes, &sb_bytes);
  std::memset(codes, 0, (size_t)cb_bytes);
  std::memset(scales, 0, (size_t)sb_bytes);
  float amax = 0.0f;
  size_t total = (size_t)v.P * v.R * v.C;
  for (size_t i = 0; i < total; ++i) { float a = std::fabs(src[i]); if (a > amax) amax = a; }
  *tensor_amax = amax;
  const float tscale = tensor_scale_of(amax_in >= 0.0f ? amax_in : amax);
  *tensor_scale = tscale;
  int Rb = (v.R + br - 1) / br, Cb = v.Cp / bc;
#pragma omp parallel for schedule(static)
  for (int p = 0; p < v.P; ++p) {
    for (int rb = 0; rb < Rb; ++rb) {
      for (int cb = 0; cb < Cb; ++cb) {
        float bmax = 0.0f;
        for (int r = rb * br; r < (rb + 1) * br && r < v.R; ++r)
          for (int c = cb * bc; c < (cb + 1) * bc && c < v.C; ++c) {
            float a = std::fabs(src[src_index(v, p, r, c)]);
            if (a > bmax) bmax = a;
          }
        int sc = block_scale_code(bmax, tscale);
        scales[scale_index(v, br, bc, p, rb, cb)] = (uint8_t)sc;
        float bscale = (float)decode_elem(E4M3, sc);
        for (int r = rb * br; r < (rb + 1) * br && r < v.R; ++r)
          for (int c = cb * bc; c < (cb + 1) * bc && c < v.C; ++c) {
            size_t si = src_index(v, p, r, c);
            int code = ts_elem_code(src[si], bscale, tscale, stochastic != 0, stochastic ? sr_bits(seed, (uint64_t)si) : 0u);
            put_code(codes, E2M1, code_index(v, p, r, c), code);
          }
      }
    }
  }
  return 0;
}

// Fake quantization of that format: element value x block scale x tensor scale (Sec. III-A).
int orc_dequant_ts(const int* d, int role, int br, int bc, const uint8_t* codes, const uint8_t* scales, float tensor_scale, double* out) {
  Conv cv = conv_from(d);
  View v = view_of(cv, role);
#pragma omp parallel for schedule(static)
  for (int p = 0; p < v.P; ++p)
    for (int r = 0; r < v.R; ++r)
      for (int c = 0; c < v.C; ++c) {
        int code = get_code(codes, E2M1, code_index(v, p, r, c));
        int sc = scales[scale_index(v, br, bc, p, r / br, c / bc)];
        out[src_index(v, p, r, c)] = decode_elem(E2M1, code) * decode_elem(E4M3, sc) * (double)tensor_scale;
      }
  return 0;
}
int orc_block_scale_code(float block_amax, float tscale) { return block_scale_code(block_amax, tscale); }
int orc_ts_elem_code(float x, float bscale, float tscale) { return ts_elem_code(x, bscale, tscale, false, 0u); }

// sizes of X'_{Cin,N} built from the stored quantized activation
int orc_im2col_sizes(const int* d, int fmt, int br, int bc, int64_t* codes_bytes, int64_t* scales_bytes) {
  Conv c = conv_from(d);
  int Cp = (c.Cin + 31) / 32 * 32;
  int64_t rows = (int64_t)c.Ho() * c.Wo() * c.N;
  *codes_bytes = rows * c.Kh * c.Kw * Cp * fmt_info(fmt).store_bits / 8;
  *scales_bytes = (int64_t)c.Ho() * c.Wo() * ((c.N + br - 1) / br) * c.Kh * c.Kw * (Cp / bc);
  return 0;
}

// Channel-batch-first im2col (Sec. IV-A) of the already-quantized activation: column (ho,wo,n),
// row (kh,kw,cin) of X'_{Cin,N} is the stored code of X at (ho*s+kh-p, wo*s+kw-p, n, cin); the
// block scales travel with the blocks.  Out-of-image taps are all-zero bytes (codes and scale).
// out codes: [Ho][Wo][N][Kh][Kw][Cp], out scales: [Ho][Wo][ceil(N/br)][Kh][Kw][Cp/bc].
int orc_cbf_im2col(const int* d, int fmt, int br, int bc, const uint8_t* codes, const uint8_t* scales,
                   uint8_t* out_codes, uint8_t* out_scales) {
  Conv c = conv_from(d);
  View v = view_of(c, ROLE_X);
  int Ho = c.Ho(), Wo = c.Wo(), Cp = v.Cp, Rb = (c.N + br - 1) / br, Cb = Cp / bc;
  int64_t cbz, sbz;
  orc_im2col_sizes(d, fmt, br, bc, &cbz, &sbz);
  std::memset(out_codes, 0, (size_t)cbz);
  std::memset(out_scales, 0, (size_t)sbz);
#pragma omp parallel for schedule(static)
  for (int ho = 0; ho < Ho; ++ho)
    for (int wo = 0; wo < Wo; ++wo)
      for (int kh = 0; kh < c.Kh; ++kh)
        for (int kw = 0; kw < c.Kw; ++kw) {
          int h = ho * c.sh + kh - c.ph, w = wo * c.sw + kw - c.pw;
          if (h < 0 || h >= c.H || w < 0 || w >= c.W) continue;
          int p = h * c.W + w;
          for (int n = 0; n < c.N; ++n)
            for (int ci = 0; ci < Cp; ++ci) {
              size_t o = ((((size_t)(ho * Wo + wo) * c.N + n) * c.Kh + kh) * c.Kw + kw) * Cp + ci;
              put_code(out_codes, fmt, o, get_code(codes, fmt, code_index(v, p, n, ci)));
            }
          for (int rb = 0; rb < Rb; ++rb)
            for (int cb = 0; cb < Cb; ++cb) {
              size_t o = ((((size_t)(ho * Wo + wo) * Rb + rb) * c.Kh + kh) * c.Kw + kw) * Cb + cb;
              out_scales[o] = scales[scale_index(v, br, bc, p, rb, cb)];
            }
        }
  return 0;
}

// ---- the three convolutions, as their plain definitions on dequantized tensors --------------
// All tensors double, logical order (X, G_X: NCHW; W, G_W: OIHW; Y, G_Y: N.Cout.Ho.Wo).
// `*_abs` receives sum |a_i * b_i| of the same terms (the parity bound's right-hand side).

// Eq. 1: Y = W * X (cross-correlation, zero padding)
static void fwd_point(const Conv& c, const double* X, const double* Wt, int n, int co, int ho, int wo, double* y, double* ya) {
  double acc = 0.0, aabs = 0.0;
  for (int ci = 0; ci < c.Cin; ++ci)
    for (int kh = 0; kh < c.Kh; ++kh)
      for (int kw = 0; kw < c.Kw; ++kw) {
        int h = ho * c.sh + kh - c.ph, w = wo * c.sw + kw - c.pw;
        if (h < 0 || h >= c.H || w < 0 || w >= c.W) continue;
        double t = Wt[(((size_t)co * c.Cin + ci) * c.Kh + kh) * c.Kw + kw] * X[(((size_t)n * c.Cin + ci) * c.H + h) * c.W + w];
        acc += t;
        aabs += std::fabs(t);
      }
  *y = acc;
  *ya = aabs;
}

// Eq. 2 / G_X' = W_f^T . G_Yf followed by col2im: the exact adjoint of Eq. 1 w.r.t. X
static void bwd_data_point(const Conv& c, const double* Wt, const double* G, int n, int ci, int h, int w, double* gx, double* gxa) {
  int Ho = c.Ho(), Wo = c.Wo();
  double acc = 0.0, aabs = 0.0;
  for (int co = 0; co < c.Cout; ++co)
    for (int kh = 0; kh < c.Kh; ++kh)
      for (int kw = 0; kw < c.Kw; ++kw) {
        int hn = h + c.ph - kh, wn = w + c.pw - kw;
        if (hn < 0 || wn < 0 || hn % c.sh != 0 || wn % c.sw != 0) continue;
        int ho = hn / c.sh, wo = wn / c.sw;
        if (ho >= Ho || wo >= Wo) continue;
        double t = Wt[(((size_t)co * c.Cin + ci) * c.Kh + kh) * c.Kw + kw] * G[(((size_t)n * c.Cout + co) * Ho + ho) * Wo + wo];
        acc += t;
        aabs += std::fabs(t);
      }
  *gx = acc;
  *gxa = aabs;
}

// Eq. 3: G_W[co,ci,:,:] = sum_n G_Y[n,co] * X[n,ci]
static void bwd_weight_point(const Conv& c, const double* G, const double* X, int co, int ci, int kh, int kw, double* gw, double* gwa) {
  int Ho = c.Ho(), Wo = c.Wo();
  double acc = 0.0, aabs = 0.0;
  for (int n = 0; n < c.N; ++n)
    for (int ho = 0; ho < Ho; ++ho)
      for (int wo = 0; wo < Wo; ++wo) {
        int h = ho * c.sh + kh - c.ph, w = wo * c.sw + kw - c.pw;
        if (h < 0 || h >= c.H || w < 0 || w >= c.W) continue;
        double t = G[(((size_t)n * c.Cout + co) * Ho + ho) * Wo + wo] * X[(((size_t)n * c.Cin + ci) * c.H + h) * c.W + w];
        acc += t;
        aabs += std::fabs(t);
      }
  *gw = acc;
  *gwa = aabs;
}

// idx: flat indices into the output tensor (nullptr => every element, count = tensor size)
int orc_conv_fwd(const int* d, const double* X, const double* Wt, const int64_t* idx, int64_t count, double* y, double* yabs) {
  Conv c = conv_from(d);
  int Ho = c.Ho(), Wo = c.Wo();
  if (!idx) count = (int64_t)c.N * c.Cout * Ho * Wo;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t f = idx ? idx[i] : i;
    int wo = (int)(f % Wo); f /= Wo;
    int ho = (int)(f % Ho); f /= Ho;
    int co = (int)(f % c.Cout); f /= c.Cout;
    fwd_point(c, X, Wt, (int)f, co, ho, wo, &y[i], &yabs[i]);
  }
  return 0;
}

int orc_conv_bwd_data(const int* d, const double* Wt, const double* G, const int64_t* idx, int64_t count, double* gx, double* gxabs) {
  Conv c = conv_from(d);
  if (!idx) count = (int64_t)c.N * c.Cin * c.H * c.W;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t f = idx ? idx[i] : i;
    int w = (int)(f % c.W); f /= c.W;
    int h = (int)(f % c.H); f /= c.H;
    int ci = (int)(f % c.Cin); f /= c.Cin;
    bwd_data_point(c, Wt, G, (int)f, ci, h, w, &gx[i], &gxabs[i]);
  }
  return 0;
}

int orc_conv_bwd_weight(const int* d, const double* G, const double* X, const int64_t* idx, int64_t count, double* gw, double* gwabs) {
  Conv c = conv_from(d);
  if (!idx) count = (int64_t)c.Cout * c.Cin * c.Kh * c.Kw;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t i = 0; i < count; ++i) {
    int64_t f = idx ? idx[i] : i;
    int kw = (int)(f % c.Kw); f /= c.Kw;
    int kh = (int)(f % c.Kh); f /= c.Kh;
    int ci = (int)(f % c.Cin); f /= c.Cin;
    bwd_weight_point(c, G, X, (int)f, ci, kh, kw, &gw[i], &gwabs[i]);
  }
  return 0;
}

}  // extern "C"
