// CPU oracle for Block Data Representations (BDR) / shared-microexponent (MX) quantization.
//
// TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct restatement of the
// paper's definitions.  Nothing on the product (CUDA) path may include, link, import or call it;
// it shares no header, helper, table or constant with the CUDA library.  Only the tests, the smoke
// check and the benchmark's CPU-baseline leg use it.
//
// What each function follows:
//   * block structure (k1 blocks, k2 sub-blocks, bits/element)  -- Section III, "Block Data
//     Representations" paragraph and the bits-per-element formula (m+1)+d1/k1+d2/k2;
//   * the quantizer Q(.)                                        -- Appendix (proof of Theorem 1):
//     shared exponent = private exponent of the largest element, the m-digit form
//     (-1)^s * (sum_{j<m} Q_-j 2^-j) * 2^E, the sub-block shift tau <= beta = 2^d2-1 and the
//     error bounds 2^(E-m) / 2^(E-tau-m);
//   * QSNR                                                      -- Section IV-A, Eq. 3;
//   * Theorem 1 bound                                           -- Section IV-C, Theorem 1;
//   * INT quantization with an FP32 max-scale                   -- Section II, Eq. 1 and Eq. 2;
//   * FP8 / VSQ as two-level schemes                            -- Section III, Table I;
//   * a first-level maximum supplied from outside ("delayed scaling") and the packing efficiency of
//     a tile in fixed-width memory lines                          -- Section IV-B, Fig. 7 caption and the
//     memory-footprint paragraph;
//   * the dot product as the hardware pipeline computes it        -- Section IV-B, Fig. 6 and its text;
//   * an FP32 parent scale above the two levels (three-level)     -- Section III, last paragraph.
//
// Readings taken where the paper is silent (all listed in the design notes of the repository):
//   ties round to even by default (ties-away selectable); a magnitude that would round to 2^m is
//   clamped to 2^m-1 and the shared exponent is never bumped; the private exponent of zeros and
//   fp32 subnormals is the raw exponent field (0); a short last block behaves as if zero padded;
//   the sign bit of the input is kept even when the magnitude quantizes to zero; any Inf/NaN in a
//   block turns the whole block into quiet NaNs with exponent byte 0xFF.
//
// Parity pins: every function here is pinned by tests (closed forms, invariants, brute force,
// textbook special cases, hand-worked examples).  The VSQ kind, for which the paper gives the
// principle but no formula, is pinned by hand-worked groups (sub-scales that round up, round down,
// tie, reach the top code and flush to zero; both tie rules; per-group first-level scale) and by its
// reductions (equal per-vector maxima => per-tensor INT; a 16-bit sub-scale => INT with one FP32
// scale per vector, within a derived bound).  The hardware dot product and the parent scale, which
// the paper describes in words only, are pinned by hand-worked examples and by the cases in which they
// must reduce to the exact dot product / the two-level quantizer.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared bdr_oracle.cpp -o liboracle_bdr.so -lpthread

#include <cfenv>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

extern "C" {

typedef struct {
    int32_t k1, d1, k2, d2, m, scale_kind, rounding;
} orc_config;

enum { ORC_POW2 = 0, ORC_FP32_INT = 1, ORC_FP32_FP = 2, ORC_FP32_VSQ = 3 };
enum { ORC_RNE = 0, ORC_RNA = 1 };
enum { ORC_OK = 0, ORC_BAD = -1 };

}  // extern "C"

namespace {

inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// A "line" is the 1-D run along the quantization axis: row r for axis=1, column c for axis=0.
struct LineView {
    int64_t nlines, len, line_stride, elem_stride;
};
inline LineView make_view(int64_t rows, int64_t cols, int64_t ld, int axis) {
    if (axis == 1) return {rows, cols, ld, 1};
    return {cols, rows, 1, ld};
}

// Round the non-negative rational M / 2^sh to the nearest integer.
inline uint64_t round_shift(uint64_t M, int sh, int rounding) {
    if (sh <= 0) return M << (-sh);
    if (sh >= 63) return 0;  // M < 2^24, so the quotient is far below 1/2
    uint64_t fl = M >> sh;
    uint64_t rem = M & ((1ull << sh) - 1);
    uint64_t half = 1ull << (sh - 1);
    if (rem > half) fl += 1;
    else if (rem == half && (rounding == ORC_RNA || (fl & 1))) fl += 1;
    return fl;
}

// Round a non-negative real to the nearest integer with the chosen tie rule.
inline double round_real(double t, int rounding) {
    double fl = std::floor(t);
    double rem = t - fl;  // exact for the magnitudes used here
    if (rem > 0.5) return fl + 1.0;
    if (rem < 0.5) return fl;
    if (rounding == ORC_RNA) return fl + 1.0;
    return (std::fmod(fl, 2.0) == 0.0) ? fl : fl + 1.0;
}

bool config_ok(const orc_config* c) {
    if (!c) return false;
    if (c->rounding != ORC_RNE && c->rounding != ORC_RNA) return false;
    switch (c->scale_kind) {
        case ORC_POW2:
            return c->d1 == 8 && c->k1 >= 1 && c->k2 >= 1 && c->k1 % c->k2 == 0 && c->d2 >= 0 &&
                   c->d2 <= 3 && c->m >= 1 && c->m <= 8;
        case ORC_FP32_INT:
            return c->k1 >= 0 && c->m >= 1 && c->m <= 15;
        case ORC_FP32_FP:
            return c->k1 >= 0 && c->d2 >= 2 && c->d2 <= 5 && c->m >= 1 && c->m <= 7;
        case ORC_FP32_VSQ:
            return c->k1 >= 0 && c->k2 >= 1 && c->d2 >= 1 && c->d2 <= 16 && c->m >= 1 && c->m <= 15 &&
                   (c->k1 == 0 || c->k1 % c->k2 == 0);
    }
    return false;
}

// ---------------------------------------------------------------------------------------------
// POW2 kind: one k1-block of one line.  `n` real elements (n <= k1); the rest is zero padding.
// Outputs (any may be null): F (exponent byte), tau[k1/k2], code[k1], deq[n].
// Appendix, proof of Theorem 1: E is the private exponent of the largest element; an element in a
// sub-block shifted by tau keeps m magnitude digits of weight 2^(E-tau) ... 2^(E-tau-m+1).
// ---------------------------------------------------------------------------------------------
void pow2_block(const orc_config& c, const float* x, int64_t stride, int n, uint8_t* F_out,
                uint8_t* tau_out, uint16_t* code_out, float* deq, int64_t deq_stride) {
    const int k1 = c.k1, k2 = c.k2, m = c.m;
    const int beta = (1 << c.d2) - 1;
    const int nsub = k1 / k2;
    const uint32_t qmax = (1u << m) - 1;

    // private exponents: the raw fp32 exponent field (zeros and subnormals -> 0)
    int F = 0;
    bool nonfinite = false;
    for (int i = 0; i < n; ++i) {
        int f = (f2u(x[i * stride]) >> 23) & 0xFF;
        if (f == 255) nonfinite = true;
        if (f > F) F = f;
    }
    if (nonfinite) {
        if (F_out) *F_out = 0xFF;
        for (int j = 0; j < nsub; ++j) if (tau_out) tau_out[j] = 0;
        for (int i = 0; i < k1; ++i) if (code_out) code_out[i] = 0;
        for (int i = 0; i < n; ++i) if (deq) deq[i * deq_stride] = u2f(0x7FC00000u);
        return;
    }
    if (F_out) *F_out = (uint8_t)F;

    for (int j = 0; j < nsub; ++j) {
        int Fj = 0;
        for (int i = j * k2; i < (j + 1) * k2 && i < n; ++i) {
            int f = (f2u(x[i * stride]) >> 23) & 0xFF;
            if (f > Fj) Fj = f;
        }
        int tau = F - Fj;
        if (tau > beta) tau = beta;
        if (tau_out) tau_out[j] = (uint8_t)tau;

        for (int i = j * k2; i < (j + 1) * k2; ++i) {
            if (i >= n) {  // zero padding: code of +0
                if (code_out) code_out[i] = 0;
                continue;
            }
            uint32_t u = f2u(x[i * stride]);
            uint32_t s = u >> 31;
            int f = (u >> 23) & 0xFF;
            uint64_t M = (u & 0x7FFFFFu) | (f ? 0x800000u : 0u);  // 24-bit significand
            int fe = f ? f : 1;                                     // |x| = M * 2^(fe-150)
            // |x| / 2^p with p = (F-127) - tau - (m-1)  equals  M / 2^sh
            int sh = 24 - m - tau - (fe - F);
            uint64_t q = round_shift(M, sh, c.rounding);
            if (q > qmax) q = qmax;
            if (code_out) code_out[i] = (uint16_t)((s << m) | q);
            if (deq) {
                int p = (F - 127) - tau - (m - 1);
                float mag = (float)std::ldexp((double)q, p);  // exact: q < 2^8, p >= -149
                deq[i * deq_stride] = u2f(f2u(mag) | (s << 31));
            }
        }
    }
}

// Second, independent formulation of the same block (real arithmetic in double, no bit twiddling
// of significands); used only to cross-check pow2_block.
void pow2_block_alt(const orc_config& c, const float* x, int64_t stride, int n, float* deq,
                    int64_t deq_stride) {
    const int k1 = c.k1, k2 = c.k2, m = c.m;
    const int beta = (1 << c.d2) - 1;
    auto priv_exp = [](float v) -> int {  // floor(log2|v|) floored at -127, 0 -> -127
        double a = std::fabs((double)v);
        if (a < std::ldexp(1.0, -126)) return -127;
        int e;
        std::frexp(a, &e);  // a = f * 2^e, f in [0.5,1)
        return e - 1;
    };
    int E = -127;
    for (int i = 0; i < n; ++i) {
        if (!std::isfinite(x[i * stride])) {
            for (int t = 0; t < n; ++t) deq[t * deq_stride] = u2f(0x7FC00000u);
            return;
        }
        E = std::max(E, priv_exp(x[i * stride]));
    }
    for (int j = 0; j < k1 / k2; ++j) {
        int Ej = -127;
        for (int i = j * k2; i < (j + 1) * k2 && i < n; ++i) Ej = std::max(Ej, priv_exp(x[i * stride]));
        int tau = std::min(E - Ej, beta);
        int p = E - tau - (m - 1);
        for (int i = j * k2; i < (j + 1) * k2 && i < n; ++i) {
            double a = std::fabs((double)x[i * stride]);
            double t = std::ldexp(a, -p);  // exact in double
            double q = round_real(t, c.rounding);
            double qmax = std::ldexp(1.0, m) - 1.0;
            if (q > qmax) q = qmax;
            double v = std::ldexp(q, p);
            deq[i * deq_stride] = std::signbit(x[i * stride]) ? -(float)v : (float)v;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// FP32-scaled comparator kinds (Section II Eq. 1-2; Section III Table I).  All fp32 operations
// are single IEEE round-to-nearest operations (file is built with -ffp-contract=off).
// ---------------------------------------------------------------------------------------------
inline float absmax(const float* x, int64_t stride, int64_t n) {
    float a = 0.f;
    for (int64_t i = 0; i < n; ++i) a = std::fmax(a, std::fabs(x[i * stride]));
    return a;
}

// Round |v| to the nearest value of a small float format with `eb` exponent bits and `mb`
// explicit mantissa bits (implicit leading one, gradual underflow), saturating at fmax.
float minifloat_round(float v, int eb, int mb, int rounding) {
    int bias = (1 << (eb - 1)) - 1;
    double fmax;
    if (eb == 4 && mb == 3) fmax = 448.0;  // E4M3 "fn": top exponent is finite, one NaN code
    else fmax = (2.0 - std::ldexp(1.0, -mb)) * std::ldexp(1.0, (1 << eb) - 2 - bias);  // IEEE-like
    double a = std::fabs((double)v);
    if (a == 0.0) return v;
    int emin = 1 - bias;
    int e;
    std::frexp(a, &e);
    e -= 1;  // floor(log2 a)
    if (e < emin) e = emin;
    double step = std::ldexp(1.0, e - mb);
    double q = round_real(a / step, rounding) * step;  // a/step exact in double
    if (q > fmax) q = fmax;
    return std::signbit(v) ? -(float)q : (float)q;
}

inline float with_sign(float mag, float like) { return u2f((f2u(mag) & 0x7FFFFFFFu) | (f2u(like) & 0x80000000u)); }

// One scale group of the INT kind: Eq. 1 (s = max/(2^(b-1)-1), here m = b-1) and Eq. 2.
void int_group(const orc_config& c, const float* x, int64_t stride, int64_t n, float amax, float* deq,
               int64_t dstride) {
    float qmax = (float)((1 << c.m) - 1);
    float s = amax / qmax;
    for (int64_t i = 0; i < n; ++i) {
        float v = x[i * stride];
        if (!(s > 0.f)) { deq[i * dstride] = with_sign(0.f, v); continue; }
        float t = std::fabs(v) / s;
        float q = (float)round_real((double)t, c.rounding);
        if (q > qmax) q = qmax;
        deq[i * dstride] = with_sign(q * s, v);
    }
}

void fp_group(const orc_config& c, const float* x, int64_t stride, int64_t n, float amax, float* deq,
              int64_t dstride) {
    float fmax = std::fabs(minifloat_round(std::numeric_limits<float>::max(), c.d2, c.m, c.rounding));
    float s = amax / fmax;
    for (int64_t i = 0; i < n; ++i) {
        float v = x[i * stride];
        if (!(s > 0.f)) { deq[i * dstride] = with_sign(0.f, v); continue; }
        float y = v / s;
        float yq = minifloat_round(y, c.d2, c.m, c.rounding);
        deq[i * dstride] = with_sign(std::fabs(yq * s), v);
    }
}

// VSQ group: FP32 first-level scale gamma over the group, unsigned d2-bit integer sub-scale per k2.
void vsq_group(const orc_config& c, const float* x, int64_t stride, int64_t n, float amax, float* deq,
               int64_t dstride) {
    float qmax = (float)((1 << c.m) - 1);
    float umax = (float)((1u << c.d2) - 1);
    float smax = amax / qmax;      // the largest per-vector ideal scale
    float gamma = smax / umax;
    for (int64_t v0 = 0; v0 < n; v0 += c.k2) {
        int64_t cnt = std::min<int64_t>(c.k2, n - v0);
        float av = absmax(x + v0 * stride, stride, cnt);
        float sv = av / qmax;
        float u = 0.f;
        if (gamma > 0.f) {
            u = (float)round_real((double)(sv / gamma), c.rounding);
            if (u > umax) u = umax;
        }
        float eff = u * gamma;
        for (int64_t i = v0; i < v0 + cnt; ++i) {
            float v = x[i * stride];
            if (!(eff > 0.f)) { deq[i * dstride] = with_sign(0.f, v); continue; }
            float t = std::fabs(v) / eff;
            float q = (float)round_real((double)t, c.rounding);
            if (q > qmax) q = qmax;
            deq[i * dstride] = with_sign(q * eff, v);
        }
    }
}

void quantize_lines(const orc_config& c, const float* x, float* y, const LineView& v, int64_t l0, int64_t l1,
                    float tensor_amax, bool alt) {
    for (int64_t l = l0; l < l1; ++l) {
        const float* xl = x + l * v.line_stride;
        float* yl = y + l * v.line_stride;
        if (c.scale_kind == ORC_POW2) {
            for (int64_t b0 = 0; b0 < v.len; b0 += c.k1) {
                int n = (int)std::min<int64_t>(c.k1, v.len - b0);
                if (alt) pow2_block_alt(c, xl + b0 * v.elem_stride, v.elem_stride, n, yl + b0 * v.elem_stride, v.elem_stride);
                else pow2_block(c, xl + b0 * v.elem_stride, v.elem_stride, n, nullptr, nullptr, nullptr,
                                yl + b0 * v.elem_stride, v.elem_stride);
            }
        } else {
            int64_t g = c.k1 == 0 ? v.len : c.k1;
            for (int64_t b0 = 0; b0 < v.len; b0 += g) {
                int64_t n = std::min<int64_t>(g, v.len - b0);
                const float* xb = xl + b0 * v.elem_stride;
                float* yb = yl + b0 * v.elem_stride;
                float amax = c.k1 == 0 ? tensor_amax : absmax(xb, v.elem_stride, n);
                if (c.scale_kind == ORC_FP32_INT) int_group(c, xb, v.elem_stride, n, amax, yb, v.elem_stride);
                else if (c.scale_kind == ORC_FP32_FP) fp_group(c, xb, v.elem_stride, n, amax, yb, v.elem_stride);
                else vsq_group(c, xb, v.elem_stride, n, amax, yb, v.elem_stride);
            }
        }
    }
}

// little-endian, LSB-first bit stream writer/reader
inline void put_bits(uint8_t* base, int64_t bitpos, int nbits, uint32_t val) {
    for (int b = 0; b < nbits; ++b) {
        int64_t p = bitpos + b;
        if ((val >> b) & 1u) base[p >> 3] |= (uint8_t)(1u << (p & 7));
    }
}
inline uint32_t get_bits(const uint8_t* base, int64_t bitpos, int nbits) {
    uint32_t v = 0;
    for (int b = 0; b < nbits; ++b) {
        int64_t p = bitpos + b;
        v |= (uint32_t)((base[p >> 3] >> (p & 7)) & 1u) << b;
    }
    return v;
}

inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

}  // namespace

extern "C" {

int orc_config_check(const orc_config* c) { return config_ok(c) ? ORC_OK : ORC_BAD; }

// Section III: total bits per element = (m+1) + d1/k1 + d2/k2.
double orc_bits_per_element(const orc_config* c) {
    double b = c->m + 1;
    if (c->k1 > 0) b += (double)c->d1 / c->k1;
    if (c->k2 > 0) b += (double)c->d2 / c->k2;
    return b;
}

// Section IV-C, Theorem 1 (d1 = 8, beta = 2^d2 - 1).
double orc_theorem1_bound_db(const orc_config* c, int64_t N) {
    double beta = (double)((1 << c->d2) - 1);
    double w = std::pow(2.0, 2.0 * beta);
    double nk = (double)std::min<int64_t>(N, c->k1);
    return 6.02 * c->m + 10.0 * std::log10(w / (nk + (w - 1.0) * c->k2));
}

// Section IV-A, Eq. 3 on whole-tensor sums.
double orc_qsnr_db(double err2, double sig2) {
    if (sig2 == 0.0) return std::numeric_limits<double>::quiet_NaN();
    if (err2 == 0.0) return std::numeric_limits<double>::infinity();
    return -10.0 * std::log10(err2 / sig2);
}

// Quantize-dequantize.  x, y: fp32 [rows, ld] row-major (only cols columns used).  sums (nullable)
// receives {sum (Q-x)^2, sum x^2} in fp64 over the tensor.  nthreads > 1 splits lines over
// std::threads (the blocks are independent); the arithmetic is the same.
// first_level_amax (nullable): for the FP32-scaled kinds with one scale per tensor (k1 = 0), the maximum that
// the first-level scale is derived from when it does not come from the tensor itself -- Section IV-B, Fig. 7
// caption: the INT / FP / VSQ points use the absolute maximum over a window of PAST vectors ("delayed
// scaling"); values beyond it saturate at the top code.  NULL: the current tensor's own maximum.
static int quant_dequant_impl(const orc_config* c, const float* x, float* y, int64_t rows, int64_t cols, int64_t ld,
                              int axis, double* sums, int alt, int nthreads, const float* first_level_amax) {
    if (!config_ok(c) || !x || !y || rows < 0 || cols < 0 || ld < cols || (axis != 0 && axis != 1)) return ORC_BAD;
    if (alt && c->scale_kind != ORC_POW2) return ORC_BAD;
    if (first_level_amax && (c->scale_kind == ORC_POW2 || c->k1 != 0 || !(*first_level_amax >= 0.f))) return ORC_BAD;
    LineView v = make_view(rows, cols, ld, axis);
    float tensor_amax = 0.f;
    if (first_level_amax) tensor_amax = *first_level_amax;
    else if (c->scale_kind != ORC_POW2 && c->k1 == 0)
        for (int64_t r = 0; r < rows; ++r) tensor_amax = std::fmax(tensor_amax, absmax(x + r * ld, 1, cols));
    if (nthreads <= 1) {
        quantize_lines(*c, x, y, v, 0, v.nlines, tensor_amax, alt != 0);
    } else {
        std::vector<std::thread> th;
        int64_t per = (v.nlines + nthreads - 1) / nthreads;
        for (int t = 0; t < nthreads; ++t) {
            int64_t l0 = t * per, l1 = std::min<int64_t>(v.nlines, l0 + per);
            if (l0 >= l1) break;
            th.emplace_back([=] { quantize_lines(*c, x, y, v, l0, l1, tensor_amax, alt != 0); });
        }
        for (auto& t : th) t.join();
    }
    if (sums) {
        double e2 = 0.0, s2 = 0.0;
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t cc = 0; cc < cols; ++cc) {
                double a = (double)x[r * ld + cc], q = (double)y[r * ld + cc];
                e2 += (q - a) * (q - a);
                s2 += a * a;
            }
        sums[0] = e2;
        sums[1] = s2;
    }
    return ORC_OK;
}

int orc_quant_dequant_mt(const orc_config* c, const float* x, float* y, int64_t rows, int64_t cols, int64_t ld,
                         int axis, double* sums, int alt, int nthreads) {
    return quant_dequant_impl(c, x, y, rows, cols, ld, axis, sums, alt, nthreads, nullptr);
}

int orc_quant_dequant_scaled(const orc_config* c, const float* x, float* y, int64_t rows, int64_t cols, int64_t ld,
                             int axis, double* sums, float first_level_amax, int nthreads) {
    return quant_dequant_impl(c, x, y, rows, cols, ld, axis, sums, 0, nthreads, &first_level_amax);
}

// Section IV-B, memory footprint: how well a tile of `tile_elems` elements packs into memory lines of
// `line_bytes` bytes -- the tile's bits (bits per element of Section III x elements) over the bits of the
// whole lines it occupies.
double orc_tile_packing_efficiency(const orc_config* c, int64_t tile_elems, int64_t line_bytes) {
    if (!config_ok(c) || tile_elems < 1 || line_bytes < 1) return -1.0;
    const double bits = orc_bits_per_element(c) * (double)tile_elems;
    const double line_bits = 8.0 * (double)line_bytes;
    const double lines = std::ceil(bits / line_bits);
    return bits / (lines * line_bits);
}

int orc_quant_dequant(const orc_config* c, const float* x, float* y, int64_t rows, int64_t cols, int64_t ld,
                      int axis, double* sums) {
    return orc_quant_dequant_mt(c, x, y, rows, cols, ld, axis, sums, 0, 1);
}

int orc_quant_dequant_alt(const orc_config* c, const float* x, float* y, int64_t rows, int64_t cols, int64_t ld,
                          int axis, double* sums) {
    return orc_quant_dequant_mt(c, x, y, rows, cols, ld, axis, sums, 1, 1);
}

// Raw (unpacked) encoding of a POW2 tensor: F[nlines][nblocks], tau[nlines][nblocks*k1/k2],
// code[nlines][nblocks*k1] (padding positions hold code 0).
int orc_encode(const orc_config* c, const float* x, int64_t rows, int64_t cols, int64_t ld, int axis, uint8_t* F,
               uint8_t* tau, uint16_t* code) {
    if (!config_ok(c) || c->scale_kind != ORC_POW2 || !x || ld < cols) return ORC_BAD;
    LineView v = make_view(rows, cols, ld, axis);
    int64_t nb = (v.len + c->k1 - 1) / c->k1;
    int nsub = c->k1 / c->k2;
    for (int64_t l = 0; l < v.nlines; ++l)
        for (int64_t b = 0; b < nb; ++b) {
            int n = (int)std::min<int64_t>(c->k1, v.len - b * c->k1);
            pow2_block(*c, x + l * v.line_stride + b * c->k1 * v.elem_stride, v.elem_stride, n,
                       F ? F + l * nb + b : nullptr, tau ? tau + (l * nb + b) * nsub : nullptr,
                       code ? code + (l * nb + b) * c->k1 : nullptr, nullptr, 0);
        }
    return ORC_OK;
}

// Packed plane geometry.  Three planes per tensor, line-major: exps (one byte per block), micro
// (LSB-first stream of d2-bit fields, one per sub-block), elems (LSB-first stream of (m+1)-bit
// codes, sign in the top bit).  Default line pitch: rounded up to 16 bytes.
int orc_packed_sizes(const orc_config* c, int64_t rows, int64_t cols, int axis, int64_t ld_out[3],
                     int64_t bytes_out[3]) {
    if (!config_ok(c) || c->scale_kind != ORC_POW2) return ORC_BAD;
    LineView v = make_view(rows, cols, cols, axis);
    int64_t nb = (v.len + c->k1 - 1) / c->k1;
    int64_t line[3] = {nb, (nb * (c->k1 / c->k2) * c->d2 + 7) / 8, (nb * c->k1 * (c->m + 1) + 7) / 8};
    for (int i = 0; i < 3; ++i) {
        ld_out[i] = round_up(line[i], 16);
        bytes_out[i] = ld_out[i] * v.nlines;
    }
    return ORC_OK;
}

int orc_pack(const orc_config* c, const float* x, int64_t rows, int64_t cols, int64_t ld, int axis, uint8_t* exps,
             uint8_t* micro, uint8_t* elems, int64_t ld_exps, int64_t ld_micro, int64_t ld_elems) {
    if (!config_ok(c) || c->scale_kind != ORC_POW2 || !x || ld < cols) return ORC_BAD;
    LineView v = make_view(rows, cols, ld, axis);
    int64_t nb = (v.len + c->k1 - 1) / c->k1;
    int nsub = c->k1 / c->k2;
    std::vector<uint8_t> tau(nsub);
    std::vector<uint16_t> code(c->k1);
    for (int64_t l = 0; l < v.nlines; ++l) {
        std::memset(exps + l * ld_exps, 0, ld_exps);
        if (ld_micro) std::memset(micro + l * ld_micro, 0, ld_micro);
        std::memset(elems + l * ld_elems, 0, ld_elems);
        for (int64_t b = 0; b < nb; ++b) {
            int n = (int)std::min<int64_t>(c->k1, v.len - b * c->k1);
            uint8_t F;
            pow2_block(*c, x + l * v.line_stride + b * c->k1 * v.elem_stride, v.elem_stride, n, &F, tau.data(),
                       code.data(), nullptr, 0);
            exps[l * ld_exps + b] = F;
            for (int j = 0; j < nsub; ++j)
                if (c->d2) put_bits(micro + l * ld_micro, (b * nsub + j) * (int64_t)c->d2, c->d2, tau[j]);
            for (int i = 0; i < c->k1; ++i)
                put_bits(elems + l * ld_elems, (b * c->k1 + i) * (int64_t)(c->m + 1), c->m + 1, code[i]);
        }
    }
    return ORC_OK;
}

// Decode packed planes back to fp32 values: (-1)^s * q * 2^(F-127-tau-(m-1)).
int orc_unpack(const orc_config* c, const uint8_t* exps, const uint8_t* micro, const uint8_t* elems, int64_t ld_exps,
               int64_t ld_micro, int64_t ld_elems, float* y, int64_t rows, int64_t cols, int64_t ld, int axis) {
    if (!config_ok(c) || c->scale_kind != ORC_POW2 || !y || ld < cols) return ORC_BAD;
    LineView v = make_view(rows, cols, ld, axis);
    int nsub_per_block = c->k1 / c->k2;
    for (int64_t l = 0; l < v.nlines; ++l)
        for (int64_t i = 0; i < v.len; ++i) {
            int64_t b = i / c->k1;
            int64_t j = b * nsub_per_block + (i % c->k1) / c->k2;
            int F = exps[l * ld_exps + b];
            float out;
            if (F == 0xFF) {
                out = u2f(0x7FC00000u);
            } else {
                int tau = c->d2 ? (int)get_bits(micro + l * ld_micro, j * (int64_t)c->d2, c->d2) : 0;
                uint32_t code = get_bits(elems + l * ld_elems, i * (int64_t)(c->m + 1), c->m + 1);
                uint32_t q = code & ((1u << c->m) - 1), s = code >> c->m;
                float mag = (float)std::ldexp((double)q, (F - 127) - tau - (c->m - 1));
                out = u2f(f2u(mag) | (s << 31));
            }
            y[l * v.line_stride + i * v.elem_stride] = out;
        }
    return ORC_OK;
}

// Element-wise rounding to a small float format (exposed so tests can pin it against a library cast).
void orc_minifloat_round(const float* in, float* out, int64_t n, int ebits, int mbits, int rounding) {
    for (int64_t i = 0; i < n; ++i) out[i] = minifloat_round(in[i], ebits, mbits, rounding);
}

// C[M,N] = A[M,K] * B[N,K]^T in fp64 (the plain definition; used as the mx_gemm reference).
void orc_gemm_nt_f64(const float* a, const float* b, int64_t M, int64_t N, int64_t K, double* c, int nthreads) {
    auto work = [=](int64_t i0, int64_t i1) {
        for (int64_t i = i0; i < i1; ++i)
            for (int64_t j = 0; j < N; ++j) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) acc += (double)a[i * K + k] * (double)b[j * K + k];
                c[i * N + j] = acc;
            }
    };
    if (nthreads <= 1) { work(0, M); return; }
    std::vector<std::thread> th;
    int64_t per = (M + nthreads - 1) / nthreads;
    for (int t = 0; t < nthreads; ++t) {
        int64_t i0 = t * per, i1 = std::min<int64_t>(M, i0 + per);
        if (i0 < i1) th.emplace_back(work, i0, i1);
    }
    for (auto& t : th) t.join();
}

// Selected entries of the same product: c[s] = sum_k A[ri[s],k] * B[ci[s],k].
void orc_gemm_nt_f64_sampled(const float* a, const float* b, int64_t K, const int64_t* ri, const int64_t* ci,
                             int64_t nsamp, double* c) {
    for (int64_t s = 0; s < nsamp; ++s) {
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k) acc += (double)a[ri[s] * K + k] * (double)b[ci[s] * K + k];
        c[s] = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// Dot product as the hardware pipeline of Section IV-B (Fig. 6) computes it, C = A B^T with both
// operands quantized along K in a POW2 format (same k1, k2, d2; the mantissa widths may differ).
// The paper describes the pipeline in words; the readings taken here (listed in the design notes):
//   1. Inside a k1-block the integer mantissa products (sign-magnitude) are summed exactly.  The
//      products of sub-block j are summed first (depth log2 k2), then aligned by the two operands'
//      shifts: the sub-block sum S_j enters the block sum with weight 2^(2 beta - tau_A,j - tau_B,j)
//      (the conditional right shift, done on a datapath widened by 2 beta bits so that nothing is
//      lost).  Block result: an integer D_b, |D_b| < 2^W, W = m_A + m_B + log2 k1 + 2 beta, worth
//      D_b * 2^(E_A,b + E_B,b - (m_A - 1) - (m_B - 1) - 2 beta).
//   2. The r/k1 block results of one pass through the pipeline (r consecutive elements of K) are
//      normalised to the largest block exponent sum e_max = max_b (F_A,b + F_B,b) -- every block takes
//      part, also one whose result is zero -- and reduced in fixed point: block b is shifted right by
//      e_max - e_b inside a frame of f magnitude bits whose top bit is the top bit of a W-bit result
//      at e_max, i.e. A_b = trunc(D_b * 2^(f - W - (e_max - e_b))), truncated toward zero (sign-
//      magnitude datapath).  The aligned integers are added exactly.
//   3. The pass's sum leaves the pipeline as an fp32 number (one rounding to nearest even), and
//      successive passes (K > r) are accumulated in fp32 in order of increasing K.
//   4. A block with the exponent byte 0xFF (Inf/NaN input) makes the result NaN.
// ---------------------------------------------------------------------------------------------
static inline int64_t shift_trunc(int64_t v, int sh) {  // v * 2^sh, truncated toward zero
    if (sh >= 0) return sh >= 62 ? 0 : v * ((int64_t)1 << sh);  // callers keep |v| 2^sh below 2^62
    if (-sh >= 63) return 0;
    const int64_t mag = (v < 0 ? -v : v) >> (-sh);
    return v < 0 ? -mag : mag;
}

int orc_gemm_hw(const orc_config* ca, const float* a, int64_t M, const orc_config* cb, const float* b, int64_t N, int64_t K,
                int r, int f, float* c) {
    if (!config_ok(ca) || !config_ok(cb) || ca->scale_kind != ORC_POW2 || cb->scale_kind != ORC_POW2) return ORC_BAD;
    if (ca->k1 != cb->k1 || ca->k2 != cb->k2 || ca->d2 != cb->d2 || ca->rounding != cb->rounding) return ORC_BAD;
    const int k1 = ca->k1, k2 = ca->k2, beta = (1 << ca->d2) - 1;
    if (!a || !b || !c || M < 0 || N < 0 || K < 0 || r < k1 || r % k1 != 0 || K % r != 0) return ORC_BAD;
    int lg = 0;
    while ((1 << lg) < k1) ++lg;
    const int W = ca->m + cb->m + lg + 2 * beta;
    if (f < 1 || f > 40 || W > 40 || r / k1 > 4096) return ORC_BAD;
    const int nb = (int)(K / k1), nsub = k1 / k2;
    // encode both operands row by row
    auto encode_rows = [&](const orc_config& cfg, const float* x, int64_t rows, std::vector<uint8_t>& F, std::vector<uint8_t>& tau,
                           std::vector<int32_t>& q) {
        F.assign(rows * nb, 0);
        tau.assign(rows * nb * nsub, 0);
        q.assign(rows * K, 0);
        std::vector<uint16_t> code(k1);
        for (int64_t i = 0; i < rows; ++i)
            for (int bb = 0; bb < nb; ++bb) {
                pow2_block(cfg, x + i * K + (int64_t)bb * k1, 1, k1, &F[i * nb + bb], &tau[(i * nb + bb) * nsub], code.data(), nullptr, 0);
                for (int e = 0; e < k1; ++e) {
                    const int32_t mag = code[e] & ((1 << cfg.m) - 1);
                    q[i * K + (int64_t)bb * k1 + e] = (code[e] >> cfg.m) & 1 ? -mag : mag;
                }
            }
    };
    std::vector<uint8_t> Fa, Fb, ta, tb;
    std::vector<int32_t> qa, qb;
    encode_rows(*ca, a, M, Fa, ta, qa);
    encode_rows(*cb, b, N, Fb, tb, qb);
    const int bpr = r / k1;  // blocks per pass
    std::vector<int64_t> D(bpr);
    std::vector<int> e(bpr);
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            float acc = 0.f;
            bool nan = false;
            for (int64_t p0 = 0; p0 < nb; p0 += bpr) {
                int emax = 0;
                for (int bb = 0; bb < bpr; ++bb) {
                    const int64_t blk = p0 + bb;
                    const int fa = Fa[i * nb + blk], fb = Fb[j * nb + blk];
                    if (fa == 255 || fb == 255) nan = true;
                    int64_t d = 0;
                    for (int sj = 0; sj < nsub; ++sj) {
                        int64_t sum = 0;
                        for (int t = 0; t < k2; ++t) {
                            const int64_t k = blk * k1 + (int64_t)sj * k2 + t;
                            sum += (int64_t)qa[i * K + k] * (int64_t)qb[j * K + k];
                        }
                        const int sh = 2 * beta - ta[(i * nb + blk) * nsub + sj] - tb[(j * nb + blk) * nsub + sj];
                        d += sum * ((int64_t)1 << sh);
                    }
                    D[bb] = d;
                    e[bb] = fa + fb;
                    emax = std::max(emax, e[bb]);
                }
                int64_t total = 0;
                for (int bb = 0; bb < bpr; ++bb) total += shift_trunc(D[bb], f - W - (emax - e[bb]));
                // value of the frame's unit: 2^(emax - 254 - (mA - 1) - (mB - 1) - 2 beta - (f - W))
                const int unit = emax - 254 - (ca->m - 1) - (cb->m - 1) - 2 * beta - (f - W);
                const float pass = (float)total;                       // one rounding to nearest even (|total| < 2^53)
                const float v = (float)std::ldexp((double)pass, unit);  // exact unless it leaves the fp32 range
                acc = acc + v;
            }
            c[i * N + j] = nan ? std::numeric_limits<float>::quiet_NaN() : acc;
        }
    return ORC_OK;
}

// Three-level scaling (Section III, last paragraph: an extension the paper only sketches): a software FP32
// parent scale over groups of k_parent consecutive elements of a line, above the power-of-two block scale and
// the microexponents.  Reading: the parent scale maps the group's largest magnitude onto the largest value a
// block with exponent 0 can hold, V = (2^m - 1) 2^-(m-1):  s = fl(amax_g / V),  x' = fl(x / s),
// Q3(x) = fl(Q(x') s) with Q the two-level quantizer on the group's k1-blocks.  A group of zeros stays zeros.
int orc_quant_dequant_parent(const orc_config* c, int64_t k_parent, const float* x, float* y, int64_t rows, int64_t cols,
                             int64_t ld, int axis, double* sums) {
    if (!config_ok(c) || c->scale_kind != ORC_POW2 || !x || !y || rows < 0 || cols < 0 || ld < cols || (axis != 0 && axis != 1))
        return ORC_BAD;
    if (k_parent < c->k1 || k_parent % c->k1 != 0) return ORC_BAD;
    LineView v = make_view(rows, cols, ld, axis);
    const float V = (float)((1 << c->m) - 1) * std::ldexp(1.0f, -(c->m - 1));
    std::vector<float> xs(k_parent), qs(k_parent);
    for (int64_t l = 0; l < v.nlines; ++l)
        for (int64_t g0 = 0; g0 < v.len; g0 += k_parent) {
            const int64_t n = std::min<int64_t>(k_parent, v.len - g0);
            const float* xg = x + l * v.line_stride + g0 * v.elem_stride;
            float* yg = y + l * v.line_stride + g0 * v.elem_stride;
            const float amax = absmax(xg, v.elem_stride, n);
            const float s = amax / V;
            if (!(s > 0.f)) {
                for (int64_t i = 0; i < n; ++i) yg[i * v.elem_stride] = with_sign(0.f, xg[i * v.elem_stride]);
                continue;
            }
            for (int64_t i = 0; i < n; ++i) xs[i] = xg[i * v.elem_stride] / s;
            for (int64_t b0 = 0; b0 < n; b0 += c->k1) {
                const int nb = (int)std::min<int64_t>(c->k1, n - b0);
                pow2_block(*c, xs.data() + b0, 1, nb, nullptr, nullptr, nullptr, qs.data() + b0, 1);
            }
            for (int64_t i = 0; i < n; ++i) yg[i * v.elem_stride] = qs[i] * s;
        }
    if (sums) {
        double e2 = 0.0, s2 = 0.0;
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t cc = 0; cc < cols; ++cc) {
                double a = (double)x[r * ld + cc], q = (double)y[r * ld + cc];
                e2 += (q - a) * (q - a);
                s2 += a * a;
            }
        sums[0] = e2;
        sums[1] = s2;
    }
    return ORC_OK;
}

}  // extern "C"
