// Packed bf16x2 arithmetic for the Table II family (k1 = 16, k2 = 2, d2 = 1, m <= 7) on bf16 tensors.
//
// A bf16 tensor arrives as 32-bit words that hold two elements each.  Everything the quantizer of
// the Appendix needs is done on both halves of a word at once with the bf16x2 instructions:
//   a  = |x| * 2^(127-F)                 exact (power-of-two scaling), a < 2
//   r  = min(a + C, C + (2^m-1) ulp)     C = 2^(7-(m-1)-tau): the bf16 adder (8-bit significand) rounds
//                                        a to a multiple of 2^(-(m-1)-tau) = ulp(C), nearest-even,
//                                        and leaves q in the seven mantissa bits of r
//   aq = r - C, Q(x) = aq * 2^(F-127)    exact
// C is a power of two (not 1.5 * 2^k as in the fp32 formulation) because a >= 0: a + C stays inside
// C's binade except for the single value 2C, which the clamp removes.  The Eq. 3 terms (aq - a, a)
// are exact bf16 values; they are squared and summed in fp32 (mixed-precision multiply-add).
// Valid for 16 <= F <= 250 (every constant and result a normal number) and ties-to-even; callers
// send other blocks (tiny, huge, Inf/NaN, ties-away) to the fp32 / integer formulation.
#pragma once

#include "bdr_device.cuh"

namespace bdr {
namespace x2 {

__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hadd2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hsub2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hmin2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hfma2(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t habs2(uint32_t a) {
    uint32_t d;
    asm("abs.bf16x2 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// Maximum that keeps NaNs (either operand NaN -> NaN), so a block with Inf/NaN reports exponent 255.
__device__ __forceinline__ uint32_t hmax2_nan(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// (d0, d1) += (lo * lo, hi * hi) for the two bf16 halves of w, with the mixed-precision multiply-add
// (bf16 operands, fp32 addend and result): the products are exact, each sum is rounded once, and no
// widening instructions are needed.
__device__ __forceinline__ void fma_sq_halves(float& d0, float& d1, uint32_t w) {
    asm("{.reg .b16 lo, hi; mov.b32 {lo, hi}, %2; fma.rn.f32.bf16 %0, lo, lo, %0; fma.rn.f32.bf16 %1, hi, hi, %1;}"
        : "+f"(d0), "+f"(d1)
        : "r"(w));
}

// 2^(2F-254) as a double: the factor that takes a block's Eq. 3 sums out of its normalised domain
__device__ __forceinline__ double pow4_weight(uint32_t F) { return __hiloint2double((int)((F << 21) + 0x30100000u), 0); }

// Where run `wi` of kRun elements starts.  A contiguous tensor is one long row (flat); otherwise a row holds
// runs_per_row runs and rows are ld elements apart.
struct RunIndex {
    FastDiv runs_per_row;
    int64_t ld;
    int flat;
    __device__ __forceinline__ void split(uint32_t wi, int64_t& row, int64_t& pos) const {
        if (flat) {
            row = 0;
            pos = wi;
        } else {
            const uint32_t r = fastdiv(wi, runs_per_row);
            row = r;
            pos = wi - r * runs_per_row.d;
        }
    }
};

constexpr uint32_t kAbs2 = 0x7FFF7FFFu, kSign2 = 0x80008000u;
constexpr int kMinF = 16, kMaxF = 250;

// constants of one mantissa width
struct Consts {
    uint32_t C0, C1;  // 2^(7-(m-1)) and the constant of a shifted sub-block (half of it; the same when d2 = 0)
    uint32_t QM;      // 2^m - 1 in both halves
    uint32_t G1;      // factor of a shifted sub-block: 2.0 (1.0 when d2 = 0)
    uint32_t SID;     // what a shifted sub-block takes off the exponent of 2^(F-127): 0x0080 per half (0 when d2 = 0)
};
__host__ __device__ __forceinline__ Consts make_consts(int m, int d2 = 1) {
    Consts k;
    const uint32_t e0 = (uint32_t)(127 + 7 - (m - 1));
    k.C0 = (e0 << 7) * 0x10001u;
    k.C1 = d2 ? ((e0 - 1) << 7) * 0x10001u : k.C0;
    k.QM = ((1u << m) - 1u) * 0x10001u;
    k.G1 = d2 ? 0x40004000u : 0x3F803F80u;
    k.SID = d2 ? 0x00800080u : 0u;
    return k;
}

// Biased shared exponent of a block given as |x| words (row direction: all 16 halves are one block).
// For non-negative bf16 the float maximum is the maximum of the bit patterns.
__device__ __forceinline__ uint32_t block_exponent(const uint32_t (&aw)[8]) {
    uint32_t mx = hmax2_nan(hmax2_nan(aw[0], aw[1]), hmax2_nan(aw[2], aw[3]));
    mx = hmax2_nan(mx, hmax2_nan(hmax2_nan(aw[4], aw[5]), hmax2_nan(aw[6], aw[7])));
    return max(mx & 0xFFFFu, mx >> 16) >> 7;
}

// Row direction: one block = eight words, sub-block j = word j.
//   yw     dequantized words (YOUT)
//   code2  per word, the two codes (sign << m | q) in bits [0, m] and [16, 16 + m] (CODE)
//   micro  the eight sub-block shifts, bit j = tau of word j (CODE)
//   pe, ps this block's Eq. 3 sums in the normalised domain (SUMS); scale by 2^(2F-254)
template <bool SUMS, bool YOUT, bool CODE>
__device__ __forceinline__ void quantize_block_row(const uint32_t (&w)[8], const uint32_t (&aw)[8], uint32_t F, int m,
                                                   const Consts& k, uint32_t (&yw)[8], uint32_t (&code2)[8],
                                                   uint32_t& micro, float& pe, float& ps) {
    const uint32_t s2 = ((254u - F) << 7) * 0x10001u;  // 2^(127-F)
    const uint32_t si2 = (F << 7) * 0x10001u;          // 2^(F-127)
    float pe0 = 0.f, pe1 = 0.f, ps0 = 0.f, ps1 = 0.f;
    uint32_t macc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t a2 = hmul2(aw[j], s2);
        // a half is >= 1.0 (0x3F80) exactly when adding 0x0080 carries into bit 14
        const bool top = ((a2 + 0x00800080u) & 0x40004000u) != 0;  // tau = 0
        uint32_t r2;
        if constexpr (SUMS) {
            // tau picks the constant; aq and a stay in the block's normalised domain for the sums
            const uint32_t C2 = top ? k.C0 : k.C1;
            r2 = hmin2(hadd2(a2, C2), C2 + k.QM);
            const uint32_t aq2 = hsub2(r2, C2);
            if constexpr (YOUT) yw[j] = hmul2(aq2, si2) | (w[j] & kSign2);
            const uint32_t d2 = hsub2(aq2, a2);  // exact
            fma_sq_halves(pe0, pe1, d2);
            fma_sq_halves(ps0, ps1, a2);
            if constexpr (CODE) macc |= (r2 << (j + 1)) & (0x100u << j);  // bit 7 of r: lowest exponent bit of C
        } else {
            // tau doubles the operand instead (exact), so the constant and the clamp are fixed
            const uint32_t g2 = top ? 0x3F803F80u : k.G1;  // 1.0 or 2.0
            r2 = hmin2(hfma2(a2, g2, k.C0), k.C0 + k.QM);
            if constexpr (YOUT) yw[j] = hmul2(hsub2(r2, k.C0), top ? si2 : si2 - k.SID) | (w[j] & kSign2);
            if constexpr (CODE) macc |= (g2 << (j + 2)) & (0x10000u << j);  // bit 14 of 2.0
        }
        if constexpr (CODE) code2[j] = (r2 & 0x007F007Fu) | ((w[j] >> (15 - m)) & (0x00010001u << m));
    }
    if constexpr (SUMS) { pe = pe0 + pe1; ps = ps0 + ps1; }
    if constexpr (CODE) {
        if constexpr (SUMS) {
            const uint32_t e0 = (uint32_t)(127 + 7 - (m - 1));  // exponent of C0: tau = bit ^ (e0 & 1)
            micro = ((macc >> 8) ^ ((e0 & 1u) ? 0xFFu : 0u)) & 0xFFu;
        } else {
            micro = (macc >> 16) & 0xFFu;
        }
    }
}

// The sixteen W-bit codes of a block, from code2[], as the little-endian bit stream (W = m + 1).
template <int W>
__device__ __forceinline__ void pack_block(const uint32_t (&code2)[8], uint32_t (&cw)[(16 * W + 31) / 32]) {
    if constexpr (W == 8) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cw[i] = __byte_perm(code2[2 * i], code2[2 * i + 1], 0x6420);
    } else {
        uint32_t f[8];  // the two codes of a word side by side: 2W bits
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = (code2[j] | (code2[j] >> (16 - W))) & ((1u << (2 * W)) - 1u);
        if constexpr (W == 3) {
            const uint32_t lo = f[0] + (f[1] << 6) + (f[2] << 12) + (f[3] << 18);
            const uint32_t hi = f[4] + (f[5] << 6) + (f[6] << 12) + (f[7] << 18);
            cw[0] = lo | (hi << 24);
            cw[1] = hi >> 8;
        } else {
            static_assert(W == 5, "code widths of Table II");
            const uint32_t g0 = f[0] + (f[1] << 10) + (f[2] << 20);
            const uint32_t g1 = f[3] + (f[4] << 10) + (f[5] << 20);
            const uint32_t g2 = f[6] + (f[7] << 10);
            cw[0] = g0 | (g1 << 30);
            cw[1] = (g1 >> 2) | (g2 << 28);
            cw[2] = g2 >> 4;
        }
    }
}

// ---- packing without dequantized output or sums: fewest integer-pipe instructions ----------------------
// The integer/logic pipe issues at half the rate of the FMA pipe, so this route keeps per-element work
// on packed floating-point instructions wherever it can:
//   * words are regrouped so that the two elements of a sub-block sit in the SAME half of two words
//     (A = {x0, x2}, B = {x1, x3} from {x0, x1}, {x2, x3}); one packed maximum then yields both
//     sub-block maxima of the pair, and everything after it treats the halves independently;
//   * tau as arithmetic: u = relu(256 pm - 255) is 0 for pm < 1 and >= 1 otherwise (pm is the scaled
//     sub-block maximum, a bf16 below 2), so g = 2 - min(u, 1) is the factor 2^tau that lines the
//     sub-block up with the fixed constant C0;
//   * the sign joins the magnitude arithmetically (m <= 6): with the constant raised by 1.0 = 2^(m-1)
//     units, r - sgn(x) has mantissa q for x >= 0 and 2^m + q for x < 0, i.e. the code itself.
// Words of the regrouped block: pair i (i = 0..3) covers elements 4i .. 4i+3.
__device__ __forceinline__ uint32_t hfma2_relu(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.relu.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

struct PairView {
    uint32_t A[4], B[4];    // regrouped words
    uint32_t aA[4], aB[4];  // their magnitudes
    uint32_t pm[4];         // sub-block maxima: low half sub-block 2i, high half sub-block 2i+1
};

__device__ __forceinline__ uint32_t pair_view(const uint32_t (&w)[8], PairView& v) {  // returns F
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v.A[i] = __byte_perm(w[2 * i], w[2 * i + 1], 0x5410);
        v.B[i] = __byte_perm(w[2 * i], w[2 * i + 1], 0x7632);
        v.aA[i] = habs2(v.A[i]);
        v.aB[i] = habs2(v.B[i]);
        v.pm[i] = hmax2_nan(v.aA[i], v.aB[i]);
    }
    const uint32_t mx = hmax2_nan(hmax2_nan(v.pm[0], v.pm[1]), hmax2_nan(v.pm[2], v.pm[3]));
    return max(mx & 0xFFFFu, mx >> 16) >> 7;
}

template <int W, bool SUMS = false>
__device__ __forceinline__ void pack_pair_view(const PairView& v, uint32_t F, uint32_t (&cw)[(16 * W + 31) / 32], uint32_t& micro,
                                               float* pe = nullptr, float* ps = nullptr) {
    constexpr int M = W - 1;
    constexpr uint32_t e0 = (uint32_t)(127 + 7 - (M - 1));
    constexpr bool kSignTrick = M <= 6;
    constexpr uint32_t C0 = ((e0 << 7) + (kSignTrick ? (1u << (M - 1)) : 0u)) * 0x10001u;  // C0 (+ 1.0 = 2^(m-1) units)
    constexpr uint32_t Cmax = C0 + ((1u << M) - 1u) * 0x10001u;
    const uint32_t s2 = ((254u - F) << 7) * 0x10001u;  // 2^(127-F)
    uint32_t macc = 0, f4[4];
    [[maybe_unused]] float pe0 = 0.f, pe1 = 0.f, ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t u = hfma2_relu(hmul2(v.pm[i], s2), 0x43804380u, 0xC37FC37Fu);  // relu(256 pm - 255)
        const uint32_t mn = hmin2(u, 0x3F803F80u);                                    // 1 - tau
        const uint32_t g = hsub2(0x40004000u, mn);                                    // 2^tau per half
        macc += g << (2 * i);
        const uint32_t tA = hmul2(v.aA[i], s2), tB = hmul2(v.aB[i], s2);
        uint32_t rA = hmin2(hfma2(tA, g, C0), Cmax);
        uint32_t rB = hmin2(hfma2(tB, g, C0), Cmax);
        if constexpr (SUMS) {
            // Eq. 3 sums in the block's normalised domain: the quantized magnitude is (r - C0) 2^-tau, the difference is exact
            const uint32_t ngi = hfma2(mn, 0xBF00BF00u, 0xBF00BF00u);  // -2^-tau
            const uint32_t dA = hfma2(hsub2(rA, C0), ngi, tA), dB = hfma2(hsub2(rB, C0), ngi, tB);
            fma_sq_halves(pe0, pe1, dA);
            fma_sq_halves(pe0, pe1, dB);
            fma_sq_halves(ps0, ps1, tA);
            fma_sq_halves(ps0, ps1, tB);
        }
        if constexpr (kSignTrick) {
            rA = hsub2(rA, (v.A[i] & kSign2) | 0x3F803F80u);  // -/+ 1.0
            rB = hsub2(rB, (v.B[i] & kSign2) | 0x3F803F80u);
            constexpr uint32_t kCode = ((1u << W) - 1u) * 0x10001u;
            const uint32_t comb = (rA & kCode) + ((rB & kCode) << W);  // halves: codes 4i, 4i+1 | codes 4i+2, 4i+3
            // the two halves side by side: 4 codes, 4W bits
            if constexpr (3 * W <= 10) f4[i] = (comb | (comb >> (16 - 2 * W))) & ((1u << (4 * W)) - 1u);  // shifted low half falls off
            else f4[i] = (comb & ((1u << (2 * W)) - 1u)) | ((comb >> (16 - 2 * W)) & (((1u << (2 * W)) - 1u) << (2 * W)));
        } else {
            // W = 8: byte 0 / 2 of each word = sign bit over the seven magnitude bits; bytes 1 / 3 are not used
            const uint32_t cA = ((v.A[i] >> 8) & 0x00800080u) | (rA & ~0x00800080u);
            const uint32_t cB = ((v.B[i] >> 8) & 0x00800080u) | (rB & ~0x00800080u);
            f4[i] = __byte_perm(cA, cB, 0x6240);
        }
    }
    if constexpr (W == 8) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cw[i] = f4[i];
    } else if constexpr (W == 3) {
        cw[0] = f4[0] + (f4[1] << 12) + (f4[2] << 24);
        cw[1] = (f4[2] >> 8) + (f4[3] << 4);
    } else {
        static_assert(W == 3 || W == 5 || W == 8, "code widths of Table II");
        cw[0] = f4[0] + (f4[1] << 20);
        cw[1] = (f4[1] >> 12) + (f4[2] << 8) + (f4[3] << 28);
        cw[2] = f4[3] >> 4;
    }
    // g is 0x3F80 + 0x80 tau per half: remove the constant part, then bit 7+2i = tau of sub-block 2i and
    // bit 23+2i = tau of sub-block 2i+1
    const uint32_t t = macc - 0x3F803F80u * 0x55u;
    micro = ((t >> 7) & 0x55u) | ((t >> 22) & 0xAAu);
    if constexpr (SUMS) { *pe = pe0 + pe1; *ps = ps0 + ps1; }
}

// Slow route for one block (exponent outside the packed range, Inf/NaN, ties-away): the fp32 /
// integer formulation on widened values.  Kept out of line so the hot loop stays small.
struct SlowOut {
    uint4 y[2];
    uint32_t cw[4];
    uint32_t F, micro;
    double e2, s2;
};
// F_ext: the shared exponent when the block is wider than these sixteen elements (k1 > 16), else 0.
template <int W, bool SUMS>
__device__ __noinline__ SlowOut quantize_block_slow(uint4 w0, uint4 w1, QParams qp, uint32_t F_ext = 0) {
    SlowOut o;
    const uint4 w[2] = {w0, w1};
    uint32_t u[kSlice], yb[kSlice], rq[kSlice], cb[kSlice / 2], tau[kSlice / 2], fj[kSlice / 2], fb[1];
    SliceWords<__nv_bfloat16>::expand(w, u);
    subblock_exponents<2>(u, fj);
    uint32_t F = 0;
#pragma unroll
    for (int j = 0; j < kSlice / 2; ++j) F = max(F, fj[j]);
    if (qp.k1 > kSlice) F = F_ext << 23;
    fb[0] = F;
    o.e2 = 0.0;
    o.s2 = 0.0;
    quantize_slice<2, kSlice, SUMS, true, true>(u, fj, fb, qp, yb, rq, cb, tau, o.e2, o.s2);
    slice_to_words(yb, o.y, (const __nv_bfloat16*)nullptr);
    o.F = F >> 23;
    uint32_t mb = 0;
#pragma unroll
    for (int j = 0; j < kSlice / 2; ++j) mb |= tau[j] << j;
    o.micro = mb;
#pragma unroll
    for (int i = 0; i < 4; ++i) o.cw[i] = 0;
    if constexpr (W > 0) {
        uint32_t words[(kSlice * W + 31) / 32];
        pack_words<W, kSlice, 2>(u, rq, cb, words);
#pragma unroll
        for (int i = 0; i < (kSlice * W + 31) / 32; ++i) o.cw[i] = words[i];
    }
    return o;
}

// ---- column direction ---------------------------------------------------------------------------------
// A "word column" is sixteen words w[r], r = 0..15: rows r of two adjacent columns (low half = the even
// column).  Each half is a block of its own, so everything runs on both halves independently: packed
// maxima give the two shared exponents, F2 holds them in place (bits 14..7 of each half), and the
// sub-block of rows 2j, 2j+1 has its maximum in pm[j].
struct WordColOut {
    uint32_t F2;           // shared exponents, (F << 7) per half
    uint32_t micro_lo, micro_hi;
    float pe_lo, pe_hi, ps_lo, ps_hi;  // Eq. 3 sums of the two blocks in their normalised domains
};

__device__ __forceinline__ bool wordcol_exponents(const uint32_t (&w)[16], uint32_t (&aw)[16], uint32_t (&pm)[8], uint32_t& F2) {
#pragma unroll
    for (int r = 0; r < 16; ++r) aw[r] = habs2(w[r]);
#pragma unroll
    for (int j = 0; j < 8; ++j) pm[j] = hmax2_nan(aw[2 * j], aw[2 * j + 1]);
    const uint32_t mx = hmax2_nan(hmax2_nan(hmax2_nan(pm[0], pm[1]), hmax2_nan(pm[2], pm[3])),
                                  hmax2_nan(hmax2_nan(pm[4], pm[5]), hmax2_nan(pm[6], pm[7])));
    F2 = mx & 0x7F807F80u;
    const uint32_t f_lo = (F2 >> 7) & 0xFFu, f_hi = F2 >> 23;
    return (f_lo - kMinF <= (uint32_t)(kMaxF - kMinF)) && (f_hi - kMinF <= (uint32_t)(kMaxF - kMinF));
}

// code streams of the two columns from the sixteen per-row code words (code of the even column in the
// low half, W clean bits; for W = 8 only bytes 0 and 2 need to be clean)
template <int W>
__device__ __forceinline__ void wordcol_streams(const uint32_t (&code)[16], uint32_t (&cl)[(16 * W + 31) / 32],
                                                uint32_t (&ch)[(16 * W + 31) / 32]) {
    if constexpr (W == 8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t p = __byte_perm(code[4 * k], code[4 * k + 1], 0x6240);      // rows 4k, 4k+1: low column | high column
            const uint32_t q = __byte_perm(code[4 * k + 2], code[4 * k + 3], 0x6240);  // rows 4k+2, 4k+3
            cl[k] = __byte_perm(p, q, 0x5410);
            ch[k] = __byte_perm(p, q, 0x7632);
        }
    } else {
        uint32_t t[8];  // rows 2j, 2j+1 side by side in each half: 2W bits
#pragma unroll
        for (int j = 0; j < 8; ++j) t[j] = code[2 * j] + (code[2 * j + 1] << W);
        if constexpr (W == 3) {
            uint32_t lo[4], hi[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t q4 = t[2 * i] + (t[2 * i + 1] << 6);  // rows 4i .. 4i+3: 12 bits per half
                lo[i] = q4 & 0xFFFFu;
                hi[i] = q4 >> 16;
            }
            cl[0] = lo[0] + (lo[1] << 12) + (lo[2] << 24);
            cl[1] = (lo[2] >> 8) + (lo[3] << 4);
            ch[0] = hi[0] + (hi[1] << 12) + (hi[2] << 24);
            ch[1] = (hi[2] >> 8) + (hi[3] << 4);
        } else {
            static_assert(W == 3 || W == 5 || W == 8, "code widths of Table II");
            uint32_t lo[8], hi[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { lo[j] = t[j] & 0xFFFFu; hi[j] = t[j] >> 16; }
            cl[0] = lo[0] + (lo[1] << 10) + (lo[2] << 20) + (lo[3] << 30);
            cl[1] = (lo[3] >> 2) + (lo[4] << 8) + (lo[5] << 18) + (lo[6] << 28);
            cl[2] = (lo[6] >> 4) + (lo[7] << 6);
            ch[0] = hi[0] + (hi[1] << 10) + (hi[2] << 20) + (hi[3] << 30);
            ch[1] = (hi[3] >> 2) + (hi[4] << 8) + (hi[5] << 18) + (hi[6] << 28);
            ch[2] = (hi[6] >> 4) + (hi[7] << 6);
        }
    }
}

// Fast path of one word column (the caller has checked both exponents with wordcol_exponents).
//   W > 0: code streams cl / ch and the micro bytes; YOUT: dequantized words; SUMS: the four partial sums.
template <int W, bool SUMS, bool YOUT>
__device__ __forceinline__ void quantize_wordcol(const uint32_t (&w)[16], const uint32_t (&aw)[16], const uint32_t (&pm)[8],
                                                 uint32_t F2, int m, uint32_t (&yw)[16],
                                                 uint32_t (&cl)[W > 0 ? (16 * W + 31) / 32 : 1],
                                                 uint32_t (&ch)[W > 0 ? (16 * W + 31) / 32 : 1], WordColOut& o) {
    constexpr bool PACK = W > 0;
    constexpr bool kPackOnly = PACK && !YOUT;  // codes (and perhaps sums) only: the formulation with the fixed constant
    constexpr bool kSignTrick = kPackOnly && W - 1 <= 6;
    const uint32_t e0 = (uint32_t)(127 + 7 - (m - 1));
    const uint32_t C0 = ((e0 << 7) + (kSignTrick ? (1u << (m - 1)) : 0u)) * 0x10001u;
    const uint32_t QM = ((1u << m) - 1u) * 0x10001u;
    const uint32_t s2 = 0x7F007F00u - F2;  // 2^(127-F) per half
    uint32_t code[16];
    uint32_t macc = 0;
    float pe0 = 0.f, pe1 = 0.f, ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t u = hfma2_relu(hmul2(pm[j], s2), 0x43804380u, 0xC37FC37Fu);  // relu(256 pm - 255): 0 iff tau = 1
        const uint32_t v = hmin2(u, 0x3F803F80u);                                   // 1.0 (tau = 0) or 0.0
        if constexpr (kPackOnly) {
            const uint32_t g = hsub2(0x40004000u, v);  // 2^tau
            macc += g << j;
            [[maybe_unused]] const uint32_t ngi = hfma2(v, 0xBF00BF00u, 0xBF00BF00u);  // -2^-tau
#pragma unroll
            for (int r = 2 * j; r < 2 * j + 2; ++r) {
                const uint32_t a2 = hmul2(aw[r], s2);
                uint32_t r2 = hmin2(hfma2(a2, g, C0), C0 + QM);
                if constexpr (SUMS) {
                    // the quantized magnitude in the block's normalised domain is (r - C0) 2^-tau; the difference is exact
                    const uint32_t d2 = hfma2(hsub2(r2, C0), ngi, a2);
                    fma_sq_halves(pe0, pe1, d2);
                    fma_sq_halves(ps0, ps1, a2);
                }
                if constexpr (kSignTrick) {
                    r2 = hsub2(r2, (w[r] & kSign2) | 0x3F803F80u);
                    code[r] = r2 & (((1u << W) - 1u) * 0x10001u);
                } else {
                    code[r] = ((w[r] >> 8) & 0x00800080u) | (r2 & ~0x00800080u);  // bytes 1 and 3 hold leftovers
                }
            }
        } else {
            const uint32_t ginv = hfma2(v, 0x3F003F00u, 0x3F003F00u);  // 2^-tau
            const uint32_t C2 = hmul2(C0, ginv);
            macc += ginv << j;
#pragma unroll
            for (int r = 2 * j; r < 2 * j + 2; ++r) {
                const uint32_t a2 = hmul2(aw[r], s2);
                const uint32_t r2 = hmin2(hadd2(a2, C2), C2 + QM);
                const uint32_t aq2 = hsub2(r2, C2);
                if constexpr (YOUT) yw[r] = hmul2(aq2, F2) | (w[r] & kSign2);
                if constexpr (SUMS) {
                    const uint32_t d2 = hsub2(aq2, a2);  // exact
                    fma_sq_halves(pe0, pe1, d2);
                    fma_sq_halves(ps0, ps1, a2);
                }
                if constexpr (PACK) {
                    if constexpr (W == 8) code[r] = ((w[r] >> 8) & 0x00800080u) | (r2 & 0x007F007Fu);
                    else code[r] = (r2 & (((1u << (W - 1)) - 1u) * 0x10001u)) | ((w[r] >> (16 - W)) & (0x00010001u << (W - 1)));
                }
            }
        }
    }
    o.F2 = F2;
    if constexpr (SUMS) { o.pe_lo = pe0; o.pe_hi = pe1; o.ps_lo = ps0; o.ps_hi = ps1; }
    if constexpr (PACK) {
        wordcol_streams<PACK ? W : 8>(code, cl, ch);
        // per half the accumulated factors are 0x3F80 + 0x80 tau (2^tau) or 0x3F80 - 0x80 tau (2^-tau), shifted by j
        const uint32_t t = kPackOnly ? macc - 0x3F803F80u * 255u : 0x3F803F80u * 255u - macc;
        o.micro_lo = (t >> 7) & 0xFFu;
        o.micro_hi = (t >> 23) & 0xFFu;
    }
}

// Slow route for one word column: the fp32 / integer formulation on each of the two blocks.
struct WordCol {
    uint32_t w[16];
};
struct WordColSlow {
    uint32_t y[16];
    uint32_t cl[4], ch[4];
    uint32_t F2, micro_lo, micro_hi;
    double e2, s2;
};
template <int W, bool SUMS>
__device__ __noinline__ WordColSlow quantize_wordcol_slow(WordCol in, QParams qp) {
    WordColSlow o;
    o.e2 = 0.0;
    o.s2 = 0.0;
    uint32_t Fs[2], ms[2], yb[2][kSlice];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t u[kSlice], rq[kSlice], cb[kSlice / 2], tau[kSlice / 2], fj[kSlice / 2], fb[1];
#pragma unroll
        for (int r = 0; r < kSlice; ++r) u[r] = h ? (in.w[r] & 0xFFFF0000u) : (in.w[r] << 16);
        subblock_exponents<2>(u, fj);
        uint32_t F = 0;
#pragma unroll
        for (int j = 0; j < kSlice / 2; ++j) F = max(F, fj[j]);
        fb[0] = F;
        quantize_slice<2, kSlice, SUMS, true, true>(u, fj, fb, qp, yb[h], rq, cb, tau, o.e2, o.s2);
        Fs[h] = F >> 23;
        uint32_t mb = 0;
#pragma unroll
        for (int j = 0; j < kSlice / 2; ++j) mb |= tau[j] << j;
        ms[h] = mb;
        uint32_t* dst = h ? o.ch : o.cl;
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = 0;
        if constexpr (W > 0) {
            uint32_t words[(kSlice * W + 31) / 32];
            pack_words<W, kSlice, 2>(u, rq, cb, words);
#pragma unroll
            for (int i = 0; i < (kSlice * W + 31) / 32; ++i) dst[i] = words[i];
        }
    }
#pragma unroll
    for (int r = 0; r < kSlice; ++r) o.y[r] = (yb[0][r] >> 16) | (yb[1][r] & 0xFFFF0000u);
    o.F2 = (Fs[0] << 7) | (Fs[1] << 23);
    o.micro_lo = ms[0];
    o.micro_hi = ms[1];
    return o;
}

// ---- decoding -----------------------------------------------------------------------------------------
// value = q * 2^p, p = F - 127 - tau - (m - 1).  The bf16 number 128 + q is built by ORing q into the
// mantissa of 128.0, and fma(128 + q, 2^p, -128 * 2^p) is exactly q * 2^p, two elements at a time.
// Needs every scale normal: kMinF <= F <= kMaxDecodeF; other blocks (and NaN blocks) go the slow way.
constexpr int kMaxDecodeF = 240;

// The two codes of sub-block j of a little-endian stream of W-bit codes, in bits [0, W) and [16, 16 + W)
// (other bits hold leftovers that the callers mask away).
template <int W, int NW>
__device__ __forceinline__ uint32_t code_pair(const uint32_t (&s)[NW], int j) {
    if constexpr (W == 8) {
        return __byte_perm(s[j >> 1], 0u, (j & 1) ? 0x4342 : 0x4140);
    } else {
        const int bit = 2 * W * j, wi = bit >> 5, sh = bit & 31;
        uint32_t f = sh == 0 ? s[wi] : (sh + 2 * W > 32 ? __funnelshift_r(s[wi], s[wi + 1], sh) : s[wi] >> sh);
        f &= (1u << (2 * W)) - 1u;
        return f * (1u + (1u << (16 - W)));  // no carries: 3W <= 16
    }
}

// Row direction: the W words s[] hold two adjacent blocks (32 codes); F0 / F1 their exponents, mb their
// microexponent bytes (block 0 in bits 0..7).  Both exponents must be in the fast range.
template <int W>
__device__ __forceinline__ void decode_two_blocks_row(const uint32_t (&s)[W], uint32_t F0, uint32_t F1, uint32_t mb,
                                                      uint32_t (&yw)[16]) {
    constexpr int M = W - 1;
    constexpr uint32_t kQ2 = ((1u << M) - 1u) * 0x10001u;
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        const uint32_t F = b ? F1 : F0, mbb = b ? mb >> 8 : mb;
        const uint32_t sc0 = ((F - (uint32_t)(M - 1)) << 7) * 0x10001u;  // 2^p for tau = 0
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t c2 = code_pair<W, W>(s, 8 * b + j);
            // tau lowers the exponent by one: sc0 - 0x0080 per half, as one multiply-add; the constant term
            // -128 * 2^p is a packed multiply (both on the FMA pipe, the integer pipe is the busy one)
            const uint32_t sc = ((mbb << (7 - j)) & 0x80u) * 0xFFFEFFFFu + sc0;
            yw[8 * b + j] = hfma2((c2 & kQ2) | 0x43004300u, sc, hmul2(sc, 0xC300C300u)) | ((c2 << (15 - M)) & kSign2);
        }
    }
}

// Slow route: the fp32 decoder on each block, then back to packed bf16.
template <int W> struct TwoBlocks {
    uint32_t s[W];
};
struct TwoBlocksOut {
    uint32_t y[16];
};
template <int W>
__device__ __noinline__ TwoBlocksOut decode_two_blocks_slow(TwoBlocks<W> in, uint32_t F0, uint32_t F1, uint32_t mb) {
    TwoBlocksOut o;
    constexpr int NW = (kSlice * W + 31) / 32;
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        uint32_t words[NW + 1], yb[kSlice];
#pragma unroll
        for (int i = 0; i <= NW; ++i) words[i] = 0;
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            if (b == 0) {
                words[i] = in.s[i];
            } else if constexpr (W % 2 == 0) {
                words[i] = in.s[W / 2 + i];
            } else {
                words[i] = __byte_perm(in.s[W / 2 + i], W / 2 + i + 1 < W ? in.s[W / 2 + i + 1] : 0u, 0x5432);
            }
        }
        decode_slice_impl<W, false>(words, (int)(b ? F1 : F0), b ? (mb >> 8) & 0xFFu : mb & 0xFFu, yb);
#pragma unroll
        for (int k = 0; k < 8; ++k) o.y[8 * b + k] = (yb[2 * k] >> 16) | (yb[2 * k + 1] & 0xFFFF0000u);
    }
    return o;
}

// Column direction: sl[] / sh[] are the streams of the even / odd column over a pair of block rows (32 codes
// each, block row i at bit 16 W i).  Decodes block row i of both columns into the sixteen row words.
// F2 = the two exponents as (F << 7) per half, mm = the two microexponent bytes (odd column in bits 16..23).
template <int W>
__device__ __forceinline__ uint32_t code_pair_col(const uint32_t (&sl)[W], const uint32_t (&sh)[W], int idx /* 0..31 */) {
    if constexpr (W == 8) {
        const int x = idx & 3;
        return __byte_perm(sl[idx >> 2], sh[idx >> 2], ((4 + x) << 12) | ((4 + x) << 8) | (x << 4) | x);  // bytes 1, 3: leftovers
    } else {
        const int bit = W * idx, wi = bit >> 5, sft = bit & 31;
        uint32_t lo = sft == 0 ? sl[wi] : (sft + W > 32 ? __funnelshift_r(sl[wi], sl[wi + 1], sft) : sl[wi] >> sft);
        const uint32_t hi = sft == 0 ? sh[wi] : (sft + W > 32 ? __funnelshift_r(sh[wi], sh[wi + 1], sft) : sh[wi] >> sft);
        lo &= (1u << W) - 1u;
        return lo + (hi << 16);  // bits above 16 + W hold leftovers
    }
}

template <int W>
__device__ __forceinline__ void decode_wordcol(const uint32_t (&sl)[W], const uint32_t (&sh)[W], int i, uint32_t F2, uint32_t mm,
                                               uint32_t (&yw)[16]) {
    constexpr int M = W - 1;
    constexpr uint32_t kQ2 = ((1u << M) - 1u) * 0x10001u;
    const uint32_t sc0 = F2 - ((uint32_t)(M - 1) << 7) * 0x10001u;  // 2^p for tau = 0, per half
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t t = (mm << (7 - j)) & 0x00800080u;
        const uint32_t sc = sc0 - t, nb = hmul2(sc, 0xC300C300u);  // 2^p and -128 * 2^p
#pragma unroll
        for (int r = 2 * j; r < 2 * j + 2; ++r) {
            const uint32_t c2 = code_pair_col<W>(sl, sh, 16 * i + r);
            yw[r] = hfma2((c2 & kQ2) | 0x43004300u, sc, nb) | ((c2 << (15 - M)) & kSign2);
        }
    }
}

// Slow route for block row i of a word column.
template <int W>
__device__ __noinline__ TwoBlocksOut decode_wordcol_slow(TwoBlocks<W> lo, TwoBlocks<W> hi, int i, uint32_t F_lo, uint32_t F_hi,
                                                         uint32_t m_lo, uint32_t m_hi) {
    TwoBlocksOut o;
    constexpr int NW = (kSlice * W + 31) / 32;
    uint32_t yb[2][kSlice];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t* s = h ? hi.s : lo.s;
        uint32_t words[NW + 1];
#pragma unroll
        for (int k = 0; k <= NW; ++k) words[k] = 0;
#pragma unroll
        for (int k = 0; k < NW; ++k) {
            const uint32_t a0 = s[k], b0 = (W % 2 == 0) ? s[(W / 2 + k) % W] : __byte_perm(s[(W / 2 + k) % W], W / 2 + k + 1 < W ? s[(W / 2 + k + 1) % W] : 0u, 0x5432);
            words[k] = i ? b0 : a0;
        }
        decode_slice_impl<W, false>(words, (int)(h ? F_hi : F_lo), h ? m_hi : m_lo, yb[h]);
    }
#pragma unroll
    for (int r = 0; r < kSlice; ++r) o.y[r] = (yb[0][r] >> 16) | (yb[1][r] & 0xFFFF0000u);
    return o;
}

}  // namespace x2
}  // namespace bdr
