// bdr_qsnr: the design-space sweep of Section IV -- QSNR (Eq. 3) of one tensor under many
// configurations, reading the tensor once per group of 16 families of configurations.
//
// The host merges configurations that differ only in the mantissa width m into families of up to
// eight members (same k1, k2, d2, kind and tie rule).  A work unit of a CTA is four tiles of 4096
// consecutive elements of a line (a row, or a column for axis 0) held in shared memory as fp32 bit
// patterns, each with a pyramid of block-maximum exponent bytes for block sizes 2, 4, ..., 1024 (every k1
// and k2 of the grid is one of its levels).  All warps of the CTA then work on the same family at the
// same time, one 16-element slice per thread and tile: exponents and shifts are computed once per slice,
// the loop over the family's mantissa widths only changes the rounding constant and the clamp, and
// sum (Q(x)-x)^2 is formed as in the quantize kernels.  A lane's sums are reduced once per family into
// per-CTA accumulators in shared memory; only at the end does a CTA touch the global sums (one atomic
// per configuration), so the tensor is read from HBM once per 16 families and the kernel is bound by
// plain ALU throughput.
//
// The comparator kinds of Table I (INT with an FP32 max-scale, Eq. 1-2; FP8-like scalar floats;
// VSQ) are evaluated in the same loop; their divisions are exact IEEE single divisions (computed by a
// multiply, a residual and a correction with the correctly rounded reciprocal, or by the divide
// instruction where that shortcut is not safe), so their dequantized values match a plain CPU
// implementation bit for bit.
#include <mutex>
#include <vector>

#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kSweepThreads = 256;
constexpr int kSweepWarps = kSweepThreads / 32;
constexpr int kTile = 4096;                    // elements per tile: a multiple of every k1 <= 1024
constexpr int kTileSlices = kTile / kSlice;    // 256
constexpr int kFamGroup = 16;                  // families (up to 8 configurations each) evaluated per tile visit

constexpr int kFamMax = 8;  // configurations (mantissa widths) per family
struct SweepCfg {            // one family, 32 bytes
    int32_t k1;
    uint8_t kind, k2, d2, rounding;
    uint8_t k2t, k1t;        // compile-time selectors: sub-block / block size inside a slice (<= 16)
    uint8_t nm, pad;
    uint32_t m_packed;       // nm mantissa widths, 4 bits each
    uint16_t idx[kFamMax];   // where each member's result goes
    __host__ __device__ int m(int i) const { return (int)((m_packed >> (4 * i)) & 0xFu); }
};
static_assert(sizeof(SweepCfg) == 32, "family record size");
static_assert(kTileSlices == kSweepThreads, "one slice per thread");

constexpr int kTilesPerUnit = 4;  // tiles a CTA keeps resident while it walks a group of families
struct SweepTile {
    uint4 x[kTile / 4];            // 16-byte chunks, chunk c stored at c ^ ((c >> 3) & 3)
    uint8_t lv[kTile];             // level l (block size 2^l) starts at lv_off(l); sizes 2048, 1024, ..., 4
};
struct SweepSmem {
    SweepTile t[kTilesPerUnit];
    double sig_warp[kSweepWarps];
    double fam_acc[kSweepWarps][8][32];  // per-lane error sums of the family a warp is working on, one row per member
};
__host__ __device__ constexpr int lv_off(int l) { return kTile - (kTile >> (l - 1)); }  // 0, 2048, 3072, ...

__device__ __forceinline__ int swz4(int c) { return c ^ ((c >> 3) & 3); }

__device__ __forceinline__ float round_to_int(float t, int rounding) {  // 0 <= t < 2^22
    if (rounding == BDR_ROUND_NEAREST_EVEN) return __fsub_rn(__fadd_rn(t, 8388608.0f), 8388608.0f);
    return floorf(__fadd_rn(t, 0.5f));
}

// ---- POW2 kind: error energy of one slice for every mantissa width of a family -----------------------
// packed fp32 arithmetic: two independent operations per instruction
__device__ __forceinline__ void add_f32x2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{.reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; add.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd;}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ void sub_f32x2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{.reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; sub.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd;}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ void fma_f32x2(float& d0, float& d1, float a0, float a1, float b0, float b1) {  // d += a * b
    asm("{.reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rd, {%0, %1}; fma.rn.f32x2 rd, ra, rb, rd; mov.b64 {%0, %1}, rd;}"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

template <int K2, int K1S>
__device__ __forceinline__ void pow2_slice(const uint32_t (&u)[kSlice], const SweepTile& sm, int s, const SweepCfg& c,
                                           double* lane_acc /* member mi at lane_acc[32 * mi] */) {
    uint32_t ej[kSlice / K2], eb[kSlice / K1S];
    if (K2 == 1) {
#pragma unroll
        for (int i = 0; i < kSlice; ++i) ej[i] = u[i] & kExpMask;
    } else {
        constexpr int l2 = K2 == 2 ? 1 : K2 == 4 ? 2 : K2 == 8 ? 3 : 4;
        const uint8_t* p = sm.lv + lv_off(l2) + s * (kSlice / K2);
#pragma unroll
        for (int j = 0; j < kSlice / K2; ++j) ej[j] = (uint32_t)p[j] << 23;
    }
    if (K1S == kSlice) {
        const int l1 = 31 - __clz(c.k1);  // log2 k1 >= 4
        eb[0] = (uint32_t)sm.lv[lv_off(l1) + ((s * kSlice) >> l1)] << 23;
    } else if (K1S == 1) {
#pragma unroll
        for (int i = 0; i < kSlice; ++i) eb[i] = u[i] & kExpMask;
    } else {
        constexpr int l1 = K1S == 2 ? 1 : K1S == 4 ? 2 : 3;
        const uint8_t* p = sm.lv + lv_off(l1) + s * (kSlice / K1S);
#pragma unroll
        for (int b = 0; b < kSlice / K1S; ++b) eb[b] = (uint32_t)p[b] << 23;
    }
    uint32_t emax = eb[0];
#pragma unroll
    for (int b = 1; b < kSlice / K1S; ++b) emax = max(emax, eb[b]);
    if (c.rounding != BDR_ROUND_NEAREST_EVEN || emax == kExpMask) {
        // ties-away or an Inf/NaN block: exact path, one member at a time
#pragma unroll 1
        for (int mi = 0; mi < c.nm; ++mi) {
            QParams qp;
            qp.k1 = c.k1; qp.k2 = c.k2; qp.d2 = c.d2; qp.m = c.m(mi); qp.rounding = c.rounding;
            qp.beta = (1 << c.d2) - 1;
            qp.qmax = (1u << qp.m) - 1u;
            uint32_t yb[kSlice], rq[kSlice], cb[kSlice / K2], tau[kSlice / K2];
            double e2 = 0.0, s2 = 0.0;
            quantize_slice_exact<K2, K1S, true>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
            lane_acc[32 * mi] += e2;
        }
        return;
    }
    // Fast path, as in quantize_slice: a = |x| * 2^(127-F) and the shifts are computed once; each
    // mantissa width only changes the rounding constant C = 1.5 * 2^(23-(m-1)-tau) and the clamp.
    const uint32_t beta23 = (uint32_t)((1 << c.d2) - 1) << 23;
#pragma unroll
    for (int b = 0; b < kSlice / K1S; ++b) {
        const uint32_t F23 = eb[b];
        const float K = __uint_as_float(max(0x7F000000u - F23, 0x00400000u));
        const double w = __hiloint2double((int)((F23 >> 2) + 0x30100000u), 0);  // 2^(2F-254)
        float a[K1S];
        uint32_t dm[K1S / K2];
#pragma unroll
        for (int i = 0; i < K1S; ++i) a[i] = __fmul_rn(fabsf(__uint_as_float(u[b * K1S + i])), K);
#pragma unroll
        for (int jj = 0; jj < K1S / K2; ++jj) dm[jj] = min(F23 - ej[b * (K1S / K2) + jj], beta23);
        if constexpr (K1S >= 2) {
            // Two elements per instruction (packed fp32 add / subtract / multiply-add; only the clamp is scalar).
            // The shift moves into the operand: at = a * 2^tau is rounded with the constant of tau = 0, so the
            // constant and the clamp are the same for the whole block, and the error comes back to a's scale
            // with one multiply-add, a - (r - C) * 2^-tau (exact).
            float at[K1S], sj[K1S / K2];
#pragma unroll
            for (int jj = 0; jj < K1S / K2; ++jj) sj[jj] = __uint_as_float(0xBF800000u - dm[jj]);  // -2^-tau
#pragma unroll
            for (int i = 0; i < K1S; ++i) at[i] = __fmul_rn(a[i], __uint_as_float(0x3F800000u + dm[i / K2]));
#pragma unroll 2
            for (int mi = 0; mi < c.nm; ++mi) {  // barely unrolled: keeps the instruction footprint of the 15 shapes small
                const int m = c.m(mi);
                const uint32_t c_base = ((uint32_t)(127 + 23 - (m - 1)) << 23) | 0x400000u;
                const float C = __uint_as_float(c_base), Cmax = __uint_as_float(c_base + (1u << m) - 1u);
                float pe0 = 0.f, pe1 = 0.f;
#pragma unroll
                for (int k = 0; k < K1S / 2; ++k) {
                    float r0, r1, e0 = a[2 * k], e1 = a[2 * k + 1];
                    add_f32x2(r0, r1, at[2 * k], at[2 * k + 1], C, C);
                    r0 = fminf(r0, Cmax);
                    r1 = fminf(r1, Cmax);
                    sub_f32x2(r0, r1, r0, r1, C, C);
                    fma_f32x2(e0, e1, r0, r1, sj[(2 * k) / K2], sj[(2 * k + 1) / K2]);  // exact
                    fma_f32x2(pe0, pe1, e0, e1, e0, e1);
                }
                lane_acc[32 * mi] = fma((double)(pe0 + pe1), w, lane_acc[32 * mi]);
            }
            continue;
        }
#pragma unroll 2
        for (int mi = 0; mi < c.nm; ++mi) {
            const int m = c.m(mi);
            const uint32_t c_base = ((uint32_t)(127 + 23 - (m - 1)) << 23) | 0x400000u;
            const uint32_t qmax = (1u << m) - 1u;
            const uint32_t c_bits = c_base - dm[0];
            const float C = __uint_as_float(c_bits), Cmax = __uint_as_float(c_bits + qmax);
            const float de = __fsub_rn(__fsub_rn(fminf(__fadd_rn(a[0], C), Cmax), C), a[0]);  // exact
            const float pe = de * de;
            lane_acc[32 * mi] = fma((double)pe, w, lane_acc[32 * mi]);
        }
    }
}

template <int K1S>
__device__ __forceinline__ void pow2_slice_k2(const uint32_t (&u)[kSlice], const SweepTile& sm, int s, const SweepCfg& c,
                                              double* e2) {
    switch (c.k2t) {
        case 1: pow2_slice<1, K1S>(u, sm, s, c, e2); break;
        case 2: if constexpr (K1S >= 2) pow2_slice<2, K1S>(u, sm, s, c, e2); break;
        case 4: if constexpr (K1S >= 4) pow2_slice<4, K1S>(u, sm, s, c, e2); break;
        case 8: if constexpr (K1S >= 8) pow2_slice<8, K1S>(u, sm, s, c, e2); break;
        default: if constexpr (K1S >= 16) pow2_slice<16, K1S>(u, sm, s, c, e2); break;
    }
}

// ---- FP32-scaled comparator kinds (one FP32 scale for the whole tensor) -----------------------------
// x / s for many x and one s.  With r = RN(1 / s): q0 = RN(x r), e = x - q0 s (exact in one fused multiply-add),
// q = RN(q0 + e r) is the correctly rounded quotient (Markstein), as long as nothing leaves the normal range
// and the significand of s is not all ones; outside these conditions the plain IEEE division is used.
// Quotients below 2^-26 may come out inexact (their residual can be subnormal); every caller rounds them
// to zero anyway.
struct Divisor {
    float s, r;
    bool fast;
};
__device__ __forceinline__ Divisor make_divisor(float s) {
    Divisor d;
    d.s = s;
    d.r = __frcp_rn(s);
    const uint32_t b = __float_as_uint(s);
    d.fast = (b & 0x7FFFFFu) != 0x7FFFFFu && b >= 0x0D800000u /*2^-100*/ && b <= 0x71800000u /*2^100*/;
    return d;
}
template <bool FAST>
__device__ __forceinline__ float divide(float x, const Divisor& d) {
    if constexpr (FAST) {
        const float q0 = __fmul_rn(x, d.r);
        return __fmaf_rn(__fmaf_rn(-q0, d.s, x), d.r, q0);
    } else {
        return __fdiv_rn(x, d.s);
    }
}
template <bool RNE>
__device__ __forceinline__ float round_int(float t) {  // 0 <= t < 2^22
    if constexpr (RNE) return __fsub_rn(__fadd_rn(t, 8388608.0f), 8388608.0f);
    else return floorf(__fadd_rn(t, 0.5f));
}

// |deq| - |x| is formed in fp64, where it is exact: with a first-level maximum that comes from elsewhere (delayed
// scaling) a value can saturate far below its magnitude, and then the fp32 difference would round.  The square goes
// to the fp64 accumulator directly: unlike on the power-of-two path the values are not normalised, so fp32 squares
// could overflow or vanish.
__device__ __forceinline__ void add_err(float deq_mag, float ax, double& e2) {
    const double d = (double)deq_mag - (double)ax;
    e2 = fma(d, d, e2);
}
__device__ __forceinline__ void all_zero_slice(const uint32_t (&u)[kSlice], double& e2) {  // scale 0: everything quantizes to 0
#pragma unroll
    for (int i = 0; i < kSlice; ++i) add_err(0.f, __uint_as_float(u[i] & 0x7FFFFFFFu), e2);
}
// The tie rule and the kind of division are the same for the whole slice: chosen once, outside the element loop.
#define BDR_SLICE_DISPATCH(FN, ...)                                             \
    do {                                                                        \
        if (c.rounding == BDR_ROUND_NEAREST_EVEN) {                             \
            if (dv.fast) FN<true, true>(__VA_ARGS__); else FN<true, false>(__VA_ARGS__);   \
        } else {                                                                \
            if (dv.fast) FN<false, true>(__VA_ARGS__); else FN<false, false>(__VA_ARGS__); \
        }                                                                       \
    } while (0)

// Eq. 2: q = RoundToInt(x / s), clamped;  descale s * q.
template <bool RNE, bool FAST>
__device__ __forceinline__ void int_elements(const uint32_t (&u)[kSlice], const Divisor& dv, float qmax, double& e2) {
#pragma unroll
    for (int i = 0; i < kSlice; ++i) {
        const float ax = __uint_as_float(u[i] & 0x7FFFFFFFu);
        add_err(__fmul_rn(fminf(round_int<RNE>(divide<FAST>(ax, dv)), qmax), dv.s), ax, e2);
    }
}
// Eq. 1: s = max / (2^(b-1) - 1) with m = b-1.
__device__ __forceinline__ void int_slice(const uint32_t (&u)[kSlice], float amax, const SweepCfg& c, double& e2) {
    const float qmax = (float)((1 << c.m(0)) - 1);
    const float s = __fdiv_rn(amax, qmax);
    if (!(s > 0.f)) return all_zero_slice(u, e2);
    const Divisor dv = make_divisor(s);
    BDR_SLICE_DISPATCH(int_elements, u, dv, qmax, e2);
}

// Scalar float with d2 exponent bits and m explicit mantissa bits under an FP32 tensor scale.
template <bool RNE, bool FAST>
__device__ __forceinline__ void fp_elements(const uint32_t (&u)[kSlice], const Divisor& dv, float fmax, int ef_min, int cm, double& e2) {
#pragma unroll
    for (int i = 0; i < kSlice; ++i) {
        const float ax = __uint_as_float(u[i] & 0x7FFFFFFFu);
        const float a = divide<FAST>(ax, dv);
        const int ef = max((int)(__float_as_uint(a) >> 23), ef_min);
        const float step = __uint_as_float((uint32_t)(ef - cm) << 23);
        const float inv_step = __uint_as_float((uint32_t)(254 - (ef - cm)) << 23);
        const float q = round_int<RNE>(__fmul_rn(a, inv_step));
        add_err(__fmul_rn(fminf(__fmul_rn(q, step), fmax), dv.s), ax, e2);
    }
}
__device__ __forceinline__ void fp_slice(const uint32_t (&u)[kSlice], float amax, const SweepCfg& c, double& e2) {
    const int cm = c.m(0);
    const int bias = (1 << (c.d2 - 1)) - 1;
    const float fmax = (c.d2 == 4 && cm == 3)
                           ? 448.0f
                           : __uint_as_float(((uint32_t)((1 << c.d2) - 2 - bias + 127) << 23) | (0x7FFFFFu & ~(0x7FFFFFu >> cm)));
    const float s = __fdiv_rn(amax, fmax);
    if (!(s > 0.f)) return all_zero_slice(u, e2);
    const Divisor dv = make_divisor(s);
    const int ef_min = 1 - bias + 127;
    BDR_SLICE_DISPATCH(fp_elements, u, dv, fmax, ef_min, cm, e2);
}

// VSQ: FP32 scale gamma for the tensor, unsigned d2-bit integer sub-scale per 16-element vector.
__device__ __forceinline__ void vsq_slice(const uint32_t (&u)[kSlice], float amax, const SweepCfg& c, double& e2) {
    const float qmax = (float)((1 << c.m(0)) - 1);
    const float umax = (float)((1u << c.d2) - 1u);
    const float gamma = __fdiv_rn(__fdiv_rn(amax, qmax), umax);
    uint32_t avb = 0;
#pragma unroll
    for (int i = 0; i < kSlice; ++i) avb = max(avb, u[i] & 0x7FFFFFFFu);
    const float sv = __fdiv_rn(__uint_as_float(avb), qmax);
    float uu = 0.f;
    if (gamma > 0.f) uu = fminf(round_to_int(__fdiv_rn(sv, gamma), c.rounding), umax);
    const float eff = __fmul_rn(uu, gamma);
    if (!(eff > 0.f)) return all_zero_slice(u, e2);
    const Divisor dv = make_divisor(eff);
    BDR_SLICE_DISPATCH(int_elements, u, dv, qmax, e2);
}

// ---- kernels ----------------------------------------------------------------------------------------------
// Largest magnitude of the tensor (as fp32 bits).  A contiguous, 16-byte aligned tensor is read with 16-byte
// loads, four in flight per thread; anything else element by element.
template <typename T>
__global__ void amax_kernel(const T* x, int64_t rows, int64_t cols, int64_t ld, uint32_t* amax_bits) {
    uint32_t m = 0;
    const int64_t total = rows * cols;
    constexpr int kPer = 16 / (int)sizeof(T);
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nthr = (int64_t)gridDim.x * blockDim.x;
    if ((ld == cols || rows == 1) && (reinterpret_cast<uintptr_t>(x) % 16) == 0) {
        const uint4* v = reinterpret_cast<const uint4*>(x);
        const int64_t nv = total / kPer;
        auto take = [&](const uint4& q) {
            if constexpr (sizeof(T) == 4) {
                m = max(max(m, q.x & 0x7FFFFFFFu), max(q.y & 0x7FFFFFFFu, max(q.z & 0x7FFFFFFFu, q.w & 0x7FFFFFFFu)));
            } else {  // two bf16 per word: the high half is already in place, the low half moves up
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) m = max(m, max(w[k] & 0x7FFF0000u, (w[k] << 16) & 0x7FFF0000u));
            }
        };
        int64_t g = tid;
        for (; g + 3 * nthr < nv; g += 4 * nthr) {
            const uint4 a = __ldg(v + g), b = __ldg(v + g + nthr), c = __ldg(v + g + 2 * nthr), d = __ldg(v + g + 3 * nthr);
            take(a); take(b); take(c); take(d);
        }
        for (; g < nv; g += nthr) take(__ldg(v + g));
        for (int64_t e = nv * kPer + tid; e < total; e += nthr) m = max(m, Elem<T>::load_bits(x + e) & 0x7FFFFFFFu);
    } else {
        for (int64_t g = tid; g < total; g += nthr) {
            const int64_t r = g / cols;
            m = max(m, Elem<T>::load_bits(x + r * ld + (g - r * cols)) & 0x7FFFFFFFu);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(amax_bits, m);
}

// First-level maximum from a window of earlier maxima (delayed scaling): the largest of n non-negative floats.
__global__ void window_amax_kernel(const float* window, int n, uint32_t* amax_bits) {
    uint32_t m = 0;
    for (int i = threadIdx.x; i < n; i += 32) {
        const uint32_t b = __float_as_uint(window[i]);
        if (b <= 0x7F800000u) m = max(m, b);  // negative values and NaNs are not maxima of magnitudes: ignored
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (threadIdx.x == 0) *amax_bits = m;
}

template <typename T>
__global__ void __launch_bounds__(kSweepThreads)
sweep_kernel(const T* x, int64_t n_lines, int64_t len, int64_t line_stride, int64_t elem_stride, const SweepCfg* fams, int n_fam,
             int n_cfg, int n_groups, int tiles_per_line, int64_t total_units, double* err_sums, double* sig_sum,
             const uint32_t* amax_bits) {
    // A line is a row (elem_stride 1, line_stride = the row pitch) or a column (elem_stride = the row pitch,
    // line_stride 1).  Tiles are numbered line by line for rows; for columns the tiles at the same position of
    // adjacent columns are neighbours, so that the four tiles of a unit share the 32-byte sectors they touch.
    extern __shared__ __align__(16) uint8_t dyn[];
    SweepSmem& sm = *reinterpret_cast<SweepSmem*>(dyn);
    double* acc = reinterpret_cast<double*>(dyn + sizeof(SweepSmem));  // [n_cfg]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c = threadIdx.x; c < n_cfg; c += kSweepThreads) acc[c] = 0.0;
    double sig_acc = 0.0;
    const float amax = __uint_as_float(*amax_bits);
    const int64_t total_tiles = n_lines * tiles_per_line;
    const bool by_column = elem_stride != 1;
    for (int64_t unit = blockIdx.x; unit < total_units; unit += gridDim.x) {
        const int64_t tgroup = unit / n_groups;              // kTilesPerUnit consecutive tiles
        const int group = (int)(unit - tgroup * n_groups);   // kFamGroup consecutive families
        const int64_t tile0 = tgroup * kTilesPerUnit;
        const int ntiles = (int)min((int64_t)kTilesPerUnit, total_tiles - tile0);
        __syncthreads();  // everyone is done with the previous unit's tiles
        for (int ti = 0; ti < ntiles; ++ti) {
            SweepTile& tl = sm.t[ti];
            const int64_t tile = tile0 + ti;
            int64_t line, tpos;
            if (by_column) {
                tpos = tile / n_lines;
                line = tile - tpos * n_lines;
            } else {
                line = tile / tiles_per_line;
                tpos = tile - line * tiles_per_line;
            }
            const int64_t t0 = tpos * kTile;
            const int n = (int)min((int64_t)kTile, len - t0);
            const T* src = x + line * line_stride + t0 * elem_stride;
            // stage: thread t owns slice t (16 elements = 4 chunks)
            const int s = threadIdx.x;
            uint32_t u[kSlice];
            if (by_column) load_slice_guarded(src + (int64_t)s * kSlice * elem_stride, elem_stride, max(0, min(kSlice, n - s * kSlice)), u);
            else load_slice_guarded(src + s * kSlice, 1, max(0, min(kSlice, n - s * kSlice)), u);
#pragma unroll
            for (int v = 0; v < 4; ++v) tl.x[swz4(4 * s + v)] = make_uint4(u[4 * v], u[4 * v + 1], u[4 * v + 2], u[4 * v + 3]);
            // exponent pyramid levels 1..4 from the slice
            uint32_t e[kSlice];
#pragma unroll
            for (int i = 0; i < kSlice; ++i) e[i] = u[i] >> 23 & 0xFFu;
#pragma unroll
            for (int l = 1; l <= 4; ++l) {
#pragma unroll
                for (int j = 0; j < (kSlice >> l); ++j) {
                    e[j] = max(e[2 * j], e[2 * j + 1]);
                    tl.lv[lv_off(l) + s * (kSlice >> l) + j] = (uint8_t)e[j];
                }
            }
            // levels 5..9 inside the warp (a warp covers 512 consecutive elements), level 10 below
            uint32_t v = e[0];
#pragma unroll
            for (int l = 5; l <= 9; ++l) {
                v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 1 << (l - 5)));
                if ((lane & ((1 << (l - 4)) - 1)) == 0) tl.lv[lv_off(l) + (s >> (l - 4))] = (uint8_t)v;
            }
            // signal energy: sum x^2 normalised by the slice exponent, widened once (first family group only)
            if (group == 0) {
                const uint32_t F23 = e[0] << 23;
                const float K = __uint_as_float(max(0x7F000000u - F23, 0x00400000u));
                float ps = 0.f;
                double sg;
                if (e[0] == 255) {
                    sg = __longlong_as_double(0x7FF8000000000000ll);
                } else {
#pragma unroll
                    for (int i = 0; i < kSlice; ++i) {
                        const float a = __fmul_rn(fabsf(__uint_as_float(u[i])), K);
                        ps = fmaf(a, a, ps);
                    }
                    sg = (double)ps * __hiloint2double((int)((F23 >> 2) + 0x30100000u), 0);
                }
                sig_acc += sg;  // per thread; reduced once at the end of the kernel
            }
        }
        __syncthreads();
        if (threadIdx.x < ntiles * (kTile / 1024)) {
            SweepTile& tl = sm.t[threadIdx.x / (kTile / 1024)];
            const int i = threadIdx.x % (kTile / 1024);
            tl.lv[lv_off(10) + i] = max(tl.lv[lv_off(9) + 2 * i], tl.lv[lv_off(9) + 2 * i + 1]);
        }
        __syncthreads();
        // All warps work on the same family at the same time (one slice per thread and tile), so the
        // whole CTA runs one instantiation of the slice code at a time and stays inside the
        // instruction cache; a lane's sums over the unit's tiles are reduced once per family.
        for (int fi = group * kFamGroup; fi < min(n_fam, (group + 1) * kFamGroup); ++fi) {
            const SweepCfg c = fams[fi];
            double* e2 = &sm.fam_acc[warp][0][lane];  // this lane's sums, member mi at e2[32 * mi]
            for (int mi = 0; mi < c.nm; ++mi) e2[32 * mi] = 0.0;
            for (int ti = 0; ti < ntiles; ++ti) {
                const SweepTile& tl = sm.t[ti];
                const int s = threadIdx.x;  // kTileSlices == kSweepThreads
                uint32_t u[kSlice];
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint4 w = tl.x[swz4(4 * s + v)];
                    u[4 * v] = w.x; u[4 * v + 1] = w.y; u[4 * v + 2] = w.z; u[4 * v + 3] = w.w;
                }
                if (c.kind == BDR_SCALE_POW2) {
                    switch (c.k1t) {
                        case 1: pow2_slice_k2<1>(u, tl, s, c, e2); break;
                        case 2: pow2_slice_k2<2>(u, tl, s, c, e2); break;
                        case 4: pow2_slice_k2<4>(u, tl, s, c, e2); break;
                        case 8: pow2_slice_k2<8>(u, tl, s, c, e2); break;
                        default: pow2_slice_k2<16>(u, tl, s, c, e2); break;
                    }
                } else if (c.kind == BDR_SCALE_FP32_INT) {
                    int_slice(u, amax, c, e2[0]);
                } else if (c.kind == BDR_SCALE_FP32_FP) {
                    fp_slice(u, amax, c, e2[0]);
                } else {
                    vsq_slice(u, amax, c, e2[0]);
                }
            }
            for (int mi = 0; mi < c.nm; ++mi) {
                const double t = warp_sum(e2[32 * mi]);
                if (lane == 0) atomicAdd(&acc[c.idx[mi]], t);  // eight warps share the slot
            }
        }
    }
    // signal energy: every thread holds a partial sum
    {
        const double sg = warp_sum(sig_acc);
        if (lane == 0) sm.sig_warp[warp] = sg;
        __syncthreads();
        sig_acc = 0.0;
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 0; w < kSweepWarps; ++w) sig_acc += sm.sig_warp[w];
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < n_cfg; c += kSweepThreads)
        if (acc[c] != 0.0) atomicAdd(err_sums + c, acc[c]);
    if (threadIdx.x == 0 && sig_acc != 0.0) atomicAdd(sig_sum, sig_acc);
}

// The configuration table travels to the device inside kernel parameters (no host buffer has to
// outlive the call, and nothing synchronises): up to kCfgChunk entries per launch.
constexpr int kCfgChunk = 96;
struct CfgChunk { SweepCfg c[kCfgChunk]; };
__global__ void upload_cfgs_kernel(CfgChunk chunk, SweepCfg* dst, int n) {
    if ((int)threadIdx.x < n) dst[threadIdx.x] = chunk.c[threadIdx.x];
}

// Eq. 3 from the accumulated sums: -10 log10(err / sig); err = 0 < sig -> +inf, sig = 0 -> NaN.
__global__ void qsnr_finalize_kernel(const double* err_sums, const double* sig_sum, int n, double* out_db) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double e = err_sums[i], s = *sig_sum;
    double q;
    if (s == 0.0 || s != s || e != e) q = __longlong_as_double(0x7FF8000000000000ll);
    else if (e == 0.0) q = __longlong_as_double(0x7FF0000000000000ll);
    else q = -10.0 * log10(e / s);
    out_db[i] = q;
}

// The same for n independent {error, signal} pairs, as the quantize kernels accumulate them.
__global__ void qsnr_pairs_kernel(const double* sums, int n, double* out_db) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double e = sums[2 * i], s = sums[2 * i + 1];
    double q;
    if (s == 0.0 || s != s || e != e) q = __longlong_as_double(0x7FF8000000000000ll);
    else if (e == 0.0) q = __longlong_as_double(0x7FF0000000000000ll);
    else q = -10.0 * log10(e / s);
    out_db[i] = q;
}

// workspace layout: [n] error sums | signal sum | amax bits (+pad to 16) | [n] SweepCfg
static constexpr size_t ws_cfg_offset(int n) { return (((size_t)n + 1) * 8 + 16 + 15) / 16 * 16; }

constexpr int64_t sweep_workspace_bytes(int n) { return (int64_t)((ws_cfg_offset(n) + (size_t)n * sizeof(SweepCfg) + 255) / 256 * 256); }

static bool is_pow2i(int v) { return v > 0 && (v & (v - 1)) == 0; }

// Validate one configuration for the sweep and translate it into a one-member family.
static int make_sweep_cfg(const bdr_config_t& c, int index, SweepCfg* out) {
    if (c.rounding != BDR_ROUND_NEAREST_EVEN && c.rounding != BDR_ROUND_NEAREST_AWAY) return BDR_ERR_BAD_CONFIG;
    SweepCfg s = {};
    s.k1 = c.k1; s.kind = (uint8_t)c.scale_kind; s.rounding = (uint8_t)c.rounding;
    s.k2t = 1; s.k1t = 1; s.nm = 1;
    switch (c.scale_kind) {
        case BDR_SCALE_POW2:
            if (c.d1 != 8 || c.k1 < 1 || c.k2 < 1 || c.k1 % c.k2 != 0 || c.d2 < 0 || c.d2 > 3 || c.m < 1 || c.m > 8)
                return BDR_ERR_BAD_CONFIG;
            if (!is_pow2i(c.k1) || !is_pow2i(c.k2) || c.k1 > 1024) return BDR_ERR_UNSUPPORTED;
            s.k1t = (uint8_t)(c.k1 < kSlice ? c.k1 : kSlice);
            s.k2t = (uint8_t)(c.d2 == 0 ? s.k1t : c.k2);  // d2 = 0: every shift is zero whatever k2 is
            if (c.d2 != 0 && c.k2 > kSlice) return BDR_ERR_UNSUPPORTED;
            break;
        case BDR_SCALE_FP32_INT:
            if (c.m < 1 || c.m > 15) return BDR_ERR_BAD_CONFIG;
            if (c.k1 != 0) return BDR_ERR_UNSUPPORTED;
            break;
        case BDR_SCALE_FP32_FP:
            if (c.d2 < 2 || c.d2 > 5 || c.m < 1 || c.m > 7) return BDR_ERR_BAD_CONFIG;
            if (c.k1 != 0) return BDR_ERR_UNSUPPORTED;
            break;
        case BDR_SCALE_FP32_VSQ:
            if (c.k2 < 1 || c.d2 < 1 || c.d2 > 16 || c.m < 1 || c.m > 15) return BDR_ERR_BAD_CONFIG;
            if (c.k1 != 0 || c.k2 != kSlice) return BDR_ERR_UNSUPPORTED;
            break;
        default: return BDR_ERR_BAD_CONFIG;
    }
    s.k2 = (uint8_t)(c.scale_kind == BDR_SCALE_POW2 ? s.k2t : c.k2);  // the effective sub-block size
    s.d2 = (uint8_t)c.d2;
    s.m_packed = (uint32_t)c.m;
    s.idx[0] = (uint16_t)index;
    *out = s;
    return BDR_OK;
}

// Merge configurations that differ only in m into families of up to kFamMax members.
static void build_families(const std::vector<SweepCfg>& singles, std::vector<SweepCfg>* fams) {
    for (const SweepCfg& c : singles) {
        bool merged = false;
        if (c.kind == BDR_SCALE_POW2) {
            for (SweepCfg& f : *fams) {
                if (f.kind == c.kind && f.k1 == c.k1 && f.k2 == c.k2 && f.d2 == c.d2 && f.rounding == c.rounding && f.nm < kFamMax) {
                    f.m_packed |= c.m_packed << (4 * f.nm);
                    f.idx[f.nm] = c.idx[0];
                    f.nm++;
                    merged = true;
                    break;
                }
            }
        }
        if (!merged) fams->push_back(c);
    }
}

template <typename T>
static int amax_launch(const T* x, int64_t rows, int64_t cols, int64_t ld, uint32_t* amax_bits, cudaStream_t st) {
    const int64_t total = rows * cols;
    const int grid = (int)max((int64_t)1, min((total + 1023) / 1024, (int64_t)sm_count() * 8));
    amax_kernel<T><<<grid, 256, 0, st>>>(x, rows, cols, ld, amax_bits);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T>
static int sweep_launch(const SweepCfg* host_fams, int n_fam, int n, bool need_amax, const T* x, int64_t rows, int64_t cols,
                        int64_t ld, int axis, const float* amax_window, int n_window, double* out_db, uint8_t* ws, cudaStream_t st) {
    double* err = reinterpret_cast<double*>(ws);
    double* sig = err + n;
    uint32_t* amax = reinterpret_cast<uint32_t*>(sig + 1);
    SweepCfg* dcfg = reinterpret_cast<SweepCfg*>(ws + ws_cfg_offset(n));
    if (cudaMemsetAsync(ws, 0, ws_cfg_offset(n), st) != cudaSuccess) return BDR_ERR_CUDA;
    for (int i0 = 0; i0 < n_fam; i0 += kCfgChunk) {
        CfgChunk chunk;
        const int cnt = min(kCfgChunk, n_fam - i0);
        for (int i = 0; i < cnt; ++i) chunk.c[i] = host_fams[i0 + i];
        upload_cfgs_kernel<<<1, kCfgChunk, 0, st>>>(chunk, dcfg + i0, cnt);
    }
    if (rows > 0 && cols > 0) {
        if (need_amax) {
            if (amax_window) window_amax_kernel<<<1, 32, 0, st>>>(amax_window, n_window, amax);
            else amax_launch<T>(x, rows, cols, ld, amax, st);
        }
        const int64_t n_lines = axis == 1 ? rows : cols, len = axis == 1 ? cols : rows;
        const int tiles_per_line = (int)((len + kTile - 1) / kTile);
        const int n_groups = (n_fam + kFamGroup - 1) / kFamGroup;
        const int64_t units = (n_lines * tiles_per_line + kTilesPerUnit - 1) / kTilesPerUnit * n_groups;
        const size_t smem = sizeof(SweepSmem) + (size_t)n * sizeof(double);
        auto kern = sweep_kernel<T>;
        // set on every call: the size depends on the number of configurations, and the attribute is per device
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return BDR_ERR_CUDA;
        const int grid = (int)max((int64_t)1, min(units, (int64_t)sm_count() * 2));
        kern<<<grid, kSweepThreads, smem, st>>>(x, n_lines, len, axis == 1 ? ld : 1, axis == 1 ? 1 : ld, dcfg, n_fam, n, n_groups,
                                                tiles_per_line, units, err, sig, amax);
    }
    qsnr_finalize_kernel<<<(n + 127) / 128, 128, 0, st>>>(err, sig, n, out_db);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// ---- built-in scratch for callers that cannot allocate ---------------------------------------------
// bdr_qsnr_static keeps its scratch in this file-scope device array instead of taking a workspace
// pointer.  Every GPU that loads the library holds these bytes until the process exits.  In host
// code the array's name is only a stand-in symbol, not a device address, so the address a kernel can
// use is looked up once per device with cudaGetSymbolAddress (below) while that device is current.
constexpr int kStaticMaxCfgs = 512;
constexpr size_t kStaticScratchBytes = 20736;
static_assert(kStaticScratchBytes == (size_t)sweep_workspace_bytes(kStaticMaxCfgs), "the built-in scratch holds exactly the documented maximum");
static __device__ __align__(256) unsigned char g_qsnr_static_scratch[kStaticScratchBytes];

// Device address of the built-in scratch on the current device (set up on first use per device).
static int static_scratch_ptr(uint8_t** out) {
    static std::mutex mu;
    static uint8_t* cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BDR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_qsnr_static_scratch) != cudaSuccess || !p) return BDR_ERR_CUDA;
        cached[dev] = static_cast<uint8_t*>(p);
    }
    *out = cached[dev];
    return BDR_OK;
}

}  // namespace bdr

using namespace bdr;

extern "C" {

int64_t bdr_qsnr_workspace_bytes(int n_cfgs) { return n_cfgs < 1 ? 0 : sweep_workspace_bytes(n_cfgs); }

static int qsnr_impl(const bdr_config_t* cfgs, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                     int axis, const float* amax_window, int n_window, double* qsnr_db_dev, void* workspace, int64_t workspace_bytes,
                     void* stream) {
    constexpr int kMaxCfgs = 4096;  // per-CTA accumulators live in shared memory
    if (!cfgs || !qsnr_db_dev) return BDR_ERR_NULL;
    if (n_cfgs < 1 || n_cfgs > kMaxCfgs) return BDR_ERR_SIZE;
    if (dt != BDR_F32 && dt != BDR_BF16) return BDR_ERR_UNSUPPORTED;
    if (axis != 0 && axis != 1) return BDR_ERR_BAD_CONFIG;
    if (rows < 0 || cols < 0 || ld < cols) return BDR_ERR_SIZE;
    if (!x && rows > 0 && cols > 0) return BDR_ERR_NULL;
    if ((uintptr_t)x % (dt == BDR_F32 ? 4 : 2) || (uintptr_t)qsnr_db_dev % 8) return BDR_ERR_MISALIGNED;
    std::vector<SweepCfg> singles(n_cfgs), table;
    bool need_amax = false;
    for (int i = 0; i < n_cfgs; ++i) {
        const int rc = make_sweep_cfg(cfgs[i], i, &singles[i]);
        if (rc) return rc;
        need_amax |= cfgs[i].scale_kind != BDR_SCALE_POW2;
    }
    build_families(singles, &table);
    const int n_fam = (int)table.size();
    // Rows shorter than a tile would leave the 4096-element tiles mostly empty.  When the rows are contiguous and every
    // configuration's blocks (and VSQ vectors) divide the row length, no block straddles two rows, so the tensor is the
    // same problem as one long row.
    if (axis == 1 && rows > 1 && ld == cols && cols > 0) {
        bool whole = true;
        for (int i = 0; i < n_cfgs && whole; ++i) {
            const int64_t g = cfgs[i].scale_kind == BDR_SCALE_POW2 ? cfgs[i].k1 : (cfgs[i].scale_kind == BDR_SCALE_FP32_VSQ ? cfgs[i].k2 : 1);
            whole = g > 0 && cols % g == 0;
        }
        if (whole) {
            cols *= rows;
            rows = 1;
            ld = cols;
        }
    }
    if (!workspace || workspace_bytes < sweep_workspace_bytes(n_cfgs)) return BDR_ERR_WORKSPACE;
    if ((uintptr_t)workspace % 16) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_F32)
        return sweep_launch<float>(table.data(), n_fam, n_cfgs, need_amax, (const float*)x, rows, cols, ld, axis, amax_window, n_window,
                                   qsnr_db_dev, (uint8_t*)workspace, st);
    return sweep_launch<__nv_bfloat16>(table.data(), n_fam, n_cfgs, need_amax, (const __nv_bfloat16*)x, rows, cols, ld, axis, amax_window,
                                       n_window, qsnr_db_dev, (uint8_t*)workspace, st);
}

int bdr_qsnr(const bdr_config_t* cfgs, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
             int axis, double* qsnr_db_dev, void* workspace, int64_t workspace_bytes, void* stream) {
    return qsnr_impl(cfgs, n_cfgs, x, dt, rows, cols, ld, axis, nullptr, 0, qsnr_db_dev, workspace, workspace_bytes, stream);
}

int bdr_qsnr_delayed(const bdr_config_t* cfgs, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                     int axis, const float* amax_window_dev, int n_window, double* qsnr_db_dev, void* workspace,
                     int64_t workspace_bytes, void* stream) {
    if (n_window < 1) return BDR_ERR_SIZE;
    if (!amax_window_dev) return BDR_ERR_NULL;
    if ((uintptr_t)amax_window_dev % 4) return BDR_ERR_MISALIGNED;
    return qsnr_impl(cfgs, n_cfgs, x, dt, rows, cols, ld, axis, amax_window_dev, n_window, qsnr_db_dev, workspace, workspace_bytes,
                     stream);
}

int bdr_amax(const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* amax_dev, void* stream) {
    if (!amax_dev) return BDR_ERR_NULL;
    if (dt != BDR_F32 && dt != BDR_BF16) return BDR_ERR_UNSUPPORTED;
    if (rows < 0 || cols < 0 || ld < cols) return BDR_ERR_SIZE;
    if (rows == 0 || cols == 0) return BDR_OK;
    if (!x) return BDR_ERR_NULL;
    if ((uintptr_t)x % (dt == BDR_F32 ? 4 : 2) || (uintptr_t)amax_dev % 4) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    // magnitudes are non-negative floats, whose order is the order of their bit patterns
    if (dt == BDR_F32) return amax_launch<float>((const float*)x, rows, cols, ld, reinterpret_cast<uint32_t*>(amax_dev), st);
    return amax_launch<__nv_bfloat16>((const __nv_bfloat16*)x, rows, cols, ld, reinterpret_cast<uint32_t*>(amax_dev), st);
}

int bdr_qsnr_from_sums(const double* sums_dev, int n, double* qsnr_db_dev, void* stream) {
    if (!sums_dev || !qsnr_db_dev) return BDR_ERR_NULL;
    if (n < 0) return BDR_ERR_SIZE;
    if ((uintptr_t)sums_dev % 8 || (uintptr_t)qsnr_db_dev % 8) return BDR_ERR_MISALIGNED;
    if (n == 0) return BDR_OK;
    qsnr_pairs_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(sums_dev, n, qsnr_db_dev);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

int bdr_qsnr_static_max_cfgs(void) { return kStaticMaxCfgs; }

int bdr_qsnr_static(const bdr_config_t* cfgs, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols,
                    int64_t ld, int axis, double* qsnr_db_dev, void* stream) {
    static_assert(kStaticScratchBytes % 256 == 0, "scratch size is a multiple of its alignment");
    if (n_cfgs > kStaticMaxCfgs) return BDR_ERR_SIZE;  // more configurations than the built-in scratch holds
    if (n_cfgs >= 1 && sweep_workspace_bytes(n_cfgs) > (int64_t)kStaticScratchBytes) return BDR_ERR_SIZE;
    uint8_t* scratch = nullptr;
    const int rc = static_scratch_ptr(&scratch);  // first call on a device resolves the symbol's address
    if (rc) return rc;
    return qsnr_impl(cfgs, n_cfgs, x, dt, rows, cols, ld, axis, nullptr, 0, qsnr_db_dev, scratch, (int64_t)kStaticScratchBytes, stream);
}

}  // extern "C"
