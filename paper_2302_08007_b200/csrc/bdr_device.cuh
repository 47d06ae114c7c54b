// Device-side building blocks shared by the quantize / pack / unpack / sweep kernels.
//
// Notation follows the paper's Appendix: F is the biased shared exponent of a k1-block (the fp32
// exponent field of its largest element, E = F - 127), tau the shift of a k2-sub-block
// (tau = min(F - F_sub, beta), beta = 2^d2 - 1), m the number of magnitude digits, q the integer
// magnitude (0 .. 2^m - 1) and p = E - tau - (m - 1) the exponent of one unit of q.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bdr.h"

namespace bdr {

// Launch-time constants of one POW2 configuration.
struct QParams {
    int k1, k2, d2, m, rounding;
    int beta;       // 2^d2 - 1
    uint32_t qmax;  // 2^m - 1
};

constexpr int kSlice = 16;  // elements a thread keeps in registers at a time

__device__ __forceinline__ int exp_field(uint32_t u) { return (int)((u >> 23) & 0xFFu); }

// 2^p as fp32 bits for -149 <= p <= 127 (subnormal powers included).
__device__ __forceinline__ uint32_t pow2_bits(int p) {
    return p >= -126 ? (uint32_t)(p + 127) << 23 : 1u << (p + 149);
}

// Exact integer formulation of one element (any tie rule, any exponent): |x| = M * 2^(fe-150),
// |x| / 2^p = M / 2^sh.  Returns q (clamped) and the dequantized bit pattern.
__device__ __forceinline__ void quant_elem_exact(uint32_t u, int F, int tau, const QParams& qp, uint32_t& q,
                                                 uint32_t& ybits) {
    const int f = exp_field(u);
    const uint32_t M = (u & 0x7FFFFFu) | (f ? 0x800000u : 0u);
    const int fe = f ? f : 1;
    const int sh = 24 - qp.m - tau - (fe - F);  // >= 8 for every legal configuration
    uint32_t qq = 0;
    if (sh <= 25) {
        const uint32_t fl = M >> sh;
        const uint32_t rem = M & ((1u << sh) - 1u);
        const uint32_t half = 1u << (sh - 1);
        qq = fl + ((rem > half) || (rem == half && (qp.rounding == BDR_ROUND_NEAREST_AWAY || (fl & 1u))) ? 1u : 0u);
    }
    qq = min(qq, qp.qmax);
    q = qq;
    const int p = F - 127 - tau - (qp.m - 1);
    const float mag = __fmul_rn(__uint2float_rn(qq), __uint_as_float(pow2_bits(p)));  // exact
    ybits = __float_as_uint(mag) | (u & 0x80000000u);
}

// Fast formulation for ties-to-even: adding C = 1.5 * 2^(p+23) makes the fp32 adder round |x| to a
// multiple of 2^p (nearest, ties to even) and leaves q in the low mantissa bits of the sum.
// Valid while C is finite, i.e. F <= kFastMaxF.
constexpr int kFastMaxF = 230;
// shared-exponent range in which the Eq. 3 terms of a block are summed in fp32 before widening
constexpr int kSumMinF = 96, kSumMaxF = 158;

struct SubScale {
    uint32_t Cbits;  // bits of C
    float C;
};

__device__ __forceinline__ SubScale make_subscale(int F, int tau, int m) {
    SubScale s;
    s.Cbits = ((uint32_t)(F - tau - m + 24) << 23) | 0x400000u;
    s.C = __uint_as_float(s.Cbits);
    return s;
}

__device__ __forceinline__ void quant_elem_fast(uint32_t u, const SubScale& s, uint32_t qmax, uint32_t& q,
                                                uint32_t& ybits, float& abs_x, float& abs_q) {
    abs_x = __uint_as_float(u & 0x7FFFFFFFu);
    const float t = __fadd_rn(abs_x, s.C);
    q = min(__float_as_uint(t) - s.Cbits, qmax);
    abs_q = __fsub_rn(__uint_as_float(s.Cbits + q), s.C);
    ybits = __float_as_uint(abs_q) | (u & 0x80000000u);
}

// ---- element I/O --------------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kBytes = 4;
    __device__ static __forceinline__ uint32_t load_bits(const float* p) { return __float_as_uint(*p); }
    __device__ static __forceinline__ void store_bits(float* p, uint32_t b) { *p = __uint_as_float(b); }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kBytes = 2;
    __device__ static __forceinline__ uint32_t load_bits(const __nv_bfloat16* p) {
        return (uint32_t)(*reinterpret_cast<const uint16_t*>(p)) << 16;
    }
    // every value this library produces from bf16 inputs (or from m <= 8 codes within bf16's
    // exponent range) has its low 16 fp32 bits clear, so truncation is exact
    __device__ static __forceinline__ void store_bits(__nv_bfloat16* p, uint32_t b) {
        *reinterpret_cast<uint16_t*>(p) = (uint16_t)(b >> 16);
    }
};

// Load / store one 16-element slice as fp32 bit patterns with 128-bit accesses.
__device__ __forceinline__ void load_slice_vec(const float* p, uint32_t (&u)[kSlice]) {
    const uint4* v = reinterpret_cast<const uint4*>(p);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 w = __ldg(v + i);
        u[4 * i] = w.x; u[4 * i + 1] = w.y; u[4 * i + 2] = w.z; u[4 * i + 3] = w.w;
    }
}
__device__ __forceinline__ void load_slice_vec(const __nv_bfloat16* p, uint32_t (&u)[kSlice]) {
    const uint4* v = reinterpret_cast<const uint4*>(p);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint4 w = __ldg(v + i);
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            u[8 * i + 2 * k] = ws[k] << 16;
            u[8 * i + 2 * k + 1] = ws[k] & 0xFFFF0000u;
        }
    }
}
__device__ __forceinline__ void store_slice_vec(float* p, const uint32_t (&y)[kSlice]) {
    uint4* v = reinterpret_cast<uint4*>(p);
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = make_uint4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
}
__device__ __forceinline__ void store_slice_vec(__nv_bfloat16* p, const uint32_t (&y)[kSlice]) {
    uint4* v = reinterpret_cast<uint4*>(p);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint32_t ws[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) ws[k] = (y[8 * i + 2 * k] >> 16) | (y[8 * i + 2 * k + 1] & 0xFFFF0000u);
        v[i] = make_uint4(ws[0], ws[1], ws[2], ws[3]);
    }
}

// Guarded scalar versions for ragged tails and unaligned tensors: elements at index >= n read as +0.
template <typename T>
__device__ __forceinline__ void load_slice_guarded(const T* p, int64_t stride, int n, uint32_t (&u)[kSlice]) {
#pragma unroll
    for (int i = 0; i < kSlice; ++i) u[i] = i < n ? Elem<T>::load_bits(p + i * stride) : 0u;
}
template <typename T>
__device__ __forceinline__ void store_slice_guarded(T* p, int64_t stride, int n, const uint32_t (&y)[kSlice]) {
#pragma unroll
    for (int i = 0; i < kSlice; ++i)
        if (i < n) Elem<T>::store_bits(p + i * stride, y[i]);
}

// ---- per-thread asynchronous prefetch ring (global -> shared, read back by the issuing thread) --------
// A thread queues 16-byte copies several loop iterations ahead and later reads only what it queued
// itself, so a wait_group is all the synchronisation needed and the bytes in flight per SM no longer
// depend on how many registers the kernel uses.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// 16-byte words of one slice (as fetched) -> fp32 bit patterns
template <typename T> struct SliceWords;
template <> struct SliceWords<float> {
    static constexpr int kVecs = 4;
    __device__ static __forceinline__ void expand(const uint4 (&w)[4], uint32_t (&u)[kSlice]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) { u[4 * i] = w[i].x; u[4 * i + 1] = w[i].y; u[4 * i + 2] = w[i].z; u[4 * i + 3] = w[i].w; }
    }
};
template <> struct SliceWords<__nv_bfloat16> {
    static constexpr int kVecs = 2;
    __device__ static __forceinline__ void expand(const uint4 (&w)[2], uint32_t (&u)[kSlice]) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t ws[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) { u[8 * i + 2 * k] = ws[k] << 16; u[8 * i + 2 * k + 1] = ws[k] & 0xFFFF0000u; }
        }
    }
};

// ---- block reduction of the two Eq. 3 sums ------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Every thread of the CTA calls this once; adds the CTA totals to sums[0..1] with two atomics.
__device__ __forceinline__ void block_accumulate_sums(double err2, double sig2, double* sums) {
    __shared__ double sh[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    err2 = warp_sum(err2);
    sig2 = warp_sum(sig2);
    if (lane == 0) { sh[0][warp] = err2; sh[1][warp] = sig2; }
    __syncthreads();
    if (warp == 0) {
        double e = lane < nwarp ? sh[0][lane] : 0.0, s = lane < nwarp ? sh[1][lane] : 0.0;
        e = warp_sum(e);
        s = warp_sum(s);
        if (lane == 0) { atomicAdd(sums, e); atomicAdd(sums + 1, s); }
    }
}

}  // namespace bdr

namespace bdr {

// ---- one 16-element slice ------------------------------------------------------------------------
// Exponent fields are kept in place (bits 30..23, "e23" values) so no per-element shift is needed.
constexpr uint32_t kExpMask = 0x7F800000u;

// Sub-block maxima of the exponent fields (k2 <= 16), as e23 values.
template <int K2>
__device__ __forceinline__ void subblock_exponents(const uint32_t (&u)[kSlice], uint32_t (&ej)[kSlice / K2]) {
#pragma unroll
    for (int j = 0; j < kSlice / K2; ++j) {
        uint32_t e = 0;
#pragma unroll
        for (int i = 0; i < K2; ++i) e = max(e, u[j * K2 + i] & kExpMask);
        ej[j] = e;
    }
}

// Exact path for one slice: ties-away rounding, or a block that holds Inf/NaN.
template <int K2, int K1S, bool WANT_SUMS>
__device__ __forceinline__ void quantize_slice_exact(const uint32_t (&u)[kSlice], const uint32_t (&ej)[kSlice / K2],
                                                  const uint32_t (&eb)[kSlice / K1S], const QParams& qp,
                                                  uint32_t (&yb)[kSlice], uint32_t (&rq)[kSlice],
                                                  uint32_t (&cb)[kSlice / K2], uint32_t (&tau)[kSlice / K2],
                                                  double& e2, double& s2) {
#pragma unroll
    for (int j = 0; j < kSlice / K2; ++j) {
        const int F = (int)(eb[(j * K2) / K1S] >> 23);
        const int t = F == 255 ? 0 : min(F - (int)(ej[j] >> 23), qp.beta);
        tau[j] = (uint32_t)t;
        cb[j] = 0;
#pragma unroll
        for (int i = 0; i < K2; ++i) {
            const int k = j * K2 + i;
            uint32_t q = 0, y = 0x7FC00000u;
            if (F != 255) quant_elem_exact(u[k], F, t, qp, q, y);
            yb[k] = y;
            rq[k] = F == 255 ? 0u : q;
            if (WANT_SUMS) {
                const double de = (double)__uint_as_float(y) - (double)__uint_as_float(u[k]);
                const double dx = (double)__uint_as_float(u[k]);
                e2 = fma(de, de, e2);
                s2 = fma(dx, dx, s2);
            }
        }
    }
}

// Quantize the slice.  eb[] holds the shared exponent (e23) of each k1-block touching the slice
// (K1S = min(k1,16) elements each; for k1 >= 16 the single entry is the block's exponent after any
// cross-lane reduction).  Produces dequantized bit patterns (WANT_Y), and for packing (WANT_CODE)
// the sub-block shifts tau plus the magnitudes in "raw" form: q of element k is rq[k] - cb[k / K2]
// (the packer removes the per-sub-block offset cb after it has shifted the fields into place; the
// sign comes from u).  Adds this slice's Eq. 3 terms to e2 / s2 when WANT_SUMS.
//
// Fast path (ties-to-even, finite block): work in the block-normalised domain a = |x| * 2^(127-F),
// a < 2.  There the unit of q is 2^(-(m-1)-tau), so adding C = 1.5 * 2^(23-(m-1)-tau) makes the fp32
// adder round a to a multiple of that unit (nearest, ties to even) and leaves q in the low
// mantissa bits; C depends on tau only.  Every scaling is by a power of two and therefore exact
// (an element so small that a underflows rounds to q = 0 either way).  The Eq. 3 terms are summed
// in fp32 in the normalised domain (at most 16 terms of magnitude <= 4) and widened once per block
// with the exact factor 2^(2F-254).
template <int K2, int K1S, bool WANT_SUMS, bool WANT_Y = true, bool WANT_CODE = true, bool WANT_SIG = true>
__device__ __forceinline__ void quantize_slice(const uint32_t (&u)[kSlice], const uint32_t (&ej)[kSlice / K2],
                                               const uint32_t (&eb)[kSlice / K1S], const QParams& qp,
                                               uint32_t (&yb)[kSlice], uint32_t (&rq)[kSlice],
                                               uint32_t (&cb)[kSlice / K2], uint32_t (&tau)[kSlice / K2], double& e2,
                                               double& s2) {
    uint32_t emax = eb[0];
#pragma unroll
    for (int b = 1; b < kSlice / K1S; ++b) emax = max(emax, eb[b]);
    if (qp.rounding != BDR_ROUND_NEAREST_EVEN || emax == kExpMask) {
        quantize_slice_exact<K2, K1S, WANT_SUMS>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
        return;
    }
    const uint32_t c_base = ((uint32_t)(127 + 23 - (qp.m - 1)) << 23) | 0x400000u;
    const uint32_t beta23 = (uint32_t)qp.beta << 23;
#pragma unroll
    for (int b = 0; b < kSlice / K1S; ++b) {
        const uint32_t F23 = eb[b];
        const float K = __uint_as_float(max(0x7F000000u - F23, 0x00400000u));  // 2^(127-F)
        const float Kinv = __uint_as_float(max(F23, 0x00400000u));            // 2^(F-127)
        float pe = 0.f, ps = 0.f;
#pragma unroll
        for (int jj = 0; jj < K1S / K2; ++jj) {
            const int j = b * (K1S / K2) + jj;
            const uint32_t dm = min(F23 - ej[j], beta23);  // tau << 23
            const uint32_t c_bits = c_base - dm;
            if (WANT_CODE) { tau[j] = dm >> 23; cb[j] = c_bits; }
            const float C = __uint_as_float(c_bits);
            const float Cmax = __uint_as_float(c_bits + qp.qmax);
#pragma unroll
            for (int i = 0; i < K2; ++i) {
                const int k = j * K2 + i;
                const float a = __fmul_rn(fabsf(__uint_as_float(u[k])), K);
                const float r = fminf(__fadd_rn(a, C), Cmax);
                const float aq = __fsub_rn(r, C);
                if (WANT_CODE) rq[k] = __float_as_uint(r);
                if (WANT_Y) yb[k] = __float_as_uint(__fmul_rn(aq, Kinv)) | (u[k] & 0x80000000u);
                if (WANT_SUMS) {
                    const float de = __fsub_rn(aq, a);  // exact
                    pe = fmaf(de, de, pe);
                    if (WANT_SIG) ps = fmaf(a, a, ps);
                }
            }
        }
        if (WANT_SUMS) {
            const double w = __hiloint2double((int)((F23 >> 2) + 0x30100000u), 0);  // 2^(2F-254)
            e2 = fma((double)pe, w, e2);
            if (WANT_SIG) s2 = fma((double)ps, w, s2);
        }
    }
}

// Runtime-flag front end: picks the instantiation that computes only what the caller will use.
template <int K2, int K1S, bool WANT_CODE>
__device__ __forceinline__ void quantize_slice_rt(const uint32_t (&u)[kSlice], const uint32_t (&ej)[kSlice / K2],
                                                  const uint32_t (&eb)[kSlice / K1S], const QParams& qp, bool want_sums,
                                                  bool want_y, uint32_t (&yb)[kSlice], uint32_t (&rq)[kSlice],
                                                  uint32_t (&cb)[kSlice / K2], uint32_t (&tau)[kSlice / K2], double& e2,
                                                  double& s2) {
    if (want_y) {
        if (want_sums) quantize_slice<K2, K1S, true, true, WANT_CODE>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
        else quantize_slice<K2, K1S, false, true, WANT_CODE>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
    } else {
        if (want_sums) quantize_slice<K2, K1S, true, false, WANT_CODE>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
        else quantize_slice<K2, K1S, false, false, WANT_CODE>(u, ej, eb, qp, yb, rq, cb, tau, e2, s2);
    }
}

// Division by a launch-time constant without the 64-bit divide sequence (n, d < 2^31).
struct FastDiv {
    uint32_t d, mul, shift;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    uint32_t s = 0;
    while ((1ull << s) < d) ++s;
    f.shift = s;
    f.mul = (uint32_t)(((1ull << 32) * ((1ull << s) - d)) / d + 1);
    return f;
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, const FastDiv& f) {
    return (uint32_t)(((uint64_t)__umulhi(n, f.mul) + n) >> f.shift);
}

// ---- bit-stream helpers (code width W = m + 1 known at compile time) -------------------------------
// Pack N elements (raw magnitudes rq with per-sub-block offsets cb, signs from u) into the
// little-endian LSB-first stream: code i = (sign << m) | q occupies bits [i*W, i*W + W).
// A field that lies inside one word is placed with one multiply-add, rq * 2^sh, in wrap-around
// arithmetic; the offsets are removed afterwards with one multiply-add per sub-block and word
// (cb * -(sum of its 2^sh)), which leaves exactly q * 2^sh because q * 2^sh < 2^32.  Sign bits are
// ORed into a second accumulator.  The few fields that straddle two words take the plain route.
template <int W, int N, int K2>
__device__ __forceinline__ void pack_words(const uint32_t (&u)[N], const uint32_t (&rq)[N], const uint32_t (&cb)[N / K2],
                                           uint32_t (&words)[(N * W + 31) / 32]) {
    constexpr int NW = (N * W + 31) / 32, M = W - 1;
    uint32_t accq[NW], accs[NW];
#pragma unroll
    for (int w = 0; w < NW; ++w) { accq[w] = 0; accs[w] = 0; }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const int bit = i * W, wi = bit >> 5, sh = bit & 31;
        if (sh + W <= 32) {
            accq[wi] += rq[i] * (1u << sh);
            const int sp = sh + M;  // where the sign bit goes
            accs[wi] |= (sp == 31 ? u[i] : (u[i] >> (31 - sp))) & (1u << sp);
        } else {
            const uint32_t code = (rq[i] - cb[i / K2]) | ((u[i] >> 31) << M);
            accs[wi] |= code << sh;
            accs[wi + 1] |= code >> (32 - sh);
        }
    }
#pragma unroll
    for (int j = 0; j < N / K2; ++j) {
#pragma unroll
        for (int w = (j * K2 * W) >> 5; w <= (((j + 1) * K2 - 1) * W) >> 5; ++w) {
            uint32_t kc = 0;  // folds to a constant
#pragma unroll
            for (int i = j * K2; i < (j + 1) * K2; ++i) {
                const int bit = i * W, wi = bit >> 5, sh = bit & 31;
                if (wi == w && sh + W <= 32) kc += 1u << sh;
            }
            if (kc) accq[w] -= cb[j] * kc;
        }
    }
#pragma unroll
    for (int w = 0; w < NW; ++w) words[w] = accq[w] | accs[w];
}

// Decode one slice of the Table II family (k2 = 2, d2 = 1): codes are W-bit fields of the
// little-endian stream in `words`, `mbits` holds the eight sub-block shifts (one bit each).
// value = q * 2^p with p = F-127-tau-(m-1): the float 2^23 + q is built by ORing q into its
// mantissa, and fma(2^23 + q, 2^p, -2^(p+23)) is then exactly q * 2^p.  FAST requires every scale
// and constant to be a normal fp32 number (the caller checks 16 <= F <= 230 for the whole warp);
// otherwise the magnitude is converted and scaled in two exact steps, which also covers subnormal
// results and NaN blocks.
template <int W, bool FAST>
__device__ __forceinline__ void decode_slice_impl(const uint32_t (&words)[(kSlice * W + 31) / 32 + 1], int F, uint32_t mbits,
                                                  uint32_t (&yb)[kSlice]) {
    constexpr int M = W - 1;
    constexpr uint32_t kQMask = (1u << M) - 1u;
    // tau = 0 / 1: scale 2^p and bias -2^(p+23)
    const uint32_t s0 = (uint32_t)(F - (M - 1)) << 23, s1 = s0 - 0x00800000u;
    const uint32_t b0 = (s0 + (23u << 23)) | 0x80000000u, b1 = b0 - 0x00800000u;
#pragma unroll
    for (int j = 0; j < kSlice / 2; ++j) {
        const bool t1 = (mbits >> j) & 1u;
        float scale, bias;
        if (FAST) {
            scale = __uint_as_float(t1 ? s1 : s0);
            bias = __uint_as_float(t1 ? b1 : b0);
        } else {
            scale = __uint_as_float(pow2_bits(max(F - 127 - (t1 ? 1 : 0) - (M - 1), -149)));
            bias = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int k = 2 * j + i, bit = k * W, wi = bit >> 5, sh = bit & 31;
            // 32 stream bits starting at this code
            const uint32_t f = sh == 0 ? words[wi] : (sh + W > 32 ? __funnelshift_r(words[wi], words[wi + 1], sh) : words[wi] >> sh);
            const float qf = __uint_as_float(0x4B000000u | (f & kQMask));
            const float mag = FAST ? fmaf(qf, scale, bias) : __fmul_rn(__fsub_rn(qf, 8388608.0f), scale);
            const uint32_t v = __float_as_uint(mag) | ((f << (31 - M)) & 0x80000000u);
            yb[k] = (!FAST && F == 255) ? 0x7FC00000u : v;
        }
    }
}

// Warp-uniform choice between the two decoders (all 32 lanes must call this).
template <int W>
__device__ __forceinline__ void decode_slice(const uint32_t (&words)[(kSlice * W + 31) / 32 + 1], int F, uint32_t mbits,
                                             uint32_t (&yb)[kSlice]) {
    if (__all_sync(0xFFFFFFFFu, F >= 16 && F <= kFastMaxF)) decode_slice_impl<W, true>(words, F, mbits, yb);
    else decode_slice_impl<W, false>(words, F, mbits, yb);
}

// ---- warp-cooperative staging shared by the row-direction kernels ---------------------------------
constexpr int kRowThreads = 256;

// Prefetch ring.  Per iteration a warp consumes one contiguous run of 32 * kVecs 16-byte words (lane
// l owns words [l*kVecs, (l+1)*kVecs)).  The warp copies the run cooperatively -- instruction v
// moves words v*32 .. v*32+31, i.e. 512 contiguous bytes -- so every 32-byte sector is requested
// once, and stores word c at position c ^ ((c >> 3) & (kVecs-1)) so that the later per-lane 16-byte
// reads (stride kVecs words) hit eight different bank groups per quarter-warp.
template <typename T, int SPT> struct Ring {
    static constexpr int kVecs = SliceWords<T>::kVecs * SPT;  // 16-byte words per thread per iteration
    static constexpr int kStages = kVecs >= 8 ? 2 : (kVecs >= 4 ? 3 : 4);  // ~128 bytes ahead per thread
    static constexpr size_t kBytes = (size_t)kStages * kVecs * kRowThreads * 16;
    __device__ static __forceinline__ uint32_t swz(uint32_t c) { return c ^ ((c >> 3) & (kVecs >= 8 ? 7u : (uint32_t)(kVecs - 1))); }
    // warp_stage: this warp's 32*kVecs words of one stage; src: start of the warp's run in global memory
    __device__ static __forceinline__ void issue(uint4* warp_stage, const T* src, int lane) {
#pragma unroll
        for (int v = 0; v < kVecs; ++v) {
            const uint32_t c = v * 32 + lane;
            cp_async16(warp_stage + swz(c), reinterpret_cast<const uint4*>(src) + c);
        }
    }
    __device__ static __forceinline__ uint4 read(const uint4* warp_stage, int lane, int v) {
        return warp_stage[swz(lane * kVecs + v)];
    }
    // Write the warp's results through the (already consumed) stage so that global stores are as
    // coalesced as the loads: each lane drops its kVecs words at their swizzled positions, then
    // instruction v stores words v*32 .. v*32+31 (512 contiguous bytes) of the run at dst.
    __device__ static __forceinline__ void store_run(uint4* warp_stage, T* dst, int lane, const uint4 (&mine)[kVecs]) {
#pragma unroll
        for (int v = 0; v < kVecs; ++v) warp_stage[swz(lane * kVecs + v)] = mine[v];
        __syncwarp();
#pragma unroll
        for (int v = 0; v < kVecs; ++v) {
            const uint32_t c = v * 32 + lane;
            reinterpret_cast<uint4*>(dst)[c] = warp_stage[swz(c)];
        }
    }
};

// dequantized bit patterns of one slice -> the 16-byte words of the output tensor
__device__ __forceinline__ void slice_to_words(const uint32_t (&y)[kSlice], uint4 (&w)[4], const float*) {
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = make_uint4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
}
__device__ __forceinline__ void slice_to_words(const uint32_t (&y)[kSlice], uint4 (&w)[2], const __nv_bfloat16*) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint32_t ws[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) ws[k] = (y[8 * i + 2 * k] >> 16) | (y[8 * i + 2 * k + 1] & 0xFFFF0000u);
        w[i] = make_uint4(ws[0], ws[1], ws[2], ws[3]);
    }
}

}  // namespace bdr
