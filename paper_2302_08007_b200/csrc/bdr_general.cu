// General kernels: any axis, any POW2 configuration, any pitch or alignment, ragged tails.
// Correctness first; the fast paths in bdr_row.cu / bdr_col.cu / bdr_unpack.cu cover the shapes
// that matter for throughput and produce identical bytes.
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kGenThreads = 128;

// OR a field into an LSB-first bit stream whose line starts 4-byte aligned (planes are zeroed first).
__device__ __forceinline__ void or_bits(uint8_t* line, int64_t bitpos, int nbits, uint32_t val) {
    if (!val) return;
    uint32_t* w = reinterpret_cast<uint32_t*>(line) + (bitpos >> 5);
    const int sh = (int)(bitpos & 31);
    atomicOr(w, val << sh);
    if (sh + nbits > 32) atomicOr(w + 1, val >> (32 - sh));
}

__device__ __forceinline__ uint32_t get_bits(const uint8_t* line, int64_t bitpos, int nbits) {
    const uint32_t* w = reinterpret_cast<const uint32_t*>(line) + (bitpos >> 5);
    const int sh = (int)(bitpos & 31);
    uint32_t v = w[0] >> sh;
    if (sh + nbits > 32) v |= w[1] << (32 - sh);
    return v & ((1u << nbits) - 1u);
}

// One thread per (line, k1-block).
template <typename T>
__global__ void __launch_bounds__(kGenThreads)
quant_general_kernel(const T* x, T* y, int64_t nlines, int64_t len, int64_t line_stride, int64_t elem_stride,
                     int64_t nblocks, int64_t total_rounded, bdr_planes_t out, bool pack, QParams qp, double* sums) {
    double e2 = 0.0, s2 = 0.0;
    const int nsub = qp.k1 / qp.k2;
    for (int64_t g = (int64_t)blockIdx.x * kGenThreads + threadIdx.x; g < total_rounded;
         g += (int64_t)gridDim.x * kGenThreads) {
        if (g >= nlines * nblocks) continue;
        const int64_t line = g / nblocks, b = g - line * nblocks;
        const int64_t i0 = b * qp.k1;
        const int n = (int)min((int64_t)qp.k1, len - i0);
        const T* px = x + line * line_stride + i0 * elem_stride;
        T* py = y ? y + line * line_stride + i0 * elem_stride : nullptr;
        int F = 0;
        for (int i = 0; i < n; ++i) F = max(F, exp_field(Elem<T>::load_bits(px + i * elem_stride)));
        if (pack) out.exps[line * out.ld_exps + b] = (uint8_t)F;
        for (int j = 0; j < nsub; ++j) {
            int Fj = 0;
            for (int i = j * qp.k2; i < (j + 1) * qp.k2 && i < n; ++i)
                Fj = max(Fj, exp_field(Elem<T>::load_bits(px + i * elem_stride)));
            const int tau = F == 255 ? 0 : min(F - Fj, qp.beta);
            if (pack && qp.d2) or_bits(out.micro + line * out.ld_micro, (b * nsub + j) * (int64_t)qp.d2, qp.d2, (uint32_t)tau);
            for (int i = j * qp.k2; i < (j + 1) * qp.k2 && i < n; ++i) {
                const uint32_t u = Elem<T>::load_bits(px + i * elem_stride);
                uint32_t q = 0, yb = 0x7FC00000u;
                if (F != 255) quant_elem_exact(u, F, tau, qp, q, yb);
                const uint32_t code = F == 255 ? 0u : (((u >> 31) << qp.m) | q);
                if (py) Elem<T>::store_bits(py + i * elem_stride, yb);
                if (pack) or_bits(out.elems + line * out.ld_elems, (i0 + i) * (int64_t)(qp.m + 1), qp.m + 1, code);
                if (sums) {
                    const double de = (double)__uint_as_float(yb) - (double)__uint_as_float(u);
                    const double dx = (double)__uint_as_float(u);
                    e2 = fma(de, de, e2);
                    s2 = fma(dx, dx, s2);
                }
            }
        }
    }
    if (sums) block_accumulate_sums(e2, s2, sums);
}

// One thread per element.
template <typename T>
__global__ void __launch_bounds__(kGenThreads)
unpack_general_kernel(bdr_planes_t in, T* y, int64_t nlines, int64_t len, int64_t line_stride, int64_t elem_stride,
                      int axis, QParams qp) {
    const int nsub = qp.k1 / qp.k2;
    const int64_t total = nlines * len;
    for (int64_t g = (int64_t)blockIdx.x * kGenThreads + threadIdx.x; g < total; g += (int64_t)gridDim.x * kGenThreads) {
        // consecutive threads walk the contiguous dimension of y
        const int64_t line = axis == 1 ? g / len : g % nlines;
        const int64_t i = axis == 1 ? g % len : g / nlines;
        const int64_t b = i / qp.k1;
        const int F = in.exps[line * in.ld_exps + b];
        uint32_t yb = 0x7FC00000u;
        if (F != 255) {
            const int64_t j = b * nsub + (i - b * qp.k1) / qp.k2;
            const int tau = qp.d2 ? (int)get_bits(in.micro + line * in.ld_micro, j * (int64_t)qp.d2, qp.d2) : 0;
            const uint32_t code = get_bits(in.elems + line * in.ld_elems, i * (int64_t)(qp.m + 1), qp.m + 1);
            const uint32_t q = code & qp.qmax;
            const int p = max(F - 127 - tau - (qp.m - 1), -149);
            yb = __float_as_uint(__fmul_rn(__uint2float_rn(q), __uint_as_float(pow2_bits(p)))) | ((code >> qp.m) << 31);
        }
        Elem<T>::store_bits(y + line * line_stride + i * elem_stride, yb);
    }
}

// Three-level scaling (Section III, last paragraph): an FP32 parent scale per group of k_parent consecutive elements of a
// line above the two-level quantizer.  One warp per group (k_parent <= 1024): a lane holds the group's 16-element slices
// lane, lane + 32; group maximum by shuffle; s = amax / V with V = (2^m - 1) 2^-(m-1); x' = x / s (IEEE division); the
// two-level quantizer on x' (k1 <= 16: the blocks of a slice; the exact integer formulation); y = Q(x') s.
__global__ void __launch_bounds__(kGenThreads)
parent_scale_kernel(const float* x, float* y, int64_t nlines, int64_t len, int64_t line_stride, int64_t elem_stride, int k_parent,
                    QParams qp, double* sums) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kGenThreads + threadIdx.x) >> 5, nwarps = ((int64_t)gridDim.x * kGenThreads) >> 5;
    const int64_t gpl = (len + k_parent - 1) / k_parent, total = nlines * gpl;
    const float V = (float)qp.qmax * __uint_as_float((uint32_t)(127 - (qp.m - 1)) << 23);
    double e2 = 0.0, s2 = 0.0;
    for (int64_t g = warp0; g < total; g += nwarps) {
        const int64_t line = g / gpl, g0 = (g - line * gpl) * k_parent;
        const int n = (int)min((int64_t)k_parent, len - g0);
        const float* xg = x + line * line_stride + g0 * elem_stride;
        float* yg = y ? y + line * line_stride + g0 * elem_stride : nullptr;
        uint32_t u[2][kSlice];
        uint32_t am = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e0 = (lane + 32 * h) * kSlice;
            load_slice_guarded(xg + (int64_t)e0 * elem_stride, elem_stride, max(0, min(kSlice, n - e0)), u[h]);
#pragma unroll
            for (int i = 0; i < kSlice; ++i) am = max(am, u[h][i] & 0x7FFFFFFFu);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
        const float s = __fdiv_rn(__uint_as_float(am), V);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e0 = (lane + 32 * h) * kSlice;
            const int cnt = max(0, min(kSlice, n - e0));
            if (cnt == 0) continue;
            uint32_t yb[kSlice];
            if (!(s > 0.f)) {
#pragma unroll
                for (int i = 0; i < kSlice; ++i) yb[i] = u[h][i] & 0x80000000u;
            } else {
                uint32_t xs[kSlice];
#pragma unroll
                for (int i = 0; i < kSlice; ++i) xs[i] = __float_as_uint(__fdiv_rn(__uint_as_float(u[h][i]), s));
                for (int b0 = 0; b0 < kSlice; b0 += qp.k1) {        // the slice's k1-blocks (k1 <= 16)
                    int F = 0;
                    for (int i = 0; i < qp.k1; ++i) F = max(F, exp_field(xs[b0 + i]));
                    for (int j0 = b0; j0 < b0 + qp.k1; j0 += qp.k2) {
                        int Fj = 0;
                        for (int i = 0; i < qp.k2; ++i) Fj = max(Fj, exp_field(xs[j0 + i]));
                        const int tau = F == 255 ? 0 : min(F - Fj, qp.beta);
                        for (int i = 0; i < qp.k2; ++i) {
                            uint32_t q = 0, yq = 0x7FC00000u;
                            if (F != 255) quant_elem_exact(xs[j0 + i], F, tau, qp, q, yq);
                            yb[j0 + i] = __float_as_uint(__fmul_rn(__uint_as_float(yq), s));
                        }
                    }
                }
            }
            if (yg) store_slice_guarded(yg + (int64_t)e0 * elem_stride, elem_stride, cnt, yb);
            if (sums) {
                for (int i = 0; i < cnt; ++i) {
                    const double a = (double)__uint_as_float(u[h][i]), d = (double)__uint_as_float(yb[i]) - a;
                    e2 = fma(d, d, e2);
                    s2 = fma(a, a, s2);
                }
            }
        }
    }
    if (sums) block_accumulate_sums(e2, s2, sums);
}

// The same for the common shape: rows along the contiguous dimension, k1 = 16, groups of 16 * 2^j <= 1024 elements that tile
// the row, 16-byte aligned rows.  A thread owns one 16-element slice (one block) of a group -- two when the group has 64 slices --
// loaded and stored with 16-byte accesses; the group maximum goes round the group's lanes by shuffle; x / s is the correctly
// rounded quotient computed with the rounded reciprocal, a residual and a correction (one reciprocal per group; plain division
// where that shortcut is not safe); the two-level quantizer is the adder formulation of quantize_slice.
struct PsDivisor {
    float s, r;
    bool fast;
};
__device__ __forceinline__ PsDivisor ps_make_divisor(float s) {
    PsDivisor d;
    d.s = s;
    d.r = __frcp_rn(s);
    const uint32_t b = __float_as_uint(s);
    d.fast = (b & 0x7FFFFFu) != 0x7FFFFFu && b >= 0x0D800000u /*2^-100*/ && b <= 0x71800000u /*2^100*/;
    return d;
}
// x / d.s, correctly rounded.  Fast route: q0 = RN(x r), e = x - q0 s (exact in one fused multiply-add), q = RN(q0 + e r); valid
// while nothing leaves the normal range: the residual is a multiple of ulp(q0) ulp(s), so x and q0 are kept above 2^-100 (s lies
// within 2^+-100, and |x| <= amax makes the quotient smaller than 2); anything else takes the division instruction.
__device__ __forceinline__ float ps_divide(float x, const PsDivisor& d) {
    const float q0 = __fmul_rn(x, d.r);
    const bool ok = d.fast && (__float_as_uint(x) & 0x7FFFFFFFu) >= 0x0D800000u && (__float_as_uint(q0) & 0x7FFFFFFFu) >= 0x0D800000u;
    if (ok) return __fmaf_rn(__fmaf_rn(-q0, d.s, x), d.r, q0);
    return __fdiv_rn(x, d.s);
}

template <int K2>
__global__ void __launch_bounds__(kGenThreads)
parent_scale_rows_kernel(const float* x, float* y, int64_t rows, int64_t cols, int64_t ld, int slices_per_group, QParams qp, double* sums) {
    const int lanes = min(slices_per_group, 32), per_lane = slices_per_group > 32 ? 2 : 1;   // lanes of a group, slices per lane
    const int64_t spr = cols / kSlice / per_lane;                                              // threads per row
    const int64_t total = rows * spr;
    const float V = (float)qp.qmax * __uint_as_float((uint32_t)(127 - (qp.m - 1)) << 23);
    double e2 = 0.0, s2 = 0.0;
    const int64_t nthreads = (int64_t)gridDim.x * kGenThreads;
    const int64_t rounded = (total + 31) / 32 * 32;   // whole warps take part in the shuffles
    for (int64_t t = (int64_t)blockIdx.x * kGenThreads + threadIdx.x; t < rounded; t += nthreads) {
        const bool live = t < total;
        const int64_t row = live ? t / spr : 0, pos = live ? t - row * spr : 0;
        // with two slices per lane a warp is one group: lane l owns slices l and l + 32 of it
        const int64_t slice0 = per_lane == 2 ? (pos / 32) * 64 + (pos & 31) : pos;
        uint32_t u[2][kSlice];
        uint32_t am = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (h < per_lane && live) {
                load_slice_vec(x + row * ld + (slice0 + 32 * h) * kSlice, u[h]);
#pragma unroll
                for (int i = 0; i < kSlice; ++i) am = max(am, u[h][i] & 0x7FFFFFFFu);
            }
        }
        for (int o = lanes >> 1; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
        if (!live) continue;
        const float s = __fdiv_rn(__uint_as_float(am), V);
        const PsDivisor dv = ps_make_divisor(s);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (h >= per_lane) break;
            uint32_t yb[kSlice];
            if (!(s > 0.f)) {
#pragma unroll
                for (int i = 0; i < kSlice; ++i) yb[i] = u[h][i] & 0x80000000u;
            } else {
                uint32_t xs[kSlice], ej[kSlice / K2], fb[1], rq[kSlice], cb[kSlice / K2], tau[kSlice / K2];
#pragma unroll
                for (int i = 0; i < kSlice; ++i) xs[i] = __float_as_uint(ps_divide(__uint_as_float(u[h][i]), dv));
                subblock_exponents<K2>(xs, ej);
                uint32_t F = 0;
#pragma unroll
                for (int j = 0; j < kSlice / K2; ++j) F = max(F, ej[j]);
                fb[0] = F;
                double de = 0.0, ds = 0.0;
                quantize_slice<K2, kSlice, false, true, false>(xs, ej, fb, qp, yb, rq, cb, tau, de, ds);
#pragma unroll
                for (int i = 0; i < kSlice; ++i) yb[i] = __float_as_uint(__fmul_rn(__uint_as_float(yb[i]), s));
            }
            if (y) store_slice_vec(y + row * ld + (slice0 + 32 * h) * kSlice, yb);
            if (sums) {
#pragma unroll
                for (int i = 0; i < kSlice; ++i) {
                    const double a = (double)__uint_as_float(u[h][i]), d = (double)__uint_as_float(yb[i]) - a;
                    e2 = fma(d, d, e2);
                    s2 = fma(a, a, s2);
                }
            }
        }
    }
    if (sums) block_accumulate_sums(e2, s2, sums);
}

template <int K2>
static int launch_parent_rows(const float* x, float* y, int64_t rows, int64_t cols, int64_t ld, int k_parent, const QParams& qp, double* sums,
                              cudaStream_t st) {
    const int spg = k_parent / kSlice;
    const int64_t total = rows * (cols / kSlice / (spg > 32 ? 2 : 1));
    const int grid = (int)max((int64_t)1, min((total + kGenThreads - 1) / kGenThreads, (int64_t)sm_count() * 16));
    parent_scale_rows_kernel<K2><<<grid, kGenThreads, 0, st>>>(x, y, rows, cols, ld, spg, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

int quant_parent_scale(const float* x, float* y, int64_t rows, int64_t cols, int64_t ld, int axis, int k_parent, const QParams& qp,
                       double* sums, cudaStream_t st) {
    const bool pow2 = (k_parent & (k_parent - 1)) == 0;
    if (axis == 1 && qp.k1 == kSlice && pow2 && k_parent >= kSlice && k_parent <= 1024 && cols % k_parent == 0 && ld % 4 == 0 &&
        ((uintptr_t)x | (uintptr_t)y) % 16 == 0 && rows > 0 && cols > 0) {
        switch (qp.k2) {
            case 1: return launch_parent_rows<1>(x, y, rows, cols, ld, k_parent, qp, sums, st);
            case 2: return launch_parent_rows<2>(x, y, rows, cols, ld, k_parent, qp, sums, st);
            case 4: return launch_parent_rows<4>(x, y, rows, cols, ld, k_parent, qp, sums, st);
            case 8: return launch_parent_rows<8>(x, y, rows, cols, ld, k_parent, qp, sums, st);
            case 16: return launch_parent_rows<16>(x, y, rows, cols, ld, k_parent, qp, sums, st);
        }
    }
    const int64_t nlines = axis == 1 ? rows : cols, len = axis == 1 ? cols : rows;
    const int64_t line_stride = axis == 1 ? ld : 1, elem_stride = axis == 1 ? 1 : ld;
    const int64_t groups = nlines * ((len + k_parent - 1) / k_parent);
    if (groups == 0) return BDR_OK;
    const int grid = (int)max((int64_t)1, min((groups * 32 + kGenThreads - 1) / kGenThreads, (int64_t)sm_count() * 16));
    parent_scale_kernel<<<grid, kGenThreads, 0, st>>>(x, y, nlines, len, line_stride, elem_stride, k_parent, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Row gather from a packed table (axis-1 planes of [n_rows, len]): output line l is the decoded row idx[l].
// One thread per element; an index outside the table gives a row of quiet NaNs and leaves BDR_ERR_SIZE in *status.
template <typename T>
__global__ void __launch_bounds__(kGenThreads)
gather_rows_kernel(bdr_planes_t in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t len, int64_t ld, QParams qp,
                   int* status) {
    const int nsub = qp.k1 / qp.k2;
    const int64_t total = n_idx * len;
    for (int64_t g = (int64_t)blockIdx.x * kGenThreads + threadIdx.x; g < total; g += (int64_t)gridDim.x * kGenThreads) {
        const int64_t l = g / len, i = g - l * len;
        const int64_t line = idx[l];
        uint32_t yb = 0x7FC00000u;
        if (line < 0 || line >= n_rows) {
            if (i == 0) atomicCAS(status, 0, (int)BDR_ERR_SIZE);
        } else {
            const int64_t b = i / qp.k1;
            const int F = in.exps[line * in.ld_exps + b];
            if (F != 255) {
                const int64_t j = b * nsub + (i - b * qp.k1) / qp.k2;
                const int tau = qp.d2 ? (int)get_bits(in.micro + line * in.ld_micro, j * (int64_t)qp.d2, qp.d2) : 0;
                const uint32_t code = get_bits(in.elems + line * in.ld_elems, i * (int64_t)(qp.m + 1), qp.m + 1);
                const uint32_t q = code & qp.qmax;
                const int p = max(F - 127 - tau - (qp.m - 1), -149);
                yb = __float_as_uint(__fmul_rn(__uint2float_rn(q), __uint_as_float(pow2_bits(p)))) | ((code >> qp.m) << 31);
            }
        }
        Elem<T>::store_bits(y + l * ld + i, yb);
    }
}

template <typename T>
int gather_rows_general(const bdr_planes_t& in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t len, int64_t ld,
                        const QParams& qp, int* status, cudaStream_t st) {
    const int64_t total = n_idx * len;
    if (total == 0) return BDR_OK;
    const int grid = (int)max((int64_t)1, min((total + kGenThreads - 1) / kGenThreads, (int64_t)sm_count() * 16));
    gather_rows_kernel<T><<<grid, kGenThreads, 0, st>>>(in, n_rows, idx, y, n_idx, len, ld, qp, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}
template int gather_rows_general<float>(const bdr_planes_t&, int64_t, const int64_t*, float*, int64_t, int64_t, int64_t, const QParams&, int*,
                                        cudaStream_t);
template int gather_rows_general<__nv_bfloat16>(const bdr_planes_t&, int64_t, const int64_t*, __nv_bfloat16*, int64_t, int64_t, int64_t,
                                                const QParams&, int*, cudaStream_t);

template <typename T>
int quant_general(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const bdr_planes_t* out,
                  const QParams& qp, double* sums, cudaStream_t st) {
    const int64_t nlines = axis == 1 ? rows : cols, len = axis == 1 ? cols : rows;
    const int64_t line_stride = axis == 1 ? ld : 1, elem_stride = axis == 1 ? 1 : ld;
    const int64_t nblocks = (len + qp.k1 - 1) / qp.k1;
    bdr_planes_t pl = {};
    if (out) {
        pl = *out;
        if (cudaMemsetAsync(pl.exps, 0, (size_t)(nlines * pl.ld_exps), st) != cudaSuccess) return BDR_ERR_CUDA;
        if (qp.d2 && pl.micro && cudaMemsetAsync(pl.micro, 0, (size_t)(nlines * pl.ld_micro), st) != cudaSuccess)
            return BDR_ERR_CUDA;
        if (cudaMemsetAsync(pl.elems, 0, (size_t)(nlines * pl.ld_elems), st) != cudaSuccess) return BDR_ERR_CUDA;
    }
    const int64_t total = nlines * nblocks;
    if (total == 0) return BDR_OK;
    const int64_t rounded = (total + kGenThreads - 1) / kGenThreads * kGenThreads;
    const int grid = (int)max((int64_t)1, min(rounded / kGenThreads, (int64_t)sm_count() * 16));
    quant_general_kernel<T><<<grid, kGenThreads, 0, st>>>(x, y, nlines, len, line_stride, elem_stride, nblocks, rounded,
                                                          pl, out != nullptr, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T>
int unpack_general(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const QParams& qp,
                   cudaStream_t st) {
    const int64_t nlines = axis == 1 ? rows : cols, len = axis == 1 ? cols : rows;
    const int64_t line_stride = axis == 1 ? ld : 1, elem_stride = axis == 1 ? 1 : ld;
    const int64_t total = nlines * len;
    if (total == 0) return BDR_OK;
    const int grid = (int)max((int64_t)1, min((total + kGenThreads - 1) / kGenThreads, (int64_t)sm_count() * 16));
    unpack_general_kernel<T><<<grid, kGenThreads, 0, st>>>(in, y, nlines, len, line_stride, elem_stride, axis, qp);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template int quant_general<float>(const float*, float*, int64_t, int64_t, int64_t, int, const bdr_planes_t*,
                                  const QParams&, double*, cudaStream_t);
template int quant_general<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, int64_t, int64_t, int64_t, int,
                                          const bdr_planes_t*, const QParams&, double*, cudaStream_t);
template int unpack_general<float>(const bdr_planes_t&, float*, int64_t, int64_t, int64_t, int, const QParams&,
                                   cudaStream_t);
template int unpack_general<__nv_bfloat16>(const bdr_planes_t&, __nv_bfloat16*, int64_t, int64_t, int64_t, int,
                                           const QParams&, cudaStream_t);

}  // namespace bdr
