// Column-direction (axis 0) quantize-dequantize for every POW2 configuration that the Table II kernels do not take
// (any k1 <= 1024, k2 <= 16, d2, m; fp32 and bf16; optional fused Eq. 3 sums; no packed planes).
//
// A lane owns one column (fp32) or two adjacent columns (bf16: one 32-bit word per row), so a warp reads 128 contiguous
// bytes of every row it touches, and the eight warps of a CTA take eight adjacent column groups of the same rows.  A
// work unit is one k1-block of rows (at least 16 rows) of a column group:
//   * blocks longer than 16 rows first get their shared exponent from a pass over the block's rows (the maximum of the
//     raw exponent fields; the rows are read again right after, from L2);
//   * then the block is walked in slices of 16 rows: the slice sits in registers, sub-block exponents come from the
//     slice itself, and the slice quantizer of the row kernels does the rest (adder formulation, exact integer
//     formulation for ties-away and Inf/NaN blocks).
// Rows past the end of the tensor read as zeros, which is the zero padding of a short last block.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kCaThreads = 256;
constexpr int kCaWarps = kCaThreads / 32;

template <typename T> struct CaWord;
template <> struct CaWord<float> {
    static constexpr int kCols = 1;
    __device__ static uint32_t load(const float* p) { return __float_as_uint(__ldg(p)); }
    __device__ static void store(float* p, uint32_t w) { *p = __uint_as_float(w); }
    __device__ static uint32_t col_bits(uint32_t w, int) { return w; }
};
template <> struct CaWord<__nv_bfloat16> {
    static constexpr int kCols = 2;
    __device__ static uint32_t load(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint32_t*>(p)); }
    __device__ static void store(__nv_bfloat16* p, uint32_t w) { *reinterpret_cast<uint32_t*>(p) = w; }
    __device__ static uint32_t col_bits(uint32_t w, int c) { return c ? (w & 0xFFFF0000u) : (w << 16); }  // widened exactly
};

template <typename T, int K2, int K1S>
__global__ void __launch_bounds__(kCaThreads)
quant_col_any_kernel(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, QParams qp, double* sums, int64_t n_col_groups,
                     int64_t n_units) {
    using CW = CaWord<T>;
    constexpr int CPL = CW::kCols;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int kb = max(qp.k1, kSlice);  // rows per unit: one block, or the 16 / k1 blocks of a slice
    const bool want_sums = sums != nullptr, want_y = y != nullptr;
    double e2 = 0.0, s2 = 0.0;
    for (int64_t unit = (int64_t)blockIdx.x * kCaWarps + warp; unit < n_units; unit += (int64_t)gridDim.x * kCaWarps) {
        const int64_t rb = unit / n_col_groups, cg = unit - rb * n_col_groups;
        const int64_t col = (cg * 32 + lane) * CPL;
        if (col >= cols) continue;
        const int64_t r0 = rb * kb;
        const int nrows = (int)min((int64_t)kb, rows - r0);
        const T* xc = x + r0 * ld + col;
        T* yc = want_y ? y + r0 * ld + col : nullptr;
        // shared exponents of a block longer than one slice
        uint32_t Fblk[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) Fblk[c] = 0;
        if (qp.k1 > kSlice) {
            int r = 0;
            for (; r + 8 <= nrows; r += 8) {
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = CW::load(xc + (int64_t)(r + i) * ld);
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int c = 0; c < CPL; ++c) Fblk[c] = max(Fblk[c], CW::col_bits(w[i], c) & kExpMask);
            }
            for (; r < nrows; ++r) {
                const uint32_t w = CW::load(xc + (int64_t)r * ld);
#pragma unroll
                for (int c = 0; c < CPL; ++c) Fblk[c] = max(Fblk[c], CW::col_bits(w, c) & kExpMask);
            }
        }
        for (int s0 = 0; s0 < nrows; s0 += kSlice) {
            const int cnt = min(kSlice, nrows - s0);
            uint32_t w[kSlice], yo[kSlice];
#pragma unroll
            for (int i = 0; i < kSlice; ++i) w[i] = i < cnt ? CW::load(xc + (int64_t)(s0 + i) * ld) : 0u;
#pragma unroll
            for (int i = 0; i < kSlice; ++i) yo[i] = 0u;
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                uint32_t u[kSlice], ej[kSlice / K2], eb[kSlice / K1S], yb[kSlice], rq[kSlice], cb[kSlice / K2], tau[kSlice / K2];
#pragma unroll
                for (int i = 0; i < kSlice; ++i) u[i] = CW::col_bits(w[i], c);
                subblock_exponents<K2>(u, ej);
                if (K1S == kSlice && qp.k1 > kSlice) {
                    eb[0] = Fblk[c];
                } else {
#pragma unroll
                    for (int b = 0; b < kSlice / K1S; ++b) {
                        uint32_t m = 0;
#pragma unroll
                        for (int j = 0; j < K1S / K2; ++j) m = max(m, ej[b * (K1S / K2) + j]);
                        eb[b] = m;
                    }
                }
                quantize_slice_rt<K2, K1S, false>(u, ej, eb, qp, want_sums, want_y, yb, rq, cb, tau, e2, s2);
                if (want_y) {
#pragma unroll
                    for (int i = 0; i < kSlice; ++i) {
                        if (CPL == 1) yo[i] = yb[i];
                        else yo[i] |= c ? (yb[i] & 0xFFFF0000u) : (yb[i] >> 16);  // exact: m <= 8 significant bits
                    }
                }
            }
            if (want_y) {
#pragma unroll
                for (int i = 0; i < kSlice; ++i)
                    if (i < cnt) CW::store(yc + (int64_t)(s0 + i) * ld, yo[i]);
            }
        }
    }
    if (want_sums) block_accumulate_sums(e2, s2, sums);
}

template <typename T, int K2, int K1S>
static int launch_col_any(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums, cudaStream_t st) {
    constexpr int CPL = CaWord<T>::kCols;
    const int kb = std::max(qp.k1, (int)kSlice);
    const int64_t n_cg = (cols + 32 * CPL - 1) / (32 * CPL), n_rb = (rows + kb - 1) / kb, n_units = n_cg * n_rb;
    if (n_units == 0) return BDR_OK;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((n_units + kCaWarps - 1) / kCaWarps, (int64_t)sm_count() * 8));
    quant_col_any_kernel<T, K2, K1S><<<grid, kCaThreads, 0, st>>>(x, y, rows, cols, ld, qp, sums, n_cg, n_units);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T, int K1S>
static int col_any_k2(int k2, const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums, cudaStream_t st) {
    switch (k2) {
        case 1: return launch_col_any<T, 1, K1S>(x, y, rows, cols, ld, qp, sums, st);
        case 2: if constexpr (K1S >= 2) return launch_col_any<T, 2, K1S>(x, y, rows, cols, ld, qp, sums, st); break;
        case 4: if constexpr (K1S >= 4) return launch_col_any<T, 4, K1S>(x, y, rows, cols, ld, qp, sums, st); break;
        case 8: if constexpr (K1S >= 8) return launch_col_any<T, 8, K1S>(x, y, rows, cols, ld, qp, sums, st); break;
        case 16: if constexpr (K1S >= 16) return launch_col_any<T, 16, K1S>(x, y, rows, cols, ld, qp, sums, st); break;
    }
    return BDR_ERR_UNSUPPORTED;
}

// Any POW2 configuration with k1 a power of two <= 1024 and k2 <= 16 (or d2 = 0).  bf16 needs an even number of columns, an even
// pitch and 4-byte aligned tensors (two columns travel in one word).  BDR_ERR_UNSUPPORTED sends the caller to the general kernel.
template <typename T>
int quant_colwise_any(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp_in, double* sums, cudaStream_t st) {
    QParams qp = qp_in;
    const int k2 = qp.d2 == 0 ? std::min(qp.k1, (int)kSlice) : qp.k2;  // d2 = 0: every shift is zero whatever k2 is
    if (k2 > kSlice || qp.k1 > 1024) return BDR_ERR_UNSUPPORTED;
    qp.k2 = k2;
    if (sizeof(T) == 2 && ((cols | ld) % 2 != 0 || ((uintptr_t)x | (uintptr_t)y) % 4 != 0)) return BDR_ERR_UNSUPPORTED;
    switch (qp.k1) {
        case 1: return col_any_k2<T, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 2: return col_any_k2<T, 2>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 4: return col_any_k2<T, 4>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 8: return col_any_k2<T, 8>(k2, x, y, rows, cols, ld, qp, sums, st);
        default: return col_any_k2<T, 16>(k2, x, y, rows, cols, ld, qp, sums, st);
    }
}
template int quant_colwise_any<float>(const float*, float*, int64_t, int64_t, int64_t, const QParams&, double*, cudaStream_t);
template int quant_colwise_any<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, int64_t, int64_t, int64_t, const QParams&, double*,
                                              cudaStream_t);

}  // namespace bdr
