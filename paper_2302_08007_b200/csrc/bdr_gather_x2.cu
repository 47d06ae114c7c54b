// Embedding-table lookups from MX-packed storage (Section V, inferencing: in memory-bound models the embedding tables are
// kept in MX format too): output row l = decoded row idx[l] of a [n_rows, dim] table packed along its rows.
// Fast path for the Table II formats.  A thread decodes one item of 32 consecutive elements (two blocks): it fetches the
// item's W code words, its two exponent bytes and its two microexponent bytes straight from the table (the rows are
// chosen at random, so there is nothing to stage: a row of 128 elements is 48 - 128 bytes of codes plus 8 + 8 bytes of
// scales), decodes them with the packed bf16x2 arithmetic of bdr_x2.cuh and writes 64 bytes (bf16) or 128 bytes (fp32,
// widened exactly).  Consecutive threads take consecutive items of the same output row, so the writes are contiguous.
// Bound by HBM latency and bandwidth on the random reads; an index outside the table gives a row of quiet NaNs and
// leaves BDR_ERR_SIZE in the status word.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kGxThreads = 256;

template <int W, typename T>
__global__ void __launch_bounds__(kGxThreads)
gather_rows_x2_kernel(bdr_planes_t in, int64_t n_rows, const int64_t* __restrict__ idx, T* y, int64_t n_items, uint32_t items_per_row,
                      int64_t ld, int* status) {
    const int64_t stride = (int64_t)gridDim.x * kGxThreads;
    for (int64_t g = (int64_t)blockIdx.x * kGxThreads + threadIdx.x; g < n_items; g += stride) {
        const int64_t l = g / items_per_row;
        const uint32_t it = (uint32_t)(g - l * items_per_row);
        const int64_t row = __ldg(idx + l);
        uint32_t yw[16];
        if (row < 0 || row >= n_rows) {
            if (it == 0) atomicCAS(status, 0, (int)BDR_ERR_SIZE);
#pragma unroll
            for (int k = 0; k < 16; ++k) yw[k] = 0x7FC07FC0u;
        } else {
            uint32_t s[W];
            const uint8_t* codes = in.elems + row * in.ld_elems + (int64_t)it * 4 * W;
            if constexpr (W == 8) {
                const uint4 a = __ldg(reinterpret_cast<const uint4*>(codes)), b = __ldg(reinterpret_cast<const uint4*>(codes) + 1);
                s[0] = a.x; s[1] = a.y; s[2] = a.z; s[3] = a.w;
                s[4] = b.x; s[5] = b.y; s[6] = b.z; s[7] = b.w;
            } else {
#pragma unroll
                for (int k = 0; k < W; ++k) s[k] = __ldg(reinterpret_cast<const uint32_t*>(codes) + k);
            }
            const uint32_t Fw = __ldg(reinterpret_cast<const uint16_t*>(in.exps + row * in.ld_exps) + it);
            const uint32_t mw = __ldg(reinterpret_cast<const uint16_t*>(in.micro + row * in.ld_micro) + it);
            const uint32_t F0 = Fw & 0xFFu, F1 = Fw >> 8;
            if ((F0 - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF)) && (F1 - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF))) {
                x2::decode_two_blocks_row<W>(s, F0, F1, mw, yw);
            } else {
                x2::TwoBlocks<W> in2;
#pragma unroll
                for (int k = 0; k < W; ++k) in2.s[k] = s[k];
                const x2::TwoBlocksOut o = x2::decode_two_blocks_slow<W>(in2, F0, F1, mw);
#pragma unroll
                for (int k = 0; k < 16; ++k) yw[k] = o.y[k];
            }
        }
        if constexpr (sizeof(T) == 2) {
            uint4* dst = reinterpret_cast<uint4*>(y + l * ld + (int64_t)it * 32);
#pragma unroll
            for (int k = 0; k < 4; ++k) dst[k] = make_uint4(yw[4 * k], yw[4 * k + 1], yw[4 * k + 2], yw[4 * k + 3]);
        } else {  // a bf16 value widens to fp32 by appending sixteen zero bits
            uint4* dst = reinterpret_cast<uint4*>(y + l * ld + (int64_t)it * 32);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                dst[k] = make_uint4(yw[2 * k] << 16, yw[2 * k] & 0xFFFF0000u, yw[2 * k + 1] << 16, yw[2 * k + 1] & 0xFFFF0000u);
        }
    }
}

template <int W, typename T>
static int launch_gather_x2(const bdr_planes_t& in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t dim, int64_t ld,
                            int* status, cudaStream_t st) {
    const int64_t n_items = n_idx * (dim / 32);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((n_items + kGxThreads - 1) / kGxThreads, (int64_t)sm_count() * 32));
    gather_rows_x2_kernel<W, T><<<grid, kGxThreads, 0, st>>>(in, n_rows, idx, y, n_items, (uint32_t)(dim / 32), ld, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Table II formats, rows of whole 32-element items, 16-byte aligned output rows.  BDR_ERR_UNSUPPORTED sends the caller to
// the general kernel.
template <typename T>
int gather_rows_mx_x2(const bdr_planes_t& in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t dim, int64_t ld,
                      const QParams& qp, int* status, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1) return BDR_ERR_UNSUPPORTED;
    if (dim % 32 != 0 || dim / 32 >= (1ll << 31) || ((uintptr_t)y % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return launch_gather_x2<3, T>(in, n_rows, idx, y, n_idx, dim, ld, status, st);
        case 4: return launch_gather_x2<5, T>(in, n_rows, idx, y, n_idx, dim, ld, status, st);
        case 7: return launch_gather_x2<8, T>(in, n_rows, idx, y, n_idx, dim, ld, status, st);
    }
    return BDR_ERR_UNSUPPORTED;
}
template int gather_rows_mx_x2<float>(const bdr_planes_t&, int64_t, const int64_t*, float*, int64_t, int64_t, int64_t, const QParams&, int*,
                                      cudaStream_t);
template int gather_rows_mx_x2<__nv_bfloat16>(const bdr_planes_t&, int64_t, const int64_t*, __nv_bfloat16*, int64_t, int64_t, int64_t,
                                              const QParams&, int*, cudaStream_t);

}  // namespace bdr
