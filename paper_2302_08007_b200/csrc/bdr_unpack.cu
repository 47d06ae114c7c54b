// Row-direction (axis 1) unpack fast path for the k1 = 16, k2 = 2 family: the mirror image of the
// packing kernel.  A warp pulls the packed bytes of 32 consecutive slices (512 elements) with
// coalesced 16-byte loads into shared memory, each lane decodes its own slice from there and
// writes it with 128-bit stores.
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kUnpackThreads = 256;

template <typename T, int W>
__global__ void __launch_bounds__(kUnpackThreads)
unpack_rowwise_mx_kernel(bdr_planes_t in, T* y, int64_t rows, int64_t cols, int64_t ld, QParams qp) {
    constexpr int kWarps = kUnpackThreads / 32;
    constexpr int kElemBytes = 2 * W;
    constexpr int kStage = (32 * kElemBytes + 32 + 96 + 15) / 16 * 16;
    __shared__ __align__(16) uint8_t stage_all[kWarps][kStage];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* stage = stage_all[warp];
    uint8_t* st_exps = stage + 32 * kElemBytes;
    uint8_t* st_micro = st_exps + 32;
    const int64_t warps_per_row = cols / 512;
    const int64_t total = rows * warps_per_row;
    for (int64_t wi = (int64_t)blockIdx.x * kWarps + warp; wi < total; wi += (int64_t)gridDim.x * kWarps) {
        const int64_t row = wi / warps_per_row;
        const int64_t slice0 = (wi - row * warps_per_row) * 32;
        const uint4* g_elems = reinterpret_cast<const uint4*>(in.elems + row * in.ld_elems + slice0 * kElemBytes);
        uint4* s4 = reinterpret_cast<uint4*>(stage);
        for (int v = lane; v < 32 * kElemBytes / 16; v += 32) s4[v] = __ldg(g_elems + v);
        if (lane < 2) {
            reinterpret_cast<uint4*>(st_exps)[lane] =
                __ldg(reinterpret_cast<const uint4*>(in.exps + row * in.ld_exps + slice0) + lane);
        } else if (lane - 2 < 2 * qp.d2) {
            reinterpret_cast<uint4*>(st_micro)[lane - 2] =
                __ldg(reinterpret_cast<const uint4*>(in.micro + row * in.ld_micro + slice0 * qp.d2) + (lane - 2));
        }
        __syncwarp();
        uint32_t words[(kSlice * W + 31) / 32 + 1];
#pragma unroll
        for (int i = 0; i < (kSlice * W + 31) / 32 + 1; ++i) words[i] = 0;
        if (W == 8) {
            const uint4 w = *reinterpret_cast<const uint4*>(stage + lane * kElemBytes);
            words[0] = w.x; words[1] = w.y; words[2] = w.z; words[3] = w.w;
        } else {
            const uint16_t* src = reinterpret_cast<const uint16_t*>(stage + lane * kElemBytes);
#pragma unroll
            for (int h = 0; h < W; ++h) words[h >> 1] |= (uint32_t)src[h] << ((h & 1) * 16);
        }
        const int F = st_exps[lane];
        uint32_t mbits = 0;
        for (int b = 0; b < qp.d2; ++b) mbits |= (uint32_t)st_micro[lane * qp.d2 + b] << (8 * b);
        uint32_t yb[kSlice];
        decode_slice<W>(words, F, mbits, qp, yb);
        store_slice_vec(y + row * ld + (slice0 + lane) * kSlice, yb);
        __syncwarp();
    }
}

template <typename T, int W>
static int launch_unpack_row(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                             cudaStream_t st) {
    const int64_t total = rows * (cols / 512);
    const int64_t need = (total + kUnpackThreads / 32 - 1) / (kUnpackThreads / 32);
    const int grid = (int)max((int64_t)1, min(need, (int64_t)sm_count() * 8));
    unpack_rowwise_mx_kernel<T, W><<<grid, kUnpackThreads, 0, st>>>(in, y, rows, cols, ld, qp);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T>
int unpack_rowwise_mx(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                      cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || cols % 512 != 0) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)y % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    switch (qp.m + 1) {
        case 2: return launch_unpack_row<T, 2>(in, y, rows, cols, ld, qp, st);
        case 3: return launch_unpack_row<T, 3>(in, y, rows, cols, ld, qp, st);
        case 4: return launch_unpack_row<T, 4>(in, y, rows, cols, ld, qp, st);
        case 5: return launch_unpack_row<T, 5>(in, y, rows, cols, ld, qp, st);
        case 6: return launch_unpack_row<T, 6>(in, y, rows, cols, ld, qp, st);
        case 7: return launch_unpack_row<T, 7>(in, y, rows, cols, ld, qp, st);
        case 8: return launch_unpack_row<T, 8>(in, y, rows, cols, ld, qp, st);
        case 9: return launch_unpack_row<T, 9>(in, y, rows, cols, ld, qp, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

template int unpack_rowwise_mx<float>(const bdr_planes_t&, float*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);
template int unpack_rowwise_mx<__nv_bfloat16>(const bdr_planes_t&, __nv_bfloat16*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);

}  // namespace bdr
