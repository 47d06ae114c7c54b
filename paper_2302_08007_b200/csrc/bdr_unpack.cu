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
unpack_rowwise_mx_kernel(bdr_planes_t in, T* y, FastDiv warps_per_row, uint32_t total, int64_t ld, QParams qp) {
    constexpr int kWarps = kUnpackThreads / 32;
    constexpr int kElemBytes = 2 * W;
    constexpr int kStage = (32 * kElemBytes + 32 + 96 + 15) / 16 * 16;
    constexpr int kStages = 3;  // packed bytes are prefetched two iterations ahead with cp.async
    __shared__ __align__(16) uint8_t stage_all[kWarps][kStages][kStage];
    using R = Ring<T, 1>;  // only its swizzled, coalesced store path is used here
    __shared__ __align__(16) uint4 out_stage[kWarps][32 * R::kVecs];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t stride = gridDim.x * kWarps;
    const uint32_t w0 = blockIdx.x * kWarps + warp;
    const int n_elem_vecs = 32 * kElemBytes / 16, n_micro_vecs = 2;  // d2 = 1: one byte per slice
    auto issue = [&](uint32_t wi, int st) {
        if (wi < total) {
            const int64_t row = fastdiv(wi, warps_per_row);
            const int64_t slice0 = (int64_t)(wi - (uint32_t)row * warps_per_row.d) * 32;
            uint8_t* stage = stage_all[warp][st];
            for (int v = lane; v < n_elem_vecs + 2 + n_micro_vecs; v += 32) {
                if (v < n_elem_vecs)
                    cp_async16(stage + v * 16, in.elems + row * in.ld_elems + slice0 * kElemBytes + v * 16);
                else if (v < n_elem_vecs + 2)
                    cp_async16(stage + 32 * kElemBytes + (v - n_elem_vecs) * 16,
                               in.exps + row * in.ld_exps + slice0 + (v - n_elem_vecs) * 16);
                else
                    cp_async16(stage + 32 * kElemBytes + 32 + (v - n_elem_vecs - 2) * 16,
                               in.micro + row * in.ld_micro + slice0 + (v - n_elem_vecs - 2) * 16);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) issue(w0 + s * stride, s);
    int rs = 0;
    for (uint32_t wi = w0; wi < total; wi += stride) {
        issue(wi + (kStages - 1) * stride, (rs + kStages - 1) % kStages);
        cp_async_wait<kStages - 1>();
        __syncwarp();  // the slice a lane decodes was fetched by other lanes
        const uint8_t* stage = stage_all[warp][rs];
        const uint8_t* st_exps = stage + 32 * kElemBytes;
        const uint8_t* st_micro = st_exps + 32;
        rs = (rs + 1) % kStages;
        const int64_t row = fastdiv(wi, warps_per_row);
        const int64_t slice0 = (int64_t)(wi - (uint32_t)row * warps_per_row.d) * 32;
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
        const uint32_t mbits = st_micro[lane];
        uint32_t yb[kSlice];
        decode_slice<W>(words, F, mbits, yb);
        uint4 mine[R::kVecs];
        slice_to_words(yb, mine, (const T*)nullptr);
        R::store_run(out_stage[warp], y + row * ld + slice0 * kSlice, lane, mine);  // 512 contiguous bytes per store instruction
        __syncwarp();  // everyone is done with both stages before they are refilled
    }
}

template <typename T, int W>
static int launch_unpack_row(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                             cudaStream_t st) {
    const int64_t total = rows * (cols / 512);
    if (total >= (1ll << 31) - (1ll << 24)) return BDR_ERR_UNSUPPORTED;
    const int64_t need = (total + kUnpackThreads / 32 - 1) / (kUnpackThreads / 32);
    const int grid = (int)max((int64_t)1, min(need, (int64_t)sm_count() * 8));
    unpack_rowwise_mx_kernel<T, W><<<grid, kUnpackThreads, 0, st>>>(in, y, make_fastdiv((uint32_t)(cols / 512)), (uint32_t)total, ld, qp);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T>
int unpack_rowwise_mx(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                      cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || cols % 512 != 0) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)y % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return launch_unpack_row<T, 3>(in, y, rows, cols, ld, qp, st);
        case 4: return launch_unpack_row<T, 5>(in, y, rows, cols, ld, qp, st);
        case 7: return launch_unpack_row<T, 8>(in, y, rows, cols, ld, qp, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

template int unpack_rowwise_mx<float>(const bdr_planes_t&, float*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);
template int unpack_rowwise_mx<__nv_bfloat16>(const bdr_planes_t&, __nv_bfloat16*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);

}  // namespace bdr
