// Column-direction (axis 0) fast paths for the k1 = 16, k2 = 2 family: blocks run down the strided
// dimension, and the packed planes come out in the transposed (column-major, reduction-contiguous)
// layout that the backward-pass GEMMs consume (Section V: "transpose, then quantize").
//
// A CTA owns a tile of 64 columns x 32 row-blocks (512 rows).  Each warp takes one 16-row block at a
// time; a lane owns two adjacent columns, so every row access of the warp is one contiguous,
// fully coalesced segment.  The lane's codes are staged in shared memory as [row-block][column]
// items; the CTA then gathers them per column and writes each column's 32 row-blocks as one
// contiguous run of 64*W bytes (and 32 exponent bytes, 32*d2 microexponent bytes), so the transposed
// planes are written with whole 16-byte vectors and whole 32-byte sectors.
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kColThreads = 256;
constexpr int kColWarps = kColThreads / 32;
constexpr int kTileCols = 64;
constexpr int kTileBlocks = 32;  // 16-row blocks per tile

// two adjacent columns of one row, as fp32 bit patterns
__device__ __forceinline__ void load_pair(const float* p, uint32_t& a, uint32_t& b) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    a = v.x; b = v.y;
}
__device__ __forceinline__ void load_pair(const __nv_bfloat16* p, uint32_t& a, uint32_t& b) {
    const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(p));
    a = v << 16; b = v & 0xFFFF0000u;
}
__device__ __forceinline__ void store_pair(float* p, uint32_t a, uint32_t b) {
    *reinterpret_cast<uint2*>(p) = make_uint2(a, b);
}
__device__ __forceinline__ void store_pair(__nv_bfloat16* p, uint32_t a, uint32_t b) {
    *reinterpret_cast<uint32_t*>(p) = (a >> 16) | (b & 0xFFFF0000u);
}

template <int W>
struct ColStage {
    static constexpr int kW = W > 0 ? W : 1;
    uint16_t elems[kTileBlocks][kTileCols][kW];  // 2W bytes per (row-block, column)
    uint8_t exps[kTileBlocks][kTileCols];
    uint8_t micro[kTileBlocks][kTileCols][3];
};

// one row's pair of columns as fetched (4 bytes of bf16, 8 bytes of fp32)
template <typename T> struct PairWord;
template <> struct PairWord<float> {
    using type = uint2;
    __device__ static __forceinline__ void fetch(type* smem, const float* g) { cp_async8(smem, g); }
    __device__ static __forceinline__ void split(type w, uint32_t& a, uint32_t& b) { a = w.x; b = w.y; }
};
template <> struct PairWord<__nv_bfloat16> {
    using type = uint32_t;
    __device__ static __forceinline__ void fetch(type* smem, const __nv_bfloat16* g) { cp_async4(smem, g); }
    __device__ static __forceinline__ void split(type w, uint32_t& a, uint32_t& b) { a = w << 16; b = w & 0xFFFF0000u; }
};
template <typename T> struct ColRing {
    static constexpr int kStages = sizeof(T) == 2 ? 3 : 2;
    static constexpr size_t kBytes = (size_t)kStages * kSlice * kColThreads * sizeof(typename PairWord<T>::type);
};

template <typename T, int W, bool SUMS, bool YOUT>  // W = m + 1 when packing, 0 when only y / sums are wanted
__global__ void __launch_bounds__(kColThreads, 2)
quant_colwise_mx_kernel(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, bdr_planes_t out, QParams qp,
                        double* sums) {
    using PW = typename PairWord<T>::type;
    constexpr int kStages = ColRing<T>::kStages;
    extern __shared__ __align__(16) uint8_t dyn_smem[];
    PW* ring = reinterpret_cast<PW*>(dyn_smem);  // [stage][row of the block][thread]
    ColStage<W>& st = *reinterpret_cast<ColStage<W>*>(dyn_smem + ColRing<T>::kBytes);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kTileCols;
    const int64_t tb0 = (int64_t)blockIdx.y * kTileBlocks;
    const int64_t nblocks = rows / kSlice;
    const int64_t c = c0 + 2 * lane;
    double e2 = 0.0, s2 = 0.0;
    auto issue = [&](int bl, int stg) {
        if (bl < kTileBlocks && tb0 + bl < nblocks) {
            const T* px = x + (tb0 + bl) * kSlice * ld + c;
#pragma unroll
            for (int r = 0; r < kSlice; ++r) PairWord<T>::fetch(&ring[(stg * kSlice + r) * kColThreads + threadIdx.x], px + r * ld);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) issue(warp + s * kColWarps, s);
    int rs = 0;
    for (int bl = warp; bl < kTileBlocks; bl += kColWarps) {
        const int64_t b = tb0 + bl;
        if (b >= nblocks) break;
        issue(bl + (kStages - 1) * kColWarps, (rs + kStages - 1) % kStages);
        cp_async_wait<kStages - 1>();
        uint32_t u[2][kSlice];
#pragma unroll
        for (int r = 0; r < kSlice; ++r)
            PairWord<T>::split(ring[(rs * kSlice + r) * kColThreads + threadIdx.x], u[0][r], u[1][r]);
        rs = (rs + 1) % kStages;
        uint32_t yb[2][kSlice];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t rq[kSlice], cb[kSlice / 2], tau[kSlice / 2];
            uint32_t fj[kSlice / 2], fb[1];
            subblock_exponents<2>(u[h], fj);
            uint32_t F = 0;
#pragma unroll
            for (int j = 0; j < kSlice / 2; ++j) F = max(F, fj[j]);
            fb[0] = F;
            quantize_slice<2, kSlice, SUMS, YOUT, (W > 0)>(u[h], fj, fb, qp, yb[h], rq, cb, tau, e2, s2);
            if (W > 0) {
                uint32_t words[(kSlice * ColStage<W>::kW + 31) / 32];
                pack_words<ColStage<W>::kW, kSlice, 2>(u[h], rq, cb, words);
#pragma unroll
                for (int k = 0; k < ColStage<W>::kW; ++k)
                    st.elems[bl][2 * lane + h][k] = (uint16_t)(words[k >> 1] >> ((k & 1) * 16));
                st.exps[bl][2 * lane + h] = (uint8_t)(F >> 23);
                uint32_t mbits = 0;  // d2 = 1
#pragma unroll
                for (int j = 0; j < kSlice / 2; ++j) mbits |= tau[j] << j;
                st.micro[bl][2 * lane + h][0] = (uint8_t)mbits;
            }
        }
        if (YOUT) {
            T* py = y + b * kSlice * ld + c;
#pragma unroll
            for (int r = 0; r < kSlice; ++r) store_pair(py + r * ld, yb[0][r], yb[1][r]);
        }
    }
    if (W > 0) {
        constexpr int kW = ColStage<W>::kW;
        __syncthreads();
        // elems: each column's run is kTileBlocks * 2W = 64W bytes = 4W vectors of 16 bytes
        for (int idx = threadIdx.x; idx < kTileCols * 4 * kW; idx += kColThreads) {
            const int ci = idx % kTileCols, v = idx / kTileCols;
            uint32_t w4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int h0 = 8 * v + 2 * i, h1 = h0 + 1;
                w4[i] = (uint32_t)st.elems[h0 / kW][ci][h0 % kW] | ((uint32_t)st.elems[h1 / kW][ci][h1 % kW] << 16);
            }
            *reinterpret_cast<uint4*>(out.elems + (c0 + ci) * out.ld_elems + tb0 * 2 * kW + v * 16) =
                make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        // exps: 32 bytes per column; micro: 32*d2 bytes per column
        for (int idx = threadIdx.x; idx < kTileCols * 2; idx += kColThreads) {
            const int ci = idx % kTileCols, v = idx / kTileCols;
            uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 16; ++i) w4[i >> 2] |= (uint32_t)st.exps[16 * v + i][ci] << ((i & 3) * 8);
            *reinterpret_cast<uint4*>(out.exps + (c0 + ci) * out.ld_exps + tb0 + v * 16) =
                make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        for (int idx = threadIdx.x; idx < kTileCols * 2; idx += kColThreads) {  // d2 = 1
            const int ci = idx % kTileCols, v = idx / kTileCols;
            uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 16; ++i) w4[i >> 2] |= (uint32_t)st.micro[16 * v + i][ci][0] << ((i & 3) * 8);
            *reinterpret_cast<uint4*>(out.micro + (c0 + ci) * out.ld_micro + tb0 + v * 16) =
                make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
    }
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

// Mirror image: gather each column's packed run with coalesced 16-byte loads, scatter it into
// [row-block][column] items in shared memory, then decode with lanes on adjacent column pairs.
template <typename T, int W>
__global__ void __launch_bounds__(kColThreads)
unpack_colwise_mx_kernel(bdr_planes_t in, T* y, int64_t rows, int64_t cols, int64_t ld, QParams qp) {
    __shared__ __align__(16) ColStage<W> st;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kTileCols;
    const int64_t tb0 = (int64_t)blockIdx.y * kTileBlocks;
    for (int idx = threadIdx.x; idx < kTileCols * 4 * W; idx += kColThreads) {
        const int v = idx % (4 * W), ci = idx / (4 * W);  // consecutive threads walk one column's run
        const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(in.elems + (c0 + ci) * in.ld_elems + tb0 * 2 * W + v * 16));
        const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int h = 8 * v + i;
            st.elems[h / W][ci][h % W] = (uint16_t)(w4[i >> 1] >> ((i & 1) * 16));
        }
    }
    for (int idx = threadIdx.x; idx < kTileCols * 2; idx += kColThreads) {
        const int v = idx % 2, ci = idx / 2;
        const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(in.exps + (c0 + ci) * in.ld_exps + tb0 + v * 16));
        const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
        for (int i = 0; i < 16; ++i) st.exps[16 * v + i][ci] = (uint8_t)(w4[i >> 2] >> ((i & 3) * 8));
    }
    for (int idx = threadIdx.x; idx < kTileCols * 2; idx += kColThreads) {
        const int v = idx % 2, ci = idx / 2;
        const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(in.micro + (c0 + ci) * in.ld_micro + tb0 + v * 16));
        const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int t = 16 * v + i;
            st.micro[t][ci][0] = (uint8_t)(w4[i >> 2] >> ((i & 3) * 8));
        }
    }
    __syncthreads();
    const int64_t c = c0 + 2 * lane;
    for (int bl = warp; bl < kTileBlocks; bl += kColWarps) {
        const int64_t b = tb0 + bl;
        uint32_t yb[2][kSlice];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t words[(kSlice * W + 31) / 32 + 1];
#pragma unroll
            for (int i = 0; i < (kSlice * W + 31) / 32 + 1; ++i) words[i] = 0;
#pragma unroll
            for (int k = 0; k < W; ++k) words[k >> 1] |= (uint32_t)st.elems[bl][2 * lane + h][k] << ((k & 1) * 16);
            const uint32_t mbits = st.micro[bl][2 * lane + h][0];
            decode_slice<W>(words, st.exps[bl][2 * lane + h], mbits, yb[h]);
        }
        T* py = y + b * kSlice * ld + c;
#pragma unroll
        for (int r = 0; r < kSlice; ++r) store_pair(py + r * ld, yb[0][r], yb[1][r]);
    }
}

template <typename T, int W, bool SUMS, bool YOUT>
static int launch_col(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                      const QParams& qp, double* sums, cudaStream_t st) {
    const dim3 grid((unsigned)(cols / kTileCols), (unsigned)((rows / kSlice + kTileBlocks - 1) / kTileBlocks));
    bdr_planes_t pl = {};
    if (out) pl = *out;
    auto kern = quant_colwise_mx_kernel<T, W, SUMS, YOUT>;
    const size_t smem = ColRing<T>::kBytes + (W > 0 ? sizeof(ColStage<W>) : 16);
    static PerDevice once;  // per instantiation
    if (kernel_setup(once, kern, kColThreads, smem) < 1) return BDR_ERR_CUDA;
    kern<<<grid, kColThreads, smem, st>>>(x, y, rows, cols, ld, pl, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T, int W>
static int col_flags(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                     const QParams& qp, double* sums, cudaStream_t st) {
    if (sums) return y ? launch_col<T, W, true, true>(x, y, rows, cols, ld, out, qp, sums, st)
                       : launch_col<T, W, true, false>(x, y, rows, cols, ld, out, qp, sums, st);
    if (y) return launch_col<T, W, false, true>(x, y, rows, cols, ld, out, qp, sums, st);
    if constexpr (W > 0) return launch_col<T, W, false, false>(x, y, rows, cols, ld, out, qp, sums, st);
    return BDR_ERR_NULL;
}

// Fast path for the Table II family (k1 = 16, k2 = 2, d2 = 1; packing: m = 2, 4, 7).
template <typename T>
int quant_colwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                     const QParams& qp, double* sums, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || cols % kTileCols != 0 || rows % kSlice != 0) return BDR_ERR_UNSUPPORTED;
    if (out && rows % (kSlice * kTileBlocks) != 0) return BDR_ERR_UNSUPPORTED;
    if ((((uintptr_t)x | (uintptr_t)y) % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    if (rows / kSlice / kTileBlocks > 65535) return BDR_ERR_UNSUPPORTED;
    if (!out) return col_flags<T, 0>(x, y, rows, cols, ld, out, qp, sums, st);
    switch (qp.m) {
        case 2: return col_flags<T, 3>(x, y, rows, cols, ld, out, qp, sums, st);
        case 4: return col_flags<T, 5>(x, y, rows, cols, ld, out, qp, sums, st);
        case 7: return col_flags<T, 8>(x, y, rows, cols, ld, out, qp, sums, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

template <typename T, int W>
static int launch_unpack_col(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                             cudaStream_t st) {
    const dim3 grid((unsigned)(cols / kTileCols), (unsigned)(rows / (kSlice * kTileBlocks)));
    unpack_colwise_mx_kernel<T, W><<<grid, kColThreads, 0, st>>>(in, y, rows, cols, ld, qp);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T>
int unpack_colwise_mx(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                      cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || cols % kTileCols != 0 || rows % (kSlice * kTileBlocks) != 0)
        return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)y % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    if (rows / (kSlice * kTileBlocks) > 65535) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return launch_unpack_col<T, 3>(in, y, rows, cols, ld, qp, st);
        case 4: return launch_unpack_col<T, 5>(in, y, rows, cols, ld, qp, st);
        case 7: return launch_unpack_col<T, 8>(in, y, rows, cols, ld, qp, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

template int quant_colwise_mx<float>(const float*, float*, int64_t, int64_t, int64_t, const bdr_planes_t*, const QParams&, double*, cudaStream_t);
template int quant_colwise_mx<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, int64_t, int64_t, int64_t, const bdr_planes_t*, const QParams&, double*, cudaStream_t);
template int unpack_colwise_mx<float>(const bdr_planes_t&, float*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);
template int unpack_colwise_mx<__nv_bfloat16>(const bdr_planes_t&, __nv_bfloat16*, int64_t, int64_t, int64_t, const QParams&, cudaStream_t);

}  // namespace bdr
