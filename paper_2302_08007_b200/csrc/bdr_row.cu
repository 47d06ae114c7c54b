// Row-direction (axis 1) kernels: quantize-dequantize with fused Eq. 3 sums for every POW2
// configuration, and the packing fast path for the k1 = 16, k2 = 2 (MX) family.
//
// Thread mapping: one thread owns SPT consecutive 16-element slices of a row (128-bit loads); a
// k1-block wider than a thread's elements is shared by G = k1 / (16*SPT) adjacent lanes, which
// agree on the shared exponent with a shuffle-xor maximum.  Rows are padded to whole blocks so a
// lane group never straddles rows.
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kThreads = 256;

template <typename T, int K2, int K1S, int SPT>
__global__ void __launch_bounds__(kThreads)
quant_rowwise_kernel(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, int64_t units_per_row,
                     int64_t total_units, int group_lanes, QParams qp, bool vec_ok, double* sums) {
    constexpr int kUnit = kSlice * SPT;  // elements per thread per iteration
    double e2 = 0.0, s2 = 0.0;
    // total_units is a multiple of 32, so whole warps iterate together (shuffles need every lane)
    for (int64_t g = (int64_t)blockIdx.x * kThreads + threadIdx.x; g < total_units;
         g += (int64_t)gridDim.x * kThreads) {
        const int64_t row = g / units_per_row;
        const int64_t col0 = (g - row * units_per_row) * kUnit;
        const bool live = row < rows;
        uint32_t u[SPT][kSlice];
        int fj[SPT][kSlice / K2];
        int fb[SPT][kSlice / K1S];
#pragma unroll
        for (int s = 0; s < SPT; ++s) {
            const int64_t c0 = col0 + s * kSlice;
            const int n = live ? (int)max((int64_t)0, min((int64_t)kSlice, cols - c0)) : 0;
            if (n == kSlice && vec_ok) load_slice_vec(x + row * ld + c0, u[s]);
            else load_slice_guarded(x + row * ld + c0, 1, n, u[s]);
            subblock_exponents<K2>(u[s], fj[s]);
#pragma unroll
            for (int b = 0; b < kSlice / K1S; ++b) {
                int f = 0;
#pragma unroll
                for (int j = 0; j < K1S / K2; ++j) f = max(f, fj[s][b * (K1S / K2) + j]);
                fb[s][b] = f;
            }
        }
        if (K1S == kSlice && qp.k1 > kSlice) {  // block spans the thread's slices and maybe lanes
            int F = fb[0][0];
#pragma unroll
            for (int s = 1; s < SPT; ++s) F = max(F, fb[s][0]);
            for (int o = group_lanes >> 1; o > 0; o >>= 1) F = max(F, __shfl_xor_sync(0xFFFFFFFFu, F, o));
#pragma unroll
            for (int s = 0; s < SPT; ++s) fb[s][0] = F;
        }
#pragma unroll
        for (int s = 0; s < SPT; ++s) {
            uint32_t yb[kSlice], code[kSlice], tau[kSlice / K2];
            if (sums) quantize_slice<K2, K1S, true>(u[s], fj[s], fb[s], qp, yb, code, tau, e2, s2);
            else quantize_slice<K2, K1S, false>(u[s], fj[s], fb[s], qp, yb, code, tau, e2, s2);
            if (y) {
                const int64_t c0 = col0 + s * kSlice;
                const int n = live ? (int)max((int64_t)0, min((int64_t)kSlice, cols - c0)) : 0;
                if (n == kSlice && vec_ok) store_slice_vec(y + row * ld + c0, yb);
                else store_slice_guarded(y + row * ld + c0, 1, n, yb);
            }
        }
    }
    if (sums) block_accumulate_sums(e2, s2, sums);
}

// ---- packing fast path: k1 = 16, k2 = 2, code width W = m + 1 -------------------------------------
// One warp handles 32 consecutive slices (512 elements) of one row per iteration.  Each lane
// assembles its slice's 2W bytes of codes in registers, the warp stages them in shared memory and
// writes whole 16-byte vectors, so every plane is written with full-width coalesced stores.
template <typename T, int W>
__global__ void __launch_bounds__(kThreads)
pack_rowwise_mx_kernel(const T* x, T* y_dq, int64_t rows, int64_t cols, int64_t ld, bdr_planes_t out, QParams qp,
                       double* sums) {
    constexpr int kWarps = kThreads / 32;
    constexpr int kElemBytes = 2 * W;                  // per slice
    constexpr int kStage = 32 * kElemBytes + 32 + 96;  // elems | exps | micro (<= 3 bytes per slice)
    __shared__ __align__(16) uint8_t stage_all[kWarps][(kStage + 15) / 16 * 16];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* stage = stage_all[warp];
    uint8_t* st_exps = stage + 32 * kElemBytes;
    uint8_t* st_micro = st_exps + 32;

    const int64_t warps_per_row = cols / 512;
    const int64_t total = rows * warps_per_row;
    double e2 = 0.0, s2 = 0.0;
    for (int64_t wi = (int64_t)blockIdx.x * kWarps + warp; wi < total; wi += (int64_t)gridDim.x * kWarps) {
        const int64_t row = wi / warps_per_row;
        const int64_t slice0 = (wi - row * warps_per_row) * 32;  // first slice of the warp in its row
        const int64_t col = (slice0 + lane) * kSlice;
        uint32_t u[kSlice], yb[kSlice], code[kSlice], tau[kSlice / 2];
        int fj[kSlice / 2], fb[1];
        load_slice_vec(x + row * ld + col, u);
        subblock_exponents<2>(u, fj);
        int F = 0;
#pragma unroll
        for (int j = 0; j < kSlice / 2; ++j) F = max(F, fj[j]);
        fb[0] = F;
        if (sums) quantize_slice<2, kSlice, true>(u, fj, fb, qp, yb, code, tau, e2, s2);
        else quantize_slice<2, kSlice, false>(u, fj, fb, qp, yb, code, tau, e2, s2);
        if (y_dq) store_slice_vec(y_dq + row * ld + col, yb);

        uint32_t words[(kSlice * W + 31) / 32];
        codes_to_words<W>(code, words);
        if (W % 2 == 0 && W % 8 == 0) {  // 16 bytes per slice
            *reinterpret_cast<uint4*>(stage + lane * kElemBytes) = make_uint4(words[0], words[1], words[2], words[3]);
        } else {
            uint16_t* dst = reinterpret_cast<uint16_t*>(stage + lane * kElemBytes);
#pragma unroll
            for (int h = 0; h < W; ++h) dst[h] = (uint16_t)(words[h >> 1] >> ((h & 1) * 16));
        }
        st_exps[lane] = (uint8_t)F;
        uint32_t mbits = 0;
#pragma unroll
        for (int j = 0; j < kSlice / 2; ++j) mbits |= tau[j] << (j * qp.d2);
        for (int b = 0; b < qp.d2; ++b) st_micro[lane * qp.d2 + b] = (uint8_t)(mbits >> (8 * b));
        __syncwarp();
        uint4* g_elems = reinterpret_cast<uint4*>(out.elems + row * out.ld_elems + slice0 * kElemBytes);
        const uint4* s4 = reinterpret_cast<const uint4*>(stage);
        for (int v = lane; v < 32 * kElemBytes / 16; v += 32) g_elems[v] = s4[v];
        if (lane < 2) {
            reinterpret_cast<uint4*>(out.exps + row * out.ld_exps + slice0)[lane] =
                reinterpret_cast<const uint4*>(st_exps)[lane];
        } else if (lane - 2 < 2 * qp.d2) {
            reinterpret_cast<uint4*>(out.micro + row * out.ld_micro + slice0 * qp.d2)[lane - 2] =
                reinterpret_cast<const uint4*>(st_micro)[lane - 2];
        }
        __syncwarp();
    }
    if (sums) block_accumulate_sums(e2, s2, sums);
}

// ---- host launchers --------------------------------------------------------------------------------
static int grid_for(int64_t units, int per_cta) {
    const int64_t need = (units + per_cta - 1) / per_cta;
    const int64_t cap = (int64_t)sm_count() * 8;
    return (int)max((int64_t)1, min(need, cap));
}

template <typename T, int K2, int K1S, int SPT>
static int launch_quant_row(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                            cudaStream_t st) {
    constexpr int kUnit = kSlice * SPT;
    const int64_t padded = (cols + qp.k1 - 1) / qp.k1 * qp.k1;  // whole blocks
    const int64_t upr = (padded + kUnit - 1) / kUnit;
    int64_t total = rows * upr;
    total = (total + 31) / 32 * 32;
    const int group = qp.k1 > kUnit ? qp.k1 / kUnit : 1;
    const bool vec_ok = (((uintptr_t)x | (uintptr_t)y) % 16 == 0) && (ld * sizeof(T)) % 16 == 0;
    if (total == 0) return BDR_OK;
    quant_rowwise_kernel<T, K2, K1S, SPT><<<grid_for(total, kThreads), kThreads, 0, st>>>(
        x, y, rows, cols, ld, upr, total, group, qp, vec_ok, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T, int K1S, int SPT>
static int dispatch_k2(int k2, const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                       double* sums, cudaStream_t st) {
    switch (k2) {
        case 1: return launch_quant_row<T, 1, K1S, SPT>(x, y, rows, cols, ld, qp, sums, st);
        case 2: if constexpr (K1S >= 2) return launch_quant_row<T, 2, K1S, SPT>(x, y, rows, cols, ld, qp, sums, st); break;
        case 4: if constexpr (K1S >= 4) return launch_quant_row<T, 4, K1S, SPT>(x, y, rows, cols, ld, qp, sums, st); break;
        case 8: if constexpr (K1S >= 8) return launch_quant_row<T, 8, K1S, SPT>(x, y, rows, cols, ld, qp, sums, st); break;
        case 16: if constexpr (K1S >= 16) return launch_quant_row<T, 16, K1S, SPT>(x, y, rows, cols, ld, qp, sums, st); break;
    }
    return BDR_ERR_UNSUPPORTED;
}

template <typename T>
int quant_rowwise(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp_in, double* sums,
                  cudaStream_t st) {
    QParams qp = qp_in;
    // d2 = 0: every shift is zero whatever k2 is; use the widest sub-block the slice allows
    int k2 = qp.d2 == 0 ? min(qp.k1, kSlice) : qp.k2;
    if (k2 > kSlice) return BDR_ERR_UNSUPPORTED;  // caller falls back to the general kernel
    qp.k2 = k2;
    switch (qp.k1) {
        case 1: return dispatch_k2<T, 1, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 2: return dispatch_k2<T, 2, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 4: return dispatch_k2<T, 4, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 8: return dispatch_k2<T, 8, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
        case 1024: return dispatch_k2<T, 16, 2>(k2, x, y, rows, cols, ld, qp, sums, st);
        default: return dispatch_k2<T, 16, 1>(k2, x, y, rows, cols, ld, qp, sums, st);  // 16 .. 512
    }
}

template <typename T, int W>
static int launch_pack_row(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                           const QParams& qp, double* sums, cudaStream_t st) {
    const int64_t total = rows * (cols / 512);
    if (total == 0) return BDR_OK;
    pack_rowwise_mx_kernel<T, W><<<grid_for(total, kThreads / 32), kThreads, 0, st>>>(x, y, rows, cols, ld, out, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Returns BDR_ERR_UNSUPPORTED when the shape / configuration is outside the fast path.
template <typename T>
int pack_rowwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                    const QParams& qp, double* sums, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || cols % 512 != 0) return BDR_ERR_UNSUPPORTED;
    if ((((uintptr_t)x | (uintptr_t)y) % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    switch (qp.m + 1) {
        case 2: return launch_pack_row<T, 2>(x, y, rows, cols, ld, out, qp, sums, st);
        case 3: return launch_pack_row<T, 3>(x, y, rows, cols, ld, out, qp, sums, st);
        case 4: return launch_pack_row<T, 4>(x, y, rows, cols, ld, out, qp, sums, st);
        case 5: return launch_pack_row<T, 5>(x, y, rows, cols, ld, out, qp, sums, st);
        case 6: return launch_pack_row<T, 6>(x, y, rows, cols, ld, out, qp, sums, st);
        case 7: return launch_pack_row<T, 7>(x, y, rows, cols, ld, out, qp, sums, st);
        case 8: return launch_pack_row<T, 8>(x, y, rows, cols, ld, out, qp, sums, st);
        case 9: return launch_pack_row<T, 9>(x, y, rows, cols, ld, out, qp, sums, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

template int quant_rowwise<float>(const float*, float*, int64_t, int64_t, int64_t, const QParams&, double*, cudaStream_t);
template int quant_rowwise<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, int64_t, int64_t, int64_t,
                                          const QParams&, double*, cudaStream_t);
template int pack_rowwise_mx<float>(const float*, float*, int64_t, int64_t, int64_t, const bdr_planes_t&,
                                    const QParams&, double*, cudaStream_t);
template int pack_rowwise_mx<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, int64_t, int64_t, int64_t,
                                            const bdr_planes_t&, const QParams&, double*, cudaStream_t);

}  // namespace bdr
