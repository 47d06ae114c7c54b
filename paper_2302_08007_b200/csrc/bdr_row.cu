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

constexpr int kThreads = kRowThreads;

// Quantize the SPT slices a thread holds (shared exponents across lanes when k1 spans them).
template <int K2, int K1S, int SPT, bool SUMS, bool YOUT>
__device__ __forceinline__ void quantize_unit(const uint32_t (&u)[SPT][kSlice], const QParams& qp, int group_lanes,
                                              uint32_t (&yb)[SPT][kSlice], double& e2, double& s2) {
    uint32_t fj[SPT][kSlice / K2];
    uint32_t fb[SPT][kSlice / K1S];
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
        subblock_exponents<K2>(u[s], fj[s]);
#pragma unroll
        for (int b = 0; b < kSlice / K1S; ++b) {
            uint32_t f = 0;
#pragma unroll
            for (int j = 0; j < K1S / K2; ++j) f = max(f, fj[s][b * (K1S / K2) + j]);
            fb[s][b] = f;
        }
    }
    if (K1S == kSlice && qp.k1 > kSlice) {  // block spans the thread's slices and maybe lanes
        uint32_t F = fb[0][0];
#pragma unroll
        for (int s = 1; s < SPT; ++s) F = max(F, fb[s][0]);
        for (int o = group_lanes >> 1; o > 0; o >>= 1) F = max(F, __shfl_xor_sync(0xFFFFFFFFu, F, o));
#pragma unroll
        for (int s = 0; s < SPT; ++s) fb[s][0] = F;
    }
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
        uint32_t rq[kSlice], cb[kSlice / K2], tau[kSlice / K2];
        quantize_slice<K2, K1S, SUMS, YOUT, false>(u[s], fj[s], fb[s], qp, yb[s], rq, cb, tau, e2, s2);
    }
}

template <typename T, int K2, int K1S, int SPT, bool SUMS, bool YOUT>
__global__ void __launch_bounds__(kThreads)
quant_rowwise_kernel(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, FastDiv units_per_row,
                     uint32_t total_units, int group_lanes, QParams qp, bool vec_ok, bool all_full, double* sums) {
    constexpr int kUnit = kSlice * SPT;  // elements per thread per iteration
    constexpr int kVecs = Ring<T, SPT>::kVecs, kStages = Ring<T, SPT>::kStages;
    extern __shared__ __align__(16) uint4 ring[];  // [stage][warp][32*kVecs words]
    double e2 = 0.0, s2 = 0.0;
    const uint32_t stride = gridDim.x * kThreads;
    const uint32_t g0 = blockIdx.x * kThreads + threadIdx.x;
    // total_units is a multiple of 32, so whole warps iterate together (shuffles need every lane)
    if (all_full) {
        // every unit is a full, 16-byte aligned run of the tensor and a warp's 32 units are contiguous
        // (units_per_row % 32 == 0): feed them through the prefetch ring
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const uint32_t gw0 = g0 - lane;  // the warp's first unit
        auto stage_ptr = [&](int stage) { return ring + ((size_t)stage * (kThreads / 32) + warp) * 32 * kVecs; };
        auto issue = [&](uint32_t gw, int stage) {
            if (gw < total_units) {
                const uint32_t row = fastdiv(gw, units_per_row);
                Ring<T, SPT>::issue(stage_ptr(stage), x + (int64_t)row * ld + (int64_t)(gw - row * units_per_row.d) * kUnit, lane);
            }
            cp_async_commit();
        };
#pragma unroll
        for (int s = 0; s < kStages - 1; ++s) issue(gw0 + s * stride, s);
        int stage = 0;
        for (uint32_t g = g0; g < total_units; g += stride) {
            __syncwarp();  // all lanes are done with the stage that is refilled next
            issue(g - lane + (kStages - 1) * stride, (stage + kStages - 1) % kStages);
            cp_async_wait<kStages - 1>();
            __syncwarp();  // a lane's words were fetched by other lanes
            uint32_t u[SPT][kSlice], yb[SPT][kSlice];
#pragma unroll
            for (int s = 0; s < SPT; ++s) {
                uint4 w[SliceWords<T>::kVecs];
#pragma unroll
                for (int v = 0; v < SliceWords<T>::kVecs; ++v)
                    w[v] = Ring<T, SPT>::read(stage_ptr(stage), lane, s * SliceWords<T>::kVecs + v);
                SliceWords<T>::expand(w, u[s]);
            }
            quantize_unit<K2, K1S, SPT, SUMS, YOUT>(u, qp, group_lanes, yb, e2, s2);
            if (YOUT) {
                const uint32_t gw = g - lane;  // the warp's first unit: its 32 units are one contiguous run
                const uint32_t row = fastdiv(gw, units_per_row);
                T* dst = y + (int64_t)row * ld + (int64_t)(gw - row * units_per_row.d) * kUnit;
                uint4 mine[kVecs];
#pragma unroll
                for (int s = 0; s < SPT; ++s) {
                    uint4 w[SliceWords<T>::kVecs];
                    slice_to_words(yb[s], w, (const T*)nullptr);
#pragma unroll
                    for (int v = 0; v < SliceWords<T>::kVecs; ++v) mine[s * SliceWords<T>::kVecs + v] = w[v];
                }
                __syncwarp();  // every lane has read its input words from this stage
                Ring<T, SPT>::store_run(stage_ptr(stage), dst, lane, mine);
            }
            stage = (stage + 1) % kStages;
        }
    } else {
        for (uint32_t g = g0; g < total_units; g += stride) {
            const int64_t row = fastdiv(g, units_per_row);
            const int64_t col0 = (int64_t)(g - (uint32_t)row * units_per_row.d) * kUnit;
            const bool live = row < rows;
            uint32_t u[SPT][kSlice], yb[SPT][kSlice];
#pragma unroll
            for (int s = 0; s < SPT; ++s) {
                const int64_t c0 = col0 + s * kSlice;
                const int n = live ? (int)max((int64_t)0, min((int64_t)kSlice, cols - c0)) : 0;
                if (n == kSlice && vec_ok) load_slice_vec(x + row * ld + c0, u[s]);
                else load_slice_guarded(x + row * ld + c0, 1, n, u[s]);
            }
            quantize_unit<K2, K1S, SPT, SUMS, YOUT>(u, qp, group_lanes, yb, e2, s2);
            if (YOUT) {
#pragma unroll
                for (int s = 0; s < SPT; ++s) {
                    const int64_t c0 = col0 + s * kSlice;
                    const int n = live ? (int)max((int64_t)0, min((int64_t)kSlice, cols - c0)) : 0;
                    if (n == kSlice && vec_ok) store_slice_vec(y + row * ld + c0, yb[s]);
                    else store_slice_guarded(y + row * ld + c0, 1, n, yb[s]);
                }
            }
        }
    }
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

// ---- packing fast path: k1 = 16, k2 = 2, code width W = m + 1 -------------------------------------
// One warp handles 64 consecutive slices (1024 elements) per iteration, two adjacent slices per
// lane; the input comes through the prefetch ring.  A lane's 32 codes are exactly W 32-bit words,
// which it assembles in registers; the warp stages them in shared memory and writes whole
// 16-byte vectors, so every plane is written with full-width coalesced stores.
constexpr int kPackSPT = 2;
template <int W> struct PackStage {
    static constexpr int kElemBytes = 32 * kPackSPT * 2 * W;  // per warp iteration
    static constexpr int kExpBytes = 32 * kPackSPT;
    static constexpr int kMicroBytes = 32 * kPackSPT;         // d2 = 1: one byte per slice
    static constexpr int kBytes = kElemBytes + kExpBytes + kMicroBytes;  // a multiple of 16
};

template <typename T, int W, bool SUMS, bool YDQ>
__global__ void __launch_bounds__(kThreads)
pack_rowwise_mx_kernel(const T* x, T* y_dq, FastDiv warps_per_row, uint32_t total, int64_t ld, bdr_planes_t out,
                       QParams qp, double* sums) {
    constexpr int kWarps = kThreads / 32;
    using R = Ring<T, kPackSPT>;
    constexpr int kVecs = R::kVecs, kStages = R::kStages, kSV = SliceWords<T>::kVecs;
    constexpr int kWarpElems = 32 * kPackSPT * kSlice;  // 1024
    extern __shared__ __align__(16) uint4 ring[];  // [stage][warp][32*kVecs words], then the per-warp staging
    uint8_t* stage_base = reinterpret_cast<uint8_t*>(ring + kStages * kVecs * kThreads);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* stage = stage_base + warp * PackStage<W>::kBytes;
    uint8_t* st_exps = stage + PackStage<W>::kElemBytes;
    uint8_t* st_micro = st_exps + PackStage<W>::kExpBytes;

    const uint32_t stride = gridDim.x * kWarps;
    const uint32_t w0 = blockIdx.x * kWarps + warp;
    auto stage_ptr = [&](int st) { return ring + ((size_t)st * kWarps + warp) * 32 * kVecs; };
    auto issue = [&](uint32_t wi, int st) {
        if (wi < total) {
            const uint32_t row = fastdiv(wi, warps_per_row);
            R::issue(stage_ptr(st), x + (int64_t)row * ld + (int64_t)(wi - row * warps_per_row.d) * kWarpElems, lane);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) issue(w0 + s * stride, s);
    int rs = 0;
    double e2 = 0.0, s2 = 0.0;
    for (uint32_t wi = w0; wi < total; wi += stride) {
        issue(wi + (kStages - 1) * stride, (rs + kStages - 1) % kStages);  // trailing __syncwarp below covers reuse
        cp_async_wait<kStages - 1>();
        __syncwarp();  // a lane's words were fetched by other lanes
        const int64_t row = fastdiv(wi, warps_per_row);
        const int64_t slice0 = (int64_t)(wi - (uint32_t)row * warps_per_row.d) * (32 * kPackSPT);  // warp's first slice in its row
        uint4 ymine[YDQ ? kVecs : 1];
#pragma unroll
        for (int s = 0; s < kPackSPT; ++s) {  // one slice at a time keeps the live register set small
            uint32_t u[kSlice], yb[kSlice], rq[kSlice], cb[kSlice / 2], tau[kSlice / 2];
            uint32_t fj[kSlice / 2], fb[1];
            uint4 w[kSV];
#pragma unroll
            for (int v = 0; v < kSV; ++v) w[v] = R::read(stage_ptr(rs), lane, s * kSV + v);
            SliceWords<T>::expand(w, u);
            subblock_exponents<2>(u, fj);
            uint32_t F = 0;
#pragma unroll
            for (int j = 0; j < kSlice / 2; ++j) F = max(F, fj[j]);
            fb[0] = F;
            quantize_slice<2, kSlice, SUMS, YDQ, true>(u, fj, fb, qp, yb, rq, cb, tau, e2, s2);
            if (YDQ) {
                uint4 wy[kSV];
                slice_to_words(yb, wy, (const T*)nullptr);
#pragma unroll
                for (int v = 0; v < kSV; ++v) ymine[s * kSV + v] = wy[v];
            }
            uint32_t words[(kSlice * W + 31) / 32];
            pack_words<W, kSlice, 2>(u, rq, cb, words);
            const int sl = kPackSPT * lane + s;  // slice index within the warp's run
            if (W % 2 == 0) {
                uint32_t* dst = reinterpret_cast<uint32_t*>(stage + sl * 2 * W);
#pragma unroll
                for (int h = 0; h < W / 2; ++h) dst[h] = words[h];
            } else {
                uint16_t* dst = reinterpret_cast<uint16_t*>(stage + sl * 2 * W);
#pragma unroll
                for (int h = 0; h < W; ++h) dst[h] = (uint16_t)(words[h >> 1] >> ((h & 1) * 16));
            }
            st_exps[sl] = (uint8_t)(F >> 23);
            uint32_t mb = 0;  // d2 = 1: one bit per sub-block
#pragma unroll
            for (int j = 0; j < kSlice / 2; ++j) mb |= tau[j] << j;
            st_micro[sl] = (uint8_t)mb;
        }
        if (YDQ) {
            __syncwarp();  // every lane has read its input words from this stage
            R::store_run(stage_ptr(rs), y_dq + row * ld + slice0 * kSlice, lane, reinterpret_cast<const uint4(&)[kVecs]>(ymine));
        }
        rs = (rs + 1) % kStages;
        __syncwarp();
        uint4* g_elems = reinterpret_cast<uint4*>(out.elems + row * out.ld_elems + slice0 * 2 * W);
        const uint4* s4 = reinterpret_cast<const uint4*>(stage);
        for (int v = lane; v < PackStage<W>::kElemBytes / 16; v += 32) g_elems[v] = s4[v];
        constexpr int n_exp_vecs = PackStage<W>::kExpBytes / 16, n_micro_vecs = 32 * kPackSPT / 16;
        if (lane < n_exp_vecs) {
            reinterpret_cast<uint4*>(out.exps + row * out.ld_exps + slice0)[lane] =
                reinterpret_cast<const uint4*>(st_exps)[lane];
        } else if (lane - n_exp_vecs < n_micro_vecs) {
            reinterpret_cast<uint4*>(out.micro + row * out.ld_micro + slice0)[lane - n_exp_vecs] =
                reinterpret_cast<const uint4*>(st_micro)[lane - n_exp_vecs];
        }
        __syncwarp();
    }
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

// ---- host launchers --------------------------------------------------------------------------------
static int grid_for(int64_t units, int per_cta) {
    const int64_t need = (units + per_cta - 1) / per_cta;
    const int64_t cap = (int64_t)sm_count() * 8;
    return (int)max((int64_t)1, min(need, cap));
}

template <typename T, int K2, int K1S, int SPT, bool SUMS, bool YOUT>
static int launch_quant_row_flags(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                                  cudaStream_t st) {
    constexpr int kUnit = kSlice * SPT;
    if (ld == cols && cols % qp.k1 == 0) {  // contiguous tensor of whole blocks: one long row, no row arithmetic
        cols *= rows;
        ld = cols;
        rows = 1;
    }
    const int64_t padded = (cols + qp.k1 - 1) / qp.k1 * qp.k1;  // whole blocks
    const int64_t upr = (padded + kUnit - 1) / kUnit;
    int64_t total = rows * upr;
    total = (total + 31) / 32 * 32;
    const int group = qp.k1 > kUnit ? qp.k1 / kUnit : 1;
    const bool vec_ok = (((uintptr_t)x | (uintptr_t)y) % 16 == 0) && (ld * sizeof(T)) % 16 == 0;
    const bool all_full = vec_ok && padded == cols && cols % kUnit == 0 && upr % 32 == 0;
    if (total == 0) return BDR_OK;
    if (total >= (1ll << 31) - (1ll << 24)) return BDR_ERR_UNSUPPORTED;  // 32-bit unit indices (incl. prefetch look-ahead)
    auto kern = quant_rowwise_kernel<T, K2, K1S, SPT, SUMS, YOUT>;
    const size_t smem = Ring<T, SPT>::kBytes;
    static PerDevice once;  // per instantiation
    if (kernel_setup(once, kern, kThreads, smem) < 1) return BDR_ERR_CUDA;
    kern<<<grid_for(total, kThreads), kThreads, smem, st>>>(x, y, rows, cols, ld, make_fastdiv((uint32_t)upr), (uint32_t)total, group, qp,
                                                            vec_ok, all_full, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T, int K2, int K1S, int SPT>
static int launch_quant_row(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                            cudaStream_t st) {
    if (sums) return y ? launch_quant_row_flags<T, K2, K1S, SPT, true, true>(x, y, rows, cols, ld, qp, sums, st)
                       : launch_quant_row_flags<T, K2, K1S, SPT, true, false>(x, y, rows, cols, ld, qp, sums, st);
    return launch_quant_row_flags<T, K2, K1S, SPT, false, true>(x, y, rows, cols, ld, qp, sums, st);
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
        default:  // 16 .. 512; two slices per thread for 2-byte elements (64 bytes per thread either way)
            if (sizeof(T) == 2 && cols % 32 == 0) return dispatch_k2<T, 16, 2>(k2, x, y, rows, cols, ld, qp, sums, st);
            return dispatch_k2<T, 16, 1>(k2, x, y, rows, cols, ld, qp, sums, st);
    }
}

template <typename T, int W, bool SUMS, bool YDQ>
static int launch_pack_row(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                           const QParams& qp, double* sums, cudaStream_t st) {
    if (ld == cols) {  // contiguous tensor, tight planes: one long row
        cols *= rows;
        ld = cols;
        rows = 1;
    }
    const int64_t total = rows * (cols / 1024);
    if (total == 0) return BDR_OK;
    if (total >= (1ll << 31) - (1ll << 24)) return BDR_ERR_UNSUPPORTED;
    auto kern = pack_rowwise_mx_kernel<T, W, SUMS, YDQ>;
    const size_t smem = Ring<T, kPackSPT>::kBytes + (kThreads / 32) * PackStage<W>::kBytes;
    static PerDevice once;  // per instantiation
    if (kernel_setup(once, kern, kThreads, smem) < 1) return BDR_ERR_CUDA;
    kern<<<grid_for(total, kThreads / 32), kThreads, smem, st>>>(x, y, make_fastdiv((uint32_t)(cols / 1024)), (uint32_t)total, ld, out, qp, sums);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <typename T, int W>
static int pack_row_flags(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                          const QParams& qp, double* sums, cudaStream_t st) {
    if (sums) return y ? launch_pack_row<T, W, true, true>(x, y, rows, cols, ld, out, qp, sums, st)
                       : launch_pack_row<T, W, true, false>(x, y, rows, cols, ld, out, qp, sums, st);
    return y ? launch_pack_row<T, W, false, true>(x, y, rows, cols, ld, out, qp, sums, st)
             : launch_pack_row<T, W, false, false>(x, y, rows, cols, ld, out, qp, sums, st);
}

// Fast path for the Table II family (k1 = 16, k2 = 2, d2 = 1; m = 2, 4, 7).  Returns
// BDR_ERR_UNSUPPORTED for every other configuration or shape (the general kernel covers those).
template <typename T>
int pack_rowwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                    const QParams& qp, double* sums, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1) return BDR_ERR_UNSUPPORTED;
    if (ld == cols ? (rows * cols) % 1024 != 0 || cols % 16 != 0 : cols % 1024 != 0) return BDR_ERR_UNSUPPORTED;
    if ((((uintptr_t)x | (uintptr_t)y) % 16) || (ld * sizeof(T)) % 16) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return pack_row_flags<T, 3>(x, y, rows, cols, ld, out, qp, sums, st);
        case 4: return pack_row_flags<T, 5>(x, y, rows, cols, ld, out, qp, sums, st);
        case 7: return pack_row_flags<T, 8>(x, y, rows, cols, ld, out, qp, sums, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

#ifndef BDR_ROW_DTYPE
#define BDR_ROW_DTYPE float
#endif
template int quant_rowwise<BDR_ROW_DTYPE>(const BDR_ROW_DTYPE*, BDR_ROW_DTYPE*, int64_t, int64_t, int64_t, const QParams&, double*,
                                          cudaStream_t);
template int pack_rowwise_mx<BDR_ROW_DTYPE>(const BDR_ROW_DTYPE*, BDR_ROW_DTYPE*, int64_t, int64_t, int64_t, const bdr_planes_t&,
                                            const QParams&, double*, cudaStream_t);

}  // namespace bdr
