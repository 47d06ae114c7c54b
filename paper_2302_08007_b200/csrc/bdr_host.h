// Host-side declarations shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "bdr.h"

namespace bdr {

struct QParams;

int sm_count();  // SMs of the current device (cached per device)

constexpr int kMaxDevices = 64;

// A positive integer remembered per device by one call site (a zero-initialised static object).
// cudaFuncSetAttribute and the occupancy query apply to the device that is current, so the launchers keep
// one of these per kernel instantiation: the set-up runs the first time each device launches the kernel,
// not the first time the process does.  The set-up is idempotent, so two threads that race on the first
// call of a device both run it and store the same value.
class PerDevice {
    std::atomic<int> v_[kMaxDevices];

   public:
    // value remembered for `dev`, running `setup` (returns > 0, or <= 0 on failure, which is not remembered)
    // when there is none yet; -1 when `dev` is out of range
    template <typename F>
    int get(int dev, F&& setup) {
        if (dev < 0 || dev >= kMaxDevices) return -1;
        int v = v_[dev].load(std::memory_order_acquire);
        if (v > 0) return v;
        v = setup();
        if (v > 0) v_[dev].store(v, std::memory_order_release);
        return v;
    }
};

inline int current_device() {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// Per-device set-up of one kernel: raises its dynamic shared-memory limit to `smem` and returns how many of
// its CTAs fit on an SM (>= 1); <= 0 when the attribute could not be set on the current device.
template <typename K>
int kernel_setup(PerDevice& once, K kern, int threads, size_t smem) {
    return once.get(current_device(), [&]() -> int {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, threads, smem) != cudaSuccess || n < 1) n = 1;
        return n;
    });
}

// axis-1 kernels (bdr_row.cu); BDR_ERR_UNSUPPORTED = not covered, use the general kernel
template <typename T>
int quant_rowwise(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                  cudaStream_t st);
template <typename T>
int pack_rowwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                    const QParams& qp, double* sums, cudaStream_t st);

// bf16 tensors in the Table II family on packed bf16x2 arithmetic (bdr_row_x2.cu)
int quant_rowwise_mx_x2(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                        double* sums, cudaStream_t st);
int pack_rowwise_mx_x2(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld,
                       const bdr_planes_t& out, const QParams& qp, double* sums, cudaStream_t st);

int quant_colwise_qd_x2(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                        double* sums, cudaStream_t st);
int quant_colwise_mx_x2(const __nv_bfloat16* x, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld,
                        const bdr_planes_t* out, const QParams& qp, double* sums, cudaStream_t st);  // bdr_col_x2.cu

// both directions from one read of the tensor (bdr_pack2_x2.cu)
int pack2_mx_x2(const __nv_bfloat16* x, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& rout, const bdr_planes_t& cout_,
                const QParams& qp, double* sums_row, double* sums_col, cudaStream_t st);

// axis-0 fast path for k1 = 16, k2 = 2 (bdr_col.cu)
template <typename T>
int quant_colwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                     const QParams& qp, double* sums, cudaStream_t st);

// axis-0 quantize-dequantize of every other POW2 configuration with k2 <= 16 (bdr_col_any.cu)
template <typename T>
int quant_colwise_any(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums, cudaStream_t st);

// general kernels: any axis, any POW2 configuration, any alignment (bdr_general.cu)
template <typename T>
int quant_general(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const bdr_planes_t* out,
                  const QParams& qp, double* sums, cudaStream_t st);
template <typename T>
int unpack_general(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const QParams& qp,
                   cudaStream_t st);

// FP32 parent scale per k_parent elements above the two-level quantizer, fp32 tensors, k1 <= 16 (bdr_general.cu)
int quant_parent_scale(const float* x, float* y, int64_t rows, int64_t cols, int64_t ld, int axis, int k_parent, const QParams& qp,
                       double* sums, cudaStream_t st);

// rows of a packed table selected by device-side indices (bdr_general.cu)
template <typename T>
int gather_rows_general(const bdr_planes_t& in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t len, int64_t ld,
                        const QParams& qp, int* status, cudaStream_t st);

// the same for the Table II formats on packed bf16x2 arithmetic, one thread per 32 elements (bdr_gather_x2.cu)
template <typename T>
int gather_rows_mx_x2(const bdr_planes_t& in, int64_t n_rows, const int64_t* idx, T* y, int64_t n_idx, int64_t dim, int64_t ld,
                      const QParams& qp, int* status, cudaStream_t st);

// Packed MX4 / MX6 operands -> E4M3 bytes plus one power-of-two scale byte per 32 elements (bdr_reencode_f8.cu)
// Order in which the GEMM kernels' clusters walk over the 256 x 256 tiles of C: bands of band_rows tile rows, column by
// column inside a band (band_rows = 1 is row-major order).  With bands of eight the 74 tiles in flight share eight 256-row
// panels of A and about ten of B, which stay in L2, and every panel of B is fetched once per band; in row-major order a
// round of tiles touches every panel of B, and an operand larger than L2 is then read from HBM once per round.
__host__ __device__ inline void gemm_tile_coords(int t, int tiles_m, int tiles_n, int band_rows, int& tm, int& tn) {
    const int per_band = band_rows * tiles_n;
    const int band = t / per_band, r = t - band * per_band;
    const int left = tiles_m - band * band_rows;
    const int rows = band_rows < left ? band_rows : left;
    tn = r / rows;
    tm = band * band_rows + (r - tn * rows);
}
// Bands pay when the operands (bytes as the GEMM reads them) and the tiles of C being written no longer fit in L2 together
// (126 MB on the target); for operands of 64 MiB (4096^3 in bf16) row-major order measured 3 % faster.
inline int gemm_band_rows(int64_t operand_bytes) { return operand_bytes > (64ll << 20) ? 8 : 1; }

struct ZeroTiles {   // `count` tiles of 256 x 256 floats of c (row pitch ldc), tiles tile0 .. in the order of gemm_tile_coords
    float* c;
    int64_t ldc;
    int tiles_n, tile0, count, tiles_m, band_rows;
};
int reencode_rowwise_e4m3(const bdr_planes_t& a, int m_a, const bdr_planes_t& b, int m_b, int64_t M, int64_t N, int64_t K,
                          uint8_t* out_a, uint8_t* out_b, uint8_t* sf_a, uint8_t* sf_b, int* inexact, const ZeroTiles& z,
                          cudaStream_t st);
int unpack_rowwise_mx_x2(const bdr_planes_t& in, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                         cudaStream_t st, bool chained = false);  // bdr_unpack_x2.cu
int unpack_colwise_mx_x2(const bdr_planes_t& in, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                         cudaStream_t st);  // bdr_unpack_col_x2.cu

// unpack fast paths for k1 = 16, k2 = 2 (bdr_unpack.cu)
template <typename T>
int unpack_rowwise_mx(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                      cudaStream_t st);
template <typename T>
int unpack_colwise_mx(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                      cudaStream_t st);

}  // namespace bdr
