// Host-side declarations shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bdr.h"

namespace bdr {

struct QParams;

int sm_count();  // SMs of the current device (cached per device)

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

// axis-0 fast path for k1 = 16, k2 = 2 (bdr_col.cu)
template <typename T>
int quant_colwise_mx(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                     const QParams& qp, double* sums, cudaStream_t st);

// general kernels: any axis, any POW2 configuration, any alignment (bdr_general.cu)
template <typename T>
int quant_general(const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const bdr_planes_t* out,
                  const QParams& qp, double* sums, cudaStream_t st);
template <typename T>
int unpack_general(const bdr_planes_t& in, T* y, int64_t rows, int64_t cols, int64_t ld, int axis, const QParams& qp,
                   cudaStream_t st);

// Packed MX4 / MX6 operands -> E4M3 bytes plus one power-of-two scale byte per 32 elements (bdr_reencode_f8.cu)
struct ZeroTiles {   // `count` tiles of 256 x 256 floats of c (row pitch ldc, tiles_n tiles per row of tiles), from tile0 on
    float* c;
    int64_t ldc;
    int tiles_n, tile0, count;
};
int reencode_rowwise_e4m3(const bdr_planes_t& a, int m_a, const bdr_planes_t& b, int m_b, int64_t M, int64_t N, int64_t K,
                          uint8_t* out_a, uint8_t* out_b, uint8_t* sf_a, uint8_t* sf_b, int* inexact, const ZeroTiles& z,
                          cudaStream_t st);
int unpack_rowwise_mx_x2(const bdr_planes_t& in, __nv_bfloat16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                         cudaStream_t st);  // bdr_unpack_x2.cu
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
