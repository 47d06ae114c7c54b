// C-ABI entry points: argument validation on the host, then dispatch to the kernels.
#include <mutex>

#include <type_traits>

#include "bdr_async.cuh"
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

__device__ int g_device_status = 0;  // sticky: the first bounded wait that runs out leaves BDR_ERR_TIMEOUT here

bool make_tensor_map_u16(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows,
                         bool swizzle128) {
    typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One warp arms a barrier that nothing will ever complete and waits on it with the kernels' own bounded wait,
// cut down to a few hundred polls (well under a millisecond): the wait runs out, the warp reports it the way
// the streaming kernels do, and the kernel ends normally.
__global__ void bounded_wait_selftest_kernel(int* status) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = async::smem_u32(&bar);
    if (threadIdx.x == 0) {
        async::mbar_init(b, 1);
        async::fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0 && !async::mbar_wait<256>(b, 0)) async::report_timeout(status);
}

int* device_status_word() {
    static int* cached[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<int*>(p);
    }
    return cached[dev];
}

int sm_count() {
    static int cached[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

static bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// Definition-level check of a POW2 tuple, then what the kernels can run.
int check_pow2_config(const bdr_config_t* c, QParams* qp) {
    if (!c) return BDR_ERR_NULL;
    if (c->scale_kind != BDR_SCALE_POW2) {
        if (c->scale_kind < 0 || c->scale_kind > BDR_SCALE_FP32_VSQ) return BDR_ERR_BAD_CONFIG;
        return BDR_ERR_UNSUPPORTED;
    }
    if (c->rounding != BDR_ROUND_NEAREST_EVEN && c->rounding != BDR_ROUND_NEAREST_AWAY) return BDR_ERR_BAD_CONFIG;
    if (c->d1 != 8 || c->k1 < 1 || c->k2 < 1 || c->k1 % c->k2 != 0 || c->d2 < 0 || c->d2 > 3 || c->m < 1 || c->m > 8)
        return BDR_ERR_BAD_CONFIG;
    if (!is_pow2(c->k1) || !is_pow2(c->k2) || c->k1 > 1024) return BDR_ERR_UNSUPPORTED;
    if (qp) {
        qp->k1 = c->k1; qp->k2 = c->k2; qp->d2 = c->d2; qp->m = c->m; qp->rounding = c->rounding;
        qp->beta = (1 << c->d2) - 1;
        qp->qmax = (1u << c->m) - 1u;
    }
    return BDR_OK;
}

static int check_tensor(const void* x, int dt, int64_t rows, int64_t cols, int64_t ld, int axis) {
    if (dt != BDR_F32 && dt != BDR_BF16) return BDR_ERR_UNSUPPORTED;
    if (axis != 0 && axis != 1) return BDR_ERR_BAD_CONFIG;
    if (rows < 0 || cols < 0 || ld < cols) return BDR_ERR_SIZE;
    if (!x) return (rows == 0 || cols == 0) ? BDR_OK : BDR_ERR_NULL;  // an empty tensor has no storage
    if ((uintptr_t)x % (dt == BDR_F32 ? 4 : 2)) return BDR_ERR_MISALIGNED;
    return BDR_OK;
}

static void line_bytes(const bdr_config_t* c, int64_t len, int64_t out[3]) {
    const int64_t nb = (len + c->k1 - 1) / c->k1;
    out[0] = nb;
    out[1] = (nb * (c->k1 / c->k2) * c->d2 + 7) / 8;
    out[2] = (nb * c->k1 * (c->m + 1) + 7) / 8;
}

static int check_planes(const bdr_config_t* c, const bdr_planes_t* p, int64_t len) {
    if (!p || !p->exps || !p->elems || (c->d2 > 0 && !p->micro)) return BDR_ERR_NULL;
    int64_t need[3];
    line_bytes(c, len, need);
    if (p->ld_exps < need[0] || p->ld_elems < need[2] || (c->d2 > 0 && p->ld_micro < need[1])) return BDR_ERR_SIZE;
    if (((uintptr_t)p->exps | (uintptr_t)p->elems | (uintptr_t)(c->d2 ? p->micro : nullptr)) % 16) return BDR_ERR_MISALIGNED;
    if ((p->ld_exps | p->ld_elems | (c->d2 ? p->ld_micro : 0)) % 16) return BDR_ERR_MISALIGNED;
    return BDR_OK;
}

// True when every plane line is filled exactly by its natural bytes (no pitch padding to zero).
static bool planes_tight(const bdr_config_t* c, const bdr_planes_t* p, int64_t len) {
    int64_t need[3];
    line_bytes(c, len, need);
    return p->ld_exps == need[0] && p->ld_elems == need[2] && (c->d2 == 0 || p->ld_micro == need[1]);
}

template <typename T>
static int quant_dispatch(const QParams& qp, const T* x, T* y, int64_t rows, int64_t cols, int64_t ld, int axis,
                          const bdr_planes_t* out, bool tight, double* sums, cudaStream_t st) {
    if (rows == 0 || cols == 0) return BDR_OK;
    int rc = BDR_ERR_UNSUPPORTED;
    if (axis == 1) {
        if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            if (out) { if (tight) rc = pack_rowwise_mx_x2(x, y, rows, cols, ld, *out, qp, sums, st); }
            else rc = quant_rowwise_mx_x2(x, y, rows, cols, ld, qp, sums, st);
            if (rc != BDR_ERR_UNSUPPORTED) return rc;
        }
        if (out) { if (tight) rc = pack_rowwise_mx<T>(x, y, rows, cols, ld, *out, qp, sums, st); }
        else rc = quant_rowwise<T>(x, y, rows, cols, ld, qp, sums, st);
    } else {
        if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            if (!out) rc = quant_colwise_qd_x2(x, y, rows, cols, ld, qp, sums, st);
            if (rc == BDR_ERR_UNSUPPORTED && (!out || tight)) rc = quant_colwise_mx_x2(x, y, rows, cols, ld, out, qp, sums, st);
            if (rc != BDR_ERR_UNSUPPORTED) return rc;
        }
        if (!out || tight) rc = quant_colwise_mx<T>(x, y, rows, cols, ld, out, qp, sums, st);
        if (rc == BDR_ERR_UNSUPPORTED && !out) rc = quant_colwise_any<T>(x, y, rows, cols, ld, qp, sums, st);
    }
    if (rc == BDR_ERR_UNSUPPORTED) rc = quant_general<T>(x, y, rows, cols, ld, axis, out, qp, sums, st);
    return rc;
}

}  // namespace bdr

using namespace bdr;

extern "C" {

const char* bdr_strerror(int status) {
    switch (status) {
        case BDR_OK: return "ok";
        case BDR_ERR_NULL: return "a required pointer is NULL";
        case BDR_ERR_BAD_CONFIG: return "configuration outside the BDR definition";
        case BDR_ERR_UNSUPPORTED: return "valid request that no kernel of this library covers";
        case BDR_ERR_MISALIGNED: return "pointer or pitch breaks an alignment rule";
        case BDR_ERR_SIZE: return "bad size or pitch";
        case BDR_ERR_WORKSPACE: return "workspace missing or too small";
        case BDR_ERR_CUDA: return "CUDA call or kernel launch failed";
        case BDR_ERR_TIMEOUT: return "bounded device-side wait ran out";
    }
    return "unknown status";
}

int bdr_device_status(void) {
    int* word = device_status_word();
    int v = 0;
    if (!word || cudaMemcpy(&v, word, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return BDR_ERR_CUDA;
    return v;
}

int bdr_device_status_reset(void) {
    int* word = device_status_word();
    int v = 0;
    if (!word || cudaMemcpy(&v, word, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return BDR_ERR_CUDA;
    if (v != 0 && cudaMemset(word, 0, sizeof(v)) != cudaSuccess) return BDR_ERR_CUDA;
    return v;
}

int bdr_selftest_bounded_wait(int* status_dev, void* stream) {
    if (!status_dev) return BDR_ERR_NULL;
    if ((uintptr_t)status_dev % 4) return BDR_ERR_MISALIGNED;
    bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(status_dev);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

int bdr_selftest_host(void) {
    // PerDevice: the set-up runs once per device, a failed set-up is not remembered, bad indices are refused
    static PerDevice once;
    int runs[kMaxDevices] = {};
    auto setup_for = [&](int dev) { return [&runs, dev]() -> int { ++runs[dev]; return 10 + dev; }; };
    const int order[] = {0, 1, 0, 63, 1, 0, 63};
    for (int dev : order)
        if (once.get(dev, setup_for(dev)) != 10 + dev) return BDR_ERR_CUDA;
    if (runs[0] != 1 || runs[1] != 1 || runs[63] != 1 || runs[2] != 0) return BDR_ERR_CUDA;
    int failures = 0;
    if (once.get(2, [&]() -> int { ++failures; return 0; }) != 0) return BDR_ERR_CUDA;  // fails: nothing is remembered ...
    if (once.get(2, [&]() -> int { ++failures; return 7; }) != 7) return BDR_ERR_CUDA;  // ... so the next call sets up again
    if (once.get(2, [&]() -> int { ++failures; return 9; }) != 7 || failures != 2) return BDR_ERR_CUDA;
    if (once.get(-1, setup_for(0)) != -1 || once.get(kMaxDevices, setup_for(0)) != -1 || runs[0] != 1) return BDR_ERR_CUDA;
    return BDR_OK;
}

int bdr_packed_sizes(const bdr_config_t* cfg, int64_t rows, int64_t cols, int axis, int64_t ld_out[3],
                     int64_t bytes_out[3]) {
    if (!cfg || !ld_out || !bytes_out) return BDR_ERR_NULL;
    if (cfg->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
    if (cfg->d1 != 8 || cfg->k1 < 1 || cfg->k2 < 1 || cfg->k1 % cfg->k2 != 0 || cfg->d2 < 0 || cfg->d2 > 3 ||
        cfg->m < 1 || cfg->m > 8)
        return BDR_ERR_BAD_CONFIG;
    if (axis != 0 && axis != 1) return BDR_ERR_BAD_CONFIG;
    if (rows < 0 || cols < 0) return BDR_ERR_SIZE;
    const int64_t nlines = axis == 1 ? rows : cols, len = axis == 1 ? cols : rows;
    int64_t need[3];
    line_bytes(cfg, len, need);
    for (int i = 0; i < 3; ++i) {
        ld_out[i] = (need[i] + 15) / 16 * 16;
        bytes_out[i] = ld_out[i] * nlines;
    }
    return BDR_OK;
}

double bdr_tile_packing_efficiency(const bdr_config_t* c, int64_t tile_elems, int64_t line_bytes) {
    if (!c || tile_elems < 1 || line_bytes < 1 || c->m < 1 || c->k1 < 0 || c->k2 < 0 || c->d1 < 0 || c->d2 < 0) return -1.0;
    // integer arithmetic in units of 1 / (k1 k2) bit, so that no rounding decides the number of lines
    const int64_t k1 = c->k1 > 0 ? c->k1 : 1, k2 = c->k2 > 0 ? c->k2 : 1;
    const int64_t unit = k1 * k2;
    const int64_t per_elem = (int64_t)(c->m + 1) * unit + (c->k1 > 0 ? (int64_t)c->d1 * k2 : 0) + (c->k2 > 0 ? (int64_t)c->d2 * k1 : 0);
    const int64_t bits = per_elem * tile_elems, line = line_bytes * 8 * unit;
    const int64_t lines = (bits + line - 1) / line;
    return (double)bits / (double)(lines * line);
}

int bdr_quant_dequant(const bdr_config_t* cfg, const void* x, void* y, bdr_dtype_t dt, int64_t rows, int64_t cols,
                      int64_t ld, int axis, double* qsnr_sums_dev, void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if ((rc = check_tensor(x, dt, rows, cols, ld, axis))) return rc;
    if (rows == 0 || cols == 0) return BDR_OK;
    if (!y && !qsnr_sums_dev) return BDR_ERR_NULL;
    if (y && (uintptr_t)y % (dt == BDR_F32 ? 4 : 2)) return BDR_ERR_MISALIGNED;
    if (qsnr_sums_dev && (uintptr_t)qsnr_sums_dev % 8) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_F32)
        return quant_dispatch<float>(qp, (const float*)x, (float*)y, rows, cols, ld, axis, nullptr, false, qsnr_sums_dev, st);
    return quant_dispatch<__nv_bfloat16>(qp, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, rows, cols, ld, axis, nullptr,
                                         false, qsnr_sums_dev, st);
}

int bdr_pack(const bdr_config_t* cfg, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, int axis,
             const bdr_planes_t* out, void* y_dq, double* qsnr_sums_dev, void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if ((rc = check_tensor(x, dt, rows, cols, ld, axis))) return rc;
    if (rows == 0 || cols == 0) return BDR_OK;
    if ((rc = check_planes(cfg, out, axis == 1 ? cols : rows))) return rc;
    if (y_dq && (uintptr_t)y_dq % (dt == BDR_F32 ? 4 : 2)) return BDR_ERR_MISALIGNED;
    if (qsnr_sums_dev && (uintptr_t)qsnr_sums_dev % 8) return BDR_ERR_MISALIGNED;
    const bool tight = planes_tight(cfg, out, axis == 1 ? cols : rows);
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_F32)
        return quant_dispatch<float>(qp, (const float*)x, (float*)y_dq, rows, cols, ld, axis, out, tight, qsnr_sums_dev, st);
    return quant_dispatch<__nv_bfloat16>(qp, (const __nv_bfloat16*)x, (__nv_bfloat16*)y_dq, rows, cols, ld, axis, out,
                                         tight, qsnr_sums_dev, st);
}

int bdr_pack2(const bdr_config_t* cfg, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
              const bdr_planes_t* out_rows, const bdr_planes_t* out_cols, double* qsnr_sums_rows_dev, double* qsnr_sums_cols_dev,
              void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if ((rc = check_tensor(x, dt, rows, cols, ld, 1))) return rc;
    if (rows == 0 || cols == 0) return BDR_OK;
    if ((rc = check_planes(cfg, out_rows, cols))) return rc;
    if ((rc = check_planes(cfg, out_cols, rows))) return rc;
    if ((qsnr_sums_rows_dev && (uintptr_t)qsnr_sums_rows_dev % 8) || (qsnr_sums_cols_dev && (uintptr_t)qsnr_sums_cols_dev % 8)) return BDR_ERR_MISALIGNED;
    const bool tight_r = planes_tight(cfg, out_rows, cols), tight_c = planes_tight(cfg, out_cols, rows);
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_BF16 && tight_r && tight_c) {
        rc = pack2_mx_x2((const __nv_bfloat16*)x, rows, cols, ld, *out_rows, *out_cols, qp, qsnr_sums_rows_dev, qsnr_sums_cols_dev, st);
        if (rc != BDR_ERR_UNSUPPORTED) return rc;
    }
    // any other shape, dtype or configuration: one pass per direction (the same bytes, the tensor is read twice)
    if (dt == BDR_F32) {
        rc = quant_dispatch<float>(qp, (const float*)x, nullptr, rows, cols, ld, 1, out_rows, tight_r, qsnr_sums_rows_dev, st);
        if (rc) return rc;
        return quant_dispatch<float>(qp, (const float*)x, nullptr, rows, cols, ld, 0, out_cols, tight_c, qsnr_sums_cols_dev, st);
    }
    rc = quant_dispatch<__nv_bfloat16>(qp, (const __nv_bfloat16*)x, nullptr, rows, cols, ld, 1, out_rows, tight_r, qsnr_sums_rows_dev, st);
    if (rc) return rc;
    return quant_dispatch<__nv_bfloat16>(qp, (const __nv_bfloat16*)x, nullptr, rows, cols, ld, 0, out_cols, tight_c, qsnr_sums_cols_dev, st);
}

int bdr_quant_dequant_parent(const bdr_config_t* cfg, int k_parent, const void* x, void* y, bdr_dtype_t dt, int64_t rows, int64_t cols,
                             int64_t ld, int axis, double* qsnr_sums_dev, void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if (k_parent < cfg->k1 || k_parent % cfg->k1 != 0) return BDR_ERR_BAD_CONFIG;
    if ((rc = check_tensor(x, dt, rows, cols, ld, axis))) return rc;
    if (dt != BDR_F32 || cfg->k1 > 16 || k_parent > 1024 || k_parent % 16 != 0) return BDR_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return BDR_OK;
    if (!y && !qsnr_sums_dev) return BDR_ERR_NULL;
    if ((y && (uintptr_t)y % 4) || (qsnr_sums_dev && (uintptr_t)qsnr_sums_dev % 8)) return BDR_ERR_MISALIGNED;
    return quant_parent_scale((const float*)x, (float*)y, rows, cols, ld, axis, k_parent, qp, qsnr_sums_dev, (cudaStream_t)stream);
}

int bdr_gather_rows(const bdr_config_t* cfg, const bdr_planes_t* table, int64_t n_rows, int64_t dim, const int64_t* idx_dev,
                    int64_t n_idx, void* y, bdr_dtype_t dt, int64_t ld, void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if (n_rows < 0 || n_idx < 0) return BDR_ERR_SIZE;
    if ((rc = check_tensor(y, dt, n_idx, dim, ld, 1))) return rc;
    if (n_idx == 0 || dim == 0) return BDR_OK;
    if (!idx_dev) return BDR_ERR_NULL;
    if ((uintptr_t)idx_dev % 8) return BDR_ERR_MISALIGNED;
    if ((rc = check_planes(cfg, table, dim))) return rc;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_F32) {
        rc = gather_rows_mx_x2<float>(*table, n_rows, idx_dev, (float*)y, n_idx, dim, ld, qp, status, st);
        if (rc != BDR_ERR_UNSUPPORTED) return rc;
        return gather_rows_general<float>(*table, n_rows, idx_dev, (float*)y, n_idx, dim, ld, qp, status, st);
    }
    rc = gather_rows_mx_x2<__nv_bfloat16>(*table, n_rows, idx_dev, (__nv_bfloat16*)y, n_idx, dim, ld, qp, status, st);
    if (rc != BDR_ERR_UNSUPPORTED) return rc;
    return gather_rows_general<__nv_bfloat16>(*table, n_rows, idx_dev, (__nv_bfloat16*)y, n_idx, dim, ld, qp, status, st);
}

int bdr_unpack(const bdr_config_t* cfg, const bdr_planes_t* in, void* y, bdr_dtype_t dt, int64_t rows, int64_t cols,
               int64_t ld, int axis, void* stream) {
    QParams qp;
    int rc = check_pow2_config(cfg, &qp);
    if (rc) return rc;
    if ((rc = check_tensor(y, dt, rows, cols, ld, axis))) return rc;
    if (rows == 0 || cols == 0) return BDR_OK;
    if ((rc = check_planes(cfg, in, axis == 1 ? cols : rows))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == BDR_F32) {
        rc = axis == 1 ? unpack_rowwise_mx<float>(*in, (float*)y, rows, cols, ld, qp, st)
                       : unpack_colwise_mx<float>(*in, (float*)y, rows, cols, ld, qp, st);
        if (rc == BDR_ERR_UNSUPPORTED) rc = unpack_general<float>(*in, (float*)y, rows, cols, ld, axis, qp, st);
    } else {
        rc = BDR_ERR_UNSUPPORTED;
        rc = axis == 1 ? unpack_rowwise_mx_x2(*in, (__nv_bfloat16*)y, rows, cols, ld, qp, st)
                       : unpack_colwise_mx_x2(*in, (__nv_bfloat16*)y, rows, cols, ld, qp, st);
        if (rc != BDR_ERR_UNSUPPORTED) return rc;
        rc = axis == 1 ? unpack_rowwise_mx<__nv_bfloat16>(*in, (__nv_bfloat16*)y, rows, cols, ld, qp, st)
                       : unpack_colwise_mx<__nv_bfloat16>(*in, (__nv_bfloat16*)y, rows, cols, ld, qp, st);
        if (rc == BDR_ERR_UNSUPPORTED) rc = unpack_general<__nv_bfloat16>(*in, (__nv_bfloat16*)y, rows, cols, ld, axis, qp, st);
    }
    return rc;
}

}  // extern "C"
