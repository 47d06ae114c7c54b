// Column-direction (axis 0) quantize-dequantize of bf16 tensors in the Table II family (k1 = 16, k2 = 2,
// d2 = 1, m <= 7, ties-to-even) on packed bf16x2 arithmetic, without packed planes.
//
// Nothing has to be transposed when no planes are written: a block is 16 consecutive rows of one column,
// so a CTA works on slabs of 16 rows x kQCols columns and moves every row of a slab with one bulk copy of
// kQCols * 2 contiguous bytes (the same long transfers the row-direction kernel uses; 2-D tile boxes of
// 256-byte row segments measured about 10 % slower).  A thread owns two adjacent word columns (four
// columns: 8 bytes of every row), reads them down the slab without bank conflicts, quantizes the two
// halves of every word as two independent blocks, writes the dequantized words back over the slab, and
// after a CTA barrier the slab leaves row by row with bulk stores.  Three slabs rotate: one computing,
// one draining, one or two loading.  The first 16 threads are the producers, one row of the slab each.
#include <algorithm>

#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;

template <int QCOLS> struct QSlab {
    static constexpr int kCols = QCOLS;
    static constexpr int kThreads = QCOLS / 4;          // four columns per thread
    static constexpr int kRowBytes = QCOLS * 2;
    static constexpr int kBytes = kSlice * kRowBytes;   // 16 rows
    static constexpr int kStages = 3;
    static constexpr int kSmem = kStages * kBytes + 64; // + barriers
};

template <int QCOLS, bool SUMS, bool YOUT>
__global__ void __launch_bounds__(QSlab<QCOLS>::kThreads)
col_qd_x2_kernel(const bf16* x, bf16* y, int64_t ld, int n_col_slabs, int n_slabs, QParams qp, double* sums, int* status) {
    using SL = QSlab<QCOLS>;
    constexpr int S = SL::kStages;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t ring0 = async::smem_u32(smem);
    const uint32_t bars = ring0 + S * SL::kBytes;
    const int tid = threadIdx.x;
    const int m = qp.m;
    const bool producer = tid < kSlice;  // thread r moves row r of every slab

    auto slab_origin = [&](int s, int64_t& row0, int64_t& col0) {
        const int br = s / n_col_slabs, cs = s - br * n_col_slabs;
        row0 = (int64_t)br * kSlice;
        col0 = (int64_t)cs * QCOLS;
    };
    auto load_row = [&](int s, int stg) {  // producers only
        int64_t row0, col0;
        slab_origin(s, row0, col0);
        const uint32_t bar = bars + 8 * stg;
        async::mbar_expect_tx(bar, SL::kRowBytes);
        async::bulk_load(ring0 + stg * SL::kBytes + tid * SL::kRowBytes, x + (row0 + tid) * ld + col0, SL::kRowBytes, bar);
    };
    if (tid == 0) {
#pragma unroll
        for (int k = 0; k < S; ++k) async::mbar_init(bars + 8 * k, kSlice);
        async::fence_barrier_init();
    }
    __syncthreads();
    // slabs in flight before the loop: with output, a stage is refilled only after its store has been read out,
    // which happens one iteration later, so two loads lead; without output all three stages load at once
    constexpr int kLead = YOUT ? S - 1 : S;
    if (producer) {
#pragma unroll
        for (int k = 0; k < kLead; ++k) {
            const int64_t s = (int64_t)blockIdx.x + (int64_t)k * gridDim.x;
            if (s < n_slabs) load_row((int)s, k);
        }
    }
    uint32_t phase = 0;
    int stg = 0;
    double e2 = 0.0, s2 = 0.0;
    bool failed = false;
    for (int64_t s = blockIdx.x; s < n_slabs; s += gridDim.x) {
        if (!failed && !async::mbar_wait(bars + 8 * stg, phase)) {
            async::report_timeout(status);
            failed = true;
        }
        const uint32_t mine = ring0 + stg * SL::kBytes + tid * 8;
        uint32_t wc[2][16];
#pragma unroll
        for (int r = 0; r < kSlice; ++r) {
            const uint2 v = async::lds64(mine + r * SL::kRowBytes);
            wc[0][r] = v.x;
            wc[1][r] = v.y;
        }
        if constexpr (!YOUT) {
            __syncthreads();  // every thread has read the stage: refill it
            const int64_t nxt = s + (int64_t)S * gridDim.x;
            if (producer && !failed && nxt < n_slabs) load_row((int)nxt, stg);
        }
#pragma unroll
        for (int c = 0; c < 2; ++c) {  // the thread's two word columns
            uint32_t aw[16], pm[8], yw[16], cl[1], ch[1], F2;
            x2::WordColOut o;
            if (x2::wordcol_exponents(wc[c], aw, pm, F2)) {
                x2::quantize_wordcol<0, SUMS, YOUT>(wc[c], aw, pm, F2, m, yw, cl, ch, o);
                if constexpr (SUMS) {
                    const double wl = x2::pow4_weight((F2 >> 7) & 0xFFu), wh = x2::pow4_weight(F2 >> 23);
                    e2 = fma((double)o.pe_lo, wl, e2);
                    e2 = fma((double)o.pe_hi, wh, e2);
                    s2 = fma((double)o.ps_lo, wl, s2);
                    s2 = fma((double)o.ps_hi, wh, s2);
                }
            } else {
                x2::WordCol in;
#pragma unroll
                for (int r = 0; r < 16; ++r) in.w[r] = wc[c][r];
                const x2::WordColSlow so = x2::quantize_wordcol_slow<0, SUMS>(in, qp);
#pragma unroll
                for (int r = 0; r < 16; ++r) yw[r] = so.y[r];
                if constexpr (SUMS) { e2 += so.e2; s2 += so.s2; }
            }
            if constexpr (YOUT) {
#pragma unroll
                for (int r = 0; r < 16; ++r) wc[c][r] = yw[r];
            }
        }
        if constexpr (YOUT) {
#pragma unroll
            for (int r = 0; r < kSlice; ++r) async::sts64(mine + r * SL::kRowBytes, wc[0][r], wc[1][r]);
            async::fence_proxy_async();
            __syncthreads();  // the whole slab holds results
            if (producer) {
                int64_t row0, col0;
                slab_origin((int)s, row0, col0);
                async::bulk_store(y + (row0 + tid) * ld + col0, ring0 + stg * SL::kBytes + tid * SL::kRowBytes, SL::kRowBytes);
                async::bulk_commit();
                async::bulk_wait_read<1>();  // the previous slab's row has left its stage: that stage takes the slab two ahead
                const int64_t nxt = s + (int64_t)kLead * gridDim.x;
                if (!failed && nxt < n_slabs) load_row((int)nxt, stg + kLead >= S ? stg + kLead - S : stg + kLead);
            }
        }
        if (++stg == S) { stg = 0; phase ^= 1; }
    }
    if (YOUT && producer) async::bulk_wait_all();
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

template <int QCOLS, bool SUMS, bool YOUT>
static int launch_col_qd(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums, cudaStream_t st) {
    using SL = QSlab<QCOLS>;
    auto kern = col_qd_x2_kernel<QCOLS, SUMS, YOUT>;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, SL::kThreads, SL::kSmem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    const int n_cs = (int)(cols / QCOLS);
    const int64_t n_slabs = (int64_t)n_cs * (rows / kSlice);
    if (n_slabs == 0) return BDR_OK;
    const int grid = (int)std::min<int64_t>(n_slabs, (int64_t)sm_count() * blocks_per_sm);
    kern<<<grid, SL::kThreads, SL::kSmem, st>>>(x, y, ld, n_cs, (int)n_slabs, qp, sums, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

constexpr int kQCols = 512;

// Fast path without planes: whole slabs of 16 rows x kQCols columns, 16-byte aligned rows.
// BDR_ERR_UNSUPPORTED sends the caller to the tile kernel and the generic column kernels.
int quant_colwise_qd_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                        cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || qp.m > 7 || qp.rounding != BDR_ROUND_NEAREST_EVEN) return BDR_ERR_UNSUPPORTED;
    if (rows % kSlice != 0 || cols % kQCols != 0) return BDR_ERR_UNSUPPORTED;
    if ((((uintptr_t)x | (uintptr_t)y) % 16) || (ld * 2) % 16) return BDR_ERR_UNSUPPORTED;
    if ((cols / kQCols) * (rows / kSlice) >= (1ll << 30)) return BDR_ERR_UNSUPPORTED;
    if (sums) return y ? launch_col_qd<kQCols, true, true>(x, y, rows, cols, ld, qp, sums, st)
                       : launch_col_qd<kQCols, true, false>(x, y, rows, cols, ld, qp, sums, st);
    if (y) return launch_col_qd<kQCols, false, true>(x, y, rows, cols, ld, qp, sums, st);
    return BDR_ERR_NULL;
}

}  // namespace bdr
