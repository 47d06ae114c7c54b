// Row-direction (axis 1) kernels for bf16 tensors in the Table II family (k1 = 16, k2 = 2, d2 = 1,
// m <= 7, ties-to-even), built on the packed bf16x2 quantizer: two elements per instruction, so the
// kernels stay bound by HBM rather than by instruction issue.  Thread mapping, prefetch ring and
// coalesced stores are those of the generic row kernels: a lane owns two adjacent 16-element blocks
// (64 bytes) of a warp's contiguous 2 KB run per iteration.
#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;
constexpr int kX2SPT = 2;

__device__ __forceinline__ void words_of(const uint4& v0, const uint4& v1, uint32_t (&w)[8]) {
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w;
    w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
}

// Per-warp pipeline.  A warp streams runs of 2048 elements (4 KB) through a small ring in shared memory:
// lane 0 keeps two runs in flight with one bulk copy each (with ~16-24 warps per SM, well over 100 KB per
// SM).  A run is handled as two halves of 1024 elements; in each a lane owns 64 consecutive bytes (two
// blocks).  Dequantized values are written back over the run's input in its stage and leave with one
// bulk store of 4 KB (measured: faster than 32-byte stores from registers); the packed planes of a run
// are collected per warp in a small double-buffered staging area and leave with one bulk store each
// (256 W code bytes, 128 exponent bytes, 128 microexponent bytes).  Bulk stores are grouped per run;
// "all but the latest group have been read" frees what the previous run used.
constexpr int kX2Threads = 128;
constexpr int kX2Warps = kX2Threads / 32;
constexpr int kX2Ahead = 2;  // runs in flight per warp
constexpr int kX2Sub = 2;                                    // halves per run
constexpr int kSubElems = 32 * kX2SPT * kSlice;              // 1024
constexpr int kX2RunElems = kX2Sub * kSubElems;              // 2048
constexpr int kRunBytes = kX2RunElems * 2;
// Stages per warp: with dequantized output the results are written back into the stage they came from and
// leave with a bulk store, so a third stage is needed while that store drains.
template <bool YOUT> struct X2Ring {
    static constexpr int kStages = YOUT ? kX2Ahead + 1 : kX2Ahead;
    static constexpr int kBytes = kX2Warps * kStages * kRunBytes;
};
constexpr int kX2BarBytes = 128;  // barriers of 8 bytes, padded
static_assert(kX2Warps * (kX2Ahead + 1) * 8 <= kX2BarBytes, "barrier area");

template <int W> struct X2PackStage {
    static constexpr int kElemBytes = kX2RunElems / 8 * W;
    static constexpr int kExpBytes = kX2RunElems / 16;
    static constexpr int kMicroBytes = kX2RunElems / 16;
    static constexpr int kBytes = W > 0 ? kElemBytes + kExpBytes + kMicroBytes : 0;  // a multiple of 128
};

struct RunIndex : x2::RunIndex {
    __device__ __forceinline__ int64_t elem_offset(uint32_t wi) const {
        int64_t row, pos;
        split(wi, row, pos);
        return row * ld + pos * kX2RunElems;
    }
};

// W = 0: quantize-dequantize (any m <= 7, from qp); W = m + 1: also write the packed planes.
template <int W, bool SUMS, bool YOUT>
__global__ void __launch_bounds__(kX2Threads)
row_mx_x2_kernel(const bf16* x, bf16* y, RunIndex ri, uint32_t total, bdr_planes_t out, QParams qp, double* sums, int* status) {
    using PS = X2PackStage<W>;
    constexpr bool PACK = W > 0;
    constexpr bool kPackOnly = PACK && !SUMS && !YOUT;
    constexpr int S = X2Ring<YOUT>::kStages;
    constexpr int kX2RingBytes = X2Ring<YOUT>::kBytes;
    constexpr int NCW = PACK ? (16 * W + 31) / 32 : 1;  // words of one block's codes (the last one half full when W is odd)
    extern __shared__ __align__(128) uint8_t smem[];  // ring [warp][stage][4 KB], barriers, staging [warp][2]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring0 = async::smem_u32(smem) + warp * S * kRunBytes;
    const uint32_t bars = async::smem_u32(smem) + kX2RingBytes + warp * S * 8;
    const uint32_t stage0 = async::smem_u32(smem) + kX2RingBytes + kX2BarBytes + warp * 2 * PS::kBytes;
    const int m = PACK ? W - 1 : qp.m;
    const x2::Consts k = x2::make_consts(m, PACK ? 1 : qp.d2);
    const int group_lanes = qp.k1 >> 5;  // lanes that share a block when k1 >= 64 (1 when the lane's two blocks form one)
    const uint32_t stride = gridDim.x * kX2Warps;
    const uint32_t w0 = blockIdx.x * kX2Warps + warp;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < S; ++s) async::mbar_init(bars + 8 * s, 1);
        async::fence_barrier_init();
#pragma unroll
        for (int s = 0; s < kX2Ahead; ++s) {
            const uint32_t wi = w0 + s * stride;
            if (wi < total) {
                async::mbar_expect_tx(bars + 8 * s, kRunBytes);
                async::bulk_load(ring0 + s * kRunBytes, x + ri.elem_offset(wi), kRunBytes, bars + 8 * s);
            }
        }
    }
    int st = 0;
    uint32_t phase = 0, half = 0;
    double e2 = 0.0, s2 = 0.0;
    for (uint32_t wi = w0; wi < total; wi += stride) {
        __syncwarp();  // lane 0 has finished the previous iteration's hand-over (staging half is free)
        if (!async::mbar_wait(bars + 8 * st, phase)) {
            async::report_timeout(status);
            // Nothing more is issued.  The loads queued for this and the next kX2Ahead - 1 runs may still be on
            // their way into this CTA's shared memory: give each of them one further bounded wait, so that the
            // CTA does not knowingly leave with a copy in flight (if one still does not land, the CTA leaves
            // all the same: the wait must end).
            if (lane == 0) {
                for (int s = 0; s < kX2Ahead; ++s) {
                    if ((uint64_t)wi + (uint64_t)s * stride >= total) break;
                    int ds = st + s;
                    uint32_t dp = phase;
                    if (ds >= S) { ds -= S; dp ^= 1; }
                    async::mbar_wait(bars + 8 * ds, dp);
                }
            }
            break;
        }
        const uint32_t stage = stage0 + half * PS::kBytes;
#pragma unroll
        for (int sub = 0; sub < kX2Sub; ++sub) {
            const uint32_t mine = ring0 + st * kRunBytes + sub * (kSubElems * 2) + lane * 64;
            if constexpr (!PACK) {
                // quantize-dequantize: blocks of 16 .. 1024 elements.  The two 16-element blocks of the lane give
                // their exponents first; wider blocks take the maximum over the lane's pair and, from 64
                // elements on, over the k1 / 32 adjacent lanes that share the block.
                uint4 vv[kX2SPT][2];
                uint32_t w[kX2SPT][8], aw[kX2SPT][8], Fb[kX2SPT];
#pragma unroll
                for (int s = 0; s < kX2SPT; ++s) {
                    vv[s][0] = async::lds128(mine + 32 * s);
                    vv[s][1] = async::lds128(mine + 32 * s + 16);
                    words_of(vv[s][0], vv[s][1], w[s]);
#pragma unroll
                    for (int j = 0; j < 8; ++j) aw[s][j] = x2::habs2(w[s][j]);
                    Fb[s] = x2::block_exponent(aw[s]);
                }
                if (group_lanes > 0) {  // the same for every thread
                    uint32_t F = max(Fb[0], Fb[1]);
                    for (int o = group_lanes >> 1; o > 0; o >>= 1) F = max(F, __shfl_xor_sync(0xFFFFFFFFu, F, o));
                    Fb[0] = F;
                    Fb[1] = F;
                }
#pragma unroll
                for (int s = 0; s < kX2SPT; ++s) {
                    uint32_t yw[8];
                    const uint32_t F = Fb[s];
                    if (F - x2::kMinF <= (uint32_t)(x2::kMaxF - x2::kMinF)) {
                        float pe = 0.f, ps = 0.f;
                        uint32_t code2[8], micro;
                        x2::quantize_block_row<SUMS, YOUT, false>(w[s], aw[s], F, m, k, yw, code2, micro, pe, ps);
                        if constexpr (SUMS) {
                            const double wgt = x2::pow4_weight(F);
                            e2 = fma((double)pe, wgt, e2);
                            s2 = fma((double)ps, wgt, s2);
                        }
                    } else {
                        const x2::SlowOut o = x2::quantize_block_slow<0, SUMS>(vv[s][0], vv[s][1], qp, F);
                        if constexpr (SUMS) { e2 += o.e2; s2 += o.s2; }
                        if constexpr (YOUT) {
                            yw[0] = o.y[0].x; yw[1] = o.y[0].y; yw[2] = o.y[0].z; yw[3] = o.y[0].w;
                            yw[4] = o.y[1].x; yw[5] = o.y[1].y; yw[6] = o.y[1].z; yw[7] = o.y[1].w;
                        }
                    }
                    if constexpr (YOUT) {  // back into the stage, over the block's input
                        async::sts128(mine + 32 * s, make_uint4(yw[0], yw[1], yw[2], yw[3]));
                        async::sts128(mine + 32 * s + 16, make_uint4(yw[4], yw[5], yw[6], yw[7]));
                    }
                }
            }
            [[maybe_unused]] uint32_t cw[kX2SPT][NCW], Fs[kX2SPT], mbs[kX2SPT];
            if constexpr (PACK) {
#pragma unroll
            for (int s = 0; s < kX2SPT; ++s) {
                const uint4 v0 = async::lds128(mine + 32 * s), v1 = async::lds128(mine + 32 * s + 16);
                uint32_t w[8], yw[8];
                words_of(v0, v1, w);
                x2::PairView pv;
                uint32_t aw[8], F;
                if constexpr (kPackOnly) {
                    F = x2::pair_view(w, pv);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) aw[j] = x2::habs2(w[j]);
                    F = x2::block_exponent(aw);
                }
                if (F - x2::kMinF <= (uint32_t)(x2::kMaxF - x2::kMinF)) {
                    if constexpr (kPackOnly) {
                        x2::pack_pair_view<PACK ? W : 8>(pv, F, cw[s], mbs[s]);
                        Fs[s] = F;
                    } else {
                        float pe = 0.f, ps = 0.f;
                        uint32_t code2[8];
                        x2::quantize_block_row<SUMS, YOUT, PACK>(w, aw, F, m, k, yw, code2, mbs[s], pe, ps);
                        if constexpr (PACK) {
                            x2::pack_block<PACK ? W : 8>(code2, cw[s]);
                            Fs[s] = F;
                        }
                        if constexpr (SUMS) {
                            const double wgt = x2::pow4_weight(F);
                            e2 = fma((double)pe, wgt, e2);
                            s2 = fma((double)ps, wgt, s2);
                        }
                    }
                } else {
                    const x2::SlowOut o = x2::quantize_block_slow<W, SUMS>(v0, v1, qp);
                    if constexpr (PACK) {
#pragma unroll
                        for (int i = 0; i < NCW; ++i) cw[s][i] = o.cw[i];
                        Fs[s] = o.F;
                        mbs[s] = o.micro;
                    }
                    if constexpr (SUMS) { e2 += o.e2; s2 += o.s2; }
                    if constexpr (YOUT) {
                        yw[0] = o.y[0].x; yw[1] = o.y[0].y; yw[2] = o.y[0].z; yw[3] = o.y[0].w;
                        yw[4] = o.y[1].x; yw[5] = o.y[1].y; yw[6] = o.y[1].z; yw[7] = o.y[1].w;
                    }
                }
                if constexpr (YOUT) {  // back into the stage, over the block's input
                    async::sts128(mine + 32 * s, make_uint4(yw[0], yw[1], yw[2], yw[3]));
                    async::sts128(mine + 32 * s + 16, make_uint4(yw[4], yw[5], yw[6], yw[7]));
                }
            }
            }
            if constexpr (PACK) {
                // the lane's 32 codes as W words: block 1 follows block 0 at bit 16 W
                const uint32_t dst = stage + sub * (kSubElems / 8 * W) + lane * 4 * W;
                if constexpr (W == 8) {
                    async::sts128(dst, make_uint4(cw[0][0], cw[0][1], cw[0][2], cw[0][3]));
                    async::sts128(dst + 16, make_uint4(cw[1][0], cw[1][1], cw[1][2], cw[1][3]));
                } else {
#pragma unroll
                    for (int i = 0; i < W / 2; ++i) async::sts32(dst + 4 * i, cw[0][i]);
                    async::sts32(dst + 4 * (W / 2), cw[0][W / 2] | (cw[1][0] << 16));
#pragma unroll
                    for (int i = 0; i < W / 2; ++i) async::sts32(dst + 4 * (W / 2 + 1 + i), __byte_perm(cw[1][i], cw[1][i + 1], 0x5432));
                }
                async::sts16(stage + PS::kElemBytes + sub * (kSubElems / 16) + 2 * lane, Fs[0] | (Fs[1] << 8));
                async::sts16(stage + PS::kElemBytes + PS::kExpBytes + sub * (kSubElems / 16) + 2 * lane, mbs[0] | (mbs[1] << 8));
            }
        }
        if constexpr (PACK || YOUT) async::fence_proxy_async();
        __syncwarp();  // every lane has consumed stage st (and filled the staging half)
        if (lane == 0) {
            if constexpr (YOUT) {
                async::bulk_store(y + ri.elem_offset(wi), ring0 + st * kRunBytes, kRunBytes);
                if constexpr (!PACK) {
                    async::bulk_commit();
                    async::bulk_wait_read<1>();  // the previous run's store has left its stage, which is refilled below
                }
            }
            if constexpr (PACK) {
                int64_t row, pos;
                ri.split(wi, row, pos);
                const int64_t blk0 = pos * (kX2RunElems / 16);  // first block of the run within its row
                async::bulk_store(out.elems + row * out.ld_elems + blk0 * 2 * W, stage, PS::kElemBytes);
                async::bulk_store(out.exps + row * out.ld_exps + blk0, stage + PS::kElemBytes, PS::kExpBytes);
                async::bulk_store(out.micro + row * out.ld_micro + blk0, stage + PS::kElemBytes + PS::kExpBytes, PS::kMicroBytes);
                async::bulk_commit();
                async::bulk_wait_read<1>();  // the other staging half (used next) has been read out
            }
            const uint32_t next = wi + kX2Ahead * stride;
            const int nst = st + kX2Ahead >= S ? st + kX2Ahead - S : st + kX2Ahead;  // YOUT: the previous run's stage; else this one
            if (next < total) {
                async::mbar_expect_tx(bars + 8 * nst, kRunBytes);
                async::bulk_load(ring0 + nst * kRunBytes, x + ri.elem_offset(next), kRunBytes, bars + 8 * nst);
            }
        }
        half ^= 1;
        if (++st == S) { st = 0; phase ^= 1; }
    }
    if ((PACK || YOUT) && lane == 0) async::bulk_wait_all();
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

// ---- host launchers --------------------------------------------------------------------------------
// packing: the Table II family; quantize-dequantize: blocks of 16 .. 1024 elements with one-bit shifts per pair of
// elements, or without shifts (d2 = 0, where k2 does not matter)
static bool x2_config(const QParams& qp, bool pack) {
    if (qp.m > 7 || qp.rounding != BDR_ROUND_NEAREST_EVEN) return false;
    if (pack) return qp.k1 == 16 && qp.k2 == 2 && qp.d2 == 1;
    const bool k1_ok = qp.k1 >= 16 && qp.k1 <= 1024 && (qp.k1 & (qp.k1 - 1)) == 0;
    return k1_ok && ((qp.k2 == 2 && qp.d2 == 1) || qp.d2 == 0);
}

// One wave of resident CTAs: every warp then streams many runs through its prefetch ring instead of
// paying the ring's start-up again in a second, partly filled wave.
static int x2_grid(int64_t total_warps, int blocks_per_sm) {
    const int64_t need = (total_warps + kX2Threads / 32 - 1) / (kX2Threads / 32);
    return (int)max((int64_t)1, min(need, (int64_t)sm_count() * blocks_per_sm));
}

template <int W, bool SUMS, bool YOUT>
static int launch_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out, const QParams& qp,
                     double* sums, cudaStream_t st) {
    const int64_t rpr = cols / kX2RunElems, total = rows * rpr;
    if (total == 0) return BDR_OK;
    if (total >= (1ll << 31) - (1ll << 24)) return BDR_ERR_UNSUPPORTED;  // 32-bit run indices (incl. look-ahead)
    auto kern = row_mx_x2_kernel<W, SUMS, YOUT>;
    const size_t smem = X2Ring<YOUT>::kBytes + kX2BarBytes + kX2Warps * 2 * X2PackStage<W>::kBytes;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, kX2Threads, smem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    bdr_planes_t pl = {};
    if (out) pl = *out;
    RunIndex ri;
    ri.runs_per_row = make_fastdiv((uint32_t)rpr);
    ri.ld = ld;
    ri.flat = rows == 1 ? 1 : 0;
    kern<<<x2_grid(total, blocks_per_sm), kX2Threads, smem, st>>>(x, y, ri, (uint32_t)total, pl, qp, sums, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <int W>
static int x2_flags(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out, const QParams& qp,
                    double* sums, cudaStream_t st) {
    if (sums) return y ? launch_x2<W, true, true>(x, y, rows, cols, ld, out, qp, sums, st)
                       : launch_x2<W, true, false>(x, y, rows, cols, ld, out, qp, sums, st);
    if (y) return launch_x2<W, false, true>(x, y, rows, cols, ld, out, qp, sums, st);
    if constexpr (W > 0) return launch_x2<W, false, false>(x, y, rows, cols, ld, out, qp, sums, st);
    return BDR_ERR_NULL;
}

// Shapes: whole 2048-element runs, 32-byte aligned (a contiguous tensor whose rows hold whole blocks counts as
// one long row).
static bool x2_shape(const void* x, const void* y, int64_t& rows, int64_t& cols, int64_t& ld, int k1 = 16) {
    if ((((uintptr_t)x | (uintptr_t)y) % 32) || (ld * 2) % 32) return false;
    if (ld == cols && cols % k1 == 0) {
        cols *= rows;
        ld = cols;
        rows = 1;
    }
    return cols % kX2RunElems == 0;
}

int quant_rowwise_mx_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp, double* sums,
                        cudaStream_t st) {
    if (!x2_config(qp, false) || !x2_shape(x, y, rows, cols, ld, qp.k1)) return BDR_ERR_UNSUPPORTED;
    return x2_flags<0>(x, y, rows, cols, ld, nullptr, qp, sums, st);
}

// The caller guarantees tight planes (line pitch = the line's natural bytes).
int pack_rowwise_mx_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& out,
                       const QParams& qp, double* sums, cudaStream_t st) {
    if (!x2_config(qp, true) || !x2_shape(x, y, rows, cols, ld)) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return x2_flags<3>(x, y, rows, cols, ld, &out, qp, sums, st);
        case 4: return x2_flags<5>(x, y, rows, cols, ld, &out, qp, sums, st);
        case 7: return x2_flags<8>(x, y, rows, cols, ld, &out, qp, sums, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
