// Dual-direction packing of a bf16 tensor in the Table II family (k1 = 16, k2 = 2, d2 = 1, m in {2, 4, 7},
// ties-to-even): the tensor is read from memory ONCE and both packed copies are written, the one quantized
// along the rows and the one quantized along the columns ("transpose, then quantize").  Section V, Fig. 8:
// every tensor of a training step feeds one matrix product of the forward pass and one of the backward pass,
// each reducing over a different dimension, so each tensor is quantized along both.
//
// A CTA of eight warps owns tiles of 256 rows x 128 columns; warp w takes block rows 2w and 2w+1 of a tile,
// each a box of 16 rows x 128 columns (4 KB) fetched as two 2-D TMA tile loads of 64 columns (128-byte rows,
// 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7), which makes both access patterns below
// free of bank conflicts) into the warp's own ring.  A box is used twice while it sits in shared memory:
//   * column direction: a lane owns four adjacent columns (8 bytes of every row) = two word columns, i.e. four
//     blocks of 16 rows; codes are staged per tile as [block-row pair][column] items and, after a CTA barrier,
//     each column's 16 blocks leave as one contiguous run of the column-major planes;
//   * row direction: the same box read as 64 items of 32 consecutive elements of a row (two blocks, 64 bytes);
//     a lane takes two items, and a row's 8 blocks leave as one contiguous run of the row-major planes.
// The arithmetic is the packed bf16x2 formulation of bdr_x2.cuh in both directions; blocks outside its exponent
// range take the out-of-line fp32 / integer formulation, so every byte equals what the two single-direction
// calls write.  Every wait is bounded.
#include <algorithm>

#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;

constexpr int kP2Threads = 256;
constexpr int kP2Warps = kP2Threads / 32;
constexpr int kP2TileCols = 128;
constexpr int kP2TileBlocks = 2 * kP2Warps;  // 16 block rows = 256 rows
constexpr int kP2TileRows = kP2TileBlocks * kSlice;
constexpr int kP2BoxBytes = kSlice * kP2TileCols * 2;  // 4 KB
constexpr int kP2Stages = 2;
constexpr int kP2RingBytes = kP2Warps * kP2Stages * kP2BoxBytes;
constexpr int kP2BarBytes = 256;

template <int W> struct P2Stage {
    // column direction, per tile -- codes: W even: [block row 16][column 128] items of 2W bytes, columns XOR-swizzled by
    // the block row; W odd: [block-row pair 8][column 128] items of 4W bytes.  Exponent / microexponent bytes [block row][column].
    static constexpr int kColElemBytes = kP2TileBlocks * kP2TileCols * 2 * W;
    static constexpr int kColExpBytes = kP2TileBlocks * kP2TileCols;
    // row direction, per warp and box (odd W only: W = 8 stores 32 aligned bytes per item straight from registers):
    // [row 16][16 W bytes]
    static constexpr int kRowBytes = W == 8 ? 0 : kSlice * 16 * W;
    static constexpr int kBytes = kColElemBytes + 2 * kColExpBytes + kP2Warps * kRowBytes;
};

__device__ __forceinline__ void p2_words_of(const uint4& a, const uint4& b, uint32_t (&w)[8]) {
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}

template <int W, bool SUMS>
__global__ void __launch_bounds__(kP2Threads, 2)
pack2_x2_kernel(const __grid_constant__ CUtensorMap xmap, int n_col_tiles, int n_tiles, bdr_planes_t rout, bdr_planes_t cout_,
                QParams qp, double* sums_row, double* sums_col, int* status) {
    using PS = P2Stage<W>;
    constexpr int NCW = (16 * W + 31) / 32;
    constexpr int S = kP2Stages;
    constexpr int M = W - 1;
    extern __shared__ __align__(1024) uint8_t smem[];  // ring [warp][stage][4 KB] (1 KB aligned: swizzle atoms), barriers, column staging, row staging
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring0 = async::smem_u32(smem) + warp * S * kP2BoxBytes;
    const uint32_t bars = async::smem_u32(smem) + kP2RingBytes + warp * 32;
    const uint32_t st_elems = async::smem_u32(smem) + kP2RingBytes + kP2BarBytes;
    const uint32_t st_exps = st_elems + PS::kColElemBytes, st_micro = st_exps + PS::kColExpBytes;
    const uint32_t st_row = st_micro + PS::kColExpBytes + warp * PS::kRowBytes;

    auto issue = [&](int t, int i, int stg) {  // lane 0 only: box i of tile t into stage stg
        const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
        async::mbar_expect_tx(bars + 8 * stg, kP2BoxBytes);
        const int row0 = rt * kP2TileRows + (2 * warp + i) * kSlice;
        async::tma_load_2d(ring0 + stg * kP2BoxBytes, &xmap, ct * kP2TileCols, row0, bars + 8 * stg);
        async::tma_load_2d(ring0 + stg * kP2BoxBytes + kP2BoxBytes / 2, &xmap, ct * kP2TileCols + kP2TileCols / 2, row0, bars + 8 * stg);
    };
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < S; ++k) async::mbar_init(bars + 8 * k, 1);
        async::fence_barrier_init();
        if ((int)blockIdx.x < n_tiles) {
            issue(blockIdx.x, 0, 0);
            issue(blockIdx.x, 1, 1);
        }
    }
    __syncwarp();
    uint32_t phase = 0;
    double e2c = 0.0, s2c = 0.0, e2r = 0.0, s2r = 0.0;
    bool failed = false;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
        uint32_t cw0[4][NCW];  // column codes of block row 2*warp (odd W: held until the pair is complete)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int stg = i;  // two boxes per tile, two stages: box i always lives in stage i
            const int bl = 2 * warp + i;
            if (!failed && !async::mbar_wait(bars + 8 * stg, phase)) {
                async::report_timeout(status);
                failed = true;
            }
            const uint32_t box = ring0 + stg * kP2BoxBytes;
            // ---- column direction: the lane's two word columns ------------------------------------------------
            {
                // the lane's 8 bytes of row r: half box lane / 16, chunk (lane % 16) / 2 of the row, swizzled by the row
                const uint32_t mine = box + (lane >> 4) * (kP2BoxBytes / 2) + (lane & 1) * 8;
                const uint32_t chunk = ((lane & 15) >> 1) << 4;
                uint32_t Fb[4], Mb[4];
                [[maybe_unused]] uint32_t wboth[2][16];
                if constexpr (!SUMS) {  // both word columns with one load per row (the sums variant has no registers to spare)
#pragma unroll
                    for (int r = 0; r < kSlice; ++r) {
                        const uint2 v2 = async::lds64(mine + r * 128 + (chunk ^ ((r & 7) << 4)));
                        wboth[0][r] = v2.x;
                        wboth[1][r] = v2.y;
                    }
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t wc[16];
#pragma unroll
                    for (int r = 0; r < kSlice; ++r) {
                        if constexpr (!SUMS) wc[r] = wboth[c][r];
                        else wc[r] = async::lds32(mine + 4 * c + r * 128 + (chunk ^ ((r & 7) << 4)));
                    }
                    uint32_t aw[16], pm[8], yw[16], cl[NCW], ch[NCW], F2;
                    x2::WordColOut o;
                    if (x2::wordcol_exponents(wc, aw, pm, F2)) {
                        x2::quantize_wordcol<W, SUMS, false>(wc, aw, pm, F2, M, yw, cl, ch, o);
                        if constexpr (SUMS) {
                            const double wl = x2::pow4_weight((F2 >> 7) & 0xFFu), wh = x2::pow4_weight(F2 >> 23);
                            e2c = fma((double)o.pe_lo, wl, e2c);
                            e2c = fma((double)o.pe_hi, wh, e2c);
                            s2c = fma((double)o.ps_lo, wl, s2c);
                            s2c = fma((double)o.ps_hi, wh, s2c);
                        }
                    } else {
                        x2::WordCol in;
#pragma unroll
                        for (int r = 0; r < 16; ++r) in.w[r] = wc[r];
                        const x2::WordColSlow so = x2::quantize_wordcol_slow<W, SUMS>(in, qp);
#pragma unroll
                        for (int k = 0; k < NCW; ++k) { cl[k] = so.cl[k]; ch[k] = so.ch[k]; }
                        o.F2 = so.F2;
                        o.micro_lo = so.micro_lo;
                        o.micro_hi = so.micro_hi;
                        if constexpr (SUMS) { e2c += so.e2; s2c += so.s2; }
                    }
                    Fb[2 * c] = (o.F2 >> 7) & 0xFFu;
                    Fb[2 * c + 1] = o.F2 >> 23;
                    Mb[2 * c] = o.micro_lo;
                    Mb[2 * c + 1] = o.micro_hi;
                    if constexpr (W % 2 == 0) {
                        // 2W bytes = one 16-byte item per (block row, column); columns swizzled by the block row
                        const uint32_t rowb = st_elems + bl * (kP2TileCols * 16);
                        const int col = 4 * lane + 2 * c;
                        async::sts128(rowb + ((col ^ (bl & 7)) * 16), make_uint4(cl[0], cl[1], cl[2], cl[3]));
                        async::sts128(rowb + (((col + 1) ^ (bl & 7)) * 16), make_uint4(ch[0], ch[1], ch[2], ch[3]));
                    } else if (i == 0) {
#pragma unroll
                        for (int k = 0; k < NCW; ++k) { cw0[2 * c][k] = cl[k]; cw0[2 * c + 1][k] = ch[k]; }
                    } else {
                        // the pair's 32 codes of a column as W words: block row 2w+1 follows 2w at bit 16 W
                        const uint32_t item = st_elems + ((warp * kP2TileCols + 4 * lane + 2 * c) * W) * 4;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t(&a)[NCW] = cw0[2 * c + h];
                            const uint32_t(&b)[NCW] = h ? ch : cl;
                            const uint32_t dst = item + h * W * 4;
#pragma unroll
                            for (int k = 0; k < W / 2; ++k) async::sts32(dst + 4 * k, a[k]);
                            async::sts32(dst + 4 * (W / 2), a[W / 2] | (b[0] << 16));
#pragma unroll
                            for (int k = 0; k < W / 2; ++k) async::sts32(dst + 4 * (W / 2 + 1 + k), __byte_perm(b[k], b[k + 1], 0x5432));
                        }
                    }
                }
                async::sts32(st_exps + bl * kP2TileCols + 4 * lane, Fb[0] | (Fb[1] << 8) | (Fb[2] << 16) | (Fb[3] << 24));
                async::sts32(st_micro + bl * kP2TileCols + 4 * lane, Mb[0] | (Mb[1] << 8) | (Mb[2] << 16) | (Mb[3] << 24));
            }
            // ---- row direction: item = 32 consecutive elements of a row (two blocks); 64 items per box ------------
            const int64_t grow0 = (int64_t)rt * kP2TileRows + bl * kSlice;  // first row of the box
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int it = lane + 32 * k, row = it >> 2, pair = it & 3;
                const uint32_t src = box + (pair >> 1) * (kP2BoxBytes / 2) + row * 128;
                const uint32_t c0 = (uint32_t)(pair & 1) << 6, sw = (uint32_t)(row & 7) << 4;
                uint4 v[4];
                if constexpr (!SUMS) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) v[g] = async::lds128(src + ((c0 + 16 * g) ^ sw));
                    if (k == 1) {
                        __syncwarp();  // every lane has read the box for the last time: refill the stage with box i of the next tile
                        if (lane == 0 && !failed && t + (int)gridDim.x < n_tiles) issue(t + gridDim.x, i, stg);
                    }
                }
                uint32_t cw[2][NCW], Fs[2], mbs[2];
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if constexpr (SUMS) {  // the sums variant has no registers to spare: one block's 32 bytes at a time
                        v[2 * s] = async::lds128(src + ((c0 + 32 * s) ^ sw));
                        v[2 * s + 1] = async::lds128(src + ((c0 + 32 * s + 16) ^ sw));
                        if (k == 1 && s == 1) {
                            __syncwarp();
                            if (lane == 0 && !failed && t + (int)gridDim.x < n_tiles) issue(t + gridDim.x, i, stg);
                        }
                    }
                    uint32_t w[8];
                    p2_words_of(v[2 * s], v[2 * s + 1], w);
                    x2::PairView pv;
                    const uint32_t F = x2::pair_view(w, pv);
                    if (F - x2::kMinF <= (uint32_t)(x2::kMaxF - x2::kMinF)) {
                        if constexpr (!SUMS) {
                            x2::pack_pair_view<W>(pv, F, cw[s], mbs[s]);
                        } else {
                            float pe, ps;
                            x2::pack_pair_view<W, true>(pv, F, cw[s], mbs[s], &pe, &ps);
                            const double wgt = x2::pow4_weight(F);
                            e2r = fma((double)pe, wgt, e2r);
                            s2r = fma((double)ps, wgt, s2r);
                        }
                        Fs[s] = F;
                    } else {
                        const x2::SlowOut o = x2::quantize_block_slow<W, SUMS>(v[2 * s], v[2 * s + 1], qp);
#pragma unroll
                        for (int q = 0; q < NCW; ++q) cw[s][q] = o.cw[q];
                        Fs[s] = o.F;
                        mbs[s] = o.micro;
                        if constexpr (SUMS) { e2r += o.e2; s2r += o.s2; }
                    }
                }
                const int64_t grow = grow0 + row;
                const int blk = ct * (kP2TileCols / 16) + 2 * pair;  // first of the item's two blocks within the row
                if constexpr (W == 8) {
                    uint4* dst = reinterpret_cast<uint4*>(rout.elems + grow * rout.ld_elems + (int64_t)blk * 16);
                    dst[0] = make_uint4(cw[0][0], cw[0][1], cw[0][2], cw[0][3]);
                    dst[1] = make_uint4(cw[1][0], cw[1][1], cw[1][2], cw[1][3]);
                } else {
                    // the item's 32 codes as W words: block 1 follows block 0 at bit 16 W
                    const uint32_t dst = st_row + row * (16 * W) + pair * 4 * W;
#pragma unroll
                    for (int q = 0; q < W / 2; ++q) async::sts32(dst + 4 * q, cw[0][q]);
                    async::sts32(dst + 4 * (W / 2), cw[0][W / 2] | (cw[1][0] << 16));
#pragma unroll
                    for (int q = 0; q < W / 2; ++q) async::sts32(dst + 4 * (W / 2 + 1 + q), __byte_perm(cw[1][q], cw[1][q + 1], 0x5432));
                }
                *reinterpret_cast<uint16_t*>(rout.exps + grow * rout.ld_exps + blk) = (uint16_t)(Fs[0] | (Fs[1] << 8));
                *reinterpret_cast<uint16_t*>(rout.micro + grow * rout.ld_micro + blk) = (uint16_t)((mbs[0] & 0xFFu) | (mbs[1] << 8));
            }
            if constexpr (W != 8) {
                __syncwarp();
                // a row's eight blocks = 16 W bytes = W vectors of 16 bytes, contiguous in the row's plane line
                for (int idx = lane; idx < kSlice * W; idx += 32) {
                    const int row = idx / W, vv = idx - row * W;
                    const uint4 q = async::lds128(st_row + row * (16 * W) + 16 * vv);
                    *reinterpret_cast<uint4*>(rout.elems + (grow0 + row) * rout.ld_elems + (int64_t)ct * (16 * W) + 16 * vv) = q;
                }
                __syncwarp();  // the staging area is free for the next box
            }
        }
        phase ^= 1;
        // ---- column planes of the tile: gather the staged items column by column ---------------------------------
        __syncthreads();
        const int64_t blk0 = (int64_t)rt * kP2TileBlocks;  // first block of the tile within a column
        for (int idx = threadIdx.x; idx < kP2TileCols * 2 * W; idx += kP2Threads) {
            const int c = idx / (2 * W), v = idx - c * (2 * W);
            uint4 q;
            if constexpr (W % 2 == 0) {
                q = async::lds128(st_elems + v * (kP2TileCols * 16) + ((c ^ (v & 7)) * 16));
            } else {
                uint32_t x4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int wd = 4 * v + k, pr = wd / W, kk = wd - pr * W;
                    x4[k] = async::lds32(st_elems + ((pr * kP2TileCols + c) * W + kk) * 4);
                }
                q = make_uint4(x4[0], x4[1], x4[2], x4[3]);
            }
            *reinterpret_cast<uint4*>(cout_.elems + ((int64_t)ct * kP2TileCols + c) * cout_.ld_elems + blk0 * 2 * W + v * 16) = q;
        }
        for (int idx = threadIdx.x; idx < kP2TileCols * 2; idx += kP2Threads) {
            const int c = idx & (kP2TileCols - 1), which = idx / kP2TileCols;
            const uint32_t src = (which ? st_micro : st_exps) + c;
            uint32_t x4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int b = 0; b < 16; ++b) x4[b >> 2] |= async::lds8(src + b * kP2TileCols) << ((b & 3) * 8);
            uint8_t* base = which ? cout_.micro + ((int64_t)ct * kP2TileCols + c) * cout_.ld_micro
                                  : cout_.exps + ((int64_t)ct * kP2TileCols + c) * cout_.ld_exps;
            *reinterpret_cast<uint4*>(base + blk0) = make_uint4(x4[0], x4[1], x4[2], x4[3]);
        }
        __syncthreads();
    }
    if constexpr (SUMS) {
        block_accumulate_sums(e2r, s2r, sums_row);
        __syncthreads();  // the reduction's scratch is reused
        block_accumulate_sums(e2c, s2c, sums_col);
    }
}

// ---- host side ----------------------------------------------------------------------------------------
template <int W, bool SUMS>
static int launch_pack2(const bf16* x, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& rout, const bdr_planes_t& cout_,
                        const QParams& qp, double* sums_row, double* sums_col, cudaStream_t st) {
    auto kern = pack2_x2_kernel<W, SUMS>;
    const size_t smem = kP2RingBytes + kP2BarBytes + P2Stage<W>::kBytes;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, kP2Threads, smem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    CUtensorMap xmap;
    if (!make_tensor_map_u16(&xmap, x, rows, cols, ld, kP2TileCols / 2, kSlice, true)) return BDR_ERR_CUDA;
    const int n_ct = (int)(cols / kP2TileCols);
    const int64_t n_tiles = (int64_t)n_ct * (rows / kP2TileRows);
    const int grid = (int)std::min<int64_t>(n_tiles, (int64_t)sm_count() * blocks_per_sm);
    kern<<<grid, kP2Threads, smem, st>>>(xmap, n_ct, (int)n_tiles, rout, cout_, qp, sums_row, sums_col, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Fast path: Table II formats, ties-to-even, whole tiles of 256 rows x 128 columns (and whole pairs of them along the
// row, so that the row-major exponent plane needs no padding), 16-byte aligned rows, tight planes (the caller checks
// tightness).  BDR_ERR_UNSUPPORTED sends the caller to two single-direction calls.
int pack2_mx_x2(const bf16* x, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t& rout, const bdr_planes_t& cout_,
                const QParams& qp, double* sums_row, double* sums_col, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || qp.rounding != BDR_ROUND_NEAREST_EVEN) return BDR_ERR_UNSUPPORTED;
    if (rows % kP2TileRows != 0 || cols % (2 * kP2TileCols) != 0) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)x % 16) || (ld * 2) % 16) return BDR_ERR_UNSUPPORTED;
    if ((int64_t)(cols / kP2TileCols) * (rows / kP2TileRows) >= (1ll << 30) || rows >= (1ll << 31) || cols >= (1ll << 31)) return BDR_ERR_UNSUPPORTED;
    if ((sums_row == nullptr) != (sums_col == nullptr)) return BDR_ERR_UNSUPPORTED;
    const bool sums = sums_row != nullptr;
    switch (qp.m) {
        case 2: return sums ? launch_pack2<3, true>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st)
                            : launch_pack2<3, false>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st);
        case 4: return sums ? launch_pack2<5, true>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st)
                            : launch_pack2<5, false>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st);
        case 7: return sums ? launch_pack2<8, true>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st)
                            : launch_pack2<8, false>(x, rows, cols, ld, rout, cout_, qp, sums_row, sums_col, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
