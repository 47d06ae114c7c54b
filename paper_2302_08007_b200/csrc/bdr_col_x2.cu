// Column-direction (axis 0) kernels for bf16 tensors in the Table II family (k1 = 16, k2 = 2, d2 = 1,
// m <= 7, ties-to-even) on packed bf16x2 arithmetic: a 32-bit word holds one row of two adjacent
// columns, and the two halves are quantized as two independent blocks by the same instructions.
//
// A CTA has eight warps; a warp works on boxes of 16 rows x 128 columns (4 KB), each fetched with one 2-D TMA
// tile load into the warp's own ring, two boxes in flight; a lane owns four adjacent columns (8 bytes
// of every row).  Dequantized values are written back over the box in shared memory and leave with one
// TMA tile store (a third stage covers the time that store needs to drain).
// When planes are written, a CTA owns tiles of 128 columns x 256 rows and warp w takes block rows 2w and
// 2w+1 of every tile.  The packed planes are column-major -- the transposed layout the backward-pass
// GEMMs read -- so codes are first staged per tile in shared memory (layouts at CStage);
// after a CTA barrier the tile's columns are gathered and each column's 16 blocks leave as one
// contiguous run (32 W code bytes, 16 exponent bytes, 16 microexponent bytes).  Without planes the
// eight warps of a CTA take eight adjacent column groups of the same 32 rows instead.
#include <algorithm>

#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;

constexpr int kCThreads = 256;
constexpr int kCWarps = kCThreads / 32;
constexpr int kCTileCols = 128;
constexpr int kCTileBlocks = 2 * kCWarps;  // 16 block rows = 256 rows
constexpr int kCTileRows = kCTileBlocks * kSlice;
constexpr int kCBoxBytes = kSlice * kCTileCols * 2;  // 4 KB
// Stages per warp: two boxes are kept in flight; with dequantized output the results are written back into
// the box they came from and leave with one TMA tile store, so a third stage is needed while it drains.
template <bool YOUT> struct CRing {
    static constexpr int kStages = YOUT ? 3 : 2;
    static constexpr int kBytes = kCWarps * kStages * kCBoxBytes;
};
constexpr int kCBarBytes = 256;

template <int W> struct CStage {
    // codes: W even: [block row 16][column 128] items of 2W bytes, columns XOR-swizzled by the block row;
    //        W odd:  per column its whole run of 8 W words (block-row pair p at word W p), column c in row
    //                (c % 4) * 32 + c / 4, rows 8 W + 1 words apart: the lanes of a warp write their k-th columns to
    //                different banks and the write-out reads a run's words without any index arithmetic
    static constexpr int kOddPitchWords = 8 * W + 1;
    static constexpr int kElemBytes = W % 2 ? kCTileCols * kOddPitchWords * 4 : kCTileBlocks * kCTileCols * 2 * W;
    static constexpr int kExpBytes = kCTileBlocks * kCTileCols;  // [block row][column]
    static constexpr int kBytes = W > 0 ? kElemBytes + 2 * kExpBytes : 0;
};

// W = 0: quantize-dequantize / sums only (any m <= 7, from qp); W = m + 1: also write the packed planes.
template <int W, bool SUMS, bool YOUT>
__global__ void __launch_bounds__(kCThreads, 2)
col_mx_x2_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap ymap, int n_col_tiles, int n_tiles,
                 bdr_planes_t out, QParams qp, double* sums, int* status) {
    using CS = CStage<W>;
    constexpr bool PACK = W > 0;
    constexpr int NCW = PACK ? (16 * W + 31) / 32 : 1;
    constexpr int S = CRing<YOUT>::kStages;
    constexpr int kCRingBytes = CRing<YOUT>::kBytes;
    extern __shared__ __align__(128) uint8_t smem[];  // ring [warp][stage][4 KB], barriers, staging
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring0 = async::smem_u32(smem) + warp * S * kCBoxBytes;
    const uint32_t bars = async::smem_u32(smem) + kCRingBytes + warp * 32;
    const uint32_t st_elems = async::smem_u32(smem) + kCRingBytes + kCBarBytes;
    const uint32_t st_exps = st_elems + CS::kElemBytes, st_micro = st_exps + CS::kExpBytes;
    const int m = PACK ? W - 1 : qp.m;

    // Where the warp's i-th box (i = 0, 1) of the CTA's t-th work unit sits.  When planes are written, a unit is
    // a tile of 256 rows x 128 columns and warp w owns block rows 2w, 2w+1 (a column's 16 blocks are staged
    // together).  Without planes nothing ties the warps together, so the eight warps take eight adjacent
    // column groups of the same 32 rows: the CTA then touches 2 KB of every row at a time instead of 256 bytes.
    auto box_origin = [&](int t, int i, int& col0, int& row0) {
        if constexpr (PACK) {
            const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
            col0 = ct * kCTileCols;
            row0 = rt * kCTileRows + (2 * warp + i) * kSlice;
        } else {
            const int g = t * kCWarps + warp, bp = g / n_col_tiles, ct = g - bp * n_col_tiles;
            col0 = ct * kCTileCols;
            row0 = (2 * bp + i) * kSlice;
        }
    };
    auto issue = [&](int t, int i, int stg) {  // lane 0 only
        int col0, row0;
        box_origin(t, i, col0, row0);
        async::mbar_expect_tx(bars + 8 * stg, kCBoxBytes);
        async::tma_load_2d(ring0 + stg * kCBoxBytes, &xmap, col0, row0, bars + 8 * stg);
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
    int stg = 0;  // stage of the current step; steps alternate between the tile's two block rows
    double e2 = 0.0, s2 = 0.0;
    bool failed = false;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
        uint32_t cw0[4][NCW];  // codes of block row 2*warp (odd W: held until the pair is complete)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int bl = 2 * warp + i;
            if (!failed && !async::mbar_wait(bars + 8 * stg, phase)) {
                async::report_timeout(status);
                failed = true;
            }
            // Packing with sums or with dequantized output are the variants with the most live registers: there the
            // second word column is loaded only when the first is done (and, without output, the stage is refilled
            // after that), which keeps 16 registers free.
            constexpr bool kLate = PACK && (SUMS || YOUT);
            uint32_t wc[2][16];
            const uint32_t mine = ring0 + stg * kCBoxBytes + lane * 8;
            if constexpr (!kLate) {
#pragma unroll
                for (int r = 0; r < kSlice; ++r) {
                    const uint2 v = async::lds64(mine + r * (kCTileCols * 2));
                    wc[0][r] = v.x;
                    wc[1][r] = v.y;
                }
                if constexpr (!YOUT) {
                    __syncwarp();  // every lane has read the stage: refill it with the same block row of the next tile
                    if (lane == 0 && !failed && t + (int)gridDim.x < n_tiles) issue(t + gridDim.x, i, stg);
                }
            }
            uint32_t Fb[4], Mb[4];
#pragma unroll
            for (int c = 0; c < 2; ++c) {  // the lane's two word columns
                if constexpr (kLate) {
#pragma unroll
                    for (int r = 0; r < kSlice; ++r) wc[c][r] = async::lds32(mine + 4 * c + r * (kCTileCols * 2));
                    if constexpr (!YOUT) {
                        if (c == 1) {
                            __syncwarp();
                            if (lane == 0 && !failed && t + (int)gridDim.x < n_tiles) issue(t + gridDim.x, i, stg);
                        }
                    }
                }
                uint32_t aw[16], pm[8], yw[16], cl[NCW], ch[NCW], F2;
                x2::WordColOut o;
                if (x2::wordcol_exponents(wc[c], aw, pm, F2)) {
                    x2::quantize_wordcol<W, SUMS, YOUT>(wc[c], aw, pm, F2, m, yw, cl, ch, o);
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
                    const x2::WordColSlow so = x2::quantize_wordcol_slow<W, SUMS>(in, qp);
#pragma unroll
                    for (int r = 0; r < 16; ++r) yw[r] = so.y[r];
#pragma unroll
                    for (int k = 0; k < NCW; ++k) { cl[k] = so.cl[k]; ch[k] = so.ch[k]; }
                    o.F2 = so.F2;
                    o.micro_lo = so.micro_lo;
                    o.micro_hi = so.micro_hi;
                    if constexpr (SUMS) { e2 += so.e2; s2 += so.s2; }
                }
                if constexpr (YOUT && kLate) {  // results over the word column's input right away
#pragma unroll
                    for (int r = 0; r < 16; ++r) async::sts32(mine + 4 * c + r * (kCTileCols * 2), yw[r]);
                } else if constexpr (YOUT) {
#pragma unroll
                    for (int r = 0; r < 16; ++r) wc[c][r] = yw[r];  // reuse the input registers for the output rows
                }
                if constexpr (PACK) {
                    Fb[2 * c] = (o.F2 >> 7) & 0xFFu;
                    Fb[2 * c + 1] = o.F2 >> 23;
                    Mb[2 * c] = o.micro_lo;
                    Mb[2 * c + 1] = o.micro_hi;
                    if constexpr (W % 2 == 0) {
                        // 2W bytes = one 16-byte item per (block row, column); columns swizzled by the block row
                        const uint32_t rowb = st_elems + bl * (kCTileCols * 16);
                        const int col = 4 * lane + 2 * c;
                        async::sts128(rowb + ((col ^ (bl & 7)) * 16), make_uint4(cl[0], cl[1], cl[2], cl[3]));
                        async::sts128(rowb + (((col + 1) ^ (bl & 7)) * 16), make_uint4(ch[0], ch[1], ch[2], ch[3]));
                    } else if (i == 0) {
#pragma unroll
                        for (int k = 0; k < NCW; ++k) { cw0[2 * c][k] = cl[k]; cw0[2 * c + 1][k] = ch[k]; }
                    } else {
                        // the pair's 32 codes of a column as W words: block row 2w+1 follows 2w at bit 16 W
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t(&a)[NCW] = cw0[2 * c + h];
                            const uint32_t(&b)[NCW] = h ? ch : cl;
                            const uint32_t dst = st_elems + (((2 * c + h) * 32 + lane) * CS::kOddPitchWords + warp * W) * 4;
#pragma unroll
                            for (int k = 0; k < W / 2; ++k) async::sts32(dst + 4 * k, a[k]);
                            async::sts32(dst + 4 * (W / 2), a[W / 2] | (b[0] << 16));
#pragma unroll
                            for (int k = 0; k < W / 2; ++k) async::sts32(dst + 4 * (W / 2 + 1 + k), __byte_perm(b[k], b[k + 1], 0x5432));
                        }
                    }
                }
            }
            if constexpr (YOUT) {
                // results over the box's input, then one tile store; the stage of the previous step (whose store
                // has been read out by then) takes the box two steps ahead
                if constexpr (!kLate) {
#pragma unroll
                    for (int r = 0; r < kSlice; ++r) async::sts64(mine + r * (kCTileCols * 2), wc[0][r], wc[1][r]);
                }
                async::fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    int col0, row0;
                    box_origin(t, i, col0, row0);
                    async::tma_store_2d(&ymap, col0, row0, ring0 + stg * kCBoxBytes);
                    async::bulk_commit();
                    async::bulk_wait_read<1>();
                    if (!failed && t + (int)gridDim.x < n_tiles) issue(t + gridDim.x, i, stg + 2 >= S ? stg + 2 - S : stg + 2);
                }
            }
            if constexpr (PACK) {
                async::sts32(st_exps + bl * kCTileCols + 4 * lane, Fb[0] | (Fb[1] << 8) | (Fb[2] << 16) | (Fb[3] << 24));
                async::sts32(st_micro + bl * kCTileCols + 4 * lane, Mb[0] | (Mb[1] << 8) | (Mb[2] << 16) | (Mb[3] << 24));
            }
            if (++stg == S) { stg = 0; phase ^= 1; }
        }
        if constexpr (PACK) {
            __syncthreads();
            // codes: column c of the tile owns 32 W contiguous bytes of its plane line = 2W vectors of 16 bytes
            const int64_t blk0 = (int64_t)rt * kCTileBlocks;  // first block of the tile within a column
            for (int idx = threadIdx.x; idx < kCTileCols * 2 * W; idx += kCThreads) {
                const int c = idx / (2 * W), v = idx - c * (2 * W);
                uint4 q;
                if constexpr (W % 2 == 0) {
                    // vector v covers bytes 16v .. 16v+15 of the run: W = 8 -> exactly block row v
                    q = async::lds128(st_elems + v * (kCTileCols * 16) + ((c ^ (v & 7)) * 16));
                } else {
                    // column c's run is kept whole in row (c % 4) * 32 + c / 4, rows an odd number of words apart
                    const uint32_t src = st_elems + ((((c & 3) * 32 + (c >> 2)) * CS::kOddPitchWords) + 4 * v) * 4;
                    q = make_uint4(async::lds32(src), async::lds32(src + 4), async::lds32(src + 8), async::lds32(src + 12));
                }
                *reinterpret_cast<uint4*>(out.elems + ((int64_t)ct * kCTileCols + c) * out.ld_elems + blk0 * 2 * W + v * 16) = q;
            }
            // exponents and microexponents: 16 bytes per column each
            for (int idx = threadIdx.x; idx < kCTileCols * 2; idx += kCThreads) {
                const int c = idx & (kCTileCols - 1), which = idx / kCTileCols;
                const uint32_t src = (which ? st_micro : st_exps) + c;
                uint32_t x4[4] = {0, 0, 0, 0};
#pragma unroll
                for (int b = 0; b < 16; ++b) x4[b >> 2] |= async::lds8(src + b * kCTileCols) << ((b & 3) * 8);
                uint8_t* base = which ? out.micro + ((int64_t)ct * kCTileCols + c) * out.ld_micro
                                      : out.exps + ((int64_t)ct * kCTileCols + c) * out.ld_exps;
                *reinterpret_cast<uint4*>(base + blk0) = make_uint4(x4[0], x4[1], x4[2], x4[3]);
            }
            __syncthreads();
        }
    }
    if (YOUT && lane == 0) async::bulk_wait_all();
    if (SUMS) block_accumulate_sums(e2, s2, sums);
}

// ---- host side ----------------------------------------------------------------------------------------
template <int W, bool SUMS, bool YOUT>
static int launch_col_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                         const QParams& qp, double* sums, cudaStream_t st) {
    auto kern = col_mx_x2_kernel<W, SUMS, YOUT>;
    const size_t smem = CRing<YOUT>::kBytes + kCBarBytes + CStage<W>::kBytes;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, kCThreads, smem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    CUtensorMap xmap, ymap;
    if (!make_tensor_map_u16(&xmap, x, rows, cols, ld, kCTileCols, kSlice)) return BDR_ERR_CUDA;
    if (!make_tensor_map_u16(&ymap, y ? y : x, rows, cols, ld, kCTileCols, kSlice)) return BDR_ERR_CUDA;
    const int n_ct = (int)(cols / kCTileCols);
    const int64_t n_tiles = (int64_t)n_ct * (rows / kCTileRows);
    bdr_planes_t pl = {};
    if (out) pl = *out;
    const int grid = (int)std::min<int64_t>(n_tiles, (int64_t)sm_count() * blocks_per_sm);
    kern<<<grid, kCThreads, smem, st>>>(xmap, ymap, n_ct, (int)n_tiles, pl, qp, sums, status);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <int W>
static int col_x2_flags(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                        const QParams& qp, double* sums, cudaStream_t st) {
    if (sums) return y ? launch_col_x2<W, true, true>(x, y, rows, cols, ld, out, qp, sums, st)
                       : launch_col_x2<W, true, false>(x, y, rows, cols, ld, out, qp, sums, st);
    if (y) return launch_col_x2<W, false, true>(x, y, rows, cols, ld, out, qp, sums, st);
    if constexpr (W > 0) return launch_col_x2<W, false, false>(x, y, rows, cols, ld, out, qp, sums, st);
    return BDR_ERR_NULL;
}

// Fast path: whole tiles of 256 rows x 128 columns, 16-byte aligned rows; planes (if any) tight.
// BDR_ERR_UNSUPPORTED sends the caller to the generic column kernels.
int quant_colwise_mx_x2(const bf16* x, bf16* y, int64_t rows, int64_t cols, int64_t ld, const bdr_planes_t* out,
                        const QParams& qp, double* sums, cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1 || qp.m > 7 || qp.rounding != BDR_ROUND_NEAREST_EVEN) return BDR_ERR_UNSUPPORTED;
    if (rows % kCTileRows != 0 || cols % kCTileCols != 0) return BDR_ERR_UNSUPPORTED;
    if ((((uintptr_t)x | (uintptr_t)y) % 16) || (ld * 2) % 16) return BDR_ERR_UNSUPPORTED;
    if ((int64_t)(cols / kCTileCols) * (rows / kCTileRows) >= (1ll << 30) || rows >= (1ll << 31) || cols >= (1ll << 31)) return BDR_ERR_UNSUPPORTED;
    if (!out) return col_x2_flags<0>(x, y, rows, cols, ld, out, qp, sums, st);
    switch (qp.m) {
        case 2: return col_x2_flags<3>(x, y, rows, cols, ld, out, qp, sums, st);
        case 4: return col_x2_flags<5>(x, y, rows, cols, ld, out, qp, sums, st);
        case 7: return col_x2_flags<8>(x, y, rows, cols, ld, out, qp, sums, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
