// Column-direction (axis 0) unpack to bf16 for the Table II family on packed bf16x2 arithmetic: the
// mirror image of the column packing kernel in bdr_col_x2.cu.  A CTA (eight warps) owns tiles of 64
// columns x 256 rows.  The packed planes are column-major, so a tile's input is, per column, one run
// of 32 W code bytes, 16 exponent bytes and 16 microexponent bytes; all threads fetch these runs with
// coalesced 16-byte cp.async copies into a double-buffered staging area (the next tile is in flight
// while the current one is decoded).  Warp w then decodes block rows 2w and 2w+1: a lane owns one word
// column (two adjacent columns, decoded in the two halves of a word), the warp's 16 x 64 results go
// through a 2 KB box in shared memory and leave with one 2-D TMA tile store per block row.
// One word column per lane keeps the kernel at 64 registers, so four CTAs share an SM, and 64-column
// tiles give an 8192 x 8192 tensor 4096 tiles, which divide evenly over them.  Measured on that tensor
// the time does not depend on how the results leave (plain stores or tile stores), on the number of
// resident CTAs between two and five, or on the length of the input runs: the mix of 16 KB-strided
// reads and writes holds it at about 5.2 TB/s.
#include <algorithm>

#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;

constexpr int kUCThreads = 256;
constexpr int kUCWarps = kUCThreads / 32;
constexpr int kUCTileCols = 64;
constexpr int kUCTileBlocks = 2 * kUCWarps;  // 16 block rows
constexpr int kUCTileRows = kUCTileBlocks * kSlice;

template <int W> struct UCStage {
    static constexpr int kPitch = kUCTileBlocks * 2 * W + 16;  // code bytes of one column, padded so columns spread over banks
    // Column c is kept in row (c % 2) * 32 + c / 2: the lanes of a warp (two adjacent columns each) then read
    // from 32 consecutive rows, i.e. from different banks, when they fetch their even or their odd column.
    __host__ __device__ static constexpr int row_of(int c) { return (c & 1) * 32 + (c >> 1); }
    static constexpr int kElemBytes = kUCTileCols * kPitch;
    static constexpr int kExpBytes = kUCTileCols * 16;
    static constexpr int kBytes = kElemBytes + 2 * kExpBytes;
};

__device__ __forceinline__ void uc_cp16(uint32_t smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}

constexpr int kUCBoxBytes = kSlice * 64 * 2;  // a warp's output box: 16 rows x 64 columns

template <int W, int CTAS>
__global__ void __launch_bounds__(kUCThreads, CTAS)
unpack_col_x2_kernel(bdr_planes_t in, const __grid_constant__ CUtensorMap ymap, int n_col_tiles, int n_tiles) {
    using ST = UCStage<W>;
    extern __shared__ __align__(128) uint8_t smem[];  // two staging buffers (codes | exponents | microexponents), output boxes
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t base = async::smem_u32(smem);
    const uint32_t obox = base + 2 * ST::kBytes + warp * kUCBoxBytes;
    auto fetch = [&](int t, int buf) {
        const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
        const int64_t blk0 = (int64_t)rt * kUCTileBlocks;
        const uint32_t b = base + buf * ST::kBytes;
        for (int idx = threadIdx.x; idx < kUCTileCols * 2 * W; idx += kUCThreads) {
            const int c = idx / (2 * W), v = idx - c * (2 * W);
            uc_cp16(b + ST::row_of(c) * ST::kPitch + v * 16, in.elems + ((int64_t)ct * kUCTileCols + c) * in.ld_elems + blk0 * 2 * W + v * 16);
        }
        for (int idx = threadIdx.x; idx < kUCTileCols * 2; idx += kUCThreads) {
            const int c = idx & (kUCTileCols - 1), which = idx / kUCTileCols;
            const uint8_t* src = which ? in.micro + ((int64_t)ct * kUCTileCols + c) * in.ld_micro
                                       : in.exps + ((int64_t)ct * kUCTileCols + c) * in.ld_exps;
            uc_cp16(b + ST::kElemBytes + which * ST::kExpBytes + ST::row_of(c) * 16, src + blk0);
        }
    };
    int buf = 0;
    if ((int)blockIdx.x < n_tiles) fetch(blockIdx.x, 0);
    cp_async_commit();
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        if (t + (int)gridDim.x < n_tiles) fetch(t + gridDim.x, buf ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();  // the tile's bytes were fetched by all threads
        const int rt = t / n_col_tiles, ct = t - rt * n_col_tiles;
        const uint32_t b = base + buf * ST::kBytes;
        {
            uint32_t s[2][W], Fp[2], mp[2];  // the lane's word column: two adjacent columns
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int col = 2 * lane + c;
                if constexpr (W == 8) {
                    const uint32_t src = b + ST::row_of(col) * ST::kPitch + warp * 4 * W;
                    const uint4 a0 = async::lds128(src), a1 = async::lds128(src + 16);
                    s[c][0] = a0.x; s[c][1] = a0.y; s[c][2] = a0.z; s[c][3] = a0.w;
                    s[c][4] = a1.x; s[c][5] = a1.y; s[c][6] = a1.z; s[c][7] = a1.w;
                } else {
                    // W words at word offset W * warp of the column's row.  The row pitch is a multiple of 16 bytes, so
                    // 32-bit loads at the same offset would put the 32 lanes (32 rows) on only eight banks; instead
                    // the two aligned 16-byte chunks that contain the words are loaded (conflict-free) and the W
                    // words are picked out: they start at word (W * warp) mod 4 of the eight, the same for the warp.
                    const uint32_t first = b + ST::row_of(col) * ST::kPitch + (((W * warp) >> 2) << 4);
                    const uint4 a0 = async::lds128(first), a1 = async::lds128(first + 16);
                    const uint32_t L[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                    switch ((W * warp) & 3) {
                        case 0:
#pragma unroll
                            for (int k = 0; k < W; ++k) s[c][k] = L[k];
                            break;
                        case 1:
#pragma unroll
                            for (int k = 0; k < W; ++k) s[c][k] = L[(1 + k) & 7];
                            break;
                        case 2:
#pragma unroll
                            for (int k = 0; k < W; ++k) s[c][k] = L[(2 + k) & 7];
                            break;
                        default:
#pragma unroll
                            for (int k = 0; k < W; ++k) s[c][k] = L[(3 + k) & 7];
                            break;
                    }
                }
                Fp[c] = async::lds16(b + ST::kElemBytes + ST::row_of(col) * 16 + 2 * warp);
                mp[c] = async::lds16(b + ST::kElemBytes + ST::kExpBytes + ST::row_of(col) * 16 + 2 * warp);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {  // block rows 2*warp and 2*warp + 1
                uint32_t yw[16];
                const uint32_t F_lo = (Fp[0] >> (8 * i)) & 0xFFu, F_hi = (Fp[1] >> (8 * i)) & 0xFFu;
                const uint32_t m_lo = (mp[0] >> (8 * i)) & 0xFFu, m_hi = (mp[1] >> (8 * i)) & 0xFFu;
                if ((F_lo - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF)) && (F_hi - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF))) {
                    x2::decode_wordcol<W>(s[0], s[1], i, (F_lo << 7) | (F_hi << 23), m_lo | (m_hi << 16), yw);
                } else {
                    x2::TwoBlocks<W> lo, hi;
#pragma unroll
                    for (int k = 0; k < W; ++k) { lo.s[k] = s[0][k]; hi.s[k] = s[1][k]; }
                    const x2::TwoBlocksOut o = x2::decode_wordcol_slow<W>(lo, hi, i, F_lo, F_hi, m_lo, m_hi);
#pragma unroll
                    for (int r = 0; r < 16; ++r) yw[r] = o.y[r];
                }
                // the 16 x 64 box goes through the warp's shared-memory box and leaves with one tile store
                if (lane == 0) async::bulk_wait_read<0>();  // the previous box has been read out
                __syncwarp();
#pragma unroll
                for (int r = 0; r < kSlice; ++r) async::sts32(obox + r * 128 + 4 * lane, yw[r]);
                async::fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    async::tma_store_2d(&ymap, ct * kUCTileCols, rt * kUCTileRows + (2 * warp + i) * kSlice, obox);
                    async::bulk_commit();
                }
            }
        }
        __syncthreads();  // everyone is done with this buffer before it is refilled
        buf ^= 1;
    }
    if (lane == 0) async::bulk_wait_all();
}

template <int W, int CTAS>
static int launch_unpack_col_x2(const bdr_planes_t& in, bf16* y, int64_t rows, int64_t cols, int64_t ld, cudaStream_t st) {
    auto kern = unpack_col_x2_kernel<W, CTAS>;
    const size_t smem = 2 * UCStage<W>::kBytes + kUCWarps * kUCBoxBytes;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, kUCThreads, smem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    CUtensorMap ymap;
    if (!make_tensor_map_u16(&ymap, y, rows, cols, ld, 64, kSlice)) return BDR_ERR_CUDA;
    const int n_ct = (int)(cols / kUCTileCols);
    const int64_t n_tiles = (int64_t)n_ct * (rows / kUCTileRows);
    const int grid = (int)std::min<int64_t>(n_tiles, (int64_t)sm_count() * blocks_per_sm);
    kern<<<grid, kUCThreads, smem, st>>>(in, ymap, n_ct, (int)n_tiles);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Whole tiles of 256 rows x 64 columns, 16-byte aligned output rows.
int unpack_colwise_mx_x2(const bdr_planes_t& in, bf16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                         cudaStream_t st) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1) return BDR_ERR_UNSUPPORTED;
    if (rows % kUCTileRows != 0 || cols % kUCTileCols != 0 || rows == 0 || cols == 0) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)y % 16) || (ld * 2) % 16) return BDR_ERR_UNSUPPORTED;
    if ((int64_t)(cols / kUCTileCols) * (rows / kUCTileRows) >= (1ll << 30) || rows >= (1ll << 31) || cols >= (1ll << 31)) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {  // staging buffers and CTAs per SM as measured: four CTAs of 64 registers, three for the widest codes
        case 2: return launch_unpack_col_x2<3, 4>(in, y, rows, cols, ld, st);
        case 4: return launch_unpack_col_x2<5, 4>(in, y, rows, cols, ld, st);
        case 7: return launch_unpack_col_x2<8, 3>(in, y, rows, cols, ld, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
