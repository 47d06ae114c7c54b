// Block-scaled 8-bit GEMM for MX4 / MX6 operands that the re-encoding kernel has written as E4M3
// elements with one power-of-two scale byte per 32 elements along K (bdr_reencode_f8.cu): C = A * B^T on
// tcgen05.mma.kind::mxf8f6f4.block_scale, which multiplies the scales into the products in hardware and runs at
// twice the bf16 rate.  Every product and scale is exact; only the fp32 accumulation rounds.
//
// Same structure as the bf16 kernel in mx_gemm_dense.cuh (persistent, one cluster of two CTAs per SM pair,
// 256 x 256 tiles of C), with these differences:
//   * a K step is 128 elements (128-byte rows, 128-byte swizzle), four MMAs of K = 32;
//   * every stage also carries the scale atoms of its K chunk -- 512 bytes for this CTA's 128 rows of A
//     and 1024 bytes for all 256 rows of the B tile (each CTA's tensor memory needs the scales of every
//     column it accumulates) -- fetched with plain bulk copies on the stage's barrier; a warp of its own in
//     the leader CTA copies them to the tensor memory of both CTAs (tcgen05.cp, 32 lanes x 128 bits
//     replicated over the four lane quarters) as soon as the stage has landed and commits to a
//     "scales ready" barrier that the MMA thread waits on (issued from the MMA thread itself the three copies
//     per K step cost 17 % of the kernel: they serialise with its MMAs; from another thread they overlap);
//     the MMA picks the scale byte of its K = 32 slice with the scale-factor id in the instruction descriptor;
//   * tensor memory holds one 256-column accumulator plus 12 scale columns per stage, so the epilogue
//     does not overlap the next tile's main loop through a second buffer; instead each epilogue warp
//     pulls its 32 x 128 block into registers, releases the accumulator, and only then stores;
//   * when the last round of tiles would keep at most half of the clusters busy, each of its tiles is
//     computed as two halves of the K range by two clusters that add (red.global.add) into a tile the
//     re-encoding launch has cleared.
// The kernel does nothing when *gate is non-zero (the operands were not representable).
// Every wait is bounded.  (textually included by mx_gemm.cu after mx_gemm_dense.cuh)
#pragma once

namespace bdr {

constexpr int kFBK = 128;                                   // K elements (bytes) per stage
constexpr int kFStages = 6;
constexpr int kFTileBytes = 2 * kPairRows * kFBK;           // A 16 KB + B half 16 KB
constexpr int kFSfaBytes = 512, kFSfbBytes = 1024;
constexpr int kFStageBytes = kFTileBytes + 2048;            // tiles, then scales of A, then scales of B (1024-byte multiple)
constexpr int kFTxBytes = kFTileBytes + kFSfaBytes + kFSfbBytes;
constexpr int kFEpiWarps = 8;
constexpr int kFThreads = (3 + kFEpiWarps) * 32;            // producer, MMA / relay, 8 epilogue warps, scale copier
constexpr int kFCopyWarp = 2 + kFEpiWarps;
constexpr size_t kFSmemBytes = (size_t)kFStages * kFStageBytes + 1024 /*bookkeeping*/ + 1024 /*alignment*/;
constexpr uint32_t kFSfCol0 = 256;                          // first scale column in tensor memory
constexpr uint32_t kFSfColsPerStage = 12;                   // 4 (A: 128 rows) + 8 (B: 256 rows)

struct F8Bars {
    uint64_t full[kFStages], full_local[kFStages], empty[kFStages], sf_ready[kFStages], tmem_full, tmem_empty;
    uint32_t tmem_base;
    int failed;
};

struct F8Maps {
    CUtensorMap a, b;  // u8 [rows, K], box 128 x 128, 128-byte swizzle
};

// Instruction descriptor of kind::mxf8f6f4.block_scale: A = B = E4M3 (format 0), both K-major, N = 256
// (bits 17-22, N / 8), E8M0 scales (bit 23), M = 256 over the CTA pair (bits 24-28, M / 16); the
// scale-factor ids of A (bits 29-30) and B (bits 4-5) select the byte of the scale column.
constexpr uint32_t kF8InstrDesc = ((uint32_t)(256 >> 3) << 17) | (1u << 23) | ((uint32_t)(256 >> 4) << 24);

// Shared-memory descriptor of a scale atom for tcgen05.cp: 32 rows of 16 bytes, no swizzle, 8-row groups
// 128 bytes apart.
__device__ __forceinline__ uint64_t make_sf_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;            // leading byte offset (a single 16-byte column: unused)
    d |= (uint64_t)(128 >> 4) << 32;   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;            // descriptor version of this architecture
    return d;
}
__device__ __forceinline__ void sf_copy2(uint32_t tmem_dst, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(tmem_dst), "l"(desc) : "memory");
}
__device__ __forceinline__ void umma_commit2_leader(uint64_t* bar) {  // arrives on the leader CTA's barrier only
    const uint16_t mask = 1;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void umma2_mxf8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate,
                                           uint32_t tmem_sfa, uint32_t tmem_sfb) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(tmem_sfa), "r"(tmem_sfb)
        : "memory");
}
__device__ __forceinline__ void bulk_load_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kFThreads, 1)
mxf8_gemm_pair_kernel(const __grid_constant__ F8Maps maps, const uint8_t* sf_a, const uint8_t* sf_b, int tiles_m, int tiles_n, int band_rows, int nk,
                      int tiles_full, int n_items, float* c, int64_t ldc, const int* gate) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* stages = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    F8Bars& bars = *reinterpret_cast<F8Bars*>(stages + kFStages * kFStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    // Work items: the first tiles_full tiles with their whole K range (a multiple of the cluster count: whole
    // rounds), then every remaining tile as two items of half the K range each, which add their results into a
    // zeroed C tile -- so a last round that would keep less than half of the clusters busy takes half as long.
    auto item_of = [&](int i, int& t, int& k0, int& cnt, bool& add) {
        if (i < tiles_full) { t = i; k0 = 0; cnt = nk; add = false; }
        else { const int j = i - tiles_full; t = tiles_full + (j >> 1); cnt = nk >> 1; k0 = (j & 1) * cnt; add = true; }
    };
    const int64_t row_tiles_a = (int64_t)tiles_m * 2, row_tiles_b = (int64_t)tiles_n * 2;  // 128-row tiles of the scale atoms

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFStages; ++s) {
            mbar_init(&bars.full[s], 2);        // leader: its own bytes (arrive.expect_tx) + the peer's relay
            mbar_init(&bars.full_local[s], 1);  // peer: its own bytes
            mbar_init(&bars.empty[s], 1);       // multicast commit of the MMAs that read the stage
            mbar_init(&bars.sf_ready[s], 1);    // leader: commit of the stage's scale copies
        }
        mbar_init(&bars.tmem_full, 1);                  // multicast commit after a tile's last K step
        mbar_init(&bars.tmem_empty, 2 * kFEpiWarps);    // leader: every epilogue warp of both CTAs
        bars.failed = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc2_cols(&bars.tmem_base, 512);  // 256 accumulator columns + 72 scale columns
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars.tmem_base;

    // Everything above touched no global memory: under a programmatic dependent launch it overlaps the tail of the
    // re-encoding kernel.  From here on the operands, the cleared tiles of C and the gate are needed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const bool open = !(gate && *gate != 0);  // the same for every thread of the grid

    if (!open) {
        // the operands were not representable: nothing to do but to give the tensor memory back
    } else if (warp == 0) {
        // ---------------- producer: operand tiles by TMA, scale atoms by bulk copy ----------------
        if (lane == 0) {
            uint64_t* const my_full = rank == 0 ? bars.full : bars.full_local;
            bool ok = true;
            uint32_t it = 0;  // running K-step count across tiles
            for (int i = cluster_id; i < n_items && ok; i += n_clusters) {
                int t, k0, cnt;
                bool add;
                item_of(i, t, k0, cnt, add);
                int tm, tn;
                gemm_tile_coords(t, tiles_m, tiles_n, band_rows, tm, tn);
                const int row_a = (tm * 2 + (int)rank) * kPairRows, row_b = (tn * 2 + (int)rank) * kPairRows;
                for (int kk = k0; kk < k0 + cnt; ++kk, ++it) {
                    const int stage = it % kFStages;
                    if (it >= kFStages) {
                        ok = mbar_wait(&bars.empty[stage], ((it / kFStages) - 1) & 1);
                        if (!ok) break;
                    }
                    uint8_t* dst = stages + stage * kFStageBytes;
                    mbar_expect_tx(&my_full[stage], kFTxBytes);
                    tma_load_2d(dst, &maps.a, kk * kFBK, row_a, &my_full[stage]);
                    tma_load_2d(dst + kPairRows * kFBK, &maps.b, kk * kFBK, row_b, &my_full[stage]);
                    bulk_load_g2s(dst + kFTileBytes, sf_a + ((int64_t)kk * row_tiles_a + tm * 2 + (int)rank) * 512, kFSfaBytes,
                                  &my_full[stage]);
                    bulk_load_g2s(dst + kFTileBytes + kFSfaBytes, sf_b + ((int64_t)kk * row_tiles_b + tn * 2) * 512, kFSfbBytes,
                                  &my_full[stage]);
                }
            }
            if (!ok) bars.failed = 1;
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            uint32_t it = 0;
            if (rank == 0) {
                // ---------------- MMA issuer (leader CTA) ----------------
                int tcount = 0;
                for (int i = cluster_id; i < n_items && ok; i += n_clusters, ++tcount) {
                    int t, k0, cnt;
                    bool add;
                    item_of(i, t, k0, cnt, add);
                    if (tcount >= 1) {  // the epilogues of both CTAs hold the previous tile in registers
                        ok = mbar_wait_cluster(&bars.tmem_empty, (tcount - 1) & 1);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    for (int kk = 0; kk < cnt; ++kk, ++it) {
                        const int stage = it % kFStages;
                        ok = mbar_wait_cluster(&bars.sf_ready[stage], (it / kFStages) & 1);  // data landed, scales copied
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sa = smem_u32(stages + stage * kFStageBytes);
                        const uint32_t tsfa = tmem_base + kFSfCol0 + (uint32_t)stage * kFSfColsPerStage, tsfb = tsfa + 4;
                        const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + kPairRows * kFBK);
#pragma unroll
                        for (int k = 0; k < kFBK / 32; ++k)  // 32 bytes of K per MMA; scale byte k of the columns
                            umma2_mxf8(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k),
                                       kF8InstrDesc | ((uint32_t)k << 29) | ((uint32_t)k << 4), (kk | k) != 0, tsfa, tsfb);
                        umma_commit2(&bars.empty[stage]);
                    }
                    if (ok) umma_commit2(&bars.tmem_full);
                }
            } else {
                // ---------------- relay (peer CTA): "my half of the stage has landed" ----------------
                for (int i = cluster_id; i < n_items && ok; i += n_clusters) {
                    int t, k0, cnt;
                    bool add;
                    item_of(i, t, k0, cnt, add);
                    for (int kk = 0; kk < cnt; ++kk, ++it) {
                        const int stage = it % kFStages;
                        ok = mbar_wait(&bars.full_local[stage], (it / kFStages) & 1);
                        if (!ok) break;
                        mbar_arrive_cluster(&bars.full[stage], 0);
                    }
                }
            }
            if (!ok) bars.failed = 1;
        }
        __syncwarp();
        tc_fence_before();
    } else if (warp == kFCopyWarp) {
        // ---------------- scale copier (leader CTA): shared memory -> tensor memory of both CTAs ----------------
        if (lane == 0 && rank == 0) {
            bool ok = true;
            uint32_t it = 0;
            for (int i = cluster_id; i < n_items && ok; i += n_clusters) {
                int t, k0, cnt;
                bool add;
                item_of(i, t, k0, cnt, add);
                for (int kk = 0; kk < cnt; ++kk, ++it) {
                    const int stage = it % kFStages;
                    // (the stage's previous MMAs are done: the producer refilled it only after their commit)
                    ok = mbar_wait_cluster(&bars.full[stage], (it / kFStages) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sf = smem_u32(stages + stage * kFStageBytes) + kFTileBytes;
                    const uint32_t tsfa = tmem_base + kFSfCol0 + (uint32_t)stage * kFSfColsPerStage;
                    sf_copy2(tsfa, make_sf_desc(sf));
                    sf_copy2(tsfa + 4, make_sf_desc(sf + kFSfaBytes));
                    sf_copy2(tsfa + 8, make_sf_desc(sf + kFSfaBytes + 512));
                    umma_commit2_leader(&bars.sf_ready[stage]);
                }
            }
            if (!ok) bars.failed = 1;
        }
        __syncwarp();
        tc_fence_before();
    } else {
        // ---------------- epilogue: this CTA's 128 x 256 block of each tile ----------------
        const int ew = warp - 2;
        const int lane_base = (warp & 3) * 32;     // the tensor-memory lanes this warp may read
        const int col_base = (ew >> 2) * 128;      // two warps share a lane quarter: 128 columns each
        bool ok = true;
        int tcount = 0;
        for (int i = cluster_id; i < n_items; i += n_clusters, ++tcount) {
            int t, k0, cnt;
            bool add;
            item_of(i, t, k0, cnt, add);
            ok = ok && mbar_wait(&bars.tmem_full, tcount & 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            int tm, tn;
            gemm_tile_coords(t, tiles_m, tiles_n, band_rows, tm, tn);
            float* crow = c + ((int64_t)(tm * 2 + (int)rank) * kPairRows + lane_base + lane) * ldc + (int64_t)tn * 256 + col_base;
            uint32_t v[4][32];
#pragma unroll
            for (int q = 0; q < 4; ++q)
                tmem_ld32_nowait(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(col_base + 32 * q), v[q]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(&bars.tmem_empty, 0);  // the next tile may overwrite the accumulator
            if (!add) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4*>(crow + 32 * q + 4 * j) = make_uint4(v[q][4 * j], v[q][4 * j + 1], v[q][4 * j + 2], v[q][4 * j + 3]);
            } else {  // half of the K range: add to the zeroed tile (two terms, so the order does not matter)
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        red_add_v4(crow + 32 * q + 4 * j, v[q][4 * j], v[q][4 * j + 1], v[q][4 * j + 2], v[q][4 * j + 3]);
            }
        }
        if (!ok) bars.failed = 1;
        tc_fence_before();
    }
    __syncthreads();
    cluster_sync_all();  // the peer may still be signalling this CTA's barriers
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, 512);
    }
    if (threadIdx.x == 0 && bars.failed) atomicExch(&g_gemm_status, (int)BDR_ERR_TIMEOUT);
}

// Clears `z.count` tiles of 256 x 256 floats (for callers of the GEMM kernel that do not come through the re-encoding
// launch, which clears them on the side); grid (z.count, 4), 256 threads.
static bool make_f8_map(CUtensorMap* out, const void* base, int64_t rows, int64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K};
    const cuuint32_t box[2] = {(cuuint32_t)kFBK, (cuuint32_t)kPairRows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// How the tiles of an M x N product are handed out: n_clusters clusters, tiles_full tiles with their whole K
// range, the remaining tiles (fewer than half the cluster count) in two halves of K each.
using F8Plan = GemmPlan;
static F8Plan plan_gemm_f8(int64_t M, int64_t N, int64_t K) { return plan_gemm(M, N, K / kFBK, (M + N) * K); }

// a_e4m3 [M, K], b_e4m3 [N, K] bytes, contiguous; scale atoms ordered [K / 128][rows / 128][512];
// M, N multiples of 256, K a multiple of 128.  The tiles plan.tiles_full .. of C must hold zeros.
static int launch_gemm_f8(const uint8_t* a_e4m3, const uint8_t* b_e4m3, const uint8_t* sf_a, const uint8_t* sf_b, int64_t M, int64_t N,
                          int64_t K, const F8Plan& plan, float* c, int64_t ldc, const int* gate, cudaStream_t st) {
    static PerDevice once;
    if (once.get(current_device(), [&]() -> int {  // no occupancy query: cluster kernel, one CTA per SM
            return cudaFuncSetAttribute(mxf8_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFSmemBytes) == cudaSuccess ? 1 : 0;
        }) < 1)
        return BDR_ERR_CUDA;
    F8Maps maps;
    if (!make_f8_map(&maps.a, a_e4m3, M, K) || !make_f8_map(&maps.b, b_e4m3, N, K)) return BDR_ERR_CUDA;
    // programmatic dependent launch: the kernel may start while the re-encoding kernel before it in the stream is
    // draining; it waits (griddepcontrol.wait) before it reads anything that kernel wrote
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * plan.n_clusters));
    cfg.blockDim = dim3(kFThreads);
    cfg.dynamicSmemBytes = kFSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, mxf8_gemm_pair_kernel, maps, sf_a, sf_b, plan.tiles_m, plan.tiles_n, plan.band_rows, (int)(K / kFBK),
                                             plan.tiles_full, plan.n_items, c, ldc, gate);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

}  // namespace bdr
