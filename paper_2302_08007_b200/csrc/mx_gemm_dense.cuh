// Second phase of the two-phase mx_gemm: C = A * B^T for bf16 operands that the unpack kernels have
// written to a caller-provided workspace.  Decoding inside the GEMM repeats the decode of every
// operand row once per tile of the other dimension (16 times at 4096^3); decoding once to bf16 costs
// two extra passes over the operands and lets the GEMM itself run from TMA.
//
// Persistent kernel, one cluster of two CTAs per SM pair; a cluster walks over 256 x 256 tiles of C.
//   warp 0   : one lane issues the TMA loads of this CTA's 128 rows of A and its 128-row half of the B
//              tile (boxes of 64 K elements, 128-byte swizzle) into a six-stage ring
//   warp 1   : leader CTA: one lane issues tcgen05.mma.cta_group::2 (M 256, N 256, K 16) into one of
//              two accumulator buffers in tensor memory (256 fp32 columns each) and commits (multicast)
//              to free the stage in both CTAs and, after the last K step, to hand the buffer to the
//              epilogue;  peer CTA: relays "my stage is full" to the leader's barrier
//   warps 2-9: epilogue, tcgen05.ld of the CTA's 128 x 256 block and 16-byte stores, overlapping the
//              next tile's main loop through the second accumulator buffer
// When the last round of tiles would keep at most half of the clusters busy (4096^3: 256 tiles on 74 clusters leave 34), each
// of its tiles is computed as two halves of the K range by two clusters that add (red.global.add) into a tile cleared
// beforehand (zero_split_tiles): 114.6 -> 111.0 us for the whole two-phase call at 4096^3.
// Every wait is bounded; a wait that runs out sets the status word and the role leaves its loop.
// (textually included by mx_gemm.cu after mx_gemm_pair.cuh)
#pragma once

namespace bdr {

constexpr int kDStages = 6;
constexpr int kDStageBytes = 2 * kPairRows * kBK * 2;  // A 16 KB + B half 16 KB
constexpr int kDEpiWarps = 8;
constexpr int kDThreads = (2 + kDEpiWarps) * 32;
constexpr size_t kDSmemBytes = (size_t)kDStages * kDStageBytes + 1024 /*bookkeeping*/ + 1024 /*alignment*/;

struct DenseBars {
    uint64_t full[kDStages], full_local[kDStages], empty[kDStages], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int failed;
};

struct DenseMaps {
    CUtensorMap a, b;  // bf16 [rows, K], box 64 x 128, 128-byte swizzle
};

__device__ __forceinline__ void tmem_alloc2_cols(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void red_add_v4(float* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(a)), "f"(__uint_as_float(b)),
                 "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kDThreads, 1)
bf16_gemm_pair_kernel(const __grid_constant__ DenseMaps maps, int tiles_m, int tiles_n, int band_rows, int nk, int tiles_full, int n_items,
                      float* c, int64_t ldc) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* stages = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    DenseBars& bars = *reinterpret_cast<DenseBars*>(stages + kDStages * kDStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    // Work items: the first tiles_full tiles with their whole K range (a multiple of the cluster count: whole rounds), then
    // every remaining tile as two items of half the K range each, which add their results into a zeroed C tile -- so a
    // last round that would keep at most half of the clusters busy takes half as long.
    auto item_of = [&](int i, int& t, int& k0, int& cnt, bool& add) {
        if (i < tiles_full) { t = i; k0 = 0; cnt = nk; add = false; }
        else { const int j = i - tiles_full; t = tiles_full + (j >> 1); cnt = nk >> 1; k0 = (j & 1) * cnt; add = true; }
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDStages; ++s) {
            mbar_init(&bars.full[s], 2);        // leader: its own TMA bytes (arrive.expect_tx) + the peer's relay
            mbar_init(&bars.full_local[s], 1);  // peer: its own TMA bytes
            mbar_init(&bars.empty[s], 1);       // multicast commit of the MMAs that read the stage
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars.tmem_full[b], 1);                 // multicast commit after a tile's last K step
            mbar_init(&bars.tmem_empty[b], 2 * kDEpiWarps);   // leader: every epilogue warp of both CTAs
        }
        bars.failed = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc2_cols(&bars.tmem_base, 512);  // two accumulator buffers of 256 columns
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars.tmem_base;

    // Nothing above touched global memory: under a programmatic dependent launch it overlaps the tail of the
    // unpack kernel that writes operand B.  From here on the operands are needed.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint64_t* const my_full = rank == 0 ? bars.full : bars.full_local;
            bool ok = true;
            uint32_t it = 0;  // running K-step count across tiles
            for (int i = cluster_id; i < n_items && ok; i += n_clusters) {
                int t, k0, cnt, tm, tn;
                bool add;
                item_of(i, t, k0, cnt, add);
                gemm_tile_coords(t, tiles_m, tiles_n, band_rows, tm, tn);
                const int row_a = (tm * 2 + (int)rank) * kPairRows, row_b = (tn * 2 + (int)rank) * kPairRows;
                for (int kk = k0; kk < k0 + cnt; ++kk, ++it) {
                    const int stage = it % kDStages;
                    if (it >= kDStages) {
                        ok = mbar_wait(&bars.empty[stage], ((it / kDStages) - 1) & 1);
                        if (!ok) break;
                    }
                    uint8_t* dst = stages + stage * kDStageBytes;
                    mbar_expect_tx(&my_full[stage], kDStageBytes);
                    tma_load_2d(dst, &maps.a, kk * kBK, row_a, &my_full[stage]);
                    tma_load_2d(dst + kPairRows * kBK * 2, &maps.b, kk * kBK, row_b, &my_full[stage]);
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
                    const int buf = tcount & 1;
                    if (tcount >= 2) {  // the epilogues of both CTAs have drained this buffer
                        ok = mbar_wait_cluster(&bars.tmem_empty[buf], ((tcount >> 1) - 1) & 1);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
                    for (int kk = 0; kk < cnt; ++kk, ++it) {
                        const int stage = it % kDStages;
                        ok = mbar_wait_cluster(&bars.full[stage], (it / kDStages) & 1);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sa = smem_u32(stages + stage * kDStageBytes);
                        const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + kPairRows * kBK * 2);
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k)
                            umma2_bf16(acc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kPairInstrDesc, (kk | k) != 0);
                        umma_commit2(&bars.empty[stage]);
                    }
                    if (ok) umma_commit2(&bars.tmem_full[buf]);
                }
            } else {
                // ---------------- relay (peer CTA): "my half of the stage has landed" ----------------
                for (int i = cluster_id; i < n_items && ok; i += n_clusters) {
                    int t, k0, cnt;
                    bool add;
                    item_of(i, t, k0, cnt, add);
                    for (int kk = 0; kk < cnt; ++kk, ++it) {
                        const int stage = it % kDStages;
                        ok = mbar_wait(&bars.full_local[stage], (it / kDStages) & 1);
                        if (!ok) break;
                        mbar_arrive_cluster(&bars.full[stage], 0);
                    }
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
            const int buf = tcount & 1;
            ok = ok && mbar_wait(&bars.tmem_full[buf], (tcount >> 1) & 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            int tm, tn;
            gemm_tile_coords(t, tiles_m, tiles_n, band_rows, tm, tn);
            float* crow = c + ((int64_t)(tm * 2 + (int)rank) * kPairRows + lane_base + lane) * ldc + (int64_t)tn * 256 + col_base;
#pragma unroll 1
            for (int cc = 0; cc < 128; cc += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(buf * 256 + col_base + cc), v);
                if (!add) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<uint4*>(crow + cc + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                } else {
#pragma unroll
                    for (int q = 0; q < 8; ++q) red_add_v4(crow + cc + 4 * q, v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(&bars.tmem_empty[buf], 0);
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

static bool make_dense_map(CUtensorMap* out, const void* base, int64_t rows, int64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)kPairRows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// clears `count` tiles of c from tile0 on (tile order of gemm_tile_coords): grid (count, 4), 256 threads
__global__ void zero_tiles_kernel(ZeroTiles z) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see zero_split_tiles
    const int t = z.tile0 + (int)blockIdx.x;
    int tm, tn;
    gemm_tile_coords(t, z.tiles_m, z.tiles_n, z.band_rows, tm, tn);
    for (int idx = (int)blockIdx.y * 64 * 64 + (int)threadIdx.x; idx < ((int)blockIdx.y + 1) * 64 * 64; idx += 256) {
        const int r = idx >> 6, ch = idx & 63;  // 64 rows per block, 64 chunks of 16 bytes per row
        *reinterpret_cast<uint4*>(z.c + ((int64_t)tm * 256 + r) * z.ldc + (int64_t)tn * 256 + ch * 4) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");  // launched as a programmatic dependent: do not finish before the grid in front
}

// How the tiles of C are shared out: whole rounds of full tiles, and a last round that would keep at most half of the
// clusters busy as twice as many items of half the K range (which add into tiles cleared beforehand).
struct GemmPlan {
    int tiles_m, tiles_n, band_rows, n_clusters, tiles_full, n_items;
    int split_tiles() const { return tiles_m * tiles_n - tiles_full; }
};
static GemmPlan plan_gemm(int64_t M, int64_t N, int64_t k_steps, int64_t operand_bytes) {
    GemmPlan p;
    p.tiles_m = (int)(M / 256);
    p.tiles_n = (int)(N / 256);
    p.band_rows = gemm_band_rows(operand_bytes);
    const int T = p.tiles_m * p.tiles_n, cmax = sm_count() / 2;
    p.n_clusters = std::min(T, cmax);
    const int rest = T % cmax;
    const bool split = rest > 0 && 2 * rest <= cmax && k_steps % 2 == 0;
    p.tiles_full = split ? T - rest : T;
    p.n_items = p.tiles_full + 2 * (T - p.tiles_full);
    if (split) p.n_clusters = std::min(p.n_items, cmax);
    return p;
}
// chained: launched as a programmatic dependent of the kernel before it in the stream, whose output it does not touch: it
// runs while that kernel drains, lets the kernel behind it start at once, and does not finish before the one in front
// (so whoever waits for the end of such a chain has every link's results).
static int zero_split_tiles(const GemmPlan& plan, float* c, int64_t ldc, cudaStream_t st, bool chained = false) {
    if (plan.split_tiles() == 0) return BDR_OK;
    const ZeroTiles z = {c, ldc, plan.tiles_n, plan.tiles_full, plan.split_tiles(), plan.tiles_m, plan.band_rows};
    if (!chained) {
        zero_tiles_kernel<<<dim3((unsigned)z.count, 4), 256, 0, st>>>(z);
        return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)z.count, 4);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, zero_tiles_kernel, z);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// a_bf16 [M, K], b_bf16 [N, K], both contiguous; M, N multiples of 256, K a multiple of 64.  The tiles plan.tiles_full ..
// of C must hold zeros (zero_split_tiles).
static int launch_gemm_dense(const void* a_bf16, const void* b_bf16, int64_t M, int64_t N, int64_t K, const GemmPlan& plan, float* c,
                             int64_t ldc, cudaStream_t st) {
    static PerDevice once;
    if (once.get(current_device(), [&]() -> int {  // no occupancy query: cluster kernel, one CTA per SM
            return cudaFuncSetAttribute(bf16_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDSmemBytes) == cudaSuccess ? 1 : 0;
        }) < 1)
        return BDR_ERR_CUDA;
    DenseMaps maps;
    if (!make_dense_map(&maps.a, a_bf16, M, K) || !make_dense_map(&maps.b, b_bf16, N, K)) return BDR_ERR_CUDA;
    const int n_clusters = plan.n_clusters;
    // programmatic dependent launch: set-up may overlap the tail of the kernel before it in the stream; the kernel
    // waits (griddepcontrol.wait) before it reads anything
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * n_clusters));
    cfg.blockDim = dim3(kDThreads);
    cfg.dynamicSmemBytes = kDSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, bf16_gemm_pair_kernel, maps, plan.tiles_m, plan.tiles_n, plan.band_rows, (int)(K / kBK), plan.tiles_full,
                                             plan.n_items, c, ldc);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

}  // namespace bdr
