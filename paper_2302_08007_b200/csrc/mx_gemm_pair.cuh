// mx_gemm, 2-CTA version: a cluster of two CTAs computes a 256 x 256 tile of C with
// tcgen05.mma.cta_group::2 (each CTA owns 128 rows of the accumulator in its own tensor memory and
// supplies its 128 rows of A and its 128-row half of the B tile from its own shared memory).
//
// Per CTA:  one thread of warp 8 streams the packed bytes of the CTA's 256 operand rows into shared
// memory with 2-D TMA tile loads (cp.async.bulk.tensor, one per plane: 128 rows x 256 K-elements of
// codes, exponents or microexponents; no multicast; completion on an mbarrier), so no thread ever
// waits on an uncoalesced global load;  warps 0-7 (one thread per row)
// decode those bytes to bf16 and store them in the K-major 128-byte-swizzled operand stages;  in the
// leader CTA one thread of warp 9 issues the MMAs once the decoders of BOTH CTAs have arrived on its
// "full" barrier, and tcgen05.commit (multicast to both CTAs) releases the stage and, at the end,
// signals the epilogue;  warps 0-7 then drain their CTA's accumulator with tcgen05.ld.
// Every wait is bounded; a wait that runs out sets the status word and the CTA falls through to the
// final cluster barrier, frees its tensor memory and returns.
// (textually included by mx_gemm.cu, which defines the shared PTX wrappers, the decoder and the status word)
#pragma once

namespace bdr {

constexpr int kPairRows = 128;                  // rows of A and of the B half per CTA
constexpr int kChunkK = 256;                    // K elements per exponent / microexponent tile (16 bytes per row)
constexpr int kEChunkK = 128;                   // K elements per code tile (two K steps): small, so more operand stages fit
constexpr int kStepsPerEChunk = kEChunkK / kBK; // 2
constexpr int kDecodeGroups = 2;                // decode groups of 8 warps (one thread per row); group g takes K steps g, g+2, ...
constexpr int kGroupWarps = 2 * kPairRows / 32; // 8
constexpr int kPairDecodeWarps = kDecodeGroups * kGroupWarps;
constexpr int kEpilogueWarps2 = 16;             // warps that drain the accumulator (4 lane groups x 4 column quarters)
constexpr int kLoaderWarp = kPairDecodeWarps, kMmaWarp = kPairDecodeWarps + 1;
constexpr int kPairThreads = (kPairDecodeWarps + 2) * 32;
constexpr int kPairStageBytes = 2 * kPairRows * kBK * 2;  // A 16 KB + B half 16 KB

// Packed bytes as the TMA writes them, dense row-major, for the 128 rows of one operand:
// codes of one 128-element K chunk [128][16 W bytes], and per 256-element K chunk the exponent and
// microexponent bytes [128][16] each.
template <int W> struct ChunkPlanes {
    static constexpr int kElemRow = kEChunkK * W / 8;      // 48 / 80 / 128 bytes of codes per row
    static constexpr int kBytes = kPairRows * kElemRow;    // a multiple of 128
};
constexpr int kXmPlane = kPairRows * 16;                   // one exponent or microexponent tile
constexpr int kXmBytes = 4 * kXmPlane;                     // A exps | A micro | B exps | B micro
constexpr int kMaxPk = 2;                                  // code-chunk buffers (and exponent buffers)
template <int WA, int WB> struct PairSmem {
    static constexpr int kPk = kMaxPk;
    static constexpr int kPackedBytes = ChunkPlanes<WA>::kBytes + ChunkPlanes<WB>::kBytes;  // one code buffer
    static constexpr int kBudget = 224 * 1024 - kPk * kPackedBytes - 2 * kXmBytes - 1024;
    // the MMA round trip (decoders -> leader's barrier -> MMA -> multicast commit -> decoders) is long:
    // as many operand stages as fit
    static constexpr int kStages = kBudget / kPairStageBytes >= 6 ? 6 : kBudget / kPairStageBytes;
    static_assert(kStages >= 2, "operand stages do not fit");
    static constexpr size_t kBytes = (size_t)kStages * kPairStageBytes + kPk * kPackedBytes + 2 * kXmBytes + 1024 /*bookkeeping*/ + 1024 /*alignment*/;
};

struct PairMaps {  // tensor maps of the three planes of A and of B (uint8 elements, rows x row bytes)
    CUtensorMap a_elems, a_exps, a_micro, b_elems, b_exps, b_micro;
};

struct PairBars {
    uint64_t full[6], empty[6], accum, pk_full[kMaxPk], pk_empty[kMaxPk];
    uint32_t tmem_base;
    int failed;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_cluster(uint64_t* bar, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(bar)), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kSuspendHintNs)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// 2-D tile load: box starts at byte x of row y (x must be a multiple of 16)
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// arrive (once the issuing thread's earlier MMAs have completed) on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma_commit2(uint64_t* bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D = fp32, A = B = bf16, both K-major, N = 256, M = 256 (128 rows per CTA)
constexpr uint32_t kPairInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

// pk0: shared-memory address of this operand's codes in code buffer 0 (buffers are pk_stride apart);
// xm0: address of this operand's exponent tile in exponent buffer 0 (its microexponents follow at
// +kXmPlane; buffers are kXmBytes apart).  `half` selects which two of the row's four 16-element
// blocks of a K step this thread decodes.
template <int W>
__device__ __forceinline__ bool pair_decode_rows(uint32_t pk0, uint32_t pk_stride, uint32_t xm0, int r, int group, uint32_t tile_off,
                                                 uint32_t stages_addr, int n_stages, PairBars& bars, int nk, int lane) {
    constexpr int NW = kBK * W / 32;  // code words of one K step (four blocks): 6 / 10 / 16
    // Decode group `group` takes every kDecodeGroups-th K step, so while one group sits in its
    // barrier / fence phase the others are decoding and the SM keeps issuing.
    for (int kk = group; kk < nk; kk += kDecodeGroups) {
        const int ech = kk / kStepsPerEChunk, ks = kk % kStepsPerEChunk, buf = ech % kMaxPk;
        {
            bool ok = mbar_wait(&bars.pk_full[buf], (ech / kMaxPk) & 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) return false;
        }
        const uint32_t ebase = pk0 + buf * pk_stride + r * ChunkPlanes<W>::kElemRow + ks * (kBK * W / 8);  // 8-byte aligned
        uint32_t w[NW];
#pragma unroll
        for (int i = 0; i < NW / 2; ++i) { const uint2 v = ld_shared_v2(ebase + 8 * i); w[2 * i] = v.x; w[2 * i + 1] = v.y; }
        // exponent / microexponent bytes of this K step: 4 bytes each within the row's 16 (256 K elements)
        const uint32_t xm = xm0 + ((kk / 4) & 1) * kXmBytes + r * 16 + 4 * (kk & 3);
        const uint32_t exps4 = ld_shared_b32(xm), micro4 = ld_shared_b32(xm + kXmPlane);
        const int stage = kk % n_stages;
        if (kk >= n_stages) {
            bool ok = mbar_wait(&bars.empty[stage], ((kk / n_stages) - 1) & 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) return false;
        }
        const uint32_t tile = stages_addr + stage * kPairStageBytes + tile_off;
        const bool safe = __all_sync(0xFFFFFFFFu, exps_safe<W>(exps4));  // warp-uniform decoder choice
#pragma unroll
        for (int bb = 0; bb < kBK / kSlice; ++bb) {
            uint32_t o[8];
            if (safe) decode_block_bf16<W, NW, true>(w, bb * kSlice * W, (exps4 >> (8 * bb)) & 0xFFu, (micro4 >> (8 * bb)) & 0xFFu, o);
            else decode_block_bf16<W, NW, false>(w, bb * kSlice * W, (exps4 >> (8 * bb)) & 0xFFu, (micro4 >> (8 * bb)) & 0xFFu, o);
            st_shared_v4(tile + (((2 * bb) ^ (r & 7)) << 4), o[0], o[1], o[2], o[3]);
            st_shared_v4(tile + (((2 * bb + 1) ^ (r & 7)) << 4), o[4], o[5], o[6], o[7]);
        }
        fence_proxy_async();  // generic-proxy stores -> visible to the tensor core's (async proxy) reads
        __syncwarp();
        if (lane == 0) {
            mbar_arrive_cluster(&bars.full[stage], 0);   // the leader CTA counts both CTAs' decoders
            mbar_arrive(&bars.pk_empty[buf]);            // each warp reads a code chunk once (its K step of the two)
        }
    }
    return true;
}

template <int WA, int WB>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
mx_gemm_pair_kernel(const __grid_constant__ PairMaps maps, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc, const int* gate) {
    if (gate && *gate == 0) return;  // a fall-back launch that is not needed (the same for every thread of the grid)
    using SM = PairSmem<WA, WB>;
    constexpr int kStages = SM::kStages;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* stages = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int kPk = SM::kPk;
    uint8_t* pk_base = stages + kStages * kPairStageBytes;        // kPk code buffers of SM::kPackedBytes each
    uint8_t* xm_base = pk_base + kPk * SM::kPackedBytes;          // two exponent / microexponent buffers
    PairBars& bars = *reinterpret_cast<PairBars*>(xm_base + 2 * kXmBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int64_t m0 = ((int64_t)(blockIdx.x >> 1) * 2 + rank) * kPairRows;  // this CTA's rows of A and C
    const int64_t n0 = (int64_t)blockIdx.y * 256;                             // the pair's columns
    const int64_t nb0 = n0 + (int64_t)rank * kPairRows;                       // this CTA's half of the B tile
    const int nk = (int)(K / kBK), nchunks = (int)(K / kEChunkK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 6; ++s) { mbar_init(&bars.full[s], 2 * kGroupWarps); mbar_init(&bars.empty[s], 1); }  // 8 warps x 2 CTAs per K step
        mbar_init(&bars.accum, 1);
        for (int i = 0; i < kMaxPk; ++i) { mbar_init(&bars.pk_full[i], 1); mbar_init(&bars.pk_empty[i], kStepsPerEChunk * kGroupWarps); }  // each K step of the chunk is read by one group
        bars.failed = 0;
        fence_barrier_init();
    }
    if (warp == kMmaWarp) tmem_alloc2(&bars.tmem_base, 256);  // 256 fp32 columns x 128 lanes in each CTA
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers are initialised before anyone signals across the cluster
    tc_fence_after();
    const uint32_t tmem_base = bars.tmem_base;

    if (warp < kPairDecodeWarps) {
        // ---------------- decoders: threads t and t+256 share row t (A rows 0-127, then the B half's 128 rows) ----------------
        const int half = warp / kGroupWarps;        // decode group
        const int row256 = (int)threadIdx.x & 255;  // consecutive lanes hold consecutive rows (conflict-free swizzled stores)
        const bool is_a = row256 < kPairRows;
        const int r = is_a ? row256 : row256 - kPairRows;
        const uint32_t tile_off = (uint32_t)((is_a ? 0 : kPairRows * kBK * 2) + (r >> 3) * 1024 + (r & 7) * 128);
        bool ok;
        if (is_a) ok = pair_decode_rows<WA>(smem_u32(pk_base), SM::kPackedBytes, smem_u32(xm_base), r, half, tile_off, smem_u32(stages),
                                            kStages, bars, nk, lane);
        else ok = pair_decode_rows<WB>(smem_u32(pk_base) + ChunkPlanes<WA>::kBytes, SM::kPackedBytes, smem_u32(xm_base) + 2 * kXmPlane, r,
                                       half, tile_off, smem_u32(stages), kStages, bars, nk, lane);
        if (!ok) bars.failed = 1;

        // ---------------- epilogue: this CTA's 128 x 256 block of C ----------------
        bool done = ok && warp < kEpilogueWarps2 && mbar_wait(&bars.accum, 0);
        done = __all_sync(0xFFFFFFFFu, done);
        if (warp >= kEpilogueWarps2) {
            // the remaining decode warps have no accumulator lanes to drain
        } else if (done) {
            tc_fence_after();
            const int lane_base = (warp & 3) * 32, col_base = (warp >> 2) * 64;  // 16 warps: 4 lane groups x 4 column quarters
            float* crow = c + (m0 + lane_base + lane) * ldc + n0 + col_base;
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(col_base + cc), v);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<uint4*>(crow + cc + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            }
        } else {
            bars.failed = 1;
        }
        tc_fence_before();
    } else if (warp == kLoaderWarp) {
        // ---------------- loader: TMA tile loads, codes per 128 K elements, exponents per 256 ----------------
        if (lane == 0) {
            bool ok = true;
            for (int ch = 0; ch < nchunks; ++ch) {
                const int buf = ch % kPk;
                if (ch >= kPk) {
                    ok = mbar_wait(&bars.pk_empty[buf], ((ch / kPk) - 1) & 1);
                    if (!ok) break;
                }
                uint8_t* pa = pk_base + (size_t)buf * SM::kPackedBytes;
                uint8_t* pb = pa + ChunkPlanes<WA>::kBytes;
                const bool with_xm = (ch & 1) == 0;  // exponent tiles cover two code chunks and ride on the even one's barrier
                mbar_expect_tx(&bars.pk_full[buf], (uint32_t)(SM::kPackedBytes + (with_xm ? kXmBytes : 0)));
                tma_load_2d(pa, &maps.a_elems, ch * ChunkPlanes<WA>::kElemRow, (int)m0, &bars.pk_full[buf]);
                tma_load_2d(pb, &maps.b_elems, ch * ChunkPlanes<WB>::kElemRow, (int)nb0, &bars.pk_full[buf]);
                if (with_xm) {
                    // buffer (ch/2)&1 was last read during code chunk ch-3, which pk_empty above has confirmed done
                    uint8_t* xm = xm_base + (size_t)((ch >> 1) & 1) * kXmBytes;
                    tma_load_2d(xm, &maps.a_exps, (ch >> 1) * 16, (int)m0, &bars.pk_full[buf]);
                    tma_load_2d(xm + kXmPlane, &maps.a_micro, (ch >> 1) * 16, (int)m0, &bars.pk_full[buf]);
                    tma_load_2d(xm + 2 * kXmPlane, &maps.b_exps, (ch >> 1) * 16, (int)nb0, &bars.pk_full[buf]);
                    tma_load_2d(xm + 3 * kXmPlane, &maps.b_micro, (ch >> 1) * 16, (int)nb0, &bars.pk_full[buf]);
                }
            }
            if (!ok) bars.failed = 1;
        }
        __syncwarp();
    } else {
        // ---------------- MMA issuer: one lane of the leader CTA ----------------
        if (rank == 0 && lane == 0) {
            bool ok = true;
            for (int kk = 0; kk < nk; ++kk) {
                const int stage = kk % kStages;
                ok = mbar_wait_cluster(&bars.full[stage], (kk / kStages) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = smem_u32(stages + stage * kPairStageBytes);
                const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + kPairRows * kBK * 2);
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k)
                    umma2_bf16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kPairInstrDesc, (kk | k) != 0);
                umma_commit2(&bars.empty[stage]);  // both CTAs may refill the stage once these MMAs have read it
            }
            if (ok) umma_commit2(&bars.accum);     // accumulators complete in both CTAs
            else bars.failed = 1;
        }
        __syncwarp();
        tc_fence_before();
    }
    __syncthreads();
    cluster_sync_all();  // the peer may still be reading this CTA's shared memory / signalling its barriers
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, 256);
    }
    if (threadIdx.x == 0 && bars.failed) atomicExch(&g_gemm_status, (int)BDR_ERR_TIMEOUT);
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}
// plane viewed as a [rows, row_bytes] byte matrix with pitch `ld`; box = 128 rows x box_bytes
static bool make_plane_map(CUtensorMap* out, const uint8_t* base, int64_t rows, int64_t row_bytes, int64_t ld, int box_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld};
    const cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)kPairRows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int WA, int WB>
int launch_gemm_pair(const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc,
                     const int* gate, cudaStream_t st) {
    auto kern = mx_gemm_pair_kernel<WA, WB>;
    const size_t smem = PairSmem<WA, WB>::kBytes;
    static PerDevice once;  // per instantiation
    if (once.get(current_device(), [&]() -> int {  // no occupancy query: cluster kernel, one CTA per SM
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess ? 1 : 0;
        }) < 1)
        return BDR_ERR_CUDA;
    PairMaps maps;
    const bool ok = make_plane_map(&maps.a_elems, a.elems, M, K * WA / 8, a.ld_elems, ChunkPlanes<WA>::kElemRow) &&
                    make_plane_map(&maps.a_exps, a.exps, M, K / 16, a.ld_exps, 16) &&
                    make_plane_map(&maps.a_micro, a.micro, M, K / 16, a.ld_micro, 16) &&
                    make_plane_map(&maps.b_elems, b.elems, N, K * WB / 8, b.ld_elems, ChunkPlanes<WB>::kElemRow) &&
                    make_plane_map(&maps.b_exps, b.exps, N, K / 16, b.ld_exps, 16) &&
                    make_plane_map(&maps.b_micro, b.micro, N, K / 16, b.ld_micro, 16);
    if (!ok) return BDR_ERR_UNSUPPORTED;  // caller falls back to the single-CTA kernel
    const dim3 grid((unsigned)(M / 128), (unsigned)(N / 256));  // x: CTAs (two per 256-row pair), y: column tiles
    kern<<<grid, kPairThreads, smem, st>>>(maps, M, N, K, c, ldc, gate);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

}  // namespace bdr
