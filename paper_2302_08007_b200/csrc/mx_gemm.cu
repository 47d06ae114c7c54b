// mx_gemm: C[M,N] = deq(A)[M,K] * deq(B)[N,K]^T with both operands given as packed MX planes
// quantized along K (Section V: both inputs of a tensor operation are MX-quantized along the
// reduction dimension).  The packed bytes are decoded to bf16 inside the kernel -- every MX value
// with m <= 7 is exact in bf16 -- and multiplied on the 5th-generation tensor cores
// (tcgen05.mma, kind::f16, fp32 accumulation in tensor memory).
//
// One CTA computes a 128 x 256 tile of C.  Warps 0-7 are decoders: per 64-wide K step they read the
// packed codes / exponents / microexponents of the tile's 128 A rows and 256 B rows straight from
// global memory (the operands live in L2), rebuild bf16 values with packed bf16x2 arithmetic and
// store them in shared memory in the K-major, 128-byte-swizzled layout the tensor core reads.
// Warp 8 issues the MMAs (4 x K=16 per stage) and signals stage reuse / accumulator completion
// through tcgen05.commit on mbarriers.  After the last K step warps 0-7 read the accumulator from
// tensor memory (tcgen05.ld) and store C.  Every wait is bounded: if one runs out the kernel
// records BDR_ERR_TIMEOUT in a status word, skips the remaining work, frees its tensor memory and
// returns.
#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 4;
constexpr int kDecodeWarps = 8;
constexpr int kGemmThreads = (kDecodeWarps + 1) * 32;
constexpr int kABytes = kBM * kBK * 2;  // 16 KB
constexpr int kBBytes = kBN * kBK * 2;  // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr uint32_t kSpinLimit = 1u << 20;  // bounded waits (each try_wait itself blocks for a while)

__device__ int g_gemm_status = 0;  // sticky: first failing launch leaves BDR_ERR_TIMEOUT here

// ---- PTX wrappers ----------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, M = 128, N = 256, K = 16.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of the accumulator -> 32 registers per thread.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 64 bf16 (128 bytes),
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, N = 256, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

// ---- decoding ---------------------------------------------------------------------------------------------
// bf16 bits of 2^(e-127) for a biased exponent e that may be <= 0 (bf16 subnormals) -- 0 below that.
__device__ __forceinline__ uint32_t bf16_pow2(int e) {
    return e >= 1 ? (uint32_t)e << 7 : (e >= -6 ? 1u << (6 + e) : 0u);
}

// Decode one 16-element block (k1 = 16, k2 = 2, d2 = 1, code width W = m + 1) into 8 bf16x2 words.
// A code pair t (2W stream bits) is spread to the two halves of a word, the magnitudes are ORed
// into the mantissa of bf16 128.0 (0x4300 | q = 128 + q exactly, q < 128), 128 is subtracted and the
// result multiplied by the sub-block's power-of-two scale with packed bf16x2 arithmetic; both steps
// are exact.  The sign bit is ORed in last.
template <int W>
__device__ __forceinline__ void decode_block_bf16(const uint32_t (&words)[(kSlice * W + 31) / 32 + 1], uint32_t F, uint32_t micro,
                                                  uint32_t (&out)[8]) {
    constexpr int M = W - 1;
    constexpr uint32_t kQ2 = ((1u << M) - 1u) * 0x00010001u;
    const int e0 = (int)F - (M - 1);  // biased exponent of one unit of q at tau = 0
    uint32_t s0 = bf16_pow2(e0), s1 = bf16_pow2(e0 - 1);
    if (F == 255) { s0 = 0x7FC0u; s1 = 0x7FC0u; }  // Inf/NaN block -> NaN
    s0 *= 0x00010001u;
    s1 *= 0x00010001u;
    const __nv_bfloat162 k128 = __floats2bfloat162_rn(128.f, 128.f);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int bit = 2 * j * W, wi = bit >> 5, sh = bit & 31;
        const uint32_t t = sh == 0 ? words[wi] : (sh + 2 * W > 32 ? __funnelshift_r(words[wi], words[wi + 1], sh) : words[wi] >> sh);
        uint32_t u;
        if (W == 8) u = __byte_perm(t, 0, 0x4140);                 // bytes [b0, 0, b1, 0]
        else u = (t & ((1u << W) - 1u)) | ((t << (16 - W)) & (((1u << W) - 1u) << 16));
        uint32_t mag = (u & kQ2) | 0x43004300u;
        uint32_t sgn = (u << (15 - M)) & 0x80008000u;
        uint32_t sc = (micro >> j) & 1u ? s1 : s0;
        __nv_bfloat162 q = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&mag), k128);
        __nv_bfloat162 v = __hmul2(q, *reinterpret_cast<__nv_bfloat162*>(&sc));
        out[j] = *reinterpret_cast<uint32_t*>(&v) | sgn;
    }
}

struct GemmSmem {
    uint64_t full[kStages], empty[kStages], accum;
    uint32_t tmem_base;
    int failed;
};

template <int WA, int WB>
__global__ void __launch_bounds__(kGemmThreads, 1)
mx_gemm_kernel(bdr_planes_t a, bdr_planes_t b, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // tiles first (1024-byte aligned for the swizzle), bookkeeping after them
    uint8_t* tiles = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    GemmSmem& gs = *reinterpret_cast<GemmSmem*>(tiles + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t m0 = (int64_t)blockIdx.y * kBM, n0 = (int64_t)blockIdx.x * kBN;
    const int nk = (int)(K / kBK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&gs.full[s], kDecodeWarps); mbar_init(&gs.empty[s], 1); }
        mbar_init(&gs.accum, 1);
        gs.failed = 0;
        fence_barrier_init();
    }
    if (warp == kDecodeWarps) tmem_alloc(&gs.tmem_base, kBN);  // 256 fp32 columns x 128 lanes
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = gs.tmem_base;

    if (warp < kDecodeWarps) {
        // ---------------- decoders ----------------
        // Work item = half a row of the K step (2 blocks = 32 elements); 768 items, 3 per thread.
        // Consecutive lanes take consecutive rows, so the eight 16-byte stores of a quarter-warp land
        // in eight different swizzled positions (no bank conflicts).
        bool ok = true;
        for (int kk = 0; kk < nk && ok; ++kk) {
            const int stage = kk % kStages;
            if (kk >= kStages) {
                ok = mbar_wait(&gs.empty[stage], ((kk / kStages) - 1) & 1);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
            }
            uint8_t* sa = tiles + stage * kStageBytes;
#pragma unroll 1
            for (int it = 0; it < 3; ++it) {
                const int item = it * 256 + (int)threadIdx.x;  // 0..767
                const int half = item / (kBM + kBN), row = item - half * (kBM + kBN);
                const bool is_a = row < kBM;
                const int r = is_a ? row : row - kBM;
                const bdr_planes_t& pl = is_a ? a : b;
                const int64_t grow = (is_a ? m0 : n0) + r;
                const int64_t blk = (int64_t)kk * (kBK / kSlice) + half * 2;  // first of the item's two blocks
                uint8_t* tile = sa + (is_a ? 0 : kABytes) + (r >> 3) * 1024 + (r & 7) * 128;
                const uint32_t exps2 = *reinterpret_cast<const uint16_t*>(pl.exps + grow * pl.ld_exps + blk);
                const uint32_t micro2 = *reinterpret_cast<const uint16_t*>(pl.micro + grow * pl.ld_micro + blk);
                if (is_a) {
                    constexpr int NW = (2 * kSlice * WA + 31) / 32;  // words of two blocks
                    const uint32_t* src = reinterpret_cast<const uint32_t*>(pl.elems + grow * pl.ld_elems + blk * 2 * WA);
                    uint32_t w[NW + 1];
#pragma unroll
                    for (int i = 0; i < NW; ++i) w[i] = __ldg(src + i);
                    w[NW] = 0;
#pragma unroll
                    for (int bb = 0; bb < 2; ++bb) {
                        uint32_t words[(kSlice * WA + 31) / 32 + 1];
#pragma unroll
                        for (int i = 0; i < (kSlice * WA + 31) / 32 + 1; ++i) {
                            const int bit = bb * kSlice * WA + 32 * i, wi = bit >> 5, sh = bit & 31;
                            words[i] = wi > NW ? 0u : (sh == 0 ? w[wi] : __funnelshift_r(w[wi], wi + 1 <= NW ? w[wi + 1] : 0u, sh));
                        }
                        uint32_t o[8];
                        decode_block_bf16<WA>(words, (exps2 >> (8 * bb)) & 0xFFu, (micro2 >> (8 * bb)) & 0xFFu, o);
                        const int chunk = (half * 2 + bb) * 2;  // 16-byte chunk index of the block's first 8 elements
                        *reinterpret_cast<uint4*>(tile + ((chunk ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                        *reinterpret_cast<uint4*>(tile + (((chunk + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                } else {
                    constexpr int NW = (2 * kSlice * WB + 31) / 32;
                    const uint32_t* src = reinterpret_cast<const uint32_t*>(pl.elems + grow * pl.ld_elems + blk * 2 * WB);
                    uint32_t w[NW + 1];
#pragma unroll
                    for (int i = 0; i < NW; ++i) w[i] = __ldg(src + i);
                    w[NW] = 0;
#pragma unroll
                    for (int bb = 0; bb < 2; ++bb) {
                        uint32_t words[(kSlice * WB + 31) / 32 + 1];
#pragma unroll
                        for (int i = 0; i < (kSlice * WB + 31) / 32 + 1; ++i) {
                            const int bit = bb * kSlice * WB + 32 * i, wi = bit >> 5, sh = bit & 31;
                            words[i] = wi > NW ? 0u : (sh == 0 ? w[wi] : __funnelshift_r(w[wi], wi + 1 <= NW ? w[wi + 1] : 0u, sh));
                        }
                        uint32_t o[8];
                        decode_block_bf16<WB>(words, (exps2 >> (8 * bb)) & 0xFFu, (micro2 >> (8 * bb)) & 0xFFu, o);
                        const int chunk = (half * 2 + bb) * 2;
                        *reinterpret_cast<uint4*>(tile + ((chunk ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                        *reinterpret_cast<uint4*>(tile + (((chunk + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
            }
            fence_proxy_async();  // make the generic-proxy stores visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&gs.full[stage]);
        }
        if (!ok) gs.failed = 1;

        // ---------------- epilogue ----------------
        bool done = ok && mbar_wait(&gs.accum, 0);
        done = __all_sync(0xFFFFFFFFu, done);
        if (done) {
            tc_fence_after();
            const int lane_base = (warp & 3) * 32;            // a warp may only touch its own 32 TMEM lanes
            const int col_base = (warp >> 2) * (kBN / 2);     // warps 0-3: columns 0-127, warps 4-7: 128-255
            float* crow = c + (m0 + lane_base + lane) * ldc + n0 + col_base;
#pragma unroll 1
            for (int cc = 0; cc < kBN / 2; cc += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(col_base + cc), r);
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<uint4*>(crow + cc + 4 * v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
            }
        } else {
            gs.failed = 1;
        }
        tc_fence_before();
    } else {
        // ---------------- MMA issuer (one lane) ----------------
        if (lane == 0) {
            bool ok = true;
            for (int kk = 0; kk < nk; ++kk) {
                const int stage = kk % kStages;
                ok = mbar_wait(&gs.full[stage], (kk / kStages) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = smem_u32(tiles + stage * kStageBytes);
                const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + kABytes);
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k)  // 32 bytes of K per MMA: advance the start address by 2 units
                    umma_bf16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kInstrDesc, (kk | k) != 0);
                umma_commit(&gs.empty[stage]);  // stage may be overwritten once these MMAs have read it
            }
            if (ok) umma_commit(&gs.accum);     // accumulator complete
            else gs.failed = 1;
        }
        __syncwarp();
        tc_fence_before();
    }
    __syncthreads();
    if (warp == kDecodeWarps) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kBN);
    }
    if (threadIdx.x == 0 && gs.failed) atomicExch(&g_gemm_status, (int)BDR_ERR_TIMEOUT);
}

template <int WA, int WB>
static int launch_gemm(const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc,
                       cudaStream_t st) {
    auto kern = mx_gemm_kernel<WA, WB>;
    const size_t smem = (size_t)kStages * kStageBytes + sizeof(GemmSmem) + 1024;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return BDR_ERR_CUDA;
        attr_done = true;
    }
    const dim3 grid((unsigned)(N / kBN), (unsigned)(M / kBM));
    kern<<<grid, kGemmThreads, smem, st>>>(a, b, M, N, K, c, ldc);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <int WA>
static int gemm_pick_b(int mb, const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, float* c,
                       int64_t ldc, cudaStream_t st) {
    switch (mb) {
        case 2: return launch_gemm<WA, 3>(a, b, M, N, K, c, ldc, st);
        case 4: return launch_gemm<WA, 5>(a, b, M, N, K, c, ldc, st);
        case 7: return launch_gemm<WA, 8>(a, b, M, N, K, c, ldc, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr

using namespace bdr;

extern "C" {

int mx_gemm(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
            int64_t N, int64_t K, float* c, int64_t ldc, void* stream) {
    if (!cfg_a || !cfg_b || !a || !b || !c) return BDR_ERR_NULL;
    for (const bdr_config_t* cf : {cfg_a, cfg_b}) {
        if (cf->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
        if (cf->d1 != 8 || cf->k1 < 1 || cf->k2 < 1 || cf->k1 % cf->k2 != 0 || cf->d2 < 0 || cf->d2 > 3 || cf->m < 1 || cf->m > 8)
            return BDR_ERR_BAD_CONFIG;
        if (cf->k1 != 16 || cf->k2 != 2 || cf->d2 != 1 || (cf->m != 2 && cf->m != 4 && cf->m != 7)) return BDR_ERR_UNSUPPORTED;
    }
    if (M < 0 || N < 0 || K < 0 || ldc < N) return BDR_ERR_SIZE;
    if (M == 0 || N == 0) return BDR_OK;
    if (M % kBM || N % kBN || K % kBK || K == 0) return BDR_ERR_UNSUPPORTED;
    if (M / kBM > 65535) return BDR_ERR_UNSUPPORTED;
    for (const bdr_planes_t* p : {a, b}) {
        if (!p->exps || !p->micro || !p->elems) return BDR_ERR_NULL;
        if (((uintptr_t)p->exps | (uintptr_t)p->micro | (uintptr_t)p->elems) % 16) return BDR_ERR_MISALIGNED;
        if ((p->ld_exps | p->ld_micro | p->ld_elems) % 16) return BDR_ERR_MISALIGNED;
    }
    if (a->ld_exps < K / 16 || a->ld_micro < K / 16 || a->ld_elems < K * (cfg_a->m + 1) / 8) return BDR_ERR_SIZE;
    if (b->ld_exps < K / 16 || b->ld_micro < K / 16 || b->ld_elems < K * (cfg_b->m + 1) / 8) return BDR_ERR_SIZE;
    if ((uintptr_t)c % 16 || ldc % 4) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    switch (cfg_a->m) {
        case 2: return gemm_pick_b<3>(cfg_b->m, *a, *b, M, N, K, c, ldc, st);
        case 4: return gemm_pick_b<5>(cfg_b->m, *a, *b, M, N, K, c, ldc, st);
        case 7: return gemm_pick_b<8>(cfg_b->m, *a, *b, M, N, K, c, ldc, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

int mx_gemm_status(void) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)) != cudaSuccess) return BDR_ERR_CUDA;
    return v;
}

}  // extern "C"
