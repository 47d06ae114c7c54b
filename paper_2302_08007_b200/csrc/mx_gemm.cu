// mx_gemm: C[M,N] = deq(A)[M,K] * deq(B)[N,K]^T with both operands given as packed MX planes
// quantized along K (Section V: both inputs of a tensor operation are MX-quantized along the
// reduction dimension).  The packed bytes are decoded to bf16 -- every MX value with m <= 7 is exact in
// bf16 -- and multiplied on the 5th-generation tensor cores (tcgen05.mma, fp32 accumulation in tensor
// memory).  This file holds the shared PTX wrappers, the packed-byte decoder, the C-ABI entry points and the
// kernels, the last three as textually included headers:
//   * mx_gemm_kernel (below): one CTA per 128 x 256 tile of C, for shapes the paired kernel does not take.
//     Warps 0-11 decode, one thread per tile row (128 A rows + 256 B rows): per 64-wide K step a thread reads
//     its row's packed codes / exponents / microexponents from global memory one step ahead of use, rebuilds
//     bf16 values with packed bf16x2 arithmetic and stores them in shared memory in the K-major,
//     128-byte-swizzled layout the tensor core reads.  Warp 12 issues the MMAs (kind::f16, 4 x K=16 per stage)
//     and signals stage reuse / accumulator completion through tcgen05.commit on mbarriers; warps 0-7 then
//     read the accumulator from tensor memory (tcgen05.ld) and store C.
//   * mx_gemm_pair.cuh: the same decode-inside-the-GEMM scheme for a cluster of two CTAs on a 256 x 256 tile
//     (cta_group::2), packed planes brought in by TMA; what mx_gemm runs when M and K are multiples of 256.
//   * mx_gemm_dense.cuh: bf16 x bf16 persistent kernel for operands decoded once into a workspace (mx_gemm_ws).
//   * mx_gemm_f8.cuh: E4M3 x E4M3 block-scaled kernel for operands re-encoded into a workspace (mx_gemm_f8).
// Every wait is bounded: if one runs out the kernel records BDR_ERR_TIMEOUT in a status word, skips the
// remaining work, frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "bdr_device.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 3;       // bf16 operand stages (48 KB each)
// packed-byte prefetch ring: K steps in flight per decode thread (shared memory budget decides)
template <int W> struct RingDepth { static constexpr int value = W >= 8 ? 2 : 4; };
constexpr int kDecodeWarps = (kBM + kBN) / 32;  // 12: one decode thread per tile row
constexpr int kEpilogueWarps = 8;
constexpr int kGemmThreads = (kDecodeWarps + 1) * 32;
constexpr int kABytes = kBM * kBK * 2;  // 16 KB
constexpr int kBBytes = kBN * kBK * 2;  // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr uint32_t kSpinLimit = 1u << 18;     // bounded waits: this many polls ...
constexpr uint32_t kSuspendHintNs = 2000;     // ... each of which may sleep about this long in hardware

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
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kSuspendHintNs)
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
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
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
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    tmem_ld32_nowait(taddr, r);
    tmem_ld_wait();
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

__device__ __forceinline__ uint2 ld_shared_v2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_shared_b32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t bf16x2_fma(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_mul(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Decode one 16-element block (k1 = 16, k2 = 2, d2 = 1, code width W = m + 1) that starts at stream
// bit `bit0` of w[] into 8 bf16x2 words.  A code pair t (2W stream bits) is spread to the two halves
// of a word; the magnitudes are ORed into the mantissa of bf16 128.0 (0x4300 | q = 128 + q exactly,
// q < 128); one packed fused multiply-add with the sub-block's power-of-two scale s and the
// constant -128 s then gives q * s exactly (the exact result is representable, so the single
// rounding changes nothing).  The sign bit is ORed in last.
template <int W, int NWORDS, bool SAFE>
__device__ __forceinline__ void decode_block_bf16(const uint32_t (&w)[NWORDS], int bit0, uint32_t F, uint32_t micro, uint32_t (&out)[8]) {
    constexpr int M = W - 1;
    constexpr uint32_t kQ2 = ((1u << M) - 1u) * 0x00010001u;
    // scale of one unit of q: 2^(F-127-tau-(m-1)); the constant term -128 * scale needs exponent + 7.
    // SAFE (decided by the caller for the whole warp): 2 <= e0 <= 247, so both scales and both
    // constants are normal bf16 numbers and one fused multiply-add per pair does the job.
    const int e0 = (int)F - (M - 1);
    uint32_t s0, s1, n0 = 0, n1 = 0;
    if (SAFE) {
        s0 = ((uint32_t)e0 << 7) * 0x00010001u;
        s1 = s0 - 0x00800080u;
        n0 = (s0 + 0x03800380u) | 0x80008000u;  // -(2^7 * s0)
        n1 = n0 - 0x00800080u;
    } else {
        s0 = bf16_pow2(e0) * 0x00010001u;
        s1 = bf16_pow2(e0 - 1) * 0x00010001u;
        if (F == 255) { s0 = 0x7FC07FC0u; s1 = s0; }  // Inf/NaN block -> NaN
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int bit = bit0 + 2 * j * W, wi = bit >> 5, sh = bit & 31;
        const uint32_t t = sh == 0 ? w[wi] : (sh + 2 * W > 32 ? __funnelshift_r(w[wi], wi + 1 < NWORDS ? w[wi + 1] : 0u, sh) : w[wi] >> sh);
        uint32_t u;
        if (W == 8) u = __byte_perm(t, 0, 0x4140);        // bytes [b0, 0, b1, 0]
        else if (3 * W <= 16) u = (t & ((1u << (2 * W)) - 1u)) * ((1u << (16 - W)) + 1u);  // t | t << (16-W), no overlap
        else u = (t & ((1u << W) - 1u)) | (t << (16 - W));
        const uint32_t mag = (u & kQ2) | 0x43004300u;
        const bool t1 = (micro >> j) & 1u;
        uint32_t v;
        if (SAFE) v = bf16x2_fma(mag, t1 ? s1 : s0, t1 ? n1 : n0);
        else v = bf16x2_mul(bf16x2_fma(mag, 0x3F803F80u, 0xC300C300u), t1 ? s1 : s0);  // subtract 128, then scale: both exact
        out[j] = v | ((u << (15 - M)) & 0x80008000u);
    }
}

// true when every block exponent in the word (4 bytes, one per block) allows the SAFE decoder
template <int W>
__device__ __forceinline__ bool exps_safe(uint32_t exps4) {
    constexpr int M = W - 1;
    bool ok = true;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int e0 = (int)((exps4 >> (8 * b)) & 0xFFu) - (M - 1);
        ok = ok && e0 >= 2 && e0 <= 247;
    }
    return ok;
}

struct GemmSmem {
    uint64_t full[kStages], empty[kStages], accum;
    uint32_t tmem_base;
    int failed;
};

// Bytes of one row's packed data for one K step, padded so that ring slots stay 8-byte aligned.
template <int W> struct RowStep {
    static constexpr int kElemBytes = kBK * W / 8;        // 24 / 40 / 64
    static constexpr int kBytes = kElemBytes + 8;         // + 4 exponent bytes + 4 microexponent bytes
    static constexpr int kRingBytes = kBytes * RingDepth<W>::value;  // one thread's ring
};
template <int WA, int WB> struct RingStride {
    static constexpr int value = RowStep<WA>::kRingBytes > RowStep<WB>::kRingBytes ? RowStep<WA>::kRingBytes : RowStep<WB>::kRingBytes;
};

// The decode loop of one thread: its row's 64 elements (4 blocks) per K step.  The row's packed
// bytes travel through a private ring in shared memory that cp.async fills kRing-1 steps ahead.
template <int W>
__device__ __forceinline__ bool decode_rows(const bdr_planes_t& pl, int64_t grow, int r, uint32_t tile_off, uint32_t tiles_addr,
                                            uint8_t* ring_base, GemmSmem& gs, int nk, int lane) {
    constexpr int NW = kBK * W / 32;  // 32-bit words of codes per K step: 6 / 10 / 16
    constexpr int kSlot = RowStep<W>::kBytes;
    constexpr int kRing = RingDepth<W>::value;
    const uint8_t* ge = pl.elems + grow * pl.ld_elems;
    const uint8_t* gx = pl.exps + grow * pl.ld_exps;
    const uint8_t* gm = pl.micro + grow * pl.ld_micro;
    uint8_t* ring = ring_base;  // this thread's private ring
    auto issue = [&](int kk) {
        if (kk < nk) {
            uint8_t* slot = ring + (kk % kRing) * kSlot;
#pragma unroll
            for (int i = 0; i < RowStep<W>::kElemBytes / 8; ++i) cp_async8(slot + 8 * i, ge + (size_t)kk * RowStep<W>::kElemBytes + 8 * i);
            cp_async4(slot + RowStep<W>::kElemBytes, gx + 4 * kk);
            cp_async4(slot + RowStep<W>::kElemBytes + 4, gm + 4 * kk);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int i = 0; i < kRing - 1; ++i) issue(i);
    for (int kk = 0; kk < nk; ++kk) {
        issue(kk + kRing - 1);
        cp_async_wait<kRing - 1>();
        const uint32_t* slot = reinterpret_cast<const uint32_t*>(ring + (kk % kRing) * kSlot);
        uint32_t w[NW];
#pragma unroll
        for (int i = 0; i < NW; ++i) w[i] = slot[i];
        const uint32_t exps4 = slot[NW], micro4 = slot[NW + 1];
        const int stage = kk % kStages;
        if (kk >= kStages) {
            bool ok = mbar_wait(&gs.empty[stage], ((kk / kStages) - 1) & 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) return false;
        }
        const uint32_t tile = tiles_addr + stage * kStageBytes + tile_off;
        const bool safe = __all_sync(0xFFFFFFFFu, exps_safe<W>(exps4));  // warp-uniform choice of decoder
#pragma unroll
        for (int bb = 0; bb < kBK / kSlice; ++bb) {
            uint32_t o[8];
            if (safe) decode_block_bf16<W, NW, true>(w, bb * kSlice * W, (exps4 >> (8 * bb)) & 0xFFu, (micro4 >> (8 * bb)) & 0xFFu, o);
            else decode_block_bf16<W, NW, false>(w, bb * kSlice * W, (exps4 >> (8 * bb)) & 0xFFu, (micro4 >> (8 * bb)) & 0xFFu, o);
            st_shared_v4(tile + (((2 * bb) ^ (r & 7)) << 4), o[0], o[1], o[2], o[3]);
            st_shared_v4(tile + (((2 * bb + 1) ^ (r & 7)) << 4), o[4], o[5], o[6], o[7]);
        }
        fence_proxy_async();  // make the generic-proxy stores visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive(&gs.full[stage]);
    }
    return true;
}

template <int WA, int WB>
__global__ void __launch_bounds__(kGemmThreads, 1)
mx_gemm_kernel(bdr_planes_t a, bdr_planes_t b, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc, const int* gate) {
    if (gate && *gate == 0) return;  // a fall-back launch that is not needed (the same for every thread of the grid)
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // tiles first (1024-byte aligned for the swizzle), bookkeeping after them
    uint8_t* tiles = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    GemmSmem& gs = *reinterpret_cast<GemmSmem*>(tiles + kStages * kStageBytes);
    uint8_t* ring_base = tiles + kStages * kStageBytes + 256 + (size_t)threadIdx.x * RingStride<WA, WB>::value;  // this thread's packed-byte ring
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
        // Thread t owns tile row t (A rows 0-127, then B rows 0-255).  Consecutive lanes hold
        // consecutive rows, so the eight 16-byte stores of a quarter-warp land in eight different
        // swizzled positions (no bank conflicts).  The packed bytes of K step kk+1 are fetched into
        // registers before step kk is decoded.
        const bool is_a = warp < kBM / 32;  // warp-uniform
        const int r = is_a ? (int)threadIdx.x : (int)threadIdx.x - kBM;
        const bdr_planes_t& pl = is_a ? a : b;
        const int64_t grow = (is_a ? m0 : n0) + r;
        const uint32_t tile_off = (uint32_t)((is_a ? 0 : kABytes) + (r >> 3) * 1024 + (r & 7) * 128);
        bool ok = true;
        if (is_a) ok = decode_rows<WA>(pl, grow, r, tile_off, smem_u32(tiles), ring_base, gs, nk, lane);
        else ok = decode_rows<WB>(pl, grow, r, tile_off, smem_u32(tiles), ring_base, gs, nk, lane);
        if (!ok) gs.failed = 1;

        // ---------------- epilogue ----------------
        bool done = ok && warp < kEpilogueWarps && mbar_wait(&gs.accum, 0);
        done = __all_sync(0xFFFFFFFFu, done);
        if (warp >= kEpilogueWarps) {
            // decoders 8-11 have no accumulator lanes to drain
        } else if (done) {
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

}  // namespace bdr

#include "mx_gemm_pair.cuh"
#include "mx_gemm_dense.cuh"
#include "mx_gemm_f8.cuh"

namespace bdr {

template <int WA, int WB>
static int launch_gemm(const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, float* c, int64_t ldc,
                       const int* gate, cudaStream_t st) {
    auto kern = mx_gemm_kernel<WA, WB>;
    const size_t smem = (size_t)kStages * kStageBytes + 256 + (size_t)(kBM + kBN) * RingStride<WA, WB>::value + 1024;
    static PerDevice once;  // per instantiation
    if (kernel_setup(once, kern, kGemmThreads, smem) < 1) return BDR_ERR_CUDA;
    const dim3 grid((unsigned)(N / kBN), (unsigned)(M / kBM));
    kern<<<grid, kGemmThreads, smem, st>>>(a, b, M, N, K, c, ldc, gate);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <int WA>
static int gemm_pick_b(int mb, const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, float* c,
                       int64_t ldc, const int* gate, cudaStream_t st) {
    // 2-CTA kernel when the shape allows whole 256-row pairs and 256-element K chunks
    const bool pair = M % 256 == 0 && K % kChunkK == 0 && M / 128 <= 0x7FFFFFFF && N / 256 <= 65535;
    switch (mb) {
        case 2: { const int rc = pair ? launch_gemm_pair<WA, 3>(a, b, M, N, K, c, ldc, gate, st) : BDR_ERR_UNSUPPORTED;
                  return rc == BDR_ERR_UNSUPPORTED ? launch_gemm<WA, 3>(a, b, M, N, K, c, ldc, gate, st) : rc; }
        case 4: { const int rc = pair ? launch_gemm_pair<WA, 5>(a, b, M, N, K, c, ldc, gate, st) : BDR_ERR_UNSUPPORTED;
                  return rc == BDR_ERR_UNSUPPORTED ? launch_gemm<WA, 5>(a, b, M, N, K, c, ldc, gate, st) : rc; }
        case 7: { const int rc = pair ? launch_gemm_pair<WA, 8>(a, b, M, N, K, c, ldc, gate, st) : BDR_ERR_UNSUPPORTED;
                  return rc == BDR_ERR_UNSUPPORTED ? launch_gemm<WA, 8>(a, b, M, N, K, c, ldc, gate, st) : rc; }
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr

using namespace bdr;

// mx_gemm with an optional device-side gate: with gate != nullptr the kernel runs only if *gate != 0
static int mx_gemm_gated(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
                         int64_t N, int64_t K, float* c, int64_t ldc, const int* gate, void* stream) {
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
        case 2: return gemm_pick_b<3>(cfg_b->m, *a, *b, M, N, K, c, ldc, gate, st);
        case 4: return gemm_pick_b<5>(cfg_b->m, *a, *b, M, N, K, c, ldc, gate, st);
        case 7: return gemm_pick_b<8>(cfg_b->m, *a, *b, M, N, K, c, ldc, gate, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

extern "C" {

// Scratch memory lent to mx_gemm by the caller (bdr_set_workspace), per device.
struct LentWorkspace { void* ptr; int64_t bytes; };
static LentWorkspace g_lent[kMaxDevices] = {};
static std::mutex g_lent_mu;  // bdr_set_workspace on one thread, mx_gemm on another

int bdr_set_workspace(void* workspace, int64_t workspace_bytes) {
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return BDR_ERR_CUDA;
    if (workspace && ((uintptr_t)workspace % 256 || workspace_bytes < 0)) return BDR_ERR_MISALIGNED;
    std::lock_guard<std::mutex> lock(g_lent_mu);
    g_lent[dev].ptr = workspace;
    g_lent[dev].bytes = workspace ? workspace_bytes : 0;
    return BDR_OK;
}

int mx_gemm_ws(const bdr_config_t*, const bdr_planes_t*, const bdr_config_t*, const bdr_planes_t*, int64_t, int64_t, int64_t, float*,
               int64_t, void*, int64_t, void*);
int mx_gemm_f8(const bdr_config_t*, const bdr_planes_t*, const bdr_config_t*, const bdr_planes_t*, int64_t, int64_t, int64_t, float*,
               int64_t, void*, int64_t, void*);
int64_t mx_gemm_workspace_bytes(int64_t, int64_t, int64_t);
int64_t mx_gemm_f8_workspace_bytes(int64_t, int64_t, int64_t);

int mx_gemm(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
            int64_t N, int64_t K, float* c, int64_t ldc, void* stream) {
    // with scratch memory lent by the caller the two-phase kernels are the faster way to the same product
    LentWorkspace w = {};
    if (cfg_a && cfg_b && M > 0 && N > 0 && M % 256 == 0 && N % 256 == 0 && K % 256 == 0) {
        const int dev = current_device();
        if (dev >= 0 && dev < kMaxDevices) {
            std::lock_guard<std::mutex> lock(g_lent_mu);
            w = g_lent[dev];
        }
    }
    if (w.ptr) {
        int rc = BDR_ERR_UNSUPPORTED;
        if (cfg_a->m <= 4 && cfg_b->m <= 4 && w.bytes >= mx_gemm_f8_workspace_bytes(M, N, K))
            rc = mx_gemm_f8(cfg_a, a, cfg_b, b, M, N, K, c, ldc, w.ptr, w.bytes, stream);
        else if (w.bytes >= mx_gemm_workspace_bytes(M, N, K))
            rc = mx_gemm_ws(cfg_a, a, cfg_b, b, M, N, K, c, ldc, w.ptr, w.bytes, stream);
        if (rc != BDR_ERR_UNSUPPORTED && rc != BDR_ERR_WORKSPACE) return rc;
    }
    return mx_gemm_gated(cfg_a, a, cfg_b, b, M, N, K, c, ldc, nullptr, stream);
}

// Workspace of mx_gemm_f8: both operands as E4M3 bytes, their scale atoms, and the flag word.
int64_t mx_gemm_f8_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0) return 0;
    return ((M + N) * K + (M + N) * K / 32 + 255) / 256 * 256 + 256;
}

int mx_gemm_f8(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
               int64_t N, int64_t K, float* c, int64_t ldc, void* workspace, int64_t workspace_bytes, void* stream) {
    if (!cfg_a || !cfg_b || !a || !b || !c) return BDR_ERR_NULL;
    for (const bdr_config_t* cf : {cfg_a, cfg_b}) {
        if (cf->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
        if (cf->d1 != 8 || cf->k1 < 1 || cf->k2 < 1 || cf->k1 % cf->k2 != 0 || cf->d2 < 0 || cf->d2 > 3 || cf->m < 1 || cf->m > 8)
            return BDR_ERR_BAD_CONFIG;
        if (cf->k1 != 16 || cf->k2 != 2 || cf->d2 != 1 || (cf->m != 2 && cf->m != 4)) return BDR_ERR_UNSUPPORTED;
    }
    if (M < 0 || N < 0 || K < 0 || ldc < N) return BDR_ERR_SIZE;
    if (M == 0 || N == 0) return BDR_OK;
    if (M % 256 || N % 256 || K % 256 || K == 0) return BDR_ERR_UNSUPPORTED;
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31) || (M / 256) * (N / 256) >= (1ll << 30)) return BDR_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < mx_gemm_f8_workspace_bytes(M, N, K)) return BDR_ERR_WORKSPACE;
    if ((uintptr_t)workspace % 256) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* wa = static_cast<uint8_t*>(workspace);
    uint8_t* wb = wa + M * K;
    uint8_t* sfa = wb + N * K;
    uint8_t* sfb = sfa + M * K / 32;
    int* flag = reinterpret_cast<int*>(wa + mx_gemm_f8_workspace_bytes(M, N, K) - 256);
    // the fall-back's argument checks run first, so that nothing is launched for a call that would fail later
    for (const bdr_planes_t* p : {a, b}) {
        if (!p->exps || !p->micro || !p->elems) return BDR_ERR_NULL;
        if (((uintptr_t)p->exps | (uintptr_t)p->micro | (uintptr_t)p->elems) % 16) return BDR_ERR_MISALIGNED;
        if ((p->ld_exps | p->ld_micro | p->ld_elems) % 16) return BDR_ERR_MISALIGNED;
    }
    if (a->ld_exps < K / 16 || a->ld_micro < K / 16 || a->ld_elems < K * (cfg_a->m + 1) / 8) return BDR_ERR_SIZE;
    if (b->ld_exps < K / 16 || b->ld_micro < K / 16 || b->ld_elems < K * (cfg_b->m + 1) / 8) return BDR_ERR_SIZE;
    if ((uintptr_t)c % 16 || ldc % 4) return BDR_ERR_MISALIGNED;
    if (cudaMemsetAsync(flag, 0, sizeof(int), st) != cudaSuccess) return BDR_ERR_CUDA;
    const F8Plan plan = plan_gemm_f8(M, N, K);
    const ZeroTiles z = {c, ldc, plan.tiles_n, plan.tiles_full, plan.split_tiles(), plan.tiles_m, plan.band_rows};
    int rc = reencode_rowwise_e4m3(*a, cfg_a->m, *b, cfg_b->m, M, N, K, wa, wb, sfa, sfb, flag, z, st);  // phase 1
    if (rc != BDR_OK) return rc;
    rc = launch_gemm_f8(wa, wb, sfa, sfb, M, N, K, plan, c, ldc, flag, st);                               // phase 2, if exact
    if (rc != BDR_OK) return rc;
    return mx_gemm_gated(cfg_a, a, cfg_b, b, M, N, K, c, ldc, flag, stream);                           // else the bf16 kernel
}

int mx_gemm_e4m3(const uint8_t* a, const uint8_t* scales_a, const uint8_t* b, const uint8_t* scales_b, int64_t M, int64_t N, int64_t K,
                 float* c, int64_t ldc, void* stream) {
    if (!a || !scales_a || !b || !scales_b || !c) return BDR_ERR_NULL;
    if (M < 0 || N < 0 || K < 0 || ldc < N) return BDR_ERR_SIZE;
    if (M == 0 || N == 0) return BDR_OK;
    if (M % 256 || N % 256 || K % 256 || K == 0) return BDR_ERR_UNSUPPORTED;
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31) || (M / 256) * (N / 256) >= (1ll << 30)) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)a | (uintptr_t)b | (uintptr_t)scales_a | (uintptr_t)scales_b | (uintptr_t)c) % 16 || ldc % 4) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    const F8Plan plan = plan_gemm_f8(M, N, K);
    if (plan.split_tiles() > 0) {
        const ZeroTiles z = {c, ldc, plan.tiles_n, plan.tiles_full, plan.split_tiles(), plan.tiles_m, plan.band_rows};
        zero_tiles_kernel<<<dim3((unsigned)z.count, 4), 256, 0, st>>>(z);
        if (cudaGetLastError() != cudaSuccess) return BDR_ERR_CUDA;
    }
    return launch_gemm_f8(a, b, scales_a, scales_b, M, N, K, plan, c, ldc, nullptr, st);
}

int bdr_reencode_e4m3(const bdr_config_t* cfg, const bdr_planes_t* in, int64_t rows, int64_t K, uint8_t* out, uint8_t* scales,
                      int* inexact_dev, void* stream) {
    if (!cfg || !in || !out || !scales || !inexact_dev) return BDR_ERR_NULL;
    if (cfg->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
    if (cfg->d1 != 8 || cfg->k1 < 1 || cfg->k2 < 1 || cfg->k1 % cfg->k2 != 0 || cfg->d2 < 0 || cfg->d2 > 3 || cfg->m < 1 || cfg->m > 8)
        return BDR_ERR_BAD_CONFIG;
    if (cfg->k1 != 16 || cfg->k2 != 2 || cfg->d2 != 1 || (cfg->m != 2 && cfg->m != 4)) return BDR_ERR_UNSUPPORTED;
    if (rows < 0 || K < 0) return BDR_ERR_SIZE;
    if (rows == 0 || K == 0) return BDR_OK;
    if (rows % 128 || K % 128) return BDR_ERR_UNSUPPORTED;
    if (!in->exps || !in->micro || !in->elems) return BDR_ERR_NULL;
    if (((uintptr_t)in->exps | (uintptr_t)in->micro | (uintptr_t)in->elems | (uintptr_t)out | (uintptr_t)scales) % 16) return BDR_ERR_MISALIGNED;
    if ((in->ld_exps | in->ld_micro | in->ld_elems) % 4) return BDR_ERR_MISALIGNED;
    if (in->ld_exps < K / 16 || in->ld_micro < K / 16 || in->ld_elems < K * (cfg->m + 1) / 8) return BDR_ERR_SIZE;
    const bdr_planes_t none = {};
    const ZeroTiles z = {nullptr, 0, 1, 0, 0, 1, 1};
    return reencode_rowwise_e4m3(*in, cfg->m, none, cfg->m, rows, 0, K, out, nullptr, scales, nullptr, inexact_dev, z, (cudaStream_t)stream);
}

int64_t mx_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0) return 0;
    return ((M + N) * K * 2 + 255) / 256 * 256;
}

int mx_gemm_ws(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
               int64_t N, int64_t K, float* c, int64_t ldc, void* workspace, int64_t workspace_bytes, void* stream) {
    if (!cfg_a || !cfg_b || !a || !b || !c) return BDR_ERR_NULL;
    for (const bdr_config_t* cf : {cfg_a, cfg_b}) {
        if (cf->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
        if (cf->d1 != 8 || cf->k1 < 1 || cf->k2 < 1 || cf->k1 % cf->k2 != 0 || cf->d2 < 0 || cf->d2 > 3 || cf->m < 1 || cf->m > 8)
            return BDR_ERR_BAD_CONFIG;
        if (cf->k1 != 16 || cf->k2 != 2 || cf->d2 != 1 || (cf->m != 2 && cf->m != 4 && cf->m != 7)) return BDR_ERR_UNSUPPORTED;
    }
    if (M < 0 || N < 0 || K < 0 || ldc < N) return BDR_ERR_SIZE;
    if (M == 0 || N == 0) return BDR_OK;
    if (M % 256 || N % 256 || K % kBK || K == 0) return BDR_ERR_UNSUPPORTED;
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31) || (M / 256) * (N / 256) >= (1ll << 30)) return BDR_ERR_UNSUPPORTED;
    for (const bdr_planes_t* p : {a, b}) {
        if (!p->exps || !p->micro || !p->elems) return BDR_ERR_NULL;
        if (((uintptr_t)p->exps | (uintptr_t)p->micro | (uintptr_t)p->elems) % 16) return BDR_ERR_MISALIGNED;
        if ((p->ld_exps | p->ld_micro | p->ld_elems) % 16) return BDR_ERR_MISALIGNED;
    }
    if (a->ld_exps < K / 16 || a->ld_micro < K / 16 || a->ld_elems < K * (cfg_a->m + 1) / 8) return BDR_ERR_SIZE;
    if (b->ld_exps < K / 16 || b->ld_micro < K / 16 || b->ld_elems < K * (cfg_b->m + 1) / 8) return BDR_ERR_SIZE;
    if ((uintptr_t)c % 16 || ldc % 4) return BDR_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < mx_gemm_workspace_bytes(M, N, K)) return BDR_ERR_WORKSPACE;
    if ((uintptr_t)workspace % 256) return BDR_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    __nv_bfloat16* wa = static_cast<__nv_bfloat16*>(workspace);
    __nv_bfloat16* wb = wa + M * K;
    const bdr_config_t* cfs[2] = {cfg_a, cfg_b};
    const bdr_planes_t* pls[2] = {a, b};
    __nv_bfloat16* outs[2] = {wa, wb};
    const int64_t rows[2] = {M, N};
    const GemmPlan plan = plan_gemm(M, N, K / kBK, (M + N) * K * 2);
    bool first_fast = false;
    for (int i = 0; i < 2; ++i) {  // phase 1: both operands to bf16, once
        QParams qp;
        qp.k1 = 16; qp.k2 = 2; qp.d2 = 1; qp.m = cfs[i]->m; qp.rounding = cfs[i]->rounding; qp.beta = 1; qp.qmax = (1u << cfs[i]->m) - 1u;
        // the second decode starts while the first drains (it is chained only when the first ran on the same kernel family)
        int rc = unpack_rowwise_mx_x2(*pls[i], outs[i], rows[i], K, K, qp, st, i == 1 && first_fast);
        if (i == 0) first_fast = rc == BDR_OK;
        if (rc == BDR_ERR_UNSUPPORTED) rc = unpack_rowwise_mx<__nv_bfloat16>(*pls[i], outs[i], rows[i], K, K, qp, st);
        if (rc == BDR_ERR_UNSUPPORTED) rc = unpack_general<__nv_bfloat16>(*pls[i], outs[i], rows[i], K, K, 1, qp, st);
        if (rc != BDR_OK) return rc;
        // the tiles that two clusters add into are cleared between the two decodes, as a link of the same chain
        if (i == 0 && zero_split_tiles(plan, c, ldc, st, true) != BDR_OK) return BDR_ERR_CUDA;
    }
    return launch_gemm_dense(wa, wb, M, N, K, plan, c, ldc, st);  // phase 2
}

int mx_gemm_status(void) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)) != cudaSuccess) return BDR_ERR_CUDA;
    return v;
}

}  // extern "C"
