// Row-direction (axis 1) unpack to bf16 for the Table II family on packed bf16x2 arithmetic: the mirror
// image of the packing kernel in bdr_row_x2.cu.  A warp streams runs of 2048 elements: lane 0 brings
// the run's 256 W code bytes, 128 exponent bytes and 128 microexponent bytes into a three-stage ring
// with three bulk copies on one barrier; each lane decodes four blocks (two per half run) and writes
// every block with one 32-byte store.
#include "bdr_async.cuh"
#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

using bf16 = __nv_bfloat16;

constexpr int kUThreads = 128;
constexpr int kUWarps = kUThreads / 32;
constexpr int kUStages = 3;
constexpr int kURunElems = 2048;
constexpr int kUHalfElems = 1024;
constexpr int kUBarBytes = 128;

template <int W> struct UStage {
    static constexpr int kElemBytes = kURunElems / 8 * W;
    static constexpr int kExpBytes = kURunElems / 16;
    static constexpr int kBytes = kElemBytes + 2 * kExpBytes;  // a multiple of 128
};

using URunIndex = x2::RunIndex;

template <int W>
__global__ void __launch_bounds__(kUThreads)
unpack_row_x2_kernel(bdr_planes_t in, bf16* y, URunIndex ri, uint32_t total, int* status) {
    using US = UStage<W>;
    constexpr int S = kUStages;
    // a kernel launched behind this one as a programmatic dependent (the second phase of mx_gemm_ws) may begin its
    // set-up now; it still waits for this grid to finish before it reads y.  Without such a launch: no effect
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    extern __shared__ __align__(128) uint8_t smem[];  // ring [warp][stage][codes | exponents | microexponents], barriers
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring0 = async::smem_u32(smem) + warp * S * US::kBytes;
    const uint32_t bars = async::smem_u32(smem) + kUWarps * S * US::kBytes + warp * S * 8;
    const uint32_t stride = gridDim.x * kUWarps;
    const uint32_t w0 = blockIdx.x * kUWarps + warp;
    auto load = [&](uint32_t wi, int st) {  // lane 0 only
        int64_t row, pos;
        ri.split(wi, row, pos);
        const int64_t blk0 = pos * (kURunElems / 16);
        const uint32_t dst = ring0 + st * US::kBytes, bar = bars + 8 * st;
        async::mbar_expect_tx(bar, US::kBytes);
        async::bulk_load(dst, in.elems + row * in.ld_elems + blk0 * 2 * W, US::kElemBytes, bar);
        async::bulk_load(dst + US::kElemBytes, in.exps + row * in.ld_exps + blk0, US::kExpBytes, bar);
        async::bulk_load(dst + US::kElemBytes + US::kExpBytes, in.micro + row * in.ld_micro + blk0, US::kExpBytes, bar);
    };
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < S; ++s) async::mbar_init(bars + 8 * s, 1);
        async::fence_barrier_init();
#pragma unroll
        for (int s = 0; s < S; ++s)
            if (w0 + s * stride < total) load(w0 + s * stride, s);
    }
    __syncwarp();
    int st = 0;
    uint32_t phase = 0;
    for (uint32_t wi = w0; wi < total; wi += stride) {
        if (!async::mbar_wait(bars + 8 * st, phase)) {
            async::report_timeout(status);
            // Nothing more is issued.  The copies queued for this and the next S - 1 runs may still be on their way into
            // this CTA's shared memory: one further bounded wait for each, so that the CTA does not knowingly leave with
            // a copy in flight (if one still does not land, the CTA leaves all the same: the wait must end).
            if (lane == 0) {
                for (int k = 0; k < S; ++k) {
                    if ((uint64_t)wi + (uint64_t)k * stride >= total) break;
                    int ds = st + k;
                    uint32_t dp = phase;
                    if (ds >= S) { ds -= S; dp ^= 1; }
                    async::mbar_wait(bars + 8 * ds, dp);
                }
            }
            break;
        }
        const uint32_t stage = ring0 + st * US::kBytes;
        uint32_t s[2][W], Fw[2], mw[2];
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            const uint32_t src = stage + sub * (kUHalfElems / 8 * W) + lane * 4 * W;
            if constexpr (W == 8) {
                const uint4 a = async::lds128(src), b = async::lds128(src + 16);
                s[sub][0] = a.x; s[sub][1] = a.y; s[sub][2] = a.z; s[sub][3] = a.w;
                s[sub][4] = b.x; s[sub][5] = b.y; s[sub][6] = b.z; s[sub][7] = b.w;
            } else {
#pragma unroll
                for (int k = 0; k < W; ++k) s[sub][k] = async::lds32(src + 4 * k);
            }
            Fw[sub] = async::lds16(stage + US::kElemBytes + sub * (kUHalfElems / 16) + 2 * lane);
            mw[sub] = async::lds16(stage + US::kElemBytes + US::kExpBytes + sub * (kUHalfElems / 16) + 2 * lane);
        }
        __syncwarp();  // every lane has read stage st
        if (lane == 0 && wi + S * stride < total) load(wi + S * stride, st);
        int64_t row, pos;
        ri.split(wi, row, pos);
        bf16* yrun = y + row * ri.ld + pos * kURunElems + lane * 32;
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            const uint32_t F0 = Fw[sub] & 0xFFu, F1 = Fw[sub] >> 8;
            uint32_t yw[16];
            if ((F0 - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF)) && (F1 - x2::kMinF <= (uint32_t)(x2::kMaxDecodeF - x2::kMinF))) {
                x2::decode_two_blocks_row<W>(s[sub], F0, F1, mw[sub], yw);
            } else {
                x2::TwoBlocks<W> in2;
#pragma unroll
                for (int k = 0; k < W; ++k) in2.s[k] = s[sub][k];
                const x2::TwoBlocksOut o = x2::decode_two_blocks_slow<W>(in2, F0, F1, mw[sub]);
#pragma unroll
                for (int k = 0; k < 16; ++k) yw[k] = o.y[k];
            }
            async::stg256(yrun + sub * kUHalfElems, yw);
            async::stg256(yrun + sub * kUHalfElems + 16, yw + 8);
        }
        if (++st == S) { st = 0; phase ^= 1; }
    }
    // Launched as a programmatic dependent of the kernel before it (the second operand's decode behind the first's in
    // mx_gemm_ws: the two do not depend on each other, so this one starts while that one drains), this grid must not
    // finish first: whoever waits for this grid then also has the other one's results.  Otherwise: no effect.
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int W>
static int launch_unpack_x2(const bdr_planes_t& in, bf16* y, int64_t rows, int64_t cols, int64_t ld, bool flat, cudaStream_t st, bool chained) {
    const int64_t rpr = cols / kURunElems, total = rows * rpr;
    if (total == 0) return BDR_OK;
    if (total >= (1ll << 31) - (1ll << 24)) return BDR_ERR_UNSUPPORTED;
    auto kern = unpack_row_x2_kernel<W>;
    const size_t smem = kUWarps * kUStages * UStage<W>::kBytes + kUBarBytes;
    static PerDevice once;  // per instantiation
    const int blocks_per_sm = kernel_setup(once, kern, kUThreads, smem);
    if (blocks_per_sm < 1) return BDR_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return BDR_ERR_CUDA;
    const int64_t need = (total + kUWarps - 1) / kUWarps;
    const int grid = (int)max((int64_t)1, min(need, (int64_t)sm_count() * blocks_per_sm));
    URunIndex ri;
    ri.runs_per_row = make_fastdiv((uint32_t)rpr);
    ri.ld = ld;
    ri.flat = flat ? 1 : 0;
    if (!chained) {
        kern<<<grid, kUThreads, smem, st>>>(in, y, ri, (uint32_t)total, status);
        return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kUThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, in, y, ri, (uint32_t)total, status);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Whole 2048-element runs, 32-byte aligned output rows; a contiguous tensor with tight planes is one long row.
// chained: launch as a programmatic dependent of the kernel before it in the stream, which must be another launch of this
// function whose output this one does not read (see the end of the kernel).
int unpack_rowwise_mx_x2(const bdr_planes_t& in, bf16* y, int64_t rows, int64_t cols, int64_t ld, const QParams& qp,
                         cudaStream_t st, bool chained) {
    if (qp.k1 != 16 || qp.k2 != 2 || qp.d2 != 1) return BDR_ERR_UNSUPPORTED;
    if (((uintptr_t)y % 32) || (ld * 2) % 32 || cols % 16 != 0) return BDR_ERR_UNSUPPORTED;
    const int W = qp.m + 1;
    bool flat = false;
    if (rows > 1 && ld == cols && in.ld_elems == cols / 8 * W && in.ld_exps == cols / 16 && in.ld_micro == cols / 16) {
        cols *= rows;
        ld = cols;
        rows = 1;
    }
    flat = rows == 1;
    if (cols % kURunElems != 0) return BDR_ERR_UNSUPPORTED;
    switch (qp.m) {
        case 2: return launch_unpack_x2<3>(in, y, rows, cols, ld, flat, st, chained);
        case 4: return launch_unpack_x2<5>(in, y, rows, cols, ld, flat, st, chained);
        case 7: return launch_unpack_x2<8>(in, y, rows, cols, ld, flat, st, chained);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
