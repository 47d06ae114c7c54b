// Exact re-encoding of packed MX operands (k1 = 16, k2 = 2, d2 = 1, m <= 4: MX4 and MX6 of Table II) onto
// the block-scaled 8-bit tensor-core format: E4M3 elements with one power-of-two scale (an 8-bit
// exponent, "E8M0") per 32 elements along K.
//
// A decoded element is +-q * 2^(F - 127 - (m-1) - tau) with q < 2^m <= 16: at most four significant
// bits, which is what E4M3 holds.  Two neighbouring 16-element blocks share one scale byte
// sb = max(F0, F1) - 7 (scale 2^(sb-127)), so an element becomes q * 2^t with
// t = 7 - (m-1) - (max(F0,F1) - F) - tau <= 6, at most 15 * 2^4 = 240 < 448.  E4M3 holds every multiple of
// 2^-9 with four significant bits, so the element is exact whenever t >= -9, i.e. whenever the two block
// exponents of a group differ by less than about 12; below that it is still exact if q is a multiple of
// 2^(-9-t).  Anything else (also blocks with F < 16 that are not all zero, and F = 255) cannot be
// represented: the kernel then raises *inexact and the caller's product falls back to the bf16 path.
//
// Scale bytes are written in the layout the tensor core's scale-factor copy expects: for every tile of
// 128 rows x 128 K a 512-byte atom with byte (r % 32) * 16 + (r / 32) * 4 + (k / 32) for row r of the
// tile, atoms ordered [K chunk][row tile].
#include <cuda_fp16.h>

#include "bdr_x2.cuh"
#include "bdr_host.h"

namespace bdr {

constexpr int kF8Threads = 128;
constexpr int kF8Warps = kF8Threads / 32;
constexpr int kF8Rows = 2;                               // rows per warp, all in flight at once
constexpr int kF8StripRows = kF8Warps * kF8Rows;        // rows per CTA (divides 128)

__device__ __forceinline__ uint32_t cvt_e4m3x2(uint32_t h2) {
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(d) : "r"(h2));
    return d;
}
__device__ __forceinline__ uint32_t f16x2_sub(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t f16x2_mul(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// bits [pos, pos + len) of x with a left and a right shift (kept apart from the optimiser, which would turn them
// into a shift and a mask, two operations of the integer pipe; the left shift can go to the multiplier)
__device__ __forceinline__ uint32_t field_of(uint32_t x, int pos, int len) {
    uint32_t t, f;
    asm("shl.b32 %0, %1, %2;" : "=r"(t) : "r"(x), "r"(32 - pos - len));
    asm("shr.u32 %0, %1, %2;" : "=r"(f) : "r"(t), "r"(32 - len));
    return f;
}

// One 16-element block: W code words (LSB-first stream of 16 (m+1)-bit codes starting at bit 0 of w[0])
// -> 16 E4M3 bytes in o[0..3].  d = (group exponent - this block's exponent), micro: tau bit per pair.
// Returns true if some element is not representable.
template <int W>
__device__ __forceinline__ bool reencode_block(const uint32_t* w, int bit0, int d, uint32_t micro, uint32_t* o) {
    constexpr int m = W - 1;
    constexpr uint32_t qmask = (1u << m) - 1u, cmask = (1u << W) - 1u;
    bool bad = false;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int b0 = bit0 + 2 * j * W;  // two codes, 2 W <= 10 bits, from at most two words
        const uint32_t lo = w[b0 >> 5], hi = w[((b0 + 2 * W - 1) >> 5)];
        const uint32_t two = __funnelshift_r(lo, hi, b0 & 31);
        const uint32_t c0 = two & cmask, c1 = (two >> W) & cmask;
        const uint32_t q0 = c0 & qmask, q1 = c1 & qmask;
        const int t = 7 - (m - 1) - d - (int)((micro >> j) & 1u);
        // q as fp16 through 1024 + q, times 2^max(t, -14): exact
        const uint32_t qh = f16x2_sub(0x64006400u | q0 | (q1 << 16), 0x64006400u);
        const uint32_t sc = (uint32_t)(15 + max(t, -14)) << 10;
        uint32_t v = f16x2_mul(qh, sc * 0x10001u);
        if (t < -9) {  // rare: the low bits of q fall below the finest E4M3 step
            const uint32_t lost = (1u << min(-9 - t, 4)) - 1u;
            bad |= ((q0 | q1) & lost) != 0;
        }
        v |= ((c0 >> m) << 15) | ((c1 >> m) << 31);
        const uint32_t e2 = cvt_e4m3x2(v);
        if (j & 1) o[j >> 1] |= e2 << 16;
        else o[j >> 1] = e2;
    }
    return bad;
}

// The general formulation of a group, out of line: any exponent gap, zero blocks, tiny and NaN blocks.
template <int W>
struct GroupWords { uint32_t w[W]; };
struct GroupOut { uint32_t o[8]; uint32_t sb; bool bad; };
template <int W>
__device__ __noinline__ GroupOut reencode_group_slow(GroupWords<W> in, uint32_t F2, uint32_t m2) {
    GroupOut r;
    const int F0 = (int)(F2 & 0xFFu), F1 = (int)(F2 >> 8);
    const int S = max(F0, F1);
    r.sb = 0;
    r.bad = false;
    if (S >= 16 && S < 255) {
        r.sb = (uint32_t)(S - 7);
        // a block with F < 16 beside a normal one is representable only if it is all zero: d = 64 sends every t
        // below -14, where any non-zero q raises the flag
        const int d0 = (F0 >= 16) ? S - F0 : 64, d1 = (F1 >= 16) ? S - F1 : 64;
        r.bad |= reencode_block<W>(in.w, 0, d0, m2 & 0xFFu, r.o);
        r.bad |= reencode_block<W>(in.w, 16 * W, d1, m2 >> 8, r.o + 4);
    } else {
        // exponents outside the range handled here: zeros if every magnitude is zero, else not representable
        r.bad |= reencode_block<W>(in.w, 0, 64, 0, r.o);
        r.bad |= reencode_block<W>(in.w, 16 * W, 64, 0, r.o + 4);
        r.bad |= S == 255;
    }
    return r;
}

// One 32-element group: the lane's W code words, two exponent bytes and two microexponent bytes -> 32 bytes
// at `dst` and the group's scale byte (returned).
//
// Fast path (both exponents >= 16, at most 13 - m binades apart): packed bf16x2 arithmetic as in the
// unpack kernels, with the block exponent replaced by 14 - d, so that q * scale comes out as the bf16
// number whose exponent field IS the E4M3 exponent field (bf16 subnormals line up with E4M3 subnormals
// the same way).  The E4M3 byte is then bits 4..10 of the bf16 pattern, and the sign comes straight from
// the code.
template <int W>
__device__ __forceinline__ uint32_t reencode_group(const uint32_t (&w)[W], uint32_t F2, uint32_t m2, uint8_t* dst, bool& bad) {
    constexpr int M = W - 1;
    constexpr uint32_t kQ2 = ((1u << M) - 1u) * 0x10001u;
    const int F0 = (int)(F2 & 0xFFu), F1 = (int)(F2 >> 8);
    const int S = max(F0, F1), lo = min(F0, F1);
    uint32_t o[8];
    uint32_t sb;
    if (lo >= 16 && S < 255 && S - lo <= 13 - M) {
        sb = (uint32_t)(S - 7);
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            const uint32_t Fp = (uint32_t)(14 - (S - (b ? F1 : F0))), mbb = b ? m2 >> 8 : m2;
            const uint32_t sc0 = ((Fp - (uint32_t)(M - 1)) << 7) * 0x10001u;  // scale 2^p for tau = 0, both halves
            uint32_t v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // the pair's 2 W code bits (a field inside one word comes out with a left and a right shift, no
                // mask), copied three times by one multiply: code 0 ends up with its magnitude at bits 0.. and
                // its sign at bit 15, code 1 with its magnitude at bits 16.. and its sign at bit 31
                const int bit = 2 * W * (8 * b + j), wi = bit >> 5, sh = bit & 31;
                uint32_t f;
                if (sh + 2 * W > 32) f = __funnelshift_r(w[wi], w[wi + 1], sh) & ((1u << (2 * W)) - 1u);
                else f = field_of(w[wi], sh, 2 * W);
                const uint32_t c3 = f * (1u + (1u << (16 - W)) + (1u << (32 - 2 * W)));
                // tau lowers the exponent by one: sc0 - 0x0080 per half, as one multiply-add; the constant term
                // -128 * 2^p is a packed multiply (both on the FMA pipe, the integer pipe is the busy one)
                const uint32_t sc = ((mbb << (7 - j)) & 0x80u) * 0xFFFEFFFFu + sc0;
                const uint32_t y = x2::hfma2((c3 & kQ2) | 0x43004300u, sc, x2::hmul2(sc, 0xC300C300u));  // (128 + q) 2^p - 128 2^p
                // bits 4..10 of each half move to bits 8..14 (a multiply) and the sign bits join them: the E4M3
                // bytes are bytes 1 and 3
                v[j] = y * 16u + (c3 & x2::kSign2);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) o[4 * b + k] = __byte_perm(v[2 * k], v[2 * k + 1], 0x7531);
        }
    } else {
        GroupWords<W> in;
#pragma unroll
        for (int k = 0; k < W; ++k) in.w[k] = w[k];
        const GroupOut r = reencode_group_slow<W>(in, F2, m2);
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = r.o[k];
        sb = r.sb;
        bad |= r.bad;
    }
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
    return sb;
}

// A warp takes a row segment of 32 groups (1024 elements), one group per lane, so the code words, the
// exponent bytes and the output bytes of a warp are contiguous; every thread has kF8Rows rows in flight.
// The four scale bytes of a 128-element K chunk travel to the lane of the chunk's first group and leave
// as one word of the chunk's atom.
template <int W>
__device__ __forceinline__ void reencode_rows(const bdr_planes_t& in, int64_t K, int64_t row0, int64_t seg, uint8_t* out, uint8_t* sf,
                                              int64_t row_tiles, int* inexact) {
    const int lane = threadIdx.x & 31;
    const int64_t group = seg * 32 + lane;
    const bool live = group * 32 < K;
    uint32_t w[kF8Rows][W], F2[kF8Rows], m2[kF8Rows];
    if (live) {
#pragma unroll
        for (int i = 0; i < kF8Rows; ++i) {
            const int64_t row = row0 + i;
            const uint32_t* codes = reinterpret_cast<const uint32_t*>(in.elems + row * in.ld_elems + group * 4 * W);
#pragma unroll
            for (int k = 0; k < W; ++k) w[i][k] = __ldg(codes + k);
            F2[i] = __ldg(reinterpret_cast<const uint16_t*>(in.exps + row * in.ld_exps + group * 2));
            m2[i] = __ldg(reinterpret_cast<const uint16_t*>(in.micro + row * in.ld_micro + group * 2));
        }
    }
    bool bad = false;
#pragma unroll
    for (int i = 0; i < kF8Rows; ++i) {
        const int64_t row = row0 + i;
        uint32_t sb = 0;
        if (live) sb = reencode_group<W>(w[i], F2[i], m2[i], out + row * K + group * 32, bad);
        uint32_t sb4 = sb | (__shfl_down_sync(0xFFFFFFFFu, sb, 1) << 8);
        sb4 |= __shfl_down_sync(0xFFFFFFFFu, sb4, 2) << 16;
        if (live && (lane & 3) == 0) {
            const int r = (int)(row & 127);
            *reinterpret_cast<uint32_t*>(sf + ((group >> 2) * row_tiles + (row >> 7)) * 512 + (r & 31) * 16 + (r >> 5) * 4) = sb4;
        }
    }
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicExch(inexact, 1);
}

// grid (row strips of A + row strips of B + tiles of C to clear, K segments): a CTA's warps take kF8Rows
// consecutive rows each
template <int WA, int WB>
__global__ void __launch_bounds__(kF8Threads)
reencode_e4m3_kernel(bdr_planes_t a, bdr_planes_t b, int a_strips, int b_strips, int64_t M, int64_t N, int64_t K, uint8_t* out_a,
                     uint8_t* out_b, uint8_t* sf_a, uint8_t* sf_b, int* inexact, ZeroTiles z) {
    // a kernel launched behind this one as a programmatic dependent may begin its own set-up now (it still
    // waits for this grid to finish before it reads what is written here); without such a launch: no effect
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5;
    if ((int)blockIdx.x >= a_strips + b_strips) {
        // extra CTAs: clear the 256 x 256 tiles of C that the GEMM kernel accumulates into
        const int t = z.tile0 + ((int)blockIdx.x - a_strips - b_strips);
        int tm, tn;
        gemm_tile_coords(t, z.tiles_m, z.tiles_n, z.band_rows, tm, tn);
        const int rows_per = (256 + (int)gridDim.y - 1) / (int)gridDim.y;
        const int r0 = (int)blockIdx.y * rows_per, r1 = min(256, r0 + rows_per);
        for (int idx = r0 * 64 + (int)threadIdx.x; idx < r1 * 64; idx += kF8Threads) {  // 64 chunks of 16 bytes per row
            const int r = idx >> 6, ch = idx & 63;
            *reinterpret_cast<uint4*>(z.c + ((int64_t)tm * 256 + r) * z.ldc + (int64_t)tn * 256 + ch * 4) = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    if ((int)blockIdx.x < a_strips) {
        const int64_t row0 = ((int64_t)blockIdx.x * kF8Warps + warp) * kF8Rows;
        reencode_rows<WA>(a, K, row0, blockIdx.y, out_a, sf_a, M / 128, inexact);
    } else {
        const int64_t row0 = ((int64_t)((int)blockIdx.x - a_strips) * kF8Warps + warp) * kF8Rows;
        reencode_rows<WB>(b, K, row0, blockIdx.y, out_b, sf_b, N / 128, inexact);
    }
}

template <int WA, int WB>
static int launch_reencode(const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, uint8_t* out_a, uint8_t* out_b,
                           uint8_t* sf_a, uint8_t* sf_b, int* inexact, const ZeroTiles& z, cudaStream_t st) {
    const int a_strips = (int)(M / kF8StripRows), b_strips = (int)(N / kF8StripRows);
    const dim3 grid((unsigned)(a_strips + b_strips + z.count), (unsigned)((K + 1023) / 1024));
    if (grid.x == 0) return BDR_OK;
    reencode_e4m3_kernel<WA, WB><<<grid, kF8Threads, 0, st>>>(a, b, a_strips, b_strips, M, N, K, out_a, out_b, sf_a, sf_b, inexact, z);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

// Operand A [M, K] and operand B [N, K] (either may have zero rows) in one launch.  M and N are multiples of
// 128, K a multiple of 128; m_a, m_b in {2, 4}; outputs 32-byte aligned, K bytes per row; scale atoms as
// described above, M * K / 32 and N * K / 32 bytes.  *inexact is set to 1 (never cleared) when an
// element cannot be represented.  z.count tiles of 256 x 256 floats of z.c are cleared on the side.
int reencode_rowwise_e4m3(const bdr_planes_t& a, int m_a, const bdr_planes_t& b, int m_b, int64_t M, int64_t N, int64_t K,
                          uint8_t* out_a, uint8_t* out_b, uint8_t* sf_a, uint8_t* sf_b, int* inexact, const ZeroTiles& z,
                          cudaStream_t st) {
    if (M % 128 || N % 128 || K % 128 || K <= 0) return BDR_ERR_UNSUPPORTED;
    if ((M + N) / kF8StripRows + z.count > 0x7FFFFFFF || (K + 1023) / 1024 > 65535) return BDR_ERR_UNSUPPORTED;
    if (m_a == 2 && m_b == 2) return launch_reencode<3, 3>(a, b, M, N, K, out_a, out_b, sf_a, sf_b, inexact, z, st);
    if (m_a == 2 && m_b == 4) return launch_reencode<3, 5>(a, b, M, N, K, out_a, out_b, sf_a, sf_b, inexact, z, st);
    if (m_a == 4 && m_b == 2) return launch_reencode<5, 3>(a, b, M, N, K, out_a, out_b, sf_a, sf_b, inexact, z, st);
    if (m_a == 4 && m_b == 4) return launch_reencode<5, 5>(a, b, M, N, K, out_a, out_b, sf_a, sf_b, inexact, z, st);
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr
