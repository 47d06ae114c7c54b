// mx_gemm_hw: C = A B^T computed the way the dot-product pipeline of Section IV-B (Fig. 6) computes it, from packed
// MX operands (Table II family, quantized along K).  Not a faster GEMM: a bit-faithful model of the narrow datapath,
// for studying what its fixed-point reduction does to a product.
//
//   * inside a 16-element block the integer mantissa products are summed exactly; the sum of sub-block j (two
//     products) carries the weight 2^(2 - tau_A,j - tau_B,j) (the conditional right shifts by the microexponents,
//     on a datapath two bits wider, so nothing is lost).  Here: the operands are decoded to the integers
//     +-q * 2^(1 - tau) as fp32 numbers (at most 8 significant bits), their products and the 16-term sum
//     (< 2^20) are exact in fp32, so plain (packed) multiply-adds give the block result D_b;
//   * the r/16 block results of a pass are aligned to the largest exponent sum e_max = max_b (F_A,b + F_B,b)
//     inside a frame of f magnitude bits and truncated toward zero: A_b = trunc(D_b * 2^(f - W - (e_max - e_b))),
//     W = m_A + m_B + 6 -- one exact fp32 multiplication by a power of two and one float-to-integer conversion
//     that rounds toward zero -- and added as integers;
//   * the pass's sum becomes an fp32 number (round to nearest even), is scaled by its power of two through fp64
//     (exact; overflow and underflow as a cast from double), and successive passes are added in fp32 in order.
// A CTA of 256 threads computes a 64 x 64 tile, a thread 4 x 4 outputs; per step of 64 elements of K the decoded
// operands sit in shared memory K-major (two packed blocks per thread are fetched one step ahead into registers).
#include <cuda_runtime.h>
#include <stdint.h>

#include "bdr.h"
#include "bdr_host.h"

namespace bdr {

constexpr int kHwTile = 64;      // rows of A and rows of B per CTA
constexpr int kHwStep = 64;      // elements of K per step (four blocks)
constexpr int kHwThreads = 256;

// d += a * b on two independent fp32 lanes; the pairs stay in 64-bit registers across the block's sixteen steps
__device__ __forceinline__ void hw_fma2(unsigned long long& d, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long hw_dup(float a) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(a));
    return r;
}
__device__ __forceinline__ void hw_split(unsigned long long d, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(d)); }

// One item = 32 consecutive elements of a row (two blocks): W words of codes, two exponent bytes, two microexponent bytes.
template <int W> struct HwItem {
    uint32_t cw[W];
    uint32_t exps, micro;  // 16 bits each
};

template <int W>
__device__ __forceinline__ void hw_fetch(const bdr_planes_t& p, int64_t row, int64_t blk /* even */, HwItem<W>& it) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.elems + row * p.ld_elems + blk * 2 * W);
#pragma unroll
    for (int i = 0; i < W; ++i) it.cw[i] = __ldg(src + i);
    it.exps = *reinterpret_cast<const uint16_t*>(p.exps + row * p.ld_exps + blk);
    it.micro = *reinterpret_cast<const uint16_t*>(p.micro + row * p.ld_micro + blk);
}

// +-q * 2^(1 - tau) of the item's 32 elements into the K-major tile: element e of half h goes to
// tile[(32 h + e) * 64 + (row ^ (h << 4))] (the XOR keeps groups of four rows together and spreads the two halves,
// which neighbouring lanes hold, over different banks)
template <int W>
__device__ __forceinline__ void hw_decode(const HwItem<W>& it, float* tile, int row, int half) {
    constexpr int M = W - 1;
    float* dst = tile + (32 * half) * kHwTile + (row ^ (half << 4));
#pragma unroll
    for (int e = 0; e < 32; ++e) {
        const int bit = e * W, wi = bit >> 5, sh = bit & 31;
        uint32_t code = sh == 0 ? it.cw[wi] : (sh + W > 32 ? __funnelshift_r(it.cw[wi], it.cw[wi + 1 < W ? wi + 1 : wi], sh) : it.cw[wi] >> sh);
        code &= (1u << W) - 1u;
        const uint32_t q = code & ((1u << M) - 1u);
        const uint32_t tau = (it.micro >> (e >> 1)) & 1u;
        const float mag = (float)(int)(q << (1u - tau));
        dst[e * kHwTile] = __uint_as_float(__float_as_uint(mag) | ((code >> M) << 31));
    }
}

__device__ __forceinline__ bool hw_has_ff_byte(uint32_t w) { return (((w & 0x7F7F7F7Fu) + 0x01010101u) & w & 0x80808080u) != 0; }

// LONG: a pass spans several steps (r > 64) and its state lives across them.
template <int WA, int WB, bool LONG>
__global__ void __launch_bounds__(kHwThreads, 2)
mx_gemm_hw_kernel(bdr_planes_t a, bdr_planes_t b, int64_t K, int r, int f, float* c, int64_t ldc) {
    __shared__ __align__(16) float As[kHwStep * kHwTile], Bs[kHwStep * kHwTile];
    __shared__ uint32_t Fa[kHwTile], Fb[kHwTile];  // the step's four exponent bytes of every row
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t row0 = (int64_t)blockIdx.y * kHwTile, col0 = (int64_t)blockIdx.x * kHwTile;
    // decode duty: threads 0..127 take A (row = t / 2, half = t % 2), threads 128..255 the same for B
    const int duty = tid & 127, drow = duty >> 1, dhalf = duty & 1;
    const bool dutyA = tid < 128;
    constexpr int W = (WA - 1) + (WB - 1) + 4 + 2;  // m_A + m_B + log2 16 + 2 beta: bits of a block result
    const int bpr = r >> 4, passes = kHwStep / r;                   // blocks per pass, passes per step
    const int fbase = 127 + f - W;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    bool bad_a[4] = {false, false, false, false}, bad_b[4] = {false, false, false, false};
    [[maybe_unused]] int emax_p[LONG ? 4 : 1][4], total_p[LONG ? 4 : 1][4];  // state of a pass that spans several steps
    HwItem<WA> ia;
    HwItem<WB> ib;
    if (dutyA) hw_fetch<WA>(a, row0 + drow, 2 * dhalf, ia);
    else hw_fetch<WB>(b, col0 + drow, 2 * dhalf, ib);
    const int64_t steps = K / kHwStep;
    for (int64_t s = 0; s < steps; ++s) {
        // the step's operands into shared memory
        if (dutyA) {
            hw_decode<WA>(ia, As, drow, dhalf);
            reinterpret_cast<uint16_t*>(Fa)[2 * drow + dhalf] = (uint16_t)ia.exps;
        } else {
            hw_decode<WB>(ib, Bs, drow, dhalf);
            reinterpret_cast<uint16_t*>(Fb)[2 * drow + dhalf] = (uint16_t)ib.exps;
        }
        __syncthreads();
        if (s + 1 < steps) {  // next step's packed bytes travel while this step is computed
            if (dutyA) hw_fetch<WA>(a, row0 + drow, 4 * (s + 1) + 2 * dhalf, ia);
            else hw_fetch<WB>(b, col0 + drow, 4 * (s + 1) + 2 * dhalf, ib);
        }
        uint32_t fa[4], fb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            fa[i] = Fa[4 * ty + i];
            fb[i] = Fb[4 * tx + i];
            bad_a[i] |= hw_has_ff_byte(fa[i]);
            bad_b[i] |= hw_has_ff_byte(fb[i]);
        }
        // one block of 16 elements of K: exact block results D_b, aligned to the pass's largest exponent inside the f-bit frame,
        // truncated toward zero, added as integers
        auto do_block = [&](int bb, const int (&base)[4][4], int (&total)[4][4]) {
            const int swz = (bb >> 1) << 4;  // the half (32 elements) this block belongs to
            const float* ap = As + (16 * bb) * kHwTile + ((4 * ty) ^ swz);
            const float* bp = Bs + (16 * bb) * kHwTile + ((4 * tx) ^ swz);
            unsigned long long D2[4][2];  // (row i; columns 0, 1) and (row i; columns 2, 3)
#pragma unroll
            for (int i = 0; i < 4; ++i) D2[i][0] = D2[i][1] = 0ull;
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) {
                const float4 av = *reinterpret_cast<const float4*>(ap + kk * kHwTile);
                const ulonglong2 bv = *reinterpret_cast<const ulonglong2*>(bp + kk * kHwTile);
                const float ar[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const unsigned long long aa = hw_dup(ar[i]);
                    hw_fma2(D2[i][0], aa, bv.x);
                    hw_fma2(D2[i][1], aa, bv.y);
                }
            }
            int ea[4], eb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                ea[i] = (int)((fa[i] >> (8 * bb)) & 0xFFu);
                eb[i] = (int)((fb[i] >> (8 * bb)) & 0xFFu);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float D[4];
                hw_split(D2[i][0], D[0], D[1]);
                hw_split(D2[i][1], D[2], D[3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int field = base[i][j] + ea[i] + eb[j];  // exponent field of 2^(f - W - (e_max - e))
                    const float scale = __uint_as_float((uint32_t)max(field, 0) << 23);
                    total[i][j] += __float2int_rz(D[j] * scale);
                }
            }
        };
        // end of a pass: the integer sum becomes an fp32 number, takes its power of two, joins the fp32 accumulator
        auto finish_pass = [&](const int (&emax)[4][4], const int (&total)[4][4]) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // the frame's unit: 2^(e_max - 254 - (m_A - 1) - (m_B - 1) - 2 - (f - W))
                    const int unit = emax[i][j] - 254 - (WA - 2) - (WB - 2) - 2 - (f - W);
                    const double v = (double)(float)total[i][j] * __hiloint2double((1023 + unit) << 20, 0);
                    acc[i][j] = __fadd_rn(acc[i][j], (float)v);
                }
        };
        if constexpr (!LONG) {  // whole passes inside the step
            for (int p = 0; p < passes; ++p) {
                const int b0 = p * bpr;
                int emax[4][4], total[4][4], base[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) emax[i][j] = 0;
                for (int bb = b0; bb < b0 + bpr; ++bb) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            emax[i][j] = max(emax[i][j], (int)((fa[i] >> (8 * bb)) & 0xFFu) + (int)((fb[j] >> (8 * bb)) & 0xFFu));
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        total[i][j] = 0;
                        base[i][j] = fbase - emax[i][j];
                    }
                for (int bb = b0; bb < b0 + bpr; ++bb) do_block(bb, base, total);
                finish_pass(emax, total);
            }
        } else {  // a pass spans r / 64 steps: its largest exponent sums come from the exponent planes when it starts
            const int spp = r / kHwStep;
            if (s % spp == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        emax_p[i][j] = 0;
                        total_p[i][j] = 0;
                    }
                for (int wd = 0; wd < spp; ++wd) {  // word wd: the four exponent bytes of step s + wd
                    uint32_t wa[4], wb[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        wa[i] = __ldg(reinterpret_cast<const uint32_t*>(a.exps + (row0 + 4 * ty + i) * a.ld_exps + 4 * (s + wd)));
                        wb[i] = __ldg(reinterpret_cast<const uint32_t*>(b.exps + (col0 + 4 * tx + i) * b.ld_exps + 4 * (s + wd)));
                    }
#pragma unroll
                    for (int bb = 0; bb < 4; ++bb)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                emax_p[i][j] = max(emax_p[i][j], (int)((wa[i] >> (8 * bb)) & 0xFFu) + (int)((wb[j] >> (8 * bb)) & 0xFFu));
                }
            }
            int base[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) base[i][j] = fbase - emax_p[i][j];
            for (int bb = 0; bb < 4; ++bb) do_block(bb, base, total_p);
            if (s % spp == spp - 1) finish_pass(emax_p, total_p);
        }
        __syncthreads();  // everyone is done with the step's tiles
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float4 o;
        const float nanv = __uint_as_float(0x7FC00000u);
        o.x = (bad_a[i] || bad_b[0]) ? nanv : acc[i][0];
        o.y = (bad_a[i] || bad_b[1]) ? nanv : acc[i][1];
        o.z = (bad_a[i] || bad_b[2]) ? nanv : acc[i][2];
        o.w = (bad_a[i] || bad_b[3]) ? nanv : acc[i][3];
        *reinterpret_cast<float4*>(c + (row0 + 4 * ty + i) * ldc + col0 + 4 * tx) = o;
    }
}

template <int WA, int WB>
static int launch_hw(const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, int r, int f, float* c, int64_t ldc,
                     cudaStream_t st) {
    const dim3 grid((unsigned)(N / kHwTile), (unsigned)(M / kHwTile));
    if (r > kHwStep) mx_gemm_hw_kernel<WA, WB, true><<<grid, kHwThreads, 0, st>>>(a, b, K, r, f, c, ldc);
    else mx_gemm_hw_kernel<WA, WB, false><<<grid, kHwThreads, 0, st>>>(a, b, K, r, f, c, ldc);
    return cudaGetLastError() == cudaSuccess ? BDR_OK : BDR_ERR_CUDA;
}

template <int WA>
static int pick_b(int mb, const bdr_planes_t& a, const bdr_planes_t& b, int64_t M, int64_t N, int64_t K, int r, int f, float* c, int64_t ldc,
                  cudaStream_t st) {
    switch (mb) {
        case 2: return launch_hw<WA, 3>(a, b, M, N, K, r, f, c, ldc, st);
        case 4: return launch_hw<WA, 5>(a, b, M, N, K, r, f, c, ldc, st);
        case 7: return launch_hw<WA, 8>(a, b, M, N, K, r, f, c, ldc, st);
    }
    return BDR_ERR_UNSUPPORTED;
}

}  // namespace bdr

using namespace bdr;

extern "C" int mx_gemm_hw(const bdr_config_t* cfg_a, const bdr_planes_t* a, const bdr_config_t* cfg_b, const bdr_planes_t* b, int64_t M,
                          int64_t N, int64_t K, int r, int f, float* c, int64_t ldc, void* stream) {
    if (!cfg_a || !cfg_b || !a || !b || !c) return BDR_ERR_NULL;
    for (const bdr_config_t* cf : {cfg_a, cfg_b}) {
        if (cf->scale_kind != BDR_SCALE_POW2) return BDR_ERR_UNSUPPORTED;
        if (cf->d1 != 8 || cf->k1 < 1 || cf->k2 < 1 || cf->k1 % cf->k2 != 0 || cf->d2 < 0 || cf->d2 > 3 || cf->m < 1 || cf->m > 8)
            return BDR_ERR_BAD_CONFIG;
        if (cf->k1 != 16 || cf->k2 != 2 || cf->d2 != 1 || (cf->m != 2 && cf->m != 4 && cf->m != 7)) return BDR_ERR_UNSUPPORTED;
    }
    if (M < 0 || N < 0 || K < 0 || ldc < N) return BDR_ERR_SIZE;
    if (r != 16 && r != 32 && r != 64 && r != 128 && r != 256 && r != 512 && r != 1024) return BDR_ERR_UNSUPPORTED;
    if (f < 1 || f > 25) return BDR_ERR_SIZE;
    if (M == 0 || N == 0) return BDR_OK;
    if (M % kHwTile || N % kHwTile || K % kHwStep || K % r || K == 0) return BDR_ERR_UNSUPPORTED;
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
        case 2: return pick_b<3>(cfg_b->m, *a, *b, M, N, K, r, f, c, ldc, st);
        case 4: return pick_b<5>(cfg_b->m, *a, *b, M, N, K, r, f, c, ldc, st);
        case 7: return pick_b<8>(cfg_b->m, *a, *b, M, N, K, r, f, c, ldc, st);
    }
    return BDR_ERR_UNSUPPORTED;
}
