/*
 * bdr.h -- C ABI of the B200 (sm_100a) Block Data Representations / shared-microexponent library.
 *
 * Every entry point takes plain pointers and sizes.  Unless a parameter says "host", a pointer is
 * a DEVICE pointer to memory that the caller allocated and keeps alive until the work queued on
 * `stream` has finished.  The library allocates no device memory, never synchronises a stream and
 * leaves every result on the device.  `stream` is a cudaStream_t passed as void* (NULL = the
 * legacy default stream).  Return value: BDR_OK (0) or a negative bdr_status_t; all argument
 * validation happens on the host before anything is launched, so a failing call has queued no work
 * (BDR_ERR_CUDA reports a failed launch).  The first call of an entry point on a device sets kernel
 * attributes and may look up the address of a library-owned status word: make that call outside stream
 * capture; later calls can be captured into CUDA graphs.
 *
 * Layout conventions
 *   A tensor is a row-major 2-D array [rows, cols] with a row pitch of `ld` ELEMENTS (ld >= cols).
 *   `axis` is the quantization (= reduction) direction: axis 1 = along the contiguous dimension
 *   ("row-wise"), axis 0 = along the strided dimension ("column-wise").  A "line" is one row
 *   (axis 1) or one column (axis 0); lines are cut into ceil(len/k1) blocks of k1 consecutive
 *   elements; a short last block behaves as if it were zero padded.  Blocks never span lines.
 *
 * Packed layout (three planes per tensor, line-major: line l starts at plane + l*ld_plane bytes)
 *   exps  : one byte per block, the biased shared exponent F (0xFF marks a block that held Inf/NaN)
 *   micro : little-endian, LSB-first stream of d2-bit fields, field j = shift tau of sub-block j of
 *           the line (empty when d2 = 0)
 *   elems : little-endian, LSB-first stream of (m+1)-bit codes, code i = (sign << m) | magnitude of
 *           element i of the line; positions of the zero padding hold code 0
 *   This spends exactly (m+1) + d1/k1 + d2/k2 bits per element (Section III) whenever a line needs
 *   no padding.  For axis 0 the planes are laid out column by column, i.e. they are byte-identical
 *   to the axis-1 planes of the transposed tensor (the "transpose, then quantize" copy that the
 *   backward pass needs, Section V).
 */
#ifndef BDR_H_
#define BDR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* How the two scale levels are encoded (Section III, Table I). */
typedef enum {
    BDR_SCALE_POW2 = 0,     /* MX / BFP / MSFP: block scale 2^E (d1 = 8 bits), sub-block scale 2^-tau */
    BDR_SCALE_FP32_INT = 1, /* INT: FP32 scale from the maximum (Section II, Eq. 1-2); m = bits - 1   */
    BDR_SCALE_FP32_FP = 2,  /* FP8-like: FP32 scale + per-element d2-bit exponent, m explicit bits    */
    BDR_SCALE_FP32_VSQ = 3  /* VSQ: FP32 scale + unsigned d2-bit integer sub-scale per k2 elements    */
} bdr_scale_kind_t;

typedef enum { BDR_ROUND_NEAREST_EVEN = 0, BDR_ROUND_NEAREST_AWAY = 1 } bdr_rounding_t;
typedef enum { BDR_F32 = 0, BDR_BF16 = 1 } bdr_dtype_t;

/* The BDR parameter tuple of Section III (k1, d1, k2, d2, m) plus scale kind and tie rule.
 * POW2 kind: d1 must be 8, k2 divides k1, 0 <= d2 <= 3, 1 <= m <= 8; the CUDA kernels additionally
 * need k1 and k2 to be powers of two with k1 <= 1024 (else BDR_ERR_UNSUPPORTED).
 * FP32_* kinds are accepted by bdr_qsnr only, with k1 = 0 meaning one scale for the whole tensor. */
typedef struct {
    int32_t k1, d1, k2, d2, m, scale_kind, rounding;
} bdr_config_t;

/* Device pointers to the three packed planes and their line pitches in bytes.  Pitches must be
 * multiples of 16 and plane bases 16-byte aligned.  `micro` may be NULL when d2 = 0. */
typedef struct {
    uint8_t *exps, *micro, *elems;
    int64_t ld_exps, ld_micro, ld_elems;
} bdr_planes_t;

typedef enum {
    BDR_OK = 0,
    BDR_ERR_NULL = -1,        /* a required pointer is NULL                                          */
    BDR_ERR_BAD_CONFIG = -2,  /* parameter tuple outside the definition (k2 does not divide k1, ...)  */
    BDR_ERR_UNSUPPORTED = -3, /* valid, but no kernel for it (non power-of-two k1, FP32 kind in pack) */
    BDR_ERR_MISALIGNED = -4,  /* pointer or pitch breaks a stated alignment rule                      */
    BDR_ERR_SIZE = -5,        /* negative size, ld < cols, size over the stated maximum               */
    BDR_ERR_WORKSPACE = -6,   /* workspace missing or too small                                       */
    BDR_ERR_CUDA = -7,        /* a CUDA call or kernel launch failed                                  */
    BDR_ERR_TIMEOUT = -8      /* a bounded device-side wait ran out (see bdr_device_status, mx_gemm_status) */
} bdr_status_t;

/* Text for a status code (host; never NULL). */
const char* bdr_strerror(int status);

/* Kernels that stage data with asynchronous bulk copies wait for them with a bounded number of
 * polls.  A wait that runs out makes the warp stop early (its part of the output is then
 * incomplete) and leaves BDR_ERR_TIMEOUT in a sticky per-device word.  This host call returns
 * that word for the current device: BDR_OK, BDR_ERR_TIMEOUT, BDR_ERR_SIZE (an index that bdr_gather_rows found
 * outside its table), or BDR_ERR_CUDA if it cannot be read.  It synchronises with the device (one word is
 * copied back), so call it after the work of interest, not between launches.  bdr_device_status_reset
 * returns the word in the same way and clears it (the first failure sticks until then). */
int bdr_device_status(void);
int bdr_device_status_reset(void);

/* Self-tests of the library's failure handling.  (The paper has no counterpart.)
 * bdr_selftest_bounded_wait queues a one-warp kernel that waits, with the same bounded wait the streaming
 * kernels use (cut down to a few hundred polls, well under a millisecond), on a barrier that nothing
 * completes.  The wait runs out by design; the kernel then reports BDR_ERR_TIMEOUT into `status_dev` (one
 * int of device memory that the caller zeroed: NOT the library's own sticky word, which stays clean) and
 * ends normally, so the context stays usable.  It shows that a wait that gives up is reported and does not
 * hang the GPU.  bdr_selftest_host checks, without any CUDA call, the per-device bookkeeping that decides when
 * a kernel's launch attributes are set (once per device, not once per process); BDR_OK when it holds. */
int bdr_selftest_bounded_wait(int* status_dev, void* stream);
int bdr_selftest_host(void);

/* Section III bits-per-element formula realised as plane sizes (host only).  ld_out / bytes_out
 * (host arrays of 3: exps, micro, elems) receive the default line pitches (rounded up to 16 bytes)
 * and total plane sizes for a [rows, cols] tensor quantized along `axis`. */
int bdr_packed_sizes(const bdr_config_t* cfg /*host*/, int64_t rows, int64_t cols, int axis,
                     int64_t ld_out[3] /*host*/, int64_t bytes_out[3] /*host*/);

/* Q(x): quantize to the format and write the dequantized values back in the input's dtype and
 * layout (Appendix: shared exponent = private exponent of the block's largest element; sub-block
 * shift tau <= 2^d2-1; m-digit magnitude rounded to nearest, clamped at 2^m-1).
 *   x, y          [rows, ld] of `dt`; y may alias x; y may be NULL when only the sums are wanted
 *   qsnr_sums_dev NULL, or 2 doubles that this call ADDS {sum (Q(x)-x)^2, sum x^2} to (Eq. 3);
 *                 the caller zeroes them
 * POW2 kind only.  Every shape, pitch and alignment is accepted; which kernel runs only changes the speed,
 * never the result.  Fastest: bf16 tensors in the Table II family (k1 = 16, k2 = 2, d2 = 1, m <= 7,
 * ties-to-even) with 32-byte aligned rows of whole 2048-element runs (axis 1; a contiguous tensor counts
 * as one long row) or whole tiles of 256 rows x 128 columns (axis 0); along axis 1 the same kernel also
 * takes k1 = 32 .. 1024 (powers of two) and formats without shifts (d2 = 0); next, fp32 or bf16 with 16-byte
 * aligned rows of whole 16-element slices (axis 1), and along axis 0 every configuration with k2 <= 16 (bf16: an
 * even number of columns and an even pitch); anything else takes a slower general kernel. */
int bdr_quant_dequant(const bdr_config_t* cfg /*host*/, const void* x, void* y, bdr_dtype_t dt,
                      int64_t rows, int64_t cols, int64_t ld, int axis, double* qsnr_sums_dev,
                      void* stream);

/* Three-level scaling, the extension sketched at the end of Section III: a software FP32 parent scale over groups of
 * k_parent consecutive elements of a line (the paper: "an even coarser granularity at up to ~1K") above the power-of-two
 * block scale and the microexponents.  This library's reading: the parent scale maps the group's largest magnitude onto
 * the largest value a block with exponent 0 can hold, V = (2^m - 1) 2^-(m-1):  s = amax_g / V,  x' = x / s,
 * y = Q(x') s with Q the two-level quantizer of bdr_quant_dequant (IEEE fp32 division and multiplication).  Arguments
 * as bdr_quant_dequant.  fp32 tensors, k1 <= 16, k_parent a multiple of 16 (and of k1) up to 1024.  Fastest (about half
 * the copy bandwidth): k1 = 16, k_parent a power of two, whole groups along contiguous 16-byte aligned rows (axis 1);
 * other shapes take one warp per group with element-wise loads. */
int bdr_quant_dequant_parent(const bdr_config_t* cfg /*host*/, int k_parent, const void* x, void* y, bdr_dtype_t dt,
                             int64_t rows, int64_t cols, int64_t ld, int axis, double* qsnr_sums_dev, void* stream);

/* Quantize and write the packed planes (layout above); optionally also the dequantized tensor
 * (y_dq, same dtype/pitch as x, may be NULL) and the Eq. 3 sums.  Every byte of every plane line
 * up to its pitch is written (padding bytes are zero). */
int bdr_pack(const bdr_config_t* cfg /*host*/, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols,
             int64_t ld, int axis, const bdr_planes_t* out /*host struct of device pointers*/, void* y_dq,
             double* qsnr_sums_dev, void* stream);

/* bdr_pack along both directions at once: out_rows receives exactly what bdr_pack(axis = 1) writes and out_cols
 * exactly what bdr_pack(axis = 0) writes (the planes of the transposed tensor), from ONE read of x.  Section V,
 * Fig. 8: every tensor of a training step is an operand of one matrix product in the forward pass and of one in
 * the backward pass, reduced over different dimensions, so it is quantized along both ("transpose, then quantize"
 * for the second copy).  The optional sums are those of bdr_pack for the two directions (each 2 doubles, added to;
 * pass both or neither for the single-read kernel).
 * Single-read kernel: bf16, Table II formats (k1 = 16, k2 = 2, d2 = 1, m in {2, 4, 7}), ties-to-even, rows a
 * multiple of 256, cols a multiple of 256, 16-byte aligned rows, planes with their natural pitches; its algorithmic
 * traffic is 2 + 2 bits/8 bytes per element against 2 (2 + bits/8) for two calls.  Anything else is served by one
 * pass per direction, with the same bytes as result. */
int bdr_pack2(const bdr_config_t* cfg /*host*/, const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
              const bdr_planes_t* out_rows /*host struct*/, const bdr_planes_t* out_cols /*host struct*/,
              double* qsnr_sums_rows_dev, double* qsnr_sums_cols_dev, void* stream);

/* Decode packed planes to values (-1)^s * q * 2^(F-127-tau-(m-1)) of dtype `dt` in a [rows, ld]
 * tensor; the inverse of bdr_pack's planes -> Q(x). */
int bdr_unpack(const bdr_config_t* cfg /*host*/, const bdr_planes_t* in /*host struct*/, void* y, bdr_dtype_t dt,
               int64_t rows, int64_t cols, int64_t ld, int axis, void* stream);

/* Rows of a packed table, decoded: y[i, :] = the dequantized row idx_dev[i] of a [n_rows, dim] table stored as axis-1
 * planes (what bdr_pack(axis = 1) wrote), for i < n_idx.  Section V (inferencing): in memory-bound models such as
 * recommendation models the embedding tables are kept in MX format as well, so a lookup reads (m+1) + 1 bits per
 * element instead of 16 or 32.  idx_dev: n_idx int64 indices on the device; y [n_idx, ld] of `dt`.  Any POW2
 * configuration.  An index outside [0, n_rows) cannot be seen by the host: its output row is filled with quiet
 * NaNs and BDR_ERR_SIZE is left in the sticky word that bdr_device_status returns. */
int bdr_gather_rows(const bdr_config_t* cfg /*host*/, const bdr_planes_t* table /*host struct*/, int64_t n_rows, int64_t dim,
                    const int64_t* idx_dev, int64_t n_idx, void* y, bdr_dtype_t dt, int64_t ld, void* stream);

/* Eq. 3 from accumulated sums: qsnr_db_dev[i] = -10 log10(sums_dev[2i] / sums_dev[2i+1]) for n pairs
 * {sum (Q(x)-x)^2, sum x^2} as bdr_quant_dequant / bdr_pack accumulate them (device pointers, 8-byte aligned;
 * a zero error sum over a non-zero signal gives +inf, a zero signal NaN).  The sums stay usable: they are
 * only read. */
int bdr_qsnr_from_sums(const double* sums_dev, int n, double* qsnr_db_dev, void* stream);

/* Bytes of device scratch that bdr_qsnr needs for n_cfgs configurations (host only). */
int64_t bdr_qsnr_workspace_bytes(int n_cfgs);

/* The design-space sweep of Section IV: QSNR (Eq. 3, in dB, ratio of whole-tensor sums) of one
 * tensor under n_cfgs configurations, reading the tensor once per group of configurations.
 *   cfgs         host array.  POW2 entries as above, with k2 <= 16 whenever d2 > 0 (BDR_ERR_UNSUPPORTED beyond).
 *                FP32_INT (1 <= m <= 15), FP32_FP (a scalar float with d2 = 2..5 exponent bits and m = 1..7
 *                explicit mantissa bits, bias 2^(d2-1)-1, gradual underflow, top exponent reserved except
 *                for d2 = 4, m = 3, which is E4M3 with maximum 448; E5M2 is d2 = 5, m = 2) and FP32_VSQ
 *                (k2 = 16, 1 <= d2 <= 16, 1 <= m <= 15) entries need k1 = 0: one FP32 scale for the whole
 *                tensor, from the current amax
 *   qsnr_db_dev  n_cfgs doubles, written (not accumulated)
 *   workspace    device scratch of at least bdr_qsnr_workspace_bytes(n_cfgs) bytes, 16-byte aligned;
 *                contents are overwritten
 * 1 <= n_cfgs <= 4096.  axis 1: rows are the lines; axis 0: columns are the lines (blocks and VSQ vectors
 * run down a column; the loads are strided, so this direction reads slower, which matters little to a
 * kernel that is bound by arithmetic). */
int bdr_qsnr(const bdr_config_t* cfgs /*host*/, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows,
             int64_t cols, int64_t ld, int axis, double* qsnr_db_dev, void* workspace, int64_t workspace_bytes,
             void* stream);

/* The sweep with a first-level maximum that comes from elsewhere (Section IV-B, Fig. 7 caption: the INT, FP and VSQ
 * points take their FP32 first-level scale from the absolute maximum over a window of PAST vectors, "delayed
 * scaling").  amax_window_dev holds n_window >= 1 non-negative floats on the device (the maxima of earlier tensors,
 * e.g. written by bdr_amax); the FP32_* entries derive their scale from the largest of them instead of from x, and
 * values of x beyond it saturate at the top code.  POW2 entries are unaffected.  Everything else as bdr_qsnr. */
int bdr_qsnr_delayed(const bdr_config_t* cfgs /*host*/, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows,
                     int64_t cols, int64_t ld, int axis, const float* amax_window_dev, int n_window,
                     double* qsnr_db_dev, void* workspace, int64_t workspace_bytes, void* stream);

/* Eq. 1's maximum: *amax_dev = max(*amax_dev, max |x|) over a [rows, ld] tensor (one float on the device; the
 * caller zeroes it, or leaves an earlier maximum in it to extend a window). */
int bdr_amax(const void* x, bdr_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* amax_dev, void* stream);

/* Section IV-B, memory footprint (host only): the fraction of the fetched bits that are payload when a tile of
 * tile_elems elements ((m+1) + d1/k1 + d2/k2 bits each, Section III) is stored in whole memory lines of line_bytes
 * bytes; the paper's setting is a 256-element tile and a 64-byte interface.  Negative for a bad argument. */
double bdr_tile_packing_efficiency(const bdr_config_t* cfg /*host*/, int64_t tile_elems, int64_t line_bytes);

/* The same sweep as bdr_qsnr for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart; this is a convenience of this library.)  Think of a monitoring hook that runs inside
 * another framework's training step, or a serving loop with a fixed memory plan: all device memory
 * already belongs to that framework's pool, a cudaMalloc could fail, and it would stall the GPU
 * because allocation and free synchronise the device.  This entry point therefore allocates nothing:
 * its scratch is an array built into the library (about 20 KB that every GPU loading the library
 * holds until the process ends).
 *   - at most bdr_qsnr_static_max_cfgs() (= 512) configurations per call; more is BDR_ERR_SIZE
 *   - inputs, outputs, validation and results are exactly those of bdr_qsnr
 *   - the first call on each device looks up the array's device address (a host-side query, no
 *     allocation); make that first call outside any stream capture
 *   - all calls on a device share the one array: it is cleared at the start of every call, and two
 *     calls whose GPU work overlaps (different streams, or threads) race on it -- serialise them */
int bdr_qsnr_static_max_cfgs(void);
int bdr_qsnr_static(const bdr_config_t* cfgs /*host*/, int n_cfgs, const void* x, bdr_dtype_t dt, int64_t rows,
                    int64_t cols, int64_t ld, int axis, double* qsnr_db_dev, void* stream);

/* C[M,N] (fp32, row pitch ldc elements) = deq(A)[M,K] * deq(B)[N,K]^T with both operands given as
 * packed planes quantized along K (axis 1 planes of A and of B), decoded to bf16 inside the kernel
 * and accumulated in fp32 on the tensor cores (Section V: both inputs of a tensor operation are
 * MX-quantized along the reduction dimension).  The result equals the fp32-accumulated product of
 * the dequantized operands; only the summation order is unspecified.
 * Needs the Table II formats (k1 = 16, k2 = 2, d2 = 1, m in {2, 4, 7}; A and B may differ), M a
 * multiple of 128, N a multiple of 256, K a multiple of 64, c 16-byte aligned and ldc a multiple
 * of 4; anything else is BDR_ERR_UNSUPPORTED.  Blocks whose shared exponent lies below 2^-120
 * decode to zero (bf16 has no finer values).  A device-side wait that runs out is reported by
 * mx_gemm_status(), not by this call. */
int mx_gemm(const bdr_config_t* cfg_a /*host*/, const bdr_planes_t* a /*host struct*/,
            const bdr_config_t* cfg_b /*host*/, const bdr_planes_t* b /*host struct*/, int64_t M, int64_t N,
            int64_t K, float* c, int64_t ldc, void* stream);

/* Lends the library scratch memory on the current device (or takes it back: workspace = NULL).  While it is
 * lent, mx_gemm uses it to compute the same product through the faster two-phase kernels (mx_gemm_f8 when
 * both formats have m <= 4, else mx_gemm_ws) whenever M, N and K are multiples of 256 and the memory is large
 * enough (mx_gemm_f8_workspace_bytes / mx_gemm_workspace_bytes); otherwise mx_gemm works without scratch as
 * before.  The memory stays the caller's: 256-byte aligned device memory that must outlive every mx_gemm call
 * issued while it is lent; its contents are overwritten by those calls, which therefore have to be ordered
 * with respect to each other (one stream, or events).  Host call, no device work. */
int bdr_set_workspace(void* workspace, int64_t workspace_bytes);

/* mx_gemm in two phases, for callers that can lend scratch memory: both operands are first decoded to
 * bf16 in `workspace` (once each, by the unpack kernels), then multiplied by a tensor-core kernel that
 * streams the bf16 operands with TMA.  mx_gemm decodes inside the GEMM and so repeats the decode of an
 * operand row for every tile of the other dimension; for large M and N this entry point is the faster
 * one.  Same result as mx_gemm (only the summation order is unspecified), same format rules.
 * Needs M and N multiples of 256, K a multiple of 64, and a 256-byte aligned workspace of at least
 * mx_gemm_workspace_bytes(M, N, K) = 2 (M + N) K bytes (rounded up to 256), whose contents are
 * overwritten; BDR_ERR_WORKSPACE if it is missing or too small.  Values below bf16's subnormal range
 * (|v| < 2^-133) are truncated toward zero. */
int64_t mx_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
int mx_gemm_ws(const bdr_config_t* cfg_a /*host*/, const bdr_planes_t* a /*host struct*/,
               const bdr_config_t* cfg_b /*host*/, const bdr_planes_t* b /*host struct*/, int64_t M, int64_t N,
               int64_t K, float* c, int64_t ldc, void* workspace, int64_t workspace_bytes, void* stream);

/* mx_gemm for MX4 / MX6 operands (k1 = 16, k2 = 2, d2 = 1, m in {2, 4}; A and B may differ) on the 8-bit
 * block-scaled tensor-core path, which runs at twice the bf16 rate.  (The paper has no counterpart: it maps
 * the format onto the scaled 8-bit matrix instruction of the target GPU.  A decoded element
 * q * 2^(E - tau - m + 1), Section III, has at most four significant bits, so it is an exact E4M3 number
 * once the exponent of the larger of two neighbouring 16-element blocks is taken out as the 32-element
 * scale.)  Phase 1 re-encodes both operands into `workspace`, phase 2 multiplies them; every product is
 * exact and accumulation is fp32, so the result agrees with mx_gemm up to summation order.  Operands
 * that cannot be represented (neighbouring block exponents more than about 12 apart with non-zero
 * elements in the smaller block, block exponents below 16, Inf/NaN blocks) are detected on the device
 * in phase 1; the call then computes C with mx_gemm's kernel instead, without host involvement.
 * Needs M, N and K multiples of 256 and a 256-byte aligned workspace of at least
 * mx_gemm_f8_workspace_bytes(M, N, K) bytes (about (M + N) K * 33 / 32), whose contents are overwritten. */
int64_t mx_gemm_f8_workspace_bytes(int64_t M, int64_t N, int64_t K);
int mx_gemm_f8(const bdr_config_t* cfg_a /*host*/, const bdr_planes_t* a /*host struct*/,
               const bdr_config_t* cfg_b /*host*/, const bdr_planes_t* b /*host struct*/, int64_t M, int64_t N,
               int64_t K, float* c, int64_t ldc, void* workspace, int64_t workspace_bytes, void* stream);

/* Phase 1 of mx_gemm_f8 on its own: packed planes of an MX4 / MX6 operand [rows, K] (axis-1 planes) ->
 *   out      rows * K bytes (device), row-major E4M3 elements
 *   scales   rows * K / 32 bytes (device): for every 128 rows x 128 K a 512-byte atom holding the scale
 *            exponent (value 2^(byte - 127)) of row r, K group g (32 elements) at (r % 32) * 16 + (r / 32) * 4 + g;
 *            atoms ordered [K / 128][rows / 128]
 *   inexact_dev  one int (device): set to 1 if some element is not representable, if a block with an
 *            exponent field below 16 holds a non-zero element, or if a block has the exponent field 255
 *            (the bytes of `out` are then unspecified); never cleared by this call
 * so that element = E4M3(out) * 2^(scale - 127) exactly.  rows and K multiples of 128; 16-byte aligned
 * pointers. */
int bdr_reencode_e4m3(const bdr_config_t* cfg /*host*/, const bdr_planes_t* in /*host struct*/, int64_t rows, int64_t K,
                      uint8_t* out, uint8_t* scales, int* inexact_dev, void* stream);

/* Phase 2 of mx_gemm_f8 on its own, for operands that were re-encoded earlier (weights that do not change
 * between calls, say): C = A B^T from E4M3 bytes a [M, K], b [N, K] (row-major, contiguous) and their scale
 * atoms as bdr_reencode_e4m3 writes them.  The caller has checked that no re-encoding raised `inexact`.
 * M, N, K multiples of 256; 16-byte aligned pointers; device memory; fp32 accumulate and output. */
int mx_gemm_e4m3(const uint8_t* a, const uint8_t* scales_a, const uint8_t* b, const uint8_t* scales_b, int64_t M,
                 int64_t N, int64_t K, float* c, int64_t ldc, void* stream);

/* C = A B^T as the dot-product pipeline of Section IV-B (Fig. 6) computes it, bit for bit, from the same packed
 * operands as mx_gemm.  The paper describes the pipeline in words; this library's reading: inside a 16-element block
 * the integer mantissa products are summed exactly, the two products of sub-block j entering with the weight
 * 2^(2 - tau_A,j - tau_B,j) (the conditional right shifts by the microexponents); the r/16 block results of one pass
 * (r consecutive elements of K) are aligned to the largest exponent sum F_A + F_B of the pass inside a frame of f
 * magnitude bits whose top bit is the top bit of a block result at that exponent, truncated toward zero, and added
 * as integers; the pass's sum is rounded to fp32 (nearest even) and passes are accumulated in fp32 in order of
 * increasing K.  The paper chooses f = min(25, the format's dynamic range), which is 25 for every format with an
 * 8-bit shared exponent.  With a frame wide enough for the exponent spread of a pass the result is the exact dot
 * product of the dequantized operands rounded once per pass; narrower frames drop low bits of the smaller blocks.
 * Table II formats (A and B may differ), r a power of two from 16 to 1024 that divides K, 1 <= f <= 25, M and N multiples
 * of 64, K a multiple of 64, c 16-byte aligned with ldc a multiple of 4.  A block with the exponent byte 0xFF makes its row's (column's)
 * outputs NaN.  Runs on the ordinary arithmetic units (the alignment is per block and output), not the tensor cores. */
int mx_gemm_hw(const bdr_config_t* cfg_a /*host*/, const bdr_planes_t* a /*host struct*/,
               const bdr_config_t* cfg_b /*host*/, const bdr_planes_t* b /*host struct*/, int64_t M, int64_t N,
               int64_t K, int r, int f, float* c, int64_t ldc, void* stream);

/* BDR_OK, or BDR_ERR_TIMEOUT if any mx_gemm launch on the current device gave up a bounded wait
 * (sticky).  Host call; synchronises with the device (it copies one word back). */
int mx_gemm_status(void);

#ifdef __cplusplus
}
#endif
#endif /* BDR_H_ */
