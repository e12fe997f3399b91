/*
 * mxp.h -- C ABI of libmxp: MXFP4 / MXFP4+ ("MX+") block quantization, decode and
 * GEMM on NVIDIA B200 (sm_100a).
 *
 * Format (paper Sec. 2 Eq. 1, Sec. 4.1, Sec. 4.2):
 *   - a block is 32 consecutive elements of a row; every block has one E8M0 scale byte
 *     (biased by 127) holding shared_exp = floor(log2 BM) - 2, BM = the block's absolute
 *     maximum (first one if several are equal);
 *   - elements are 4-bit E2M1 codes (sign, 2 exponent bits with bias 1, 1 mantissa bit),
 *     element 2j in the low nibble of byte j, rounded to nearest with ties to the even
 *     code and saturating at 6;
 *   - in MXFP4+ mode the BM element stores 3 mantissa bits instead (E0M3, value
 *     4 + m/2 on the scaled grid, exponent implied) and a per-block index byte holds its
 *     position in bits 4:0 (bits 7:5 are written 0 and ignored on read);
 *   - in MX++ mode (Sec. 4.3) the scale byte and the BM are those of MXFP4+, and the
 *     other elements (NBMs) use shared_exp_new = CLIP(max2 - 2 + 1, {shared_exp - 7,
 *     shared_exp}), max2 = the largest floor(log2|x|) among the non-zero NBMs (lower clip
 *     if there are none); delta = shared_exp - shared_exp_new sits in bits 7:5 of the
 *     index byte; an NBM decodes to 2^(shared_exp - delta) times its E2M1 value;
 *   - a block whose BM has floor(log2 BM) <= -125 is flushed: scale byte 0, all-zero
 *     nibbles, index 0; scale byte 0 decodes to 32 zeros in both modes;
 *   - a block holding Inf/NaN gets scale byte 0xFF and zero data (not defined by the
 *     paper; decodes to NaN).
 *
 * Conventions for every entry point:
 *   - every data pointer is caller-owned DEVICE memory unless stated otherwise; the
 *     library never allocates, frees or keeps it;
 *   - matrices are row-major; blocks run along the contiguous dimension (cols = K), so
 *     the GEMM's B operand is passed as N x K ("weights as [out, in]");
 *   - `cuda_stream` is a cudaStream_t (NULL = the legacy default stream); work is
 *     enqueued on it and the call returns without synchronising;
 *   - errors are return codes; nothing is launched when a call returns
 *     MXP_ERR_INVALID_ARG / MXP_ERR_UNSUPPORTED / MXP_ERR_WORKSPACE.
 */
#ifndef MXP_H_
#define MXP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MXP_OK = 0,
    MXP_ERR_INVALID_ARG = 1, /* null / misaligned pointer, bad size, bad enum */
    MXP_ERR_UNSUPPORTED = 2, /* valid request this build has no kernel for */
    MXP_ERR_WORKSPACE = 3,   /* workspace missing or too small */
    MXP_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
    MXP_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (see mxp_gemm_status) */
} mxp_status;

typedef enum {
    MXP_MODE_MXFP4 = 0,
    MXP_MODE_MXFP4_PLUS = 1, /* MX+  (Sec. 4.1): BM with 3 mantissa bits, index byte */
    MXP_MODE_MXFP4_PP = 2,   /* MX++ (Sec. 4.3): MX+ and a finer shared exponent for the NBMs */
    /* The same scheme at the other element widths (Table of MX formats, Sec. 4.1-4.2):
     * mxp_quantize and mxp_dequantize, and operands of the packed x packed mxp_gemm with its
     * full workspace (MXFP8 codes are read as stored; an MXFP6+ operand costs one more pass
     * over K, its BM being entered as the sum of two E2M3 values, an MXFP8+ operand two more,
     * its BM being the sum of three E4M3 values); as weights of the weight-only mxp_gemm (bf16
     * activations) with the workspace mxp_gemm_workspace_bytes(..., a_dense = 1, ...) gives, at
     * any M, K % 128 == 0; also of mxp_gemm_prepack / mxp_gemm_prepacked;
     * the other GEMM forms (decode kernels, chained and re-tiled forms) reject them. */
    MXP_MODE_MXFP6 = 3,      /* E2M3 elements, emax 2 */
    MXP_MODE_MXFP6_PLUS = 4, /* ... with the BM as sign + 5 mantissa bits: 4 + m/8, index byte */
    MXP_MODE_MXFP8 = 5,      /* E4M3 elements, emax 8 */
    MXP_MODE_MXFP8_PLUS = 6  /* ... with the BM as sign + 7 mantissa bits: 256 + 2 m, index byte */
} mxp_mode;
typedef enum { MXP_F32 = 0, MXP_BF16 = 1 } mxp_dtype;

/* A packed operand: three row-major device planes.  MXFP6 modes: `nibbles` holds rows * cols
 * 6-bit codes, code i of a row in bits 6i..6i+5 of the little-endian bit stream (3/4 byte per
 * element); MXFP8 modes: one byte per element. */
typedef struct {
    const uint8_t *nibbles;  /* rows * cols / 2 bytes, 16-byte aligned                */
    const uint8_t *scales;   /* rows * cols / 32 bytes, E8M0                          */
    const uint8_t *bm_index; /* rows * cols / 32 bytes; may be NULL iff mode == MXFP4 */
    int64_t rows, cols;      /* cols % 32 == 0                                        */
    mxp_mode mode;
} mxp_packed;

/*
 * Quantize (Eq. 1 shared scale; Sec. 4.1 BM re-encoding and flush rule; Sec. 4.2 layout).
 *   src      rows x cols elements of `src_dt`, row stride `ld_src` elements
 *            (ld_src >= cols, ld_src % 8 == 0, 16-byte aligned base)
 *   nibbles  out, rows * cols / 2 bytes (16-byte aligned)
 *   scales   out, rows * cols / 32 bytes
 *   bm_index out, rows * cols / 32 bytes; required for MXFP4+, may be NULL for MXFP4
 *            (when given in MXFP4 mode it is filled with zeros)
 * cols must be a multiple of 32.  rows == 0 or cols == 0 is a no-op returning MXP_OK.
 * MXFP6 / MXFP8 modes: the same with emax 2 / 8 in Eq. 1 and the flush rule, E2M3 / E4M3
 * element casts (round to nearest even, saturating at 7.5 / 448) and `nibbles` sized
 * rows * cols * 3 / 4 resp. rows * cols bytes; in the + modes the BM is stored as its sign and
 * 5 resp. 7 mantissa bits (scaled value 4 + m/8 resp. 256 + 2 m).
 */
mxp_status mxp_quantize(const void *src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                        int64_t ld_src, mxp_mode mode, uint8_t *nibbles, uint8_t *scales,
                        uint8_t *bm_index, void *cuda_stream);

/*
 * mxp_quantize with channel reordering fused in (Sec. 8, "Scattering outliers with channel
 * reordering": outlier channels are spread over the blocks so that more of them become a
 * block's BM; the reordering costs nothing extra because it happens where the quantizer
 * touches the data anyway).  Position c of every quantized row holds source channel
 * order[c]:  out = quantize(src[:, order]).  Both operands of a GEMM must use the same
 * ordering along K for the product to be unchanged.
 *   order   device, `cols` entries of int32, 16-byte aligned, read for every row.  Meant to
 *           be a permutation of 0..cols-1; the library does not check that: entries are
 *           clamped to cols-1 and applied as a gather.
 *   src     as for mxp_quantize, but only element-aligned (rows are read channel by channel)
 *   modes   MXFP4, MXFP4+, MXFP4++; the 6- and 8-bit modes return MXP_ERR_UNSUPPORTED.
 * Everything else (planes, sizes, errors) as mxp_quantize.
 *
 * mxp_channel_order builds such an ordering on the HOST from per-channel outlier counts, by
 * the rule of the same passage: channels sorted by count, most first (equal counts keep
 * channel order); the cols/32 highest go one to each block, at its first position, in that
 * order; the remaining channels fill the other positions front to back, first the half with
 * the fewer outliers and then the half with the more, each half from its highest count down
 * (an odd remainder gives the extra channel to the first-placed half).  How outliers are
 * counted (threshold, calibration samples) is the caller's business.
 *   outlier_count, order   host arrays of `cols` entries; cols % 32 == 0.
 */
mxp_status mxp_quantize_reordered(const void *src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                                  int64_t ld_src, const int32_t *order, mxp_mode mode,
                                  uint8_t *nibbles, uint8_t *scales, uint8_t *bm_index,
                                  void *cuda_stream);
mxp_status mxp_channel_order(const int64_t *outlier_count, int64_t cols, int32_t *order);

/*
 * NVFP4 and NVFP4+ (Sec. 8, "Applicability of MX+ to NVFP4").  NVFP4: E2M1 elements in blocks
 * of 16 along the row, one E4M3 scale byte per block, one fp32 scale for the tensor.  NVFP4+
 * gives the block's largest-magnitude element (BM) three mantissa bits in place of its
 * exponent and mantissa bits (value 4 + m/2 times the block's scale, as in MXFP4+) and stores
 * a 4-bit BM index per block; blocks whose scale byte is 00000010b or less keep the plain
 * NVFP4 form and index 0.
 *
 *   tensor_scale  the per-tensor fp32 scale, chosen by the caller, 2^-100 <= ts <= 2^100,
 *                 MXP_ERR_INVALID_ARG otherwise (the usual
 *                 choice: largest magnitude of the tensor / (6 * 448), so that block scales
 *                 use the E4M3 range; a larger value pushes more blocks into the fallback)
 *   plus          0: NVFP4, != 0: NVFP4+
 *   nibbles       rows*cols/2 bytes, element 2j of a row in the low nibble of byte j
 *   scales        rows*cols/16 bytes, E4M3 (sign bit 0), row-major; 2-byte aligned
 *   bm_index      rows*cols/32 bytes: two 4-bit indices per byte, the even block of a row in
 *                 the low nibble; NULL allowed iff plus == 0 (then not written / not read)
 *   cols % 32 == 0; src / dst rows 16-byte aligned (ld % 8 == 0), nibbles 16-byte aligned.
 *
 * What is computed is the definition in real numbers, not a floating-point recipe (the codes
 * are those of exact arithmetic; the CPU oracle of the test suite states the same in binary64):
 *   q = amax / (6 * tensor_scale);  scale byte = the E4M3 value nearest to q, ties to the even
 *   byte, saturating at 448;  d = value(scale byte) * tensor_scale;  element codes = the E2M1
 *   value nearest to |x| / d, ties to the even code, saturating at 6, sign of x kept;  scale
 *   byte 0: all codes 0;  BM (first of equal maxima), NVFP4+ only: m = the integer nearest to
 *   (clamp(amax / d, 4, 8) - 4) * 2, ties to even, at most 7.  Decode: x = +-E * d, E the E2M1
 *   value or 4 + m/2, rounded once (nearest even) to the destination type, fp32 or bf16.
 * Inf / NaN inputs are outside the contract.
 */
mxp_status mxp_nvfp4_quantize(const void *src, mxp_dtype src_dt, int64_t rows, int64_t cols,
                              int64_t ld_src, float tensor_scale, int plus, uint8_t *nibbles,
                              uint8_t *scales, uint8_t *bm_index, void *cuda_stream);
mxp_status mxp_nvfp4_dequantize(const uint8_t *nibbles, const uint8_t *scales,
                                const uint8_t *bm_index, int64_t rows, int64_t cols,
                                float tensor_scale, int plus, void *dst, mxp_dtype dst_dt,
                                int64_t ld_dst, void *cuda_stream);

/*
 * Decode (Eq. 3): dst[r][c] = (-1)^s * 2^(scale - 127) * E, E = 4 + m/2 for the BM
 * element of an MXFP4+ block, the E2M1 value otherwise.  Exact in both output types.
 *   p       host pointer to the operand descriptor (its planes are device memory)
 *   dst     rows x cols of `dst_dt`, row stride `ld_dst` elements (ld_dst % 8 == 0,
 *           16-byte aligned base)
 */
mxp_status mxp_dequantize(const mxp_packed *p, void *dst, mxp_dtype dst_dt, int64_t ld_dst,
                          void *cuda_stream);

/*
 * GEMM on MX / MX+ operands (problem statement of Sec. 5; Eq. 3 for the weight-only
 * form; Eq. 4 / Algorithm 1 for the direct form):
 *     D[M,N] = dec(A)[M,K] * dec(B)[N,K]^T, fp32 accumulation.
 * Exactly one of A_dense_bf16 / A_packed is non-NULL:
 *   - A_dense_bf16 (device, bf16, row stride lda elements): weight-only form, the
 *     weights B are decoded inside the kernel and multiplied with bf16 activations
 *     (up to 64 rows: streamed decode kernels, no workspace needed -- they bring each chunk of
 *     256 activations into half-precision range by a power of two, so an activation more than
 *     2^28 below the largest of its chunk is rounded at 2^-39 of that largest one; more rows, given
 *     mxp_gemm_workspace_bytes(..., a_dense = 1, ...) bytes of workspace: the tensor-core
 *     kernel, the activations entering as the exact sum of two E4M3 planes with a
 *     power-of-two scale per block of 32 -- elements more than 2^9 below their block's
 *     maximum are rounded at 2^-17 of that maximum; with less workspace a slower
 *     general kernel answers; MXFP6(+) / MXFP8(+) weights take the tensor-core kernel at every
 *     M and return MXP_ERR_WORKSPACE without its workspace);
 *   - A_packed (host pointer to a descriptor): both operands are consumed by the
 *     block-scaled tensor-core path; any combination of MXFP4 / MXFP4+ modes.  With the full
 *     workspace: MXFP4 x MXFP4 runs FP4 instructions on the stored planes; one MXFP4+ operand
 *     against an MXFP4 one runs the same main pass with every BM replaced by its upper part
 *     BM_H plus Eq. 4's residual (BM_L) as a sparse tensor-core instruction (Sec. 5.2,
 *     Algorithm 1: "sparse MMA"), 1.5 times the plain MXFP4 tensor work; two MXFP4+ operands
 *     run one pass on 6-bit codes that hold the decoded values of Eq. 3 exactly, 2 times.
 *   B_packed   host pointer to the descriptor of the N x K weight operand
 *   D          M x N of `d_dt` (bf16 rounded to nearest even, or fp32), row stride ldd
 *              elements (ldd >= N; 16-byte aligned rows let the epilogue use wide stores)
 *   workspace  device scratch, 256-byte aligned, of at least
 *              mxp_gemm_min_workspace_bytes(...) bytes (MXP_ERR_WORKSPACE otherwise); may be
 *              NULL when that size is 0.  With mxp_gemm_workspace_bytes(...) bytes the
 *              tensor-core form first re-tiles the scales and, for MX+ operands, widens the
 *              4-bit codes to 6-bit E2M3 codes (E4M3 bytes for MX++; either is exact for every
 *              E2M1 value and for the BM values of Eq. 3) inside the workspace and then runs
 *              its fastest kernel; with less
 *              it runs kernels that work on the packed planes in place (Eq. 4 / Algorithm 1:
 *              BM split and residual MMAs), which are slower.  Same result either way.
 *              Its first 16 bytes are a status block written by the kernels (see
 *              mxp_gemm_status).  The workspace holds nothing the caller has to keep
 *              between calls.
 * K % 32 == 0 always; the tensor-core form further needs K % 128 == 0.
 */
mxp_status mxp_gemm(int64_t M, int64_t N, int64_t K, const void *A_dense_bf16, int64_t lda,
                    const mxp_packed *A_packed, const mxp_packed *B_packed, void *D,
                    mxp_dtype d_dt, int64_t ldd, void *workspace, size_t workspace_bytes,
                    void *cuda_stream);

/* Bytes of workspace with which mxp_gemm runs its fastest kernel for this problem
 * (a_dense != 0: weight-only form), and the least it accepts. */
size_t mxp_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dense,
                                mxp_mode a_mode, mxp_mode b_mode);
size_t mxp_gemm_min_workspace_bytes(int64_t M, int64_t N, int64_t K, int a_dense,
                                    mxp_mode a_mode, mxp_mode b_mode);

/*
 * Weights prepared once.  mxp_gemm with the full workspace re-tiles the scales of both
 * operands and prepares the MX+ ones (split per Eq. 4, or widened to E2M3 / E4M3 codes) on
 * every call (see `workspace` above).  For an operand that does not change between calls (the
 * N x K weights) that work can be done once.  Which form a GEMM reads depends on both
 * operands' modes; mxp_gemm_prepack_form tells:
 *   MXP_PREPACK_PLAIN  scale atoms only: B is MXFP4 and A is MXFP4 or MXFP4+
 *   MXP_PREPACK_WIDE   12 bytes per 16 elements: E2M3 codes (exact for every E2M1 value and
 *                      for the BM values of Eq. 3), packed; the tensor map spreads them into
 *                      the 16-byte slots the tensor core reads.  B is MXFP4, MXFP4+ or MXFP6
 *                      and the pairing is not one of the two above or below: both operands
 *                      MX+, the wider modes, and the weight-only tensor-core path
 *   MXP_PREPACK_WIDE8  16 bytes per 16 elements: E4M3 bytes, where B is MX++ or MXFP8
 *   MXP_PREPACK_WIDE_X2   B is MXFP6+: two planes of E2M3 codes (its BM is the sum of two)
 *   MXP_PREPACK_WIDE8_X3  B is MXFP8+: three planes of E4M3 bytes (its BM is the sum of three)
 *   MXP_PREPACK_SPLIT  B is MXFP4+ and A is MXFP4: Eq. 4's split for the sparse residual
 *                      instruction -- B's nibble plane with BM_H in every BM's place, BM_L
 *                      compressed 2:1, and the metadata that says where each BM_L sits
 *   mxp_gemm_prepack_form   the form (an mxp_prepack_form) of B's copy that mxp_gemm_prepacked
 *                           reads for these two modes
 *   mxp_gemm_prepack_bytes  bytes of that form of a rows x K operand.  0: shape or form not
 *                           supported (K % 128 != 0).
 *   mxp_gemm_prepack        writes that form of `P` into `out` (device, 256-byte aligned,
 *                           `out_bytes` >= the size above).  Asynchronous on `cuda_stream`.
 *   mxp_gemm_prepacked      mxp_gemm's packed-operand form with B's prepacked copy:
 *                           `B_prepacked` must come from mxp_gemm_prepack(B_packed, form) with
 *                           form == mxp_gemm_prepack_form(A's mode, B's mode), and
 *                           `B_prepacked_bytes` must be mxp_gemm_prepack_bytes(N, K, form): the
 *                           call checks that before any launch (MXP_ERR_INVALID_ARG), so a copy
 *                           made for another shape or another pairing of modes is refused
 *                           instead of being read past its end.  B_packed still describes the
 *                           operand (planes, shape, mode).  Needs M > 128 and
 *                           N > 128 and mxp_gemm_workspace_bytes(...) of workspace
 *                           (MXP_ERR_UNSUPPORTED / MXP_ERR_WORKSPACE otherwise; fall back
 *                           to mxp_gemm).  Same result as mxp_gemm.
 * The paper describes the format and its decode (Sec. 4, Eq. 3), not this staging: it is
 * an implementation device of this library.
 *   mxp_gemm_dense_prepacked  the weight-only form (bf16 activations, more than one tile's
 *                           worth of rows is where it pays: see mxp_gemm) with B's prepacked
 *                           copy in its widened form, MXP_PREPACK_WIDE or, for MX++ weights,
 *                           MXP_PREPACK_WIDE8 (size checked as above).  Workspace
 *                           (device, 256-byte aligned): at least
 *                           mxp_gemm_dense_prepacked_workspace_bytes(M, K) bytes (0: shape
 *                           not supported), which hold the activations' two planes and
 *                           scales.  Any M >= 1; 4-bit weight modes; K % 128 == 0.  Same
 *                           result as mxp_gemm's tensor-core weight-only path.
 */
typedef enum {
    MXP_PREPACK_PLAIN = 0,
    MXP_PREPACK_WIDE = 1,
    MXP_PREPACK_SPLIT = 2,
    MXP_PREPACK_WIDE8 = 3,
    MXP_PREPACK_WIDE_X2 = 4,
    MXP_PREPACK_WIDE8_X3 = 5
} mxp_prepack_form;
int mxp_gemm_prepack_form(mxp_mode a_mode, mxp_mode b_mode);
size_t mxp_gemm_prepack_bytes(int64_t rows, int64_t K, int form);
mxp_status mxp_gemm_prepack(const mxp_packed *P, int form, void *out, size_t out_bytes,
                            void *cuda_stream);
mxp_status mxp_gemm_prepacked(int64_t M, int64_t N, int64_t K, const mxp_packed *A_packed,
                              const mxp_packed *B_packed, const void *B_prepacked,
                              size_t B_prepacked_bytes, void *D, mxp_dtype d_dt, int64_t ldd,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t mxp_gemm_dense_prepacked_workspace_bytes(int64_t M, int64_t K);
mxp_status mxp_gemm_dense_prepacked(int64_t M, int64_t N, int64_t K, const void *A_dense_bf16,
                                    int64_t lda, const mxp_packed *B_packed,
                                    const void *B_prepacked, size_t B_prepacked_bytes, void *D,
                                    mxp_dtype d_dt, int64_t ldd, void *workspace,
                                    size_t workspace_bytes, void *cuda_stream);

/*
 * Quantization fused with the preparation of the GEMM operand (Sec. 5, software integration:
 * the activations are quantized right before the matrix multiply that consumes them).
 *   mxp_quantize_gemm_ready  mxp_quantize of an M x K bf16 matrix with contiguous rows
 *                            (ld_src == K; MXFP4 or MXFP4+; anything else MXP_ERR_UNSUPPORTED)
 *                            that also writes, into `workspace`, the operand in the form the
 *                            streamed tensor-core kernel reads (what mxp_gemm_prepacked would
 *                            otherwise derive from the packed planes in a launch of its own)
 *                            and clears the workspace's status block.  `b_mode`: the mode of
 *                            the operand the result will be multiplied with; it decides the
 *                            form, as for mxp_gemm: an MXFP4+ A against an MXFP4 B is split per
 *                            Eq. 4 for the sparse residual instruction (needs K % 256 == 0),
 *                            every other pairing is widened.  `workspace`: device, 256-byte
 *                            aligned, at least mxp_gemm_workspace_bytes(M, N, K, 0, mode,
 *                            b_mode) bytes for the GEMM it will serve; M > 128, K % 128 == 0.
 *   mxp_gemm_ready           mxp_gemm_prepacked for an A prepared that way in the same
 *                            `workspace` (nothing may have written to it in between) and a B
 *                            prepacked in the form mxp_gemm_prepack_form(A's mode, B's mode)
 *                            says, except that an MXFP4 A against an MXFP4+ B reads the widened
 *                            forms here (size checked as for mxp_gemm_prepacked): one launch.
 *                            Same result as mxp_gemm.
 */
mxp_status mxp_quantize_gemm_ready(const void *src, mxp_dtype src_dt, int64_t M, int64_t K,
                                   int64_t ld_src, mxp_mode mode, mxp_mode b_mode,
                                   uint8_t *nibbles, uint8_t *scales, uint8_t *bm_index,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);
mxp_status mxp_gemm_ready(int64_t M, int64_t N, int64_t K, const mxp_packed *A_packed,
                          const mxp_packed *B_packed, const void *B_prepacked,
                          size_t B_prepacked_bytes, void *D, mxp_dtype d_dt, int64_t ldd,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The weight-only form of mxp_gemm for a chain of decode GEMMs on one stream (Sec. 7.1:
 * "conversion before computation", the memory-bound token-generation phase, where one such
 * GEMM follows another and each streams its own weights once).  Same operation and result
 * as mxp_gemm(A_dense_bf16, B_packed); the difference is when the grid may start: it is
 * launched as a programmatic dependent of the preceding kernel on `cuda_stream`, so its
 * CTAs are scheduled while that kernel drains and begin streaming B's planes at once.
 * Ordering that still holds: A is read and D is written only after the preceding kernel has
 * completed and its writes are visible.  Ordering the caller gives up: B's three planes
 * (nibbles, scales, bm_index) must not be written by the kernel that precedes this call on
 * the stream (weights quantised once, ahead of the decode loop, satisfy this; quantising B
 * immediately before this call does not: use mxp_gemm there).  Every streamed weight-only
 * kernel of this library releases its own dependents when it starts, so a chain of these
 * calls overlaps launch to launch; after any other kernel the call behaves like mxp_gemm.
 * May be captured into a CUDA graph (the launches become programmatic dependency edges).
 *
 *   M <= 64, N % 16 == 0, K % 256 == 0, pointers 16-byte aligned, lda % 8 == 0; otherwise
 *   MXP_ERR_UNSUPPORTED and nothing is launched (use mxp_gemm).
 *   status_block   device pointer (16 bytes, 16-byte aligned) or NULL.  NOT cleared by the
 *                  call (a clear between the kernels would break the chain): zero it once,
 *                  the first bounded wait that runs out in any call of the chain leaves
 *                  MXP_ERR_TIMEOUT there; read it with mxp_gemm_status.
 */
mxp_status mxp_gemm_decode_chained(int64_t M, int64_t N, int64_t K, const void *A_dense_bf16,
                                   int64_t lda, const mxp_packed *B_packed, void *D,
                                   mxp_dtype d_dt, int64_t ldd, void *status_block,
                                   void *cuda_stream);

/*
 * The weight-only form for decode shapes (1 <= M <= 16) with the weights re-tiled once (Sec. 7.1:
 * the memory-bound token-generation phase; Eq. 3 decode, BM split per Eq. 4).  The GEMM streams
 * every weight byte exactly once, straight into the FP4 tensor cores:
 *   mxp_gemm_decode_prepack_bytes  bytes of the re-tiled form of an N x K weight operand in
 *                            mode MXFP4 or MXFP4+ on the CURRENT device (the tiling depends on
 *                            its SM count); 0: not supported (K % 256 != 0, other modes).
 *   mxp_gemm_decode_prepack  writes that form into `out` (device, 256-byte aligned, out_bytes >=
 *                            the size above).  A re-ordering of the stored 4-bit codes, scales
 *                            and BM indices; for MXFP4+ the BM's code is replaced by its upper
 *                            part BM_H (an E2M1 value) and the lower part BM_L is kept in a
 *                            record byte per block.  Blocks with scale byte 0 become zeros.
 *   mxp_gemm_decode_workspace_bytes  device scratch one call needs (0: M or K not supported):
 *                            a status block and the activations' operand images.
 *   mxp_gemm_decode_prepacked  D[M,N] = A(bf16)[M,K] * dec(B)[N,K]^T.  `b_mode`, N, K must be
 *                            those B_prepacked was made with, and B_prepacked_bytes the size
 *                            mxp_gemm_decode_prepack_bytes gives for them (checked before any
 *                            launch: MXP_ERR_INVALID_ARG).  The activations become five FP4
 *                            digit planes per row (balanced base 8, a block scale per plane: an
 *                            element within 2^5 of the largest magnitude of its block of 32 is
 *                            exact, a smaller one is rounded at 2^-13 of that magnitude's
 *                            binade -- far inside the GEMM's error bound, which is relative to
 *                            the row norm).  Up to three rows (two with MXFP4+ weights), when
 *                            the planes of all of K fit shared memory: one launch, every CTA
 *                            converts the rows for itself.  Otherwise two launches: a small
 *                            kernel writes the planes to the workspace and the GEMM is launched
 *                            as its programmatic dependent and starts streaming weights at once.
 *                            chained != 0: the first kernel is itself launched as a
 *                            programmatic dependent of whatever precedes it on the stream, with
 *                            the promise and the status-block rule of mxp_gemm_decode_chained
 *                            (B_prepacked not written by the preceding kernel; status block
 *                            not cleared).  M > 16 or unsupported shapes: MXP_ERR_UNSUPPORTED
 *                            (use mxp_gemm).  Same result as mxp_gemm within its bound; one-hot
 *                            activation rows return decoded weights bit for bit.
 *   mxp_gemm_decode_prepacked_next  the same call with a hint: `next_B_prepacked` (device, the
 *                            output of mxp_gemm_decode_prepack for any shape, with its size; NULL
 *                            and 0: no hint) names the weights of the call expected next on this
 *                            stream, a decoder's next layer.  About a third of a call's time --
 *                            its last MMAs and stores, the switch to the next call's CTAs, their
 *                            first copies' latency -- moves no weights; once a CTA's own weights
 *                            have all but landed it asks for the head of the next call's (what
 *                            its ring will hold first) to be fetched into L2, from where that
 *                            call streams them faster than from HBM.  Nothing waits for the
 *                            fetch and the result does not depend on it; a pointer and size that
 *                            do not describe readable device memory are the caller's error
 *                            (alignment and NULL / 0 pairing are checked: MXP_ERR_INVALID_ARG).
 * The paper describes the format and its decode, not this staging.
 */
size_t mxp_gemm_decode_prepack_bytes(int64_t N, int64_t K, mxp_mode b_mode);
size_t mxp_gemm_decode_workspace_bytes(int64_t M, int64_t K);
mxp_status mxp_gemm_decode_prepack(const mxp_packed *B_packed, void *out, size_t out_bytes,
                                   void *cuda_stream);
mxp_status mxp_gemm_decode_prepacked(int64_t M, int64_t N, int64_t K, const void *A_dense_bf16,
                                     int64_t lda, mxp_mode b_mode, const void *B_prepacked,
                                     size_t B_prepacked_bytes, void *D, mxp_dtype d_dt,
                                     int64_t ldd, void *workspace, size_t workspace_bytes,
                                     int chained, void *cuda_stream);
mxp_status mxp_gemm_decode_prepacked_next(int64_t M, int64_t N, int64_t K,
                                          const void *A_dense_bf16, int64_t lda, mxp_mode b_mode,
                                          const void *B_prepacked, size_t B_prepacked_bytes,
                                          void *D, mxp_dtype d_dt, int64_t ldd, void *workspace,
                                          size_t workspace_bytes, int chained,
                                          const void *next_B_prepacked,
                                          size_t next_B_prepacked_bytes, void *cuda_stream);

/*
 * Reads back (synchronously, after synchronising `cuda_stream`) the status block a GEMM
 * left in `workspace`: MXP_OK, or MXP_ERR_TIMEOUT if a bounded wait inside a kernel gave
 * up (the output is then undefined but the context stays usable).
 */
mxp_status mxp_gemm_status(const void *workspace, void *cuda_stream);

/*
 * How fast the SMs were clocked during the last GEMM that ran the streamed tensor-core kernel
 * with this `workspace` (the path taken when the workspace has mxp_gemm_workspace_bytes(...)
 * bytes; measurement aid, no counterpart in the paper).  The kernel's first CTA reads the SM
 * cycle counter and the GPU's nanosecond timer when it starts and after its last tile;
 * *sm_cycles / *nanoseconds is the SM clock in GHz the kernel really ran at, which a dense
 * tensor-core kernel at the board's power limit holds well below the nominal maximum.
 * Synchronises `cuda_stream`.  `workspace`: device, >= 256 bytes; the outputs are host
 * pointers.  MXP_ERR_UNSUPPORTED when the workspace holds no stamp (another kernel ran).
 */
mxp_status mxp_gemm_clock_stamp(const void *workspace, void *cuda_stream, uint64_t *sm_cycles,
                                uint64_t *nanoseconds);

/*
 * Self-test of the bounded device-side waits (the paper has no counterpart: it is how this
 * library's kernels report a wait that runs out instead of hanging).  Launches one warp
 * that waits, for at most `limit_cycles` SM clock cycles (1 .. 2e9), on a barrier nothing
 * signals.  Afterwards mxp_gemm_status(workspace, stream) must return MXP_ERR_TIMEOUT, and
 * the device must be usable as before.  `workspace`: device, 16-byte aligned, >= 16 bytes.
 */
mxp_status mxp_wait_selftest(void *workspace, size_t workspace_bytes, int64_t limit_cycles,
                             void *cuda_stream);

/*
 * Issue-rate probe for the roofline denominator: runs `iters` back-to-back tensor-core
 * instructions per CTA on operands resident in shared memory (no global traffic) on
 * every SM and returns the elapsed milliseconds in *ms (synchronises the device).
 *   kind 0: kind::mxf4 block-scaled E2M1 x E2M1 (128 x 256 x 64 per instruction)
 *   kind 1: kind::mxf8f6f4 block-scaled E2M3 x E2M3 (128 x 256 x 32 per instruction)
 *   kind 2: as kind 0 plus the three scale-factor copies (tcgen05.cp) a 128 x 256 tile needs
 *           per 128 elements of K, into one TMEM buffer
 *   kind 3: as kind 2 with the copies alternating between two TMEM buffers
 *   kind 4: the sparse form (Sec. 5.2, "sparse MMA"): one tcgen05.mma.sp of 128 x 256 x 128
 *           per group, A stored 2:1 compressed
 *   kind 5: two dense instructions of kind 0 and one sparse one per group: the instruction mix
 *           of a main pass plus a sparse residual pass over the same 128 elements of K
 * `iters` counts groups (128 elements of K for the FP4 kinds, 64 for kind 1).
 * *flops receives 2 * M * N * K of the groups summed over CTAs (for kind 5 the K of the main
 * pass only: the residual instruction is overhead).
 * The paper has no counterpart; it exists so that fractions of peak have a measured
 * denominator on the device the library runs on.
 */
mxp_status mxp_tensor_peak_probe(int kind, int iters, double *ms, double *flops);

/*
 * The packed-operand form of mxp_gemm for callers that cannot allocate device memory
 * (the paper has no counterpart; this is a deployment convenience).
 *
 * Who needs it: code that runs inside another framework's memory pool and must not call
 * cudaMalloc behind its back, plugins loaded after the pool has taken the whole device,
 * and callers with no allocator of their own to ask for the GEMM's small workspace.
 * Here that workspace (the status block the kernel's bounded waits report into) lives in
 * a fixed device array inside the library: 4096 bytes that every GPU which loads libmxp
 * holds until the process exits.  The call allocates and frees nothing, on the host or
 * the device; A, B and D are still the caller's memory, with the same layout rules as
 * mxp_gemm.  A problem whose workspace need exceeds those 4096 bytes is rejected with
 * MXP_ERR_WORKSPACE before anything is launched.
 *
 * With so little scratch the call always runs the kernels that work on the packed planes in
 * place (Eq. 4 / Algorithm 1 with dense residual passes), never the faster ones that first
 * prepare the operands in a workspace: on the 8192 x 28672 x 8192 prefill shape about 0.89 ms
 * for MXFP4 x MXFP4 against 0.68 ms, 1.8 ms for one MXFP4+ operand against 0.95 ms, and
 * 2.6 ms for two against 1.3 ms.  MX++ and the 6- and 8-bit modes need the workspace forms:
 * MXP_ERR_UNSUPPORTED here.
 *
 * The first call on a device looks up the array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.  The
 * remembered address belongs to the device's context: after cudaDeviceReset the library
 * must be reloaded before this entry point is used again.
 * All calls on a device share the one array and it keeps what the previous call left:
 * the status block is cleared on `cuda_stream` at the start of every call, but two calls
 * whose kernels overlap on the GPU (different streams) race on it; serialise them.
 *
 *   kernel_status  host pointer or NULL.  When given, the call synchronises `cuda_stream`
 *                  and stores MXP_OK or MXP_ERR_TIMEOUT (what mxp_gemm_status would
 *                  report); when NULL the call stays asynchronous.
 */
mxp_status mxp_gemm_noalloc(int64_t M, int64_t N, int64_t K, const mxp_packed *A_packed,
                            const mxp_packed *B_packed, void *D, mxp_dtype d_dt, int64_t ldd,
                            mxp_status *kernel_status, void *cuda_stream);

/*
 * Test and measurement aid (no counterpart in the paper): forces a kernel choice that the
 * dispatch of mxp_gemm would otherwise make by shape, so that every kernel can be reached with
 * any operands.  Process-wide and not synchronised with calls in flight; value 0 gives the
 * choice back to the library.  Not meant for production use.
 *   MXP_KNOB_INPLACE_KERNEL      packed x packed mxp_gemm: 1 = the in-place single-CTA kernel,
 *                                2 = the in-place CTA-pair kernel (either also keeps the call
 *                                away from the streamed kernel on prepacked operands)
 *   MXP_KNOB_STREAM_HALVES       streamed kernel: 1 / 2 = output tile of one / two halves
 *   MXP_KNOB_WEIGHT_ONLY_KERNEL  weight-only mxp_gemm: 1 = the general kernel, 2 = the streamed
 *                                decode kernel where it applies (either keeps M > 64 calls
 *                                away from the tensor-core path)
 *   MXP_KNOB_ONE_SIDED           one MXFP4+ operand against an MXFP4 one: 1 = the single pass on
 *                                widened codes instead of the sparse residual instruction (the
 *                                prepacked form of B such calls read is then MXP_PREPACK_WIDE)
 * Returns MXP_ERR_INVALID_ARG for an unknown knob or a value outside 0..2.
 */
typedef enum {
    MXP_KNOB_INPLACE_KERNEL = 0,
    MXP_KNOB_STREAM_HALVES = 1,
    MXP_KNOB_WEIGHT_ONLY_KERNEL = 2,
    MXP_KNOB_ONE_SIDED = 3,
    MXP_KNOB_COUNT_ = 4
} mxp_knob;
mxp_status mxp_debug_override(int knob, int value);

const char *mxp_status_string(mxp_status s);

/* Library version string, e.g. "mxp 0.1 sm_100a". */
const char *mxp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MXP_H_ */
