/*
 * ufp4.h — C ABI of libufp4: the UFP4 training hot path on NVIDIA B200 (sm_100a).
 *
 * Two operations, as the paper states them:
 *   1. the blockwise quantizer of Sec. 2.1 (s_B = max|x_j| / g_max, q_i = rho_G(x_i / s_B), rho_G = RTNE or SR) fused
 *      with the 16-point Random Hadamard Transform of Sec. 2.2 (H'_16 = S_16 H_16), in the configuration of
 *      Sec. 4 / Table 1: 1x16 blocks, one scale per block, RHT block 16, RTNE for X and W, SR for dY;
 *   2. the low-precision GEMM of Sec. 2.2, Y^ = Q_G(X H') Q_G(W H')^T, for the three training products fwd_y, bwd_dx
 *      and bwd_dw, each reducing over the dimension its operands were rotated and blocked along.
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned and sized by the caller unless a parameter says "host".  The library
 *     allocates no device memory and keeps no per-call state.  Work is enqueued on the caller's CUDA stream
 *     (a cudaStream_t passed as void*; NULL = the default stream) and the call returns without synchronizing.
 *   - Errors the host can see (null pointers, shapes, alignment, enums, too-small workspace) return a negative
 *     ufp4_status and launch nothing.  Conditions only the device can see set bits in *dev_status (device int32,
 *     optional): UFP4_DEV_NONFINITE, UFP4_DEV_EXP_WINDOW, UFP4_DEV_WAIT_TIMEOUT.  Bits are OR-ed in, never cleared.
 *   - A quantized tensor is logically [rows][k] with k the reduction dimension; codes are packed two per byte along k
 *     (element 2j in bits 3:0 of byte j, element 2j+1 in bits 7:4); there is one scale per 16 consecutive k.
 *   - All three training GEMMs are the same contraction C[m][n] = sum_k A[m][k] * B[n][k] on k-contiguous operands:
 *       fwd_y : A = rows variant of X  [T][K],  B = row variant of W  [N][K]   -> Y  [T][N]
 *       bwd_dx: A = row variant of dY  [T][N],  B = col variant of W  [K][N]   -> dX [T][K]
 *       bwd_dw: A = col variant of dY  [N][T],  B = col variant of X  [K][T]   -> dW [N][K]
 *     Both operands of a product must have been quantized with the same seed_rht and rht_block along the shared
 *     dimension (Sec. 2.2: the identity X W^T = (X H')(W H')^T needs the same H'); the library cannot check this.
 */
#ifndef UFP4_H_
#define UFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    UFP4_OK = 0,
    UFP4_ERR_NULL = -1,        /* a required pointer is NULL */
    UFP4_ERR_SHAPE = -2,       /* a dimension is non-positive or not a multiple of what the operation needs */
    UFP4_ERR_ALIGN = -3,       /* a pointer or leading dimension breaks the stated alignment */
    UFP4_ERR_ENUM = -4,        /* an enum value is out of range */
    UFP4_ERR_UNSUPPORTED = -5, /* a valid combination this build does not implement */
    UFP4_ERR_CUDA = -6,        /* a CUDA runtime call failed (launch error, no sm_100 device, ...) */
    UFP4_ERR_WORKSPACE = -7    /* workspace missing or smaller than ufp4_gemm_workspace_bytes() */
} ufp4_status;

/* Data-element grids (Sec. 2.1; Sec. 3.1 prints the E2M1 magnitudes).  INT4 and E1M2 are the same uniform grid:
 * INT4 stores q in [-7,7] as a two's-complement nibble with g_max = 7; E1M2 stores sign|e|mm with values q/4 and
 * g_max = 1.75, so its block scale is exactly 4x the INT4 one.  E2M1 is the comparison grid {0,.5,1,1.5,2,3,4,6}
 * stored as sign|ee|m.  Zero is always encoded as nibble 0x0.
 * E2M1_MAX4 / E2M1_MAX2 are the range-restricted E2M1 of Sec. 5.4 (App. B's `max_fpx` = 4 / 2): the quantizer scales by
 * g_max = 4 / 2 and rounds onto the E2M1 levels not above it (max_fpx = 2 keeps {0,.5,1,1.5,2}); the codes are E2M1
 * codes, so the GEMM and diagnostics calls read such a tensor exactly like an E2M1 one. */
typedef enum {
    UFP4_GRID_INT4 = 0, UFP4_GRID_E1M2 = 1, UFP4_GRID_E2M1 = 2, UFP4_GRID_E2M1_MAX4 = 3, UFP4_GRID_E2M1_MAX2 = 4
} ufp4_grid;

/* Rounding rule rho_G (Sec. 2.1).  RTNE: nearest level, ties to the even code.  SR: between neighbouring levels
 * g_a <= t < g_b the upper one is taken with probability (t - g_a)/(g_b - g_a), resolved to 1/256 by one random byte
 * per element from Philox4x32-10 keyed by seed_sr and the block index (Table 1: SR on dY only). */
typedef enum { UFP4_ROUND_RTNE = 0, UFP4_ROUND_SR = 1 } ufp4_round;

/* Which dimension the 16-element blocks (and the RHT) run along (Sec. 2.2, last paragraph: the reduction dimension
 * of the product the tensor feeds).  ROW: along the last dimension.  COL: along the first dimension, output stored
 * transposed.  BOTH: both variants from one pass over the input. */
typedef enum { UFP4_AXIS_ROW = 0, UFP4_AXIS_COL = 1, UFP4_AXIS_BOTH = 2 } ufp4_axis;

/* Block-scale format.  FP32: s = RN(amax / g_max), Table 1's "FP32 single-level".  POW2: that value rounded up to a
 * power of two, still stored as FP32 (Sec. 4 leaves the scale hierarchy open "depending on hardware efficiency"); it
 * is the format the tensor-core GEMM path folds into its 8-bit operands exactly.  E4M3_TENSOR: an E4M3 byte per
 * block times one FP32 per tensor (the two-level layout Sec. 2.1's footnote attributes to NVFP4). */
typedef enum {
    UFP4_SCALE_FP32 = 0, UFP4_SCALE_POW2 = 1, UFP4_SCALE_E4M3_TENSOR = 2,
    /* One power-of-two scale per 32 consecutive elements: the 1x32 blocks with an E8M0 scale that Sec. 2.1's footnote
     * attributes to MXFP4, here on any grid.  amax is taken over the 32 (rotated) elements, the scale is the next
     * power of two >= amax / g_max and is stored, as FP32, for both 16-element halves, so that the GEMM and
     * diagnostics calls read such a tensor exactly like a POW2 one.  The reduction dimension must be a multiple of 32.
     * The quantizer serves this format with its plain kernel (see rht_block). */
    UFP4_SCALE_E8M0_B32 = 3
} ufp4_scale_fmt;

/* Which training product a GEMM call computes.  All are C = A B^T on k-contiguous operands; the value matters only to
 * the grouped call, where fwd_y / bwd_dx split the rows of A (and C) by group and bwd_dw splits the reduction. */
typedef enum { UFP4_FWD_Y = 0, UFP4_BWD_DX = 1, UFP4_BWD_DW = 2 } ufp4_layout;

/* Bits of *dev_status. */
enum {
    UFP4_DEV_NONFINITE = 1,    /* a block held Inf/NaN: its codes and scale are unspecified */
    UFP4_DEV_EXP_WINDOW = 2,   /* tensor-core GEMM: a block scale lay outside the exponent window of its row and was
                                  flushed to zero; re-run with the exact path (see ufp4_gemm) */
    UFP4_DEV_WAIT_TIMEOUT = 4  /* a bounded pipeline wait inside a kernel gave up; the output is invalid */
};

/* A quantized tensor (device pointers, caller-owned). */
typedef struct ufp4_qtensor {
    void *codes;               /* uint8 [rows][ld_codes_bytes]; the first k/2 bytes of a row are used; 16-B aligned */
    void *scales;              /* float [rows][ld_scales] (FP32, POW2) or uint8 [rows][ld_scales] (E4M3_TENSOR)      */
    const float *tensor_scale; /* device pointer to one float; E4M3_TENSOR only (input to the quantizer), else NULL  */
    int64_t rows;              /* logical rows                                                                       */
    int64_t k;                 /* reduction dimension, multiple of 16                                                */
    int64_t ld_codes_bytes;    /* row pitch of codes in bytes, multiple of 16, >= k/2                                */
    int64_t ld_scales;         /* row pitch of scales in elements, >= k/16                                           */
    int32_t grid;              /* ufp4_grid                                                                          */
    int32_t scale_fmt;         /* ufp4_scale_fmt                                                                     */
} ufp4_qtensor;

/* Library version (major*10000 + minor*100 + patch). */
int ufp4_version(void);

/* Static, NUL-terminated description of a status code. */
const char *ufp4_status_string(int status);

/* The 16 RHT signs of a seed (host computation): bit i set means eps_i = -1 (Sec. 2.2, S_16 = diag(eps)).
 * Bits are the low 16 bits of word 0 of Philox4x32-10 with counter (0,0,0,0x52485400) and key (lo32, hi32) of seed. */
uint32_t ufp4_rht_sign_mask(uint64_t seed_rht);

/* The sign bits of the wider RHT blocks (32 / 64 / 128, the sizes App. B lists beside the selected 16): all 128 bits of
 * the same Philox output, bit i (word i / 32, bit i % 32) set meaning eps_i = -1; the mask above is its first 16 bits.
 * Host computation; out is host memory. */
void ufp4_rht_signs(uint64_t seed_rht, uint32_t out[4]);

/* Densely packed sizes of a [rows][k] quantized tensor (ld_codes_bytes = k/2 rounded up to 16, ld_scales = k/16). */
int ufp4_qtensor_bytes(int64_t rows, int64_t k, int scale_fmt, size_t *codes_bytes, size_t *scales_bytes);

/*
 * Fused RHT + blockwise quantizer (Sec. 2.1 quantizer; Sec. 2.2 RHT; Sec. 4 / Table 1 settings; Sec. 5.5 describes
 * the fusion: rotate before scale estimation and packing, no rotated tensor is materialised).
 *
 *   x          BF16 [rows][cols], row pitch ld elements; 16-B aligned, ld % 8 == 0
 *   axis       ROW needs cols % 16 == 0 and fills *out_row = [rows][cols];
 *              COL needs rows % 16 == 0 and cols % 16 == 0 and fills *out_col = [cols][rows];
 *              BOTH fills both from a single read of x
 *   rht_block  0 (no rotation), 16 (the recipe's choice, Table 1), or 32 / 64 / 128 (App. B's other candidates: the
 *              reduction dimension of each requested variant must then be a multiple of rht_block; the rotated values
 *              are scaled by RN(1 / sqrt(rht_block)) in FP32 and their 16-element blocks quantized as usual; a plain,
 *              slower kernel)
 *   seed_rht   selects the sign vector (ufp4_rht_sign_mask); along COL the sign of row r is eps_(r mod 16)
 *   seed_sr    key of the SR random bytes; counter = (lo32(b), hi32(b), variant, 0x53520000), b = index of the block in
 *              the variant's dense [rows][k/16] scale array, variant 0 = row, 1 = col
 *   out_row / out_col   describe caller-allocated outputs; rows, k, grid and scale_fmt must match the call, and for
 *              E4M3_TENSOR tensor_scale must point at the FP32 tensor scale to use
 *
 * Per block, in FP32: v = x (o) eps; butterfly stages h = 1,2,4,8; x' = v/4; amax = max|x'|; s = RN(amax/g_max);
 * y = RN(x' * RN(g_max/amax)); q = rho_G(y).  Blocks with amax == 0 or amax < 2^-100 store scale 0 and codes 0.
 * Inputs must be finite (else UFP4_DEV_NONFINITE) and |x'| <= 2^120.  Output is bit-reproducible.
 */
int ufp4_quantize(const void *x, int64_t rows, int64_t cols, int64_t ld, int axis, int rht_block, int grid,
                  int rounding, int scale_fmt, uint64_t seed_rht, uint64_t seed_sr, const ufp4_qtensor *out_row,
                  const ufp4_qtensor *out_col, int32_t *dev_status, void *stream);

/*
 * The same quantizer over a batch of equally shaped matrices x[e] = x + e * batch_stride (elements), e.g. the expert
 * weights [E][N][K] of an MoE layer (Sec. 5 trains MoE models; the quantizer itself is Sec. 2.1 / 2.2 as above).
 * Outputs are stacked along rows: *out_row = [batch * rows][cols], *out_col = [batch * cols][rows] (matrix e owns rows
 * [e * cols, (e+1) * cols) of it).  batch_stride % 8 == 0.  RTNE only (weights are never stochastically rounded,
 * Table 1); SR returns UFP4_ERR_UNSUPPORTED when batch > 1.
 */
int ufp4_quantize_batched(const void *x, int64_t batch, int64_t batch_stride, int64_t rows, int64_t cols, int64_t ld,
                          int axis, int rht_block, int grid, int rounding, int scale_fmt, uint64_t seed_rht,
                          uint64_t seed_sr, const ufp4_qtensor *out_row, const ufp4_qtensor *out_col,
                          int32_t *dev_status, void *stream);

/*
 * Several independent tensors in one call (a layer's X, W and dY): the same as calling ufp4_quantize for args[0],
 * args[1], ... in this order on `stream`, except that the kernel of each tensor after the first is launched as a
 * programmatic dependent of the one before it, so that its thread blocks fill the last, partly empty wave of its
 * predecessor instead of waiting for it to drain.  INDEPENDENT means: no tensor of the call reads or overwrites what
 * another one writes (inputs may be shared).  Work enqueued on the stream afterwards sees all outputs complete, as
 * after separate calls.  All argument sets are checked before anything is launched: on an error (the status of the first
 * offending set) nothing has been enqueued.  args: HOST array of `count` entries, read during the call only.
 */
typedef struct ufp4_quantize_args {
    const void *x;                       /* device, BF16 [rows][ld]                                   */
    int64_t rows, cols, ld;
    int32_t axis, rht_block, grid, rounding, scale_fmt;
    int32_t reserved;                    /* 0                                                         */
    uint64_t seed_rht, seed_sr;
    const ufp4_qtensor *out_row, *out_col;
} ufp4_quantize_args;
int ufp4_quantize_multi(int count, const ufp4_quantize_args *args, int32_t *dev_status, void *stream);

/*
 * Self-check of the quantizer's scale arithmetic (Sec. 2.1: s_B = amax / g_max and x_i / s_B).  The kernel evaluates
 * amax / g and g / amax with short FMA sequences instead of the generic division; this call compares both sequences
 * with the IEEE-754 division for every FP32 mantissa at eight exponents of the supported range and g in {7, 1.75, 6},
 * and adds the number of differing results to *dev_mismatches (device int32, zeroed by the caller; expected 0).
 */
int ufp4_selftest_division(int32_t *dev_mismatches, void *stream);

/* Workspace the GEMM calls need for these operands and this path request (0 for the exact path). */
size_t ufp4_gemm_workspace_bytes(const ufp4_qtensor *A, const ufp4_qtensor *B, int path);

/* GEMM paths (given a workspace of ufp4_gemm_workspace_bytes(A, B, path); without one AUTO falls back to EXACT).
 * AUTO:    TENSOR when both operands use power-of-two scales (1 x 16 or 1 x 32); when both use E4M3 x tensor scales, NVF4
 *          for plain products and FP16 for grouped ones; else SPLIT.
 * EXACT:   CUDA-core kernel: integer block partials (dp4a) promoted with the two FP32 block scales, FP64 running sum;
 *          every grid and scale format, no workspace; the slow reference path.
 * TENSOR:  tcgen05 / TMEM kernel on 8-bit floating-point operands into which code x 2^e is folded exactly (POW2 scales
 *          only); blocks whose exponent lies outside a row's window set UFP4_DEV_EXP_WINDOW.
 * PROMOTE: tcgen05 computes the exact integer partial of every 16-element block (BF16 operands, K = 16 per MMA) and the
 *          CUDA cores promote it with sA * sB into FP32 accumulators; every grid and scale format (Table 1's FP32 scales).
 *          A row-grouped product needs group_n % 4 == 0 on this path (else UFP4_ERR_UNSUPPORTED; AUTO moves on to EXACT).
 * SPLIT:   tcgen05 / TMEM kernel on FP16 operands: each dequantized value, relative to a per-row power-of-two
 *          reference, is split into two FP16 pieces (22 significant bits) and the product taken by three MMAs per K
 *          step; every grid and scale format (Table 1's FP32 scales), plain and grouped; blocks more than 2^26 below
 *          a row's largest scale are flushed and set UFP4_DEV_EXP_WINDOW.
 * FP16:    the same kernels with one FP16 piece per value and one MMA per K step, for operands that BOTH carry
 *          E4M3 block scales times a per-tensor FP32 scale (the two-level hierarchy Sec. 2.1's footnote names):
 *          level x E4M3 value has at most 7 significant bits, so it is exact in FP16 without a row reference or an
 *          exponent window, and the two tensor scales multiply the result once (they enter as RN(ts x E4M3 value) in
 *          the definition: a relative difference of 2^-24 per operand, far inside the bound below).  Any other scale
 *          format: UFP4_ERR_UNSUPPORTED.
 * MX:      tcgen05 / TMEM kernel with the hardware's own block scaling (kind::mxf8f6f4, one UE8M0 scale per 32 elements,
 *          Sec. 2.1's footnote on MXFP4): the operand element is the bare code as an 8-bit float and the tensor core
 *          applies the scales, so there is no per-row reference and no window relative to the rest of the row.  Both
 *          operands must carry power-of-two scales: UFP4_SCALE_E8M0_B32 is exact by construction (nothing is ever
 *          flushed), UFP4_SCALE_POW2 folds the gap between the two 16-blocks of a 32-group into the elements (a block
 *          more than 2^14 below its neighbour is flushed and sets UFP4_DEV_EXP_WINDOW).  Plain and reduction-grouped
 *          products; a row-grouped product returns UFP4_ERR_UNSUPPORTED.  On request only: on the same operands TENSOR
 *          is the faster path (its accumulators are double-buffered and it copies no scales inside the main loop), so
 *          MX is the choice for rows whose block exponents spread beyond TENSOR's window.
 * NVF4:    tcgen05 / TMEM kernel on the FP4 tensor path (kind::mxf4nvf4) with the hardware applying one UE4M3 scale per
 *          16 elements, for operands that BOTH carry E4M3 block scales times a per-tensor FP32 scale.  That path knows
 *          the E2M1 levels only (Sec. 1): an E2M1 tensor is read as it stands (one MMA per 64-element step, nothing is
 *          decoded but the scale layout), a uniform code q is split into two E2M1 values, q / 2 = hi + lo, and the
 *          product taken plane by plane (four MMAs per step for two uniform tensors, two when one of them is E2M1).
 *          Exact like FP16 (no window, the tensor scales multiply the result once).  Plain products only. */
typedef enum {
    UFP4_PATH_AUTO = 0, UFP4_PATH_EXACT = 1, UFP4_PATH_TENSOR = 2, UFP4_PATH_PROMOTE = 3, UFP4_PATH_SPLIT = 4,
    UFP4_PATH_FP16 = 5, UFP4_PATH_MX = 6, UFP4_PATH_NVF4 = 7
} ufp4_gemm_path;

/* Which path ufp4_gemm would take for these operands and this request (given a sufficient workspace), or a negative
 * status.  *kernel_launches (optional, host) receives the number of kernels one
 * such call enqueues. */
int ufp4_gemm_path_taken(const ufp4_qtensor *A, const ufp4_qtensor *B, int path, int *kernel_launches);

/*
 * C[m][n] = sum_k a[m][k] * b[n][k], a = value(code) * scale (Sec. 2.2, Y^ = Q_G(XH') Q_G(WH')^T).
 *   A [M][K], B [N][K] quantized tensors with equal k; grids may differ
 *   C       FP32 (c_is_bf16 == 0) or BF16 [M][ldc], ldc in elements, 16-B aligned rows
 *   workspace / workspace_bytes   >= ufp4_gemm_workspace_bytes(A, B, path); may be NULL/0 when that is 0
 * Accumulation is FP32 or better; the result differs from the exact sum by at most 1e-5 * sum_k |a_k b_k|.
 */
int ufp4_gemm(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int layout, int path,
              void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/*
 * The same product with a quantizing epilogue (Sec. 5.5: "end-to-end training overhead still depends on full-system
 * integration"): C = A B^T is rounded to BF16, as it would be stored for the next layer, and leaves the kernel already
 * quantized the way ufp4_quantize(C, AXIS_BOTH, rht_block, UFP4_GRID_INT4, UFP4_ROUND_RTNE, scale_fmt, seed_rht) would
 * quantize it: out_row [M][N] with its 1 x 16 blocks (and the RHT) along N, out_col [N][M] with them along M.  Either
 * output may be NULL; C_bf16 [M][ldc] (optional, may be NULL) receives the BF16 product itself.  The FP32 product is
 * never written: 1.5 B per element leave the kernel instead of 4.
 *   A, B       POW2 scales (the tensor-core path); M and N multiples of 16
 *   outputs    grid UFP4_GRID_INT4, scale_fmt UFP4_SCALE_FP32 or UFP4_SCALE_POW2 (the same for both); rht_block 16 or 0
 *   workspace  ufp4_gemm_workspace_bytes(A, B, UFP4_PATH_TENSOR)
 * For consumers that round to nearest (the next layer's X); SR consumers go through ufp4_quantize.  The codes are those
 * of the BF16-rounded tensor-core result: where the exact product lies within the GEMM bound of a BF16 rounding
 * boundary, the BF16 value, and with it codes of its block, can differ from those of the exactly rounded product.
 */
int ufp4_gemm_quantized(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C_bf16, int64_t ldc, int rht_block,
                        uint64_t seed_rht, const ufp4_qtensor *out_row, const ufp4_qtensor *out_col, void *workspace,
                        size_t workspace_bytes, int32_t *dev_status, void *stream);

/*
 * MoE-grouped variant: one call for all experts.  offsets is a DEVICE int64 [num_groups+1] array of row offsets
 * (offsets[0] = 0, every offset a multiple of 128; padding rows must hold zero codes or zero scales), and
 * host_offsets the same values in HOST memory (the launch geometry is sized from them).
 *   FWD_Y, BWD_DX: A [total][K] with rows grouped; B [num_groups * N][K] (expert e owns rows [e*N, (e+1)*N));
 *                  C [total][N]: C[t][:] = A[t][:] . B_e(t)^T
 *   BWD_DW:        A [N][total], B [Kout][total] (reduction dimension grouped); C [num_groups * N][Kout]:
 *                  C_e = sum over k in [offsets[e], offsets[e+1]) of A[:,k] B[:,k]^T; an empty group writes zeros
 */
int ufp4_gemm_grouped(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int layout,
                      int path, const int64_t *offsets, const int64_t *host_offsets, int num_groups, int64_t group_n,
                      void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/*
 * Tensor diagnostics of Sec. 3 on a BF16 matrix x [rows][cols] and its row variant q_row (FP32 or POW2 scales), with
 * x' = x H'_n per n-element chunk for rht_block n = 16, 32, 64 or 128 (the quantizer's FP32 butterflies; cols must be a
 * multiple of n) or x' = x for rht_block == 0, and
 * xq = level * scale.  dev_out (device, 19 doubles) receives
 *   [0] sum x'^2   [1] sum (xq - x')^2   [2] sum xq x'      -> alpha = [2] / [0] (Eq. 3), NMSE = [1] / [0] (Sec. 3.3;
 *                                                              Delta SQNR of Eq. 7 is 10 log10 of the ratio of two NMSEs)
 *   [3 + i]  number of elements whose code has magnitude level i, i = 0..7 -> p_i of Eq. 6 (effective bucket ratio)
 *   [11 + i] sum over those elements of (level_i - |x'| / s) in grid units -> Sec. 3.1's E[rho_G(t) - t] per bin
 *            (elements of zero-scale blocks are counted in [3 + i] but add nothing here)
 * The three sums of squares are FP32 inside a 16-block and FP64 across blocks (relative error below 1e-6), the
 * per-level error sums FP32 per thread and FP64 across threads; everything is added in a fixed order: the result is
 * reproducible.  workspace >= ufp4_diagnose_workspace_bytes(rows, cols) bytes of device memory.
 * Not on the training hot path: a measurement pass (one read of x, codes and scales).
 */
size_t ufp4_diagnose_workspace_bytes(int64_t rows, int64_t cols);
int ufp4_diagnose(const void *x, int64_t rows, int64_t cols, int64_t ld, const ufp4_qtensor *q_row, int rht_block,
                  uint64_t seed_rht, double *dev_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The quantities of Sec. 3 from the 19 sums of ufp4_diagnose (both arrays in HOST memory; plain host arithmetic, no
 * launch).  out (11 doubles):
 *   [0] alpha = sum xq x' / sum x'^2, the operand projection of Eq. 3
 *   [1] NMSE  = sum (xq - x')^2 / sum x'^2 (Sec. 3.3; Eq. 7's Delta SQNR is 10 log10 of the ratio of two of these)
 *   [2] B_eff = exp(-sum_i p_i ln(p_i + 1e-12)) / 8, Eq. 6 over the K = 8 magnitude levels (zero included)
 *   [3 + i] mean of (level_i - |x'| / s) over the elements on level i, Sec. 3.1's per-bin bias; NaN for an unused level
 * [0] and [1] are NaN for an all-zero tensor.  Returns UFP4_ERR_NULL for a null pointer.
 */
int ufp4_diagnose_ratios(const double *sums, double *out);

/*
 * ufp4_gemm without any device allocation by anyone (the paper has no counterpart to this entry point; it exists for
 * the library's users).  Some callers cannot provide the workspace ufp4_gemm's tensor-core path needs: a process
 * whose device memory has all been handed to a framework's pool, or code running at a point where calling cudaMalloc
 * is not allowed or would stall the whole device (it synchronises the device).  For them this call computes the same
 * C[m][n] = sum_k a[m][k] * b[n][k] as ufp4_gemm(..., UFP4_PATH_TENSOR, ...) with its scratch (the decoded 8-bit
 * operands and the per-row reference scales) in a fixed device array that is part of the library image.
 *   - Limit: the scratch the shapes need, ufp4_gemm_workspace_bytes(A, B, UFP4_PATH_TENSOR), must not exceed
 *     ufp4_gemm_noalloc_max_scratch_bytes() (16 MiB: e.g. A of 2048 and B of 2040 rows at K = 4096 fit, 2048 and 2048 rows
 *     do not, because the reference scales and the tile list share the array); beyond it the call
 *     returns UFP4_ERR_WORKSPACE and launches nothing.  Every GPU that loads the library holds those 16 MiB until exit.
 *   - Both operands must use UFP4_SCALE_POW2 (else UFP4_ERR_UNSUPPORTED).  C as in ufp4_gemm.
 *   - The first call on each device looks up the array's device address (that device must be current); make that first
 *     call outside any stream capture.  The call itself calls no cudaMalloc / cudaFree and no allocating library.
 *   - All calls share the one array and it keeps the last call's contents; each call rewrites every byte it reads, so
 *     nothing needs clearing, but two calls that overlap on the GPU (different streams, or different host threads)
 *     race on it: serialise them on one stream.
 */
int ufp4_gemm_noalloc(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16,
                      int32_t *dev_status, void *stream);

/*
 * Test hook for the failure path of the tensor-core kernels (TENSOR, SPLIT and FP16 paths; the paper has no
 * counterpart).  Every wait of those kernels on a copy or on the tensor cores is bounded: after poll_limit polls (0 =
 * the default, 2^24) the waiting role raises a flag in shared memory, the other roles see it in their own waits, the
 * kernel returns normally (tensor memory released, cluster barriers met) and UFP4_DEV_WAIT_TIMEOUT is OR-ed into
 * *dev_status.  With skip_loads = 1 the launches that follow issue no operand loads at all, so the first wait of the
 * MMA-issuing thread runs out by construction, with no copy and no MMA in flight: that is how the tests exercise the
 * path without faulting or hanging anything.  Process-wide until reset with (0, 0); C is left undefined by such a call.
 * Returns UFP4_ERR_ENUM unless skip_loads is 0 or 1.
 */
int ufp4_debug_wait_injection(uint32_t poll_limit, int skip_loads);

/*
 * Measurement aid (the paper has no counterpart; not on the hot path): cycles a scheduler of this GPU needs per group of
 * warp instructions, for the instruction kinds the quantizer is made of: host_cycles (HOST, 8 doubles) receives
 *   [0] add.rn.f32x2   [1] two add.rn.f32   [2] lop3   [3] mad.lo.u32   [4] f32x2 add + lop3   [5] f32x2 add + mad
 *   [6] f32x2 add + two lop3   [7] two add.rn.f32 + lop3
 * measured with one CTA of 1024 threads per SM on independent chains.  dev_scratch: device memory, 256-byte aligned, at
 * least (SM count x 4096 + 256) bytes.  Synchronizes the stream.
 */
int ufp4_probe_issue_rates(void *dev_scratch, size_t scratch_bytes, double *host_cycles, void *stream);

/*
 * Measurement aid (not on the hot path): cycles one SM needs to decode one pipeline stage of packed nibbles in shared
 * memory (a CTA pair's share of a 256 x 256 x 128 step: 256 rows x 128 elements = 32768 elements) into the swizzled
 * E5M2 operand tiles of the folded tensor-core path, with that path's decode arithmetic, when the stage is shared by
 *   [0] 128   [1] 256   [2] 512   [3] 1024
 * threads of one CTA per SM (host_cycles: HOST, 4 doubles).  The product kernel consumes such a stage every ~890 cycles;
 * this is the measurement behind keeping the decode a pass of its own.  dev_scratch as for ufp4_probe_issue_rates.
 * Synchronizes the stream.
 */
int ufp4_probe_decode_rate(void *dev_scratch, size_t scratch_bytes, double *host_cycles, void *stream);

/* Size in bytes of the fixed scratch array behind ufp4_gemm_noalloc. */
size_t ufp4_gemm_noalloc_max_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* UFP4_H_ */
