/*
 * UFP4 oracle — TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, single-threaded CPU statement of what the UFP4 hot path computes, written from the paper's
 * definitions so that a reader can check it against them by eye.  It shares no code, header, table or constant
 * generator with the CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * What each function follows:
 *   orc_hadamard_matrix   Sec. 2.2, the Sylvester recursion H_2n = 1/sqrt(2) [[H,H],[H,-H]], H_1 = [1]
 *   orc_rht16_f32         Sec. 2.2, H'_16 = S_16 H_16 applied to a row vector (signs first, then Hadamard), FP32
 *   orc_rht_f32           the same for the RHT block sizes 32 / 64 / 128 of App. B's search space
 *   orc_quantize          Sec. 2.1, s_B = max|x_j| / g_max, q_i = rho_G(x_i / s_B); Sec. 4 / Table 1 (1x16 blocks,
 *                         FP32 single-level scale, RHT block 16); Sec. 2.2 last paragraph (blocks and RHT run along
 *                         the reduction dimension, so a tensor has a "row" and a "col" variant)
 *   orc_round_rtne        Sec. 2.1 (nearest level, deterministic tie-break) and Eq. 1 (bin edges are midpoints)
 *   orc_round_sr          Sec. 2.1, Pr[q = g_b] = (x/s - g_a) / (g_b - g_a)
 *   orc_dequantize        Sec. 2.1, "Q_G(T) ... denotes the dequantized numerical tensor"
 *   orc_gemm_f64          Sec. 2.2, Y^ = Q_G(X H') Q_G(W H')^T as a plain FP64 triple loop
 *   orc_bin_bias          Sec. 3.1, b_G = E[rho_G(t) - t] restricted to the bin of each level
 *   orc_diagnose          Sec. 3.2 Eq. 3 (operand projection alpha), Sec. 3.3 (NMSE, Eq. 7) and Eq. 6 (level counts
 *                         behind the effective bucket ratio, orc_b_eff), plus the per-bin bias sums again
 *
 * Readings taken where the paper is silent (each is restated in the repository's design notes):
 *   - E1M2 levels are {0,...,7}/4 (g_max 1.75); INT4 is the symmetric integer grid {-7..7} (g_max 7); both are the
 *     same uniform grid, differing only in nibble encoding and a factor 4 in the stored scale.
 *   - x/s is evaluated as x * inv with inv = RN(g_max / amax) (one FP32 division per block), s = RN(amax / g_max).
 *   - RTNE ties go to the level with the even code.
 *   - One 16-entry sign vector per seed, shared by every block; bit i of the low 16 bits of word 0 of
 *     Philox4x32-10(counter (0,0,0,0x52485400), key = seed) set means eps_i = -1.
 *   - Butterfly stages run h = 1, 2, 4, 8 in FP32, then one exact multiply by 1/4.
 *   - SR draws one Philox4x32-10 block per 16-element quant block: counter (lo32(b), hi32(b), variant, 0x53520000),
 *     key = seed; the 16 little-endian bytes of the four output words are the elements' random bytes r;
 *     round up iff p * 256 > r + 0.5, p being the exact fractional position between the two neighbouring levels.
 *   - A block with amax == 0 or amax < 2^-100 is stored as scale 0, codes 0.  Zero is always nibble 0x0.
 *   - RHT blocks of 32 / 64 / 128 (App. B): sign i of the block is bit i of all 128 bits of that Philox output;
 *     butterfly stages h = 1, 2, ..., n/2 in FP32, then one multiplication by the FP32 value nearest 1/sqrt(n); the
 *     quant blocks stay 16 wide and are taken from the rotated chunk.
 *   - 1x32 blocks with an E8M0 scale (Sec. 2.1's footnote on MXFP4): amax over the 32 rotated elements, scale = the
 *     next power of two >= amax / g_max (E8M0 holds exactly the powers of two), shared by the two 16-element halves;
 *     rotation, rounding, SR draws and block indices stay per 16 elements.
 *   - Range-restricted E2M1 (Sec. 5.4, `max_fpx` of App. B): g_max = max_fpx in the scale, and rho_G rounds onto the
 *     E2M1 levels not above max_fpx (max_fpx = 2 keeps {0, 0.5, 1, 1.5, 2}); encoding and dequantization are E2M1's.
 *
 * Parity pins: see tests/test_oracle_pins.py.  The E4M3-with-tensor-scale mode has no counterpart in the paper and
 * is pinned only by brute force: "parity unpinned" by the paper for that mode.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* E2M1_MAX4 / E2M1_MAX2: the E2M1 codebook with the magnitudes above 4 / above 2 left unused (the range-restricted
 * E2M1 of Sec. 5.4 and App. B's `max_fpx`): g_max = 4 / 2, same nibble encoding as E2M1. */
enum { ORC_GRID_INT4 = 0, ORC_GRID_E1M2 = 1, ORC_GRID_E2M1 = 2, ORC_GRID_E2M1_MAX4 = 3, ORC_GRID_E2M1_MAX2 = 4 };
enum { ORC_ROUND_RTNE = 0, ORC_ROUND_SR = 1 };
/* E8M0_B32: one power-of-two scale shared by 32 consecutive elements (the 1x32 blocks with an E8M0 scale that Sec. 2.1's
 * footnote attributes to MXFP4), stored as that FP32 power of two for both 16-element halves. */
enum { ORC_SCALE_FP32 = 0, ORC_SCALE_POW2 = 1, ORC_SCALE_E4M3_TENSOR = 2, ORC_SCALE_E8M0_B32 = 3 };
enum { ORC_AXIS_ROW = 0, ORC_AXIS_COL = 1 };

/* ---------------------------------------------------------------- codebooks (Sec. 2.1, Sec. 3.1) */

static const double LEVELS_INT4[8] = {0, 1, 2, 3, 4, 5, 6, 7};
static const double LEVELS_E1M2[8] = {0, 0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75};
static const double LEVELS_E2M1[8] = {0, 0.5, 1, 1.5, 2, 3, 4, 6};

static const double *levels_of(int grid) {
    switch (grid) {
        case ORC_GRID_INT4: return LEVELS_INT4;
        case ORC_GRID_E1M2: return LEVELS_E1M2;
        default: return LEVELS_E2M1;
    }
}

/* Number of non-negative levels in use: a range-restricted grid keeps the levels up to its g_max. */
int orc_num_levels(int grid) { return grid == ORC_GRID_E2M1_MAX4 ? 7 : (grid == ORC_GRID_E2M1_MAX2 ? 5 : 8); }

/* Non-negative level i (0..7) of a grid's codebook; exported so tests can read the codebook. */
double orc_level(int grid, int i) { return levels_of(grid)[i & 7]; }

double orc_gmax(int grid) { return levels_of(grid)[orc_num_levels(grid) - 1]; }

/* ---------------------------------------------------------------- Philox4x32-10 (Salmon et al., SC'11) */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 16 RHT signs of a seed: bit i set means eps_i = -1. */
uint32_t orc_rht_sign_mask(uint64_t seed) {
    uint32_t ctr[4] = {0, 0, 0, 0x52485400u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[0] & 0xFFFFu;
}

/* The sign bits of RHT blocks up to 128 wide: bit i of the 128-bit output of the same Philox call (word i / 32,
 * bit i % 32) set means eps_i = -1; the 16-point mask above is its first 16 bits. */
void orc_rht_signs(uint64_t seed, uint32_t out[4]) {
    uint32_t ctr[4] = {0, 0, 0, 0x52485400u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    orc_philox4x32_10(ctr, key, out);
}

/* The 16 random bytes of quant block b of a variant (0 = row, 1 = col). */
void orc_sr_bytes(uint64_t seed_sr, uint64_t block_index, uint32_t variant, uint8_t r[16]) {
    uint32_t ctr[4] = {(uint32_t)block_index, (uint32_t)(block_index >> 32), variant, 0x53520000u};
    uint32_t key[2] = {(uint32_t)seed_sr, (uint32_t)(seed_sr >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    for (int w = 0; w < 4; ++w)
        for (int b = 0; b < 4; ++b) r[4 * w + b] = (uint8_t)(out[w] >> (8 * b));
}

/* ---------------------------------------------------------------- Hadamard / RHT (Sec. 2.2) */

/* H_n by the Sylvester recursion, row-major n x n, n a power of two.  The recursion is run on the +-1 pattern and
 * the n factors 1/sqrt(2) are applied once as 1/sqrt(n), so that H_16 has entries exactly +-1/4. */
void orc_hadamard_matrix(int n, double *H) {
    H[0] = 1.0;
    for (int m = 1; m < n; m *= 2)
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) {
                double h = H[i * n + j];
                H[i * n + (j + m)] = h;
                H[(i + m) * n + j] = h;
                H[(i + m) * n + (j + m)] = -h;
            }
    double c = 1.0 / sqrt((double)n);
    for (int i = 0; i < n * n; ++i) H[i] *= c;
}

/* v <- (v o eps) H_16 in FP32: signs, then butterfly stages h = 1,2,4,8, then the exact factor 1/4. */
void orc_rht16_f32(float v[16], uint32_t sign_mask) {
    for (int i = 0; i < 16; ++i)
        if ((sign_mask >> i) & 1u) v[i] = -v[i];
    for (int h = 1; h < 16; h *= 2)
        for (int i = 0; i < 16; ++i)
            if ((i & h) == 0) {
                float a = v[i], b = v[i + h];
                v[i] = a + b;
                v[i + h] = a - b;
            }
    for (int i = 0; i < 16; ++i) v[i] = 0.25f * v[i];
}

/* v <- (v o eps) H_n in FP32 for n = 32, 64, 128 (App. B lists these block sizes beside the selected 16): signs, the
 * butterfly stages h = 1, 2, ..., n/2 in that order, then one multiplication by the FP32 value nearest to 1/sqrt(n)
 * (exact for n = 64). */
void orc_rht_f32(float *v, int n, const uint32_t signs[4]) {
    for (int i = 0; i < n; ++i)
        if ((signs[i >> 5] >> (i & 31)) & 1u) v[i] = -v[i];
    for (int h = 1; h < n; h *= 2)
        for (int i = 0; i < n; ++i)
            if ((i & h) == 0) {
                float a = v[i], b = v[i + h];
                v[i] = a + b;
                v[i + h] = a - b;
            }
    const float c = (float)(1.0 / sqrt((double)n));
    for (int i = 0; i < n; ++i) v[i] = c * v[i];
}

/* ---------------------------------------------------------------- rounding rules (Sec. 2.1) */

/* RTNE of a normalised magnitude a >= 0 onto a grid: index of the nearest level, ties to the even index,
 * values above the top level saturate to it. */
int orc_round_rtne(double a, int grid) {
    const double *L = levels_of(grid);
    const int n = orc_num_levels(grid);
    int best = 0;
    double best_d = fabs(a - L[0]);
    for (int i = 1; i < n; ++i) {
        double d = fabs(a - L[i]);
        if (d < best_d || (d == best_d && (i % 2 == 0))) {
            best = i;
            best_d = d;
        }
    }
    return best;
}

/* SR of a normalised magnitude a >= 0 with random byte r: between neighbours g_a <= a < g_b the upper one is
 * taken iff p * 256 > r + 0.5, p = (a - g_a) / (g_b - g_a); at or above the top level the top level is taken. */
int orc_round_sr(double a, int grid, int r) {
    const double *L = levels_of(grid);
    const int n = orc_num_levels(grid);
    if (a >= L[n - 1]) return n - 1;
    int lo = 0;
    for (int i = 1; i < n; ++i)
        if (L[i] <= a) lo = i;
    double p = (a - L[lo]) / (L[lo + 1] - L[lo]);
    return (p * 256.0 > (double)r + 0.5) ? lo + 1 : lo;
}

static uint8_t encode_nibble(int grid, int negative, int level_index) {
    if (level_index == 0) return 0;
    if (grid == ORC_GRID_INT4) {
        int q = negative ? -level_index : level_index;
        return (uint8_t)(q & 0xF);
    }
    return (uint8_t)((negative ? 8 : 0) | level_index);
}

/* Value of a 4-bit code in grid units. */
double orc_nibble_value(int grid, int nibble) {
    nibble &= 0xF;
    if (grid == ORC_GRID_INT4) {
        int q = (nibble & 8) ? nibble - 16 : nibble;
        return (double)q;
    }
    double mag = levels_of(grid)[nibble & 7];
    return (nibble & 8) ? -mag : mag;
}

/* ---------------------------------------------------------------- E4M3 helpers (two-level scale mode only) */

double orc_e4m3_value(int byte) {
    int e = (byte >> 3) & 0xF, m = byte & 7;
    double v = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (byte & 0x80) ? -v : v;
}

/* Nearest non-negative finite E4M3 value (ties to even code), saturating at 448 (code 0x7E). */
int orc_e4m3_encode(float u) {
    if (!(u > 0.0f)) return 0;
    int best = 0;
    double best_d = fabs((double)u - 0.0);
    for (int c = 1; c <= 0x7E; ++c) {
        double d = fabs((double)u - orc_e4m3_value(c));
        if (d < best_d || (d == best_d && (c % 2 == 0))) {
            best = c;
            best_d = d;
        }
    }
    return best;
}

/* ---------------------------------------------------------------- the blockwise quantizer (Sec. 2.1, Sec. 4) */

typedef struct {
    int grid, rounding, scale_fmt, rht_block;
    uint32_t sign_mask;
    uint64_t seed_sr;
    float tensor_scale;
} orc_params;

/* Effective FP32 scale of a stored block scale. */
static float effective_scale(int scale_fmt, float stored_f32, uint8_t stored_byte, float tensor_scale) {
    if (scale_fmt == ORC_SCALE_E4M3_TENSOR) return tensor_scale * (float)orc_e4m3_value(stored_byte);
    return stored_f32;
}

/* One 16-element block.  x: the block's values (BF16 widened to FP32).  Outputs: 16 nibbles, the stored scale
 * (FP32 and, for the E4M3 mode, the byte), and optionally the normalised values y. */
static void quantize_block(const float x[16], const orc_params *p, uint64_t block_index, uint32_t variant,
                           uint8_t nib[16], float *scale_f32, uint8_t *scale_byte, float *y_out, float amax_shared) {
    float v[16];
    memcpy(v, x, sizeof(v));
    if (p->rht_block == 16) orc_rht16_f32(v, p->sign_mask);

    float amax = 0.0f;
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
    if (amax_shared >= 0.0f) amax = amax_shared;      /* the scale block is wider than this block: its amax is given */

    const float g = (float)orc_gmax(p->grid);
    float s = 0.0f, inv = 0.0f;
    uint8_t sb = 0;
    int zero_block = (amax == 0.0f) || (amax < 0x1p-100f);
    if (!zero_block) {
        if (p->scale_fmt == ORC_SCALE_FP32) {
            s = amax / g;
            inv = g / amax;
        } else if (p->scale_fmt == ORC_SCALE_POW2 || p->scale_fmt == ORC_SCALE_E8M0_B32) {
            float z = amax / g;
            int e;
            float m = frexpf(z, &e); /* z = m * 2^e, m in [0.5, 1) */
            s = (m == 0.5f) ? z : ldexpf(1.0f, e);
            inv = 1.0f / s;
        } else {
            float z = amax / g;
            float u = z / p->tensor_scale;
            sb = (uint8_t)orc_e4m3_encode(u);
            s = effective_scale(ORC_SCALE_E4M3_TENSOR, 0.0f, sb, p->tensor_scale);
            if (sb == 0 || s == 0.0f) zero_block = 1;
            else inv = 1.0f / s;
        }
    }
    if (zero_block) {
        for (int i = 0; i < 16; ++i) {
            nib[i] = 0;
            if (y_out) y_out[i] = 0.0f;
        }
        *scale_f32 = 0.0f;
        *scale_byte = 0;
        return;
    }

    uint8_t r[16];
    if (p->rounding == ORC_ROUND_SR) orc_sr_bytes(p->seed_sr, block_index, variant, r);

    for (int i = 0; i < 16; ++i) {
        float y = v[i] * inv;
        if (y_out) y_out[i] = y;
        double a = fabs((double)y);
        int idx = (p->rounding == ORC_ROUND_SR) ? orc_round_sr(a, p->grid, r[i]) : orc_round_rtne(a, p->grid);
        nib[i] = encode_nibble(p->grid, y < 0.0f, idx);
    }
    *scale_f32 = s;
    *scale_byte = sb;
}

/*
 * Quantize a BF16 matrix x[rows][cols] (row pitch ld elements) along one axis.
 *   axis ROW: blocks are 16 consecutive elements of a row; outputs codes[rows][cols/2], scales[rows][cols/16].
 *   axis COL: blocks are 16 consecutive elements of a column; outputs are stored transposed,
 *             codes[cols][rows/2], scales[cols][rows/16].
 * Element 2j of an output row sits in bits 3:0 of byte j, element 2j+1 in bits 7:4.
 * scales is float[] for FP32 / POW2 and uint8_t[] for E4M3_TENSOR.  y_out (optional) receives the normalised
 * pre-rounding values in the output's [R][k] order.  Returns 0, or -1 on a bad shape / argument.
 */
int orc_quantize_window(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, int axis, int rht_block, int grid,
                        int rounding, int scale_fmt, uint64_t seed_rht, uint64_t seed_sr, float tensor_scale,
                        uint8_t *codes, void *scales, float *y_out, int64_t out_row0, int64_t kb0, int64_t full_nkb);

int orc_quantize(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, int axis, int rht_block, int grid,
                 int rounding, int scale_fmt, uint64_t seed_rht, uint64_t seed_sr, float tensor_scale,
                 uint8_t *codes, void *scales, float *y_out) {
    int64_t K = (axis == ORC_AXIS_ROW) ? cols : rows;
    return orc_quantize_window(x, rows, cols, ld, axis, rht_block, grid, rounding, scale_fmt, seed_rht, seed_sr,
                               tensor_scale, codes, scales, y_out, 0, 0, K / 16);
}

/*
 * The same quantizer on a window of a larger tensor: x[rows][cols] is the part of the full tensor whose first output
 * row (row for axis ROW, column for axis COL) is out_row0 and whose first 16-element block along the reduction axis is
 * kb0, the full tensor having full_nkb blocks along that axis.  Only the SR draws depend on where a block sits in the
 * full tensor (Philox counter = index of the block in the full variant's scales array); everything else is the
 * window's own.  kb0 must be a multiple of the RHT block (and of 2 for 1x32 scale blocks) counted in 16-blocks.
 */
int orc_quantize_window(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, int axis, int rht_block, int grid,
                        int rounding, int scale_fmt, uint64_t seed_rht, uint64_t seed_sr, float tensor_scale,
                        uint8_t *codes, void *scales, float *y_out, int64_t out_row0, int64_t kb0, int64_t full_nkb) {
    if (!x || !codes || !scales) return -1;
    if (out_row0 < 0 || kb0 < 0 || full_nkb < 1) return -1;
    if (rht_block != 0 && rht_block != 16 && rht_block != 32 && rht_block != 64 && rht_block != 128) return -1;
    if (grid < 0 || grid > 4 || rounding < 0 || rounding > 1 || scale_fmt < 0 || scale_fmt > 3) return -1;
    int64_t R = (axis == ORC_AXIS_ROW) ? rows : cols; /* output rows   */
    int64_t K = (axis == ORC_AXIS_ROW) ? cols : rows; /* reduction dim */
    if (K % 16 != 0 || R <= 0 || K <= 0) return -1;
    if (rht_block > 16 && K % rht_block != 0) return -1;
    if (scale_fmt == ORC_SCALE_E8M0_B32 && K % 32 != 0) return -1;

    /* RHT blocks wider than the quant block: the whole rht_block-wide chunk is rotated first, then its 16-element
     * blocks are quantized without further rotation. */
    const int wide = rht_block > 16;
    uint32_t signs[4];
    orc_rht_signs(seed_rht, signs);
    orc_params p = {grid, rounding, scale_fmt, wide ? 0 : rht_block, orc_rht_sign_mask(seed_rht), seed_sr, tensor_scale};
    int64_t nkb = K / 16;
    float chunk[128];
    for (int64_t o = 0; o < R; ++o)
        for (int64_t kb = 0; kb < nkb; ++kb) {
            float xb[16];
            if (wide && (kb * 16) % rht_block == 0) {
                for (int i = 0; i < rht_block; ++i) {
                    int64_t k = kb * 16 + i;
                    uint16_t h = (axis == ORC_AXIS_ROW) ? x[o * ld + k] : x[k * ld + o];
                    uint32_t u = (uint32_t)h << 16;
                    memcpy(&chunk[i], &u, 4);
                }
                orc_rht_f32(chunk, rht_block, signs);
            }
            for (int i = 0; i < 16; ++i) {
                int64_t k = kb * 16 + i;
                if (wide) {
                    xb[i] = chunk[k % rht_block];
                    continue;
                }
                uint16_t h = (axis == ORC_AXIS_ROW) ? x[o * ld + k] : x[k * ld + o];
                uint32_t u = (uint32_t)h << 16;
                memcpy(&xb[i], &u, 4);
            }
            /* 1x32 scale blocks: amax over this 16-element block and its neighbour (kb ^ 1), both after rotation */
            float amax_shared = -1.0f;
            if (scale_fmt == ORC_SCALE_E8M0_B32) {
                float nb[16];
                int64_t kn = kb ^ 1;
                for (int i = 0; i < 16; ++i) {
                    int64_t k = kn * 16 + i;
                    if (wide) {
                        nb[i] = chunk[k % rht_block];       /* the neighbour lies in the same rotated chunk */
                        continue;
                    }
                    uint16_t h = (axis == ORC_AXIS_ROW) ? x[o * ld + k] : x[k * ld + o];
                    uint32_t u = (uint32_t)h << 16;
                    memcpy(&nb[i], &u, 4);
                }
                float own[16];
                memcpy(own, xb, sizeof(own));
                if (p.rht_block == 16) {
                    orc_rht16_f32(nb, p.sign_mask);
                    orc_rht16_f32(own, p.sign_mask);
                }
                amax_shared = 0.0f;
                for (int i = 0; i < 16; ++i) amax_shared = fmaxf(amax_shared, fmaxf(fabsf(nb[i]), fabsf(own[i])));
            }
            uint8_t nib[16];
            float sf;
            uint8_t sbyte;
            uint64_t b = (uint64_t)((out_row0 + o) * full_nkb + (kb0 + kb));
            quantize_block(xb, &p, b, (uint32_t)axis, nib, &sf, &sbyte, y_out ? y_out + (o * K + kb * 16) : NULL,
                           amax_shared);
            for (int j = 0; j < 8; ++j) codes[o * (K / 2) + kb * 8 + j] = (uint8_t)(nib[2 * j] | (nib[2 * j + 1] << 4));
            if (scale_fmt == ORC_SCALE_E4M3_TENSOR) ((uint8_t *)scales)[o * nkb + kb] = sbyte;
            else ((float *)scales)[o * nkb + kb] = sf;
        }
    return 0;
}

/* Dequantize rows [r0, r1) of a quantized tensor codes[R][K/2], scales[R][K/16] into out[(r1-r0)][K] (FP64). */
void orc_dequantize(const uint8_t *codes, const void *scales, int64_t K, int grid, int scale_fmt,
                    float tensor_scale, int64_t r0, int64_t r1, double *out) {
    int64_t nkb = K / 16;
    for (int64_t r = r0; r < r1; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int nibble = (k & 1) ? (byte >> 4) : (byte & 0xF);
            float s = (scale_fmt == ORC_SCALE_E4M3_TENSOR)
                          ? effective_scale(scale_fmt, 0.0f, ((const uint8_t *)scales)[r * nkb + k / 16], tensor_scale)
                          : ((const float *)scales)[r * nkb + k / 16];
            out[(r - r0) * K + k] = orc_nibble_value(grid, nibble) * (double)s;
        }
}

/* ---------------------------------------------------------------- GEMM on dequantized values (Sec. 2.2) */

/* C[m][n] = sum_k A[m][k] B[n][k] and S[m][n] = sum_k |A[m][k] B[n][k]|, FP64, plain triple loop. */
void orc_gemm_f64(const double *A, const double *B, int64_t M, int64_t N, int64_t K, double *C, double *S) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double c = 0.0, s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double pr = A[m * K + k] * B[n * K + k];
                c += pr;
                s += fabs(pr);
            }
            C[m * N + n] = c;
            if (S) S[m * N + n] = s;
        }
}

/* The same sum for a list of (m, n) pairs, over the reduction range [k0, k1), straight from the quantized tensors
 * (for problem sizes whose full product is too slow to form on a CPU). */
void orc_gemm_sampled(const uint8_t *a_codes, const void *a_scales, int a_grid, int a_scale_fmt, float a_ts,
                      const uint8_t *b_codes, const void *b_scales, int b_grid, int b_scale_fmt, float b_ts,
                      int64_t K, int64_t k0, int64_t k1, int64_t n_samples, const int64_t *im, const int64_t *in,
                      double *c_out, double *s_out) {
    double *ra = (double *)malloc(sizeof(double) * (size_t)K);
    double *rb = (double *)malloc(sizeof(double) * (size_t)K);
    for (int64_t t = 0; t < n_samples; ++t) {
        orc_dequantize(a_codes, a_scales, K, a_grid, a_scale_fmt, a_ts, im[t], im[t] + 1, ra);
        orc_dequantize(b_codes, b_scales, K, b_grid, b_scale_fmt, b_ts, in[t], in[t] + 1, rb);
        double c = 0.0, s = 0.0;
        for (int64_t k = k0; k < k1; ++k) {
            double pr = ra[k] * rb[k];
            c += pr;
            s += fabs(pr);
        }
        c_out[t] = c;
        if (s_out) s_out[t] = s;
    }
    free(ra);
    free(rb);
}

/* ---------------------------------------------------------------- Shrinkage-Bias measurement (Sec. 3.1) */

/* For each non-negative level i: count of elements whose code has magnitude level i, and the sum of
 * (level - |y|) over them, in grid units.  mean = sum / count is E[rho_G(t) - t | t in bin i]. */
void orc_bin_bias(const float *y, const uint8_t *codes, int64_t n, int grid, int64_t count[8], double sum[8]) {
    for (int i = 0; i < 8; ++i) {
        count[i] = 0;
        sum[i] = 0.0;
    }
    for (int64_t e = 0; e < n; ++e) {
        uint8_t byte = codes[e / 2];
        int nibble = (e & 1) ? (byte >> 4) : (byte & 0xF);
        double mag = fabs(orc_nibble_value(grid, nibble));
        int idx = 0;
        const double *L = levels_of(grid);
        for (int i = 0; i < 8; ++i)
            if (L[i] == mag) idx = i;
        count[idx] += 1;
        sum[idx] += mag - fabs((double)y[e]);
    }
}

/* ---------------------------------------------------------------- tensor diagnostics (Sec. 3.2 Eq. 3, Sec. 3.3 Eq. 6-7) */

/* For the row variant (codes, FP32 scales) of the BF16 matrix x [rows][cols], with x' = x H'_n per n-element chunk
 * (rht_block n = 16, 32, 64 or 128; FP32 butterflies as in the quantizer) or x' = x (rht_block == 0) and
 * xq = level * scale:
 *   out[0] = sum x'^2, out[1] = sum (xq - x')^2, out[2] = sum xq x'            (Eq. 3: alpha = out[2] / out[0];
 *                                                                               Sec. 3.3: NMSE = out[1] / out[0])
 *   out[3 + i]  = number of elements whose code has magnitude level i           (Eq. 6: p_i = out[3 + i] / n)
 *   out[11 + i] = sum over those elements of (level_i - |x'| / s), grid units   (Sec. 3.1 per-bin bias; a zero-scale
 *                                                                               block contributes 0 to it)
 * All sums in FP64, elements in storage order. */
void orc_diagnose(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, const uint8_t *codes, int64_t ld_codes,
                  const float *scales, int64_t ld_scales, int grid, int rht_block, uint64_t seed_rht, double out[19]) {
    const double *L = levels_of(grid);
    const uint32_t sign_mask = orc_rht_sign_mask(seed_rht);
    uint32_t signs[4];
    orc_rht_signs(seed_rht, signs);
    float chunk[128];
    for (int i = 0; i < 19; ++i) out[i] = 0.0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < cols / 16; ++b) {
            float v[16];
            if (rht_block > 16) {
                if ((16 * b) % rht_block == 0) {        /* a new chunk: rotate all of it */
                    for (int i = 0; i < rht_block; ++i) {
                        uint32_t bits = (uint32_t)x[r * ld + 16 * b + i] << 16;
                        memcpy(&chunk[i], &bits, 4);
                    }
                    orc_rht_f32(chunk, rht_block, signs);
                }
                memcpy(v, chunk + (16 * b) % rht_block, sizeof(v));
            } else {
                for (int i = 0; i < 16; ++i) {
                    uint32_t bits = (uint32_t)x[r * ld + 16 * b + i] << 16;
                    memcpy(&v[i], &bits, 4);
                }
                if (rht_block == 16) orc_rht16_f32(v, sign_mask);
            }
            const double s = (double)scales[r * ld_scales + b];
            for (int i = 0; i < 16; ++i) {
                const int64_t e = 16 * b + i;
                const uint8_t byte = codes[r * ld_codes + e / 2];
                const int nibble = (e & 1) ? (byte >> 4) : (byte & 0xF);
                const double val = orc_nibble_value(grid, nibble);
                const double xp = (double)v[i], xq = val * s;
                out[0] += xp * xp;
                out[1] += (xq - xp) * (xq - xp);
                out[2] += xq * xp;
                int idx = 0;
                for (int k = 0; k < 8; ++k)
                    if (L[k] == fabs(val)) idx = k;
                out[3 + idx] += 1.0;
                if (s > 0.0) out[11 + idx] += fabs(val) - fabs(xp) / s;
            }
        }
}

/* Effective bucket ratio of Eq. 6 from the eight level counts: exp(-sum p_i log(p_i + eps)) / 8, natural log,
 * eps = 1e-12 (the paper leaves eps and the base open). */
double orc_b_eff(const double count[8]) {
    double n = 0.0, ent = 0.0;
    for (int i = 0; i < 8; ++i) n += count[i];
    if (n <= 0.0) return 0.0;
    for (int i = 0; i < 8; ++i) {
        double p = count[i] / n;
        ent -= p * log(p + 1e-12);
    }
    return exp(ent) / 8.0;
}
