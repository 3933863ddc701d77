/*
 * CPU oracle for the SLiM compressed linear layer.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain, fp64 statement of what the GPU library must
 * compute.  It is used by the tests, by the smoke check and by the timed CPU
 * baseline of the benchmark; the product path never links, imports or calls
 * it, and it shares no code, header, table or helper with the CUDA sources.
 *
 * What it states (paper sections in brackets):
 *   - the layer output  Y = X W  with the compressed weight plus low-rank
 *     adapters,  W ~ W^C + L R              [Sec. 2 "Model Compression", Eq. 1;
 *                                            Sec. 3.2 "SLiM-LoRA"]
 *   - W^C is a symmetric uniform 4-bit quantized matrix with one scale per
 *     tensor                                [Sec. 3.1, Eq. 2 and Eq. 5]
 *   - pruned to the 2:4 pattern (at most two kept values in every aligned
 *     group of four along the contraction axis)         [Sec. 1, Sec. 3.2]
 *   - the adapter product costs O(2 b r d^2) and is added to the sparse
 *     product                                [App. "Rank Analysis"]
 *
 * Layout convention (nn.Linear orientation, i.e. the transpose of the paper's
 * W in R^{d_in x d_out}):  Q[d_out][d_in] int4 codes, mask[d_out][d_in],
 * L[d_out][r] (= paper R^T), R[r][d_in] (= paper L^T), X[b][d_in], Y[b][d_out]:
 *     Y[m][n] = sum_k X[m][k] * s*Q[n][k]*mask[n][k]
 *             + sum_j ( sum_k X[m][k]*R[j][k] ) * L[n][j]
 *
 * The packed storage format is not given by the paper (it delegates storage
 * to a third-party kernel); the format below is this project's definition:
 *   vals[n][g]  (one byte per group g of four columns): low nibble = code at
 *               the lower kept position, high nibble = code at the upper one,
 *               two's complement;
 *   meta[n][g/2] (one nibble per group): bits 0-1 = lower kept position,
 *               bits 2-3 = upper kept position; even g in the low nibble.
 *   A group with fewer than two kept positions is completed with the lowest
 *   positions not already kept (their codes are stored as 0) and the pair is
 *   sorted ascending.  More than two kept positions is an error.
 *
 * Every function here is pinned by tests/test_oracle_pins.py against values
 * that do not come from this file (hand-computed bytes and sums, an
 * independent float64 matrix product, closed forms, invariants).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_BAD_MASK = 3, ORACLE_CODE_RANGE = 4 };

/* bfloat16 (upper half of an IEEE binary32) to double: exact. */
static double bf16_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Sign-extend a 4-bit two's-complement nibble. */
static int sext4(unsigned nib)
{
    nib &= 0xFu;
    return (nib & 0x8u) ? (int)nib - 16 : (int)nib;
}

/*
 * Pack int4 codes and a 2:4 mask into nibble values and 2-bit position
 * metadata [format defined in the header comment; 2:4 pattern: Sec. 1].
 * codes, mask: [d_out][d_in] row-major.  vals: [d_out][d_in/4].
 * meta: [d_out][d_in/8].  d_in must be a multiple of 8.
 * Returns ORACLE_OK, or the first error found; on error, *bad_row / *bad_group
 * (if non-NULL) identify the offending group.
 */
int oracle_pack(const int8_t *codes, const uint8_t *mask, int d_out, int d_in,
                uint8_t *vals, uint8_t *meta, int *bad_row, int *bad_group)
{
    if (!codes || !mask || !vals || !meta || d_out < 1 || d_in < 8 || d_in % 8 != 0)
        return ORACLE_BAD_ARG;
    const int groups = d_in / 4;
    memset(meta, 0, (size_t)d_out * (size_t)(d_in / 8));
    for (int n = 0; n < d_out; ++n) {
        for (int g = 0; g < groups; ++g) {
            const int8_t *c = codes + (size_t)n * d_in + 4 * g;
            const uint8_t *mk = mask + (size_t)n * d_in + 4 * g;
            int keep[4] = {0, 0, 0, 0};
            int kept = 0;
            for (int i = 0; i < 4; ++i)
                if (mk[i]) { keep[i] = 1; ++kept; }
            if (kept > 2) {
                if (bad_row) *bad_row = n;
                if (bad_group) *bad_group = g;
                return ORACLE_BAD_MASK;
            }
            /* complete the pair with the lowest positions not kept; those
               slots carry the value 0 */
            int real[4] = {keep[0], keep[1], keep[2], keep[3]};
            for (int i = 0; i < 4 && kept < 2; ++i)
                if (!keep[i]) { keep[i] = 1; ++kept; }
            int pos[2], np = 0;
            for (int i = 0; i < 4; ++i)
                if (keep[i]) pos[np++] = i;          /* ascending */
            int v[2];
            for (int e = 0; e < 2; ++e) {
                if (real[pos[e]]) {
                    int code = c[pos[e]];
                    if (code < -8 || code > 7) {
                        if (bad_row) *bad_row = n;
                        if (bad_group) *bad_group = g;
                        return ORACLE_CODE_RANGE;
                    }
                    v[e] = code;
                } else {
                    v[e] = 0;
                }
            }
            vals[(size_t)n * groups + g] =
                (uint8_t)(((unsigned)v[0] & 0xFu) | (((unsigned)v[1] & 0xFu) << 4));
            unsigned m = (unsigned)pos[0] | ((unsigned)pos[1] << 2);
            meta[(size_t)n * (d_in / 8) + (g >> 1)] |= (uint8_t)(m << (4 * (g & 1)));
        }
    }
    return ORACLE_OK;
}

/*
 * Inverse of oracle_pack: dense int8 codes (0 where nothing is stored) and a
 * mask holding 1 at the two stored positions of every group.
 */
int oracle_unpack(const uint8_t *vals, const uint8_t *meta, int d_out, int d_in,
                  int8_t *codes, uint8_t *mask)
{
    if (!vals || !meta || !codes || d_out < 1 || d_in < 8 || d_in % 8 != 0)
        return ORACLE_BAD_ARG;
    const int groups = d_in / 4;
    for (int n = 0; n < d_out; ++n) {
        for (int g = 0; g < groups; ++g) {
            unsigned vb = vals[(size_t)n * groups + g];
            unsigned mb = meta[(size_t)n * (d_in / 8) + (g >> 1)];
            unsigned m = (mb >> (4 * (g & 1))) & 0xFu;
            int p0 = (int)(m & 3u), p1 = (int)((m >> 2) & 3u);
            int8_t *c = codes + (size_t)n * d_in + 4 * g;
            c[0] = c[1] = c[2] = c[3] = 0;
            if (mask) {
                uint8_t *mk = mask + (size_t)n * d_in + 4 * g;
                mk[0] = mk[1] = mk[2] = mk[3] = 0;
                mk[p0] = 1;
                mk[p1] = 1;
            }
            c[p0] = (int8_t)sext4(vb & 0xFu);
            c[p1] = (int8_t)sext4(vb >> 4);   /* p0 == p1 cannot come from oracle_pack */
        }
    }
    return ORACLE_OK;
}

/*
 * Decode-tiled copy of a packed weight: the same nibbles and position indices as
 * (vals, meta), re-ordered so that a 32-lane group that multiplies a 16-row x
 * 32-column piece reads its share as consecutive 32-bit words.  Like the packed
 * format itself this layout is the project's own (the paper leaves storage to a
 * third-party kernel, Sec. 4 "Speedup"); nothing is computed, bytes only move.
 *
 * d_out % 16 == 0, d_in % 256 == 0.  The matrix is cut into tiles of 16 rows and
 * blocks of 256 columns; (tile, block) occupies 1536 bytes.  Tiles are taken in groups
 * of four: group g = tile / 4 starts at 4 g * (d_in/256) * 1536; inside a group the
 * blocks follow each other, and inside a block the group's four tiles: (tile, block) sits at
 *     (4 g * (d_in/256) + block * 4 + (tile - 4 g)) * 1536,
 * so the 64 rows x 256 columns a group holds of one block are 6144 contiguous bytes.
 * When d_out/16 is not a multiple of four the last group is completed with padding
 * pieces: value words 0 and every index nibble 4 (positions 0 and 1), i.e. rows of
 * stored zeros.
 * Inside a (tile, block) piece, a "step" j = 0..7 is 32
 * columns (8 groups of four), a "lane" is (g, t) = (lane / 4, lane % 4):
 *   value words, bytes [0, 1024):  word (j, lane) at (j / 4) * 512 + lane * 16 + (j % 4) * 4.
 *     It holds four value bytes B_i, i = 0..3, taken from row 16 tile + g + 8 (i % 2),
 *     group 8 j + 4 (i / 2) + t of the block: the low nibble of B_i sits at bits
 *     [4 i, 4 i + 3], the high nibble at bits [16 + 4 i, 16 + 4 i + 3].
 *   index words, bytes [1024, 1536):  word (lane, jj), jj = 0..3, at 1024 + lane * 16 + jj * 4,
 *     belongs to step j = 4 (t / 2) + jj.  Bits 0-15 are the index bytes of row
 *     16 tile + g for 16 of the step's 32 columns (the first 16 when t is even, the
 *     last 16 when t is odd), as a little-endian 16-bit number; bits 16-31 the same
 *     for row 16 tile + g + 8.
 * Words are stored little-endian.  out: ceil(d_out / 64) * 64 * d_in * 3 / 8 bytes.
 */
int oracle_repack_tiled(const uint8_t *vals, const uint8_t *meta, int d_out, int d_in, uint8_t *out)
{
    if (!vals || !meta || !out || d_out < 16 || d_in < 256 || d_out % 16 != 0 || d_in % 256 != 0)
        return ORACLE_BAD_ARG;
    const int nblk = d_in / 256, tiles = d_out / 16;
    const size_t vrow = (size_t)d_in / 4, mrow = (size_t)d_in / 8;
    const int tiles4 = (tiles + 3) / 4 * 4;
    for (int tile = tiles; tile < tiles4; ++tile)               /* padding pieces of the last group */
        for (int blk = 0; blk < nblk; ++blk) {
            uint8_t *base = out + ((size_t)(4 * (tile / 4)) * nblk + (size_t)blk * 4 + tile % 4) * 1536;
            memset(base, 0, 1024);
            memset(base + 1024, 0x44, 512);
        }
    for (int tile = 0; tile < tiles; ++tile) {
        const int g4 = 4 * (tile / 4);                          /* first tile of the group */
        for (int blk = 0; blk < nblk; ++blk) {
            uint8_t *base = out + ((size_t)g4 * nblk + (size_t)blk * 4 + (tile - g4)) * 1536;
            for (int j = 0; j < 8; ++j) {
                for (int lane = 0; lane < 32; ++lane) {
                    const int g = lane / 4, t = lane % 4;
                    uint32_t w = 0;
                    for (int i = 0; i < 4; ++i) {
                        const int row = 16 * tile + g + 8 * (i % 2);
                        const int group = 64 * blk + 8 * j + 4 * (i / 2) + t;
                        const uint32_t B = vals[(size_t)row * vrow + group];
                        w |= (B & 0xFu) << (4 * i);
                        w |= (B >> 4) << (16 + 4 * i);
                    }
                    uint8_t *dst = base + (j / 4) * 512 + lane * 16 + (j % 4) * 4;
                    dst[0] = (uint8_t)w; dst[1] = (uint8_t)(w >> 8); dst[2] = (uint8_t)(w >> 16); dst[3] = (uint8_t)(w >> 24);
                }
            }
            for (int lane = 0; lane < 32; ++lane) {
                const int g = lane / 4, t = lane % 4;
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * (t / 2) + jj;
                    uint8_t *dst = base + 1024 + lane * 16 + jj * 4;
                    for (int up = 0; up < 2; ++up) {
                        const int row = 16 * tile + g + 8 * up;
                        const uint8_t *mb = meta + (size_t)row * mrow + 32 * blk + 4 * j + 2 * (t % 2);
                        dst[2 * up] = mb[0];
                        dst[2 * up + 1] = mb[1];
                    }
                }
            }
        }
    }
    return ORACLE_OK;
}

/*
 * Factored forward  Y = X (s Q)^T + (X R^T) L^T  in fp64, dense loops over the
 * whole contraction axis (the zeros of the 2:4 pattern are multiplied, not
 * skipped), no intermediate rounding  [Sec. 2 Eq. 1; Sec. 3.2; App. Rank
 * Analysis].  X, L, R are bfloat16 bit patterns.  Y is double [b][d_out].
 * rows: optional list of n_rows token indices to evaluate (NULL = all b rows,
 * in which case n_rows is ignored); Y then has n_rows rows in list order.
 */
int oracle_linear_fwd(const uint16_t *X, int b, const uint8_t *vals, const uint8_t *meta,
                      float s, const uint16_t *L, const uint16_t *R, int r,
                      int d_out, int d_in, const int32_t *rows, int n_rows, double *Y)
{
    if (!X || !vals || !meta || !Y || b < 1 || d_out < 1 || d_in < 8 || d_in % 8 != 0 || r < 0)
        return ORACLE_BAD_ARG;
    if (r > 0 && (!L || !R)) return ORACLE_BAD_ARG;
    const int nm = rows ? n_rows : b;
    int8_t *Wd = (int8_t *)malloc((size_t)d_out * d_in);
    if (!Wd) return ORACLE_BAD_ARG;
    int rc = oracle_unpack(vals, meta, d_out, d_in, Wd, NULL);
    if (rc != ORACLE_OK) { free(Wd); return rc; }
    const double sd = (double)s;
#pragma omp parallel for schedule(static)
    for (int mi = 0; mi < nm; ++mi) {
        const int m = rows ? rows[mi] : mi;
        double *xrow = (double *)malloc(sizeof(double) * (size_t)d_in);
        double *t = (double *)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        for (int k = 0; k < d_in; ++k) xrow[k] = bf16_to_double(X[(size_t)m * d_in + k]);
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int k = 0; k < d_in; ++k) acc += xrow[k] * bf16_to_double(R[(size_t)j * d_in + k]);
            t[j] = acc;
        }
        for (int n = 0; n < d_out; ++n) {
            double acc = 0.0;
            for (int k = 0; k < d_in; ++k) acc += xrow[k] * (sd * (double)Wd[(size_t)n * d_in + k]);
            double lr = 0.0;
            for (int j = 0; j < r; ++j) lr += t[j] * bf16_to_double(L[(size_t)n * r + j]);
            Y[(size_t)mi * d_out + n] = acc + lr;
        }
        free(xrow);
        free(t);
    }
    free(Wd);
    return ORACLE_OK;
}

/*
 * Dense form of the same layer: builds W_eff = s Q + L R explicitly
 * ([d_out][d_in], fp64) and returns Y = X W_eff^T  [Sec. 3.2: W ~ W^C + L R].
 * Used to check the factored routine against the unfactored definition.
 * W_eff_out (optional, [d_out][d_in]) receives the dense matrix.
 */
int oracle_linear_fwd_dense(const uint16_t *X, int b, const uint8_t *vals, const uint8_t *meta,
                            float s, const uint16_t *L, const uint16_t *R, int r,
                            int d_out, int d_in, double *Y, double *W_eff_out)
{
    if (!X || !vals || !meta || !Y || b < 1 || d_out < 1 || d_in < 8 || d_in % 8 != 0 || r < 0)
        return ORACLE_BAD_ARG;
    if (r > 0 && (!L || !R)) return ORACLE_BAD_ARG;
    int8_t *Wd = (int8_t *)malloc((size_t)d_out * d_in);
    double *We = (double *)malloc(sizeof(double) * (size_t)d_out * d_in);
    if (!Wd || !We) { free(Wd); free(We); return ORACLE_BAD_ARG; }
    int rc = oracle_unpack(vals, meta, d_out, d_in, Wd, NULL);
    if (rc != ORACLE_OK) { free(Wd); free(We); return rc; }
    const double sd = (double)s;
    for (int n = 0; n < d_out; ++n)
        for (int k = 0; k < d_in; ++k) {
            double w = sd * (double)Wd[(size_t)n * d_in + k];
            for (int j = 0; j < r; ++j)
                w += bf16_to_double(L[(size_t)n * r + j]) * bf16_to_double(R[(size_t)j * d_in + k]);
            We[(size_t)n * d_in + k] = w;
        }
    for (int m = 0; m < b; ++m)
        for (int n = 0; n < d_out; ++n) {
            double acc = 0.0;
            for (int k = 0; k < d_in; ++k)
                acc += bf16_to_double(X[(size_t)m * d_in + k]) * We[(size_t)n * d_in + k];
            Y[(size_t)m * d_out + n] = acc;
        }
    if (W_eff_out) memcpy(W_eff_out, We, sizeof(double) * (size_t)d_out * d_in);
    free(Wd);
    free(We);
    return ORACLE_OK;
}

/*
 * Inference FLOP-reduction ratio of a compressed transformer
 * [App. "Computation Reduction Analysis", Eq. 13]: dense over compressed flop
 * count for n blocks of hidden size d, feed-forward ratio a, vocabulary V,
 * 2:4 sparsity on every block linear and adapters of rank ratio rr (0 = none).
 * The batch size cancels.
 */
double oracle_flop_reduction(double d, double n, double a, double V, double rr)
{
    double dense = n * (4.0 * d * d + 2.0 * d * d * a) + d * V;
    double comp = n * (4.0 * d * d / 2.0 + 4.0 * 2.0 * d * d * rr + 2.0 * d * d * a / 2.0 +
                       2.0 * (d * d * rr + d * d * rr * a)) + d * V;
    return dense / comp;
}

/* ------------------------------------------------------------------------
 * Quantized adapters  [Sec. 3.3 "Low-rank Adapter Quantization": 4-bit AbsMax
 * group quantization, groups of 128 elements share one quantization parameter;
 * the symmetric uniform grid is that of Sec. 3.1, Eq. 2 and Eq. 5].
 *
 * The paper fixes neither the axis of the groups, nor the type of the
 * parameter, nor which of the 17 levels of Eq. 2 are kept.  Readings taken
 * here: an adapter is a row-major bf16 matrix A[rows][cols] whose rows run
 * along the contraction axis of the product it enters (R[r][d_in]: along d_in;
 * L[d_out][r]: along r); a group is 128 consecutive elements of a row (the last
 * group of a row may be shorter); the parameter of a group is stored as a bf16
 * scale = absmax / 7, so that codes are int4 in [-7, 7] (-8 never produced, but
 * decoded); the value of an element is code * scale.
 *
 * Floating point decides the codes, so the decision is taken in one stated
 * precision on both sides: scale = bf16_rne(fp32(absmax) / 7.0f) and
 * code = clamp(rint_even(fp32(a) / fp32(scale)), -8, 7), both divisions in IEEE
 * binary32; a group whose absmax is 0 gets scale 0 and codes 0.
 *
 * Storage: codes[rows][cols / 2], two per byte, the even column in the low
 * nibble, two's complement; scales[rows][ceil(cols / 128)] bf16 bit patterns.
 * 4 + 16/128 = 4.125 bits per element.
 * ---------------------------------------------------------------------- */
static float bf16_to_float(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* binary32 -> bfloat16, round to nearest even (finite inputs). */
static uint16_t float_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

int oracle_quant_adapter(const uint16_t *A, int rows, int cols, uint8_t *codes, uint16_t *scales)
{
    if (!A || !codes || !scales || rows < 1 || cols < 2 || cols % 2 != 0) return ORACLE_BAD_ARG;
    const int groups = (cols + 127) / 128;
    for (int i = 0; i < rows; ++i) {
        for (int g = 0; g < groups; ++g) {
            const int c0 = g * 128, c1 = c0 + 128 < cols ? c0 + 128 : cols;
            float absmax = 0.0f;
            for (int c = c0; c < c1; ++c) {
                float v = bf16_to_float(A[(size_t)i * cols + c]);
                if (v < 0.0f) v = -v;
                if (v > absmax) absmax = v;
            }
            const uint16_t sb = absmax > 0.0f ? float_to_bf16_rne(absmax / 7.0f) : 0;
            const float sc = bf16_to_float(sb);
            scales[(size_t)i * groups + g] = sb;
            for (int c = c0; c < c1; ++c) {
                int q = 0;
                if (sc > 0.0f) {
                    const float t = bf16_to_float(A[(size_t)i * cols + c]) / sc;
                    q = (int)nearbyintf(t);               /* default rounding mode: to nearest even */
                    if (q > 7) q = 7;
                    if (q < -8) q = -8;
                }
                uint8_t *byte = &codes[(size_t)i * (cols / 2) + c / 2];
                if (c % 2 == 0) *byte = (uint8_t)((*byte & 0xF0u) | ((unsigned)q & 0xFu));
                else            *byte = (uint8_t)((*byte & 0x0Fu) | (((unsigned)q & 0xFu) << 4));
            }
        }
    }
    return ORACLE_OK;
}

/* The values a quantized adapter stands for: out[i][c] = code * scale, exact in fp64. */
int oracle_dequant_adapter(const uint8_t *codes, const uint16_t *scales, int rows, int cols, double *out)
{
    if (!codes || !scales || !out || rows < 1 || cols < 2 || cols % 2 != 0) return ORACLE_BAD_ARG;
    const int groups = (cols + 127) / 128;
    for (int i = 0; i < rows; ++i)
        for (int c = 0; c < cols; ++c) {
            const uint8_t byte = codes[(size_t)i * (cols / 2) + c / 2];
            const int q = sext4(c % 2 == 0 ? byte & 0xFu : byte >> 4);
            out[(size_t)i * cols + c] = (double)q * bf16_to_double(scales[(size_t)i * groups + c / 128]);
        }
    return ORACLE_OK;
}

/*
 * The layer with quantized adapters: the definition of oracle_linear_fwd with L and R replaced
 * by the values their codes and scales stand for  [Sec. 3.2: W ~ W^C + L R; Sec. 3.3].
 * Lq/Ls: codes and scales of L[d_out][r]; Rq/Rs: of R[r][d_in].
 */
int oracle_linear_fwd_q(const uint16_t *X, int b, const uint8_t *vals, const uint8_t *meta, float s,
                        const uint8_t *Lq, const uint16_t *Ls, const uint8_t *Rq, const uint16_t *Rs, int r,
                        int d_out, int d_in, const int32_t *rows, int n_rows, double *Y)
{
    if (!X || !vals || !meta || !Y || b < 1 || d_out < 1 || d_in < 8 || d_in % 8 != 0 || r < 2 || r % 2 != 0)
        return ORACLE_BAD_ARG;
    if (!Lq || !Ls || !Rq || !Rs) return ORACLE_BAD_ARG;
    const int nm = rows ? n_rows : b;
    int8_t *Wd = (int8_t *)malloc((size_t)d_out * d_in);
    double *Ld = (double *)malloc(sizeof(double) * (size_t)d_out * r);
    double *Rd = (double *)malloc(sizeof(double) * (size_t)r * d_in);
    int rc = (Wd && Ld && Rd) ? ORACLE_OK : ORACLE_BAD_ARG;
    if (rc == ORACLE_OK) rc = oracle_unpack(vals, meta, d_out, d_in, Wd, NULL);
    if (rc == ORACLE_OK) rc = oracle_dequant_adapter(Lq, Ls, d_out, r, Ld);
    if (rc == ORACLE_OK) rc = oracle_dequant_adapter(Rq, Rs, r, d_in, Rd);
    if (rc != ORACLE_OK) { free(Wd); free(Ld); free(Rd); return rc; }
    const double sd = (double)s;
#pragma omp parallel for schedule(static)
    for (int mi = 0; mi < nm; ++mi) {
        const int m = rows ? rows[mi] : mi;
        double *xrow = (double *)malloc(sizeof(double) * (size_t)d_in);
        double *t = (double *)malloc(sizeof(double) * (size_t)r);
        for (int k = 0; k < d_in; ++k) xrow[k] = bf16_to_double(X[(size_t)m * d_in + k]);
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int k = 0; k < d_in; ++k) acc += xrow[k] * Rd[(size_t)j * d_in + k];
            t[j] = acc;
        }
        for (int n = 0; n < d_out; ++n) {
            double acc = 0.0;
            for (int k = 0; k < d_in; ++k) acc += xrow[k] * (sd * (double)Wd[(size_t)n * d_in + k]);
            double lr = 0.0;
            for (int j = 0; j < r; ++j) lr += t[j] * Ld[(size_t)n * r + j];
            Y[(size_t)mi * d_out + n] = acc + lr;
        }
        free(xrow);
        free(t);
    }
    free(Wd); free(Ld); free(Rd);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------
 * SLiM-Quant: the per-tensor scale search  [Sec. 3.1 "SLiM-Quant Quantization
 * Method", Eq. 2-7 and Algorithm 1; number of histogram bins: App. "Settings
 * and Hyperparameters"].
 *
 * The steps of Algorithm 1, in its order:
 *   f_abs      histogram of |W| over [0, M], M = max |W|, with
 *              B = max(512, min(d_in * d_out / 1000, 20000)) uniform bins; a bin
 *              stands for its centre x_i = (i + 1/2) M / B with weight count_i / N
 *   E(alpha)   = sum_{x_i <= alpha} p_i (alpha 2^(1-q) round(x_i 2^(q-1) / alpha) - x_i)^2
 *              + sum_{x_i >  alpha} p_i (alpha - x_i)^2              [Eq. 5, Eq. 6, Eq. 7]
 *   coarse     alpha = k M / 10, k = 1..10 ("10 uniform samples in (0, max W)"),
 *              eta_low = M / 10; alpha_low = the first minimiser
 *   fine       alpha = alpha_low - eta_low + j eta_high, j = 1..19, eta_high = eta_low / 10
 *              (the open interval (alpha_low - eta_low, alpha_low + eta_low)), capped at M;
 *              alpha* = the first minimiser over both grids
 *   quantize   code = clamp(rint(W / alpha* 2^(q-1)), -8, 7), scale s = alpha* 2^(1-q)
 * Readings where the text is garbled or silent: Eq. 2 / Eq. 5 are read as
 * code = round(clip(W / alpha, -1, 1) 2^(q-1)), value = code alpha 2^(1-q); the error model keeps
 * the paper's symmetric clip at alpha although int4 stores +8 as +7; the step sizes eta are not
 * given: ten coarse samples as the text says, and a fine step of a tenth of the coarse one; ties
 * go to the smaller alpha; q = 4.
 *
 * Floating point decides integers here (the bin of a weight, the argmin, the codes), so the
 * precision of every such decision is fixed: bin = min(B - 1, (int)((|w| / M) * B)) in binary32
 * (IEEE division, then multiplication, truncation); E(alpha) in binary64, bins added in
 * ascending order, no fused multiply-add; codes in binary32: rint((w / alpha32) * 8).
 * err_table (may be NULL) receives the 29 pairs (alpha, E(alpha)): coarse 1..10, then fine 1..19.
 * ---------------------------------------------------------------------- */
static double quant_search_error(const uint32_t *hist, int B, double M, double n_total, double alpha)
{
    double e = 0.0;
    const double width = M / (double)B;
    for (int i = 0; i < B; ++i) {
        if (!hist[i]) continue;
        const double x = ((double)i + 0.5) * width;
        const double p = (double)hist[i] / n_total;
        double d;
        if (x <= alpha) {
            const double level = rint((x * 8.0) / alpha);
            d = (alpha * 0.125) * level - x;
        } else {
            d = alpha - x;
        }
        const double dd = d * d;
        const double term = p * dd;
        e = e + term;
    }
    return e;
}

int oracle_slim_quant(const float *W, int d_out, int d_in, int8_t *codes, float *scale, double *alpha_out,
                      double *err_table)
{
    if (!W || !codes || !scale || d_out < 1 || d_in < 1) return ORACLE_BAD_ARG;
    const size_t n = (size_t)d_out * (size_t)d_in;
    float M = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        const float a = fabsf(W[i]);
        if (!(a <= 3.0e38f)) return ORACLE_BAD_ARG;          /* NaN or infinity */
        if (a > M) M = a;
    }
    if (M == 0.0f) {                                          /* nothing to quantize */
        memset(codes, 0, n);
        *scale = 0.0f;
        if (alpha_out) *alpha_out = 0.0;
        if (err_table) memset(err_table, 0, sizeof(double) * 58);
        return ORACLE_OK;
    }
    long long bins = (long long)n / 1000;
    if (bins > 20000) bins = 20000;
    if (bins < 512) bins = 512;
    const int B = (int)bins;
    uint32_t *hist = (uint32_t *)calloc((size_t)B, sizeof(uint32_t));
    if (!hist) return ORACLE_BAD_ARG;
    for (size_t i = 0; i < n; ++i) {
        const float ratio = fabsf(W[i]) / M;
        int b = (int)(ratio * (float)B);
        if (b > B - 1) b = B - 1;
        hist[b] += 1u;
    }
    const double Md = (double)M, eta_low = Md / 10.0, eta_high = eta_low / 10.0;
    double best_a = 0.0, best_e = 0.0;
    int have = 0, t = 0;
    for (int k = 1; k <= 10; ++k) {
        const double a = (Md * (double)k) / 10.0;
        const double e = quant_search_error(hist, B, Md, (double)n, a);
        if (err_table) { err_table[2 * t] = a; err_table[2 * t + 1] = e; }
        ++t;
        if (!have || e < best_e) { best_a = a; best_e = e; have = 1; }
    }
    const double a_low = best_a;
    for (int j = 1; j <= 19; ++j) {
        double a = (a_low - eta_low) + (double)j * eta_high;
        if (a > Md) a = Md;
        const double e = a > 0.0 ? quant_search_error(hist, B, Md, (double)n, a) : best_e + 1.0;
        if (err_table) { err_table[2 * t] = a; err_table[2 * t + 1] = e; }
        ++t;
        if (a > 0.0 && (e < best_e || (e == best_e && a < best_a))) { best_a = a; best_e = e; }
    }
    free(hist);
    const float a32 = (float)best_a;
    for (size_t i = 0; i < n; ++i) {
        const float v = (W[i] / a32) * 8.0f;
        int q = (int)nearbyintf(v);
        if (q > 7) q = 7;
        if (q < -8) q = -8;
        codes[i] = (int8_t)q;
    }
    *scale = a32 * 0.125f;
    if (alpha_out) *alpha_out = best_a;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------
 * The 2:4 mask of the pipeline's second step  [Sec. 3 and Fig. 1: the quantized weights are
 * sparsified by a one-shot pruning method; Sec. 3.2: "the product of the magnitude of the weights
 * and activations is a useful metric for identifying important weights"].
 * In every aligned group of four along d_in the two entries with the largest metric
 *     m[n][k] = |Q[n][k]| * xbar[k]        (xbar == NULL: m = |Q|, magnitude pruning)
 * are kept; equal metrics go to the lower index.  The metric is one binary32 multiplication.
 * xbar is the average input magnitude per input channel (non-negative, finite).
 * ---------------------------------------------------------------------- */
int oracle_mask_top2(const int8_t *codes, const float *xbar, int d_out, int d_in, uint8_t *mask)
{
    if (!codes || !mask || d_out < 1 || d_in < 4 || d_in % 4 != 0) return ORACLE_BAD_ARG;
    for (int n = 0; n < d_out; ++n)
        for (int g = 0; g < d_in / 4; ++g) {
            float m[4];
            for (int i = 0; i < 4; ++i) {
                const int k = 4 * g + i;
                const int c = codes[(size_t)n * d_in + k];
                const float a = (float)(c < 0 ? -c : c);
                if (xbar && !(xbar[k] >= 0.0f && xbar[k] <= 3.0e38f)) return ORACLE_BAD_ARG;
                m[i] = xbar ? a * xbar[k] : a;
            }
            for (int i = 0; i < 4; ++i) {
                int beaten = 0;                       /* entries that come before i in the order */
                for (int j = 0; j < 4; ++j)
                    if (j != i && (m[j] > m[i] || (m[j] == m[i] && j < i))) ++beaten;
                mask[(size_t)n * d_in + 4 * g + i] = (uint8_t)(beaten < 2);
            }
        }
    return ORACLE_OK;
}

/* Number of OpenMP threads oracle_linear_fwd will use (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif
