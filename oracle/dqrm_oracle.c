/*
 * DQRM embedding-path oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of what the quantisation-aware
 * embedding step of DQRM (Deep Quantized Recommendation Model) computes.  It
 * exists so that the CUDA library can be checked against something written
 * straight from the paper.  It shares no code with the CUDA path and nothing
 * in the product may call it; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg do.
 *
 * The paper states the method in prose and prints no formula for its
 * quantiser.  What it fixes: one FP32 scale per table (Section 4.1), a uniform
 * quantiser clipped to the table's fixed minimum and maximum (Appendix A, the
 * part on earlier QAT techniques), a scale found by traversing the whole table and
 * refreshed only periodically (Section 3.2), quantisation applied to the rows
 * a batch actually gathers (Section 3.1, Figure 2(b)), embedding gradients
 * kept as sparse (indices, values) whose values alone are quantised to INT8
 * with a scale determined by bit width and tensor distribution, and a local
 * update with the dequantised gradient (Appendix B.1).  The remaining choices
 * (symmetric range, divisor 2^(b-1)-1, round-half-to-even, true division,
 * quantise-then-pool, pass-through backward, abs-max gradient scale) are this
 * build's reading and are listed in the design notes.
 *
 * Every FP32 operation below is a single, separately rounded IEEE operation:
 * compile with -ffp-contract=off and without fast-math.
 *
 * Layout: tables are one arena [sum R_t, D] float32, row_off[t] = first arena
 * row of table t; indices are row numbers within their table, table-major;
 * bag g = t*B + i owns indices[offsets[g] .. offsets[g+1]); out and grad_out
 * are [B, T, D].
 *
 * Parity pins: see tests/test_oracle_*.py.  Every function here is pinned by
 * at least one check that does not come from this file (hand-worked cases,
 * exact rational arithmetic, numpy library routines, dense brute force).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- quantiser (Section 4.1: one scale per table; Appendix A: evenly spaced
 *      levels, the clipping range fixed by the table's min and max) --------- */

static int32_t q_max(int bits) { return (int32_t)((1u << (bits - 1)) - 1u); }
static int32_t q_min(int bits) { return -(int32_t)(1u << (bits - 1)); }

/* scale = max(absmax, 1e-8) / (2^(b-1) - 1), one FP32 divide */
float dqrm_oracle_scale_from_absmax(float absmax, int bits)
{
    const float floor_ = 1e-8f;
    float a = absmax > floor_ ? absmax : floor_;
    return a / (float)q_max(bits);
}

/* code = clamp(round_half_even(x / s), -2^(b-1), 2^(b-1)-1) */
int32_t dqrm_oracle_quantize(float x, float s, int bits)
{
    float r = rintf(x / s); /* default rounding mode: to nearest, ties to even */
    float lo = (float)q_min(bits), hi = (float)q_max(bits);
    if (r < lo) r = lo;     /* clamp before the integer cast: same result, no overflow */
    if (r > hi) r = hi;
    return (int32_t)r;
}

/* value = code * s, one FP32 multiply */
float dqrm_oracle_dequantize(int32_t q, float s) { return (float)q * s; }

float dqrm_oracle_fake_quant(float x, float s, int bits)
{
    return dqrm_oracle_dequantize(dqrm_oracle_quantize(x, s, bits), s);
}

/* ---- scale refresh (Section 3.2: traverse the table to find the scale) ---- */

void dqrm_oracle_scale_refresh(const float *tables, const int64_t *row_off, int T, int D,
                               const int32_t *bits, float *scales, float *minmax /* [T][2] or NULL */)
{
    for (int t = 0; t < T; ++t) {
        int64_t n = (row_off[t + 1] - row_off[t]) * (int64_t)D;
        const float *w = tables + row_off[t] * (int64_t)D;
        float mn = 0.0f, mx = 0.0f;
        if (n > 0) { mn = w[0]; mx = w[0]; }
        for (int64_t i = 1; i < n; ++i) {
            if (w[i] < mn) mn = w[i];
            if (w[i] > mx) mx = w[i];
        }
        float a = fabsf(mn) > fabsf(mx) ? fabsf(mn) : fabsf(mx);
        scales[t] = dqrm_oracle_scale_from_absmax(a, bits[t]);
        if (minmax) { minmax[2 * t] = mn; minmax[2 * t + 1] = mx; }
    }
}

/* ---- forward (Section 3.1 / Figure 2(b): gather the used rows, then quantise
 *      them; sum pooling over the bag) --------------------------------------- */

void dqrm_oracle_emb_fwd(const float *tables, const int64_t *row_off, int T, int D, int B,
                         const int32_t *indices, const int32_t *offsets,
                         const float *scales, const int32_t *bits,
                         float *out /* [B][T][D] */, int8_t *codes_out /* [L][D] or NULL */)
{
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    for (int t = 0; t < T; ++t) {
        const float *w = tables + row_off[t] * (int64_t)D;
        for (int i = 0; i < B; ++i) {
            int64_t g = (int64_t)t * B + i;
            for (int d = 0; d < D; ++d) acc[d] = 0.0;
            for (int32_t j = offsets[g]; j < offsets[g + 1]; ++j) {
                const float *row = w + (int64_t)indices[j] * D;
                for (int d = 0; d < D; ++d) {
                    int32_t q = dqrm_oracle_quantize(row[d], scales[t], bits[t]);
                    if (codes_out) codes_out[(int64_t)j * D + d] = (int8_t)q;
                    acc[d] += (double)dqrm_oracle_dequantize(q, scales[t]);
                }
            }
            float *o = out + ((int64_t)i * T + t) * D;
            for (int d = 0; d < D; ++d) o[d] = (float)acc[d];
        }
    }
    free(acc);
}

/* ---- backward (Section 4.3 / Appendix B.1: the embedding gradient is a sparse
 *      (indices, values) tensor over the rows the batch touched; duplicates are
 *      coalesced).  Sum pooling and a straight-through quantiser hand every
 *      lookup its bag's upstream gradient unchanged. --------------------------- */

typedef struct { int32_t row; int32_t pos; } pair_t;

static int pair_cmp(const void *a, const void *b)
{
    const pair_t *x = (const pair_t *)a, *y = (const pair_t *)b;
    if (x->row != y->row) return x->row < y->row ? -1 : 1;
    if (x->pos != y->pos) return x->pos < y->pos ? -1 : 1;
    return 0;
}

/* Returns the number of unique (table,row) pairs U.  unique_rows has room for L
 * entries, grad_rows for L*D, uniq_off for T+1. */
int64_t dqrm_oracle_emb_bwd(const float *grad_out /* [B][T][D] */, int T, int D, int B,
                            const int32_t *indices, const int32_t *offsets,
                            int32_t *unique_rows, int32_t *uniq_off, float *grad_rows)
{
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    int64_t u = 0;
    for (int t = 0; t < T; ++t) {
        uniq_off[t] = (int32_t)u;
        int32_t lo = offsets[(int64_t)t * B], hi = offsets[(int64_t)(t + 1) * B];
        int32_t n = hi - lo;
        if (n <= 0) continue;
        pair_t *p = (pair_t *)malloc(sizeof(pair_t) * (size_t)n);
        int32_t *bag_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        for (int i = 0; i < B; ++i) {
            int64_t g = (int64_t)t * B + i;
            for (int32_t j = offsets[g]; j < offsets[g + 1]; ++j) {
                p[j - lo].row = indices[j];
                p[j - lo].pos = j;
                bag_of[j - lo] = i;
            }
        }
        qsort(p, (size_t)n, sizeof(pair_t), pair_cmp);
        int32_t k = 0;
        while (k < n) {
            int32_t row = p[k].row;
            for (int d = 0; d < D; ++d) acc[d] = 0.0;
            while (k < n && p[k].row == row) { /* ascending lookup position */
                const float *g = grad_out + ((int64_t)bag_of[p[k].pos - lo] * T + t) * D;
                for (int d = 0; d < D; ++d) acc[d] += (double)g[d];
                ++k;
            }
            unique_rows[u] = row;
            for (int d = 0; d < D; ++d) grad_rows[u * D + d] = (float)acc[d];
            ++u;
        }
        free(p);
        free(bag_of);
    }
    uniq_off[T] = (int32_t)u;
    free(acc);
    return u;
}

/* ---- INT8 gradient quantiser (Appendix B.1: only the values of the sparse
 *      gradient are quantised; the scale follows from the bit width and the
 *      tensor's own distribution; one scale per parameter tensor) ------------- */

void dqrm_oracle_grad_quant_int8(const float *grad_rows, const int32_t *uniq_off, int T, int D,
                                 int8_t *codes, float *grad_scales)
{
    for (int t = 0; t < T; ++t) {
        int64_t lo = (int64_t)uniq_off[t] * D, hi = (int64_t)uniq_off[t + 1] * D;
        float a = 0.0f;
        for (int64_t i = lo; i < hi; ++i) {
            float v = fabsf(grad_rows[i]);
            if (v > a) a = v;
        }
        float s = dqrm_oracle_scale_from_absmax(a, 8);
        grad_scales[t] = s;
        for (int64_t i = lo; i < hi; ++i)
            codes[i] = (int8_t)dqrm_oracle_quantize(grad_rows[i], s, 8);
    }
}

/* ---- touched-row update (Appendix B.1: the local step uses the dequantised
 *      gradient; Section 3.1: the FP32 master copy is what is updated) -------- */

void dqrm_oracle_row_update(float *tables, const int64_t *row_off, int T, int D,
                            const int32_t *unique_rows, const int32_t *uniq_off,
                            const int8_t *codes, const float *grad_scales, float lr)
{
    for (int t = 0; t < T; ++t) {
        for (int64_t u = uniq_off[t]; u < uniq_off[t + 1]; ++u) {
            float *w = tables + (row_off[t] + (int64_t)unique_rows[u]) * D;
            for (int d = 0; d < D; ++d) {
                float g = dqrm_oracle_dequantize((int32_t)codes[u * D + d], grad_scales[t]);
                float step = lr * g;
                w[d] = w[d] - step;
            }
        }
    }
}

/* ==========================================================================
 * Data-parallel exchange of the sparse INT8 gradient (Appendix B.1, Figure
 * "Customized Data Parallelism Framework"): every rank computes its local
 * gradient, the per-tensor quantisation scales are unified across ranks, each
 * rank quantises with the unified scale, the integer gradients are summed over
 * ranks, and every rank applies the dequantised sum.  Readings taken here: the
 * scales are unified by MAX (no rank clips), the integers are summed exactly in
 * 32 bits (so no re-rounding at intermediate reduce steps, the caveat the
 * paper raises for recursive-doubling all-reduce), and the update uses the sum,
 * not the mean.
 * ========================================================================== */

/* codes = Q(grad_rows; given scales[t], 8): the quantiser of step "quantise locally
 * with the unified scale" */
void dqrm_oracle_grad_quant_int8_scaled(const float *grad_rows, const int32_t *uniq_off, int T, int D,
                                        const float *scales, int8_t *codes)
{
    for (int t = 0; t < T; ++t)
        for (int64_t i = (int64_t)uniq_off[t] * D; i < (int64_t)uniq_off[t + 1] * D; ++i)
            codes[i] = (int8_t)dqrm_oracle_quantize(grad_rows[i], scales[t], 8);
}

/* per-table max |grad_rows| (0 for a table that touched nothing) */
void dqrm_oracle_grad_absmax(const float *grad_rows, const int32_t *uniq_off, int T, int D, float *absmax)
{
    for (int t = 0; t < T; ++t) {
        float a = 0.0f;
        for (int64_t i = (int64_t)uniq_off[t] * D; i < (int64_t)uniq_off[t + 1] * D; ++i) {
            float v = fabsf(grad_rows[i]);
            if (v > a) a = v;
        }
        absmax[t] = a;
    }
}

/* Sum of the ranks' integer gradients.  Rank r holds, per table, ascending distinct rows
 * rows[r][uoff[r][t] .. uoff[r][t+1]) with codes[r][u][D].  Output: the ascending union of
 * rows per table (out_rows, out_off[T+1]) and the exact int32 sum of the codes of each row.
 * out_rows / out_sums have room for the total number of input rows.  Returns the union size. */
int64_t dqrm_oracle_dp_merge(int W, int T, int D, const int32_t *const *rows, const int32_t *const *uoff,
                             const int8_t *const *codes, int32_t *out_rows, int32_t *out_off, int32_t *out_sums)
{
    int64_t n = 0;
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)W);
    for (int t = 0; t < T; ++t) {
        out_off[t] = (int32_t)n;
        for (int r = 0; r < W; ++r) pos[r] = uoff[r][t];
        for (;;) {
            /* smallest row not yet consumed over the W ascending lists */
            int found = 0;
            int32_t best = 0;
            for (int r = 0; r < W; ++r)
                if (pos[r] < uoff[r][t + 1] && (!found || rows[r][pos[r]] < best)) { best = rows[r][pos[r]]; found = 1; }
            if (!found) break;
            out_rows[n] = best;
            for (int d = 0; d < D; ++d) out_sums[n * D + d] = 0;
            for (int r = 0; r < W; ++r)
                if (pos[r] < uoff[r][t + 1] && rows[r][pos[r]] == best) {
                    for (int d = 0; d < D; ++d) out_sums[n * D + d] += (int32_t)codes[r][(int64_t)pos[r] * D + d];
                    ++pos[r];
                }
            ++n;
        }
    }
    out_off[T] = (int32_t)n;
    free(pos);
    return n;
}

/* W[row] -= lr * ((float)sum * scale[t]) for every row of the union: three rounded FP32 operations */
void dqrm_oracle_row_update_i32(float *tables, const int64_t *row_off, int T, int D, const int32_t *rows,
                                const int32_t *off, const int32_t *sums, const float *scales, float lr)
{
    for (int t = 0; t < T; ++t)
        for (int64_t u = off[t]; u < off[t + 1]; ++u) {
            float *w = tables + (row_off[t] + (int64_t)rows[u]) * D;
            for (int d = 0; d < D; ++d) {
                float g = (float)sums[u * D + d] * scales[t];
                float step = lr * g;
                w[d] = w[d] - step;
            }
        }
}

/* ==========================================================================
 * Bit-packed export of the quantised tables and inference from them (Appendix C:
 * the INT4 embedding vectors are bit-packed into bytes to realise the 8x smaller
 * model; Table "res_tab": 2.161 GB -> 0.270 GB, 12.575 GB -> 1.572 GB).  The paper
 * gives no layout; here element d of a row sits in byte (d*b)/8 at bit offset
 * (d*b)%8, lowest bits first, as a b-bit two's-complement code, b in {2, 4, 8},
 * and a row takes D*b/8 bytes.
 * ========================================================================== */

void dqrm_oracle_pack_tables(const float *tables, const int64_t *row_off, int T, int D,
                             const float *scales, int bits, uint8_t *packed /* [sum R_t][D*bits/8] */)
{
    const int row_bytes = D * bits / 8;
    const uint32_t mask = (1u << bits) - 1u;
    for (int t = 0; t < T; ++t)
        for (int64_t r = row_off[t]; r < row_off[t + 1]; ++r) {
            uint8_t *dst = packed + r * row_bytes;
            memset(dst, 0, (size_t)row_bytes);
            for (int d = 0; d < D; ++d) {
                int32_t q = dqrm_oracle_quantize(tables[r * D + d], scales[t], bits);
                dst[(d * bits) / 8] |= (uint8_t)(((uint32_t)q & mask) << ((d * bits) % 8));
            }
        }
}

static int32_t unpack_code(const uint8_t *row, int d, int bits)
{
    uint32_t v = (row[(d * bits) / 8] >> ((d * bits) % 8)) & ((1u << bits) - 1u);
    if (v & (1u << (bits - 1))) v |= ~((1u << bits) - 1u); /* sign-extend */
    return (int32_t)v;
}

/* inference lookup from the packed tables: out[i][t][:] = sum over the bag of code * scale[t] */
void dqrm_oracle_packed_fwd(const uint8_t *packed, const int64_t *row_off, int T, int D, int B,
                            const int32_t *indices, const int32_t *offsets, const float *scales, int bits,
                            float *out)
{
    const int row_bytes = D * bits / 8;
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < B; ++i) {
            int64_t g = (int64_t)t * B + i;
            for (int d = 0; d < D; ++d) acc[d] = 0.0;
            for (int32_t j = offsets[g]; j < offsets[g + 1]; ++j) {
                const uint8_t *row = packed + (row_off[t] + (int64_t)indices[j]) * row_bytes;
                for (int d = 0; d < D; ++d) acc[d] += (double)dqrm_oracle_dequantize(unpack_code(row, d, bits), scales[t]);
            }
            float *o = out + ((int64_t)i * T + t) * D;
            for (int d = 0; d < D; ++d) o[d] = (float)acc[d];
        }
    free(acc);
}

/* ---- table-sharded forward payload (paper Section 4.3, the remark on hybrid parallelism: the
 * all-to-all that carries embedding vectors shrinks with the code width) -------------------------
 * For one-index bags the pooled vector is the dequantised row, so the owner of a table can send the
 * row's b-bit codes instead of FP32 values.  payload[i][t] holds the packed codes (layout of
 * dqrm_oracle_pack_tables) of bag (t, i)'s row.  Returns 0, or -1 when a bag does not hold exactly
 * one index. */
int dqrm_oracle_emb_fwd_codes(const float *tables, const int64_t *row_off, int T, int D, int B,
                              const int32_t *indices, const int32_t *offsets, const float *scales, int bits,
                              uint8_t *payload /* [B][T][D*bits/8] */)
{
    const int row_bytes = D * bits / 8;
    const uint32_t mask = (1u << bits) - 1u;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < B; ++i) {
            int64_t g = (int64_t)t * B + i;
            if (offsets[g + 1] - offsets[g] != 1) return -1;
            const float *row = tables + (row_off[t] + (int64_t)indices[offsets[g]]) * D;
            uint8_t *dst = payload + ((int64_t)i * T + t) * row_bytes;
            memset(dst, 0, (size_t)row_bytes);
            for (int d = 0; d < D; ++d) {
                int32_t q = dqrm_oracle_quantize(row[d], scales[t], bits);
                dst[(d * bits) / 8] |= (uint8_t)(((uint32_t)q & mask) << ((d * bits) % 8));
            }
        }
    return 0;
}

/* receiver side: out[i][t0 + j][:] = code * scales[j] for the T_blk tables of one sender */
void dqrm_oracle_decode_payload(const uint8_t *payload /* [B][T_blk][D*bits/8] */, const float *scales /* [T_blk] */,
                                int bits, int B, int T_blk, int T_total, int t0, int D, float *out /* [B][T_total][D] */)
{
    const int row_bytes = D * bits / 8;
    for (int i = 0; i < B; ++i)
        for (int j = 0; j < T_blk; ++j) {
            const uint8_t *row = payload + ((int64_t)i * T_blk + j) * row_bytes;
            float *o = out + ((int64_t)i * T_total + t0 + j) * D;
            for (int d = 0; d < D; ++d) o[d] = dqrm_oracle_dequantize(unpack_code(row, d, bits), scales[j]);
        }
}
