// Forward of the quantisation-aware embedding lookup (paper Section 3.1, Figure 2(b)):
// gather the rows a batch uses from the FP32 master table, fake-quantise each gathered
// row with the table's stored scale, and sum-pool over the bag.  No low-precision copy
// of the table exists; only the gathered rows are ever quantised.
//
// HBM-bound random row gather.  Measured on B200, a bare gather of this access pattern
// runs fastest with many resident warps and only two to four independent 128-bit loads
// per lane, so the kernels are kept lean (about 40 registers) rather than deeply
// unrolled.  blockIdx.y is the table, which makes scale, bit width and row base block
// constants.  A group of LPR lanes owns one row: a feature-16 row is one 64-byte request
// of four lanes, a feature-64 row one 256-byte request of sixteen.
//   * fwd_onehot_kernel (launched when L == T*B and no codes are asked for, the Criteo-shaped
//     training case): a warp owns 32 consecutive bags, does their bookkeeping one bag per
//     lane, then fetches the rows 32/LPR per step with NB steps in flight; the pooled value
//     is the fake-quantised row itself.  A bag that turns out not to hold exactly one index
//     is pooled by a plain loop.
//   * fwd_bags_kernel (any other batch): a lane group walks one bag at a time, NB of its
//     rows per batch, and sums them in bag order in FP64, rounded once, so the result
//     does not depend on the launch shape.
#include "common.cuh"

namespace {

constexpr int FW_THREADS = 256;
// independent rows in flight per lane group.  Measured on B200: four for rows of up to 128
// bytes, two for 256- and 512-byte rows (more resident warps beat deeper unrolling), one
// when a lane already holds several 128-bit pieces of every row
template <int LPR, int CH>
struct NBOf { static constexpr int v = CH >= 2 ? 1 : 4; };

struct FwdArgs {
    const float *tables;
    const int64_t *row_off;
    const int32_t *indices;
    const int32_t *offsets;
    const float *scales;
    const int32_t *bits;
    float *out;
    int8_t *codes_out;
    int T, D, B;
    int64_t L;
    int *status;
};

__device__ __forceinline__ void store_codes(int8_t *codes_out, int64_t j, int D, int c4, const float4 &c)
{
    char4 cc = make_char4((signed char)(int)c.x, (signed char)(int)c.y, (signed char)(int)c.z, (signed char)(int)c.w);
    *reinterpret_cast<char4 *>(codes_out + j * D + 4 * c4) = cc;
}

// clamps an index into [0, nrows) and remembers that it had to
__device__ __forceinline__ int32_t clamp_index(int32_t idx, int32_t nrows, bool &bad)
{
    bad |= (idx < 0) | (idx >= nrows);
    return min(max(idx, 0), nrows - 1);
}

// Per-table constants of a block
struct TableCtx {
    QuantScale qs;
    const float *tbl;
    int32_t nrows;
    int64_t g0;
};

__device__ __forceinline__ TableCtx table_ctx(const FwdArgs &a, int t, int D)
{
    TableCtx c;
    c.qs = dq_make_scale(__ldg(a.scales + t), __ldg(a.bits + t));
    const int64_t r0 = __ldg(a.row_off + t);
    c.nrows = (int32_t)(__ldg(a.row_off + t + 1) - r0);
    c.tbl = a.tables + r0 * D;
    c.g0 = (int64_t)t * a.B;
    return c;
}

// plain pooling of one bag (one row at a time): used for the rare bags of a one-index batch
template <int LPR, int CH>
__device__ __forceinline__ void pool_bag_plain(const FwdArgs &a, const TableCtx &tc, int D, int d4, int32_t lo,
                                               int32_t hi, float *out_row, int lane, bool &bad)
{
    if (lo < 0 || hi < lo || (int64_t)hi > a.L) { bad = true; hi = lo = 0; }
#pragma unroll 1
    for (int c = 0; c < CH; ++c) {
        const int c4 = c * LPR + lane;
        if (c4 >= d4) continue;
        double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll 1
        for (int32_t j = lo; j < hi; ++j) {
            const int32_t idx = clamp_index(__ldg(a.indices + j), tc.nrows, bad);
            float4 cd, f;
            dq_fq4(__ldg(reinterpret_cast<const float4 *>(tc.tbl + (int64_t)idx * D) + c4), tc.qs, cd, f);
            a0 += (double)f.x; a1 += (double)f.y; a2 += (double)f.z; a3 += (double)f.w;
            if (a.codes_out) store_codes(a.codes_out, j, D, c4, cd);
        }
        reinterpret_cast<float4 *>(out_row)[c4] = make_float4((float)a0, (float)a1, (float)a2, (float)a3);
    }
}

// A warp takes 32 consecutive bags of its table.  The bookkeeping of a bag (its offsets, its index,
// the range checks) is done once, by the one lane that owns the bag; the rows are then fetched
// 32/LPR at a time by all lanes, each step reading its bag's index from the owner lane by shuffle.
// Measured on B200 the kernel is bound by instruction issue, not by HBM, at 256-byte rows, which
// is why the per-bag work is kept off the per-row path.
template <int LPR, int CH, bool EXACT>
__global__ void __launch_bounds__(FW_THREADS, 5)
fwd_onehot_kernel(const FwdArgs a)
{
    constexpr int NB = NBOf<LPR, CH>::v;      // row steps in flight
    constexpr int RPW = 32 / LPR;             // rows one warp instruction covers
    constexpr int WPB = FW_THREADS / 32;
    const int D = EXACT ? 4 * LPR * CH : a.D;
    const int d4 = D >> 2;
    const int t = blockIdx.y;
    const int wlane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lane = wlane % LPR, grp = wlane / LPR;
    const TableCtx tc = table_ctx(a, t, D);
    const float4 *tbl_lane = reinterpret_cast<const float4 *>(tc.tbl) + lane;
    const int TD4 = a.T * d4;                 // 128-bit vectors between the output rows of bags i and i+1
    bool bad = false;
    const uint64_t keep = dq_policy_evict_last();

    for (int i0 = (blockIdx.x * WPB + warp) * 32; i0 < a.B; i0 += gridDim.x * (WPB * 32)) {
        // ---- lane-per-bag bookkeeping
        const int i = i0 + wlane;
        int32_t idx = 0;
        bool single = false;
        if (i < a.B) {
            const int32_t lo = __ldg(a.offsets + tc.g0 + i), hi = __ldg(a.offsets + tc.g0 + i + 1);
            idx = __ldg(a.indices + tc.g0 + i);            // right when the offsets are the identity (L == T*B)
            single = (hi - lo == 1) & (lo >= 0) & ((int64_t)hi <= a.L);
            if (single) {
                if ((int64_t)lo != tc.g0 + i) idx = __ldg(a.indices + lo);
                idx = clamp_index(idx, tc.nrows, bad);
            }
        }
        const unsigned one = __ballot_sync(0xffffffffu, single);
        unsigned rare = __ballot_sync(0xffffffffu, (i < a.B) && !single);
        float4 *out_lane = reinterpret_cast<float4 *>(a.out) + ((int64_t)i0 * a.T + t) * d4 + lane;

        // ---- rows, RPW per step, NB steps in flight
#pragma unroll 1
        for (int k0 = 0; k0 < 32; k0 += RPW * NB) {
            if ((one >> k0) == 0u) break;
            int32_t ib[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) ib[b] = __shfl_sync(0xffffffffu, idx, (k0 + b * RPW + grp) & 31);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int c4 = c * LPR + lane;
                float4 v[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int bag = k0 + b * RPW + grp;
                    if (bag < 32 && ((one >> bag) & 1u) && (EXACT || c4 < d4))
                        v[b] = dq_ld_nc_keep(tbl_lane + (int64_t)ib[b] * d4 + c * LPR, keep);   // the update reads the row again
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int bag = k0 + b * RPW + grp;
                    if (bag < 32 && ((one >> bag) & 1u) && (EXACT || c4 < d4)) {
                        float4 cd, f;
                        dq_fq4(v[b], tc.qs, cd, f);
                        __stcs(out_lane + (int64_t)bag * TD4 + c * LPR, f);   // written once, read by nobody here
                    }
                }
            }
        }
        // ---- bags that do not hold exactly one index: pooled by the first lane group, one at a time
        while (rare) {
            const int bag = __ffs(rare) - 1;
            rare &= rare - 1;
            const int ii = i0 + bag;
            if (grp == 0) {
                const int32_t l = __ldg(a.offsets + tc.g0 + ii), h = __ldg(a.offsets + tc.g0 + ii + 1);
                pool_bag_plain<LPR, CH>(a, tc, D, d4, l, h, a.out + ((int64_t)ii * a.T + t) * D, lane, bad);
            }
        }
    }
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
}

template <int LPR, int CH, bool EXACT>
__global__ void __launch_bounds__(FW_THREADS)
fwd_bags_kernel(const FwdArgs a)
{
    constexpr int NB = NBOf<LPR, CH>::v;
    constexpr int GPB = FW_THREADS / LPR;
    const int D = EXACT ? 4 * LPR * CH : a.D;
    const int d4 = D >> 2;
    const int t = blockIdx.y;
    const int lane = threadIdx.x % LPR;
    const int grp = threadIdx.x / LPR;
    const TableCtx tc = table_ctx(a, t, D);
    bool bad = false;

    for (int i = blockIdx.x * GPB + grp; i < a.B; i += gridDim.x * GPB) {
        int32_t lo = __ldg(a.offsets + tc.g0 + i), hi = __ldg(a.offsets + tc.g0 + i + 1);
        if (lo < 0 || hi < lo || (int64_t)hi > a.L) { bad = true; hi = lo = 0; }
        double acc[CH][4];
#pragma unroll
        for (int c = 0; c < CH; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.0;
        for (int32_t j0 = lo; j0 < hi; j0 += NB) {
            int32_t idx[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) idx[b] = (j0 + b < hi) ? clamp_index(__ldg(a.indices + j0 + b), tc.nrows, bad) : 0;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int c4 = c * LPR + lane;
                float4 v[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    if (j0 + b < hi && (EXACT || c4 < d4))
                        v[b] = __ldg(reinterpret_cast<const float4 *>(tc.tbl + (int64_t)idx[b] * D) + c4);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (j0 + b < hi && (EXACT || c4 < d4)) {
                        float4 cd, f;
                        dq_fq4(v[b], tc.qs, cd, f);
                        acc[c][0] += (double)f.x;
                        acc[c][1] += (double)f.y;
                        acc[c][2] += (double)f.z;
                        acc[c][3] += (double)f.w;
                        if (a.codes_out) store_codes(a.codes_out, j0 + b, D, c4, cd);
                    }
                }
            }
        }
        float4 *o = reinterpret_cast<float4 *>(a.out + ((int64_t)i * a.T + t) * D);
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int c4 = c * LPR + lane;
            if (EXACT || c4 < d4)
                o[c4] = make_float4((float)acc[c][0], (float)acc[c][1], (float)acc[c][2], (float)acc[c][3]);
        }
    }
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
}

template <int LPR, int CH, bool EXACT>
int launch2(dqrm_ctx *ctx, const FwdArgs &a, cudaStream_t st)
{
    constexpr int GPB = FW_THREADS / LPR;
    // the one-index kernel does not emit codes; a caller that asks for them gets the general kernel
    const bool onehot = a.L == (int64_t)a.T * a.B && a.codes_out == nullptr;
    const int per_block = onehot ? FW_THREADS : GPB;
    int bx = (a.B + per_block - 1) / per_block;
    const int cap = (ctx->num_sms * 32 + ctx->T - 1) / ctx->T;     // a few waves over all tables
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)ctx->T);
    if (onehot) fwd_onehot_kernel<LPR, CH, EXACT><<<grid, FW_THREADS, 0, st>>>(a);
    else fwd_bags_kernel<LPR, CH, EXACT><<<grid, FW_THREADS, 0, st>>>(a);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_FWD);
    return DQRM_OK;
}

template <int LPR, int CH>
int launch(dqrm_ctx *ctx, const FwdArgs &a, cudaStream_t st)
{
    if (a.D == 4 * LPR * CH) return launch2<LPR, CH, true>(ctx, a, st);
    return launch2<LPR, CH, false>(ctx, a, st);
}

}  // namespace

int dq_launch_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                  const float *scales, const int32_t *bits, float *out, int8_t *codes_out,
                  int B, int64_t L, cudaStream_t st)
{
    FwdArgs a{tables, ctx->d_row_off, indices, offsets, scales, bits, out, codes_out, ctx->T, ctx->D, B, L,
              ctx->d_status};
    const int d4 = ctx->D / 4;
    if (d4 <= 1) return launch<1, 1>(ctx, a, st);
    if (d4 <= 2) return launch<2, 1>(ctx, a, st);
    if (d4 <= 4) return launch<4, 1>(ctx, a, st);
    if (d4 <= 8) return launch<8, 1>(ctx, a, st);
    if (d4 <= 16) return launch<16, 1>(ctx, a, st);
    if (d4 <= 32) return launch<32, 1>(ctx, a, st);
    if (d4 <= 64) return launch<32, 2>(ctx, a, st);
    if (d4 <= 128) return launch<32, 4>(ctx, a, st);
    return launch<32, 8>(ctx, a, st);
}
