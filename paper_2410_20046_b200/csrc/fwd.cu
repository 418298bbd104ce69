// Forward of the quantisation-aware embedding lookup (paper Section 3.1, Figure 2(b)):
// gather the rows a batch uses from the FP32 master table, fake-quantise each gathered
// row with the table's stored scale, and sum-pool over the bag.  No low-precision copy
// of the table exists; only the gathered rows are ever quantised.
//
// HBM-bound random row gather: throughput is set by how many row requests an SM keeps
// in flight.  Rows therefore travel global -> shared memory with 16-byte asynchronous
// copies (cp.async), two batches deep, so the bytes in flight cost no registers and the
// occupancy stays high; every thread reads back exactly the 16-byte pieces it copied, so
// no block barrier is needed.  blockIdx.y is the table, which makes scale, bit width and
// row base block constants.  A group of LPR lanes owns one row: a feature-16 row is one
// 64-byte request of four lanes, a feature-64 row one 256-byte request of sixteen.
//   * fwd_onehot_kernel (launched when L == T*B, the Criteo-shaped case): a group has
//     NB rows of NB different one-index bags in flight per batch; the pooled value is
//     the fake-quantised row itself.  A bag that turns out not to hold exactly one index
//     takes the general routine.
//   * fwd_bags_kernel (any other batch): a group walks one bag at a time, NB of its rows
//     per batch, and sums them in bag order in FP64, rounded once, so the result does
//     not depend on the launch shape.
#include "common.cuh"

namespace {

constexpr int FW_THREADS = 256;
constexpr int FW_STAGES = 2;      // batches in flight
// rows per lane group per batch: four for rows of up to 128 features, fewer for wider rows so
// that the staging buffer stays at 32 KB per block (64 KB beyond 512 features)
template <int CH>
struct NBOf { static constexpr int v = CH >= 4 ? 1 : (CH == 2 ? 2 : 4); };

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

__device__ __forceinline__ float4 fq4(const float4 &v, const QuantScale &qs, float4 &codes)
{
    float4 deq;
    dq_fq4(v, qs, codes, deq);
    return deq;
}

__device__ __forceinline__ void store_codes(int8_t *codes_out, int64_t j, int D, int c4, const float4 &c)
{
    char4 cc = make_char4((signed char)(int)c.x, (signed char)(int)c.y, (signed char)(int)c.z, (signed char)(int)c.w);
    *reinterpret_cast<char4 *>(codes_out + j * D + 4 * c4) = cc;
}

__device__ __forceinline__ int32_t checked_index(int32_t idx, int64_t nrows, int *status)
{
    if (idx < 0 || idx >= nrows) {
        dq_report(status, DQRM_ERR_INDEX_RANGE);
        idx = idx < 0 ? 0 : (int32_t)(nrows - 1);
    }
    return idx;
}

// thread-private slot of the staging buffer: [stage][row-in-batch][vector][thread]
template <int CH>
__device__ __forceinline__ float4 *slot(float4 *buf, int stage, int b, int c)
{
    return buf + ((size_t)((stage * NBOf<CH>::v + b) * CH + c)) * FW_THREADS + threadIdx.x;
}

// one bag: NB of its rows per batch, FP64 sum in bag order
template <int LPR, int CH>
__device__ __forceinline__ void pool_bag(const FwdArgs &a, const float *tbl, int64_t nrows, const QuantScale &qs,
                                         int32_t lo, int32_t hi, float *out_row, int lane, float4 *buf)
{
    const int d4 = a.D >> 2;
    if (lo < 0 || hi < lo || (int64_t)hi > a.L) { dq_report(a.status, DQRM_ERR_INDEX_RANGE); hi = lo = 0; }
    double acc[CH][4];
#pragma unroll
    for (int c = 0; c < CH; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.0;

    auto issue = [&](int32_t j0, int stage) {
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) {
            if (j0 + b < hi) {
                const int32_t idx = checked_index(__ldg(a.indices + j0 + b), nrows, a.status);
                const float4 *row = reinterpret_cast<const float4 *>(tbl + (int64_t)idx * a.D);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int c4 = c * LPR + lane;
                    if (c4 < d4) dq_cp_async16(slot<CH>(buf, stage, b, c), row + c4);
                }
            }
        }
        dq_cp_async_commit();
    };

    int stage = 0;
    if (lo < hi) issue(lo, 0);
    for (int32_t j0 = lo; j0 < hi; j0 += NBOf<CH>::v) {
        if (j0 + NBOf<CH>::v < hi) { issue(j0 + NBOf<CH>::v, stage ^ 1); dq_cp_async_wait<1>(); }
        else dq_cp_async_wait<0>();
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) {
            if (j0 + b < hi) {
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int c4 = c * LPR + lane;
                    if (c4 < d4) {
                        float4 cd;
                        const float4 f = fq4(*slot<CH>(buf, stage, b, c), qs, cd);
                        acc[c][0] += (double)f.x;
                        acc[c][1] += (double)f.y;
                        acc[c][2] += (double)f.z;
                        acc[c][3] += (double)f.w;
                        if (a.codes_out) store_codes(a.codes_out, j0 + b, a.D, c4, cd);
                    }
                }
            }
        }
        stage ^= 1;
    }
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        const int c4 = c * LPR + lane;
        if (c4 < d4)
            reinterpret_cast<float4 *>(out_row)[c4] =
                make_float4((float)acc[c][0], (float)acc[c][1], (float)acc[c][2], (float)acc[c][3]);
    }
}

template <int LPR, int CH>
__device__ __noinline__ void pool_bag_rare(const FwdArgs &a, const float *tbl, int64_t nrows, const QuantScale &qs,
                                           int32_t lo, int32_t hi, float *out_row, int lane, float4 *buf)
{
    pool_bag<LPR, CH>(a, tbl, nrows, qs, lo, hi, out_row, lane, buf);
}

template <int LPR, int CH>
__global__ void __launch_bounds__(FW_THREADS, 4)
fwd_onehot_kernel(const FwdArgs a)
{
    extern __shared__ float4 s_buf[];            // [FW_STAGES][NBOf<CH>::v][CH][FW_THREADS]
    constexpr int GPB = FW_THREADS / LPR;
    constexpr int TILE = GPB * NBOf<CH>::v;            // bags per block per batch
    const int t = blockIdx.y;
    const int d4 = a.D >> 2;
    const int lane = threadIdx.x % LPR;
    const int grp = threadIdx.x / LPR;
    const QuantScale qs = dq_make_scale(__ldg(a.scales + t), __ldg(a.bits + t));
    const int64_t r0 = __ldg(a.row_off + t);
    const int64_t nrows = __ldg(a.row_off + t + 1) - r0;
    const float *tbl = a.tables + r0 * a.D;
    const int64_t g0 = (int64_t)t * a.B;

    // state of one batch: offsets of its NB bags and which of them hold exactly one index
    struct Batch { int32_t lo[NBOf<CH>::v], hi[NBOf<CH>::v]; unsigned one; };

    auto issue = [&](int ib, int stage, Batch &bt) {
        int32_t idx[NBOf<CH>::v];
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) {
            const int i = ib + b * GPB + grp;
            bt.lo[b] = 0; bt.hi[b] = 0; idx[b] = 0;
            if (i < a.B) {
                bt.lo[b] = __ldg(a.offsets + g0 + i);
                bt.hi[b] = __ldg(a.offsets + g0 + i + 1);
                idx[b] = __ldg(a.indices + g0 + i);          // right when offsets are the identity (L == T*B)
            }
        }
        bt.one = 0;
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) {
            const int i = ib + b * GPB + grp;
            if (i < a.B && bt.hi[b] - bt.lo[b] == 1 && bt.lo[b] >= 0 && (int64_t)bt.hi[b] <= a.L) {
                if ((int64_t)bt.lo[b] != g0 + i) idx[b] = __ldg(a.indices + bt.lo[b]);
                idx[b] = checked_index(idx[b], nrows, a.status);
                bt.one |= 1u << b;
                const float4 *row = reinterpret_cast<const float4 *>(tbl + (int64_t)idx[b] * a.D);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int c4 = c * LPR + lane;
                    if (c4 < d4) dq_cp_async16(slot<CH>(s_buf, stage, b, c), row + c4);
                }
            }
        }
        dq_cp_async_commit();
    };

    const int step = gridDim.x * TILE;
    int ib = blockIdx.x * TILE;
    if (ib >= a.B) return;
    Batch cur, nxt;
    int stage = 0;
    issue(ib, 0, cur);
    for (; ib < a.B; ib += step) {
        const bool more = ib + step < a.B;
        if (more) { issue(ib + step, stage ^ 1, nxt); dq_cp_async_wait<1>(); }
        else dq_cp_async_wait<0>();
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) {
            const int i = ib + b * GPB + grp;
            if ((cur.one >> b) & 1u) {
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int c4 = c * LPR + lane;
                    if (c4 < d4) {
                        float4 cd;
                        const float4 f = fq4(*slot<CH>(s_buf, stage, b, c), qs, cd);
                        reinterpret_cast<float4 *>(a.out + ((int64_t)i * a.T + t) * a.D)[c4] = f;
                        if (a.codes_out) store_codes(a.codes_out, cur.lo[b], a.D, c4, cd);
                    }
                }
            }
        }
        bool rare = false;
#pragma unroll
        for (int b = 0; b < NBOf<CH>::v; ++b) rare |= (ib + b * GPB + grp < a.B) && !((cur.one >> b) & 1u);
        if (rare) {
            // bags of this batch that are empty, multi-index or out of range: the general routine
            // reuses this thread's staging slots of both stages, so the prefetched batch is re-issued
            dq_cp_async_wait<0>();
#pragma unroll
            for (int b = 0; b < NBOf<CH>::v; ++b) {
                const int i = ib + b * GPB + grp;
                if (i < a.B && !((cur.one >> b) & 1u))
                    pool_bag_rare<LPR, CH>(a, tbl, nrows, qs, cur.lo[b], cur.hi[b],
                                           a.out + ((int64_t)i * a.T + t) * a.D, lane, s_buf);
            }
            if (more) issue(ib + step, stage ^ 1, nxt);
        }
        cur = nxt;
        stage ^= 1;
    }
}

template <int LPR, int CH>
__global__ void __launch_bounds__(FW_THREADS)
fwd_bags_kernel(const FwdArgs a)
{
    extern __shared__ float4 s_buf[];
    constexpr int GPB = FW_THREADS / LPR;
    const int t = blockIdx.y;
    const int lane = threadIdx.x % LPR;
    const int grp = threadIdx.x / LPR;
    const QuantScale qs = dq_make_scale(__ldg(a.scales + t), __ldg(a.bits + t));
    const int64_t r0 = __ldg(a.row_off + t);
    const int64_t nrows = __ldg(a.row_off + t + 1) - r0;
    const float *tbl = a.tables + r0 * a.D;
    const int64_t g0 = (int64_t)t * a.B;
    for (int i = blockIdx.x * GPB + grp; i < a.B; i += gridDim.x * GPB) {
        const int32_t lo = __ldg(a.offsets + g0 + i), hi = __ldg(a.offsets + g0 + i + 1);
        pool_bag<LPR, CH>(a, tbl, nrows, qs, lo, hi, a.out + ((int64_t)i * a.T + t) * a.D, lane, s_buf);
    }
}

template <int LPR, int CH>
int launch(dqrm_ctx *ctx, const FwdArgs &a, cudaStream_t st)
{
    constexpr int GPB = FW_THREADS / LPR;
    constexpr size_t SMEM = sizeof(float4) * FW_STAGES * NBOf<CH>::v * CH * FW_THREADS;   // 32 KB * CH
    static bool raised = false;
    if (SMEM > 48 * 1024 && !raised) {
        DQRM_CUDA_TRY(ctx, cudaFuncSetAttribute(fwd_onehot_kernel<LPR, CH>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM));
        DQRM_CUDA_TRY(ctx, cudaFuncSetAttribute(fwd_bags_kernel<LPR, CH>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM));
        raised = true;
    }
    const bool onehot = a.L == (int64_t)a.T * a.B;
    const int per_block = onehot ? GPB * NBOf<CH>::v : GPB;
    int bx = (a.B + per_block - 1) / per_block;
    const int cap = (ctx->num_sms * 32 + ctx->T - 1) / ctx->T;     // a few waves over all tables
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)ctx->T);
    if (onehot) fwd_onehot_kernel<LPR, CH><<<grid, FW_THREADS, SMEM, st>>>(a);
    else fwd_bags_kernel<LPR, CH><<<grid, FW_THREADS, SMEM, st>>>(a);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_FWD);
    return DQRM_OK;
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
