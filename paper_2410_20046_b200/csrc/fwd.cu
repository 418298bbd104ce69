// Forward of the quantisation-aware embedding lookup (paper Section 3.1, Figure 2(b)):
// gather the rows a batch uses from the FP32 master table, fake-quantise each gathered
// row with the table's stored scale, and sum-pool over the bag.  No low-precision copy
// of the table exists; only the gathered rows are ever quantised.
//
// HBM-bound random row gather.  A group of LPR lanes owns one row (one 128-bit load per
// lane per 4 features), so a feature-16 row is one 64-byte request of four lanes and a
// feature-64 row one 256-byte request of sixteen.  Every group keeps NB bags in flight
// (index loads first, then the NB independent row loads) to cover DRAM latency.  Bags
// are summed in bag order in FP64 and rounded once, which makes the pooled output
// independent of the launch shape.
#include "common.cuh"

namespace {

constexpr int FW_THREADS = 256;

template <int LPR, int CH, int NB>
__global__ void __launch_bounds__(FW_THREADS)
fwd_kernel(const float *__restrict__ tables, const int64_t *__restrict__ row_off,
           const int32_t *__restrict__ indices, const int32_t *__restrict__ offsets,
           const float *__restrict__ scales, const int32_t *__restrict__ bits,
           float *__restrict__ out, int8_t *__restrict__ codes_out,
           int T, int D, int B, int64_t G, int64_t L, int *__restrict__ status)
{
    const int d4 = D >> 2;
    const int lane = threadIdx.x % LPR;
    const int64_t group = ((int64_t)blockIdx.x * FW_THREADS + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t)gridDim.x * FW_THREADS / LPR;

    for (int64_t gbase = 0; gbase < G; gbase += n_groups * NB) {
        int32_t lo[NB], len[NB];
        int tb[NB];
        int64_t bag[NB];
        int maxlen = 0;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            bag[b] = gbase + (int64_t)b * n_groups + group;
            lo[b] = 0; len[b] = -1; tb[b] = 0;
            if (bag[b] < G) {
                int32_t a = __ldg(offsets + bag[b]), e = __ldg(offsets + bag[b] + 1);
                if (a < 0 || e < a || (int64_t)e > L) { dq_report(status, DQRM_ERR_INDEX_RANGE); e = a = 0; }
                lo[b] = a; len[b] = e - a;
                tb[b] = (int)(bag[b] / B);
                maxlen = max(maxlen, len[b]);
            }
        }
        float s[NB], qlo[NB], qhi[NB];
        int64_t r0[NB], nrows[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            s[b] = __ldg(scales + tb[b]);
            int bt = __ldg(bits + tb[b]);
            qlo[b] = -(float)(1 << (bt - 1));
            qhi[b] = (float)((1 << (bt - 1)) - 1);
            r0[b] = __ldg(row_off + tb[b]);
            nrows[b] = __ldg(row_off + tb[b] + 1) - r0[b];
        }
        double acc[NB][CH][4];
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int c = 0; c < CH; ++c)
                acc[b][c][0] = acc[b][c][1] = acc[b][c][2] = acc[b][c][3] = 0.0;

        for (int k = 0; k < maxlen; ++k) {
            int32_t idx[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) idx[b] = (k < len[b]) ? __ldg(indices + lo[b] + k) : 0;
            float4 v[NB][CH];
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (k < len[b]) {
                    if (idx[b] < 0 || idx[b] >= nrows[b]) {
                        dq_report(status, DQRM_ERR_INDEX_RANGE);
                        idx[b] = idx[b] < 0 ? 0 : (int32_t)(nrows[b] - 1);
                    }
                    const float4 *row = reinterpret_cast<const float4 *>(tables + (r0[b] + idx[b]) * D);
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        int c4 = c * LPR + lane;
                        if (c4 < d4) v[b][c] = __ldg(row + c4);
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (k < len[b]) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        int c4 = c * LPR + lane;
                        if (c4 < d4) {
                            int q0 = dq_code(v[b][c].x, s[b], qlo[b], qhi[b]);
                            int q1 = dq_code(v[b][c].y, s[b], qlo[b], qhi[b]);
                            int q2 = dq_code(v[b][c].z, s[b], qlo[b], qhi[b]);
                            int q3 = dq_code(v[b][c].w, s[b], qlo[b], qhi[b]);
                            acc[b][c][0] += (double)dq_dequant(q0, s[b]);
                            acc[b][c][1] += (double)dq_dequant(q1, s[b]);
                            acc[b][c][2] += (double)dq_dequant(q2, s[b]);
                            acc[b][c][3] += (double)dq_dequant(q3, s[b]);
                            if (codes_out) {
                                char4 cc = make_char4((signed char)q0, (signed char)q1, (signed char)q2, (signed char)q3);
                                *reinterpret_cast<char4 *>(codes_out + (int64_t)(lo[b] + k) * D + 4 * c4) = cc;
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (len[b] >= 0) {
                int64_t smp = bag[b] - (int64_t)tb[b] * B;
                float4 *o = reinterpret_cast<float4 *>(out + (smp * T + tb[b]) * D);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    int c4 = c * LPR + lane;
                    if (c4 < d4)
                        o[c4] = make_float4((float)acc[b][c][0], (float)acc[b][c][1],
                                            (float)acc[b][c][2], (float)acc[b][c][3]);
                }
            }
        }
    }
}

template <int LPR, int CH, int NB>
int launch(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
           const float *scales, const int32_t *bits, float *out, int8_t *codes_out,
           int B, int64_t L, cudaStream_t st)
{
    const int64_t G = (int64_t)ctx->T * B;
    const int64_t groups_per_block = FW_THREADS / LPR;
    int64_t blocks = (G + groups_per_block * NB - 1) / (groups_per_block * NB);
    int64_t cap = (int64_t)ctx->num_sms * 8;
    int grid = (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
    fwd_kernel<LPR, CH, NB><<<grid, FW_THREADS, 0, st>>>(tables, ctx->d_row_off, indices, offsets, scales, bits,
                                                         out, codes_out, ctx->T, ctx->D, B, G, L, ctx->d_status);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_FWD);
    return DQRM_OK;
}

}  // namespace

int dq_launch_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                  const float *scales, const int32_t *bits, float *out, int8_t *codes_out,
                  int B, int64_t L, cudaStream_t st)
{
    const int d4 = ctx->D / 4;
#define DQ_FWD(LPR, CH, NB) return launch<LPR, CH, NB>(ctx, tables, indices, offsets, scales, bits, out, codes_out, B, L, st)
    if (d4 <= 1) DQ_FWD(1, 1, 4);
    if (d4 <= 2) DQ_FWD(2, 1, 4);
    if (d4 <= 4) DQ_FWD(4, 1, 4);
    if (d4 <= 8) DQ_FWD(8, 1, 4);
    if (d4 <= 16) DQ_FWD(16, 1, 4);
    if (d4 <= 32) DQ_FWD(32, 1, 4);
    if (d4 <= 64) DQ_FWD(32, 2, 2);
    if (d4 <= 128) DQ_FWD(32, 4, 1);
    DQ_FWD(32, 8, 1);
#undef DQ_FWD
}
