// Row-streaming core of the INT8 gradient quantiser and the touched-row SGD update
// (paper Appendix B.1 and Section 3.1): quantise only, update only (from stored codes), or
// quantise + update fused.  A group of LPR lanes owns a contiguous range of unique rows and
// keeps a few of them in flight; rows are distinct, so the read-modify-write of the master
// rows needs no atomics.  All streams are 128-bit per lane.  Shared by the stand-alone
// kernels and by the kernel that ends a training step.
#pragma once
#include "common.cuh"

namespace rowstream {

constexpr int QU_THREADS = 256;
enum { MODE_QUANT = 0, MODE_UPDATE = 1, MODE_FUSED = 2 };

// largest t with uoff[t] <= u, skipping empty tables
__device__ __forceinline__ int table_of_row(const int32_t *uoff, int T, int64_t u)
{
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (uoff[mid] <= u) lo = mid; else hi = mid;
    }
    return lo;
}

// rows in flight per lane group: fewer when a lane already holds several vectors of every row
template <int CH> struct RowsInFlight { static constexpr int v = CH >= 4 ? 1 : (CH == 2 ? 2 : 4); };

// EXACT: the feature size is 4*LPR*CH, a compile-time constant, and the per-vector range checks fall away
inline size_t smem_bytes(int T) { return (size_t)(T + 1) * sizeof(int32_t) + (size_t)T * sizeof(float); }

// smem_raw: smem_bytes(T) bytes of shared memory; every thread of the block calls this
// TRACK: the (min, max) of every row written is stored in row_summary[arena row] as well
template <int MODE, int LPR, int CH, bool EXACT, bool TRACK = false>
__device__ __forceinline__ void
row_stream_body(unsigned char *smem_raw, float *__restrict__ tables, const int64_t *__restrict__ row_off,
                const int32_t *__restrict__ unique_rows, const int32_t *__restrict__ uniq_off,
                const float *__restrict__ grad_rows, const u32 *__restrict__ absmax,
                int8_t *__restrict__ codes, float *__restrict__ grad_scales, float lr, int T, int D_any,
                int *__restrict__ status, float2 *__restrict__ row_summary = nullptr)
{
    constexpr int NB = RowsInFlight<CH>::v;
    const int D = EXACT ? 4 * LPR * CH : D_any;
    int32_t *s_uoff = reinterpret_cast<int32_t *>(smem_raw);      // [T+1]
    float *s_scale = reinterpret_cast<float *>(s_uoff + (T + 1)); // [T] gradient scale of every table
    for (int t = threadIdx.x; t <= T; t += QU_THREADS) s_uoff[t] = uniq_off[t];
    for (int t = threadIdx.x; t < T; t += QU_THREADS) {
        const float sc = (MODE == MODE_UPDATE) ? grad_scales[t] : dq_scale_from_absmax(__uint_as_float(absmax[t]), 8);
        s_scale[t] = sc;
        if (MODE != MODE_UPDATE && blockIdx.x == 0) grad_scales[t] = sc;
    }
    __syncthreads();
    const int d4 = D >> 2;
    const int64_t U = s_uoff[T];
    const int lane = threadIdx.x % LPR;
    const int64_t group = ((int64_t)blockIdx.x * QU_THREADS + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t)gridDim.x * QU_THREADS / LPR;
    // a lane group owns a contiguous range of unique rows: its rows mostly share a table, and its reads
    // of the gradient rows and writes of the codes are sequential
    int64_t per = (U + n_groups - 1) / n_groups;
    if (per < NB) per = NB;             // few rows: fewer groups, each with a full set of rows in flight
    const int64_t u_begin = group * per, u_end = min(U, u_begin + per);
    int cur_t = -1;
    int64_t cur_end = -1, r0 = 0, nrows = 1;
    bool bad = false;
    float s = 1.f;
    QuantScale qs = dq_make_scale(1.f, 8);
    for (int64_t u = u_begin; u < u_end;) {
        if (u >= cur_end) {
            cur_t = table_of_row(s_uoff, T, u);
            cur_end = s_uoff[cur_t + 1];
            if (MODE != MODE_QUANT) { r0 = __ldg(row_off + cur_t); nrows = __ldg(row_off + cur_t + 1) - r0; }
            s = s_scale[cur_t];
            qs = dq_make_scale(s, 8);
        }
        // up to NB rows of the current table at once
        const int nb = (int)min((int64_t)NB, min(u_end, cur_end) - u);
        float4 *wrow[NB];
        float4 g[NB][CH], w[NB][CH];
        char4 cin[NB][CH];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            wrow[b] = nullptr;
            if (b < nb && MODE != MODE_QUANT) {
                // a row number outside its table is reported and kept inside the arena, never followed
                // (no branch: the rows' index loads stay in flight together)
                const int64_t row = __ldg(unique_rows + u + b);
                bad |= (row < 0) | (row >= nrows);
                wrow[b] = reinterpret_cast<float4 *>(tables + (r0 + min(max(row, (int64_t)0), nrows - 1)) * D);
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < nb) {
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int c4 = ch * LPR + lane;
                    if (EXACT || c4 < d4) {
                        if (MODE == MODE_UPDATE) cin[b][ch] = *reinterpret_cast<const char4 *>(codes + (u + b) * D + 4 * c4);
                        else g[b][ch] = __ldg(reinterpret_cast<const float4 *>(grad_rows + (u + b) * D) + c4);
                        if (MODE != MODE_QUANT) w[b][ch] = wrow[b][c4];
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < nb) {
                float row_mn = __int_as_float(0x7f800000), row_mx = __int_as_float(0xff800000);
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int c4 = ch * LPR + lane;
                    if (EXACT || c4 < d4) {
                        float4 q;                      // integer codes held as floats
                        if (MODE == MODE_UPDATE) {
                            q = make_float4((float)cin[b][ch].x, (float)cin[b][ch].y, (float)cin[b][ch].z, (float)cin[b][ch].w);
                        } else {
                            float4 dq_unused;
                            dq_fq4(g[b][ch], qs, q, dq_unused);
                            __stcs(reinterpret_cast<char4 *>(codes + (u + b) * D + 4 * c4),
                                   make_char4((signed char)(int)q.x, (signed char)(int)q.y, (signed char)(int)q.z,
                                              (signed char)(int)q.w));
                        }
                        if (MODE != MODE_QUANT) {
                            float4 x = w[b][ch];
                            x.x = __fsub_rn(x.x, __fmul_rn(lr, __fmul_rn(q.x, s)));
                            x.y = __fsub_rn(x.y, __fmul_rn(lr, __fmul_rn(q.y, s)));
                            x.z = __fsub_rn(x.z, __fmul_rn(lr, __fmul_rn(q.z, s)));
                            x.w = __fsub_rn(x.w, __fmul_rn(lr, __fmul_rn(q.w, s)));
                            wrow[b][c4] = x;
                            if (TRACK) {
                                row_mn = fminf(row_mn, fminf(fminf(x.x, x.y), fminf(x.z, x.w)));
                                row_mx = fmaxf(row_mx, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));
                            }
                        }
                    }
                }
                // (nb is the same in all lanes of a group, so all of them arrive here together)
                if (TRACK && MODE != MODE_QUANT)
                    dq_store_row_minmax<LPR>(row_summary, (reinterpret_cast<float *>(wrow[b]) - tables) / D, row_mn, row_mx);
            }
        }
        u += nb;
    }
    if (MODE != MODE_QUANT && bad) dq_report(status, DQRM_ERR_INDEX_RANGE);
}

}  // namespace rowstream
