// Data-parallel exchange of the sparse INT8 gradient, local half (paper Appendix B.1): after
// the ranks' (unique rows, INT8 codes) have been gathered, sum the integer gradients of every
// row over the ranks and apply the dequantised sum to the FP32 master rows.  The integers
// are summed exactly in 32 bits, so the result does not depend on the order of the ranks and
// no value is re-rounded on the way (the concern the paper raises for recursive-doubling
// all-reduce).  Every replica runs this on the same gathered data and stays identical.
//
//   dp_pack_kernel        turns the W per-rank row lists into one table-major index list with
//                         bags of at most 64 entries (the layout the backward's sort takes) and
//                         remembers where each entry's codes live
//   (sort + seg_emit)     the backward's index sort, with the entry's position as payload:
//                         gives the ascending union of rows per table and each row's entries
//   dp_sum_update_kernel  one lane group per union row: adds the (at most W) code rows in int32,
//                         dequantises with the unified scale, updates the master row
#include "common.cuh"

namespace {

constexpr int DP_BAG = 64;       // entries per artificial bag

struct DpLayout {
    int64_t Bp;                  // bags per table
    size_t indices, offsets, src, sort_ws, total;
};

DpLayout dp_layout(const dqrm_ctx *ctx, int64_t n_entries, int64_t max_table_entries)
{
    DpLayout y;
    y.Bp = (max_table_entries + DP_BAG - 1) / DP_BAG;
    if (y.Bp < 1) y.Bp = 1;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const int64_t n = n_entries < 1 ? 1 : n_entries;
    y.indices = take(sizeof(int32_t) * n);
    y.offsets = take(sizeof(int32_t) * ((int64_t)ctx->T * y.Bp + 1));
    y.src = take(sizeof(u32) * n);
    y.sort_ws = o;
    y.total = o + dq_bwd_ws_bytes(ctx, n_entries, (int64_t)ctx->T * y.Bp);
    return y;
}

// one block per table
__global__ void __launch_bounds__(256)
dp_pack_kernel(int W, int T, int64_t rank_stride, int64_t Bp, const int32_t *__restrict__ rows_cat,
               const int32_t *__restrict__ uoff_cat, int32_t *__restrict__ indices, int32_t *__restrict__ offsets,
               u32 *__restrict__ src)
{
    const int t = blockIdx.x;
    // entries of all ranks in the tables before t, and of this table
    __shared__ int64_t s_base, s_n;
    if (threadIdx.x == 0) {
        int64_t base = 0, n = 0;
        for (int r = 0; r < W; ++r) {
            const int32_t *uo = uoff_cat + (int64_t)r * (T + 1);
            base += uo[t] - uo[0];
            n += uo[t + 1] - uo[t];
        }
        s_base = base;
        s_n = n;
    }
    __syncthreads();
    const int64_t base = s_base, n = s_n;
    // artificial bags of DP_BAG entries; the remaining bags of the table are empty
    for (int64_t i = threadIdx.x; i < Bp; i += blockDim.x)
        offsets[(int64_t)t * Bp + i] = (int32_t)(base + min(n, i * DP_BAG));
    if (t == T - 1 && threadIdx.x == 0) offsets[(int64_t)T * Bp] = (int32_t)(base + n);
    // rank after rank
    int64_t at = base;
    for (int r = 0; r < W; ++r) {
        const int32_t *uo = uoff_cat + (int64_t)r * (T + 1);
        const int32_t lo = uo[t], hi = uo[t + 1];
        for (int32_t u = lo + threadIdx.x; u < hi; u += blockDim.x) {
            indices[at + (u - lo)] = rows_cat[(int64_t)r * rank_stride + u];
            src[at + (u - lo)] = (u32)((int64_t)r * rank_stride + u);
        }
        at += hi - lo;
    }
}

__device__ __forceinline__ int dp_table_of_row(const int32_t *uoff, int T, int64_t u)
{
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (uoff[mid] <= u) lo = mid; else hi = mid;
    }
    return lo;
}

template <int LPR, int CH>
__global__ void __launch_bounds__(256)
dp_sum_update_kernel(float *__restrict__ tables, const int64_t *__restrict__ row_off,
                     const int32_t *__restrict__ union_rows, const int32_t *__restrict__ union_off,
                     const u32 *__restrict__ seg_start, const u32 *__restrict__ vals, const u32 *__restrict__ src,
                     const int8_t *__restrict__ codes_cat, const float *__restrict__ grad_scales, float lr,
                     int32_t *__restrict__ sums_out, int T, int D, int64_t n_src, float2 *__restrict__ row_summary)
{
    extern __shared__ unsigned char smem_raw[];
    int32_t *s_uoff = reinterpret_cast<int32_t *>(smem_raw);
    for (int t = threadIdx.x; t <= T; t += blockDim.x) s_uoff[t] = union_off[t];
    __syncthreads();
    const int d4 = D >> 2;
    const int64_t U = s_uoff[T];
    const int lane = threadIdx.x % LPR;
    const int64_t group = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t)gridDim.x * blockDim.x / LPR;
    int cur_t = -1;
    int64_t cur_end = -1, r0 = 0;
    float s = 1.f;
    for (int64_t u = group; u < U; u += n_groups) {
        if (u >= cur_end) {
            cur_t = dp_table_of_row(s_uoff, T, u);
            cur_end = s_uoff[cur_t + 1];
            r0 = __ldg(row_off + cur_t);
            s = __ldg(grad_scales + cur_t);
        }
        const u32 a = seg_start[u], e = seg_start[u + 1];
        int acc[CH][4];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) acc[ch][0] = acc[ch][1] = acc[ch][2] = acc[ch][3] = 0;
        for (u32 i = a; i < e; ++i) {                      // at most one entry per rank
            const u32 pos = vals[i];
            const int64_t ent = (int64_t)src[pos];
            if (ent >= n_src) continue;                    // (cannot happen with consistent inputs)
#pragma unroll
            for (int ch = 0; ch < CH; ++ch) {
                const int c4 = ch * LPR + lane;
                if (c4 < d4) {
                    const char4 c = *reinterpret_cast<const char4 *>(codes_cat + ent * D + 4 * c4);
                    acc[ch][0] += c.x; acc[ch][1] += c.y; acc[ch][2] += c.z; acc[ch][3] += c.w;
                }
            }
        }
        const int64_t arena_row = r0 + __ldg(union_rows + u);
        float4 *wrow = reinterpret_cast<float4 *>(tables + arena_row * D);
        float row_mn = __int_as_float(0x7f800000), row_mx = __int_as_float(0xff800000);
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
            const int c4 = ch * LPR + lane;
            if (c4 < d4) {
                if (sums_out)
                    *reinterpret_cast<int4 *>(sums_out + u * D + 4 * c4) = make_int4(acc[ch][0], acc[ch][1], acc[ch][2], acc[ch][3]);
                float4 x = wrow[c4];
                x.x = __fsub_rn(x.x, __fmul_rn(lr, __fmul_rn((float)acc[ch][0], s)));
                x.y = __fsub_rn(x.y, __fmul_rn(lr, __fmul_rn((float)acc[ch][1], s)));
                x.z = __fsub_rn(x.z, __fmul_rn(lr, __fmul_rn((float)acc[ch][2], s)));
                x.w = __fsub_rn(x.w, __fmul_rn(lr, __fmul_rn((float)acc[ch][3], s)));
                wrow[c4] = x;
                row_mn = fminf(row_mn, fminf(fminf(x.x, x.y), fminf(x.z, x.w)));
                row_mx = fmaxf(row_mx, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));
            }
        }
        if (row_summary) dq_store_row_minmax<LPR>(row_summary, arena_row, row_mn, row_mx);   // (uniform per lane group)
    }
}

template <int LPR, int CH>
int launch_sum_update(dqrm_ctx *ctx, float *tables, const int32_t *union_rows, const int32_t *union_off,
                      const u32 *seg_start, const u32 *vals, const u32 *src, const int8_t *codes_cat,
                      const float *grad_scales, float lr, int32_t *sums_out, int64_t n_src, cudaStream_t st)
{
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int32_t);
    dp_sum_update_kernel<LPR, CH><<<ctx->num_sms * 8, 256, smem, st>>>(tables, ctx->d_row_off, union_rows, union_off,
                                                                       seg_start, vals, src, codes_cat, grad_scales, lr,
                                                                       sums_out, ctx->T, ctx->D, n_src,
                                                                       ctx->row_summary);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_DP_SUM_UPDATE);
    return DQRM_OK;
}

}  // namespace

// exposed by bwd.cu for this file: where the sorted payloads and the segment starts live in the sort workspace
void dq_bwd_ws_views(const dqrm_ctx *ctx, int64_t L, char *ws, const u32 **sorted_vals, const u32 **seg_start);

size_t dq_dp_ws_bytes(const dqrm_ctx *ctx, int64_t max_entries)
{
    return dp_layout(ctx, max_entries, max_entries).total;
}

int dq_launch_dp_merge_update(dqrm_ctx *ctx, float *tables, int W, int64_t rank_stride, const int32_t *rows_cat,
                              const int32_t *uoff_cat, const int8_t *codes_cat, const float *grad_scales, float lr,
                              int64_t n_entries, int64_t max_table_entries, int32_t *union_rows, int32_t *union_off,
                              int32_t *sums_out, void *ws_, size_t ws_bytes, cudaStream_t st)
{
    const DpLayout y = dp_layout(ctx, n_entries, max_table_entries);
    if (ws_bytes < y.total) return DQRM_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(ws_);
    int32_t *indices = reinterpret_cast<int32_t *>(ws + y.indices);
    int32_t *offsets = reinterpret_cast<int32_t *>(ws + y.offsets);
    u32 *src = reinterpret_cast<u32 *>(ws + y.src);
    dp_pack_kernel<<<ctx->T, 256, 0, st>>>(W, ctx->T, rank_stride, y.Bp, rows_cat, uoff_cat, indices, offsets, src);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_DP_PACK);
    ctx->payload_position = 1;
    int rc = dq_launch_bwd_sort(ctx, indices, offsets, union_rows, union_off, (int)y.Bp, n_entries, ws + y.sort_ws,
                                ws_bytes - y.sort_ws, st, nullptr);
    ctx->payload_position = 0;
    if (rc != DQRM_OK) return rc;
    if (n_entries == 0) return DQRM_OK;
    const u32 *svals = nullptr, *seg_start = nullptr;
    dq_bwd_ws_views(ctx, n_entries, ws + y.sort_ws, &svals, &seg_start);
    const int64_t n_src = (int64_t)W * rank_stride;
    const int d4 = ctx->D / 4;
#define DQ_DP(LPR, CH) \
    return launch_sum_update<LPR, CH>(ctx, tables, union_rows, union_off, seg_start, svals, src, codes_cat, grad_scales, \
                                      lr, sums_out, n_src, st)
    if (d4 <= 1) DQ_DP(1, 1);
    if (d4 <= 2) DQ_DP(2, 1);
    if (d4 <= 4) DQ_DP(4, 1);
    if (d4 <= 8) DQ_DP(8, 1);
    if (d4 <= 16) DQ_DP(16, 1);
    if (d4 <= 32) DQ_DP(32, 1);
    if (d4 <= 64) DQ_DP(32, 2);
    if (d4 <= 128) DQ_DP(32, 4);
    DQ_DP(32, 8);
#undef DQ_DP
}
