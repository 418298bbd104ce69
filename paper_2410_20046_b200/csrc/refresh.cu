// Scale refresh (paper Section 3.2): one streaming pass over the whole arena that finds
// every table's min and max and turns them into the table's quantisation scale.
//
// The pass is HBM-bound: 4 bytes read per element, nothing written.  The arena is cut
// into 64 KB chunks that a persistent grid strides over; a chunk that lies inside one
// table (all but at most T-1 of them) is reduced with 128-bit streaming loads and one
// warp reduction, a chunk that straddles tables looks the table up per 16-byte vector.
// min/max are exact and order-independent, so the result is bit-identical to a
// sequential scan.  The last block to finish folds the per-block partials and writes
// the scales (no second launch, no inter-block wait).
#include "common.cuh"

namespace {

constexpr int RF_THREADS = 512;
constexpr int RF_UNROLL = 8;
constexpr int RF_CHUNK4 = RF_THREADS * RF_UNROLL;   // vectors per chunk (64 KB of float4)

// What one vector contributes: a float4 of table elements its smallest and largest element, a float2 of
// the per-row summary (min, max of one row) its two fields.
__device__ __forceinline__ float vec_min(const float4 &v) { return fminf(fminf(v.x, v.y), fminf(v.z, v.w)); }
__device__ __forceinline__ float vec_max(const float4 &v) { return fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)); }
__device__ __forceinline__ float vec_min(const float2 &v) { return v.x; }
__device__ __forceinline__ float vec_max(const float2 &v) { return v.y; }

// order-preserving map float -> uint32 (so that unsigned min/max order like the floats)
__device__ __forceinline__ u32 f2ord(float f)
{
    u32 b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord2f(u32 o)
{
    u32 b = (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o;
    return __uint_as_float(b);
}

// V = float4: arena4 is the arena of tables, d4 = D/4 vectors per row.  V = float2: arena4 is the per-row
// summary, d4 = 1.
template <typename V>
__global__ void __launch_bounds__(RF_THREADS)
refresh_kernel(const V *__restrict__ arena4, const int64_t *__restrict__ row_off, int T, int d4,
               int64_t n4, const int32_t *__restrict__ bits, float *__restrict__ scales,
               float *__restrict__ minmax, u32 *__restrict__ partials /*[grid][T][2]*/,
               u32 *__restrict__ done)
{
    extern __shared__ unsigned char smem_raw[];
    int64_t *v4_off = reinterpret_cast<int64_t *>(smem_raw);             // [T+1] table starts in float4 units
    u32 *s_min = reinterpret_cast<u32 *>(v4_off + (T + 1));              // [T]
    u32 *s_max = s_min + T;                                              // [T]
    __shared__ bool is_last;

    for (int t = threadIdx.x; t <= T; t += RF_THREADS) v4_off[t] = row_off[t] * d4;
    for (int t = threadIdx.x; t < T; t += RF_THREADS) { s_min[t] = 0xFFFFFFFFu; s_max[t] = 0u; }
    __syncthreads();

    const int64_t n_chunks = (n4 + RF_CHUNK4 - 1) / RF_CHUNK4;
    const int lane = threadIdx.x & 31;
    for (int64_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const int64_t c0 = c * RF_CHUNK4;
        const int64_t c1 = min(c0 + (int64_t)RF_CHUNK4, n4);
        const int t0 = dq_table_of(v4_off, T, c0);
        if (c1 <= v4_off[t0 + 1]) {
            // whole chunk inside table t0
            V v[RF_UNROLL];
#pragma unroll
            for (int k = 0; k < RF_UNROLL; ++k) {
                int64_t i = c0 + k * RF_THREADS + threadIdx.x;
                if (i < c1) v[k] = __ldcs(arena4 + i);
                else v[k] = V();                                                      // skipped below
            }
            float mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);   // +inf, -inf
#pragma unroll
            for (int k = 0; k < RF_UNROLL; ++k) {
                int64_t i = c0 + k * RF_THREADS + threadIdx.x;
                if (i < c1) {
                    mn = fminf(mn, vec_min(v[k]));
                    mx = fmaxf(mx, vec_max(v[k]));
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            }
            if (lane == 0 && mn <= mx) {
                atomicMin(&s_min[t0], f2ord(mn));
                atomicMax(&s_max[t0], f2ord(mx));
            }
        } else {
            // chunk straddles a table boundary (at most T-1 such chunks in the arena)
            for (int64_t i = c0 + threadIdx.x; i < c1; i += RF_THREADS) {
                V v = __ldcs(arena4 + i);
                int t = dq_table_of(v4_off, T, i);
                float mn = vec_min(v), mx = vec_max(v);
                if (mn <= mx) {
                    atomicMin(&s_min[t], f2ord(mn));
                    atomicMax(&s_max[t], f2ord(mx));
                }
            }
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < T; t += RF_THREADS) {
        partials[((size_t)blockIdx.x * T + t) * 2 + 0] = s_min[t];
        partials[((size_t)blockIdx.x * T + t) * 2 + 1] = s_max[t];
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        u32 prev = atomicAdd(done, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // last block: fold the partials of all blocks, one warp per table
    const int warp = threadIdx.x >> 5, n_warps = RF_THREADS >> 5;
    for (int t = warp; t < T; t += n_warps) {
        u32 mn = 0xFFFFFFFFu, mx = 0u;
        for (int b = lane; b < (int)gridDim.x; b += 32) {
            mn = min(mn, __ldcg(&partials[((size_t)b * T + t) * 2 + 0]));
            mx = max(mx, __ldcg(&partials[((size_t)b * T + t) * 2 + 1]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        if (lane == 0) {
            float fmn = ord2f(mn), fmx = ord2f(mx);
            float a = fmaxf(fabsf(fmn), fabsf(fmx));
            scales[t] = dq_scale_from_absmax(a, bits[t]);
            if (minmax) { minmax[2 * t] = fmn; minmax[2 * t + 1] = fmx; }
        }
    }
    if (threadIdx.x == 0) *done = 0u;   // ready for the next call on this context
}

int refresh_grid(const dqrm_ctx *ctx) { return ctx->num_sms * 4; }

}  // namespace

size_t dq_refresh_ws_bytes(const dqrm_ctx *ctx)
{
    return align_up((size_t)refresh_grid(ctx) * ctx->T * 2 * sizeof(u32), 256);
}

int dq_launch_refresh(dqrm_ctx *ctx, const float *tables, const int32_t *bits, float *scales,
                      float *minmax, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (ws_bytes < dq_refresh_ws_bytes(ctx)) return DQRM_ERR_WORKSPACE;
    const int grid = refresh_grid(ctx);
    size_t smem = (size_t)(ctx->T + 1) * sizeof(int64_t) + (size_t)ctx->T * 2 * sizeof(u32);
    if (ctx->row_summary) {
        // every row's (min, max) is kept current by the update kernels: 8 bytes per row are read, not 4*D
        refresh_kernel<float2><<<grid, RF_THREADS, smem, st>>>(ctx->row_summary, ctx->d_row_off, ctx->T, 1,
                                                               ctx->total_rows, bits, scales, minmax,
                                                               reinterpret_cast<u32 *>(ws), ctx->d_done);
    } else {
        const int64_t n4 = ctx->total_rows * (ctx->D / 4);
        refresh_kernel<float4><<<grid, RF_THREADS, smem, st>>>(reinterpret_cast<const float4 *>(tables), ctx->d_row_off,
                                                               ctx->T, ctx->D / 4, n4, bits, scales, minmax,
                                                               reinterpret_cast<u32 *>(ws), ctx->d_done);
    }
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_REFRESH);
    return DQRM_OK;
}

namespace {

// (min, max) of every row of the arena, a lane group per row
__global__ void __launch_bounds__(256)
row_summary_kernel(const float4 *__restrict__ arena4, int d4, int lpr, int64_t total_rows, float2 *__restrict__ summary)
{
    const int lane = threadIdx.x % lpr;
    const int64_t group = ((int64_t)blockIdx.x * 256 + threadIdx.x) / lpr;
    const int64_t n_groups = (int64_t)gridDim.x * 256 / lpr;
    const unsigned lane_w = threadIdx.x & 31;
    const unsigned mask = lpr == 32 ? 0xffffffffu : (((1u << lpr) - 1u) << (lane_w / lpr * lpr));
    for (int64_t r = group; r < total_rows; r += n_groups) {
        float mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);
        for (int c = lane; c < d4; c += lpr) {
            const float4 v = __ldcs(arena4 + r * d4 + c);
            mn = fminf(mn, vec_min(v));
            mx = fmaxf(mx, vec_max(v));
        }
        for (int o = lpr >> 1; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(mask, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(mask, mx, o));
        }
        if (lane == 0) summary[r] = make_float2(mn, mx);
    }
}

}  // namespace

int dq_launch_row_summary(dqrm_ctx *ctx, const float *tables, float2 *summary, cudaStream_t st)
{
    const int d4 = ctx->D / 4;
    int lpr = 1;
    while (lpr < d4 && lpr < 32) lpr <<= 1;
    row_summary_kernel<<<ctx->num_sms * 8, 256, 0, st>>>(reinterpret_cast<const float4 *>(tables), d4, lpr,
                                                         ctx->total_rows, summary);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_REFRESH);
    return DQRM_OK;
}
