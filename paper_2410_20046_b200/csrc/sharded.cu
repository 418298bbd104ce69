// Table-sharded forward (paper Section 4.3, the remark on hybrid parallelism: the all-to-all that
// carries embedding vectors shrinks with the code width).  The rank that owns a table gathers the
// rows a one-index batch looks up, quantises them and emits the b-bit codes bit-packed (layout of
// the packed tables: element d in byte (d*b)/8 at bit offset (d*b)%8, two's complement), 32/b times
// fewer bytes than the FP32 vectors; the rank that owns the samples multiplies the codes by the
// table's scale.  Together the two kernels give exactly the training forward.
//
// fwd_codes_kernel       a warp owns 32 consecutive bags of one table: one lane per bag does the
//                        bookkeeping, the rows are then fetched 32/LPR per step (one 128-bit load per
//                        lane), quantised with the division-free quantiser and written as b/2 bytes
//                        per lane
// decode_payload_kernel  streaming: one thread per 128-bit output vector
#include "common.cuh"

namespace {

constexpr int SH_THREADS = 256;

template <int BITS>
__device__ __forceinline__ u32 pack4(const float4 &codes)
{
    const u32 m = (1u << BITS) - 1u;
    return ((u32)(int)codes.x & m) | (((u32)(int)codes.y & m) << BITS) | (((u32)(int)codes.z & m) << (2 * BITS)) |
           (((u32)(int)codes.w & m) << (3 * BITS));
}

template <int BITS>
__device__ __forceinline__ void store_quad(uint8_t *dst, int64_t v4, u32 bits4)
{
    if constexpr (BITS == 2) dst[v4] = (uint8_t)bits4;
    else if constexpr (BITS == 4) reinterpret_cast<uint16_t *>(dst)[v4] = (uint16_t)bits4;
    else reinterpret_cast<u32 *>(dst)[v4] = bits4;
}

template <int BITS>
__device__ __forceinline__ float4 load_quad(const uint8_t *src, int64_t v4)
{
    u32 v;
    if constexpr (BITS == 2) v = src[v4];
    else if constexpr (BITS == 4) v = reinterpret_cast<const uint16_t *>(src)[v4];
    else v = reinterpret_cast<const u32 *>(src)[v4];
    const int sh = 32 - BITS;
    return make_float4((float)((int)(v << sh) >> sh), (float)((int)(v << (sh - BITS)) >> sh),
                       (float)((int)(v << (sh - 2 * BITS)) >> sh), (float)((int)(v << (sh - 3 * BITS)) >> sh));
}

struct CodesArgs {
    const float *tables;
    const int64_t *row_off;
    const int32_t *indices;
    const int32_t *offsets;
    const float *scales;
    uint8_t *payload;
    int T, D, B;
    int64_t L;
    int *status;
};

template <int BITS, int LPR, int CH>
__global__ void __launch_bounds__(SH_THREADS)
fwd_codes_kernel(const CodesArgs a)
{
    constexpr int NB = CH >= 2 ? 1 : 4;
    constexpr int RPW = 32 / LPR;
    constexpr int WPB = SH_THREADS / 32;
    const int d4 = a.D >> 2;
    const int t = blockIdx.y;
    const int wlane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lane = wlane % LPR, grp = wlane / LPR;
    const QuantScale qs = dq_make_scale(__ldg(a.scales + t), BITS);
    const int64_t r0 = __ldg(a.row_off + t);
    const int32_t nrows = (int32_t)(__ldg(a.row_off + t + 1) - r0);
    const float4 *tbl_lane = reinterpret_cast<const float4 *>(a.tables + r0 * a.D) + lane;
    const int64_t g0 = (int64_t)t * a.B;
    bool bad = false;
    for (int i0 = (blockIdx.x * WPB + warp) * 32; i0 < a.B; i0 += gridDim.x * (WPB * 32)) {
        const int i = i0 + wlane;
        int32_t idx = 0;
        bool ok = false;
        if (i < a.B) {
            const int32_t lo = __ldg(a.offsets + g0 + i), hi = __ldg(a.offsets + g0 + i + 1);
            ok = (hi - lo == 1) & (lo >= 0) & ((int64_t)hi <= a.L);
            if (ok) {
                idx = __ldg(a.indices + lo);
                bad |= (idx < 0) | (idx >= nrows);
                idx = min(max(idx, 0), nrows - 1);
            } else {
                bad = true;                          // this call is defined for one-index bags only
            }
        }
        const unsigned one = __ballot_sync(0xffffffffu, ok);
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
                    if (bag < 32 && ((one >> bag) & 1u) && c4 < d4) v[b] = __ldg(tbl_lane + (int64_t)ib[b] * d4 + c * LPR);
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int bag = k0 + b * RPW + grp;
                    if (bag < 32 && ((one >> bag) & 1u) && c4 < d4) {
                        float4 cd, dq_unused;
                        dq_fq4(v[b], qs, cd, dq_unused);
                        store_quad<BITS>(a.payload, ((int64_t)(i0 + bag) * a.T + t) * d4 + c4, pack4<BITS>(cd));
                    }
                }
            }
        }
    }
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
}

template <int BITS>
__global__ void __launch_bounds__(SH_THREADS)
decode_payload_kernel(const uint8_t *__restrict__ payload, const float *__restrict__ scales, float *__restrict__ out,
                      int64_t n4, int B, int T_blk, int T_total, int t0, int d4)
{
    for (int64_t v = (int64_t)blockIdx.x * SH_THREADS + threadIdx.x; v < n4; v += (int64_t)gridDim.x * SH_THREADS) {
        const int c4 = (int)(v % d4);
        const int64_t bt = v / d4;                   // (sample, table of the block)
        const int j = (int)(bt % T_blk);
        const int64_t i = bt / T_blk;
        const float s = __ldg(scales + j);
        const float4 q = load_quad<BITS>(payload, v);
        const float2 s2 = make_float2(s, s);
        const float2 lo = __fmul2_rn(make_float2(q.x, q.y), s2), hi = __fmul2_rn(make_float2(q.z, q.w), s2);
        reinterpret_cast<float4 *>(out)[(i * T_total + t0 + j) * d4 + c4] = make_float4(lo.x, lo.y, hi.x, hi.y);
    }
}

template <int BITS, int LPR, int CH>
int launch_codes(dqrm_ctx *ctx, const CodesArgs &a, cudaStream_t st)
{
    int bx = (a.B + SH_THREADS - 1) / SH_THREADS;
    const int cap = (ctx->num_sms * 32 + ctx->T - 1) / ctx->T;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    fwd_codes_kernel<BITS, LPR, CH><<<dim3((unsigned)bx, (unsigned)ctx->T), SH_THREADS, 0, st>>>(a);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_FWD_CODES);
    return DQRM_OK;
}

template <int BITS>
int dispatch_codes(dqrm_ctx *ctx, const CodesArgs &a, cudaStream_t st)
{
    const int d4 = a.D / 4;
#define DQ_FC(LPR, CH) return launch_codes<BITS, LPR, CH>(ctx, a, st)
    if (d4 <= 1) DQ_FC(1, 1);
    if (d4 <= 2) DQ_FC(2, 1);
    if (d4 <= 4) DQ_FC(4, 1);
    if (d4 <= 8) DQ_FC(8, 1);
    if (d4 <= 16) DQ_FC(16, 1);
    if (d4 <= 32) DQ_FC(32, 1);
    if (d4 <= 64) DQ_FC(32, 2);
    if (d4 <= 128) DQ_FC(32, 4);
    DQ_FC(32, 8);
#undef DQ_FC
}

}  // namespace

int dq_launch_fwd_codes(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                        const float *scales, int bits, uint8_t *payload, int B, int64_t L, cudaStream_t st)
{
    const CodesArgs a{tables, ctx->d_row_off, indices, offsets, scales, payload, ctx->T, ctx->D, B, L, ctx->d_status};
    if (bits == 2) return dispatch_codes<2>(ctx, a, st);
    if (bits == 4) return dispatch_codes<4>(ctx, a, st);
    return dispatch_codes<8>(ctx, a, st);
}

int dq_launch_decode_payload(dqrm_ctx *ctx, const uint8_t *payload, const float *scales, int bits, float *out, int B,
                             int T_blk, int T_total, int t0, cudaStream_t st)
{
    const int d4 = ctx->D / 4;
    const int64_t n4 = (int64_t)B * T_blk * d4;
    if (n4 == 0) return DQRM_OK;
    int64_t blocks = (n4 + SH_THREADS - 1) / SH_THREADS;
    const int64_t cap = (int64_t)ctx->num_sms * 16;
    const int grid = (int)(blocks > cap ? cap : blocks);
    if (bits == 2) decode_payload_kernel<2><<<grid, SH_THREADS, 0, st>>>(payload, scales, out, n4, B, T_blk, T_total, t0, d4);
    else if (bits == 4) decode_payload_kernel<4><<<grid, SH_THREADS, 0, st>>>(payload, scales, out, n4, B, T_blk, T_total, t0, d4);
    else decode_payload_kernel<8><<<grid, SH_THREADS, 0, st>>>(payload, scales, out, n4, B, T_blk, T_total, t0, d4);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_DECODE_PAYLOAD);
    return DQRM_OK;
}
