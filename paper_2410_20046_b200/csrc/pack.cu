// Bit-packed export of the quantised embedding tables and inference lookups from the packed
// form (paper Appendix C: the INT4 vectors are bit-packed into bytes, which is what makes the
// deployed model 8x smaller: 2.161 GB -> 0.270 GB, 12.575 GB -> 1.572 GB in Table "res_tab").
// Layout (the paper gives none): element d of a row sits in byte (d*b)/8 at bit offset (d*b)%8,
// lowest bits first, as a b-bit two's-complement code, b in {2, 4, 8}; a row takes D*b/8 bytes.
//
// pack_kernel      streams the arena once (4 bytes read, b/8 bytes written per element); one
//                  thread turns one 128-bit vector of weights into b/2 bytes
// packed_fwd_kernel gathers packed rows, decodes, multiplies by the table's scale and sum-pools
//                  in bag order in FP64 - bit-identical to the training forward on the same
//                  master weights and scales
#include "common.cuh"

namespace {

constexpr int PK_THREADS = 256;
constexpr int PK_CHUNK4 = 4096;          // 128-bit vectors per chunk

template <int BITS>
__device__ __forceinline__ u32 pack4(const float4 &codes)
{
    const u32 m = (1u << BITS) - 1u;
    return ((u32)(int)codes.x & m) | (((u32)(int)codes.y & m) << BITS) | (((u32)(int)codes.z & m) << (2 * BITS)) |
           (((u32)(int)codes.w & m) << (3 * BITS));
}

template <int BITS>
__device__ __forceinline__ void store_packed(uint8_t *dst, int64_t v4, u32 bits4)
{
    if constexpr (BITS == 2) dst[v4] = (uint8_t)bits4;
    else if constexpr (BITS == 4) reinterpret_cast<uint16_t *>(dst)[v4] = (uint16_t)bits4;
    else reinterpret_cast<u32 *>(dst)[v4] = bits4;
}

template <int BITS>
__global__ void __launch_bounds__(PK_THREADS)
pack_kernel(const float4 *__restrict__ arena4, const int64_t *__restrict__ row_off, int T, int D, int64_t n4,
            const float *__restrict__ scales, uint8_t *__restrict__ packed)
{
    extern __shared__ unsigned char smem_raw[];
    int64_t *v4_off = reinterpret_cast<int64_t *>(smem_raw);       // table starts in 128-bit vectors
    const int d4 = D >> 2;
    for (int t = threadIdx.x; t <= T; t += PK_THREADS) v4_off[t] = row_off[t] * d4;
    __syncthreads();
    const int64_t n_chunks = (n4 + PK_CHUNK4 - 1) / PK_CHUNK4;
    for (int64_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const int64_t c0 = c * PK_CHUNK4, c1 = min(c0 + (int64_t)PK_CHUNK4, n4);
        const int t0 = dq_table_of(v4_off, T, c0);
        const bool one_table = c1 <= v4_off[t0 + 1];
        QuantScale qs = dq_make_scale(__ldg(scales + t0), BITS);
        for (int64_t i = c0 + threadIdx.x; i < c1; i += PK_THREADS) {
            if (!one_table) qs = dq_make_scale(__ldg(scales + dq_table_of(v4_off, T, i)), BITS);
            float4 cd, dq;
            dq_fq4(__ldcs(arena4 + i), qs, cd, dq);
            store_packed<BITS>(packed, i, pack4<BITS>(cd));
        }
    }
}

// ---- packed lookups -------------------------------------------------------------------
// A lane owns EPL consecutive elements of a row (8 when the feature size allows, else 4): one
// load of EPL*BITS/8 bytes, EPL/4 128-bit stores.
template <int BITS, int EPL>
struct Unit {
    static constexpr int BYTES = BITS * EPL / 8;
    u32 w[2];
    __device__ __forceinline__ void load(const uint8_t *__restrict__ p, int64_t u)
    {
        w[1] = 0;
        if constexpr (BYTES == 1) w[0] = __ldg(p + u);
        else if constexpr (BYTES == 2) w[0] = __ldg(reinterpret_cast<const uint16_t *>(p) + u);
        else if constexpr (BYTES == 4) w[0] = __ldg(reinterpret_cast<const u32 *>(p) + u);
        else { const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p) + u); w[0] = v.x; w[1] = v.y; }
    }
    // element k as a float: sign-extended BITS-wide field
    template <int K>
    __device__ __forceinline__ float get() const
    {
        constexpr int bit = K * BITS, word = bit / 32, off = bit % 32;
        return (float)((int)(w[word] << (32 - BITS - off)) >> (32 - BITS));
    }
    template <int Q>
    __device__ __forceinline__ float4 quad() const
    {
        return make_float4(get<4 * Q>(), get<4 * Q + 1>(), get<4 * Q + 2>(), get<4 * Q + 3>());
    }
};

__device__ __forceinline__ float4 scale4(const float4 &q, float s)
{
    const float2 s2 = make_float2(s, s);
    const float2 a = __fmul2_rn(make_float2(q.x, q.y), s2), b = __fmul2_rn(make_float2(q.z, q.w), s2);
    return make_float4(a.x, a.y, b.x, b.y);
}

struct PfArgs {
    const uint8_t *packed;
    const int64_t *row_off;
    const int32_t *indices;
    const int32_t *offsets;
    const float *scales;
    float *out;
    int T, D, B;
    int64_t L;
    int *status;
};

// pools one bag in bag order in FP64 and rounds once (any bag length, zero included)
template <int BITS, int EPL, int LPR, int CH>
__device__ __forceinline__ void pool_bag(const PfArgs &a, int64_t r0, int32_t nrows, float s, int units, int32_t lo,
                                         int32_t hi, float *out_row, int lane, bool &bad)
{
    constexpr int NB = 4;
    if (lo < 0 || hi < lo || (int64_t)hi > a.L) { bad = true; hi = lo = 0; }
    double acc[CH][EPL];
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
        for (int k = 0; k < EPL; ++k) acc[c][k] = 0.0;
    for (int32_t j0 = lo; j0 < hi; j0 += NB) {
        Unit<BITS, EPL> v[NB][CH];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (j0 + b < hi) {
                int32_t idx = __ldg(a.indices + j0 + b);
                bad |= (idx < 0) | (idx >= nrows);
                idx = min(max(idx, 0), nrows - 1);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int u = c * LPR + lane;
                    if (u < units) v[b][c].load(a.packed, (r0 + idx) * units + u);
                }
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (j0 + b < hi) {
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    if (c * LPR + lane < units) {
                        const float4 f0 = scale4(v[b][c].template quad<0>(), s);
                        acc[c][0] += (double)f0.x; acc[c][1] += (double)f0.y;
                        acc[c][2] += (double)f0.z; acc[c][3] += (double)f0.w;
                        if constexpr (EPL == 8) {
                            const float4 f1 = scale4(v[b][c].template quad<1>(), s);
                            acc[c][4] += (double)f1.x; acc[c][5] += (double)f1.y;
                            acc[c][6] += (double)f1.z; acc[c][7] += (double)f1.w;
                        }
                    }
                }
            }
        }
    }
    float4 *o = reinterpret_cast<float4 *>(out_row);
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        const int u = c * LPR + lane;
        if (u < units) {
            o[u * (EPL / 4)] = make_float4((float)acc[c][0], (float)acc[c][1], (float)acc[c][2], (float)acc[c][3]);
            if constexpr (EPL == 8)
                o[u * 2 + 1] = make_float4((float)acc[c][4], (float)acc[c][5], (float)acc[c][6], (float)acc[c][7]);
        }
    }
}

template <int BITS, int EPL, int LPR, int CH>
__global__ void __launch_bounds__(PK_THREADS)
packed_fwd_kernel(const PfArgs a)
{
    constexpr int GPB = PK_THREADS / LPR;
    const int units = a.D / EPL;
    const int t = blockIdx.y;
    const int lane = threadIdx.x % LPR, grp = threadIdx.x / LPR;
    const float s = __ldg(a.scales + t);
    const int64_t r0 = __ldg(a.row_off + t);
    const int32_t nrows = (int32_t)(__ldg(a.row_off + t + 1) - r0);
    const int64_t g0 = (int64_t)t * a.B;
    bool bad = false;
    for (int i = blockIdx.x * GPB + grp; i < a.B; i += gridDim.x * GPB)
        pool_bag<BITS, EPL, LPR, CH>(a, r0, nrows, s, units, __ldg(a.offsets + g0 + i), __ldg(a.offsets + g0 + i + 1),
                                     a.out + ((int64_t)i * a.T + t) * a.D, lane, bad);
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
}

// One index per bag (L == T*B, the Criteo shape): a warp takes 32 consecutive bags, one lane per
// bag does the bag's bookkeeping once, then the rows are fetched 32/LPR per step (the bag's index
// broadcast by shuffle), NB steps in flight; the pooled value of a one-index bag is code * scale
// itself.  A bag that turns out not to hold exactly one index goes through pool_bag.
template <int BITS, int EPL, int LPR, int CH>
__global__ void __launch_bounds__(PK_THREADS)
packed_fwd_onehot_kernel(const PfArgs a)
{
    constexpr int NB = CH >= 2 ? 1 : 4;
    constexpr int RPW = 32 / LPR;
    constexpr int WPB = PK_THREADS / 32;
    const int units = a.D / EPL;
    const int t = blockIdx.y;
    const int wlane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lane = wlane % LPR, grp = wlane / LPR;
    const float s = __ldg(a.scales + t);
    const int64_t r0 = __ldg(a.row_off + t);
    const int32_t nrows = (int32_t)(__ldg(a.row_off + t + 1) - r0);
    const int64_t g0 = (int64_t)t * a.B;
    const int TD4 = a.T * (a.D >> 2);            // 128-bit vectors between the output rows of bags i and i+1
    bool bad = false;
    for (int i0 = (blockIdx.x * WPB + warp) * 32; i0 < a.B; i0 += gridDim.x * (WPB * 32)) {
        const int i = i0 + wlane;
        int32_t idx = 0;
        bool single = false;
        if (i < a.B) {
            const int32_t lo = __ldg(a.offsets + g0 + i), hi = __ldg(a.offsets + g0 + i + 1);
            idx = __ldg(a.indices + g0 + i);            // right when the offsets are the identity (L == T*B)
            single = (hi - lo == 1) & (lo >= 0) & ((int64_t)hi <= a.L);
            if (single) {
                if ((int64_t)lo != g0 + i) idx = __ldg(a.indices + lo);
                bad |= (idx < 0) | (idx >= nrows);
                idx = min(max(idx, 0), nrows - 1);
            }
        }
        const unsigned one = __ballot_sync(0xffffffffu, single);
        unsigned rare = __ballot_sync(0xffffffffu, (i < a.B) && !single);
        float4 *out_lane = reinterpret_cast<float4 *>(a.out) + ((int64_t)i0 * a.T + t) * (a.D >> 2) + lane * (EPL / 4);
#pragma unroll 1
        for (int k0 = 0; k0 < 32; k0 += RPW * NB) {
            if ((one >> k0) == 0u) break;
            int32_t ib[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) ib[b] = __shfl_sync(0xffffffffu, idx, (k0 + b * RPW + grp) & 31);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int u = c * LPR + lane;
                Unit<BITS, EPL> v[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int bag = k0 + b * RPW + grp;
                    if (bag < 32 && ((one >> bag) & 1u) && u < units) v[b].load(a.packed, (r0 + ib[b]) * units + u);
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int bag = k0 + b * RPW + grp;
                    if (bag < 32 && ((one >> bag) & 1u) && u < units) {
                        float4 *o = out_lane + (int64_t)bag * TD4 + c * LPR * (EPL / 4);
                        o[0] = scale4(v[b].template quad<0>(), s);
                        if constexpr (EPL == 8) o[1] = scale4(v[b].template quad<1>(), s);
                    }
                }
            }
        }
        while (rare) {
            const int bag = __ffs(rare) - 1;
            rare &= rare - 1;
            const int ii = i0 + bag;
            if (grp == 0)
                pool_bag<BITS, EPL, LPR, CH>(a, r0, nrows, s, units, __ldg(a.offsets + g0 + ii),
                                             __ldg(a.offsets + g0 + ii + 1), a.out + ((int64_t)ii * a.T + t) * a.D, lane,
                                             bad);
        }
    }
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
}

template <int BITS>
int launch_pack(dqrm_ctx *ctx, const float *tables, const float *scales, uint8_t *packed, cudaStream_t st)
{
    const int64_t n4 = ctx->total_rows * (ctx->D / 4);
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int64_t);
    pack_kernel<BITS><<<ctx->num_sms * 8, PK_THREADS, smem, st>>>(reinterpret_cast<const float4 *>(tables), ctx->d_row_off,
                                                                  ctx->T, ctx->D, n4, scales, packed);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_PACK);
    return DQRM_OK;
}

template <int BITS, int EPL, int LPR, int CH>
int launch_pfwd(dqrm_ctx *ctx, const PfArgs &a, cudaStream_t st)
{
    constexpr int GPB = PK_THREADS / LPR;
    const bool onehot = a.L == (int64_t)a.T * a.B;
    const int per_block = onehot ? PK_THREADS : GPB;
    int bx = (a.B + per_block - 1) / per_block;
    const int cap = (ctx->num_sms * 32 + ctx->T - 1) / ctx->T;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)ctx->T);
    if (onehot) packed_fwd_onehot_kernel<BITS, EPL, LPR, CH><<<grid, PK_THREADS, 0, st>>>(a);
    else packed_fwd_kernel<BITS, EPL, LPR, CH><<<grid, PK_THREADS, 0, st>>>(a);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_PACKED_FWD);
    return DQRM_OK;
}

template <int BITS, int EPL>
int dispatch_pfwd2(dqrm_ctx *ctx, const PfArgs &a, cudaStream_t st)
{
    const int units = a.D / EPL;
#define DQ_PF(LPR, CH) return launch_pfwd<BITS, EPL, LPR, CH>(ctx, a, st)
    if (units <= 1) DQ_PF(1, 1);
    if (units <= 2) DQ_PF(2, 1);
    if (units <= 4) DQ_PF(4, 1);
    if (units <= 8) DQ_PF(8, 1);
    if (units <= 16) DQ_PF(16, 1);
    if (units <= 32) DQ_PF(32, 1);
    if (units <= 64) DQ_PF(32, 2);
    if (units <= 128) DQ_PF(32, 4);
    DQ_PF(32, 8);
#undef DQ_PF
}

template <int BITS>
int dispatch_pfwd(dqrm_ctx *ctx, const PfArgs &a, cudaStream_t st)
{
    if (a.D % 8 == 0) return dispatch_pfwd2<BITS, 8>(ctx, a, st);
    return dispatch_pfwd2<BITS, 4>(ctx, a, st);
}

}  // namespace

int dq_launch_pack(dqrm_ctx *ctx, const float *tables, const float *scales, int bits, uint8_t *packed, cudaStream_t st)
{
    if (bits == 2) return launch_pack<2>(ctx, tables, scales, packed, st);
    if (bits == 4) return launch_pack<4>(ctx, tables, scales, packed, st);
    return launch_pack<8>(ctx, tables, scales, packed, st);
}

int dq_launch_packed_fwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                         const float *scales, int bits, float *out, int B, int64_t L, cudaStream_t st)
{
    const PfArgs a{packed, ctx->d_row_off, indices, offsets, scales, out, ctx->T, ctx->D, B, L, ctx->d_status};
    if (bits == 2) return dispatch_pfwd<2>(ctx, a, st);
    if (bits == 4) return dispatch_pfwd<4>(ctx, a, st);
    return dispatch_pfwd<8>(ctx, a, st);
}
