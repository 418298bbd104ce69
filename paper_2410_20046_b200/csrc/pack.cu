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

template <int BITS>
__device__ __forceinline__ float4 unpack4(u32 v)
{
    // sign-extend each BITS-wide field
    const int sh = 32 - BITS;
    return make_float4((float)((int)(v << sh) >> sh), (float)((int)(v << (sh - BITS)) >> sh),
                       (float)((int)(v << (sh - 2 * BITS)) >> sh), (float)((int)(v << (sh - 3 * BITS)) >> sh));
}

template <int BITS>
__device__ __forceinline__ u32 load_packed(const uint8_t *src, int64_t v4)
{
    if constexpr (BITS == 2) return src[v4];
    else if constexpr (BITS == 4) return reinterpret_cast<const uint16_t *>(src)[v4];
    else return reinterpret_cast<const u32 *>(src)[v4];
}

template <int BITS, int LPR, int CH>
__global__ void __launch_bounds__(PK_THREADS)
packed_fwd_kernel(const uint8_t *__restrict__ packed, const int64_t *__restrict__ row_off,
                  const int32_t *__restrict__ indices, const int32_t *__restrict__ offsets,
                  const float *__restrict__ scales, float *__restrict__ out, int T, int D, int B, int64_t L,
                  int *__restrict__ status)
{
    constexpr int GPB = PK_THREADS / LPR;
    constexpr int NB = 4;
    const int d4 = D >> 2;
    const int t = blockIdx.y;
    const int lane = threadIdx.x % LPR, grp = threadIdx.x / LPR;
    const float s = __ldg(scales + t);
    const int64_t r0 = __ldg(row_off + t);
    const int32_t nrows = (int32_t)(__ldg(row_off + t + 1) - r0);
    const int64_t g0 = (int64_t)t * B;
    bool bad = false;
    for (int i = blockIdx.x * GPB + grp; i < B; i += gridDim.x * GPB) {
        int32_t lo = __ldg(offsets + g0 + i), hi = __ldg(offsets + g0 + i + 1);
        if (lo < 0 || hi < lo || (int64_t)hi > L) { bad = true; hi = lo = 0; }
        double acc[CH][4];
#pragma unroll
        for (int c = 0; c < CH; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.0;
        for (int32_t j0 = lo; j0 < hi; j0 += NB) {
            u32 v[NB][CH];
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (j0 + b < hi) {
                    int32_t idx = __ldg(indices + j0 + b);
                    bad |= (idx < 0) | (idx >= nrows);
                    idx = min(max(idx, 0), nrows - 1);
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int c4 = c * LPR + lane;
                        if (c4 < d4) v[b][c] = load_packed<BITS>(packed, (r0 + idx) * d4 + c4);
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (j0 + b < hi) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int c4 = c * LPR + lane;
                        if (c4 < d4) {
                            const float4 q = unpack4<BITS>(v[b][c]);
                            acc[c][0] += (double)__fmul_rn(q.x, s);
                            acc[c][1] += (double)__fmul_rn(q.y, s);
                            acc[c][2] += (double)__fmul_rn(q.z, s);
                            acc[c][3] += (double)__fmul_rn(q.w, s);
                        }
                    }
                }
            }
        }
        float4 *o = reinterpret_cast<float4 *>(out + ((int64_t)i * T + t) * D);
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int c4 = c * LPR + lane;
            if (c4 < d4) o[c4] = make_float4((float)acc[c][0], (float)acc[c][1], (float)acc[c][2], (float)acc[c][3]);
        }
    }
    if (bad) dq_report(status, DQRM_ERR_INDEX_RANGE);
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

template <int BITS, int LPR, int CH>
int launch_pfwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                const float *scales, float *out, int B, int64_t L, cudaStream_t st)
{
    constexpr int GPB = PK_THREADS / LPR;
    int bx = (B + GPB - 1) / GPB;
    const int cap = (ctx->num_sms * 32 + ctx->T - 1) / ctx->T;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)ctx->T);
    packed_fwd_kernel<BITS, LPR, CH><<<grid, PK_THREADS, 0, st>>>(packed, ctx->d_row_off, indices, offsets, scales, out,
                                                                  ctx->T, ctx->D, B, L, ctx->d_status);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_PACKED_FWD);
    return DQRM_OK;
}

template <int BITS>
int dispatch_pfwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                  const float *scales, float *out, int B, int64_t L, cudaStream_t st)
{
    const int d4 = ctx->D / 4;
#define DQ_PF(LPR, CH) return launch_pfwd<BITS, LPR, CH>(ctx, packed, indices, offsets, scales, out, B, L, st)
    if (d4 <= 1) DQ_PF(1, 1);
    if (d4 <= 2) DQ_PF(2, 1);
    if (d4 <= 4) DQ_PF(4, 1);
    if (d4 <= 8) DQ_PF(8, 1);
    if (d4 <= 16) DQ_PF(16, 1);
    if (d4 <= 32) DQ_PF(32, 1);
    if (d4 <= 64) DQ_PF(32, 2);
    if (d4 <= 128) DQ_PF(32, 4);
    DQ_PF(32, 8);
#undef DQ_PF
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
    if (bits == 2) return dispatch_pfwd<2>(ctx, packed, indices, offsets, scales, out, B, L, st);
    if (bits == 4) return dispatch_pfwd<4>(ctx, packed, indices, offsets, scales, out, B, L, st);
    return dispatch_pfwd<8>(ctx, packed, indices, offsets, scales, out, B, L, st);
}
