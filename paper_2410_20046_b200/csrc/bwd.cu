// Backward of the embedding lookup (paper Section 4.3 and Appendix B.1): the gradient of
// an embedding table is a sparse (indices, values) tensor over the rows the batch
// touched; lookups that hit the same row are coalesced.  Sum pooling and the
// straight-through quantiser hand every lookup its bag's upstream gradient unchanged.
//
// Pipeline (all on one stream, no inter-block waits anywhere):
//   prepare      one thread per bag: arena-row key + gradient-row payload per lookup,
//                digit histograms of every radix pass, first pass's per-tile histogram
//   per pass     scan   : per-digit exclusive scan of the tile histograms (+ digit base)
//                scatter: stable least-significant-digit scatter of (key, payload);
//                         counts the next pass's tile histogram on the way
//   seg_count / seg_emit  head flags of the sorted keys -> unique_rows, uniq_off,
//                         segment starts, first segment of every 32-entry chunk
//   seg_reduce   one lane group per 32-entry chunk of the sorted order: gathers the
//                upstream gradient rows (128-bit loads), sums runs in FP64; runs that are
//                whole segments are rounded and written, runs cut by a chunk boundary
//                leave an FP64 partial
//   seg_fixup    one warp per cut segment: adds its partials in a fixed order
// The sort is stable and every sum has a fixed shape, so results are reproducible bit
// for bit.  The per-table abs-max of the summed gradient (needed by the INT8 gradient
// quantiser) is folded into the last two kernels.
#include "common.cuh"
#include "seg_reduce.cuh"
#include "cluster_sort.cuh"

namespace {

constexpr int ST_THREADS = 256;
constexpr int ST_ITEMS = 8;
constexpr int ST_TILE = ST_THREADS * ST_ITEMS;   // 2048 entries per tile
constexpr int ST_WARPS = ST_THREADS / 32;
constexpr int NB_MAX = 512;                      // bins per pass (<= 9 bit digits)
constexpr int HIST_CHUNK = 64;                   // tiles per chunk of the radix sort's offset computation
constexpr int SEG_CHUNK = segred::CHUNK;         // sorted entries per reduce work item

struct Layout {
    int passes, digit_bits, nb;
    int ck;                                    // sorted entries per lane group of the reduce: 32, or 16
    int64_t num_tiles, num_chunks;             // num_chunks = ceil(L / ck)
    // zeroed at call start: [0, zero_small)
    size_t absmax, counters, tile_heads, zero_small, digit_base, chunk_sum, tilehist;
    size_t keys_a, vals_a, pairs_a, pairs_b, seg_start, chunk_first, long_list, partials, table_cnt, tb;
    size_t total;
};

Layout make_layout(const dqrm_ctx *ctx, int64_t L)
{
    Layout y;
    y.passes = (ctx->key_bits + 8) / 9;
    if (y.passes < 1) y.passes = 1;
    y.digit_bits = (ctx->key_bits + y.passes - 1) / y.passes;
    y.nb = 1 << y.digit_bits;
    int64_t Lc = L < 1 ? 1 : L;
    y.num_tiles = (Lc + ST_TILE - 1) / ST_TILE;
    // A chunk is walked in order by one lane group.  A batch whose 32-entry chunks would not even give every SM
    // one block of the reduce takes 16-entry chunks: twice the groups, each half as long (measured: 19 -> 14 us
    // at batch 128, but 24 -> 29 us at 208 blocks, where the extra pieces cost more than the shorter walks save).
    y.ck = SEG_CHUNK;
    {
        const int D = ctx->D;
        const int rl = D <= 4 ? 4 : D <= 8 ? 8 : D <= 16 ? 4 : D <= 64 ? 16 : 32;      // lanes per row of the reduce
        if (rl <= 16 && (Lc / SEG_CHUNK) / (256 / rl) < (int64_t)ctx->num_sms) y.ck = SEG_CHUNK / 2;
    }
    y.num_chunks = (Lc + y.ck - 1) / y.ck;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    y.absmax = take(sizeof(u32) * ctx->T);
    y.counters = take(sizeof(u32) * 8);
    y.tile_heads = take(sizeof(u32) * y.num_tiles);
    y.zero_small = o;
    y.digit_base = take(sizeof(u32) * NB_MAX);
    y.chunk_sum = take(sizeof(u32) * y.nb * ((y.num_tiles + HIST_CHUNK - 1) / HIST_CHUNK));
    y.tilehist = take(sizeof(u32) * y.nb * y.num_tiles);
    y.keys_a = take(sizeof(u32) * Lc);
    y.vals_a = take(sizeof(u32) * Lc);
    y.pairs_a = take(sizeof(uint2) * Lc);
    y.pairs_b = take(sizeof(uint2) * Lc);
    y.seg_start = take(sizeof(u32) * (Lc + ctx->T + 1));     // (lists by table: one slot more per table)
    y.table_cnt = take(sizeof(u32) * ctx->T);
    y.tb = take(sizeof(u32) * (ctx->T + 1));
    y.chunk_first = take(sizeof(u32) * y.num_chunks);
    y.long_list = take(sizeof(uint4) * y.num_chunks);
    y.partials = take(sizeof(double) * y.num_chunks * 2 * ctx->D);
    y.total = o;
    return y;
}

// counters[]: see segred::CNT_*
using segred::CNT_U;

// ---------------------------------------------------------------------------------
// one thread per bag: (arena-row key, gradient-row payload) of every lookup of the bag, as one 8-byte pair:
// the passes move pairs, so that a digit's short run in a tile still leaves as whole 32-byte sectors
__global__ void __launch_bounds__(256)
prepare_kernel(const int32_t *__restrict__ indices, const int32_t *__restrict__ offsets,
               const int64_t *__restrict__ row_off, int T, int B, int64_t G, int64_t L,
               uint2 *__restrict__ pairs, int payload_position, int *__restrict__ status)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (__ldg(offsets) != 0 || (int64_t)__ldg(offsets + G) != L) dq_report(status, DQRM_ERR_INDEX_RANGE);
    }
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < G; g += (int64_t)gridDim.x * blockDim.x) {
        int32_t a = __ldg(offsets + g), e = __ldg(offsets + g + 1);
        if (a < 0 || e < a || (int64_t)e > L) { dq_report(status, DQRM_ERR_INDEX_RANGE); continue; }
        const int t = (int)(g / B);
        const u32 payload = (u32)((g - (int64_t)t * B) * T + t);      // row of grad_out [B][T][D]
        const int64_t r0 = __ldg(row_off + t);
        const int64_t nrows = __ldg(row_off + t + 1) - r0;
        for (int32_t j = a; j < e; ++j) {
            int32_t idx = __ldg(indices + j);
            if (idx < 0 || idx >= nrows) {
                dq_report(status, DQRM_ERR_INDEX_RANGE);
                idx = idx < 0 ? 0 : (int32_t)(nrows - 1);
            }
            pairs[j] = make_uint2((u32)(r0 + idx), payload_position ? (u32)j : payload);
        }
    }
}

// Per pass, three small kernels turn the digit counts of every tile of 2048 entries into the scatter's
// offsets without a single global atomic: tilehist[tile][digit] counts; a thread per digit then walks the
// 64 tiles of a chunk and leaves the running count in their place and the chunk's total in
// chunk_sum[chunk][digit]; one block does the same over the chunks and scans the digits' totals.  The
// scatter adds the three: digit base + chunks before + tiles before within the chunk.
__global__ void __launch_bounds__(ST_THREADS)
sort_hist_kernel(const uint2 *__restrict__ pairs, int64_t L, int shift, int nb, u32 *__restrict__ tilehist)
{
    __shared__ u32 cnt[NB_MAX];
    for (int i = threadIdx.x; i < nb; i += ST_THREADS) cnt[i] = 0u;
    __syncthreads();
    const u32 mask = (u32)nb - 1u;
    const int64_t base = (int64_t)blockIdx.x * ST_TILE + threadIdx.x;
    u32 key[ST_ITEMS];
#pragma unroll
    for (int k = 0; k < ST_ITEMS; ++k) {
        const int64_t i = base + (int64_t)k * ST_THREADS;
        key[k] = i < L ? pairs[i].x : 0u;
    }
#pragma unroll
    for (int k = 0; k < ST_ITEMS; ++k)
        if (base + (int64_t)k * ST_THREADS < L) atomicAdd(&cnt[(key[k] >> shift) & mask], 1u);
    __syncthreads();
    for (int i = threadIdx.x; i < nb; i += ST_THREADS) tilehist[(size_t)blockIdx.x * nb + i] = cnt[i];
}

// block = chunk of HIST_CHUNK tiles, thread = digit
__global__ void __launch_bounds__(NB_MAX)
sort_chunk_kernel(u32 *__restrict__ tilehist, int64_t num_tiles, int nb, u32 *__restrict__ chunk_sum)
{
    const int d = threadIdx.x;
    if (d >= nb) return;
    const int64_t t0 = (int64_t)blockIdx.x * HIST_CHUNK;
    const int n = (int)min((int64_t)HIST_CHUNK, num_tiles - t0);
    u32 run = 0;
    for (int b = 0; b < n; b += 8) {
        u32 c[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) c[k] = b + k < n ? tilehist[(size_t)(t0 + b + k) * nb + d] : 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (b + k < n) { tilehist[(size_t)(t0 + b + k) * nb + d] = run; run += c[k]; }
    }
    chunk_sum[(size_t)blockIdx.x * nb + d] = run;
}

// one block, thread = digit: running counts over the chunks, then an exclusive scan of the digits' totals
__global__ void __launch_bounds__(NB_MAX)
sort_base_kernel(u32 *__restrict__ chunk_sum, int64_t num_chunks, int nb, u32 *__restrict__ digit_base)
{
    __shared__ u32 wsum[NB_MAX / 32];
    const int d = threadIdx.x, lane = d & 31, warp = d >> 5;
    u32 run = 0;
    if (d < nb) {
        for (int64_t c = 0; c < num_chunks; c += 8) {
            u32 v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = c + k < num_chunks ? chunk_sum[(size_t)(c + k) * nb + d] : 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (c + k < num_chunks) { chunk_sum[(size_t)(c + k) * nb + d] = run; run += v[k]; }
        }
    }
    u32 incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const u32 v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    u32 woff = 0;
    for (int w = 0; w < warp; ++w) woff += wsum[w];
    if (d < nb) digit_base[d] = woff + incl - run;
}

// stable scatter of one tile by one digit
// LAST: the final pass leaves keys and payloads in arrays of their own, as the kernels behind the sort read them
template <bool LAST>
__global__ void __launch_bounds__(ST_THREADS)
sort_scatter_kernel(const uint2 *__restrict__ pairs_in, uint2 *__restrict__ pairs_out,
                    u32 *__restrict__ keys_out, u32 *__restrict__ vals_out,
                    const u32 *__restrict__ tilehist, const u32 *__restrict__ chunk_sum,
                    const u32 *__restrict__ digit_base, int64_t L, int shift, int nb, int *__restrict__ status)
{
    __shared__ u32 cnt[ST_WARPS][NB_MAX];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tile = blockIdx.x;
    const u32 mask = (u32)nb - 1u;
    for (int i = threadIdx.x; i < ST_WARPS * NB_MAX; i += ST_THREADS) (&cnt[0][0])[i] = 0u;
    __syncthreads();

    u32 key[ST_ITEMS], val[ST_ITEMS], rank[ST_ITEMS];
    const int64_t base = tile * ST_TILE + (int64_t)warp * (32 * ST_ITEMS) + lane;
#pragma unroll
    for (int k = 0; k < ST_ITEMS; ++k) {
        int64_t i = base + k * 32;
        bool valid = i < L;
        const uint2 pr = valid ? pairs_in[i] : make_uint2(0u, 0u);
        key[k] = pr.x;
        val[k] = pr.y;
    }
    const u32 lt = (1u << lane) - 1u;
#pragma unroll
    for (int k = 0; k < ST_ITEMS; ++k) {
        bool valid = (base + k * 32) < L;
        u32 digit = valid ? ((key[k] >> shift) & mask) : (u32)nb;      // nb = "no item"
        u32 peers = __match_any_sync(0xffffffffu, digit);
        int leader = __ffs(peers) - 1;
        u32 pre = 0;
        if (lane == leader && valid) {
            pre = cnt[warp][digit];
            cnt[warp][digit] = pre + __popc(peers);
        }
        pre = __shfl_sync(0xffffffffu, pre, leader);
        rank[k] = pre + __popc(peers & lt);
        __syncwarp();
    }
    __syncthreads();
    // per digit: running offset over warps, starting at this tile's global offset
    for (int b = threadIdx.x; b < nb; b += ST_THREADS) {
        u32 run = digit_base[b] + chunk_sum[(size_t)(tile / HIST_CHUNK) * nb + b] + tilehist[(size_t)tile * nb + b];
#pragma unroll
        for (int w = 0; w < ST_WARPS; ++w) {
            u32 c = cnt[w][b];
            cnt[w][b] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < ST_ITEMS; ++k) {
        if ((base + k * 32) < L) {
            u32 digit = (key[k] >> shift) & mask;
            u32 pos = cnt[warp][digit] + rank[k];
            if ((int64_t)pos < L) {
                if (LAST) {
                    keys_out[pos] = key[k];
                    vals_out[pos] = val[k];
                } else {
                    pairs_out[pos] = make_uint2(key[k], val[k]);
                }
            } else {
                dq_report(status, DQRM_ERR_INDEX_RANGE);   // only reachable with inconsistent offsets
            }
        }
    }
}

// ---------------------------------------------------------------------------------
// heads of the sorted key array
__device__ __forceinline__ void load_tile_keys(const u32 *__restrict__ keys, int64_t L, int64_t i0,
                                               u32 (&k)[ST_ITEMS], u32 &prev, int &n)
{
    n = (int)max((int64_t)0, min((int64_t)ST_ITEMS, L - i0));
    prev = (i0 > 0 && i0 <= L) ? keys[i0 - 1] : 0xFFFFFFFFu;
#pragma unroll
    for (int e = 0; e < ST_ITEMS; ++e) k[e] = (e < n) ? keys[i0 + e] : 0u;
}

__global__ void __launch_bounds__(ST_THREADS)
seg_count_kernel(const u32 *__restrict__ keys, int64_t L, u32 *__restrict__ tile_heads)
{
    __shared__ u32 wsum[ST_WARPS];
    const int64_t i0 = (int64_t)blockIdx.x * ST_TILE + (int64_t)threadIdx.x * ST_ITEMS;
    u32 k[ST_ITEMS], prev; int n;
    load_tile_keys(keys, L, i0, k, prev, n);
    u32 c = 0;
#pragma unroll
    for (int e = 0; e < ST_ITEMS; ++e) {
        if (e < n) c += (i0 + e == 0 || k[e] != prev) ? 1u : 0u;
        prev = k[e];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        u32 s = 0;
        for (int w = 0; w < ST_WARPS; ++w) s += wsum[w];
        tile_heads[blockIdx.x] = s;
    }
}

__global__ void __launch_bounds__(ST_THREADS)
seg_emit_kernel(const u32 *__restrict__ keys, int64_t L, const u32 *__restrict__ tile_heads,
                const int64_t *__restrict__ row_off, int T,
                u32 *__restrict__ seg_start, u32 *__restrict__ chunk_first,
                int32_t *__restrict__ unique_rows, int32_t *__restrict__ uniq_off, u32 *__restrict__ counters, int ck)
{
    extern __shared__ unsigned char smem_raw[];
    int64_t *s_off = reinterpret_cast<int64_t *>(smem_raw);   // [T+1]
    __shared__ u32 wsum[ST_WARPS];
    __shared__ u32 s_prefix;
    // this thread's keys first: they depend on nothing, so they fly beside the loads of the prefix below
    const int64_t i0 = (int64_t)blockIdx.x * ST_TILE + (int64_t)threadIdx.x * ST_ITEMS;
    const int ck_shift = 31 - __clz(ck);
    u32 k[ST_ITEMS], prev0; int n;
    load_tile_keys(keys, L, i0, k, prev0, n);
    for (int t = threadIdx.x; t <= T; t += ST_THREADS) s_off[t] = row_off[t];
    // heads in all earlier tiles
    u32 p = 0;
    for (int64_t i = threadIdx.x; i < blockIdx.x; i += ST_THREADS) p += tile_heads[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = p;
    __syncthreads();
    if (threadIdx.x == 0) {
        u32 s = 0;
        for (int w = 0; w < ST_WARPS; ++w) s += wsum[w];
        s_prefix = s;
    }
    __syncthreads();
    const u32 tile_prefix = s_prefix;
    __syncthreads();

    u32 c = 0;
    {
        u32 prev = prev0;
#pragma unroll
        for (int e = 0; e < ST_ITEMS; ++e) {
            if (e < n) c += (i0 + e == 0 || k[e] != prev) ? 1u : 0u;
            prev = k[e];
        }
    }
    // block exclusive scan of c
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u32 incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        u32 v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    u32 woff = 0;
    for (int w = 0; w < warp; ++w) woff += wsum[w];
    u32 heads_before = tile_prefix + woff + incl - c;   // heads strictly before entry i0

    // tables of the keys: found once for the key before this thread's entries, then only advanced
    // (keys ascend), so a head costs a comparison instead of two searches
    int t_prev = -1, t = 0;
    if (n > 0) {
        if (i0 > 0) t_prev = dq_table_of(s_off, T, (int64_t)prev0);
        t = t_prev < 0 ? 0 : t_prev;
    }
    u32 prev = prev0;
#pragma unroll
    for (int e = 0; e < ST_ITEMS; ++e) {
        if (e < n) {
            const int64_t i = i0 + e;
            const bool head = (i == 0 || k[e] != prev);
            if (head) {
                const u32 u = heads_before;
                heads_before += 1;
                seg_start[u] = (u32)i;
                // a sort that refused a table leaves that table's keys undefined: keep them inside the arena and
                // the walk inside the offset list, whatever they hold
                const int64_t key = min((int64_t)k[e], s_off[T] - 1);
                while (t < T - 1 && key >= s_off[t + 1]) ++t;
                unique_rows[u] = (int32_t)max((int64_t)0, key - s_off[t]);
                for (int tt = t_prev + 1; tt <= t; ++tt) uniq_off[tt] = (int32_t)u;
                t_prev = t;
            }
            const u32 u_of_i = heads_before - 1;
            if ((i & (int64_t)(ck - 1)) == 0) chunk_first[i >> ck_shift] = u_of_i;     // ck is 16 or 32
            if (i == L - 1) {
                const u32 U = u_of_i + 1;
                seg_start[U] = (u32)L;
                for (int tt = t_prev + 1; tt <= T; ++tt) uniq_off[tt] = (int32_t)U;
                counters[CNT_U] = U;
            }
        }
        prev = k[e];
    }
}

// ---------------------------------------------------------------------------------
// RL/RV/RC: lanes per row, floats per lane vector and vectors per lane of the reduce kernel;
// LPR/CH: the same for the fix-up kernels (always 128-bit vectors)
template <int RL, int RV, int RC, int LPR, int CH>
int launch_reduce(dqrm_ctx *ctx, const Layout &y, char *ws, const u32 *keys, const u32 *vals, int32_t *unique_rows,
                  int32_t *uniq_off, const float *grad_out, float *grad_rows, int64_t L, int64_t G, cudaStream_t st)
{
    using namespace segred;
    const int64_t cap = (int64_t)ctx->num_sms * 8;
    const int64_t gpb = 256 / RL;                            // one lane group per chunk
    int64_t blocks = (y.num_chunks + gpb - 1) / gpb;
    int grid = (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
    u32 *counters = reinterpret_cast<u32 *>(ws + y.counters);
    u32 *absmax = reinterpret_cast<u32 *>(ws + y.absmax);
    const u32 *seg_start = reinterpret_cast<const u32 *>(ws + y.seg_start);
    double *partials = reinterpret_cast<double *>(ws + y.partials);
    uint4 *long_list = reinterpret_cast<uint4 *>(ws + y.long_list);
    const size_t red_smem = (size_t)(ctx->T + 1) * 3 * sizeof(u32) + (size_t)gpb * 2 * y.ck * sizeof(u32);
    ByTable bt;
    bt.table_cnt = reinterpret_cast<const u32 *>(ws + y.table_cnt);
    bt.tb = reinterpret_cast<const u32 *>(ws + y.tb);
    bt.row_off = ctx->d_row_off;
    bt.unique_rows = unique_rows;
    bt.uniq_off = uniq_off;
    const u32 *chunk_first = reinterpret_cast<const u32 *>(ws + y.chunk_first);
#define DQ_LAUNCH_REDUCE(EXACT, CK)                                                                                  \
    seg_reduce_kernel<RL, RV, RC, EXACT, CK><<<grid, 256, red_smem, st>>>(                                          \
        keys, vals, seg_start, chunk_first, uniq_off, grad_out, grad_rows, partials, long_list, counters, absmax,    \
        ctx->T, ctx->D, L, G, y.num_chunks, ctx->d_status, bt)
    const bool exact = ctx->D == RL * RV * RC;
    if constexpr (RL <= 16) {
        if (y.ck == SEG_CHUNK / 2) {
            if (exact) DQ_LAUNCH_REDUCE(true, SEG_CHUNK / 2); else DQ_LAUNCH_REDUCE(false, SEG_CHUNK / 2);
        } else {
            if (exact) DQ_LAUNCH_REDUCE(true, SEG_CHUNK); else DQ_LAUNCH_REDUCE(false, SEG_CHUNK);
        }
    } else {
        if (exact) DQ_LAUNCH_REDUCE(true, SEG_CHUNK); else DQ_LAUNCH_REDUCE(false, SEG_CHUNK);
    }
#undef DQ_LAUNCH_REDUCE
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_SEG_REDUCE);
    int64_t fblocks = (y.num_chunks + 7) / 8;                // at most one cut segment per chunk, a warp each
    int fgrid = (int)(fblocks < (int64_t)ctx->num_sms * 4 ? (fblocks < 1 ? 1 : fblocks) : (int64_t)ctx->num_sms * 4);
    const size_t fix_smem = (size_t)(256 / LPR) * ctx->D * sizeof(double);
    if (fix_smem > 48 * 1024) {
        bool &raised = ctx->smem_raised[dq_smem_slot_fixup(LPR, CH)];
        if (!raised) {
            DQRM_CUDA_TRY(ctx, cudaFuncSetAttribute(seg_fixup_kernel<LPR, CH>,
                                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fix_smem));
            raised = true;
        }
    }
    seg_fixup_kernel<LPR, CH><<<fgrid, 256, fix_smem, st>>>(partials, long_list, counters, grad_rows, absmax, ctx->D,
                                                            y.num_chunks);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_SEG_FIXUP);
    return DQRM_OK;
}

template <int CL>
cudaError_t launch_cluster_sort(dqrm_ctx *ctx, csort::Args ca, int64_t per_table, cudaStream_t st)
{
    ca.cap = csort::choose_cap(per_table, CL);
    bool &raised = ctx->smem_raised[DQ_SMEM_SLOT_CSORT + (CL == csort::CLUSTER ? 0 : 1)];
    cudaError_t e = cudaSuccess;
    if (!raised) {
        e = cudaFuncSetAttribute(csort::cluster_sort_kernel<CL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)csort::smem_bytes(12288));
        if (e == cudaSuccess && CL > 8)       // more than eight blocks in a cluster is an opt-in
            e = cudaFuncSetAttribute(csort::cluster_sort_kernel<CL>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        raised = (e == cudaSuccess);
    }
    if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(ctx->T * CL));
        cfg.blockDim = dim3(csort::THREADS);
        cfg.dynamicSmemBytes = csort::smem_bytes(ca.cap);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, csort::cluster_sort_kernel<CL>, ca);
    }
    if (e != cudaSuccess) (void)cudaGetLastError();
    return e;
}

}  // namespace

void dq_bwd_ws_views(const dqrm_ctx *ctx, int64_t L, char *ws, const u32 **sorted_vals, const u32 **seg_start)
{
    const Layout y = make_layout(ctx, L);
    *sorted_vals = reinterpret_cast<const u32 *>(ws + y.vals_a);
    *seg_start = reinterpret_cast<const u32 *>(ws + y.seg_start);
}

const u32 *dq_bwd_absmax_bits(const dqrm_ctx *ctx, int64_t L, const void *ws)
{
    return reinterpret_cast<const u32 *>(reinterpret_cast<const char *>(ws) + make_layout(ctx, L).absmax);
}

size_t dq_bwd_ws_bytes(const dqrm_ctx *ctx, int64_t L, int64_t G)
{
    (void)G;
    return make_layout(ctx, L).total;
}

// first half of the backward: everything that depends only on the indices (sort, unique rows,
// segment starts).  It needs no upstream gradient, so a training step runs it beside the forward.
int dq_launch_bwd_sort(dqrm_ctx *ctx, const int32_t *indices, const int32_t *offsets,
                       int32_t *unique_rows, int32_t *uniq_off, int B, int64_t L,
                       void *ws_, size_t ws_bytes, cudaStream_t st, const u32 **absmax_bits_out, bool lists_by_table)
{
    const Layout y = make_layout(ctx, L);
    if (ws_bytes < y.total) return DQRM_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(ws_);
    const int64_t G = (int64_t)ctx->T * B;
    if (absmax_bits_out) *absmax_bits_out = reinterpret_cast<const u32 *>(ws + y.absmax);
    const bool fits_cluster = (L + ctx->T - 1) / ctx->T <= (int64_t)csort::CLUSTER * 12288;   // (a table beyond its
    // blocks' shared memory still sorts, through global staging, but slowly)
    const bool try_cluster = ctx->sort_path != 1 && fits_cluster;
    DQRM_CUDA_TRY(ctx, cudaMemsetAsync(ws, 0, y.zero_small, st));
    dq_mark(ctx, st, DQ_K_MEMSET);
    if (L == 0) {
        DQRM_CUDA_TRY(ctx, cudaMemsetAsync(uniq_off, 0, sizeof(int32_t) * (ctx->T + 1), st));
        return DQRM_OK;
    }
    u32 *keys[1] = {reinterpret_cast<u32 *>(ws + y.keys_a)};
    u32 *vals[1] = {reinterpret_cast<u32 *>(ws + y.vals_a)};
    uint2 *pairs[2] = {reinterpret_cast<uint2 *>(ws + y.pairs_a), reinterpret_cast<uint2 *>(ws + y.pairs_b)};
    u32 *tilehist = reinterpret_cast<u32 *>(ws + y.tilehist), *chunk_sum = reinterpret_cast<u32 *>(ws + y.chunk_sum);
    u32 *digit_base = reinterpret_cast<u32 *>(ws + y.digit_base);
    const u32 *skeys = nullptr;      // sorted keys; the sorted payloads sit beside them in vals[0]
    bool sorted = false;
    // (tables far beyond the shared-memory slices sort faster with the global radix sort)
    if (try_cluster) {
        // one cluster of eight blocks per table (sixteen when so few tables would leave most SMs idle); falls
        // through to the narrower cluster, then to the global radix sort, if a launch is refused
        csort::Args ca;
        ca.indices = indices; ca.offsets = offsets; ca.row_off = ctx->d_row_off;
        ca.T = ctx->T; ca.B = B; ca.L = L;
        ca.keys_out = keys[0]; ca.vals_out = vals[0];
        // global staging of (row, payload) pairs, used only by tables too large for shared memory
        ca.gp[0] = reinterpret_cast<uint2 *>(ws + y.pairs_a); ca.gp[1] = reinterpret_cast<uint2 *>(ws + y.pairs_b);
        ca.status = ctx->d_status;
        ca.payload_position = ctx->payload_position;
        ca.tile_heads = reinterpret_cast<u32 *>(ws + y.tile_heads);
        // when dq_launch_bwd_reduce follows, the clusters number their own tables' segments and seg_emit is not run
        ca.lists_by_table = lists_by_table ? 1 : 0;
        ca.seg_start = reinterpret_cast<u32 *>(ws + y.seg_start);
        ca.chunk_first = reinterpret_cast<u32 *>(ws + y.chunk_first);
        ca.table_cnt = reinterpret_cast<u32 *>(ws + y.table_cnt);
        ca.tb = reinterpret_cast<u32 *>(ws + y.tb);
        ca.counters = reinterpret_cast<u32 *>(ws + y.counters);
        ca.ck_shift = y.ck == SEG_CHUNK ? 5 : 4;
        ca.fmt_slot = segred::CNT_FMT; ca.fmt_by_table = segred::LISTS_BY_TABLE; ca.fmt_broken = segred::LISTS_BROKEN;
        const int64_t per_table = (L + ctx->T - 1) / ctx->T;
        const bool wide = ctx->T * csort::CLUSTER_WIDE * 2 <= ctx->num_sms && per_table >= csort::CLUSTER_WIDE * 1024;
        cudaError_t e = cudaErrorUnknown;
        if (wide) e = launch_cluster_sort<csort::CLUSTER_WIDE>(ctx, ca, per_table, st);
        if (e != cudaSuccess) e = launch_cluster_sort<csort::CLUSTER>(ctx, ca, per_table, st);
        if (e == cudaSuccess) {
            dq_mark(ctx, st, DQ_K_CLUSTER_SORT);
            skeys = keys[0];
            sorted = true;
        } else {
            ctx->last_cuda_error = (int)e;
        }
    }
    if (!sorted) {
    {
        int64_t blocks = (G + 255) / 256;
        int64_t cap = (int64_t)ctx->num_sms * 8;
        int grid = (int)(blocks > cap ? cap : blocks);
        prepare_kernel<<<grid, 256, 0, st>>>(indices, offsets, ctx->d_row_off, ctx->T, B, G, L, pairs[0],
                                             ctx->payload_position, ctx->d_status);
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_PREPARE);
    }
    const int64_t hist_chunks = (y.num_tiles + HIST_CHUNK - 1) / HIST_CHUNK;
    for (int p = 0; p < y.passes; ++p) {
        const uint2 *pin = pairs[p & 1];
        const int shift = p * y.digit_bits;
        sort_hist_kernel<<<(unsigned)y.num_tiles, ST_THREADS, 0, st>>>(pin, L, shift, y.nb, tilehist);
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_SORT_SCAN);
        sort_chunk_kernel<<<(unsigned)hist_chunks, NB_MAX, 0, st>>>(tilehist, y.num_tiles, y.nb, chunk_sum);
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_SORT_SCAN);
        sort_base_kernel<<<1, NB_MAX, 0, st>>>(chunk_sum, hist_chunks, y.nb, digit_base);
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_SORT_SCAN);
        if (p + 1 < y.passes)
            sort_scatter_kernel<false><<<(unsigned)y.num_tiles, ST_THREADS, 0, st>>>(
                pin, pairs[(p + 1) & 1], nullptr, nullptr, tilehist, chunk_sum, digit_base, L, shift, y.nb, ctx->d_status);
        else
            sort_scatter_kernel<true><<<(unsigned)y.num_tiles, ST_THREADS, 0, st>>>(
                pin, nullptr, keys[0], vals[0], tilehist, chunk_sum, digit_base, L, shift, y.nb, ctx->d_status);
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_SORT_SCATTER);
    }
        skeys = keys[0];
    }
    if (sorted && lists_by_table) return DQRM_OK;      // the lists are there; unique_rows and uniq_off come with the sums
    if (!sorted) {        // (a cluster sort that did not number the segments itself has counted the segment heads of every tile)
        seg_count_kernel<<<(unsigned)y.num_tiles, ST_THREADS, 0, st>>>(skeys, L, reinterpret_cast<u32 *>(ws + y.tile_heads));
        DQRM_CUDA_TRY(ctx, cudaGetLastError());
        dq_mark(ctx, st, DQ_K_SEG_COUNT);
    }
    seg_emit_kernel<<<(unsigned)y.num_tiles, ST_THREADS, (size_t)(ctx->T + 1) * sizeof(int64_t), st>>>(
        skeys, L, reinterpret_cast<const u32 *>(ws + y.tile_heads), ctx->d_row_off, ctx->T,
        reinterpret_cast<u32 *>(ws + y.seg_start), reinterpret_cast<u32 *>(ws + y.chunk_first), unique_rows, uniq_off,
        reinterpret_cast<u32 *>(ws + y.counters), y.ck);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_SEG_EMIT);
    return DQRM_OK;
}

// second half: segmented sum of the upstream gradient over the sorted lookups
int dq_launch_bwd_reduce(dqrm_ctx *ctx, const float *grad_out, int32_t *unique_rows, int32_t *uniq_off, float *grad_rows,
                         int B, int64_t L, void *ws_, size_t ws_bytes, cudaStream_t st)
{
    const Layout y = make_layout(ctx, L);
    if (ws_bytes < y.total) return DQRM_ERR_WORKSPACE;
    if (L == 0) return DQRM_OK;
    char *ws = reinterpret_cast<char *>(ws_);
    const int64_t G = (int64_t)ctx->T * B;
    // both sort paths leave the sorted pairs in the first key / payload buffers
    const u32 *skeys = reinterpret_cast<const u32 *>(ws + y.keys_a), *svals = reinterpret_cast<const u32 *>(ws + y.vals_a);
    const int D = ctx->D, d4 = D / 4;
#define DQ_RED(RL, RV, RC, LPR, CH) \
    return launch_reduce<RL, RV, RC, LPR, CH>(ctx, y, ws, skeys, svals, unique_rows, uniq_off, grad_out, grad_rows, L, G, st)
    if (D <= 4) DQ_RED(4, 1, 1, 1, 1);
    if (D <= 8) DQ_RED(8, 1, 1, 2, 1);
    if (D <= 16) DQ_RED(4, 4, 1, 4, 1);
    if (D <= 32) DQ_RED(16, 2, 1, 8, 1);
    if (D <= 64) DQ_RED(16, 4, 1, 16, 1);
    if (d4 <= 32) DQ_RED(32, 4, 1, 32, 1);
    if (d4 <= 64) DQ_RED(32, 4, 2, 32, 2);
    if (d4 <= 128) DQ_RED(32, 4, 4, 32, 4);
    DQ_RED(32, 4, 8, 32, 8);
#undef DQ_RED
}

int dq_launch_bwd(dqrm_ctx *ctx, const float *grad_out, const int32_t *indices, const int32_t *offsets,
                  int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int B, int64_t L,
                  void *ws, size_t ws_bytes, cudaStream_t st, const u32 **absmax_bits_out)
{
    int rc = dq_launch_bwd_sort(ctx, indices, offsets, unique_rows, uniq_off, B, L, ws, ws_bytes, st, absmax_bits_out, true);
    if (rc != DQRM_OK) return rc;
    return dq_launch_bwd_reduce(ctx, grad_out, unique_rows, uniq_off, grad_rows, B, L, ws, ws_bytes, st);
}
