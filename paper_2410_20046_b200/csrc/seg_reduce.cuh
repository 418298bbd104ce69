// Segmented reduction of the upstream gradient over the sorted lookups (second half of
// the backward; paper Section 4.3 / Appendix B.1: duplicates of a row are coalesced).
//
// Input: keys[L] (arena rows, ascending), vals[L] (row of grad_out for each lookup, in
// stable order), chunk_first[c] = index of the segment that holds sorted entry 32*c,
// seg_start[] = sorted position where every segment begins; the segments are numbered over
// the whole batch or per table (see LISTS_* below), and in the second case this kernel also
// writes unique_rows and uniq_off.  Work is dealt in chunks of 32 sorted entries, one lane group per chunk,
// but a segment is summed by the group in whose chunk it BEGINS, tail in the next chunk
// included; the group sees where that tail ends from the next chunk's keys, which it loads
// with its own.  All sums are FP64 and have a shape fixed by the entry positions, so results
// are reproducible.  Only a segment whose tail is not over within the next chunk (a hot row)
// is summed in pieces: every chunk it covers leaves an FP64 partial and the segment is
// finished by one of the fix-up kernels (a warp for up to 32 pieces, a block beyond that).
// The per-table abs-max of the rounded sums is collected on the way.
#pragma once
#include <type_traits>
#include "common.cuh"

namespace segred {

constexpr int CHUNK = 32;            // sorted entries per lane group of the reduce (16 for a small batch of narrow rows)
constexpr int PREFETCH_ROW_BYTES = 512;   // rows up to this size are prefetched into L2 by the reduce's head phase
constexpr int BIG_PIECES = 32;       // cut segments with more pieces go to the block-wide fix-up
enum { CNT_LONG = 0, CNT_U = 1, CNT_BIG = 2, CNT_FMT = 3 };
// counters[CNT_FMT]: how the segment lists that the sort left are laid out.
//   LISTS_GLOBAL    seg_start[u], chunk_first[c] and uniq_off[] number the segments over the whole batch (seg_emit)
//   LISTS_BY_TABLE  the cluster sort numbered each table's segments from 0: table t's starts sit at
//                   seg_start[tb[t] + t + .] (tb[t] = first sorted position of the table, one slot more than it
//                   has segments: the last holds the table's end), chunk_first[c] counts within the table that
//                   holds entry c*CK, table_cnt[t] says how many segments the table has; unique_rows and
//                   uniq_off are then written by the reduce, which adds the tables' bases
//   LISTS_BROKEN    a table's boundary offsets were unusable (reported): nothing is summed, no row is updated
enum { LISTS_GLOBAL = 0, LISTS_BY_TABLE = 1, LISTS_BROKEN = 2 };
struct ByTable {
    const u32 *table_cnt;       // [T]
    const u32 *tb;              // [T+1]
    const int64_t *row_off;     // [T+1]
    int32_t *unique_rows;       // [U] out
    int32_t *uniq_off;          // [T+1] out
};

template <int LPR>
__device__ __forceinline__ u32 group_mask()
{
    if constexpr (LPR >= 32) {
        return 0xffffffffu;
    } else {
        const int lane = threadIdx.x & 31;
        return ((1u << LPR) - 1u) << (lane / LPR * LPR);
    }
}

template <int LPR>
__device__ __forceinline__ float group_max(float m)
{
    const u32 gm = group_mask<LPR>();
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(gm, m, o));
    return m;
}

// running abs-max of one table at a time (segment numbers only ascend along a lane group's work)
struct AbsmaxTracker {
    int t = -1;
    u32 u_end = 0;          // first segment past table t
    float m = 0.f;
};

template <int LPR>
__device__ __forceinline__ void absmax_push(AbsmaxTracker &tr, u32 *absmax)
{
    float m = group_max<LPR>(tr.m);      // called group-uniformly
    if ((threadIdx.x % LPR) == 0 && tr.t >= 0 && m > 0.f) atomicMax(&absmax[tr.t], __float_as_uint(m));
    tr.m = 0.f;
}

// s_uoff[t] = first segment (unique row) of table t, s_uoff[T] = number of segments
template <int LPR>
__device__ __forceinline__ void absmax_note(AbsmaxTracker &tr, u32 u, float m, const u32 *s_uoff, int T, u32 *absmax)
{
    if (u >= tr.u_end) {
        absmax_push<LPR>(tr, absmax);
        int lo = 0, hi = T;              // invariant: s_uoff[lo] <= u < s_uoff[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_uoff[mid] <= u) lo = mid; else hi = mid;
        }
        tr.t = lo;
        tr.u_end = s_uoff[lo + 1];
    }
    tr.m = fmaxf(tr.m, m);
}

template <int CH>
__device__ __forceinline__ float round_store(const double (&acc)[CH][4], float *dst_row, int lane, int lpr, int d4)
{
    float m = 0.f;
#pragma unroll
    for (int ch = 0; ch < CH; ++ch) {
        int c4 = ch * lpr + lane;
        if (c4 < d4) {
            float4 r = make_float4((float)acc[ch][0], (float)acc[ch][1], (float)acc[ch][2], (float)acc[ch][3]);
            *reinterpret_cast<float4 *>(dst_row + 4 * c4) = r;
            m = fmaxf(fmaxf(m, fmaxf(fabsf(r.x), fabsf(r.y))), fmaxf(fabsf(r.z), fabsf(r.w)));
        }
    }
    return m;
}

// VEC consecutive floats (1, 2 or 4) as one load
template <int VEC> struct Vec;
template <> struct Vec<1> { typedef float type; };
template <> struct Vec<2> { typedef float2 type; };
template <> struct Vec<4> { typedef float4 type; };

template <int VEC>
__device__ __forceinline__ void vec_add(double (&acc)[VEC], const typename Vec<VEC>::type &v)
{
    if constexpr (VEC == 1) { acc[0] += (double)v; }
    else if constexpr (VEC == 2) { acc[0] += (double)v.x; acc[1] += (double)v.y; }
    else { acc[0] += (double)v.x; acc[1] += (double)v.y; acc[2] += (double)v.z; acc[3] += (double)v.w; }
}

// One lane group (LPR lanes) owns one chunk of 32 sorted entries and walks in order the segments that
// BEGIN in it, NB upstream-gradient rows in flight at a time: a segment's tail in the next chunk is
// read by the same group, and a leading run that began in the chunk before is skipped, so the common
// segment that straddles a chunk boundary needs no partial sum.  Lane `lane` holds, for ch < CH, the
// VEC consecutive features starting at (ch*LPR + lane)*VEC.  Per chunk, one lane per entry compares
// neighbouring keys once (this chunk's and the next one's); the resulting bit masks of segment heads
// and the payloads (parked in shared memory) are all the walk needs, so an entry costs one shared
// load, one address, one 128-bit load, a bit test and the FP64 adds.
// (256-byte rows want four resident blocks per SM: that caps the kernel at 64 registers.  64-byte rows are capped
// at three blocks' worth, 78 registers with a few spills: alone the kernel loses a microsecond, beside the sort of
// the next batch the step gains three, because the two then fit on an SM together)
template <int LPR, int VEC, int CH, bool EXACT, int CK = 32, bool OWN = (LPR >= 8)>
__global__ void __launch_bounds__(256, (LPR == 16 && VEC == 4 && CH == 1) ? 4 : (LPR == 4 && VEC == 4) ? 3 : 1)
seg_reduce_kernel(const u32 *__restrict__ keys, const u32 *__restrict__ vals,
                  const u32 *__restrict__ seg_start, const u32 *__restrict__ chunk_first,
                  const int32_t *__restrict__ uniq_off,
                  const float *__restrict__ grad_out, float *__restrict__ grad_rows,
                  double *__restrict__ partials, uint4 *__restrict__ long_list, u32 *__restrict__ counters,
                  u32 *__restrict__ absmax, int T, int D_any,
                  int64_t L, int64_t G, int64_t num_chunks, int *__restrict__ status, const ByTable bt)
{
    // EXACT: the feature size fills the lanes exactly, so it is a compile-time constant and the
    // per-vector range checks fall away
    const int D = EXACT ? LPR * VEC * CH : D_any;
    extern __shared__ unsigned char smem_raw[];
    u32 *s_uoff = reinterpret_cast<u32 *>(smem_raw);                                     // [T+1]
    u32 *s_tb = s_uoff + (T + 1);                                                        // [T+1] (lists by table)
    u32 *s_row = s_tb + (T + 1);                                                         // [T+1] (lists by table)
    u32 *s_vals = s_row + (T + 1) + (size_t)(threadIdx.x / LPR) * (2 * CK);           // this group's [2*CK]
    // (the first T+1 threads fetch what either layout of the lists needs before the layout is known, so that the
    // kernel starts with one round trip to memory, not two)
    u32 r_tb = 0u, r_cnt = 0u, r_uo = 0u, r_row = 0u;
    if ((int)threadIdx.x <= T) {
        r_tb = bt.tb[threadIdx.x];
        r_uo = (u32)uniq_off[threadIdx.x];
        r_row = (u32)bt.row_off[threadIdx.x];      // (arena rows are 32-bit keys throughout)
    }
    if ((int)threadIdx.x < T) r_cnt = bt.table_cnt[threadIdx.x];
    const u32 fmt = counters[CNT_FMT];
    if (fmt == LISTS_BROKEN) {                    // (block-uniform)
        if (blockIdx.x == 0) {
            for (int t = threadIdx.x; t <= T; t += blockDim.x) bt.uniq_off[t] = 0;
            if (threadIdx.x == 0) counters[CNT_U] = 0u;
        }
        return;
    }
    const bool by_table = fmt == LISTS_BY_TABLE;
    if (by_table) {
        // the tables' first segments: a running sum over their segment counts (T is small against the batch; one
        // warp adds them up 32 at a time)
        if (threadIdx.x < 32) {
            u32 run = 0;
            for (int t0 = 0; t0 < T; t0 += 32) {
                const int t = t0 + (int)threadIdx.x;
                const u32 cnt = t0 == 0 ? r_cnt : (t < T ? bt.table_cnt[t] : 0u);
                u32 incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const u32 v = __shfl_up_sync(0xffffffffu, incl, o);
                    if ((int)threadIdx.x >= o) incl += v;
                }
                if (t < T) s_uoff[t] = run + incl - cnt;
                run += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (threadIdx.x == 0) s_uoff[T] = run;
        }
        for (int t = threadIdx.x; t <= T; t += blockDim.x) {
            s_tb[t] = t == (int)threadIdx.x ? r_tb : bt.tb[t];
            s_row[t] = t == (int)threadIdx.x ? r_row : (u32)bt.row_off[t];
        }
        __syncthreads();
        if (blockIdx.x == 0) {
            for (int t = threadIdx.x; t <= T; t += blockDim.x) bt.uniq_off[t] = (int32_t)s_uoff[t];
            if (threadIdx.x == 0) counters[CNT_U] = s_uoff[T];
        }
    } else {
        for (int t = threadIdx.x; t <= T; t += blockDim.x) s_uoff[t] = t == (int)threadIdx.x ? r_uo : (u32)uniq_off[t];
        __syncthreads();
    }

    typedef typename Vec<VEC>::type vec_t;
    constexpr int NB = (VEC == 4 && LPR > 4) ? 4 : 8;   // rows in flight per lane
    constexpr int EPL = CK / LPR;              // chunk entries one lane looks at
    const int dv = D / VEC;                       // vectors per row
    const int lane = threadIdx.x % LPR;
    const u32 gmask = group_mask<LPR>();
    const int gbase = (threadIdx.x & 31) / LPR * LPR;
    const vec_t *g_lane = reinterpret_cast<const vec_t *>(grad_out) + lane;
    const int64_t group = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t)gridDim.x * blockDim.x / LPR;
    AbsmaxTracker tr;
    bool bad = false;
    const uint64_t keep = dq_policy_evict_last();

    for (int64_t c = group; c < num_chunks; c += n_groups) {
        const int64_t i0 = c * CK;
        const int n = (int)(min(i0 + (int64_t)CK, L) - i0);
        const int n_next = (int)max((int64_t)0, min((int64_t)CK, L - i0 - CK));
        // Heads: entry e starts a segment when its key differs from the key before it; the same for the
        // chunk behind, whose first head tells where this chunk's last segment ends.  All loads are issued
        // before the first vote so that they are in flight together.
        u32 kc[EPL], kp[EPL], vv[EPL], kn[OWN ? EPL : 1], knp[OWN ? EPL : 1], vn[OWN ? EPL : 1];
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
            const int e = j * LPR + lane;
            const int64_t i = i0 + e;
            kc[j] = kp[j] = vv[j] = 0u;
            if (e < n) {
                vv[j] = vals[i];
                kc[j] = keys[i];
                kp[j] = i > 0 ? keys[i - 1] : ~kc[j];
            }
            if (OWN) {
                kn[j] = knp[j] = vn[j] = 0u;
                if (e < n_next) {
                    vn[j] = vals[i + CK];
                    kn[j] = keys[i + CK];
                    knp[j] = keys[i + CK - 1];
                }
            }
        }
        // OWN: did the run that enters this chunk begin in the chunk before?  (the keys ascend: it did unless the
        // key 33 entries back is still the same).  Otherwise: the key behind the chunk tells whether its last run ends
        u32 k_x = 0u;
        if (OWN) { if (i0 > CK) k_x = keys[i0 - CK - 1]; }
        else if (i0 + n < L) k_x = keys[i0 + n];
        u32 u_first = chunk_first[c];
        int t_first = 0;                          // lists by table: the table that holds the chunk's first entry
        if (by_table) {
            int lo = 0, hi = T;                   // largest t with s_tb[t] <= i0 (empty tables share a start: the last)
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if ((int64_t)s_tb[mid] <= i0) lo = mid; else hi = mid;
            }
            t_first = lo;
            u_first += s_uoff[lo];
        }
        __syncwarp(gmask);                        // the previous chunk's payloads are no longer read
        u32 heads = 0, heads_n = 0;
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
            const int e = j * LPR + lane;
            if (e < n) {
                u32 v = vv[j];
                if ((int64_t)v >= G) { bad = true; v = 0u; }
                s_vals[e] = v;
                // the walk reaches this entry's upstream-gradient row up to 32 dependent steps from now: have L2
                // fetch it meanwhile, so that all of a chunk's rows are in flight at once without holding registers
                if (PREFETCH_ROW_BYTES >= D * (int)sizeof(float)) {
                    const char *row = reinterpret_cast<const char *>(grad_out) + (int64_t)v * D * sizeof(float);
#pragma unroll
                    for (int b = 0; b < PREFETCH_ROW_BYTES; b += 128)
                        if (b < D * (int)sizeof(float)) dq_prefetch_l2(row + b);
                }
            }
            const u32 lm = LPR >= 32 ? 0xffffffffu : ((1u << LPR) - 1u);
            if (OWN) {
                if (e < n_next) {
                    u32 v = vn[j];
                    if ((int64_t)v >= G) { bad = true; v = 0u; }
                    s_vals[CK + e] = v;
                }
                const bool head_n = (e < n_next) && (kn[j] != knp[j]);
                heads_n |= ((__ballot_sync(gmask, head_n) >> gbase) & lm) << (j * LPR);
            }
            const bool head = (e < n) && (kc[j] != kp[j]);
            heads |= ((__ballot_sync(gmask, head) >> gbase) & lm) << (j * LPR);
        }
        if (by_table) {
            // every entry that starts a segment names the segment's row: segment of entry e = u_first + heads in (0, e]
            u32 base = s_row[t_first];
            const bool one_table = (int64_t)s_tb[min(t_first + 1, T)] >= i0 + n;     // (group-uniform)
#pragma unroll
            for (int j = 0; j < EPL; ++j) {
                const int e = j * LPR + lane;
                if (e < n && kc[j] != kp[j]) {
                    if (!one_table) {             // the chunk straddles tables: this key's own table
                        int lo = t_first, hi = T;
                        while (hi - lo > 1) {
                            const int mid = (lo + hi) >> 1;
                            if (s_row[mid] <= kc[j]) lo = mid; else hi = mid;
                        }
                        base = s_row[lo];
                    }
                    const u32 ue = u_first + __popc(heads & ~1u & (0xffffffffu >> (31 - e)));
                    bt.unique_rows[ue] = (int32_t)(kc[j] - base);
                }
            }
        }
        if (n_next < CK) heads_n |= 1u << n_next;   // the end of the array closes a run like a head
        const u32 k_0 = __shfl_sync(gmask, kc[0], gbase);
        // the chunk's last key sits in lane (n-1) % LPR, register (n-1) / LPR
        u32 k_last = 0u;
#pragma unroll
        for (int j = 0; j < EPL; ++j)
            if ((n - 1) / LPR == j) k_last = kc[j];
        k_last = __shfl_sync(gmask, k_last, gbase + (n - 1) % LPR);
        __syncwarp(gmask);

        // ---- which entries this group sums: [ea, eb) relative to i0, eb up to 2*CK.
        // A segment is summed where it BEGINS, together with its tail in the next chunk; a leading run that
        // began in the chunk before and ends here was summed there.  Only a segment whose tail is not over
        // within the next chunk is summed in pieces (FP64 partials, folded by the fix-up kernel).
        // (Without OWN - rows so narrow that the extra keys and payloads would cost more registers than the
        // fix-up saves - a group sums exactly its chunk and every run cut by a chunk boundary is a piece.)
        const bool any_head = heads != 0u;
        const int f = any_head ? __ffs(heads) - 1 : n;                 // first head (n: none)
        bool lead_piece, trail_long;
        int ea, eb;
        if (OWN) {
            const bool closes_here = any_head || n < CK;
            const bool began_prev = (i0 <= CK) || (k_x != k_0);
            lead_piece = f > 0 && !(closes_here && began_prev);
            ea = lead_piece ? 0 : f;
            trail_long = any_head && heads_n == 0u;
            eb = n + ((any_head && heads_n != 0u) ? __ffs(heads_n) - 1 : 0);    // (an extension only when n == CK)
        } else {
            lead_piece = f > 0;
            ea = 0;
            trail_long = !((i0 + n == L) || (k_x != k_last));
            eb = n;
        }
        if (eb <= ea) continue;                   // group-uniform
        heads &= ~1u;                             // the walk starts a run at its first entry either way
        u32 u = u_first + ((ea > 0) ? 1u : 0u);   // segment of entry ea (ea > 0: it is the chunk's first head)
        int run_start = ea;
        double acc[CH][VEC];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch)
#pragma unroll
            for (int q = 0; q < VEC; ++q) acc[ch][q] = 0.0;

        // closes run [rs, re) (chunk-relative) of segment u
        auto flush = [&](int rs, int re) {
            const bool begins = !(lead_piece && rs == 0);
            const bool ends = !(trail_long && re == eb);
            if (begins && ends) {
                float m = 0.f;
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int cv = ch * LPR + lane;
                    if (EXACT || cv < dv) {
                        float *dst = grad_rows + (int64_t)u * D + cv * VEC;
                        if constexpr (VEC == 1) { float r = (float)acc[ch][0]; *dst = r; m = fmaxf(m, fabsf(r)); }
                        else if constexpr (VEC == 2) {
                            float2 r = make_float2((float)acc[ch][0], (float)acc[ch][1]);
                            *reinterpret_cast<float2 *>(dst) = r;
                            m = fmaxf(m, fmaxf(fabsf(r.x), fabsf(r.y)));
                        } else {
                            float4 r = make_float4((float)acc[ch][0], (float)acc[ch][1], (float)acc[ch][2], (float)acc[ch][3]);
                            dq_st_keep(reinterpret_cast<float4 *>(dst), r, keep);   // quantise+update reads it next
                            m = fmaxf(fmaxf(m, fmaxf(fabsf(r.x), fabsf(r.y))), fmaxf(fabsf(r.z), fabsf(r.w)));
                        }
                    }
                }
                absmax_note<LPR>(tr, u, m, s_uoff, T, absmax);
            } else {
                double *pdst = partials + ((size_t)c * 2 + (begins ? 1 : 0)) * D;
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int cv = ch * LPR + lane;
                    if (EXACT || cv < dv) {
#pragma unroll
                        for (int q = 0; q < VEC; ++q) pdst[cv * VEC + q] = acc[ch][q];
                    }
                }
                if (begins && lane == 0) {
                    // the segment begins here: leave all the fix-up needs to know about it in one record
                    int lo = 0, hi = T;              // its table: largest t with s_uoff[t] <= u
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (s_uoff[mid] <= u) lo = mid; else hi = mid;
                    }
                    // (lists by table: the table's starts sit at seg_start[tb[t] + t + .], the slot behind its last
                    // segment holds its end)
                    const int64_t at = by_table ? (int64_t)s_tb[lo] + lo + (u - s_uoff[lo]) : (int64_t)u;
                    const u32 sa = seg_start[at], sb = seg_start[at + 1];
                    const u32 npieces = (sb - 1) / CK - sa / CK + 1;
                    const uint4 rec = make_uint4(u, sa / CK, npieces, (u32)lo);
                    // (the list has a slot per chunk and every chunk begins at most one such segment; the bound only
                    // matters for a workspace that is summed twice without a sort in between, which must not write
                    // outside the list)
                    if (npieces > BIG_PIECES) {
                        const u32 k = atomicAdd(&counters[CNT_BIG], 1u);
                        if ((int64_t)k < num_chunks) long_list[num_chunks - 1 - k] = rec;
                    } else {
                        const u32 k = atomicAdd(&counters[CNT_LONG], 1u);
                        if ((int64_t)k < num_chunks) long_list[k] = rec;
                    }
                }
            }
        };

        // whole batches of NB entries need no per-entry range checks
        auto walk = [&](int e0, auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            vec_t r[NB][CH];
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                if (FULL || e0 + k < eb) {
                    const vec_t *src = g_lane + (int64_t)s_vals[e0 + k] * dv;
#pragma unroll
                    for (int ch = 0; ch < CH; ++ch)
                        if (EXACT || ch * LPR + lane < dv) r[k][ch] = __ldcs(src + ch * LPR);   // every row is read once
                }
            }
#pragma unroll
            for (int k = 0; k < NB; ++k) {
                const int e = e0 + k;
                if (FULL || e < eb) {
                    if (e > ea && e < CK && ((heads >> e) & 1u)) {
                        flush(run_start, e);
                        u += 1;
                        run_start = e;
#pragma unroll
                        for (int ch = 0; ch < CH; ++ch)
#pragma unroll
                            for (int q = 0; q < VEC; ++q) acc[ch][q] = 0.0;
                    }
#pragma unroll
                    for (int ch = 0; ch < CH; ++ch)
                        if (EXACT || ch * LPR + lane < dv) vec_add<VEC>(acc[ch], r[k][ch]);
                }
            }
        };
        int e0 = ea;
        for (; e0 + NB <= eb; e0 += NB) walk(e0, std::true_type{});
        if (e0 < eb) walk(e0, std::false_type{});
        flush(run_start, eb);
    }
    absmax_push<LPR>(tr, absmax);      // group-uniform: all lanes of a group walk the same chunks
    if (bad) dq_report(status, DQRM_ERR_INDEX_RANGE);
}

// pieces of a listed segment: the chunk in which it begins holds the first (slot 1), later chunks slot 0
__device__ __forceinline__ const double *piece_ptr(const double *partials, int64_t c0, int64_t p, int D)
{
    return partials + ((size_t)(c0 + p) * 2 + (p == 0 ? 1 : 0)) * D;
}

template <int CH, int UN>
__device__ __forceinline__ void add_pieces(double (&acc)[CH][4], const double *partials, int64_t c0,
                                           int64_t p_begin, int64_t p_end, int64_t stride, int D, int lane,
                                           int lpr, int d4)
{
    for (int64_t p = p_begin; p < p_end; p += stride * UN) {
        double2 x[UN][CH], y[UN][CH];
#pragma unroll
        for (int k = 0; k < UN; ++k) {
            const int64_t pk = p + k * stride;
            if (pk < p_end) {
                const double *src = piece_ptr(partials, c0, pk, D);
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    int c4 = ch * lpr + lane;
                    if (c4 < d4) {
                        x[k][ch] = __ldcg(reinterpret_cast<const double2 *>(src + 4 * c4));
                        y[k][ch] = __ldcg(reinterpret_cast<const double2 *>(src + 4 * c4 + 2));
                    }
                }
            }
        }
#pragma unroll
        for (int k = 0; k < UN; ++k) {
            if (p + k * stride < p_end) {
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    int c4 = ch * lpr + lane;
                    if (c4 < d4) {
                        acc[ch][0] += x[k][ch].x; acc[ch][1] += x[k][ch].y;
                        acc[ch][2] += y[k][ch].x; acc[ch][3] += y[k][ch].y;
                    }
                }
            }
        }
    }
}

// A record of the list: x = segment (unique row), y = chunk in which it begins, z = number of pieces, w = table.

// one warp per listed segment of at most BIG_PIECES pieces
template <int LPR, int CH>
__device__ __forceinline__ void
fixup_small(const double *__restrict__ partials, const uint4 *__restrict__ long_list, u32 count,
            float *__restrict__ grad_rows, u32 *__restrict__ absmax, int D)
{
    constexpr int SG = 32 / LPR;
    const int d4 = D >> 2;
    const int wl = threadIdx.x & 31;
    const int sub = wl / LPR, lane = wl % LPR;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t s = warp; s < count; s += n_warps) {
        const uint4 rec = __ldcg(long_list + s);
        double acc[CH][4];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) acc[ch][0] = acc[ch][1] = acc[ch][2] = acc[ch][3] = 0.0;
        add_pieces<CH, 4>(acc, partials, rec.y, sub, rec.z, SG, D, lane, LPR, d4);
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
            for (int ch = 0; ch < CH; ++ch)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[ch][q] += __shfl_xor_sync(0xffffffffu, acc[ch][q], o);
        float m = 0.f;
        if (sub == 0) m = round_store<CH>(acc, grad_rows + (int64_t)rec.x * D, lane, LPR, d4);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (wl == 0 && m > 0.f) atomicMax(&absmax[rec.w], __float_as_uint(m));
    }
}

// one block per listed segment of more than BIG_PIECES pieces (the hottest rows)
template <int LPR, int CH>
__device__ __forceinline__ void
fixup_big(const double *__restrict__ partials, const uint4 *__restrict__ long_list, u32 count,
          float *__restrict__ grad_rows, u32 *__restrict__ absmax, int D, int64_t num_chunks,
          double *s_part /*[256/LPR][D]*/)
{
    constexpr int NSG = 256 / LPR;
    const int d4 = D >> 2;
    const int sub = threadIdx.x / LPR, lane = threadIdx.x % LPR;
    for (u32 s = blockIdx.x; s < count; s += gridDim.x) {
        const uint4 rec = __ldcg(long_list + (num_chunks - 1 - s));
        double acc[CH][4];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) acc[ch][0] = acc[ch][1] = acc[ch][2] = acc[ch][3] = 0.0;
        add_pieces<CH, (CH == 1 ? 8 : 4)>(acc, partials, rec.y, sub, rec.z, NSG, D, lane, LPR, d4);
        __syncthreads();
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
            int c4 = ch * LPR + lane;
            if (c4 < d4) {
                double *dst = s_part + (size_t)sub * D + 4 * c4;
                dst[0] = acc[ch][0]; dst[1] = acc[ch][1]; dst[2] = acc[ch][2]; dst[3] = acc[ch][3];
            }
        }
        __syncthreads();
        if (sub == 0) {
            // lane group 0 adds the NSG sub-sums in order
            float m = 0.f;
#pragma unroll
            for (int ch = 0; ch < CH; ++ch) {
                int c4 = ch * LPR + lane;
                if (c4 < d4) {
                    double t0 = 0, t1 = 0, t2 = 0, t3 = 0;
                    for (int g = 0; g < NSG; ++g) {
                        const double *src = s_part + (size_t)g * D + 4 * c4;
                        t0 += src[0]; t1 += src[1]; t2 += src[2]; t3 += src[3];
                    }
                    float4 r = make_float4((float)t0, (float)t1, (float)t2, (float)t3);
                    *reinterpret_cast<float4 *>(grad_rows + (int64_t)rec.x * D + 4 * c4) = r;
                    m = fmaxf(fmaxf(m, fmaxf(fabsf(r.x), fabsf(r.y))), fmaxf(fabsf(r.z), fabsf(r.w)));
                }
            }
            m = group_max<LPR>(m);
            if (lane == 0 && m > 0.f) atomicMax(&absmax[rec.w], __float_as_uint(m));
        }
    }
}

// both fix-ups in one launch: every block first takes its share of the hottest rows, then its
// warps take the other listed segments
template <int LPR, int CH>
__global__ void __launch_bounds__(256)
seg_fixup_kernel(const double *__restrict__ partials, const uint4 *__restrict__ long_list,
                 const u32 *__restrict__ counters, float *__restrict__ grad_rows, u32 *__restrict__ absmax,
                 int D, int64_t num_chunks)
{
    extern __shared__ unsigned char smem_raw[];
    double *s_part = reinterpret_cast<double *>(smem_raw);                         // [256/LPR][D]
    const u32 n_big = (u32)min((int64_t)__ldcg(counters + CNT_BIG), num_chunks);
    const u32 n_small = (u32)min((int64_t)__ldcg(counters + CNT_LONG), num_chunks);
    fixup_big<LPR, CH>(partials, long_list, n_big, grad_rows, absmax, D, num_chunks, s_part);
    fixup_small<LPR, CH>(partials, long_list, n_small, grad_rows, absmax, D);
}

}  // namespace segred
