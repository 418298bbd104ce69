// Per-table stable sort of a batch's lookups by row, one thread-block cluster per table.
//
// The lookups of a batch arrive table-major, so sorting them by arena row is T independent
// sorts of a few thousand to a few tens of thousands of keys each.  A cluster of eight
// blocks owns one table: every block holds one eighth of the table's (row, payload) pairs
// in shared memory, and a least-significant-digit radix sort (8-bit digits, only as many
// passes as the table's row count needs) moves the pairs between the blocks' shared
// memories with distributed-shared-memory stores.  Per pass: per-warp digit counts over
// the block's slice (shared-memory atomics), the eight per-block histograms are exchanged
// through DSMEM, every block derives its scatter offsets, ranks its slice in order (warp ballots, stable)
// and scatters.  Cluster barriers separate the phases; no block waits on anything else.
// Tables whose lookups do not fit the shared-memory slices use the same algorithm on
// global staging buffers.  The result - keys (arena rows) ascending, payloads (rows of
// grad_out) in the original order within equal keys - is written table-major, which is
// the globally sorted order the segmented reduction expects.  On the way out the cluster
// also finds where every row's run begins: either it numbers its table's segments itself
// (the kernel that sums them adds the tables' bases), or it counts the segment starts per
// 2048-entry tile for a kernel that numbers them over the whole batch.
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"


namespace csort {

namespace cg = cooperative_groups;

constexpr int THREADS = 512;
constexpr int WARPS = THREADS / 32;
constexpr int CLUSTER = 8;            // blocks per table
constexpr int CLUSTER_WIDE = 16;      // ... when the batch has so few tables that eight blocks each would leave most SMs idle
constexpr int BINS = 256;

struct Args {
    const int32_t *indices;
    const int32_t *offsets;
    const int64_t *row_off;
    int T, B;
    int64_t L;
    u32 *keys_out, *vals_out;       // [L] sorted result
    uint2 *gp[2];                   // [L] global staging of pairs (tables too large for shared memory)
    int cap;                        // pairs per block that fit in shared memory
    int payload_position;           // 0: payload = row of grad_out [B][T][D]; 1: payload = position of the lookup in indices
    int *status;
    u32 *tile_heads;                // [ceil(L / 2048)] zeroed by the caller: segment heads per tile of the sorted order
    // lists_by_table: instead of the per-tile head counts (from which a later kernel numbers the segments over the
    // whole batch), every cluster numbers its own table's segments from 0 and leaves
    //   seg_start[tb0 + t + u] = sorted position where the table's segment u begins, [.. + count] = the table's end
    //   chunk_first[c]         = the table's segment that holds sorted entry c << ck_shift (for c inside the table)
    //   table_cnt[t], tb[t]    = segments and first sorted position of table t (tb[T] = L)
    // and counters[fmt_slot] says so; the kernel that sums the segments adds the tables' bases
    int lists_by_table;
    u32 *seg_start, *chunk_first, *table_cnt, *tb, *counters;
    int ck_shift, fmt_slot, fmt_by_table, fmt_broken;
};

__device__ __forceinline__ u32 *remote(cg::cluster_group &cluster, u32 *p, unsigned rank)
{
    return cluster.map_shared_rank(p, rank);
}

// lanes of the warp that hold the same 8-bit digit as this lane (one call by all lanes; a lane without an
// entry matches nobody)
__device__ __forceinline__ u32 same_digit_lanes(u32 d, bool valid)
{
    const u32 peers = __match_any_sync(0xffffffffu, valid ? d : 256u + (threadIdx.x & 31));
    return valid ? peers : 0u;
}

// (no minimum of resident blocks is asked for: with one, the compiler spends registers that the kernels running
// beside the sort then lack - measured, the training step beside it went from 61 to 72 us)
template <int CL>
__global__ void __launch_bounds__(THREADS)
cluster_sort_kernel(const Args a)
{
    extern __shared__ uint2 s_dyn[];               // pair buffers [2][cap]: (row within table, payload)
    __shared__ u32 s_cnt[WARPS][BINS];
    __shared__ u32 s_hist[BINS];
    __shared__ u32 s_scan[BINS / 32];
    __shared__ u32 s_wheads[WARPS];                // write-out: segment starts in each warp's part of the slice
    __shared__ u32 s_totals[16];                   // ... and in every block's slice (each block sends its own)
    __shared__ u32 s_cbase, s_ctotal;              // ... in the blocks before this one, and in the whole table

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned c = cluster.block_rank();
    const int t = blockIdx.x / CL;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const u32 lt = (1u << lane) - 1u;

    int64_t tb0 = __ldg(a.offsets + (int64_t)t * a.B), tb1 = __ldg(a.offsets + (int64_t)(t + 1) * a.B);
    if (tb0 < 0 || tb1 < tb0 || tb1 > a.L) {
        if (threadIdx.x == 0 && c == 0) {
            dq_report(a.status, DQRM_ERR_INDEX_RANGE);
            if (a.lists_by_table) atomicMax(&a.counters[a.fmt_slot], (u32)a.fmt_broken);   // nothing downstream runs
        }
        return;                                    // uniform over the cluster
    }
    const int64_t n = tb1 - tb0;
    if (a.lists_by_table && c == 0 && threadIdx.x == 0) {
        a.tb[t] = (u32)tb0;
        if (t == a.T - 1) a.tb[a.T] = (u32)tb1;
        if (t == 0) atomicMax(&a.counters[a.fmt_slot], (u32)a.fmt_by_table);
        if (n == 0) a.table_cnt[t] = 0u;
    }
    if (n == 0) return;
    const int64_t r0 = __ldg(a.row_off + t);
    const int64_t nrows = __ldg(a.row_off + t + 1) - r0;
    const int npc = (int)(((n + CL - 1) / CL + 31) / 32 * 32);      // pairs per block
    const bool in_smem = npc <= a.cap;
    const int my_n = (int)max((int64_t)0, min((int64_t)npc, n - (int64_t)c * npc));
    // the scatter divides every destination by npc: a float reciprocal gives the quotient (a block number,
    // since pos < n <= CL * npc) to within one, and one correction step settles it
    const float npc_inv = 1.0f / (float)npc;

    // buffers of this block for stage s (shared memory slices, or this block's part of the global staging)
    // a pair travels as one 8-byte store: distributed-shared-memory traffic is bound by the number of stores
    uint2 *pb0, *pb1;
    if (in_smem) {
        pb0 = s_dyn; pb1 = s_dyn + a.cap;
    } else {
        pb0 = a.gp[0] + tb0 + (int64_t)c * npc; pb1 = a.gp[1] + tb0 + (int64_t)c * npc;
    }
    // ---- load this block's slice: key = row within the table, payload = row of grad_out ----
    // In a table of one-index bags in order (n == B and offsets = identity, the Criteo-shaped case) the bag of
    // the lookup at position p is bag p.  That is checked per lookup from the two offsets around it, which are
    // loaded together with the index, so nothing here waits on another block.  Any other lookup finds its
    // bag by a search of the offsets, which must not decrease inside the table.
    const int32_t *off_t = a.offsets + (int64_t)t * a.B;
    if (n != a.B) {
        bool dec = false;
        const int per = (a.B + CL - 1) / CL;
        const int b0 = c * per, b1 = min(a.B, b0 + per);
        for (int i = b0 + threadIdx.x; i < b1; i += THREADS) dec |= __ldg(off_t + i) > __ldg(off_t + i + 1);
        if (dec) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 &&
        (__ldg(a.offsets) != 0 || (int64_t)__ldg(a.offsets + (int64_t)a.T * a.B) != a.L))
        dq_report(a.status, DQRM_ERR_INDEX_RANGE);
    bool bad = false;
    for (int i = threadIdx.x; i < my_n; i += THREADS) {
        const int64_t p = (int64_t)c * npc + i;    // position within the table's lookups
        int32_t idx = __ldg(a.indices + tb0 + p);
        bool single = false;
        if (n == a.B) {
            const int64_t o0 = __ldg(off_t + p), o1 = __ldg(off_t + p + 1);
            single = o0 == tb0 + p && o1 == tb0 + p + 1;
            if (o0 > o1) dq_report(a.status, DQRM_ERR_INDEX_RANGE);
        }
        bad |= (idx < 0) | (idx >= nrows);
        idx = (int32_t)min((int64_t)max(idx, 0), nrows - 1);
        int64_t bag = p;
        if (!single) {                             // largest bag b with offsets[t*B + b] <= tb0 + p
            int lo = 0, hi = a.B;
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if ((int64_t)__ldg(off_t + mid) <= tb0 + p) lo = mid; else hi = mid;
            }
            bag = lo;
        }
        pb0[i] = make_uint2((u32)idx, a.payload_position ? (u32)(tb0 + p) : (u32)(bag * a.T + t));
    }
    if (bad) dq_report(a.status, DQRM_ERR_INDEX_RANGE);

    int bits = 0;
    while (((int64_t)1 << bits) < nrows) ++bits;
    const int passes = (bits + 7) / 8;
    // the slice of this block is cut into WARPS contiguous parts, walked 32 entries at a time
    const int wsz = ((my_n + WARPS - 1) / WARPS + 31) / 32 * 32;
    const int w0 = min(my_n, warp * wsz), w1 = min(my_n, w0 + wsz);

    int s = 0;
    __syncthreads();
    // a one-row table takes no pass, so no cluster barrier separates the loads above from the
    // neighbour's read of this slice's last pair in the write-out below
    if (passes == 0) cluster.sync();
    for (int pass = 0; pass < passes; ++pass) {
        const int shift = 8 * pass;
        const uint2 *src = s ? pb1 : pb0;                           // this pass reads stage s ...
        uint2 *dst = s ? pb0 : pb1;                                 // ... and fills the other one
        uint2 *gdst = s ? a.gp[0] : a.gp[1];
        for (int i = threadIdx.x; i < WARPS * BINS; i += THREADS) (&s_cnt[0][0])[i] = 0u;
        __syncthreads();
        // phase 1: digit counts of this warp's part
        for (int i = w0 + lane; i < w1; i += 32) atomicAdd(&s_cnt[warp][(src[i].x >> shift) & 255u], 1u);
        __syncthreads();
        if (threadIdx.x < BINS) {
            u32 h = 0;
#pragma unroll 8
            for (int w = 0; w < WARPS; ++w) h += s_cnt[w][threadIdx.x];
            s_hist[threadIdx.x] = h;
        }
        cluster.sync();
        // offsets: digits first, then blocks of the cluster, then warps of this block
        u32 tot = 0, pre = 0, incl = 0;
        if (threadIdx.x < BINS) {                  // one thread per digit (the first BINS / 32 warps)
            u32 h[CL];
#pragma unroll
            for (unsigned cc = 0; cc < CL; ++cc) h[cc] = *remote(cluster, &s_hist[threadIdx.x], cc);
#pragma unroll
            for (unsigned cc = 0; cc < CL; ++cc) { if (cc < c) pre += h[cc]; tot += h[cc]; }
            incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                u32 v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) s_scan[warp] = incl;
        }
        __syncthreads();
        if (threadIdx.x < BINS) {
            u32 woff = 0;
            for (int w = 0; w < warp; ++w) woff += s_scan[w];
            u32 run = woff + incl - tot + pre;      // first destination of (digit, this block)
#pragma unroll 8
            for (int w = 0; w < WARPS; ++w) {
                const u32 cnt = s_cnt[w][threadIdx.x];
                s_cnt[w][threadIdx.x] = run;
                run += cnt;
            }
        }
        __syncthreads();
        // phase 2: rank again and scatter into the owners' buffers of the other stage
        for (int i0 = w0; i0 < w1; i0 += 32) {
            const int i = i0 + lane;
            const bool valid = i < w1;
            const uint2 pr = valid ? src[i] : make_uint2(0u, 0u);
            const u32 key = pr.x;
            const u32 d = (key >> shift) & 255u;
            const u32 peers = same_digit_lanes(d, valid);
            const int leader = __ffs(peers) - 1;
            u32 base = 0;
            if (valid && lane == leader) { base = s_cnt[warp][d]; s_cnt[warp][d] = base + __popc(peers); }
            base = __shfl_sync(0xffffffffu, base, leader);
            __syncwarp();
            if (valid) {
                const u32 pos = base + __popc(peers & lt);      // position within the table, < n
                if ((int64_t)pos < n) {
                    if (in_smem) {
                        unsigned owner = (unsigned)((float)pos * npc_inv);       // within one of pos / npc
                        if (owner * (u32)npc > pos) --owner;
                        else if ((owner + 1u) * (u32)npc <= pos) ++owner;
                        const u32 j = pos - owner * npc;
                        cluster.map_shared_rank(dst, owner)[j] = pr;
                    } else {
                        gdst[tb0 + pos] = pr;
                    }
                }
            }
        }
        cluster.sync();
        s ^= 1;
    }
    // ---- write the sorted slice: arena row keys ----
    // and either count, per 2048-entry tile of the sorted order, the entries that start a new row, or number the
    // table's segments right here
    {
        const uint2 *fin = s ? pb1 : pb0;
        u32 prev_last = 0xFFFFFFFFu;               // last row of the previous block's slice (full by construction)
        if (c > 0) {
            const uint2 *pf = in_smem ? cluster.map_shared_rank(s ? pb1 : pb0, c - 1)
                                      : (s ? a.gp[1] : a.gp[0]) + tb0 + (int64_t)(c - 1) * npc;
            prev_last = pf[npc - 1].x;
        }
        if (!a.lists_by_table) {
            for (int i0 = warp * 32; i0 < my_n; i0 += THREADS) {
                const int i = i0 + lane;
                const bool valid = i < my_n;
                const int64_t j = tb0 + (int64_t)c * npc + i;
                bool head = false;
                if (valid) {
                    const uint2 pr = fin[i];
                    a.keys_out[j] = (u32)(r0 + pr.x);
                    a.vals_out[j] = pr.y;
                    const u32 before = i > 0 ? fin[i - 1].x : prev_last;
                    head = (c == 0 && i == 0) || before != pr.x;
                }
                const int64_t tile = j >> 11;
                const int64_t tile0 = __shfl_sync(0xffffffffu, tile, 0);
                const u32 m0 = __ballot_sync(0xffffffffu, head && tile == tile0);
                const u32 m1 = __ballot_sync(0xffffffffu, head && tile != tile0);
                if (lane == 0) {
                    if (m0) atomicAdd(&a.tile_heads[tile0], __popc(m0));
                    if (m1) atomicAdd(&a.tile_heads[tile0 + 1], __popc(m1));
                }
            }
        } else {
            // every warp takes a contiguous part [w0, w1) of the slice, so that the segment starts before an entry
            // are those of the blocks before, of the warps before, and a count the warp carries along
            // (a part of up to 1024 entries: lane k keeps the 32 head bits of the part's k-th round, so that the
            // second walk need not read the pairs again)
            const bool few = wsz <= 1024;
            u32 mine = 0, kept = 0;
            for (int i0 = w0, it = 0; i0 < w1; i0 += 32, ++it) {
                const int i = i0 + lane;
                bool head = false;
                if (i < w1) {
                    const int64_t j = tb0 + (int64_t)c * npc + i;
                    const uint2 pr = fin[i];
                    a.keys_out[j] = (u32)(r0 + pr.x);
                    a.vals_out[j] = pr.y;
                    const u32 before = i > 0 ? fin[i - 1].x : prev_last;
                    head = (c == 0 && i == 0) || before != pr.x;
                }
                const u32 m = __ballot_sync(0xffffffffu, head);
                if (lane == it) kept = m;
                mine += __popc(m);
            }
            if (lane == 0) s_wheads[warp] = mine;
            __syncthreads();
            if (warp == 0) {                       // the warps' bases within the block, and the block's total
                const u32 v = lane < WARPS ? s_wheads[lane] : 0u;
                u32 incl = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const u32 x = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += x;
                }
                if (lane < WARPS) s_wheads[lane] = incl - v;
                // the block's total goes into every block's shared memory, under cover of the barrier below
                // (sending or fetching made no measurable difference, here or for the passes' digit counts)
                const u32 mine_all = __shfl_sync(0xffffffffu, incl, WARPS - 1);
                if (lane < CL) *cluster.map_shared_rank(&s_totals[c], (unsigned)lane) = mine_all;
            }
            cluster.sync();                        // every block's total has arrived (and the warps' bases are here)
            if (warp == 0) {
                const u32 v = lane < CL ? s_totals[lane] : 0u;
                u32 before = lane < (int)c ? v : 0u, all = v;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    before += __shfl_xor_sync(0xffffffffu, before, o);
                    all += __shfl_xor_sync(0xffffffffu, all, o);
                }
                if (lane == 0) { s_cbase = before; s_ctotal = all; }
            }
            __syncthreads();
            const u32 base = s_cbase, total = s_ctotal;
            u32 *segs = a.seg_start + tb0 + t;
            if (c == 0 && threadIdx.x == 0) {
                a.table_cnt[t] = total;
                segs[total] = (u32)tb1;            // the slot behind the last segment holds the table's end
            }
            const u32 ck_mask = (1u << a.ck_shift) - 1u;
            u32 before_me = base + s_wheads[warp];
            for (int i0 = w0, it = 0; i0 < w1; i0 += 32, ++it) {
                const int i = i0 + lane;
                const int64_t j = tb0 + (int64_t)c * npc + i;
                u32 m;
                if (few) {
                    m = __shfl_sync(0xffffffffu, kept, it);
                } else {
                    bool again = false;
                    if (i < w1) {
                        const u32 before = i > 0 ? fin[i - 1].x : prev_last;
                        again = (c == 0 && i == 0) || before != fin[i].x;
                    }
                    m = __ballot_sync(0xffffffffu, again);
                }
                const bool head = (m >> lane) & 1u;
                if (i < w1) {
                    const u32 upto = before_me + __popc(m & (lt | (1u << lane)));     // segment starts in [0, i]
                    if (head) segs[upto - 1] = (u32)j;
                    if (((u32)j & ck_mask) == 0u) a.chunk_first[j >> a.ck_shift] = upto - 1;
                }
                before_me += __popc(m);
            }
        }
    }
    cluster.sync();      // nobody leaves while its shared memory may still be read or written
}

inline size_t smem_bytes(int cap) { return (size_t)2 * cap * sizeof(uint2); }

// pairs per block to provision in shared memory for an expected n per table sorted by `cluster` blocks
inline int choose_cap(int64_t expect_n, int cluster)
{
    int64_t npc = ((expect_n + cluster - 1) / cluster + 31) / 32 * 32;
    int64_t cap = (npc + npc / 4 + 31) / 32 * 32;         // 25 % head room for uneven tables
    if (cap < 256) cap = 256;
    if (cap > 12288) cap = 12288;                         // 192 KB of the 227 KB a block may use
    return (int)cap;
}

}  // namespace csort
