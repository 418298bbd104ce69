// Internal declarations shared by the CUDA translation units of the DQRM library.
#pragma once
#include <mutex>
#include <unordered_map>
#include <utility>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "dqrm.h"

typedef uint32_t u32;

struct dqrm_ctx {
    int T = 0, D = 0;
    int64_t total_rows = 0;
    int64_t *h_row_off = nullptr;   // [T+1] host copy
    int64_t *d_row_off = nullptr;   // [T+1]
    int *d_status = nullptr;        // device status word (first error wins)
    u32 *d_done = nullptr;          // "blocks finished" counter of the refresh kernel (self-resetting)
    int *h_status_pinned = nullptr; // pinned landing slot for dqrm_check_status
    int last_cuda_error = 0;
    int device = 0;
    int num_sms = 0;
    int key_bits = 1;               // bits of an arena row number
    int sort_path = 0;              // 0: per-table cluster sort, 1: global radix sort
    cudaStream_t side = nullptr;    // second stream: a training step sorts the indices and sums the gradient beside its forward
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t low = nullptr;     // lowest priority: the forward of a step whose next batch is being sorted elsewhere
    cudaEvent_t ev_low_fork = nullptr, ev_low_join = nullptr;
    cudaEvent_t ev_fwd = nullptr;   // recorded behind the forward of the last training step enqueued
    // host-buffer step: the upstream gradient comes in and the pooled output goes out on streams of their own
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_h_start = nullptr, ev_h_go = nullptr, ev_h_fwd = nullptr, ev_h_out = nullptr;
    // ... with two sets of staging buffers used alternately: a set is free again when the call that used it is over
    cudaEvent_t ev_h_free[2] = {nullptr, nullptr}, ev_h_idx = nullptr;
    bool h_set_used[2] = {false, false};
    unsigned host_calls = 0;
    float2 *row_summary = nullptr;  // [total_rows] (min, max) of every row, caller's memory; null: not kept
    // what the context knows, on the host, about each workspace dqrm_sort_batch has written: whether it holds a
    // sorted batch that no step has taken yet, of which size, and the event recorded behind that sort (with the
    // stream capture it was recorded in, if any)
    struct SortedBatch {
        bool fresh = false;
        int64_t L = 0;
        int B = 0;
        cudaEvent_t done = nullptr;
        bool captured = false;
        unsigned long long capture_id = 0;
    };
    std::mutex sorted_mu;
    std::unordered_map<const void *, SortedBatch> sorted;
    int overlap = 1;                // 0: keep everything on the caller's stream
    int payload_position = 0;       // sort payload: 0 = row of grad_out, 1 = position of the lookup (set by the merge)
    // kernels whose dynamic shared-memory limit has been raised on this context's device (the attribute is
    // per device, so the record lives here and not in a process-wide flag)
    bool smem_raised[32] = {};
    // launch accounting and optional per-launch timing (see dqrm_profile_*)
    int64_t launch_count = 0;
    int prof_on = 0, prof_n = 0;
    cudaEvent_t *prof_events = nullptr;   // [DQ_PROF_MAX]
    int *prof_ids = nullptr;              // [DQ_PROF_MAX] kernel id that ENDS at event i
};

enum {
    DQ_K_BEGIN = 0, DQ_K_REFRESH, DQ_K_FWD, DQ_K_MEMSET, DQ_K_PREPARE, DQ_K_SORT_SCAN, DQ_K_SORT_SCATTER,
    DQ_K_SEG_COUNT, DQ_K_SEG_EMIT, DQ_K_SEG_REDUCE, DQ_K_SEG_FIXUP, DQ_K_ABSMAX, DQ_K_QUANT, DQ_K_UPDATE,
    DQ_K_QUANT_UPDATE, DQ_K_COPY, DQ_K_SEG_FIXUP_BIG, DQ_K_CLUSTER_SORT, DQ_K_DP_PACK, DQ_K_DP_SUM_UPDATE, DQ_K_PACK, DQ_K_PACKED_FWD, DQ_K_FWD_CODES, DQ_K_DECODE_PAYLOAD, DQ_K_COUNT
};
constexpr int DQ_PROF_MAX = 4096;

// called right after every launch: counts it and, when profiling is on, drops an event
static inline void dq_mark(dqrm_ctx *ctx, cudaStream_t st, int kernel_id)
{
    if (kernel_id != DQ_K_BEGIN && kernel_id != DQ_K_MEMSET && kernel_id != DQ_K_COPY) ctx->launch_count++;
    if (ctx->prof_on && ctx->prof_n < DQ_PROF_MAX) {
        ctx->prof_ids[ctx->prof_n] = kernel_id;
        cudaEventRecord(ctx->prof_events[ctx->prof_n], st);
        ctx->prof_n++;
    }
}

#define DQRM_CUDA_TRY(ctx, call)                                   \
    do {                                                           \
        cudaError_t e_ = (call);                                   \
        if (e_ != cudaSuccess) {                                   \
            (ctx)->last_cuda_error = (int)e_;                      \
            (void)cudaGetLastError();                              \
            return DQRM_ERR_CUDA;                                  \
        }                                                          \
    } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// slots of dqrm_ctx::smem_raised
constexpr int DQ_SMEM_SLOT_CSORT = 24;
constexpr int dq_log2c(int x) { return x <= 1 ? 0 : 1 + dq_log2c(x / 2); }
constexpr int dq_smem_slot_fixup(int lpr, int ch) { return dq_log2c(lpr) * 4 + dq_log2c(ch); }

// ---------------------------------------------------------------------------------
// quantiser arithmetic: each operation is one IEEE round-to-nearest FP32 operation
// ---------------------------------------------------------------------------------
__device__ __forceinline__ float dq_scale_from_absmax(float absmax, int bits)
{
    float a = fmaxf(absmax, 1e-8f);
    return __fdiv_rn(a, (float)((1 << (bits - 1)) - 1));
}

// code = clamp(round_half_even(x / s), lo, hi); lo/hi are the integer bounds as floats
__device__ __forceinline__ int dq_code(float x, float s, float lo, float hi)
{
    float r = rintf(__fdiv_rn(x, s));
    r = fminf(fmaxf(r, lo), hi);
    return (int)r;
}

__device__ __forceinline__ float dq_dequant(int q, float s) { return __fmul_rn((float)q, s); }

// ---------------------------------------------------------------------------------
// The same codes without the IEEE-division sequence, for a scale shared by many elements,
// four elements at a time.
//
//   QuantScale holds s and r = RN(1/s).  q0 = RN(x * r) equals x/s up to a relative error
//   below 2^-22 (one rounding of r, one of the product), and RN(x/s) is within 2^-24 of
//   x/s.  Only half-integers of magnitude below 2^(b-1) decide a b-bit code (beyond them the
//   clamp gives the same code either way), and there |q0 - RN(x/s)| < 2^(b-23).  So if q0 is
//   farther than TOL = 2^(b-21) from every half-integer, rounding q0 gives the same code as
//   rounding RN(x/s).  Vectors with an element inside that window (about one in 10^4 for
//   4-bit codes) are redone with the IEEE division.  Rounding to an integer is done by
//   adding and subtracting 1.5*2^23 (round-to-nearest-even, no conversion instruction);
//   the result is the code as a float, which is also what the dequantiser multiplies.
//   The multiplies and adds use the packed two-float instructions of sm_100.
//   Bit widths above 10 and scales outside [2^-100, 2^100] always take the IEEE path.
// ---------------------------------------------------------------------------------
struct QuantScale {
    float s, r, lo, hi, tie_lim;
    bool fast;
};

__device__ __forceinline__ QuantScale dq_make_scale(float s, int bits)
{
    QuantScale q;
    q.s = s;
    q.r = __frcp_rn(s);
    q.lo = -(float)(1 << (bits - 1));
    q.hi = (float)((1 << (bits - 1)) - 1);
    q.tie_lim = 0.5f - (float)(1 << (bits - 1)) * 9.5367431640625e-07f;     // 0.5 - 2^(b-21)
    q.fast = (bits <= 10) && (s >= 7.8886090522101181e-31f) && (s <= 1.2676506002282294e+30f);
    return q;
}

// one code as a float by the plain definition
__device__ __forceinline__ float dq_codef_ieee(float x, const QuantScale &q)
{
    // "+ 0" turns the -0.0 that rintf gives for small negative quotients into the +0.0 an integer code has
    return __fadd_rn(fminf(fmaxf(rintf(__fdiv_rn(x, q.s)), q.lo), q.hi), 0.0f);
}

// codes (as floats, integer values in [lo, hi]) and dequantised values of four elements
__device__ __forceinline__ void dq_fq4(const float4 &v, const QuantScale &q, float4 &codes, float4 &deq)
{
    const float MAGIC = 12582912.0f;                   // 1.5 * 2^23
    bool done = false;
    if (q.fast) {
        const float2 r2 = make_float2(q.r, q.r), m2 = make_float2(MAGIC, MAGIC), nm2 = make_float2(-MAGIC, -MAGIC);
        const float2 neg1 = make_float2(-1.f, -1.f);
        const float2 qa = __fmul2_rn(make_float2(v.x, v.y), r2), qb = __fmul2_rn(make_float2(v.z, v.w), r2);
        const float2 ra = __fadd2_rn(__fadd2_rn(qa, m2), nm2), rb = __fadd2_rn(__fadd2_rn(qb, m2), nm2);
        const float2 da = __ffma2_rn(ra, neg1, qa), db = __ffma2_rn(rb, neg1, qb);     // q0 - rint(q0)
        const float m = fmaxf(fmaxf(fabsf(da.x), fabsf(da.y)), fmaxf(fabsf(db.x), fabsf(db.y)));
        if (m < q.tie_lim) {
            codes = make_float4(fminf(fmaxf(ra.x, q.lo), q.hi), fminf(fmaxf(ra.y, q.lo), q.hi),
                                fminf(fmaxf(rb.x, q.lo), q.hi), fminf(fmaxf(rb.y, q.lo), q.hi));
            done = true;
        }
    }
    if (!done)
        codes = make_float4(dq_codef_ieee(v.x, q), dq_codef_ieee(v.y, q), dq_codef_ieee(v.z, q), dq_codef_ieee(v.w, q));
    const float2 s2 = make_float2(q.s, q.s);
    const float2 ea = __fmul2_rn(make_float2(codes.x, codes.y), s2), eb = __fmul2_rn(make_float2(codes.z, codes.w), s2);
    deq = make_float4(ea.x, ea.y, eb.x, eb.y);
}


// 16-byte asynchronous copy global -> shared (data never passes through registers)
__device__ __forceinline__ void dq_cp_async16(void *smem_dst, const void *gmem_src)
{
    unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void dq_cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void dq_cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// asks L2 for the 128-byte line that holds p (no register, no scoreboard entry: the later load finds it there)
__device__ __forceinline__ void dq_prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p)); }

// L2 eviction priorities.  Data that a later kernel of the same step reads again (the summed gradient rows, the
// touched master rows) is marked to be evicted last; what is touched once is streamed (__ldcs / __stcs).
__device__ __forceinline__ uint64_t dq_policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float4 dq_ld_nc_keep(const float4 *p, uint64_t pol)
{
    float4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;\n"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ void dq_st_keep(float4 *p, const float4 &v, uint64_t pol)
{
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;\n"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(pol) : "memory");
}

__device__ __forceinline__ void dq_report(int *status, int code)
{
    atomicCAS(status, 0, code);   // first error wins
}

// table that owns arena row `key`: largest t with row_off[t] <= key
__device__ __forceinline__ int dq_table_of(const int64_t *row_off, int T, int64_t key)
{
    int lo = 0, hi = T;           // invariant: row_off[lo] <= key < row_off[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (row_off[mid] <= key) lo = mid; else hi = mid;
    }
    return lo;
}

// ---------------------------------------------------------------------------------
// host launchers (one per translation unit)
// ---------------------------------------------------------------------------------
// (min, max) of a row's new values, folded over the LPR lanes that hold the row (all of them call this together;
// lane groups are aligned to LPR within the warp).  In the first exchange the even lane of a pair takes over the
// pair's min and the odd lane its max, so that from then on every lane folds one value with one shuffle per
// level; the group's first lane ends up with the row's min, the second with its max, and each stores its own.
template <int LPR>
__device__ __forceinline__ void dq_store_row_minmax(float2 *__restrict__ row_summary, int64_t arena_row, float mn, float mx)
{
    if (LPR == 1) {
        row_summary[arena_row] = make_float2(mn, mx);
        return;
    }
    const unsigned lane_w = threadIdx.x & 31;
    const unsigned mask = LPR == 32 ? 0xffffffffu : (((1u << LPR) - 1u) << (lane_w / LPR * LPR));
    const bool odd = lane_w & 1u;
    const float other = __shfl_xor_sync(mask, odd ? mn : mx, 1);
    float v = odd ? fmaxf(mx, other) : fminf(mn, other);
#pragma unroll
    for (int o = 2; o < LPR; o <<= 1) {
        const float r = __shfl_xor_sync(mask, v, o);
        v = odd ? fmaxf(v, r) : fminf(v, r);
    }
    if (lane_w % LPR < 2) reinterpret_cast<float *>(row_summary + arena_row)[odd ? 1 : 0] = v;
}

size_t dq_refresh_ws_bytes(const dqrm_ctx *ctx);
int dq_launch_refresh(dqrm_ctx *ctx, const float *tables, const int32_t *bits, float *scales,
                      float *minmax, void *ws, size_t ws_bytes, cudaStream_t st);

int dq_launch_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                  const float *scales, const int32_t *bits, float *out, int8_t *codes_out,
                  int B, int64_t L, cudaStream_t st);

size_t dq_bwd_ws_bytes(const dqrm_ctx *ctx, int64_t L, int64_t G);
// per-table |grad| maxima (float bit patterns) inside a workspace that dq_launch_bwd_sort and
// dq_launch_bwd_reduce have filled
const u32 *dq_bwd_absmax_bits(const dqrm_ctx *ctx, int64_t L, const void *ws);
// absmax_bits_out: device pointer (inside ws) to per-table |grad| maxima as float bit patterns
int dq_launch_bwd(dqrm_ctx *ctx, const float *grad_out, const int32_t *indices, const int32_t *offsets,
                  int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int B, int64_t L,
                  void *ws, size_t ws_bytes, cudaStream_t st, const u32 **absmax_bits_out);

// lists_by_table: dq_launch_bwd_reduce follows on the same workspace; the cluster sort then numbers each table's
// segments itself, no separate kernel numbers them over the batch, and unique_rows / uniq_off are written by
// dq_launch_bwd_reduce.  Without it they are complete when the sort is.
int dq_launch_bwd_sort(dqrm_ctx *ctx, const int32_t *indices, const int32_t *offsets, int32_t *unique_rows,
                       int32_t *uniq_off, int B, int64_t L, void *ws, size_t ws_bytes, cudaStream_t st,
                       const u32 **absmax_bits_out, bool lists_by_table = false);
int dq_launch_bwd_reduce(dqrm_ctx *ctx, const float *grad_out, int32_t *unique_rows, int32_t *uniq_off,
                         float *grad_rows, int B, int64_t L, void *ws, size_t ws_bytes, cudaStream_t st);

size_t dq_quant_ws_bytes(const dqrm_ctx *ctx);
int dq_launch_grad_absmax(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, float *absmax,
                          cudaStream_t st);
int dq_launch_grad_quant_unified(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off,
                                 const float *unified_absmax, int8_t *codes, float *grad_scales, cudaStream_t st);
int dq_launch_pack(dqrm_ctx *ctx, const float *tables, const float *scales, int bits, uint8_t *packed, cudaStream_t st);
int dq_launch_packed_fwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                         const float *scales, int bits, float *out, int B, int64_t L, cudaStream_t st);
int dq_launch_fwd_codes(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                        const float *scales, int bits, uint8_t *payload, int B, int64_t L, cudaStream_t st);
int dq_launch_decode_payload(dqrm_ctx *ctx, const uint8_t *payload, const float *scales, int bits, float *out, int B,
                             int T_blk, int T_total, int t0, cudaStream_t st);
size_t dq_dp_ws_bytes(const dqrm_ctx *ctx, int64_t max_entries);
int dq_launch_dp_merge_update(dqrm_ctx *ctx, float *tables, int W, int64_t rank_stride, const int32_t *rows_cat,
                              const int32_t *uoff_cat, const int8_t *codes_cat, const float *grad_scales, float lr,
                              int64_t n_entries, int64_t max_table_entries, int32_t *union_rows, int32_t *union_off,
                              int32_t *sums_out, void *ws, size_t ws_bytes, cudaStream_t st);
int dq_launch_grad_quant(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, int8_t *codes,
                         float *grad_scales, void *ws, size_t ws_bytes, cudaStream_t st);
int dq_launch_row_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                         const int8_t *codes, const float *grad_scales, float lr, cudaStream_t st);
int dq_launch_row_summary(dqrm_ctx *ctx, const float *tables, float2 *summary, cudaStream_t st);
int dq_launch_quant_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                           const float *grad_rows, const u32 *absmax_bits, int8_t *codes,
                           float *grad_scales, float lr, cudaStream_t st);
