// Internal declarations shared by the CUDA translation units of the DQRM library.
#pragma once
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
    // launch accounting and optional per-launch timing (see dqrm_profile_*)
    int64_t launch_count = 0;
    int prof_on = 0, prof_n = 0;
    cudaEvent_t *prof_events = nullptr;   // [DQ_PROF_MAX]
    int *prof_ids = nullptr;              // [DQ_PROF_MAX] kernel id that ENDS at event i
};

enum {
    DQ_K_BEGIN = 0, DQ_K_REFRESH, DQ_K_FWD, DQ_K_MEMSET, DQ_K_PREPARE, DQ_K_SORT_SCAN, DQ_K_SORT_SCATTER,
    DQ_K_SEG_COUNT, DQ_K_SEG_EMIT, DQ_K_SEG_REDUCE, DQ_K_SEG_FIXUP, DQ_K_ABSMAX, DQ_K_QUANT, DQ_K_UPDATE,
    DQ_K_QUANT_UPDATE, DQ_K_COPY, DQ_K_COUNT
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
size_t dq_refresh_ws_bytes(const dqrm_ctx *ctx);
int dq_launch_refresh(dqrm_ctx *ctx, const float *tables, const int32_t *bits, float *scales,
                      float *minmax, void *ws, size_t ws_bytes, cudaStream_t st);

int dq_launch_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                  const float *scales, const int32_t *bits, float *out, int8_t *codes_out,
                  int B, int64_t L, cudaStream_t st);

size_t dq_bwd_ws_bytes(const dqrm_ctx *ctx, int64_t L, int64_t G);
// absmax_bits_out: device pointer (inside ws) to per-table |grad| maxima as float bit patterns
int dq_launch_bwd(dqrm_ctx *ctx, const float *grad_out, const int32_t *indices, const int32_t *offsets,
                  int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int B, int64_t L,
                  void *ws, size_t ws_bytes, cudaStream_t st, const u32 **absmax_bits_out);

size_t dq_quant_ws_bytes(const dqrm_ctx *ctx);
int dq_launch_grad_quant(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, int8_t *codes,
                         float *grad_scales, void *ws, size_t ws_bytes, cudaStream_t st);
int dq_launch_row_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                         const int8_t *codes, const float *grad_scales, float lr, cudaStream_t st);
int dq_launch_quant_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                           const float *grad_rows, const u32 *absmax_bits, int8_t *codes,
                           float *grad_scales, float lr, cudaStream_t st);
