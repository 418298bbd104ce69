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
};

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
