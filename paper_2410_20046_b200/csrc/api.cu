// C ABI of the DQRM embedding-path library: context, argument checks, workspace carving
// and the order of kernel launches.  No arithmetic of the method lives here.
#include <new>
#include <string.h>
#include <stdint.h>
#include "common.cuh"

namespace {

inline cudaStream_t as_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }

inline bool ws_ok(const void *ws, size_t have, size_t need)
{
    return ws != nullptr && (reinterpret_cast<uintptr_t>(ws) % 256u) == 0 && have >= need;
}

inline bool batch_ok(const dqrm_ctx *ctx, int B, int64_t L)
{
    return ctx && B > 0 && L >= 0 && L < (int64_t)1 << 31 && (int64_t)ctx->T * B < ((int64_t)1 << 31) - 1;
}

struct HostStepLayout {
    size_t indices[2], offsets[2], grad_out[2], out[2];      // two sets of staging buffers, used by alternate calls
    size_t unique_rows, uniq_off, grad_rows, codes, grad_scales, step_ws, total;
};

HostStepLayout host_layout(const dqrm_ctx *ctx, int64_t L, int64_t G)
{
    HostStepLayout y;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const int64_t Lc = L < 1 ? 1 : L;
    for (int k = 0; k < 2; ++k) {
        y.indices[k] = take(sizeof(int32_t) * Lc);
        y.offsets[k] = take(sizeof(int32_t) * (G + 1));
        y.grad_out[k] = take(sizeof(float) * G * ctx->D);
        y.out[k] = take(sizeof(float) * G * ctx->D);
    }
    y.unique_rows = take(sizeof(int32_t) * Lc);
    y.uniq_off = take(sizeof(int32_t) * (ctx->T + 1));
    y.grad_rows = take(sizeof(float) * Lc * ctx->D);
    y.codes = take((size_t)Lc * ctx->D);
    y.grad_scales = take(sizeof(float) * ctx->T);
    y.step_ws = o;
    y.total = o + dqrm_workspace_bytes(ctx, L, G);
    return y;
}

}  // namespace

extern "C" {

int dqrm_create(dqrm_ctx **out, int T, int D, const int64_t *h_row_off)
{
    if (!out) return DQRM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!h_row_off || T <= 0 || T > 2048 || D < 4 || D > 1024 || (D % 4) != 0) return DQRM_ERR_INVALID_ARG;
    if (h_row_off[0] != 0) return DQRM_ERR_INVALID_ARG;
    for (int t = 0; t < T; ++t)
        if (h_row_off[t + 1] <= h_row_off[t]) return DQRM_ERR_INVALID_ARG;
    if (h_row_off[T] >= ((int64_t)1 << 31)) return DQRM_ERR_INVALID_ARG;

    dqrm_ctx *ctx = new (std::nothrow) dqrm_ctx();
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    ctx->T = T;
    ctx->D = D;
    ctx->total_rows = h_row_off[T];
    ctx->key_bits = 1;
    while (((int64_t)1 << ctx->key_bits) < ctx->total_rows) ctx->key_bits++;
    ctx->h_row_off = new (std::nothrow) int64_t[T + 1];
    if (!ctx->h_row_off) { delete ctx; return DQRM_ERR_INVALID_ARG; }
    memcpy(ctx->h_row_off, h_row_off, sizeof(int64_t) * (T + 1));

    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_row_off, sizeof(int64_t) * (T + 1));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_done, sizeof(u32));
    if (e == cudaSuccess) e = cudaMallocHost(&ctx->h_status_pinned, sizeof(int));
    if (e == cudaSuccess) {
        // highest priority: the sort's few blocks should be placed ahead of the forward's many
        int lo_prio = 0, hi_prio = 0;
        e = cudaDeviceGetStreamPriorityRange(&lo_prio, &hi_prio);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->side, cudaStreamNonBlocking, hi_prio);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->low, cudaStreamNonBlocking, lo_prio);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_low_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_low_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fwd, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_go, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_fwd, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_out, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_free[0], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_free[1], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h_idx, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->d_row_off, h_row_off, sizeof(int64_t) * (T + 1), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->d_done, 0, sizeof(u32));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        dqrm_destroy(ctx);
        return DQRM_ERR_CUDA;
    }
    *out = ctx;
    return DQRM_OK;
}

int dqrm_destroy(dqrm_ctx *ctx)
{
    if (!ctx) return DQRM_OK;
    if (ctx->d_row_off) cudaFree(ctx->d_row_off);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_done) cudaFree(ctx->d_done);
    if (ctx->h_status_pinned) cudaFreeHost(ctx->h_status_pinned);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    if (ctx->low) cudaStreamDestroy(ctx->low);
    if (ctx->ev_low_fork) cudaEventDestroy(ctx->ev_low_fork);
    if (ctx->ev_low_join) cudaEventDestroy(ctx->ev_low_join);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ev_fwd) cudaEventDestroy(ctx->ev_fwd);
    for (auto &kv : ctx->sorted)
        if (kv.second.done) cudaEventDestroy(kv.second.done);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    if (ctx->ev_h_start) cudaEventDestroy(ctx->ev_h_start);
    if (ctx->ev_h_go) cudaEventDestroy(ctx->ev_h_go);
    if (ctx->ev_h_fwd) cudaEventDestroy(ctx->ev_h_fwd);
    if (ctx->ev_h_out) cudaEventDestroy(ctx->ev_h_out);
    if (ctx->ev_h_free[0]) cudaEventDestroy(ctx->ev_h_free[0]);
    if (ctx->ev_h_free[1]) cudaEventDestroy(ctx->ev_h_free[1]);
    if (ctx->ev_h_idx) cudaEventDestroy(ctx->ev_h_idx);
    if (ctx->prof_events) {
        for (int i = 0; i < DQ_PROF_MAX; ++i) cudaEventDestroy(ctx->prof_events[i]);
        delete[] ctx->prof_events;
    }
    delete[] ctx->prof_ids;
    delete[] ctx->h_row_off;
    delete ctx;
    return DQRM_OK;
}

size_t dqrm_workspace_bytes(const dqrm_ctx *ctx, int64_t max_lookups, int64_t max_bags)
{
    if (!ctx || max_lookups < 0 || max_bags < 0) return 0;
    size_t a = dq_refresh_ws_bytes(ctx);
    size_t b = dq_bwd_ws_bytes(ctx, max_lookups, max_bags);
    size_t c = dq_quant_ws_bytes(ctx);
    size_t m = a > b ? a : b;
    return m > c ? m : c;
}

int dqrm_check_status(dqrm_ctx *ctx, void *stream)
{
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_status_pinned, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    DQRM_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    int s = *ctx->h_status_pinned;
    if (s != 0) {
        DQRM_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st));
        DQRM_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    }
    return s;
}

int dqrm_last_cuda_error(const dqrm_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

int64_t dqrm_launch_count(const dqrm_ctx *ctx) { return ctx ? ctx->launch_count : 0; }

int dqrm_set_overlap(dqrm_ctx *ctx, int on)
{
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    ctx->overlap = on ? 1 : 0;
    return DQRM_OK;
}

int dqrm_set_sort_path(dqrm_ctx *ctx, int path)
{
    if (!ctx || path < 0 || path > 1) return DQRM_ERR_INVALID_ARG;
    ctx->sort_path = path;
    return DQRM_OK;
}

int dqrm_profile_begin(dqrm_ctx *ctx, void *stream)
{
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    if (!ctx->prof_events) {
        ctx->prof_events = new (std::nothrow) cudaEvent_t[DQ_PROF_MAX];
        ctx->prof_ids = new (std::nothrow) int[DQ_PROF_MAX];
        if (!ctx->prof_events || !ctx->prof_ids) return DQRM_ERR_INVALID_ARG;
        for (int i = 0; i < DQ_PROF_MAX; ++i) DQRM_CUDA_TRY(ctx, cudaEventCreate(&ctx->prof_events[i]));
    }
    ctx->prof_n = 0;
    ctx->prof_on = 1;
    dq_mark(ctx, as_stream(stream), DQ_K_BEGIN);
    return DQRM_OK;
}

int dqrm_profile_end(dqrm_ctx *ctx, void *stream, float *h_ms_per_kernel, int32_t *h_launches_per_kernel, int n)
{
    if (!ctx || !h_ms_per_kernel || !h_launches_per_kernel || n < DQ_K_COUNT) return DQRM_ERR_INVALID_ARG;
    ctx->prof_on = 0;
    DQRM_CUDA_TRY(ctx, cudaStreamSynchronize(as_stream(stream)));
    for (int k = 0; k < n; ++k) { h_ms_per_kernel[k] = 0.f; h_launches_per_kernel[k] = 0; }
    for (int i = 1; i < ctx->prof_n; ++i) {
        float ms = 0.f;
        DQRM_CUDA_TRY(ctx, cudaEventElapsedTime(&ms, ctx->prof_events[i - 1], ctx->prof_events[i]));
        const int id = ctx->prof_ids[i];
        if (id == DQ_K_BEGIN) continue;          // a gap between profiled calls, not a launch
        h_ms_per_kernel[id] += ms;
        h_launches_per_kernel[id] += 1;
    }
    ctx->prof_n = 0;
    return DQRM_OK;
}

const char *dqrm_kernel_name(int kernel_id)
{
    static const char *names[DQ_K_COUNT] = {
        "begin", "refresh_kernel", "fwd_kernel", "memset", "prepare_kernel", "sort_scan_kernel",
        "sort_scatter_kernel", "seg_count_kernel", "seg_emit_kernel", "seg_reduce_kernel", "seg_fixup_kernel",
        "absmax_kernel", "row_stream_kernel<quant>", "row_stream_kernel<update>", "row_stream_kernel<fused>",
        "copy", "seg_fixup_big_kernel", "cluster_sort_kernel", "dp_pack_kernel", "dp_sum_update_kernel", "pack_kernel", "packed_fwd_kernel", "fwd_codes_kernel", "decode_payload_kernel"};
    return (kernel_id >= 0 && kernel_id < DQ_K_COUNT) ? names[kernel_id] : "?";
}

int dqrm_kernel_count(void) { return DQ_K_COUNT; }

const char *dqrm_status_string(int status)
{
    switch (status) {
    case DQRM_OK: return "ok";
    case DQRM_ERR_INVALID_ARG: return "invalid argument";
    case DQRM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DQRM_ERR_CUDA: return "CUDA runtime error";
    case DQRM_ERR_INDEX_RANGE: return "index or offset out of range (detected on the device)";
    case DQRM_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case DQRM_ERR_STATIC_LIMIT: return "size exceeds the built-in scratch of an allocation-free call";
    case DQRM_ERR_NOT_SORTED: return "workspace holds no unconsumed sorted batch of this size (call dqrm_sort_batch first)";
    default: return "unknown status";
    }
}

int dqrm_scale_refresh(dqrm_ctx *ctx, const float *tables, const int32_t *bits, float *scales, float *minmax,
                       void *workspace, size_t workspace_bytes, void *stream)
{
    if (!ctx || !tables || !bits || !scales) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_refresh_ws_bytes(ctx))) return DQRM_ERR_WORKSPACE;
    return dq_launch_refresh(ctx, tables, bits, scales, minmax, workspace, workspace_bytes, as_stream(stream));
}

int dqrm_emb_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                 const float *scales, const int32_t *bits, float *out, int8_t *codes_out, int B, int64_t L,
                 void *stream)
{
    if (!batch_ok(ctx, B, L) || !tables || !offsets || !scales || !bits || !out) return DQRM_ERR_INVALID_ARG;
    if (L > 0 && !indices) return DQRM_ERR_INVALID_ARG;
    return dq_launch_fwd(ctx, tables, indices, offsets, scales, bits, out, codes_out, B, L, as_stream(stream));
}

int dqrm_emb_bwd(dqrm_ctx *ctx, const float *grad_out, const int32_t *indices, const int32_t *offsets,
                 int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int B, int64_t L,
                 void *workspace, size_t workspace_bytes, void *stream)
{
    if (!batch_ok(ctx, B, L) || !grad_out || !offsets || !uniq_off) return DQRM_ERR_INVALID_ARG;
    if (L > 0 && (!indices || !unique_rows || !grad_rows)) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_bwd_ws_bytes(ctx, L, (int64_t)ctx->T * B))) return DQRM_ERR_WORKSPACE;
    return dq_launch_bwd(ctx, grad_out, indices, offsets, unique_rows, uniq_off, grad_rows, B, L, workspace,
                         workspace_bytes, as_stream(stream), nullptr);
}

int dqrm_grad_quant_int8(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, int8_t *codes,
                         float *grad_scales, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!ctx || !grad_rows || !uniq_off || !codes || !grad_scales) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_quant_ws_bytes(ctx))) return DQRM_ERR_WORKSPACE;
    return dq_launch_grad_quant(ctx, grad_rows, uniq_off, codes, grad_scales, workspace, workspace_bytes,
                                as_stream(stream));
}

int dqrm_row_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                    const int8_t *codes, const float *grad_scales, float lr, void *stream)
{
    if (!ctx || !tables || !unique_rows || !uniq_off || !codes || !grad_scales) return DQRM_ERR_INVALID_ARG;
    return dq_launch_row_update(ctx, tables, unique_rows, uniq_off, codes, grad_scales, lr, as_stream(stream));
}

int dqrm_train_step(dqrm_ctx *ctx, float *tables, const int32_t *indices, const int32_t *offsets,
                    const float *grad_out, const float *scales, const int32_t *bits, float *out,
                    int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int8_t *codes, float *grad_scales,
                    float lr, int B, int64_t L, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!batch_ok(ctx, B, L) || !tables || !offsets || !grad_out || !scales || !bits || !out || !uniq_off ||
        !grad_scales)
        return DQRM_ERR_INVALID_ARG;
    if (L > 0 && (!indices || !unique_rows || !grad_rows || !codes)) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_bwd_ws_bytes(ctx, L, (int64_t)ctx->T * B))) return DQRM_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    if (ctx->prof_on) dq_mark(ctx, st, DQ_K_BEGIN);
    // The backward up to the summed gradient needs the indices and the upstream gradient but neither the
    // tables nor the forward's output, so it runs on the context's second stream while the forward runs on
    // the caller's (per-launch profiling keeps one stream, because its events time consecutive launches).
    // The quantise-and-update kernel writes the rows the forward reads, so it waits for both.
    const bool overlap = ctx->overlap && !ctx->prof_on && L > 0;
    cudaStream_t ss = overlap ? ctx->side : st;
    if (overlap) {
        DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork, st));
        DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    }
    int rc = dq_launch_bwd_sort(ctx, indices, offsets, unique_rows, uniq_off, B, L, workspace, workspace_bytes, ss, nullptr, true);
    if (rc == DQRM_OK)
        rc = dq_launch_bwd_reduce(ctx, grad_out, unique_rows, uniq_off, grad_rows, B, L, workspace, workspace_bytes, ss);
    int rc2 = dq_launch_fwd(ctx, tables, indices, offsets, scales, bits, out, nullptr, B, L, st);
    if (overlap) {   // join even after an error so that the caller's stream stays ordered behind the side stream
        cudaEventRecord(ctx->ev_join, ctx->side);
        cudaStreamWaitEvent(st, ctx->ev_join, 0);
    }
    if (rc != DQRM_OK) return rc;
    if (rc2 != DQRM_OK) return rc2;
    return dq_launch_quant_update(ctx, tables, unique_rows, uniq_off, grad_rows, dq_bwd_absmax_bits(ctx, L, workspace),
                                  codes, grad_scales, lr, st);
}

int dqrm_grad_absmax(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, float *absmax, void *stream)
{
    if (!ctx || !grad_rows || !uniq_off || !absmax) return DQRM_ERR_INVALID_ARG;
    return dq_launch_grad_absmax(ctx, grad_rows, uniq_off, absmax, as_stream(stream));
}

int dqrm_grad_quant_int8_unified(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off,
                                 const float *unified_absmax, int8_t *codes, float *grad_scales, void *stream)
{
    if (!ctx || !grad_rows || !uniq_off || !unified_absmax || !codes || !grad_scales) return DQRM_ERR_INVALID_ARG;
    return dq_launch_grad_quant_unified(ctx, grad_rows, uniq_off, unified_absmax, codes, grad_scales, as_stream(stream));
}

size_t dqrm_dp_workspace_bytes(const dqrm_ctx *ctx, int64_t max_entries)
{
    if (!ctx || max_entries < 0) return 0;
    return dq_dp_ws_bytes(ctx, max_entries);
}

int dqrm_dp_merge_update(dqrm_ctx *ctx, float *tables, int W, int64_t rank_stride, const int32_t *rows_cat,
                         const int32_t *uoff_cat, const int8_t *codes_cat, const float *grad_scales, float lr,
                         int64_t n_entries, int64_t max_table_entries, int32_t *union_rows, int32_t *union_off,
                         int32_t *sums_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!ctx || !tables || W < 1 || rank_stride < 0 || !uoff_cat || !grad_scales || !union_off || n_entries < 0 ||
        n_entries > (int64_t)W * rank_stride || max_table_entries < 0 || max_table_entries > n_entries ||
        n_entries >= ((int64_t)1 << 31))
        return DQRM_ERR_INVALID_ARG;
    if (n_entries > 0 && (!rows_cat || !codes_cat || !union_rows)) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, 1)) return DQRM_ERR_WORKSPACE;
    return dq_launch_dp_merge_update(ctx, tables, W, rank_stride, rows_cat, uoff_cat, codes_cat, grad_scales, lr,
                                     n_entries, max_table_entries, union_rows, union_off, sums_out, workspace,
                                     workspace_bytes, as_stream(stream));
}

int dqrm_sort_batch(dqrm_ctx *ctx, const int32_t *indices, const int32_t *offsets, int32_t *unique_rows,
                    int32_t *uniq_off, int B, int64_t L, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!batch_ok(ctx, B, L) || !offsets || !uniq_off) return DQRM_ERR_INVALID_ARG;
    if (L > 0 && (!indices || !unique_rows)) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_bwd_ws_bytes(ctx, L, (int64_t)ctx->T * B))) return DQRM_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    if (ctx->prof_on) dq_mark(ctx, st, DQ_K_BEGIN);
    const int rc = dq_launch_bwd_sort(ctx, indices, offsets, unique_rows, uniq_off, B, L, workspace, workspace_bytes, st, nullptr, true);
    {
        std::lock_guard<std::mutex> lock(ctx->sorted_mu);
        dqrm_ctx::SortedBatch &sb = ctx->sorted[workspace];
        sb.fresh = false;
        if (rc != DQRM_OK) return rc;
        if (!sb.done) DQRM_CUDA_TRY(ctx, cudaEventCreateWithFlags(&sb.done, cudaEventDisableTiming));
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        unsigned long long id = 0;
        DQRM_CUDA_TRY(ctx, cudaStreamGetCaptureInfo(st, &cs, &id));
        DQRM_CUDA_TRY(ctx, cudaEventRecord(sb.done, st));
        sb.captured = cs == cudaStreamCaptureStatusActive;
        sb.capture_id = id;
        sb.L = L;
        sb.B = B;
        sb.fresh = true;
    }
    return rc;
}

int dqrm_train_step_sorted(dqrm_ctx *ctx, float *tables, const int32_t *indices, const int32_t *offsets,
                           const float *grad_out, const float *scales, const int32_t *bits, float *out,
                           int32_t *unique_rows, int32_t *uniq_off, float *grad_rows, int8_t *codes,
                           float *grad_scales, float lr, int B, int64_t L, void *workspace, size_t workspace_bytes,
                           void *stream)
{
    if (!batch_ok(ctx, B, L) || !tables || !offsets || !grad_out || !scales || !bits || !out || !uniq_off ||
        !grad_scales)
        return DQRM_ERR_INVALID_ARG;
    if (L > 0 && (!indices || !unique_rows || !grad_rows || !codes)) return DQRM_ERR_INVALID_ARG;
    if (!ws_ok(workspace, workspace_bytes, dq_bwd_ws_bytes(ctx, L, (int64_t)ctx->T * B))) return DQRM_ERR_WORKSPACE;
    cudaEvent_t sort_done = nullptr;
    bool sort_captured = false;
    unsigned long long sort_capture_id = 0;
    {   // the workspace must hold this batch, sorted by dqrm_sort_batch and not consumed yet: the summation
        // trusts the segment lists in it and zeroes nothing itself
        std::lock_guard<std::mutex> lock(ctx->sorted_mu);
        auto it = ctx->sorted.find(workspace);
        if (it == ctx->sorted.end() || !it->second.fresh || it->second.L != L || it->second.B != B)
            return DQRM_ERR_NOT_SORTED;
        it->second.fresh = false;
        sort_done = it->second.done;
        sort_captured = it->second.captured;
        sort_capture_id = it->second.capture_id;
    }
    cudaStream_t st = as_stream(stream);
    if (ctx->prof_on) dq_mark(ctx, st, DQ_K_BEGIN);
    // the gradient summation (second stream of the context) runs beside the forward (caller's stream)
    const bool overlap = ctx->overlap && !ctx->prof_on && L > 0;
    cudaStream_t ss = overlap ? ctx->side : st;
    if (overlap) {
        DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork, st));
        DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    }
    {   // only the summation needs the sorted order: it, not the forward, is put behind the sort's event.  An event
        // recorded inside one stream capture cannot be waited for from another capture or from outside (and the
        // other way round); there the caller's own ordering of the two calls is all there is.
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        unsigned long long id = 0;
        DQRM_CUDA_TRY(ctx, cudaStreamGetCaptureInfo(st, &cs, &id));
        const bool captured = cs == cudaStreamCaptureStatusActive;
        if (captured == sort_captured && (!captured || id == sort_capture_id))
            DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ss, sort_done, 0));
    }
    int rc = dq_launch_bwd_reduce(ctx, grad_out, unique_rows, uniq_off, grad_rows, B, L, workspace, workspace_bytes, ss);
    // The forward goes to the context's lowest-priority stream: its many blocks then do not keep the next batch's
    // sort, which a pipelined loop runs on a stream of its own, from getting SMs (with the forward on the caller's
    // high-priority stream the sort's clusters started only when the forward had handed out its last block;
    // measured per step: 62.9 -> 61.2 us Kaggle-shaped, 188.0 -> 186.8 us Terabyte-shaped)
    int rc2;
    if (overlap) {
        DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_low_fork, st));
        DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->low, ctx->ev_low_fork, 0));
        rc2 = dq_launch_fwd(ctx, tables, indices, offsets, scales, bits, out, nullptr, B, L, ctx->low);
        cudaEventRecord(ctx->ev_low_join, ctx->low);
        cudaStreamWaitEvent(st, ctx->ev_low_join, 0);
    } else {
        rc2 = dq_launch_fwd(ctx, tables, indices, offsets, scales, bits, out, nullptr, B, L, st);
    }
    cudaEventRecord(ctx->ev_fwd, st);                           // for dqrm_stream_wait_forward
    if (overlap) {
        cudaEventRecord(ctx->ev_join, ctx->side);
        cudaStreamWaitEvent(st, ctx->ev_join, 0);
    }
    if (rc != DQRM_OK) return rc;
    if (rc2 != DQRM_OK) return rc2;
    return dq_launch_quant_update(ctx, tables, unique_rows, uniq_off, grad_rows, dq_bwd_absmax_bits(ctx, L, workspace),
                                  codes, grad_scales, lr, st);
}

size_t dqrm_row_summary_bytes(const dqrm_ctx *ctx)
{
    return ctx ? (size_t)ctx->total_rows * sizeof(float2) : 0;
}

int dqrm_row_summary_attach(dqrm_ctx *ctx, const float *tables, void *summary, size_t summary_bytes, void *stream)
{
    if (!ctx || !tables || !summary || ((uintptr_t)summary & 7u)) return DQRM_ERR_INVALID_ARG;
    if (summary_bytes < dqrm_row_summary_bytes(ctx)) return DQRM_ERR_WORKSPACE;
    const int rc = dq_launch_row_summary(ctx, tables, reinterpret_cast<float2 *>(summary), as_stream(stream));
    if (rc == DQRM_OK) ctx->row_summary = reinterpret_cast<float2 *>(summary);
    return rc;
}

int dqrm_row_summary_detach(dqrm_ctx *ctx)
{
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    ctx->row_summary = nullptr;
    return DQRM_OK;
}

int dqrm_stream_wait_forward(dqrm_ctx *ctx, void *stream)
{
    if (!ctx) return DQRM_ERR_INVALID_ARG;
    DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(as_stream(stream), ctx->ev_fwd, 0));
    return DQRM_OK;
}

int dqrm_emb_fwd_codes(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                       const float *scales, int bits, uint8_t *payload, int B, int64_t L, void *stream)
{
    if (!batch_ok(ctx, B, L) || !tables || !offsets || !scales || !payload || (bits != 2 && bits != 4 && bits != 8))
        return DQRM_ERR_INVALID_ARG;
    if (L != (int64_t)ctx->T * B || (L > 0 && !indices)) return DQRM_ERR_INVALID_ARG;     // one index per bag
    return dq_launch_fwd_codes(ctx, tables, indices, offsets, scales, bits, payload, B, L, as_stream(stream));
}

int dqrm_decode_payload(dqrm_ctx *ctx, const uint8_t *payload, const float *scales, int bits, float *out, int B,
                        int T_blk, int T_total, int t0, void *stream)
{
    if (!ctx || !payload || !scales || !out || B < 0 || T_blk < 0 || t0 < 0 || t0 + T_blk > T_total ||
        (bits != 2 && bits != 4 && bits != 8))
        return DQRM_ERR_INVALID_ARG;
    return dq_launch_decode_payload(ctx, payload, scales, bits, out, B, T_blk, T_total, t0, as_stream(stream));
}

size_t dqrm_packed_bytes(const dqrm_ctx *ctx, int bits)
{
    if (!ctx || (bits != 2 && bits != 4 && bits != 8)) return 0;
    return (size_t)ctx->total_rows * (size_t)(ctx->D * bits / 8);
}

int dqrm_pack_tables(dqrm_ctx *ctx, const float *tables, const float *scales, int bits, uint8_t *packed, void *stream)
{
    if (!ctx || !tables || !scales || !packed || (bits != 2 && bits != 4 && bits != 8)) return DQRM_ERR_INVALID_ARG;
    return dq_launch_pack(ctx, tables, scales, bits, packed, as_stream(stream));
}

int dqrm_packed_fwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                    const float *scales, int bits, float *out, int B, int64_t L, void *stream)
{
    if (!batch_ok(ctx, B, L) || !packed || !offsets || !scales || !out || (bits != 2 && bits != 4 && bits != 8))
        return DQRM_ERR_INVALID_ARG;
    if (L > 0 && !indices) return DQRM_ERR_INVALID_ARG;
    return dq_launch_packed_fwd(ctx, packed, indices, offsets, scales, bits, out, B, L, as_stream(stream));
}

size_t dqrm_host_step_workspace_bytes(const dqrm_ctx *ctx, int64_t max_lookups, int64_t max_bags)
{
    if (!ctx || max_lookups < 0 || max_bags < 0) return 0;
    return host_layout(ctx, max_lookups, max_bags).total;
}

int dqrm_train_step_host(dqrm_ctx *ctx, float *tables, const int32_t *h_indices, const int32_t *h_offsets,
                         const float *h_grad_out, const float *scales, const int32_t *bits, float *h_out,
                         float lr, int B, int64_t L, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!batch_ok(ctx, B, L) || !tables || !h_offsets || !h_grad_out || !scales || !bits || !h_out)
        return DQRM_ERR_INVALID_ARG;
    if (L > 0 && !h_indices) return DQRM_ERR_INVALID_ARG;
    const int64_t G = (int64_t)ctx->T * B;
    const HostStepLayout y = host_layout(ctx, L, G);
    if (!ws_ok(workspace, workspace_bytes, y.total)) return DQRM_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(workspace);
    cudaStream_t st = as_stream(stream);
    const bool plain = !ctx->overlap || ctx->prof_on || L == 0;        // everything in order on the caller's stream
    const int set = plain ? 0 : (int)(ctx->host_calls++ & 1u);
    int32_t *d_idx = reinterpret_cast<int32_t *>(ws + y.indices[set]);
    int32_t *d_off = reinterpret_cast<int32_t *>(ws + y.offsets[set]);
    float *d_go = reinterpret_cast<float *>(ws + y.grad_out[set]);
    float *d_out = reinterpret_cast<float *>(ws + y.out[set]);
    int32_t *d_ur = reinterpret_cast<int32_t *>(ws + y.unique_rows);
    int32_t *d_uo = reinterpret_cast<int32_t *>(ws + y.uniq_off);
    float *d_gr = reinterpret_cast<float *>(ws + y.grad_rows);
    int8_t *d_codes = reinterpret_cast<int8_t *>(ws + y.codes);
    float *d_gs = reinterpret_cast<float *>(ws + y.grad_scales);
    const size_t go_bytes = sizeof(float) * G * ctx->D;
    if (plain) {
        if (L > 0) DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_idx, h_indices, sizeof(int32_t) * L, cudaMemcpyHostToDevice, st));
        DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_off, h_offsets, sizeof(int32_t) * (G + 1), cudaMemcpyHostToDevice, st));
        DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_go, h_grad_out, go_bytes, cudaMemcpyHostToDevice, st));
        int rc = dqrm_train_step(ctx, tables, d_idx, d_off, d_go, scales, bits, d_out, d_ur, d_uo, d_gr, d_codes, d_gs, lr, B,
                                 L, ws + y.step_ws, workspace_bytes - y.step_ws, stream);
        if (rc != DQRM_OK) return rc;
        DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(h_out, d_out, go_bytes, cudaMemcpyDeviceToHost, st));
        return DQRM_OK;
    }
    // The two large transfers go in opposite directions and neither is needed where the other is: the upstream
    // gradient (host to device) is first read by the gradient summation, the pooled output (device to host) is
    // complete once the forward is.  Each gets a stream of the context, so that they overlap each other, the index
    // sort and the forward.  The inputs of this call land in the staging set that the call before the last one used,
    // as soon as that call is over: they do not wait for the previous call, whose kernels and output copy they
    // overlap.  The caller's stream waits for everything before the call's work on it is complete.
    if (ctx->h_set_used[set]) DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy_in, ctx->ev_h_free[set], 0));
    else {      // first use of this set: only what the caller's stream already holds comes first
        DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_h_start, st));
        DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy_in, ctx->ev_h_start, 0));
    }
    DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_idx, h_indices, sizeof(int32_t) * L, cudaMemcpyHostToDevice, ctx->copy_in));
    DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_off, h_offsets, sizeof(int32_t) * (G + 1), cudaMemcpyHostToDevice, ctx->copy_in));
    DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_h_idx, ctx->copy_in));
    DQRM_CUDA_TRY(ctx, cudaMemcpyAsync(d_go, h_grad_out, go_bytes, cudaMemcpyHostToDevice, ctx->copy_in));
    DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_h_go, ctx->copy_in));
    DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->ev_h_idx, 0));
    DQRM_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork, st));
    DQRM_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    char *step_ws = ws + y.step_ws;
    const size_t step_ws_bytes = workspace_bytes - y.step_ws;
    int rc = dq_launch_bwd_sort(ctx, d_idx, d_off, d_ur, d_uo, B, L, step_ws, step_ws_bytes, ctx->side, nullptr, true);
    if (rc == DQRM_OK) rc = dq_launch_fwd(ctx, tables, d_idx, d_off, scales, bits, d_out, nullptr, B, L, st);
    // join every stream even after an error, so that the caller's stream stays ordered behind them
    cudaEventRecord(ctx->ev_h_fwd, st);
    cudaStreamWaitEvent(ctx->copy_out, ctx->ev_h_fwd, 0);
    if (rc == DQRM_OK) cudaMemcpyAsync(h_out, d_out, go_bytes, cudaMemcpyDeviceToHost, ctx->copy_out);
    cudaEventRecord(ctx->ev_h_out, ctx->copy_out);
    // the gradient summation follows the sort on the second stream as soon as the upstream gradient has arrived
    cudaStreamWaitEvent(ctx->side, ctx->ev_h_go, 0);
    if (rc == DQRM_OK) rc = dq_launch_bwd_reduce(ctx, d_go, d_ur, d_uo, d_gr, B, L, step_ws, step_ws_bytes, ctx->side);
    cudaEventRecord(ctx->ev_join, ctx->side);
    cudaStreamWaitEvent(st, ctx->ev_join, 0);
    if (rc == DQRM_OK)
        rc = dq_launch_quant_update(ctx, tables, d_ur, d_uo, d_gr, dq_bwd_absmax_bits(ctx, L, step_ws), d_codes, d_gs, lr, st);
    cudaStreamWaitEvent(st, ctx->ev_h_out, 0);
    cudaEventRecord(ctx->ev_h_free[set], st);        // the staging set is free for the call after the next one
    ctx->h_set_used[set] = true;
    if (rc != DQRM_OK) return rc;
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    return DQRM_OK;
}

}  // extern "C"
