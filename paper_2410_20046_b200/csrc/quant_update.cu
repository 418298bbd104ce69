// INT8 gradient quantiser and touched-row SGD update (paper Appendix B.1): the values of
// the sparse embedding gradient are quantised to INT8 with one scale per table, fixed
// by the bit width and the tensor's own abs-max, and the local step is taken with the
// dequantised gradient on the FP32 master rows (Section 3.1).
//
// Three variants of one row-streaming kernel share the addressing: quantise only,
// update only (from stored codes), and quantise + update fused (the training step).
// A group of LPR lanes owns a contiguous range of unique rows and keeps a few of them in flight;
// rows are distinct, so the read-modify-write of the master rows needs no atomics.  All
// streams are 128-bit per lane.
#include <mutex>
#include "common.cuh"

namespace {

constexpr int QU_THREADS = 256;
enum { MODE_QUANT = 0, MODE_UPDATE = 1, MODE_FUSED = 2 };

// largest t with uoff[t] <= u, skipping empty tables
__device__ __forceinline__ int table_of_row(const int32_t *uoff, int T, int64_t u)
{
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (uoff[mid] <= u) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(QU_THREADS)
absmax_kernel(const float *__restrict__ grad_rows, const int32_t *__restrict__ uniq_off, int T, int D,
              u32 *__restrict__ absmax)
{
    extern __shared__ unsigned char smem_raw[];
    int32_t *s_uoff = reinterpret_cast<int32_t *>(smem_raw);      // [T+1]
    u32 *s_max = reinterpret_cast<u32 *>(s_uoff + (T + 1));       // [T]
    for (int t = threadIdx.x; t <= T; t += QU_THREADS) s_uoff[t] = uniq_off[t];
    for (int t = threadIdx.x; t < T; t += QU_THREADS) s_max[t] = 0u;
    __syncthreads();
    const int d4 = D >> 2;
    const int64_t n4 = (int64_t)s_uoff[T] * d4;
    const float4 *g4 = reinterpret_cast<const float4 *>(grad_rows);
    int cur_t = -1;
    int64_t cur_end4 = -1;
    float m = 0.f;
    for (int64_t base = (int64_t)blockIdx.x * QU_THREADS; base < n4; base += (int64_t)gridDim.x * QU_THREADS) {
        int64_t i = base + threadIdx.x;
        bool ok = i < n4;
        float v = 0.f;
        int t = cur_t;
        if (ok) {
            float4 x = __ldg(g4 + i);
            v = fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w)));
            if (i >= cur_end4) {
                t = table_of_row(s_uoff, T, i / d4);
                cur_end4 = (int64_t)s_uoff[t + 1] * d4;
            }
        }
        if (t != cur_t) {
            if (cur_t >= 0 && m > 0.f) atomicMax(&s_max[cur_t], __float_as_uint(m));
            cur_t = t;
            m = 0.f;
        }
        m = fmaxf(m, v);
    }
    if (cur_t >= 0 && m > 0.f) atomicMax(&s_max[cur_t], __float_as_uint(m));
    __syncthreads();
    for (int t = threadIdx.x; t < T; t += QU_THREADS)
        if (s_max[t]) atomicMax(&absmax[t], s_max[t]);
}

// rows in flight per lane group: fewer when a lane already holds several vectors of every row
template <int CH> struct RowsInFlight { static constexpr int v = CH >= 4 ? 1 : (CH == 2 ? 2 : 4); };

// EXACT: the feature size is 4*LPR*CH, a compile-time constant, and the per-vector range checks fall away
template <int MODE, int LPR, int CH, bool EXACT>
__global__ void __launch_bounds__(QU_THREADS)
row_stream_kernel(float *__restrict__ tables, const int64_t *__restrict__ row_off,
                  const int32_t *__restrict__ unique_rows, const int32_t *__restrict__ uniq_off,
                  const float *__restrict__ grad_rows, const u32 *__restrict__ absmax,
                  int8_t *__restrict__ codes, float *__restrict__ grad_scales, float lr, int T, int D_any,
                  int *__restrict__ status)
{
    constexpr int NB = RowsInFlight<CH>::v;
    const int D = EXACT ? 4 * LPR * CH : D_any;
    extern __shared__ unsigned char smem_raw[];
    int32_t *s_uoff = reinterpret_cast<int32_t *>(smem_raw);      // [T+1]
    float *s_scale = reinterpret_cast<float *>(s_uoff + (T + 1)); // [T] gradient scale of every table
    for (int t = threadIdx.x; t <= T; t += QU_THREADS) s_uoff[t] = uniq_off[t];
    for (int t = threadIdx.x; t < T; t += QU_THREADS) {
        const float sc = (MODE == MODE_UPDATE) ? grad_scales[t] : dq_scale_from_absmax(__uint_as_float(absmax[t]), 8);
        s_scale[t] = sc;
        if (MODE != MODE_UPDATE && blockIdx.x == 0) grad_scales[t] = sc;
    }
    __syncthreads();
    const int d4 = D >> 2;
    const int64_t U = s_uoff[T];
    const int lane = threadIdx.x % LPR;
    const int64_t group = ((int64_t)blockIdx.x * QU_THREADS + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t)gridDim.x * QU_THREADS / LPR;
    // a lane group owns a contiguous range of unique rows: its rows mostly share a table, and its reads
    // of the gradient rows and writes of the codes are sequential
    int64_t per = (U + n_groups - 1) / n_groups;
    if (per < NB) per = NB;             // few rows: fewer groups, each with a full set of rows in flight
    const int64_t u_begin = group * per, u_end = min(U, u_begin + per);
    int cur_t = -1;
    int64_t cur_end = -1, r0 = 0, nrows = 1;
    bool bad = false;
    float s = 1.f;
    QuantScale qs = dq_make_scale(1.f, 8);
    for (int64_t u = u_begin; u < u_end;) {
        if (u >= cur_end) {
            cur_t = table_of_row(s_uoff, T, u);
            cur_end = s_uoff[cur_t + 1];
            if (MODE != MODE_QUANT) { r0 = __ldg(row_off + cur_t); nrows = __ldg(row_off + cur_t + 1) - r0; }
            s = s_scale[cur_t];
            qs = dq_make_scale(s, 8);
        }
        // up to NB rows of the current table at once
        const int nb = (int)min((int64_t)NB, min(u_end, cur_end) - u);
        float4 *wrow[NB];
        float4 g[NB][CH], w[NB][CH];
        char4 cin[NB][CH];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            wrow[b] = nullptr;
            if (b < nb && MODE != MODE_QUANT) {
                // a row number outside its table is reported and kept inside the arena, never followed
                int64_t row = __ldg(unique_rows + u + b);
                if (row < 0 || row >= nrows) { bad = true; row = row < 0 ? 0 : nrows - 1; }
                wrow[b] = reinterpret_cast<float4 *>(tables + (r0 + row) * D);
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < nb) {
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int c4 = ch * LPR + lane;
                    if (EXACT || c4 < d4) {
                        if (MODE == MODE_UPDATE) cin[b][ch] = *reinterpret_cast<const char4 *>(codes + (u + b) * D + 4 * c4);
                        else g[b][ch] = __ldg(reinterpret_cast<const float4 *>(grad_rows + (u + b) * D) + c4);
                        if (MODE != MODE_QUANT) w[b][ch] = wrow[b][c4];
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b < nb) {
#pragma unroll
                for (int ch = 0; ch < CH; ++ch) {
                    const int c4 = ch * LPR + lane;
                    if (EXACT || c4 < d4) {
                        float4 q;                      // integer codes held as floats
                        if (MODE == MODE_UPDATE) {
                            q = make_float4((float)cin[b][ch].x, (float)cin[b][ch].y, (float)cin[b][ch].z, (float)cin[b][ch].w);
                        } else {
                            float4 dq_unused;
                            dq_fq4(g[b][ch], qs, q, dq_unused);
                            *reinterpret_cast<char4 *>(codes + (u + b) * D + 4 * c4) =
                                make_char4((signed char)(int)q.x, (signed char)(int)q.y, (signed char)(int)q.z,
                                           (signed char)(int)q.w);
                        }
                        if (MODE != MODE_QUANT) {
                            float4 x = w[b][ch];
                            x.x = __fsub_rn(x.x, __fmul_rn(lr, __fmul_rn(q.x, s)));
                            x.y = __fsub_rn(x.y, __fmul_rn(lr, __fmul_rn(q.y, s)));
                            x.z = __fsub_rn(x.z, __fmul_rn(lr, __fmul_rn(q.z, s)));
                            x.w = __fsub_rn(x.w, __fmul_rn(lr, __fmul_rn(q.w, s)));
                            wrow[b][c4] = x;
                        }
                    }
                }
            }
        }
        u += nb;
    }
    if (MODE != MODE_QUANT && bad) dq_report(status, DQRM_ERR_INDEX_RANGE);
}

template <int MODE, int LPR, int CH>
int launch_rows(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                const float *grad_rows, const u32 *absmax, int8_t *codes, float *grad_scales, float lr,
                cudaStream_t st)
{
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int32_t) + (size_t)ctx->T * sizeof(float);
    int grid = ctx->num_sms * 8;      // U lives on the device: a fixed grid splits the rows evenly
    if (ctx->D == 4 * LPR * CH)
        row_stream_kernel<MODE, LPR, CH, true><<<grid, QU_THREADS, smem, st>>>(
            tables, ctx->d_row_off, unique_rows, uniq_off, grad_rows, absmax, codes, grad_scales, lr, ctx->T, ctx->D,
            ctx->d_status);
    else
        row_stream_kernel<MODE, LPR, CH, false><<<grid, QU_THREADS, smem, st>>>(
            tables, ctx->d_row_off, unique_rows, uniq_off, grad_rows, absmax, codes, grad_scales, lr, ctx->T, ctx->D,
            ctx->d_status);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, MODE == MODE_QUANT ? DQ_K_QUANT : (MODE == MODE_UPDATE ? DQ_K_UPDATE : DQ_K_QUANT_UPDATE));
    return DQRM_OK;
}

template <int MODE>
int dispatch(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
             const float *grad_rows, const u32 *absmax, int8_t *codes, float *grad_scales, float lr,
             cudaStream_t st)
{
    const int d4 = ctx->D / 4;
#define DQ_ROWS(LPR, CH) \
    return launch_rows<MODE, LPR, CH>(ctx, tables, unique_rows, uniq_off, grad_rows, absmax, codes, grad_scales, lr, st)
    if (d4 <= 1) DQ_ROWS(1, 1);
    if (d4 <= 2) DQ_ROWS(2, 1);
    if (d4 <= 4) DQ_ROWS(4, 1);
    if (d4 <= 8) DQ_ROWS(8, 1);
    if (d4 <= 16) DQ_ROWS(16, 1);
    if (d4 <= 32) DQ_ROWS(32, 1);
    if (d4 <= 64) DQ_ROWS(32, 2);
    if (d4 <= 128) DQ_ROWS(32, 4);
    DQ_ROWS(32, 8);
#undef DQ_ROWS
}

}  // namespace

size_t dq_quant_ws_bytes(const dqrm_ctx *ctx) { return align_up(sizeof(u32) * ctx->T, 256); }

int dq_launch_grad_quant(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, int8_t *codes,
                         float *grad_scales, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (ws_bytes < dq_quant_ws_bytes(ctx)) return DQRM_ERR_WORKSPACE;
    u32 *absmax = reinterpret_cast<u32 *>(ws);
    DQRM_CUDA_TRY(ctx, cudaMemsetAsync(absmax, 0, sizeof(u32) * ctx->T, st));
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int32_t) + (size_t)ctx->T * sizeof(u32);
    dq_mark(ctx, st, DQ_K_MEMSET);
    absmax_kernel<<<ctx->num_sms * 8, QU_THREADS, smem, st>>>(grad_rows, uniq_off, ctx->T, ctx->D, absmax);
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_ABSMAX);
    return dispatch<MODE_QUANT>(ctx, nullptr, nullptr, uniq_off, grad_rows, absmax, codes, grad_scales, 0.f, st);
}

// per-table max |grad_rows| as floats (the bit pattern of a non-negative float orders like the uint the kernel maximises)
int dq_launch_grad_absmax(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, float *absmax,
                          cudaStream_t st)
{
    DQRM_CUDA_TRY(ctx, cudaMemsetAsync(absmax, 0, sizeof(float) * ctx->T, st));
    dq_mark(ctx, st, DQ_K_MEMSET);
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int32_t) + (size_t)ctx->T * sizeof(u32);
    absmax_kernel<<<ctx->num_sms * 8, QU_THREADS, smem, st>>>(grad_rows, uniq_off, ctx->T, ctx->D,
                                                              reinterpret_cast<u32 *>(absmax));
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    dq_mark(ctx, st, DQ_K_ABSMAX);
    return DQRM_OK;
}

// quantise with scales derived from abs-max values that were unified across ranks
int dq_launch_grad_quant_unified(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off,
                                 const float *unified_absmax, int8_t *codes, float *grad_scales, cudaStream_t st)
{
    return dispatch<MODE_QUANT>(ctx, nullptr, nullptr, uniq_off, grad_rows, reinterpret_cast<const u32 *>(unified_absmax),
                                codes, grad_scales, 0.f, st);
}

int dq_launch_row_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                         const int8_t *codes, const float *grad_scales, float lr, cudaStream_t st)
{
    return dispatch<MODE_UPDATE>(ctx, tables, unique_rows, uniq_off, nullptr, nullptr, const_cast<int8_t *>(codes),
                                 const_cast<float *>(grad_scales), lr, st);
}

int dq_launch_quant_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                           const float *grad_rows, const u32 *absmax_bits, int8_t *codes, float *grad_scales,
                           float lr, cudaStream_t st)
{
    return dispatch<MODE_FUSED>(ctx, tables, unique_rows, uniq_off, grad_rows, absmax_bits, codes, grad_scales, lr, st);
}

// ---------------------------------------------------------------------------------
// Allocation-free variant of the INT8 gradient quantiser.
//
// Some users of this library may not allocate device memory at the point where they
// quantise gradients: a plug-in that runs inside another framework's step after that
// framework has reserved the whole HBM for its own pool (a cudaMalloc there fails or
// fragments the pool), or a latency-critical loop in which the implicit device-wide
// synchronisation of cudaMalloc/cudaFree would stall every other stream.  Such callers
// have no way to provide the per-table abs-max scratch word that dqrm_grad_quant_int8
// takes from its workspace, and they cannot create a context either (dqrm_create
// allocates).  For them the scratch lives in the array below, which is part of the
// loaded module: every GPU that loads the library holds these 4 KB until the process
// exits.  The name `g_static_absmax` is only a handle in host code; the device address
// is looked up once per device with cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------------
static __device__ __align__(256) u32 g_static_absmax[DQRM_STATIC_MAX_TABLES];

namespace {

constexpr int STATIC_MAX_DEVICES = 64;
struct StaticSlot {
    u32 *absmax = nullptr;   // device address of g_static_absmax on this device
    int num_sms = 0;
    bool ready = false;
};
StaticSlot g_static_slots[STATIC_MAX_DEVICES];
std::mutex g_static_mutex;        // host threads may make a device's first call at the same time

}  // namespace

extern "C" int dqrm_grad_quant_int8_static(int T, int D, const float *grad_rows, const int32_t *uniq_off,
                                           int8_t *codes, float *grad_scales, void *stream)
{
    if (T <= 0 || D < 4 || D > 1024 || (D % 4) != 0 || !grad_rows || !uniq_off || !codes || !grad_scales)
        return DQRM_ERR_INVALID_ARG;
    if (T > DQRM_STATIC_MAX_TABLES) return DQRM_ERR_STATIC_LIMIT;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
        (void)cudaGetLastError();
        return DQRM_ERR_CUDA;
    }
    StaticSlot slot;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        StaticSlot &shared = g_static_slots[dev];
        if (!shared.ready) {
            // first call on this device: resolve the array's device address (with this device current)
            u32 *p = nullptr;
            if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_absmax) != cudaSuccess || !p ||
                cudaDeviceGetAttribute(&shared.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
                (void)cudaGetLastError();
                return DQRM_ERR_CUDA;
            }
            shared.absmax = p;
            shared.ready = true;
        }
        slot = shared;
    }
    // a stack context carries the shape to the shared launch helpers; nothing is allocated
    dqrm_ctx tmp;
    tmp.T = T;
    tmp.D = D;
    tmp.device = dev;
    tmp.num_sms = slot.num_sms;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps the previous call's maxima: clear the entries this call uses
    if (cudaMemsetAsync(slot.absmax, 0, sizeof(u32) * T, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQRM_ERR_CUDA;
    }
    const size_t smem = (size_t)(T + 1) * sizeof(int32_t) + (size_t)T * sizeof(u32);
    absmax_kernel<<<tmp.num_sms * 8, QU_THREADS, smem, st>>>(grad_rows, uniq_off, T, D, slot.absmax);
    if (cudaGetLastError() != cudaSuccess) return DQRM_ERR_CUDA;
    return dispatch<MODE_QUANT>(&tmp, nullptr, nullptr, uniq_off, grad_rows, slot.absmax, codes, grad_scales, 0.f, st);
}
