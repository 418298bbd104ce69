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
#include "row_stream.cuh"

namespace {

using namespace rowstream;

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

template <int MODE, int LPR, int CH, bool EXACT, bool TRACK = false>
__global__ void __launch_bounds__(QU_THREADS)
row_stream_kernel(float *__restrict__ tables, const int64_t *__restrict__ row_off,
                  const int32_t *__restrict__ unique_rows, const int32_t *__restrict__ uniq_off,
                  const float *__restrict__ grad_rows, const u32 *__restrict__ absmax,
                  int8_t *__restrict__ codes, float *__restrict__ grad_scales, float lr, int T, int D_any,
                  int *__restrict__ status, float2 *__restrict__ row_summary)
{
    extern __shared__ unsigned char smem_raw[];
    row_stream_body<MODE, LPR, CH, EXACT, TRACK>(smem_raw, tables, row_off, unique_rows, uniq_off, grad_rows, absmax,
                                                 codes, grad_scales, lr, T, D_any, status, row_summary);
}

template <int MODE, int LPR, int CH>
int launch_rows(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows, const int32_t *uniq_off,
                const float *grad_rows, const u32 *absmax, int8_t *codes, float *grad_scales, float lr,
                cudaStream_t st)
{
    const size_t smem = (size_t)(ctx->T + 1) * sizeof(int32_t) + (size_t)ctx->T * sizeof(float);
    int grid = ctx->num_sms * 8;      // U lives on the device: a fixed grid splits the rows evenly
    // with a row summary attached, every kernel that writes master rows keeps the rows' (min, max) current
    float2 *summary = MODE == MODE_QUANT ? nullptr : ctx->row_summary;
#define DQ_ROW_STREAM(EXACT, TRACK)                                                                               \
    row_stream_kernel<MODE, LPR, CH, EXACT, TRACK><<<grid, QU_THREADS, smem, st>>>(                                \
        tables, ctx->d_row_off, unique_rows, uniq_off, grad_rows, absmax, codes, grad_scales, lr, ctx->T, ctx->D, \
        ctx->d_status, summary)
    if (ctx->D == 4 * LPR * CH) {
        if (summary) DQ_ROW_STREAM(true, (MODE != MODE_QUANT));
        else DQ_ROW_STREAM(true, false);
    } else {
        if (summary) DQ_ROW_STREAM(false, (MODE != MODE_QUANT));
        else DQ_ROW_STREAM(false, false);
    }
#undef DQ_ROW_STREAM
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
