// Device self-check of the quantiser shortcut: over a range of FP32 bit patterns it
// compares the division-free code (dq_codef) with the plain definition
// clamp(rint(x / s)) computed with the IEEE division, and counts disagreements.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(256)
selfcheck_kernel(float s, int bits, u32 first_bits, unsigned long long count, unsigned long long *mismatches)
{
    const QuantScale q = dq_make_scale(s, bits);
    unsigned long long bad = 0;
    // four consecutive bit patterns per call, as the kernels quantise (one 128-bit vector)
    for (unsigned long long i = 4ull * ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x); i < count;
         i += 4ull * gridDim.x * blockDim.x) {
        float x[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) x[k] = __uint_as_float(first_bits + (u32)(i + k));
        float4 codes, deq;
        dq_fq4(make_float4(x[0], x[1], x[2], x[3]), q, codes, deq);
        const float got[4] = {codes.x, codes.y, codes.z, codes.w};
        const float dgot[4] = {deq.x, deq.y, deq.z, deq.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (i + k >= count || !(x[k] == x[k])) continue;      // NaN inputs are outside the contract
            const int want = dq_code(x[k], s, q.lo, q.hi);
            // bit patterns are compared, so that a -0.0 in place of +0.0 counts as a difference
            if (__float_as_uint(got[k]) != __float_as_uint((float)want) ||
                __float_as_uint(dgot[k]) != __float_as_uint(dq_dequant(want, s)))
                ++bad;
        }
    }
    if (bad) atomicAdd(mismatches, bad);
}

}  // namespace

extern "C" int dqrm_selfcheck_quantizer(dqrm_ctx *ctx, float scale, int bits, uint32_t first_bits, uint64_t count,
                                        uint64_t *mismatches, void *stream)
{
    if (!ctx || !mismatches || bits < 2 || bits > 16 || !(scale > 0.f) || count > ((uint64_t)1 << 32))
        return DQRM_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    selfcheck_kernel<<<ctx->num_sms * 8, 256, 0, st>>>(scale, bits, first_bits, (unsigned long long)count,
                                                        reinterpret_cast<unsigned long long *>(mismatches));
    DQRM_CUDA_TRY(ctx, cudaGetLastError());
    return DQRM_OK;
}
