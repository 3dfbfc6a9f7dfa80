// Measured rates of the SM pipes that bound phase 2 (paper Eq. 2) beside the tensor pipe: the special-function
// unit (one ex2 per weight), the fp32 FMA pipe, and the instruction mix the softmax spends per weight (scale-and-
// shift FMA, ex2, running-sum add, half a bf16x2 pack).  Rates are results per SM clock per SM, taken from
// clock64 inside the kernel, so they do not depend on the clock frequency of the moment; the benchmark turns them
// into a ceiling with the SM clock it samples during its timed region.
#include "psa_internal.h"
#include "sm100.cuh"

namespace psa {

namespace {

constexpr int PIPE_THREADS = 512;     // 16 warps per SM: 4 per scheduler, as many as a row tile's softmax warps x 2
constexpr int PIPE_ILP = 8;           // independent instructions in flight per thread
constexpr int PIPE_ITERS = 2048;

__device__ __forceinline__ float ex2_raw(float v) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v));
    return y;
}

// MODE 0: ex2.approx.ftz   MODE 1: fma.rn.f32   MODE 2: the softmax mix.
// Every result feeds the next iteration (8 independent chains per thread), so that nothing is loop-invariant or dead
// for the assembler to remove; the values stay bounded: x <- -0.5 * 2^x maps [-1, 0] into [-0.5, -0.25].
template <int MODE>
__global__ void __launch_bounds__(PIPE_THREADS, 1) pipe_rate_kernel(unsigned long long* cycles, float* sink, float seed) {
    float x[PIPE_ILP];
#pragma unroll
    for (int k = 0; k < PIPE_ILP; ++k) x[k] = seed - 0.03125f * k - 0.0001f * threadIdx.x;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t packed = 0;
    __syncthreads();
    const long long t0 = clock64();
#pragma unroll 4
    for (int it = 0; it < PIPE_ITERS; ++it) {
        if (MODE == 0) {
#pragma unroll
            for (int k = 0; k < PIPE_ILP; ++k) x[k] = -0.5f * ex2_raw(x[k]);          // one MUFU op + one multiply
        } else if (MODE == 1) {
#pragma unroll
            for (int k = 0; k < PIPE_ILP; ++k) x[k] = fmaf(x[k], 0.5f, seed);         // converges to 2 * seed
        } else {
#pragma unroll
            for (int k = 0; k < PIPE_ILP; k += 2) {
                // per weight: scale-and-shift, exponential, row-sum add; per pair of weights one bf16x2 pack
                const float p0 = ex2_raw(fmaf(x[k], seed, -0.25f));
                const float p1 = ex2_raw(fmaf(x[k + 1], seed, -0.25f));
                sum0 += p0;
                sum1 += p1;
                uint32_t pk;
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(p1), "f"(p0));
                packed ^= pk;
                x[k] = p0;
                x[k + 1] = p1;
            }
        }
    }
    const long long t1 = clock64();
    float acc = sum0 + sum1 + __uint_as_float(packed & 0x3f800000u);
#pragma unroll
    for (int k = 0; k < PIPE_ILP; ++k) acc += x[k];
    if (acc == 123.456f) *sink = acc;                      // keeps the results alive; never true in practice
    if ((threadIdx.x & 31) == 0) atomicMax(&cycles[blockIdx.x], (unsigned long long)(t1 - t0));
}

}  // namespace

// cycles: device array of `sms` counters per mode (3 * sms), zeroed by the caller.
cudaError_t launch_pipe_rates(unsigned long long* cycles, float* sink, int sms, cudaStream_t stream) {
    pipe_rate_kernel<0><<<sms, PIPE_THREADS, 0, stream>>>(cycles, sink, -0.5f);
    pipe_rate_kernel<1><<<sms, PIPE_THREADS, 0, stream>>>(cycles + sms, sink, -0.5f);
    pipe_rate_kernel<2><<<sms, PIPE_THREADS, 0, stream>>>(cycles + 2 * sms, sink, -0.5f);
    return cudaGetLastError();
}
double pipe_results_per_launch_per_sm() { return (double)PIPE_THREADS * PIPE_ILP * PIPE_ITERS; }

}  // namespace psa
