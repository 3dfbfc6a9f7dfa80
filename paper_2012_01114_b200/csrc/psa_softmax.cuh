// Register-level pieces of phase 2 (paper Eq. 2) shared by the attention kernels of the bf16 path:
// exp2 evaluation, the 32-score chunk routines (row maximum, exponentials packed to bf16) and the
// constants of the lazily rescaled online softmax.
#pragma once
#include "sm100.cuh"

namespace psa {

constexpr int CTRL_WARPS = 2;                       // producer, MMA issuer
constexpr int TPR = 2;                              // softmax threads per query row (each owns 64 of a block's 128 columns)
constexpr int SOFTMAX_WARPS_PER_TILE = 4 * TPR;
constexpr int ATTN_THREADS = 32 * (CTRL_WARPS + 2 * SOFTMAX_WARPS_PER_TILE);   // 576
constexpr float LOG2E = 1.4426950408889634f;
constexpr float RESCALE_THRESHOLD = 8.0f;  // log2 units: O and l are rescaled only when the row max grew by more

__device__ __forceinline__ float ex2_mufu(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// exp2 of 32 scores of one row (raw, unscaled) against the running maximum: P = exp2(s*sl2 - m), packed
// to bf16 pairs in `pk`; returns the sum of the 32 weights (before rounding).  `col0` is the column of
// s[0] inside the 128-wide block; with DIAG, columns beyond `r` carry no weight.
template <bool DIAG>
__device__ __forceinline__ float exp_chunk32(const uint32_t (&s)[32], float sl2, float neg_m, int col0, int r,
                                             uint32_t (&pk)[16]) {
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const float x0 = fmaf(__uint_as_float(s[i]), sl2, neg_m);
        const float x1 = fmaf(__uint_as_float(s[i + 1]), sl2, neg_m);
        float p0 = ex2_mufu(x0);
        float p1 = ex2_mufu(x1);
        if (DIAG) {
            if (col0 + i > r) p0 = 0.f;
            if (col0 + i + 1 > r) p1 = 0.f;
        }
        sum0 += p0;
        sum1 += p1;
        pk[i >> 1] = pack_bf16x2(p0, p1);
    }
    return sum0 + sum1;
}

template <bool DIAG>
__device__ __forceinline__ float max_chunk32(const uint32_t (&s)[32], int col0, int r, float mx) {
    // four independent accumulators: the chain of dependent maxima is 4 long, not 16 (the three-input maximum has a
    // latency of about a dozen cycles); with DIAG, columns beyond `r` are replaced by -inf first
    float a[4] = {mx, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float x0 = __uint_as_float(s[i + 2 * k]), x1 = __uint_as_float(s[i + 2 * k + 1]);
            if (DIAG) {
                if (col0 + i + 2 * k > r) x0 = -INFINITY;
                if (col0 + i + 2 * k + 1 > r) x1 = -INFINITY;
            }
            a[k] = max3(a[k], x0, x1);
        }
    }
    return fmaxf(max3(a[0], a[1], a[2]), a[3]);
}

}  // namespace psa
