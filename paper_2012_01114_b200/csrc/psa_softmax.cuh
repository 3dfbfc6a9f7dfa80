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

// Softmax over a block of S held in the quad layout (sm100.cuh): s[0..31] are 16 scores of row A (s[4g], s[4g+1])
// and 16 of row B = A + 8 (s[4g+2], s[4g+3]), columns col0 + 8g + 2(lane%4) + {0, 1}.
//
// Columns beyond cbA / cbB (the rows' last kept columns on a diagonal or ragged block) carry no weight: they are set
// to -inf once, which the maximum ignores and the exponential turns into 0, so that such blocks share all other code.
__device__ __forceinline__ void mask_quad64(uint32_t (&s)[32], int col0q, int cbA, int cbB) {
    const uint32_t ninf = 0xff800000u;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const int c = col0q + 8 * g;
        if (c > cbA) s[4 * g] = ninf;
        if (c + 1 > cbA) s[4 * g + 1] = ninf;
        if (c > cbB) s[4 * g + 2] = ninf;
        if (c + 1 > cbB) s[4 * g + 3] = ninf;
    }
}
__device__ __forceinline__ void max_quad64(const uint32_t (&s)[32], float& mA, float& mB) {
    float a0 = mA, a1 = -INFINITY, b0 = mB, b1 = -INFINITY;
#pragma unroll
    for (int g = 0; g < 8; g += 2) {
        a0 = max3(a0, __uint_as_float(s[4 * g]), __uint_as_float(s[4 * g + 1]));
        b0 = max3(b0, __uint_as_float(s[4 * g + 2]), __uint_as_float(s[4 * g + 3]));
        a1 = max3(a1, __uint_as_float(s[4 * g + 4]), __uint_as_float(s[4 * g + 5]));
        b1 = max3(b1, __uint_as_float(s[4 * g + 6]), __uint_as_float(s[4 * g + 7]));
    }
    mA = fmaxf(a0, a1);
    mB = fmaxf(b0, b1);
}
// P = exp2(s*sl2 - m) for the 32 scores, packed to bf16 pairs in the layout tmem_st_quad32 expects (pk[2g] row A,
// pk[2g+1] row B); the rows' sums of weights (before rounding) are added to sumA / sumB.
__device__ __forceinline__ void exp_quad64(const uint32_t (&s)[32], float sl2, float negmA, float negmB, uint32_t (&pk)[16],
                                           float& sumA, float& sumB) {
    float sa0 = 0.f, sa1 = 0.f, sb0 = 0.f, sb1 = 0.f;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const float p0 = ex2_mufu(fmaf(__uint_as_float(s[4 * g]), sl2, negmA));
        const float p1 = ex2_mufu(fmaf(__uint_as_float(s[4 * g + 1]), sl2, negmA));
        const float p2 = ex2_mufu(fmaf(__uint_as_float(s[4 * g + 2]), sl2, negmB));
        const float p3 = ex2_mufu(fmaf(__uint_as_float(s[4 * g + 3]), sl2, negmB));
        sa0 += p0; sa1 += p1; sb0 += p2; sb1 += p3;
        pk[2 * g] = pack_bf16x2(p0, p1);
        pk[2 * g + 1] = pack_bf16x2(p2, p3);
    }
    sumA += sa0 + sa1;
    sumB += sb0 + sb1;
}
// Sum (or maximum) over the four threads of a quad, which hold the same two rows.
__device__ __forceinline__ float quad_max(float v) {
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

}  // namespace psa
