// fp32 storage, fp32 arithmetic path on CUDA cores with element-exact skipping: a weight that the
// scheme does not need is never computed (paper Sec. 4.1, 5.1), so issued MACs equal the paper's
// element counts (Sec. 3.2, 4.2, 5.2).  Meant for small problems and as the full-precision path;
// the throughput path is the bf16 tensor-core one.
#include "psa_internal.h"

namespace psa {

namespace {

constexpr int PROJ_TILE = 16;

// out[w][r, c] = sum_k X[r, k] W[w][k, c]      (paper Sec. 3.1: the projections are plain products)
__global__ void __launch_bounds__(PROJ_TILE* PROJ_TILE)
f32_project_kernel(const float* __restrict__ X, const float* W0, const float* W1, const float* W2, float* O0,
                   float* O1, float* O2, int rows, int D, int N, const float* __restrict__ R, DeviceCounters* dc) {
    __shared__ float xs[PROJ_TILE][PROJ_TILE + 1];
    __shared__ float ws[PROJ_TILE][PROJ_TILE + 1];
    const float* W = blockIdx.z == 0 ? W0 : (blockIdx.z == 1 ? W1 : W2);
    float* O = blockIdx.z == 0 ? O0 : (blockIdx.z == 1 ? O1 : O2);
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int r = blockIdx.y * PROJ_TILE + ty, c = blockIdx.x * PROJ_TILE + tx;
    float acc = 0.f;
    for (int k0 = 0; k0 < D; k0 += PROJ_TILE) {
        xs[ty][tx] = (r < rows && k0 + tx < D) ? X[(size_t)r * D + k0 + tx] : 0.f;
        ws[ty][tx] = (k0 + ty < D && c < N) ? W[(size_t)(k0 + ty) * N + c] : 0.f;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < PROJ_TILE; ++k) acc = fmaf(xs[ty][k], ws[k][tx], acc);
        __syncthreads();
    }
    if (r < rows && c < N) O[(size_t)r * N + c] = R ? acc + R[(size_t)r * N + c] : acc;
    if (tx == 0 && ty == 0) {
        const int vr = min(PROJ_TILE, rows - blockIdx.y * PROJ_TILE), vc = min(PROJ_TILE, N - blockIdx.x * PROJ_TILE);
        atomicAdd(&dc->proj_macs, (unsigned long long)vr * vc * D);
    }
}

constexpr int ROWS_PER_BLOCK = 4;  // one warp per query row
constexpr int KEY_TILE = 32;

// MODE 0: all three phases for FULL / MASKED.
// MODE 1: phase 1 of the symmetric scheme: S_ij for j <= i, stored at (i,j) and at its mirror (j,i)
//         (the reuse of paper Sec. 4.1: the mirror costs a store, no MACs).
// MODE 2: phases 2 and 3 reading the weights' pre-softmax values from S.
template <int MODE>
__global__ void __launch_bounds__(ROWS_PER_BLOCK * 32)
f32_attn_kernel(const float* __restrict__ Q, const float* __restrict__ K, const float* __restrict__ V,
                float* __restrict__ out, float* __restrict__ S, int n, int H, int d, float scale, int masked,
                DeviceCounters* dc) {
    extern __shared__ float sm[];
    float* ks = sm;                                   // [KEY_TILE][d + 1]
    float* qs = ks + KEY_TILE * (d + 1);              // [ROWS_PER_BLOCK][d]
    float* sc = qs + ROWS_PER_BLOCK * d;              // [ROWS_PER_BLOCK][n]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.z, h = blockIdx.y;
    const int i = blockIdx.x * ROWS_PER_BLOCK + warp;
    const bool live = i < n;
    const size_t ld = (size_t)H * d;                                  // row pitch of Q, K, V, out
    const size_t base = ((size_t)b * n) * ld + (size_t)h * d;
    const bool lower = (MODE == 1) || masked;                          // only j <= i is needed
    const int jend = live ? (lower ? i + 1 : n) : 0;                   // this warp's keys: [0, jend)
    const int last_row = min(n - 1, (int)blockIdx.x * ROWS_PER_BLOCK + ROWS_PER_BLOCK - 1);
    const int jend_block = lower ? last_row + 1 : n;
    float* myS = S ? S + ((size_t)(b * H + h) * n) * n : nullptr;
    float* mysc = sc + warp * n;
    unsigned long long dots = 0;

    if (MODE != 2) {
        if (live)
            for (int c = lane; c < d; c += 32) qs[warp * d + c] = Q[base + (size_t)i * ld + c];
        for (int j0 = 0; j0 < jend_block; j0 += KEY_TILE) {
            __syncthreads();
            for (int t = threadIdx.x; t < KEY_TILE * d; t += blockDim.x) {
                const int jj = t / d, c = t - jj * d;
                ks[jj * (d + 1) + c] = (j0 + jj < n) ? K[base + (size_t)(j0 + jj) * ld + c] : 0.f;
            }
            __syncthreads();
            const int j = j0 + lane;
            if (j < jend) {                                            // phase 1, Eq. 1: one weight per lane
                float acc = 0.f;
                const float* kr = ks + lane * (d + 1);
                const float* qr = qs + warp * d;
                for (int c = 0; c < d; ++c) acc = fmaf(qr[c], kr[c], acc);
                acc *= scale;
                ++dots;
                if (MODE == 1) {
                    myS[(size_t)i * n + j] = acc;
                    myS[(size_t)j * n + i] = acc;
                } else {
                    mysc[j] = acc;
                }
            }
        }
    } else {
        for (int j = lane; j < jend; j += 32) mysc[j] = myS[(size_t)i * n + j];
    }
    for (int off = 16; off; off >>= 1) dots += __shfl_xor_sync(0xffffffffu, dots, off);
    if (MODE != 2 && lane == 0 && dots) atomicAdd(&dc->qk_macs, dots * (unsigned long long)d);
    if (MODE == 1 || !live) return;
    __syncwarp();

    // phase 2, Eq. 2: exponent-accumulate over the kept weights, then normalisation
    float mx = -INFINITY;
    for (int j = lane; j < jend; j += 32) mx = fmaxf(mx, mysc[j]);
    for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    float sum = 0.f;
    for (int j = lane; j < jend; j += 32) {
        const float e = expf(mysc[j] - mx);
        mysc[j] = e;
        sum += e;
    }
    for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    __syncwarp();
    const float inv = 1.f / sum;

    // phase 3, Eq. 3: lanes own output components, keys are walked in order
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j = 0; j < jend; ++j) {
        const float w = mysc[j];
        const float* vr = V + base + (size_t)j * ld;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int c = lane + 32 * t;
            if (c < d) acc[t] = fmaf(w, vr[c], acc[t]);
        }
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int c = lane + 32 * t;
        if (c < d) out[base + (size_t)i * ld + c] = acc[t] * inv;
    }
    if (lane == 0) {
        atomicAdd(&dc->pv_macs, (unsigned long long)jend * d);
        atomicAdd(&dc->exps, (unsigned long long)jend);
    }
}

size_t attn_smem_bytes(int n, int d) {
    return sizeof(float) * ((size_t)KEY_TILE * (d + 1) + (size_t)ROWS_PER_BLOCK * d + (size_t)ROWS_PER_BLOCK * n);
}

}  // namespace

cudaError_t f32_project(const float* X, const float* const W[3], float* const out[3], int nW, int rows, int D,
                        int N, const float* residual, DeviceCounters* dc, cudaStream_t stream) {
    dim3 block(PROJ_TILE, PROJ_TILE), grid((N + PROJ_TILE - 1) / PROJ_TILE, (rows + PROJ_TILE - 1) / PROJ_TILE, nW);
    f32_project_kernel<<<grid, block, 0, stream>>>(X, W[0], W[1], W[2], out[0], out[1], out[2], rows, D, N, residual, dc);
    return cudaGetLastError();
}

cudaError_t f32_attention(const float* Q, const float* K, const float* V, float* out, float* S, int B, int H,
                          int n, int d, float scale, int scheme, DeviceCounters* dc, cudaStream_t stream) {
    dim3 grid((n + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK, H, B), block(ROWS_PER_BLOCK * 32);
    const size_t smem = attn_smem_bytes(n, d);
    if (scheme == PSA_SYMMETRIC) {
        f32_attn_kernel<1><<<grid, block, smem, stream>>>(Q, Q, Q, out, S, n, H, d, scale, 0, dc);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        f32_attn_kernel<2><<<grid, block, smem, stream>>>(Q, Q, Q, out, S, n, H, d, scale, 0, dc);
    } else {
        f32_attn_kernel<0><<<grid, block, smem, stream>>>(Q, K, V, out, nullptr, n, H, d, scale,
                                                          scheme == PSA_MASKED ? 1 : 0, dc);
    }
    return cudaGetLastError();
}

}  // namespace psa
