// fp32 storage, fp32 arithmetic path on CUDA cores with element-exact skipping: a weight that the
// scheme does not need is never computed (paper Sec. 4.1, 5.1), so issued MACs equal the paper's
// element counts (Sec. 3.2, 4.2, 5.2).  Meant for small problems and as the full-precision path;
// the throughput path is the bf16 tensor-core one.
#include <cooperative_groups.h>

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

// ---------------------------------------------------------------- one launch for small layers
// Projections and the three phases of one (batch, head) in one CTA, everything in shared memory: the layer of a few
// dozen vectors is a few microseconds of work, and two launches with a round trip of q, k, v through global memory
// cost more than the arithmetic.  Element-exact skipping as in the kernels above: a weight the scheme does not need
// is never computed, and the census counts the multiply-accumulates actually executed.
constexpr int FS_THREADS = 512;
constexpr int FS_MAX_FLOATS = 56 * 1024;          // shared-memory budget in floats (224 KB)

struct FusedLayout {
    int xs_ld, t_ld, ds, s_ld;                    // row pitches: X, transposed q and k, v, the weight matrix S
    size_t xs, ws, qt, kt, vs, sm, rinv, total;   // offsets in floats
};
// q and k are kept transposed ([component][vector]) so that phase 1 reads four consecutive vectors of one component
// as one 16-byte access; v is kept [vector][component] for phase 3.
__host__ __device__ inline FusedLayout fused_layout(int n, int D, int d, int nW) {
    FusedLayout L;
    L.xs_ld = D + 1; L.t_ld = ((n + 3) & ~3) + 4; L.ds = d + 4; L.s_ld = n + 1;
    size_t off = 0;
    L.xs = off; off += (size_t)n * L.xs_ld; off = (off + 3) & ~size_t(3);
    L.ws = off; off += (size_t)nW * D * d;
    L.qt = off; off += (size_t)d * L.t_ld;
    L.kt = nW == 3 ? off : L.qt; if (nW == 3) off += (size_t)d * L.t_ld;
    L.vs = off; off += (size_t)n * L.ds;
    L.sm = off; off += (size_t)n * L.s_ld;
    L.rinv = off; off += n;
    L.total = off;
    return L;
}

__global__ void __launch_bounds__(FS_THREADS, 1)
f32_fused_layer_kernel(const float* __restrict__ X, const float* __restrict__ Wq, const float* __restrict__ Wk,
                       const float* __restrict__ Wv, float* __restrict__ out, int n, int H, int D, int d, float scale,
                       int scheme, DeviceCounters* dc, DeviceCounters* dc_next) {
    extern __shared__ float4 fs_smem4[];
    float* sm = reinterpret_cast<float*>(fs_smem4);
    // the counter block of the NEXT call on this workspace is cleared here, off that call's critical path
    if (blockIdx.x == 0 && threadIdx.x == 0 && dc_next) *dc_next = DeviceCounters{0, 0, 0, 0, 0, 0, 0};
    const int nW = scheme == PSA_SYMMETRIC ? 1 : 3;
    const FusedLayout L = fused_layout(n, D, d, nW);
    float* xs = sm + L.xs; float* ws = sm + L.ws; float* qt = sm + L.qt; float* kt = sm + L.kt; float* vs = sm + L.vs;
    float* S = sm + L.sm; float* rinv = sm + L.rinv;
    const int b = blockIdx.x / H, h = blockIdx.x - b * H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool lower = scheme != PSA_FULL;            // only j <= i is computed in phase 1 (masked; symmetric: then mirrored)
    const bool masked = scheme == PSA_MASKED;
    const size_t HD = (size_t)H * d;
    unsigned long long qk = 0, pv = 0, ex = 0;

    // ---- stage X[b] and this head's columns of the projection matrices (loads batched eight deep: a layer this small
    // lives on the latency of its first loads)
    {
        const float* xb = X + (size_t)b * n * D;
        for (int t0 = tid; t0 < n * D; t0 += 8 * FS_THREADS) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) { const int t = t0 + u * FS_THREADS; v[u] = t < n * D ? __ldg(xb + t) : 0.f; }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int t = t0 + u * FS_THREADS;
                if (t < n * D) { const int i = t / D; xs[i * L.xs_ld + (t - i * D)] = v[u]; }
            }
        }
        const int d4 = d / 4;
        for (int w = 0; w < nW; ++w) {
            const float* W = (w == 0 ? Wq : (w == 1 ? Wk : Wv)) + (size_t)h * d;
            float4* dst = reinterpret_cast<float4*>(ws + (size_t)w * D * d);
            for (int t0 = tid; t0 < D * d4; t0 += 4 * FS_THREADS) {
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int t = t0 + u * FS_THREADS;
                    if (t < D * d4) { const int k = t / d4; v[u] = __ldg(reinterpret_cast<const float4*>(W + (size_t)k * HD) + (t - k * d4)); }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) { const int t = t0 + u * FS_THREADS; if (t < D * d4) dst[t] = v[u]; }
            }
        }
    }
    __syncthreads();

    // ---- projections (Sec. 3.1): 4 x 4 register tiles of q, k, v
    const int tr = (n + 3) / 4, tc = d / 4;
    for (int t = tid; t < nW * tr * tc; t += FS_THREADS) {
        const int w = t / (tr * tc), rem = t - w * tr * tc;
        const int i0 = (rem / tc) * 4, c0 = (rem % tc) * 4;
        const float* wp = ws + (size_t)w * D * d + c0;
        float acc[4][4] = {};
        int row[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) row[r] = min(i0 + r, n - 1) * L.xs_ld;
        for (int k = 0; k < D; ++k) {
            const float4 wv = *reinterpret_cast<const float4*>(wp + (size_t)k * d);
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float x = xs[row[r] + k];
                acc[r][0] = fmaf(x, wv.x, acc[r][0]); acc[r][1] = fmaf(x, wv.y, acc[r][1]);
                acc[r][2] = fmaf(x, wv.z, acc[r][2]); acc[r][3] = fmaf(x, wv.w, acc[r][3]);
            }
        }
        if (w < 2) {          // q, k: transposed (rows beyond n land in the pitch's padding and are never used)
            float* dst = w == 0 ? qt : kt;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                *reinterpret_cast<float4*>(dst + (size_t)(c0 + u) * L.t_ld + i0) = make_float4(acc[0][u], acc[1][u], acc[2][u], acc[3][u]);
        }
        if (w == 2 || nW == 1) {   // v (the symmetric scheme's single projection is q, k and v at once)
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (i0 + r < n) *reinterpret_cast<float4*>(vs + (size_t)(i0 + r) * L.ds + c0) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
        }
    }
    __syncthreads();

    // ---- phase 1 (Eq. 1): S_ij = scale q_i . k_j for the weights the scheme needs, in 4 x 4 register tiles
    const int tn = (n + 3) / 4;
    for (int t = tid; t < tn * tn; t += FS_THREADS) {
        const int i0 = (t / tn) * 4, j0 = (t % tn) * 4;
        if (lower && j0 > i0 + 3) continue;                       // wholly above the diagonal: never issued
        const bool inside = i0 + 3 < n && j0 + 3 < n;
        if (inside && !(lower && j0 == i0)) {
            // a whole tile: 16 weights
            float acc[4][4] = {};
            for (int c = 0; c < d; ++c) {
                const float4 q4 = *reinterpret_cast<const float4*>(qt + (size_t)c * L.t_ld + i0);
                const float4 k4 = *reinterpret_cast<const float4*>(kt + (size_t)c * L.t_ld + j0);
                const float qv[4] = {q4.x, q4.y, q4.z, q4.w}, kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int u = 0; u < 4; ++u) acc[r][u] = fmaf(qv[r], kv[u], acc[r][u]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float v = acc[r][u] * scale;
                    S[(size_t)(i0 + r) * L.s_ld + j0 + u] = v;
                    if (scheme == PSA_SYMMETRIC) S[(size_t)(j0 + u) * L.s_ld + i0 + r] = v;   // reuse (Sec. 4.1): a store, no MACs
                }
            qk += 16ull * d;
        } else if (inside) {
            // the tile on the diagonal of a lower-triangle scheme: the 10 weights with j <= i, nothing above them
            float acc[4][4] = {};
            for (int c = 0; c < d; ++c) {
                const float4 q4 = *reinterpret_cast<const float4*>(qt + (size_t)c * L.t_ld + i0);
                const float4 k4 = *reinterpret_cast<const float4*>(kt + (size_t)c * L.t_ld + j0);
                const float qv[4] = {q4.x, q4.y, q4.z, q4.w}, kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int u = 0; u <= r; ++u) acc[r][u] = fmaf(qv[r], kv[u], acc[r][u]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int u = 0; u <= r; ++u) {
                    const float v = acc[r][u] * scale;
                    S[(size_t)(i0 + r) * L.s_ld + j0 + u] = v;
                    if (scheme == PSA_SYMMETRIC) S[(size_t)(j0 + u) * L.s_ld + i0 + r] = v;
                }
            qk += 10ull * d;
        } else {
            // a tile that the edge of the matrix crosses (n not a multiple of 4): weight by weight
            for (int r = 0; r < 4; ++r)
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + r, j = j0 + u;
                    if (i >= n || j >= n || (lower && j > i)) continue;
                    float acc = 0.f;
                    for (int c = 0; c < d; ++c) acc = fmaf(qt[(size_t)c * L.t_ld + i], kt[(size_t)c * L.t_ld + j], acc);
                    acc *= scale;
                    S[(size_t)i * L.s_ld + j] = acc;
                    if (scheme == PSA_SYMMETRIC) S[(size_t)j * L.s_ld + i] = acc;
                    qk += d;
                }
        }
    }
    __syncthreads();

    // ---- phase 2 (Eq. 2): one warp per row; the division is applied to the output row
    for (int i = warp; i < n; i += FS_THREADS / 32) {
        const int jend = masked ? i + 1 : n;
        float* row = S + (size_t)i * L.s_ld;
        float mx = -INFINITY;
        for (int j = lane; j < jend; j += 32) mx = fmaxf(mx, row[j]);
        for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float sum = 0.f;
        for (int j = lane; j < jend; j += 32) {
            const float e = expf(row[j] - mx);
            row[j] = e;
            sum += e;
        }
        for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) { rinv[i] = 1.f / sum; ex += (unsigned long long)jend; }
    }
    __syncthreads();

    // ---- phase 3 (Eq. 3): y_i = sum_j w_ij v_j over the kept weights, four output components per thread
    for (int t = tid; t < n * tc; t += FS_THREADS) {
        const int i = t / tc, c0 = (t - i * tc) * 4;
        const int jend = masked ? i + 1 : n;
        const float* row = S + (size_t)i * L.s_ld;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < jend; ++j) {
            const float w = row[j];
            const float4 v = *reinterpret_cast<const float4*>(vs + (size_t)j * L.ds + c0);
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y); acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        const float r = rinv[i];
        *reinterpret_cast<float4*>(out + ((size_t)b * n + i) * HD + (size_t)h * d + c0) = make_float4(acc.x * r, acc.y * r, acc.z * r, acc.w * r);
        pv += 4ull * jend;
    }

    // ---- census
    for (int off = 16; off; off >>= 1) {
        qk += __shfl_xor_sync(0xffffffffu, qk, off);
        pv += __shfl_xor_sync(0xffffffffu, pv, off);
        ex += __shfl_xor_sync(0xffffffffu, ex, off);
    }
    if (lane == 0) {
        if (qk) atomicAdd(&dc->qk_macs, qk);
        if (pv) atomicAdd(&dc->pv_macs, pv);
        if (ex) atomicAdd(&dc->exps, ex);
    }
    if (tid == 0) atomicAdd(&dc->proj_macs, (unsigned long long)nW * n * D * d);
}

// Asynchronous copies global -> shared (4 and 16 bytes) and the wait for all of a thread's copies.
__device__ __forceinline__ void cp_async4(float* dst, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// The same layer spread over a cluster of C CTAs (FULL and MASKED): 4-row tiles are dealt to the CTAs in turn (tile ti
// belongs to CTA ti % C, which balances the masked scheme's growing rows), each CTA projects q, k, v of its own rows,
// the CTAs read one another's k and v through distributed shared memory, and each finishes phases 1-3 for its rows.
// A layer of one head then occupies C SMs instead of one.  Tasks are one row by four columns, so that the few rows a
// CTA owns still spread over its threads; the census is element-exact as above.
__global__ void __launch_bounds__(FS_THREADS, 1)
f32_fused_cluster_kernel(const float* __restrict__ X, const float* __restrict__ Wq, const float* __restrict__ Wk,
                         const float* __restrict__ Wv, float* __restrict__ out, int n, int H, int D, int d, float scale,
                         int scheme, DeviceCounters* dc, DeviceCounters* dc_next) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    extern __shared__ float4 fs_smem4[];
    float* sm = reinterpret_cast<float*>(fs_smem4);
    const FusedLayout L = fused_layout(n, D, d, 3);
    float* xs = sm + L.xs; float* ws = sm + L.ws; float* qt = sm + L.qt; float* kt = sm + L.kt; float* vs = sm + L.vs;
    float* S = sm + L.sm; float* rinv = sm + L.rinv;
    const int head = blockIdx.x / C, b = head / H, h = head - b * H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool masked = scheme == PSA_MASKED;
    const size_t HD = (size_t)H * d;
    const int tn = (n + 3) / 4, tc = d / 4;
    const int own_tiles = rank < tn ? (tn - rank + C - 1) / C : 0;     // tiles rank, rank + C, ...
    const int own_rows = own_tiles * 4;                                // (the last tile's rows beyond n are skipped)
    auto own_row = [&](int lr) { return 4 * (rank + (lr >> 2) * C) + (lr & 3); };     // local row -> row of the head
    unsigned long long qk = 0, pv = 0, ex = 0, pj = 0;
    if (blockIdx.x == 0 && tid == 0 && dc_next) *dc_next = DeviceCounters{0, 0, 0, 0, 0, 0, 0};

    // ---- stage this CTA's rows of X[b] and the head's columns of the three projection matrices: asynchronous copies
    // straight into shared memory, all in flight at once (a layer this small lives on the latency of its first loads)
    {
        const float* xb = X + (size_t)b * n * D;
        for (int t = tid; t < own_rows * D; t += FS_THREADS) {
            const int lr = t / D, k = t - lr * D, i = own_row(lr);
            if (i < n) cp_async4(xs + i * L.xs_ld + k, xb + (size_t)i * D + k);
        }
        const int d4 = d / 4;
        for (int t = tid; t < 3 * D * d4; t += FS_THREADS) {
            const int w = t / (D * d4), rem = t - w * D * d4, k = rem / d4, c4 = rem - k * d4;
            const float* W = (w == 0 ? Wq : (w == 1 ? Wk : Wv)) + (size_t)h * d;
            cp_async16(ws + (size_t)w * D * d + (size_t)k * d + 4 * c4, W + (size_t)k * HD + 4 * c4);
        }
        cp_async_wait_all();
    }
    __syncthreads();

    // ---- projections (Sec. 3.1) of the own rows: one row by four columns per task
    for (int t = tid; t < 3 * own_rows * tc; t += FS_THREADS) {
        const int w = t / (own_rows * tc), rem = t - w * own_rows * tc;
        const int lr = rem / tc, c0 = (rem - lr * tc) * 4, i = own_row(lr);
        if (i >= n) continue;
        const float* wp = ws + (size_t)w * D * d + c0;
        const float* xr = xs + (size_t)i * L.xs_ld;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int k = 0; k < D; ++k) {
            const float4 wv = *reinterpret_cast<const float4*>(wp + (size_t)k * d);
            const float x = xr[k];
            acc.x = fmaf(x, wv.x, acc.x); acc.y = fmaf(x, wv.y, acc.y); acc.z = fmaf(x, wv.z, acc.z); acc.w = fmaf(x, wv.w, acc.w);
        }
        if (w < 2) {
            float* dst = (w == 0 ? qt : kt) + i;
            dst[(size_t)(c0 + 0) * L.t_ld] = acc.x; dst[(size_t)(c0 + 1) * L.t_ld] = acc.y;
            dst[(size_t)(c0 + 2) * L.t_ld] = acc.z; dst[(size_t)(c0 + 3) * L.t_ld] = acc.w;
        } else {
            *reinterpret_cast<float4*>(vs + (size_t)i * L.ds + c0) = acc;
        }
        pj += 4ull * D;
    }
    cluster.sync();           // every CTA's k and v rows are in its shared memory

    // ---- k and v of the other CTAs' rows, one 4-row tile (16 bytes of a transposed k component; a row of v) at a time
    for (int t = tid; t < d * tn; t += FS_THREADS) {
        const int c = t / tn, ti = t - c * tn, owner = ti % C;
        if (owner == rank) continue;
        const float* src = cluster.map_shared_rank(kt, owner);
        *reinterpret_cast<float4*>(kt + (size_t)c * L.t_ld + 4 * ti) = *reinterpret_cast<const float4*>(src + (size_t)c * L.t_ld + 4 * ti);
    }
    for (int t = tid; t < n * tc; t += FS_THREADS) {
        const int i = t / tc, c0 = (t - i * tc) * 4, owner = (i >> 2) % C;
        if (owner == rank) continue;
        const float* src = cluster.map_shared_rank(vs, owner);
        *reinterpret_cast<float4*>(vs + (size_t)i * L.ds + c0) = *reinterpret_cast<const float4*>(src + (size_t)i * L.ds + c0);
    }
    cluster.sync();           // no CTA reads another's shared memory from here on

    // ---- phase 1 (Eq. 1) for the own rows: S_ij = scale q_i . k_j, one row by four keys per task; a key beyond the
    // row's last kept one (masked: j > i; the edge: j >= n) is never computed
    for (int t = tid; t < own_rows * tn; t += FS_THREADS) {
        const int lr = t / tn, j0 = (t - lr * tn) * 4, i = own_row(lr);
        if (i >= n) continue;
        const int jlast = masked ? i : n - 1;
        if (j0 > jlast) continue;
        const int cnt = min(4, jlast - j0 + 1);                   // keys j0 .. j0 + cnt - 1 are kept
        const float* qp = qt + i;
        const float* kp = kt + j0;
        float* row = S + (size_t)i * L.s_ld + j0;
        if (cnt == 4) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int c = 0; c < d; ++c) {
                const float q = qp[(size_t)c * L.t_ld];
                const float4 k4 = *reinterpret_cast<const float4*>(kp + (size_t)c * L.t_ld);
                acc.x = fmaf(q, k4.x, acc.x); acc.y = fmaf(q, k4.y, acc.y); acc.z = fmaf(q, k4.z, acc.z); acc.w = fmaf(q, k4.w, acc.w);
            }
            row[0] = acc.x * scale; row[1] = acc.y * scale; row[2] = acc.z * scale; row[3] = acc.w * scale;
        } else {
            for (int u = 0; u < cnt; ++u) {
                float acc = 0.f;
                for (int c = 0; c < d; ++c) acc = fmaf(qp[(size_t)c * L.t_ld], kp[(size_t)c * L.t_ld + u], acc);
                row[u] = acc * scale;
            }
        }
        qk += (unsigned long long)cnt * d;
    }
    __syncthreads();

    // ---- phase 2 (Eq. 2): one warp per own row; the division is applied to the output row
    for (int lr = warp; lr < own_rows; lr += FS_THREADS / 32) {
        const int i = own_row(lr);
        if (i >= n) continue;
        const int jend = masked ? i + 1 : n;
        float* row = S + (size_t)i * L.s_ld;
        float mx = -INFINITY;
        for (int j = lane; j < jend; j += 32) mx = fmaxf(mx, row[j]);
        for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float sum = 0.f;
        for (int j = lane; j < jend; j += 32) {
            const float e = expf(row[j] - mx);
            row[j] = e;
            sum += e;
        }
        for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) { rinv[i] = 1.f / sum; ex += (unsigned long long)jend; }
    }
    __syncthreads();

    // ---- phase 3 (Eq. 3): y_i = sum_j w_ij v_j over the kept weights, four output components per task
    for (int t = tid; t < own_rows * tc; t += FS_THREADS) {
        const int lr = t / tc, c0 = (t - lr * tc) * 4, i = own_row(lr);
        if (i >= n) continue;
        const int jend = masked ? i + 1 : n;
        const float* row = S + (size_t)i * L.s_ld;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int j = 0; j < jend; ++j) {
            const float w = row[j];
            const float4 v = *reinterpret_cast<const float4*>(vs + (size_t)j * L.ds + c0);
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y); acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        const float r = rinv[i];
        *reinterpret_cast<float4*>(out + ((size_t)b * n + i) * HD + (size_t)h * d + c0) = make_float4(acc.x * r, acc.y * r, acc.z * r, acc.w * r);
        pv += 4ull * jend;
    }

    // ---- census
    for (int off = 16; off; off >>= 1) {
        qk += __shfl_xor_sync(0xffffffffu, qk, off);
        pv += __shfl_xor_sync(0xffffffffu, pv, off);
        ex += __shfl_xor_sync(0xffffffffu, ex, off);
        pj += __shfl_xor_sync(0xffffffffu, pj, off);
    }
    if (lane == 0) {
        if (qk) atomicAdd(&dc->qk_macs, qk);
        if (pv) atomicAdd(&dc->pv_macs, pv);
        if (ex) atomicAdd(&dc->exps, ex);
        if (pj) atomicAdd(&dc->proj_macs, pj);
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

bool f32_fused_fits(int n, int D, int d, int scheme) {
    if (n > 256 || d % 4 != 0 || d > 128) return false;
    return fused_layout(n, D, d, scheme == PSA_SYMMETRIC ? 1 : 3).total <= (size_t)FS_MAX_FLOATS;
}

// Heads few enough that one CTA each would leave most SMs idle are spread over clusters of up to 8 CTAs.
int f32_fused_cluster_size(int B, int H, int n, int scheme) {
    if (scheme == PSA_SYMMETRIC || B * H > 32) return 1;      // (the symmetric scheme's mirrored store crosses row owners)
    const int tn = (n + 3) / 4;
    int c = 1;
    while (c < 8 && 2 * c <= tn) c *= 2;
    return c;
}

cudaError_t f32_fused_layer(const float* X, const float* Wq, const float* Wk, const float* Wv, float* out, int B, int H,
                            int n, int D, int d, float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next,
                            cudaStream_t stream) {
    static DeviceSetup setup;
    if (device_setup(&setup, [] {
            cudaError_t e = cudaFuncSetAttribute(f32_fused_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 FS_MAX_FLOATS * (int)sizeof(float));
            if (e != cudaSuccess) return e;
            return cudaFuncSetAttribute(f32_fused_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        FS_MAX_FLOATS * (int)sizeof(float));
        }, "fp32 fused layer set-up") <= 0)
        return cudaErrorUnknown;
    const int C = f32_fused_cluster_size(B, H, n, scheme);
    if (C > 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(B * H * C);
        cfg.blockDim = dim3(FS_THREADS);
        cfg.dynamicSmemBytes = fused_layout(n, D, d, 3).total * sizeof(float);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = C;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, f32_fused_cluster_kernel, X, Wq, Wk, Wv, out, n, H, D, d, scale, scheme, dc, dc_next);
    }
    const size_t smem = fused_layout(n, D, d, scheme == PSA_SYMMETRIC ? 1 : 3).total * sizeof(float);
    f32_fused_layer_kernel<<<B * H, FS_THREADS, smem, stream>>>(X, Wq, scheme == PSA_SYMMETRIC ? Wq : Wk,
                                                               scheme == PSA_SYMMETRIC ? Wq : Wv, out, n, H, D, d, scale,
                                                               scheme, dc, dc_next);
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
