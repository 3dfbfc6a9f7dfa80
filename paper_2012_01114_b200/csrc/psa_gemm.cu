// Projection GEMM for the bf16 path (paper Sec. 3.1: q, k, v = x*Wq, x*Wk, x*Wv):
//     C_w[M, N] = A[M, K] * B_w[K, N] (+ R[M, N]),  w < nW,  bf16 row-major operands, fp32 accumulation in TMEM;
// the optional residual R is added in the epilogue (the output projection of the attention block).
//
// Persistent kernel, one CTA per SM, walking 128 x 256 output tiles (all three weight matrices in one
// launch).  Warp 0 streams operand tiles with TMA into a shared-memory ring, warp 1 issues tcgen05 MMAs
// (A K-major, B in its natural row-major form = MN-major) into one of two 256-column TMEM accumulators,
// warps 2-5 drain the other accumulator (TMEM -> registers -> bf16 -> swizzled shared memory -> TMA
// store, 64 columns at a time through two staging buffers so that the stores overlap the conversion),
// so that a tile's epilogue runs under the next tile's main loop.
#include <stdio.h>

#include <mutex>

#include "psa_internal.h"
#include "psa_tma.h"
#include "sm100.cuh"

namespace psa {

// ---------------------------------------------------------------- tensor-map helper
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_encode_once;
}  // namespace

namespace {
bool resolve_encode() {
    std::call_once(g_encode_once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    });
    if (!g_encode) { set_error_text("cuTensorMapEncodeTiled entry point not available"); return false; }
    return true;
}
}  // namespace

bool make_tensor_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_bytes,
                          uint32_t box_rows, uint32_t box_cols) {
    if (!resolve_encode()) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t es[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        set_error_text(msg);
        return false;
    }
    return true;
}

bool make_tensor_map_bf16_4d(CUtensorMap* map, const void* base, uint64_t batch, uint64_t n, uint64_t heads, uint64_t d,
                             uint32_t box_rows) {
    if (!resolve_encode()) return false;
    cuuint64_t dims[4] = {d, heads, n, batch};
    cuuint64_t strides[3] = {d * 2, heads * d * 2, n * heads * d * 2};
    cuuint32_t box[4] = {64, 1, box_rows, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled (4-D) failed with CUresult %d", (int)r);
        set_error_text(msg);
        return false;
    }
    return true;
}

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int NSUB = BN / 64;                  // 64-column sub-tiles of B and C per tile
#ifndef PSA_GEMM_STAGES
#define PSA_GEMM_STAGES 4
#endif
constexpr int STAGES = PSA_GEMM_STAGES;
constexpr int A_BYTES = BM * BK * 2;           // 16 KB, K-major [128 x 64]
constexpr int B_SUB_BYTES = BK * 64 * 2;       // 8 KB, one [64 k-rows x 64 n] sub-tile
constexpr int B_BYTES = NSUB * B_SUB_BYTES;    // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES; // 48 KB
constexpr int OUT_BYTES = 2 * BM * 64 * 2;      // 32 KB output staging: two swizzled [128 x 64] sub-tiles used in turn
constexpr int GEMM_THREADS = 192;
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES + OUT_BYTES + 1024;  // + slack for 1024-byte alignment
constexpr int TMEM_COLS = 2 * BN;              // two accumulators

struct GemmMaps {
    CUtensorMap a;
    CUtensorMap b[3];
    CUtensorMap c[3];
};

struct TileCoord {
    int w, m0, n0;
};
// Tile t of the launch: column tiles fastest, then row tiles, then the weight matrix, so that CTAs
// working side by side share the A row panel in L2.
__device__ __forceinline__ TileCoord tile_coord(int t, int mt, int nt) {
    TileCoord c;
    c.n0 = (t % nt) * BN;
    const int r = t / nt;
    c.m0 = (r % mt) * BM;
    c.w = r / mt;
    return c;
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ GemmMaps maps, int M, int N, int K, int nW, const uint16_t* __restrict__ R,
                 DeviceCounters* dc) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stage_out = smem + STAGES * STAGE_BYTES;
    __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nk = (K + BK - 1) / BK;
    const int mt = (M + BM - 1) / BM, nt = (N + BN - 1) / BN;
    const int ntiles = mt * nt * nW;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 128); }
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base_s, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;
    // (programmatic dependent launch: the set-up above overlaps the end of the kernel before this one)
    grid_launch_dependents();
    grid_dependency_wait();

    if (warp == 0 && lane == 0) {
        // ---- TMA producer: k-steps of all this CTA's tiles, numbered g = 0, 1, ... through the ring
        int g = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            const TileCoord c = tile_coord(t, mt, nt);
            for (int kt = 0; kt < nk; ++kt, ++g) {
                const int s = g % STAGES;
                if (g >= STAGES && !mbar_wait(&empty_bar[s], ((g / STAGES) - 1) & 1, abortp)) { ok = false; break; }
                uint8_t* sA = smem + s * STAGE_BYTES;
                uint8_t* sB = sA + A_BYTES;
                mbar_arrive_expect_tx(&full_bar[s], STAGE_BYTES);
                tma_load_2d(sA, &maps.a, &full_bar[s], kt * BK, c.m0);
#pragma unroll
                for (int u = 0; u < NSUB; ++u)
                    tma_load_2d(sB + u * B_SUB_BYTES, &maps.b[c.w], &full_bar[s], c.n0 + 64 * u, kt * BK);
            }
        }
        if (*abortp) {  // let copies already in flight land before the CTA goes away
            for (int k = max(0, g - STAGES); k < g; ++k) mbar_wait_drain(&full_bar[k % STAGES], (k / STAGES) & 1);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        const uint32_t idesc = umma_idesc_bf16(BM, BN, UMMA_K_MAJOR, UMMA_MN_MAJOR);
        // descriptor low words of stage 0; a stage or k-step is a constant added to them (sm100.cuh)
        const uint32_t a_lo0 = umma_desc_lo_kmajor(smem_u32(smem));
        const uint32_t b_lo0 = umma_desc_lo_mnmajor(smem_u32(smem + A_BYTES), B_SUB_BYTES);
        unsigned long long macs = 0;
        int g = 0, i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++i) {
            const int buf = i & 1;
            if (i >= 2) ok = mbar_wait(&acc_empty[buf], ((i >> 1) - 1) & 1, abortp);   // epilogue drained it
            if (!ok) break;
            tc_fence_after();
            const uint32_t acc = tmem + buf * BN;
            for (int kt = 0; kt < nk; ++kt, ++g) {
                const int s = g % STAGES;
                ok = mbar_wait(&full_bar[s], (g / STAGES) & 1, abortp);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + s * (STAGE_BYTES >> 4), b_lo = b_lo0 + s * (STAGE_BYTES >> 4);
                if (kt == 0) {
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_ss(acc, umma_desc_join(a_lo + k * (32 >> 4), UMMA_DESC_HI_SW128),
                                umma_desc_join(b_lo + k * (2048 >> 4), UMMA_DESC_HI_SW128), idesc, k != 0);
                } else {
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_ss(acc, umma_desc_join(a_lo + k * (32 >> 4), UMMA_DESC_HI_SW128),
                                umma_desc_join(b_lo + k * (2048 >> 4), UMMA_DESC_HI_SW128), idesc, 1);
                }
                umma_commit(&empty_bar[s]);
            }
            if (!ok) break;
            umma_commit(&acc_full[buf]);
            const TileCoord c = tile_coord(t, mt, nt);
            macs += (unsigned long long)min(BM, M - c.m0) * min(BN, N - c.n0) * K;
        }
        if (macs) atomicAdd(&dc->proj_macs, macs);
    }
    else if (warp >= 2) {
        // ---- epilogue: 4 warps, warp q owns TMEM lanes 32q .. 32q+31 = output rows
        const int q = warp & 3;
        const int row = q * 32 + lane;
        int i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
            const int buf = i & 1;
            if (ok) ok = mbar_wait(&acc_full[buf], (i >> 1) & 1, abortp);
            const TileCoord c = tile_coord(t, mt, nt);
            bool live = true;
#pragma unroll 1
            for (int u = 0; u < NSUB; ++u) {
                // The tile leaves in 64-column sub-tiles through two staging buffers used in turn: while the TMA store
                // of one reads its buffer, the next sub-tile is converted into the other.
                // This barrier is uniform across the four warps; it also orders the store that last used this buffer
                // (warp 2 lane 0 waited for it to have read the buffer) before the writes below.
                if (!named_bar_all(ok, 1, 128)) { live = false; break; }
                tc_fence_after();
                uint8_t* sub = stage_out + (u & 1) * 16384;
                uint32_t r[2][32];
                const uint32_t src = tmem + (static_cast<uint32_t>(q * 32) << 16) + buf * BN + u * 64;
                tmem_ld32(src, r[0]);
                tmem_ld32(src + 32, r[1]);
                tc_wait_ld();
                if (R) {
                    // residual input: C = A B + R, added in fp32 before the rounding to bf16 (R is [M, N] bf16, row-major)
                    const int grow = c.m0 + row, gcol = c.n0 + 64 * u;
                    if (grow < M && gcol < N) {
                        const uint4* rp = reinterpret_cast<const uint4*>(R + (size_t)grow * N + gcol);
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const uint4 x = __ldg(rp + g);
                            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                uint32_t* dst = &r[g >> 2][(g & 3) * 8 + 2 * e];
                                dst[0] = __float_as_uint(__uint_as_float(dst[0]) + __uint_as_float(w[e] << 16));
                                dst[1] = __float_as_uint(__uint_as_float(dst[1]) + __uint_as_float(w[e] & 0xffff0000u));
                            }
                        }
                    }
                }
#pragma unroll
                for (int c0 = 0; c0 < 2; ++c0) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {  // four 16-byte chunks of 8 bf16
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(r[c0][g * 8 + 0]), __uint_as_float(r[c0][g * 8 + 1]));
                        v.y = pack_bf16x2(__uint_as_float(r[c0][g * 8 + 2]), __uint_as_float(r[c0][g * 8 + 3]));
                        v.z = pack_bf16x2(__uint_as_float(r[c0][g * 8 + 4]), __uint_as_float(r[c0][g * 8 + 5]));
                        v.w = pack_bf16x2(__uint_as_float(r[c0][g * 8 + 6]), __uint_as_float(r[c0][g * 8 + 7]));
                        *reinterpret_cast<uint4*>(sub + swz128_offset(row, c0 * 4 + g)) = v;
                    }
                }
                if (u == NSUB - 1) {
                    tc_fence_before();
                    mbar_arrive(&acc_empty[buf]);      // the accumulator may be overwritten by tile i + 2
                }
                fence_async_smem();
                named_bar_sync(2, 128);
                if (warp == 2 && lane == 0) {
                    const int col = c.n0 + 64 * u;
                    if (col < N) tma_store_2d(&maps.c[c.w], sub, col, c.m0);
                    tma_store_commit();                // (an empty group when the sub-tile lies beyond N)
                    tma_store_wait_read_1();           // the OTHER buffer, stored one sub-tile ago, may be rewritten
                }
            }
            if (!live) { ok = false; break; }
        }
        if (warp == 2 && lane == 0) tma_store_wait_all();
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace

int bf16_project(const void* A, const void* const Bw[3], void* const C[3], int nW, int M, int K, int N,
                 const void* residual, DeviceCounters* dc, cudaStream_t stream) {
    static DeviceSetup setup;
    const int sm_count = device_setup(&setup, [] {
        return cudaFuncSetAttribute(gemm_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM);
    }, "gemm set-up");
    if (sm_count <= 0) return PSA_ERR_CUDA;
    GemmMaps maps;
    if (!make_tensor_map_bf16(&maps.a, A, M, K, (uint64_t)K * 2, BM, BK)) return PSA_ERR_CUDA;
    for (int w = 0; w < 3; ++w) {
        const int src = w < nW ? w : 0;
        if (!make_tensor_map_bf16(&maps.b[w], Bw[src], K, N, (uint64_t)N * 2, BK, 64)) return PSA_ERR_CUDA;
        if (!make_tensor_map_bf16(&maps.c[w], C[src], M, N, (uint64_t)N * 2, BM, 64)) return PSA_ERR_CUDA;
    }
    const int ntiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN) * nW;
    const int grid = ntiles < sm_count ? ntiles : sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = GEMM_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits for its predecessor itself
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_bf16_kernel, maps, M, N, K, nW, static_cast<const uint16_t*>(residual), dc);
    if (e != cudaSuccess) { set_cuda_error(e, "gemm_bf16_kernel launch"); return PSA_ERR_CUDA; }
    return PSA_OK;
}

}  // namespace psa
