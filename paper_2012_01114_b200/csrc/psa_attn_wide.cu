// Fused attention core of the bf16 path for head sizes 128 < d_k <= 256 (FULL and MASKED schemes): phases 1-3 of the
// paper (Eq. 1-3) for one (batch, head, 128-row query tile) per CTA, never materialising the weight matrix.
//
// A 256-column output accumulator leaves tensor memory room for one row tile only (S 128 + O 256 of 512 columns), and
// shared memory room for one stage of K and one of V (Q, K, V tiles of 64 KB each), so this kernel is a plain chain
// per key block -- S = Q K^T (16 MMAs of 128 x 128 x 16), softmax, O += P V (8 MMAs of 128 x 256 x 16) -- without
// the second row tile that keeps the tensor pipe busy in the kernel for d_k <= 128.  It exists so that the head sizes
// up to 256 run on the tensor cores at all; the masked scheme's blocks beyond the diagonal are absent from every loop
// here too, and only the block on the diagonal carries an element predicate.
//
// CTA layout (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer, warps 2-9 = softmax and epilogue (a warp owns
// 16 rows, read in the quad layout of sm100.cuh).  TMEM columns: S [0, 128), P (bf16) over S [0, 64), O [128, 384).
// The tensors' head size may be any multiple of 8 in (128, 256]: columns beyond d_k are zero-filled by the loads and
// dropped by the stores.
#include "psa_internal.h"
#include "psa_sched.h"
#include "psa_softmax.cuh"
#include "psa_tma.h"
#include "sm100.cuh"

namespace psa {

namespace {

constexpr int WD = 256;                                  // padded head width
constexpr int W_SUB = WD / 64;                           // 64-column sub-tiles of a tile
constexpr int W_TILE_BYTES = 128 * WD * 2;               // one Q, K or V tile: 64 KB
constexpr int W_WARPS = 8;                               // softmax warps
constexpr int W_THREADS = 32 * (2 + W_WARPS);
constexpr int W_STAGE_BYTES = 16 * 64 * 2;               // a warp's output staging buffer: 16 rows x 64 columns
constexpr int W_SMEM = 3 * W_TILE_BYTES + W_WARPS * W_STAGE_BYTES + 1024;
constexpr int W_TMEM_S = 0, W_TMEM_O = 128;

struct WMaps {
    CUtensorMap q, k, v, o;
};

struct WBars {
    uint64_t q_full, k_full, k_empty, v_full, v_empty, s_full, p_ready, o_done;
};

__global__ void __launch_bounds__(W_THREADS, 1)
attn_wide_kernel(const __grid_constant__ WMaps maps, int n, int d, int H, int nbh, int scheme, float sl2,
                 DeviceCounters* dc) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + W_TILE_BYTES;
    uint8_t* sV = sK + W_TILE_BYTES;
    uint8_t* sStage = sV + W_TILE_BYTES;
    __shared__ WBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = row_tiles(n);
    const bool masked = scheme == PSA_MASKED;
    // CTAs are numbered row tile by row tile, all heads of a tile together; the masked scheme starts with the last
    // (longest) row tile, so that the short ones fill the end of the launch
    const int it = blockIdx.x / nbh, bh = blockIdx.x - it * nbh;
    const int It = masked ? T - 1 - it : it;
    const int b = bh / H, h = bh - b * H;
    const int nkv = kv_tiles(It, T, scheme);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bars.q_full, 1);
        mbar_init(&bars.k_full, 1);
        mbar_init(&bars.k_empty, 1);
        mbar_init(&bars.v_full, 1);
        mbar_init(&bars.v_empty, 1);
        mbar_init(&bars.s_full, 1);
        mbar_init(&bars.p_ready, W_WARPS);          // one arrival per softmax warp
        mbar_init(&bars.o_done, 1);
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            bool ok = true;
            mbar_arrive_expect_tx(&bars.q_full, W_TILE_BYTES);
            for (int u = 0; u < W_SUB; ++u) tma_load_4d(sQ + u * 16384, &maps.q, &bars.q_full, 64 * u, h, It * TILE, b);
            int issued = 0;                              // key blocks whose loads were issued
            for (int j = 0; j < nkv && ok; ++j) {
                if (j > 0) ok = mbar_wait(&bars.k_empty, (j - 1) & 1, abortp);
                if (!ok) break;
                mbar_arrive_expect_tx(&bars.k_full, W_TILE_BYTES);
                for (int u = 0; u < W_SUB; ++u) tma_load_4d(sK + u * 16384, &maps.k, &bars.k_full, 64 * u, h, j * TILE, b);
                if (j > 0) ok = mbar_wait(&bars.v_empty, (j - 1) & 1, abortp);
                if (!ok) {      // K_j is in flight, V_j is not
                    mbar_wait_drain(&bars.k_full, j & 1);
                    break;
                }
                mbar_arrive_expect_tx(&bars.v_full, W_TILE_BYTES);
                for (int u = 0; u < W_SUB; ++u) tma_load_4d(sV + u * 16384, &maps.v, &bars.v_full, 64 * u, h, j * TILE, b);
                issued = j + 1;
            }
            if (*abortp) {      // let copies already issued land before shared memory is released
                mbar_wait_drain(&bars.q_full, 0);
                if (issued > 0) {
                    mbar_wait_drain(&bars.k_full, (issued - 1) & 1);
                    mbar_wait_drain(&bars.v_full, (issued - 1) & 1);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            // S_j may overwrite S_{j-1} and P_{j-1} only behind PV_{j-1}: the tensor pipe runs this thread's MMAs in
            // order, so issuing S_j after PV_{j-1} is enough.
            const uint32_t idescS = umma_idesc_bf16(128, 128, UMMA_K_MAJOR, UMMA_K_MAJOR);
            const uint32_t idescO = umma_idesc_bf16(128, WD, UMMA_K_MAJOR, UMMA_MN_MAJOR);
            const uint32_t q_lo = umma_desc_lo_kmajor(smem_u32(sQ)), k_lo = umma_desc_lo_kmajor(smem_u32(sK));
            const uint32_t v_lo = umma_desc_lo_mnmajor(smem_u32(sV), 16384);
            const uint32_t dS = tmem + W_TMEM_S, dO = tmem + W_TMEM_O;
            int done = 0;
            bool ok = mbar_wait(&bars.q_full, 0, abortp);
            for (int j = 0; j < nkv && ok; ++j) {
                ok = mbar_wait(&bars.k_full, j & 1, abortp);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < WD / 16; ++kk) {       // phase 1 (Eq. 1): S = Q K_j^T
                    const uint32_t off = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    umma_ss(dS, umma_desc_join(q_lo + off, UMMA_DESC_HI_SW128), umma_desc_join(k_lo + off, UMMA_DESC_HI_SW128),
                            idescS, kk != 0);
                }
                umma_commit(&bars.s_full);
                umma_commit(&bars.k_empty);
                ok = mbar_wait(&bars.v_full, j & 1, abortp) && mbar_wait(&bars.p_ready, j & 1, abortp);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)               // phase 3 (Eq. 3): O (+)= P_j V_j, 16 keys per MMA
                    umma_ts(dO, dS + kk * 8, umma_desc_join(v_lo + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO,
                            (j != 0 || kk != 0) ? 1u : 0u);
                umma_commit(&bars.o_done);
                umma_commit(&bars.v_empty);
                ++done;
            }
            const unsigned long long block_macs = (unsigned long long)TILE * TILE * WD;
            if (done) {
                atomicAdd(&dc->qk_macs, done * block_macs);
                atomicAdd(&dc->pv_macs, done * block_macs);
                atomicAdd(&dc->exps, done * (unsigned long long)(TILE * TILE));
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue
        const int wq = warp - 2;                                // softmax warp 0-7
        const int q = warp & 3;                                 // TMEM lane quarter this warp may access
        const int row0 = q * 32 + (wq >> 2) * 16;               // first of the warp's 16 rows inside the tile
        const int rA = row0 + (lane >> 2), rB = rA + 8;         // this thread's rows
        const int cq = 2 * (lane & 3);                          // its first column inside every group of 8
        const uint32_t lane_off = static_cast<uint32_t>(row0) << 16;
        const uint32_t tS = tmem + W_TMEM_S + lane_off, tO = tmem + W_TMEM_O + lane_off;
        uint8_t* stage = sStage + wq * W_STAGE_BYTES;
        float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;       // running maxima (log2 units) and row sums
        bool ok = true;
        for (int j = 0; j < nkv; ++j) {
            // S_j lies behind PV_{j-1} in the tensor pipe: its commit also says that O and P_{j-1} are at rest
            ok = __all_sync(0xffffffffu, mbar_wait(&bars.s_full, j & 1, abortp));
            if (!ok) break;
            const int nvalid = min(TILE, n - j * TILE);
            const bool on_diag = masked && (j == It);
            const bool diag = on_diag || nvalid < TILE;
            const int cbA = min(on_diag ? rA : TILE - 1, nvalid - 1);
            const int cbB = min(on_diag ? rB : TILE - 1, nvalid - 1);
            uint32_t s0[32], s1[32];
            tc_fence_after();
            tmem_ld_quad64(tS, s0);
            tmem_ld_quad64(tS + 64, s1);
            tc_wait_ld();
            if (diag) {
                mask_quad64(s0, cq, cbA, cbB);
                mask_quad64(s1, 64 + cq, cbA, cbB);
            }
            float bA = -INFINITY, bB = -INFINITY;
            max_quad64(s0, bA, bB);
            max_quad64(s1, bA, bB);
            bA = quad_max(bA) * sl2;
            bB = quad_max(bB) * sl2;
            float alphaA = 1.f, alphaB = 1.f;
            if (bA > mA + RESCALE_THRESHOLD) {   // also taken on the first block (m = -inf)
                alphaA = ex2_mufu(mA - bA);
                mA = bA;
            }
            if (bB > mB + RESCALE_THRESHOLD) {
                alphaB = ex2_mufu(mB - bB);
                mB = bB;
            }
            float sumA = 0.f, sumB = 0.f;
            uint32_t pk[16];
            exp_quad64(s0, sl2, -mA, -mB, pk, sumA, sumB);
            tmem_st_quad32(tS, pk);
            exp_quad64(s1, sl2, -mA, -mB, pk, sumA, sumB);
            tmem_st_quad32(tS + 32, pk);
            lA = fmaf(lA, alphaA, sumA);
            lB = fmaf(lB, alphaB, sumB);
            if (j > 0 && __any_sync(0xffffffffu, alphaA != 1.f || alphaB != 1.f)) {   // rare: a row maximum grew by > 2^8
                const int nA = __popc(__ballot_sync(0xffffffffu, (lane & 3) == 0 && alphaA != 1.f));
                const int nB = __popc(__ballot_sync(0xffffffffu, (lane & 3) == 0 && alphaB != 1.f));
                if (lane == 0) atomicAdd(&dc->rescales, (unsigned long long)(nA + nB));
#pragma unroll 1
                for (int c = 0; c < WD / 64; ++c) {
                    uint32_t v[32];
                    tmem_ld_quad64(tO + 64 * c, v);
                    tc_wait_ld();
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        v[4 * g] = __float_as_uint(__uint_as_float(v[4 * g]) * alphaA);
                        v[4 * g + 1] = __float_as_uint(__uint_as_float(v[4 * g + 1]) * alphaA);
                        v[4 * g + 2] = __float_as_uint(__uint_as_float(v[4 * g + 2]) * alphaB);
                        v[4 * g + 3] = __float_as_uint(__uint_as_float(v[4 * g + 3]) * alphaB);
                    }
                    tmem_st_quad64(tO + 64 * c, v);
                }
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.p_ready);
        }
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars.o_done, (nkv - 1) & 1, abortp));
        if (ok) {
            // ---- epilogue: y = O / l (the division of Eq. 2, applied once per output row), bf16, 64 columns at a time
            tc_fence_after();
            const float invA = 1.f / quad_sum(lA), invB = 1.f / quad_sum(lB);
#pragma unroll 1
            for (int u = 0; u < W_SUB; ++u) {
                uint32_t v[32];
                tmem_ld_quad64(tO + 64 * u, v);
                tc_wait_ld();
                if (u > 0) {                // the store that last used the buffer must have read it
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                }
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint32_t a = pack_bf16x2(__uint_as_float(v[4 * g]) * invA, __uint_as_float(v[4 * g + 1]) * invA);
                    const uint32_t bb = pack_bf16x2(__uint_as_float(v[4 * g + 2]) * invB, __uint_as_float(v[4 * g + 3]) * invB);
                    *reinterpret_cast<uint32_t*>(stage + swz128_offset(lane >> 2, g) + 2 * cq) = a;
                    *reinterpret_cast<uint32_t*>(stage + swz128_offset((lane >> 2) + 8, g) + 2 * cq) = bb;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0 && 64 * u < d) {      // (a sub-tile wholly beyond the head's columns is not stored)
                    tma_store_4d(&maps.o, stage, 64 * u, h, It * TILE + row0, b);
                    tma_store_commit();
                }
            }
            if (lane == 0) tma_store_wait_read();    // shared memory may be released; the writes complete on their own
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace

// FULL and MASKED schemes for 128 < d <= 256 (d a multiple of 8).
int bf16_attention_wide(const void* Q, const void* K, const void* V, void* out, int B, int H, int n, int d, float scale,
                        int scheme, DeviceCounters* dc, cudaStream_t stream) {
    if (d <= 128 || d > WD || d % 8) return PSA_ERR_UNSUPPORTED;
    static DeviceSetup setup;
    const int sm_count = device_setup(&setup, [] {
        return cudaFuncSetAttribute(attn_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, W_SMEM);
    }, "wide attention kernel set-up");
    if (sm_count <= 0) return PSA_ERR_CUDA;
    WMaps maps;
    if (!make_tensor_map_bf16_4d(&maps.q, Q, B, n, H, d, 128) || !make_tensor_map_bf16_4d(&maps.k, K, B, n, H, d, 128) ||
        !make_tensor_map_bf16_4d(&maps.v, V, B, n, H, d, 128) || !make_tensor_map_bf16_4d(&maps.o, out, B, n, H, d, 16))
        return PSA_ERR_CUDA;
    const long long ctas = (long long)B * H * row_tiles(n);
    if (ctas > 0x7fffffffLL) return PSA_ERR_SHAPE;
    attn_wide_kernel<<<(int)ctas, W_THREADS, W_SMEM, stream>>>(maps, n, d, H, B * H, scheme, scale * LOG2E, dc);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, "attn_wide_kernel launch"); return PSA_ERR_CUDA; }
    return PSA_OK;
}

}  // namespace psa
