// Attention core of the bf16 path: dispatch, and the two kernels of the symmetric scheme (paper Sec. 4).
//
// With query = key = value = X the weight matrix before the softmax is symmetric, w'_ij = w'_ji (paper
// Eq. 4), and the paper computes one member of each pair and reuses it.  On this machine the reuse goes
// through memory:
//
//   sym_scores_kernel   phase 1, one CTA per unordered pair of 128-row tiles {I, J}, J <= I: the block
//                       S_IJ = scale * X_I X_J^T on the tensor core, written ONCE to the scratch.  Blocks
//                       above the diagonal are neither computed nor stored.
//   sym_attn_kernel     phases 2 and 3 per 128-row tile: the row of blocks S_I,* is fetched into shared
//                       memory -- block (I, J) as stored for J <= I, block (J, I) read transposed for
//                       J > I (the reuse) -- then softmax and O += P V as in the fused kernel of the other
//                       schemes (two threads per row, P written to TMEM as bf16, V = X staged by TMA,
//                       accumulator O in TMEM, the division of Eq. 2 applied once to the output row).
//
// The scratch holds, per head, the T(T+1)/2 blocks at or below the block diagonal, each as one contiguous
// 64 KB image of its shared-memory form (four [128 rows x 32 fp32] sub-tiles in the 128-byte swizzle), so
// that a block moves between shared and global memory as one bulk copy of consecutive bytes.
//
// The fused persistent kernel of the FULL and MASKED schemes is in psa_attn_persist.cu.
#include "psa_internal.h"
#include "psa_sched.h"
#include "psa_softmax.cuh"
#include "psa_tma.h"
#include "sm100.cuh"

namespace psa {

namespace {

constexpr int S_SUB_BYTES = 128 * 32 * 4;       // one [128 rows x 32 fp32] sub-tile of a score block, 128-byte rows
constexpr int S_BLOCK_BYTES = 4 * S_SUB_BYTES;  // one 128 x 128 fp32 score block: 64 KB
#ifndef PSA_SYM_COPIES
#define PSA_SYM_COPIES 4
#endif
constexpr int S_COPIES = PSA_SYM_COPIES;        // bulk copies a block is moved in

template <int D>
struct SymCfg {
    static constexpr int SUB = D / 64;                  // 64-column sub-tiles per 128-row tile of X
    static constexpr int TILE_BYTES = 128 * D * 2;      // one X tile (bf16)
    static constexpr int VSTAGES = D == 128 ? 2 : 4;
    static constexpr int SMEM = 2 * S_BLOCK_BYTES + VSTAGES * TILE_BYTES + 1024;
    static constexpr int TMEM_P = 0, TMEM_O = 64;       // P (64 columns: 128 keys as bf16 pairs) | O (D columns)
    static constexpr int SCORES_SMEM = (S_BLOCK_BYTES > 2 * TILE_BYTES ? S_BLOCK_BYTES : 2 * TILE_BYTES) + 1024;
};

struct SymMaps {
    CUtensorMap x;     // X as [batch, n, H*d] bf16, boxes of 128 rows x 64 columns
    CUtensorMap o;     // output, like x
};

struct SymBars {
    uint64_t s_full[2], s_free[2];
    uint64_t v_full[4], v_empty[4];
    uint64_t p_ready[2], o_done[2];
};

// Phase 1 of the symmetric scheme (paper Sec. 4.1): one CTA per unordered tile pair {I, J}, J <= I, computes
// S_IJ = scale * X_I X_J^T once and stores it at block (I, J) of the scratch; the mirror block (J, I) is never
// formed: its readers take (I, J) transposed.
template <int D>
__global__ void __launch_bounds__(128)
sym_scores_kernel(const __grid_constant__ SymMaps maps, float* __restrict__ Sg, int n, int H, int bh0, float scale,
                  DeviceCounters* dc) {
    constexpr int SUB = D / 64, TILE_BYTES = 128 * D * 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + TILE_BYTES;
    uint8_t* sS = smem;                  // the finished block is staged over the operand tiles
    __shared__ uint64_t full_bar, acc_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = row_tiles(n);
    const int np = sym_pairs(T);
    const int hl = blockIdx.x / np;                 // head inside this pass
    int I, J;
    sym_pair(blockIdx.x - hl * np, &I, &J);
    const int bh = bh0 + hl, b = bh / H, h = bh - b * H;
    const int pair = blockIdx.x - hl * np;           // = I (I + 1) / 2 + J: the block's place in the head's scratch

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&full_bar, 1);
        mbar_init(&acc_bar, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_base_s, 128); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        mbar_arrive_expect_tx(&full_bar, 2 * TILE_BYTES);
        for (int u = 0; u < SUB; ++u) {
            tma_load_4d(sA + u * 16384, &maps.x, &full_bar, 64 * u, h, I * TILE, b);
            tma_load_4d(sB + u * 16384, &maps.x, &full_bar, 64 * u, h, J * TILE, b);
        }
        if (mbar_wait(&full_bar, 0, abortp)) {
            tc_fence_after();
            const uint32_t idesc = umma_idesc_bf16(128, 128, UMMA_K_MAJOR, UMMA_K_MAJOR);
            const uint32_t a = smem_u32(sA), bb = smem_u32(sB);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;
                umma_ss(tmem, umma_desc_kmajor(a + off), umma_desc_kmajor(bb + off), idesc, kk != 0);
            }
            umma_commit(&acc_bar);
            atomicAdd(&dc->qk_macs, (unsigned long long)TILE * TILE * D);
        } else {
            mbar_wait_drain(&full_bar, 0);
        }
    }
    __syncwarp();
    const bool ready = mbar_wait(&acc_bar, 0, abortp);
    if (__syncthreads_and(ready)) {
        // every MMA has read its operands: the block goes to shared memory as four [128 x 32] fp32 sub-tiles in
        // the 128-byte swizzle, each thread its own row, and from there to the scratch as one bulk copy
        tc_fence_after();
        const int r = warp * 32 + lane;
#pragma unroll 1
        for (int c0 = 0; c0 < 4; ++c0) {
            uint32_t v[32];
            tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + 32 * c0, v);
            tc_wait_ld();
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                float4 f;
                f.x = __uint_as_float(v[4 * g]) * scale;     f.y = __uint_as_float(v[4 * g + 1]) * scale;
                f.z = __uint_as_float(v[4 * g + 2]) * scale; f.w = __uint_as_float(v[4 * g + 3]) * scale;
                *reinterpret_cast<float4*>(sS + c0 * S_SUB_BYTES + swz128_offset(r, g)) = f;
            }
        }
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            float* dst = Sg + ((size_t)hl * np + pair) * (S_BLOCK_BYTES / 4);
            for (int u = 0; u < S_COPIES; ++u)
                bulk_store_1d(dst + u * (S_BLOCK_BYTES / S_COPIES / 4), sS + u * (S_BLOCK_BYTES / S_COPIES), S_BLOCK_BYTES / S_COPIES);
            tma_store_commit();
            tma_store_wait_read();   // shared memory may be released; the writes complete on their own
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 0) tmem_dealloc(tmem, 128);
}

// Phases 2 and 3 of the symmetric scheme for one 128-row tile of one head: softmax over the stored scores and
// O = P X.  320 threads: warp 0 = producer (score blocks and X tiles, bulk / TMA copies), warp 1 = MMA issuer,
// warps 2-9 = softmax and epilogue, two threads per row.  The kernel is bound by the arrival of its score blocks
// (64 KB per 128 x 128 weights), so these are double-buffered: block j + 1 is in flight while block j is in the
// softmax, and a buffer is released as soon as its scores are in registers.
constexpr int SYM_THREADS = 32 * (CTRL_WARPS + SOFTMAX_WARPS_PER_TILE);   // 320

template <int D>
__global__ void __launch_bounds__(SYM_THREADS, 1)
sym_attn_kernel(const __grid_constant__ SymMaps maps, const float* __restrict__ Sg, int n, int H, int bh0,
                DeviceCounters* dc) {
    using Cfg = SymCfg<D>;
    constexpr int VST = Cfg::VSTAGES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sS = smem;                                  // two 64 KB score blocks (stages)
    uint8_t* sV = smem + 2 * S_BLOCK_BYTES;              // VSTAGES tiles of X
    __shared__ SymBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ float xch_max[2][2][128];      // [block parity][column half][row]
    __shared__ float xch_sum[2][128];         // [column half][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = row_tiles(n);
    const int np = sym_pairs(T);
    const int hl = blockIdx.x / T;                       // head inside this pass
    const int It = blockIdx.x - hl * T;                  // row tile
    const int bh = bh0 + hl;
    const int b = bh / H, h = bh - b * H;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars.s_full[s], 1);
            mbar_init(&bars.s_free[s], 32 * SOFTMAX_WARPS_PER_TILE);
        }
        mbar_init(&bars.p_ready[0], 32 * SOFTMAX_WARPS_PER_TILE);
        mbar_init(&bars.o_done[0], 1);
        for (int s = 0; s < 4; ++s) { mbar_init(&bars.v_full[s], 1); mbar_init(&bars.v_empty[s], 1); }
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base_s, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ producer
            int s_loads = 0, v_loads = 0;
            bool ok = true;
            for (int j = 0; j < T && ok; ++j) {
                const int st = j & 1;
                // a stage is free once the softmax threads have taken block j - 2 into registers
                if (j >= 2) ok = mbar_wait(&bars.s_free[st], ((j >> 1) - 1) & 1, abortp);
                if (!ok) break;
                const int bi = j <= It ? It : j, bj = j <= It ? j : It;      // stored block (row tile, column tile)
                const float* src = Sg + ((size_t)hl * np + bi * (bi + 1) / 2 + bj) * (S_BLOCK_BYTES / 4);
                mbar_arrive_expect_tx(&bars.s_full[st], S_BLOCK_BYTES);
                for (int u = 0; u < S_COPIES; ++u)      // several copies in flight move a block faster than one
                    bulk_load_1d(sS + st * S_BLOCK_BYTES + u * (S_BLOCK_BYTES / S_COPIES), src + u * (S_BLOCK_BYTES / S_COPIES / 4),
                                 S_BLOCK_BYTES / S_COPIES, &bars.s_full[st]);
                ++s_loads;
                const int s = j % VST;
                if (j >= VST) ok = mbar_wait(&bars.v_empty[s], ((j / VST) - 1) & 1, abortp);
                if (!ok) break;
                mbar_arrive_expect_tx(&bars.v_full[s], Cfg::TILE_BYTES);
                for (int u = 0; u < Cfg::SUB; ++u)
                    tma_load_4d(sV + s * Cfg::TILE_BYTES + u * 16384, &maps.x, &bars.v_full[s], 64 * u, h, j * TILE, b);
                ++v_loads;
            }
            if (*abortp) {  // let copies already issued land before shared memory is released
                for (int c = max(0, s_loads - 2); c < s_loads; ++c) mbar_wait_drain(&bars.s_full[c & 1], (c >> 1) & 1);
                for (int c = max(0, v_loads - VST); c < v_loads; ++c) mbar_wait_drain(&bars.v_full[c % VST], (c / VST) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer: O (+)= P X_j (phase 3, Eq. 3)
            const uint32_t idescO = umma_idesc_bf16(128, D, UMMA_K_MAJOR, UMMA_MN_MAJOR);
            const uint32_t v_lo = umma_desc_lo_mnmajor(smem_u32(sV), 16384);
            const uint32_t dO = tmem + Cfg::TMEM_O, aP = tmem + Cfg::TMEM_P;
            unsigned long long pv_blocks = 0;
            bool ok = true;
            for (int j = 0; j < T && ok; ++j) {
                const int sv = j % VST;
                ok = mbar_wait(&bars.v_full[sv], (j / VST) & 1, abortp) && mbar_wait(&bars.p_ready[0], j & 1, abortp);
                if (!ok) break;
                tc_fence_after();
                const uint32_t v = v_lo + sv * (Cfg::TILE_BYTES >> 4);
                if (j == 0) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, kk != 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, 1);
                }
                ++pv_blocks;
                umma_commit(&bars.o_done[0]);
                umma_commit(&bars.v_empty[sv]);
            }
            if (pv_blocks) {
                atomicAdd(&dc->pv_macs, pv_blocks * (unsigned long long)TILE * TILE * D);
                atomicAdd(&dc->exps, pv_blocks * (unsigned long long)(TILE * TILE));
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue
        // Two threads share a query row; thread `part` owns block columns [64 part, 64 part + 64).
        constexpr int CPT = 128 / TPR, NCH = CPT / 32, OPT = D / TPR;
        constexpr float sl2 = LOG2E;                          // the stored scores carry the 1/sqrt(d) factor already
        const int sw = warp - CTRL_WARPS;
        const int part = sw >> 2;                               // which share of the row's columns
        const int q = warp & 3;                                 // TMEM lane quarter this warp may access
        const int r = q * 32 + lane;                            // row inside the tile = TMEM lane
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t tO = tmem + Cfg::TMEM_O + lane_off + part * OPT;
        const uint32_t tP = tmem + Cfg::TMEM_P + lane_off;
        const int pair_bar = 1 + q;                             // named barrier of the two warps sharing rows
        const int tile_bar = 9;                                 // named barrier of all softmax warps
        const int col_base = part * CPT;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < T; ++j) {
            const uint8_t* sblock = sS + (j & 1) * S_BLOCK_BYTES;
            ok = mbar_wait(&bars.s_full[j & 1], (j >> 1) & 1, abortp);
            ok = __all_sync(0xffffffffu, ok);
            // keys beyond the sequence (ragged last block) carry no weight; `cb` = last kept column
            const int nvalid = min(TILE, n - j * TILE);
            const bool ragged = nvalid < TILE;
            const int cb = nvalid - 1;
            float mx = -INFINITY;
            uint32_t sreg[NCH][32];
            if (ok) {
                // ---- this thread's 64 scores: from the block as stored (column tile j at or below the row tile), or
                // from the mirror block (j, I) read down its columns (the reused half)
                if (j <= It) {
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const uint8_t* sub = sblock + ((col_base >> 5) + c) * S_SUB_BYTES;
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const float4 f = *reinterpret_cast<const float4*>(sub + swz128_offset(r, g));
                            sreg[c][4 * g] = __float_as_uint(f.x); sreg[c][4 * g + 1] = __float_as_uint(f.y);
                            sreg[c][4 * g + 2] = __float_as_uint(f.z); sreg[c][4 * g + 3] = __float_as_uint(f.w);
                        }
                    }
                } else {
                    const uint8_t* sub = sblock + q * S_SUB_BYTES + (lane & 3) * 4;   // rows of the mirror block = my columns
#pragma unroll
                    for (int c = 0; c < NCH; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            sreg[c][i] = *reinterpret_cast<const uint32_t*>(sub + swz128_offset(col_base + 32 * c + i, lane >> 2));
                }
#pragma unroll
                for (int c = 0; c < NCH; ++c)
                    mx = ragged ? max_chunk32<true>(sreg[c], col_base + 32 * c, cb, mx)
                                : max_chunk32<false>(sreg[c], col_base + 32 * c, r, mx);
            }
            // the scores are in registers: the stage may take block j + 2
            mbar_arrive(&bars.s_free[j & 1]);
            // the two threads of a row exchange their half-row maxima (and leave together if either gave up a wait)
            xch_max[j & 1][part][r] = mx;
            ok = named_bar_all(ok, pair_bar, 64);
            if (!ok) break;
            mx = fmaxf(mx, xch_max[j & 1][part ^ 1][r]);
            const float mx2 = mx * sl2;
            float alpha = 1.f;
            if (mx2 > m_run + RESCALE_THRESHOLD) {   // also taken on the first block (m_run = -inf)
                alpha = ex2_mufu(m_run - mx2);
                m_run = mx2;
            }
            // P and O are still in use by PV_{j-1} until its commit.  A wait given up here is not acted on
            // before the next pair barrier, so that the two threads of a row stay together.
            if (j > 0) {
                ok = mbar_wait(&bars.o_done[0], (j - 1) & 1, abortp);
                ok = __all_sync(0xffffffffu, ok);
                tc_fence_after();
            }
            // ---- P = exp2(S * log2 e - m) as bf16 into TMEM
            float rowsum = 0.f;
            if (ok) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t pk[16];
                    const int kc = col_base + 32 * c;            // first key column of the chunk
                    rowsum += ragged ? exp_chunk32<true>(sreg[c], sl2, -m_run, kc, cb, pk)
                                     : exp_chunk32<false>(sreg[c], sl2, -m_run, kc, r, pk);
                    tmem_st16(tP + (kc >> 1), pk);
                }
            }
            l_run = fmaf(l_run, alpha, rowsum);
            if (ok && j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rare: a row maximum grew by > 2^8
                const unsigned grown = __ballot_sync(0xffffffffu, alpha != 1.f);
                if (part == 0 && lane == 0) atomicAdd(&dc->rescales, (unsigned long long)__popc(grown));
#pragma unroll
                for (int c = 0; c < OPT / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tO + 32 * c, v);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    tmem_st32(tO + 32 * c, v);
                }
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(&bars.p_ready[0]);
        }
        if (ok) ok = mbar_wait(&bars.o_done[0], (T - 1) & 1, abortp);
        xch_sum[part][r] = l_run;
        if (named_bar_all(ok, tile_bar, 32 * SOFTMAX_WARPS_PER_TILE)) {
            // ---- epilogue: y = O / l (the division of Eq. 2, applied once per output row); the first score stage,
            // which no copy targets any more, stages the bf16 tile for the TMA store
            tc_fence_after();
            const float inv = 1.f / (l_run + xch_sum[part ^ 1][r]);
            uint8_t* stage = sS;
#pragma unroll
            for (int c = 0; c < OPT / 32; ++c) {
                const int col = part * OPT + 32 * c;       // first of 32 output columns handled here
                uint32_t v[32];
                tmem_ld32(tO + 32 * c, v);
                tc_wait_ld();
                uint8_t* sub = stage + (col / 64) * 16384;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint4 o;
                    o.x = pack_bf16x2(__uint_as_float(v[g * 8 + 0]) * inv, __uint_as_float(v[g * 8 + 1]) * inv);
                    o.y = pack_bf16x2(__uint_as_float(v[g * 8 + 2]) * inv, __uint_as_float(v[g * 8 + 3]) * inv);
                    o.z = pack_bf16x2(__uint_as_float(v[g * 8 + 4]) * inv, __uint_as_float(v[g * 8 + 5]) * inv);
                    o.w = pack_bf16x2(__uint_as_float(v[g * 8 + 6]) * inv, __uint_as_float(v[g * 8 + 7]) * inv);
                    *reinterpret_cast<uint4*>(sub + swz128_offset(r, (col % 64) / 8 + g)) = o;
                }
            }
            fence_async_smem();
            named_bar_sync(tile_bar, 32 * SOFTMAX_WARPS_PER_TILE);
            if (sw == 0 && lane == 0) {
                for (int u = 0; u < Cfg::SUB; ++u)
                    tma_store_4d(&maps.o, stage + u * 16384, 64 * u, h, It * TILE, b);
                tma_store_commit();
                tma_store_wait_read();   // smem may be released; the writes complete on their own
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, 256);
}

// Heads per pass: as many as the scratch cap allows, in passes of equal size (the scratch is reused from pass
// to pass).  Passes small enough to stay in L2 were measured slower: the kernels of a small pass do not fill the GPU.
constexpr size_t SYM_SCRATCH_CAP = size_t(2) << 30;   // bytes of score scratch per pass

int sym_heads_per_pass(int B, int H, int n) {
    const size_t per_head = (size_t)sym_pairs(row_tiles(n)) * S_BLOCK_BYTES;
    const size_t all = (size_t)B * H;
    size_t hp = SYM_SCRATCH_CAP / per_head;
    if (hp < 1) hp = 1;
    if (hp > all) hp = all;
    const size_t passes = (all + hp - 1) / hp;
    return (int)((all + passes - 1) / passes);
}

// D: head size the kernels work with (64 or 128); d <= D: the tensors' head size (see the 4-D tensor maps).
template <int D>
int launch_symmetric(const void* X, void* out, float* S, int B, int H, int n, int d, float scale, DeviceCounters* dc,
                     cudaStream_t stream) {
    using Cfg = SymCfg<D>;
    static DeviceSetup setup;
    if (device_setup(&setup, [] {
            cudaError_t e = cudaFuncSetAttribute(sym_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, SymCfg<D>::SMEM);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(sym_scores_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, SymCfg<D>::SCORES_SMEM);
            return e;
        }, "cudaFuncSetAttribute(symmetric attention)") <= 0)
        return PSA_ERR_CUDA;
    const int T = row_tiles(n), np = sym_pairs(T);
    const int hp = sym_heads_per_pass(B, H, n);
    SymMaps maps;
    if (!make_tensor_map_bf16_4d(&maps.x, X, B, n, H, d, 128) || !make_tensor_map_bf16_4d(&maps.o, out, B, n, H, d, 128))
        return PSA_ERR_CUDA;
    for (int bh0 = 0; bh0 < B * H; bh0 += hp) {
        const int heads = min(hp, B * H - bh0);
        sym_scores_kernel<D><<<heads * np, 128, Cfg::SCORES_SMEM, stream>>>(maps, S, n, H, bh0, scale, dc);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { set_cuda_error(e, "sym_scores_kernel launch"); return PSA_ERR_CUDA; }
        sym_attn_kernel<D><<<heads * T, SYM_THREADS, Cfg::SMEM, stream>>>(maps, S, n, H, bh0, dc);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_cuda_error(e, "sym_attn_kernel launch"); return PSA_ERR_CUDA; }
    }
    return PSA_OK;
}

}  // namespace

size_t bf16_symmetric_scratch_bytes(int B, int H, int n) {
    return (size_t)sym_heads_per_pass(B, H, n) * sym_pairs(row_tiles(n)) * S_BLOCK_BYTES;
}

int bf16_attention(const void* Q, const void* K, const void* V, void* out, float* S, size_t s_bytes, int B, int H,
                   int n, int d, float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next, cudaStream_t stream) {
    if (scheme != PSA_SYMMETRIC && d > 128) return bf16_attention_wide(Q, K, V, out, B, H, n, d, scale, scheme, dc, stream);
    if (scheme != PSA_SYMMETRIC) return bf16_attention_persist(Q, K, V, out, B, H, n, d, scale, scheme, dc, dc_next, stream);
    if (!S || s_bytes < bf16_symmetric_scratch_bytes(B, H, n)) return PSA_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(S) & 15u) != 0) return PSA_ERR_ALIGN;
    if (d < 8 || d > 128 || d % 8) return PSA_ERR_UNSUPPORTED;
    if (d <= 64) return launch_symmetric<64>(Q, out, S, B, H, n, d, scale, dc, stream);
    return launch_symmetric<128>(Q, out, S, B, H, n, d, scale, dc, stream);
}

}  // namespace psa
