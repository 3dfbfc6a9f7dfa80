// Fused attention core for the bf16 path: phases 1-3 of the paper (Eq. 1-3) per (batch, head) and
// per pair of 128-row query tiles, never materialising the n x n weight matrix.
//
//   phase 1  S = Q K^T            tcgen05 MMA, operands staged by TMA, accumulator in TMEM
//   phase 2  softmax              two threads per query row (64 columns each) read S from TMEM, keep a
//                                 running row maximum m and row sum l (the division of Eq. 2 is
//                                 applied once to the output row), write P = exp2(..) as bf16 back
//                                 into TMEM over S
//   phase 3  O += P V             tcgen05 MMA with P read from TMEM and V (row-major = MN-major) from
//                                 shared memory, accumulator O in TMEM
//
// Which (row tile, column tile) blocks exist is decided by the tile scheduler (psa_sched.h): for
// the masked scheme (paper Sec. 5) column tiles beyond the diagonal are absent from every loop in
// this file -- not loaded, not multiplied, not exponentiated -- and only the block on the diagonal
// carries an element predicate.  For the symmetric scheme (paper Sec. 4) phase 1 is a separate
// kernel that computes one block per unordered tile pair and stores it at both mirror positions;
// this kernel then runs phases 2 and 3 reading S from that scratch.
//
// CTA layout (576 threads with two softmax threads per row, the default): warp 0 = TMA producer, warp 1 =
// MMA issuer, warps 2-9 = softmax and epilogue of row tile 0, warps 10-17 = the same for row tile 1.
// Within a tile's eight warps, warp pairs (w, w+4) share a TMEM lane quarter (32 rows) and split the
// 128 columns of S in halves; the pair agrees on the row maximum through shared memory.  (Built with
// PSA_THREADS_PER_ROW=1 each row has one thread, four warps per tile, 320 threads.)  The two row tiles ping-pong: while the
// softmax warps of one work on S_j, the tensor core runs the other's MMAs.
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [256+D,256+2D); P_t (bf16, two per column)
// overlays S_t: keys 0-63 at S_t columns [0,32), keys 64-127 at [64,96), each written by the thread that
// owns that half of the row, so no thread overwrites scores another thread still has to read.
//
// exp2 is evaluated on the special-function unit for most elements and, for a fixed fraction of
// them, by a degree-3 polynomial on the FMA pipe (range reduction by the round-to-nearest "magic
// number" addition, exponent re-inserted with an integer add), because at these tile shapes the
// special-function unit is as loaded as the tensor core.  Relative error of the polynomial:
// 1.5e-4, well inside the bf16 rounding of P.
#include "psa_internal.h"
#include "psa_sched.h"
#include "psa_softmax.cuh"
#include "psa_tma.h"
#include "sm100.cuh"

namespace psa {

namespace {

#ifndef PSA_SOFTMAX_SLEEP_NS
#define PSA_SOFTMAX_SLEEP_NS 0
#endif
#ifndef PSA_RELOAD_S
#define PSA_RELOAD_S 1
#endif

template <int D>
struct AttnCfg {
    static constexpr int SUB = D / 64;                  // 64-column sub-tiles per 128-row tile
    static constexpr int TILE_BYTES = 128 * D * 2;      // one Q, K or V tile
    static constexpr int KSTAGES = D == 128 ? 2 : 4;
    static constexpr int VSTAGES = D == 128 ? 2 : 4;
    static constexpr int SMEM = (2 + KSTAGES + VSTAGES) * TILE_BYTES + 1024;
    // With d = 64 the 512 TMEM columns have room for P outside S (S0 S1 | P0 P1 | O0 O1): S_{j+1} can then be
    // computed while the softmax of block j is still running.  With d = 128 P overlays S.
    static constexpr bool SEP_P = D == 64;
    static constexpr int TMEM_S = 0, TMEM_P = 256, TMEM_O = SEP_P ? 384 : 256;
    // of every 4 consecutive elements, this many take the polynomial exp2 (FMA pipe) instead of MUFU
    static constexpr int POLY_OF_4 = PSA_POLY_OF_4;
};

struct AttnMaps {
    CUtensorMap q, k, v, o;
};

struct AttnBars {
    uint64_t q_full[2];
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
    uint64_t s_full[2], p_ready[2], o_done[2], s_free[2];
};

template <int D, bool SYM>
__global__ void __launch_bounds__(ATTN_THREADS, 1)
attn_kernel(const __grid_constant__ AttnMaps maps, const float* __restrict__ Sg, int n, int H, int scheme, int bh0,
            int nbh, int group, float sl2, DeviceCounters* dc) {
    using Cfg = AttnCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                          // 2 tiles
    uint8_t* sK = sQ + 2 * Cfg::TILE_BYTES;                      // KSTAGES tiles
    uint8_t* sV = sK + Cfg::KSTAGES * Cfg::TILE_BYTES;           // VSTAGES tiles
    __shared__ AttnBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ float xch_max[2][2][2][128];   // [step parity][tile][column half][row]
    __shared__ float xch_sum[2][2][128];      // [tile][column half][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = row_tiles(n);
    const CtaWork work = cta_work(blockIdx.x, n, scheme == PSA_MASKED, nbh, group);
    const int bh = bh0 + work.bh;
    const int b = bh / H, h = bh - b * H;
    const int col0 = h * D;
    const int nkv0 = kv_tiles(work.tile0, T, scheme);
    const int nkv1 = work.ntiles > 1 ? kv_tiles(work.tile0 + 1, T, scheme) : 0;
    const int maxkv = max(nkv0, nkv1);
    const int last_t = work.ntiles - 1;

    // TMA requests of one Q, K or V tile (issued by thread 0 only)
    auto load_q = [&](int t) {
        mbar_arrive_expect_tx(&bars.q_full[t], Cfg::TILE_BYTES);
        for (int u = 0; u < Cfg::SUB; ++u)
            tma_load_3d(sQ + t * Cfg::TILE_BYTES + u * 16384, &maps.q, &bars.q_full[t], col0 + 64 * u,
                        (work.tile0 + t) * TILE, b);
    };
    auto load_k = [&](int j) {
        if (SYM) return;
        const int s = j % Cfg::KSTAGES;
        mbar_arrive_expect_tx(&bars.k_full[s], Cfg::TILE_BYTES);
        for (int u = 0; u < Cfg::SUB; ++u)
            tma_load_3d(sK + s * Cfg::TILE_BYTES + u * 16384, &maps.k, &bars.k_full[s], col0 + 64 * u, j * TILE, b);
    };
    auto load_v = [&](int j) {
        const int s = j % Cfg::VSTAGES;
        mbar_arrive_expect_tx(&bars.v_full[s], Cfg::TILE_BYTES);
        for (int u = 0; u < Cfg::SUB; ++u)
            tma_load_3d(sV + s * Cfg::TILE_BYTES + u * 16384, &maps.v, &bars.v_full[s], col0 + 64 * u, j * TILE, b);
    };
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(&bars.q_full[t], 1);
            mbar_init(&bars.s_full[t], 1);
            mbar_init(&bars.s_free[t], 32 * SOFTMAX_WARPS_PER_TILE);
            mbar_init(&bars.p_ready[t], 32 * SOFTMAX_WARPS_PER_TILE);
            mbar_init(&bars.o_done[t], 1);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(&bars.k_full[s], 1); mbar_init(&bars.k_empty[s], 1);
            mbar_init(&bars.v_full[s], 1); mbar_init(&bars.v_empty[s], 1);
        }
        fence_mbar_init();
        // The first operand tiles need no free-stage wait: request them now, so that their flight
        // overlaps the TMEM allocation and the CTA-wide barrier below.
        for (int t = 0; t < work.ntiles; ++t) load_q(t);
        for (int j = 0; j < maxkv && j < Cfg::KSTAGES; ++j) load_k(j);
        for (int j = 0; j < maxkv && j < Cfg::VSTAGES; ++j) load_v(j);
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
            // (Q and the first KSTAGES / VSTAGES key and value tiles were requested during set-up.)
            int jk = SYM ? 0 : min(maxkv, Cfg::KSTAGES), jv = min(maxkv, Cfg::VSTAGES);
            for (int j = 0; j < maxkv; ++j) {
                if (!SYM && j >= Cfg::KSTAGES) {
                    if (!mbar_wait(&bars.k_empty[j % Cfg::KSTAGES], ((j / Cfg::KSTAGES) - 1) & 1, abortp)) break;
                    load_k(j);
                    jk = j + 1;
                }
                if (j >= Cfg::VSTAGES) {
                    if (!mbar_wait(&bars.v_empty[j % Cfg::VSTAGES], ((j / Cfg::VSTAGES) - 1) & 1, abortp)) break;
                    load_v(j);
                    jv = j + 1;
                }
            }
            if (*abortp) {  // let copies already issued land before shared memory is released
                for (int t = 0; t < work.ntiles; ++t) mbar_wait_drain(&bars.q_full[t], 0);
                for (int j = max(0, jk - Cfg::KSTAGES); j < jk; ++j)
                    mbar_wait_drain(&bars.k_full[j % Cfg::KSTAGES], (j / Cfg::KSTAGES) & 1);
                for (int j = max(0, jv - Cfg::VSTAGES); j < jv; ++j)
                    mbar_wait_drain(&bars.v_full[j % Cfg::VSTAGES], (j / Cfg::VSTAGES) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            const uint32_t idescS = umma_idesc_bf16(128, 128, UMMA_K_MAJOR, UMMA_K_MAJOR);
            const uint32_t idescO = umma_idesc_bf16(128, D, UMMA_K_MAJOR, UMMA_MN_MAJOR);
            unsigned long long qk_blocks = 0, pv_blocks = 0;
            bool ok = true;
            constexpr bool SEP = Cfg::SEP_P && !SYM;
            // Descriptor low words of the operand bases; per MMA only a constant is added (sm100.cuh).
            const uint32_t q_lo0 = umma_desc_lo_kmajor(smem_u32(sQ)), q_lo1 = umma_desc_lo_kmajor(smem_u32(sQ + Cfg::TILE_BYTES));
            const uint32_t k_lo = umma_desc_lo_kmajor(smem_u32(sK));
            const uint32_t v_lo = umma_desc_lo_mnmajor(smem_u32(sV), 16384);
            const uint32_t tS0 = tmem + Cfg::TMEM_S, tO0 = tmem + Cfg::TMEM_O;
            // S_t = Q_t K_j^T (phase 1, Eq. 1): D/16 MMAs of 128x128x16 into the tile's S columns.
            auto mma_S = [&](int t, int j) {
                const uint32_t q = t ? q_lo1 : q_lo0, k = k_lo + (j % Cfg::KSTAGES) * (Cfg::TILE_BYTES >> 4);
                const uint32_t dS = tS0 + t * 128;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    umma_ss(dS, umma_desc_join(q + off, UMMA_DESC_HI_SW128), umma_desc_join(k + off, UMMA_DESC_HI_SW128),
                            idescS, kk != 0);
                }
                ++qk_blocks;
            };
            // One step of one row tile: O_t += P_t V_j (phase 3, Eq. 3) and, when the tile has another key
            // block, S_t for block j+1 right behind it (the tensor pipe runs them in order, so S may
            // overwrite the columns P was read from).  One commit reports both to the softmax warps.
            auto issue_step = [&](int t, int j, bool has_next) -> bool {
                const int sv = j % Cfg::VSTAGES, sk = (j + 1) % Cfg::KSTAGES;
                // operand tiles first: these are normally long complete and cost only the poll
                if (!mbar_wait(&bars.v_full[sv], (j / Cfg::VSTAGES) & 1, abortp)) return false;
                if (has_next && !mbar_wait(&bars.k_full[sk], ((j + 1) / Cfg::KSTAGES) & 1, abortp)) return false;
                if (!mbar_wait(&bars.p_ready[t], j & 1, abortp)) return false;
                tc_fence_after();
                const uint32_t v = v_lo + sv * (Cfg::TILE_BYTES >> 4);
                const uint32_t dO = tO0 + t * D, aP = tS0 + t * 128;
                (void)aP;
                if (j == 0) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + (kk >> 2) * 64 + (kk & 3) * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128),
                                idescO, kk != 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + (kk >> 2) * 64 + (kk & 3) * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128),
                                idescO, 1);
                }
                ++pv_blocks;
                if (has_next) mma_S(t, j + 1);
                umma_commit(&bars.o_done[t]);
                if (t == last_t) {
                    umma_commit(&bars.v_empty[sv]);
                    if (has_next) umma_commit(&bars.k_empty[sk]);
                }
                return true;
            };
            for (int t = 0; t < work.ntiles && ok; ++t) ok = mbar_wait(&bars.q_full[t], 0, abortp);
            if (!SYM && ok) {
                ok = mbar_wait(&bars.k_full[0], 0, abortp);
                if (ok) {
                    tc_fence_after();
                    for (int t = 0; t < work.ntiles; ++t) {
                        mma_S(t, 0);
                        umma_commit(&bars.s_full[t]);
                    }
                    umma_commit(&bars.k_empty[0]);
                }
            }
            if (!SEP) {
                for (int j = 0; j < maxkv && ok; ++j)
                    for (int t = 0; t < work.ntiles && ok; ++t) {
                        const int nkv_t = t == 0 ? nkv0 : nkv1;
                        if (j < nkv_t) ok = issue_step(t, j, !SYM && j + 1 < nkv_t);
                    }
            } else {
                // Separate P: S_t(j+1) needs only that the softmax warps have taken S_t(j) out of TMEM
                // (s_free) and PV_t(j) only P_t(j) (p_ready); the two tiles' events arrive in no fixed
                // order, so the issuer polls them without blocking and issues whatever has become possible.
                int nS[2] = {1, 1}, nPV[2] = {0, 0};
                const int nkv[2] = {nkv0, nkv1};
                const uint64_t t_start = globaltimer_ns();
                uint32_t idle = 0;
                while (ok && (nPV[0] < nkv0 || nPV[1] < nkv1)) {
                    bool progressed = false;
                    for (int t = 0; t < work.ntiles && ok; ++t) {
                        const int o = t ^ 1;
                        int j = nS[t];
                        // (the operand tile is tested, not waited for: its load may itself depend on an MMA
                        // of the other tile that this very thread has yet to issue)
                        if (j < nkv[t] && mbar_test(&bars.s_free[t], (j - 1) & 1) &&
                            mbar_test(&bars.k_full[j % Cfg::KSTAGES], (j / Cfg::KSTAGES) & 1)) {
                            const int sk = j % Cfg::KSTAGES;
                            tc_fence_after();
                            mma_S(t, j);
                            umma_commit(&bars.s_full[t]);
                            ++nS[t];
                            if (o >= work.ntiles || j >= nkv[o] || nS[o] > j) umma_commit(&bars.k_empty[sk]);
                            progressed = true;
                        }
                        j = nPV[t];
                        if (j < nkv[t] && mbar_test(&bars.p_ready[t], j & 1) &&
                            mbar_test(&bars.v_full[j % Cfg::VSTAGES], (j / Cfg::VSTAGES) & 1)) {
                            const int sv = j % Cfg::VSTAGES;
                            tc_fence_after();
                            const uint32_t v = v_lo + sv * (Cfg::TILE_BYTES >> 4);
                            const uint32_t dO = tO0 + t * D, aP = tmem + Cfg::TMEM_P + t * 64;
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
                            umma_commit(&bars.o_done[t]);
                            ++nPV[t];
                            if (o >= work.ntiles || j >= nkv[o] || nPV[o] > j) umma_commit(&bars.v_empty[sv]);
                            progressed = true;
                        }
                    }
                    if (!progressed && (++idle & 255u) == 0u) {
                        if (*abortp) ok = false;
                        else if (globaltimer_ns() - t_start > 4 * PSA_WAIT_LIMIT_NS) { *abortp = 1; ok = false; }
                    }
                }
            }
            const unsigned long long block_macs = (unsigned long long)TILE * TILE * D;
            if (qk_blocks) atomicAdd(&dc->qk_macs, qk_blocks * block_macs);
            if (pv_blocks) {
                atomicAdd(&dc->pv_macs, pv_blocks * block_macs);
                atomicAdd(&dc->exps, pv_blocks * (unsigned long long)(TILE * TILE));
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue
        // TPR threads share a query row; thread `part` owns block columns [part*CPT, (part+1)*CPT).
        constexpr int CPT = 128 / TPR;                           // score columns per thread
        constexpr int NCH = CPT / 32;                            // 32-column chunks per thread
        constexpr int OPT = D / TPR;                             // output columns per thread
        const int sw = warp - CTRL_WARPS;
        const int t = sw / SOFTMAX_WARPS_PER_TILE;              // row tile of this warp
        const int part = (sw % SOFTMAX_WARPS_PER_TILE) >> 2;    // which share of the row's columns
        const int nkv = t == 0 ? nkv0 : nkv1;
        constexpr bool SEP = Cfg::SEP_P && !SYM;
        if (t < work.ntiles) {
            const int q = warp & 3;                             // TMEM lane quarter this warp may access
            const int r = q * 32 + lane;                        // row inside the tile = TMEM lane
            const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
            const uint32_t tS = tmem + Cfg::TMEM_S + t * 128 + lane_off;
            const uint32_t tO = tmem + Cfg::TMEM_O + t * D + lane_off + part * OPT;
            const uint32_t tP = tmem + Cfg::TMEM_P + t * 64 + lane_off;     // separate-P layout only
            const int It = work.tile0 + t;
            const int pair_bar = 1 + t * 4 + q;                 // named barrier of the warps sharing rows
            const int tile_bar = 9 + t;                         // named barrier of all softmax warps of the tile
            const int col_base = part * CPT;
            const size_t npad = (size_t)T * TILE;                 // S scratch is [heads, npad, npad]
            const float* srow = SYM ? Sg + ((size_t)work.bh * npad + (size_t)It * TILE + r) * npad + col_base : nullptr;
            float m_run = -INFINITY, l_run = 0.f;
            bool ok = true;
            for (int j = 0; j < nkv; ++j) {
                if (SEP) {
                    ok = mbar_wait<PSA_SOFTMAX_SLEEP_NS>(&bars.s_full[t], j & 1, abortp);    // every S_j has its own commit
                } else {
                    // block 0 waits for the first S; later blocks for the commit that follows PV_{j-1} and S_j
                    if (j == 0) { if (!SYM) ok = mbar_wait<PSA_SOFTMAX_SLEEP_NS>(&bars.s_full[t], 0, abortp); }
                    else ok = mbar_wait<PSA_SOFTMAX_SLEEP_NS>(&bars.o_done[t], (j - 1) & 1, abortp);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (TPR == 1 && !ok) break;
                // Element predicate: on the diagonal block of the masked scheme keys beyond the row's own index,
                // and on a ragged last block keys beyond the sequence, carry no weight.  `cb` = last kept column.
                const int nvalid = min(TILE, n - j * TILE);
                const bool on_diag = (scheme == PSA_MASKED) && (j == It);
                const bool diag = on_diag || nvalid < TILE;
                const int cb = min(on_diag ? r : TILE - 1, nvalid - 1);
                float mx = -INFINITY;
                // 32 raw scores of this thread's share of the row: chunk c = block columns col_base + 32c ..
                auto load32 = [&](int c, uint32_t (&v)[32]) {
                    if (!SYM) {
                        tmem_ld32(tS + col_base + 32 * c, v);
                    } else {
                        const float4* src = reinterpret_cast<const float4*>(srow + (size_t)j * TILE + 32 * c);
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const float4 f = __ldg(src + g);
                            v[4 * g] = __float_as_uint(f.x); v[4 * g + 1] = __float_as_uint(f.y);
                            v[4 * g + 2] = __float_as_uint(f.z); v[4 * g + 3] = __float_as_uint(f.w);
                        }
                    }
                };
                uint32_t sreg[NCH][32];
                if (ok) {
                    // ---- pass 1: maximum of this thread's scores
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < NCH; ++c) load32(c, sreg[c]);
                    if (!SYM) tc_wait_ld();
#pragma unroll
                    for (int c = 0; c < NCH; ++c)
                        mx = diag ? max_chunk32<true>(sreg[c], col_base + 32 * c, cb, mx)
                                  : max_chunk32<false>(sreg[c], col_base + 32 * c, r, mx);
                }
                if (TPR == 2) {
                    // The two threads of a row meet here to exchange their half-row maxima (and to leave
                    // together if either gave up a wait).
                    xch_max[j & 1][t][part][r] = mx;
                    ok = named_bar_all(ok, pair_bar, 64);
                    if (!ok) break;
                    mx = fmaxf(mx, xch_max[j & 1][t][part ^ 1][r]);
                }
                const float mx2 = mx * sl2;
                float alpha = 1.f;
                if (mx2 > m_run + RESCALE_THRESHOLD) {   // also taken on the first block (m_run = -inf)
                    alpha = ex2_mufu(m_run - mx2);
                    m_run = mx2;
                }
                // ---- pass 2: P = exp2(S*sl2 - m) as bf16, stored over this thread's own share of S, behind
                // its own reads: keys [col_base + 32c, +32) go to S columns (col_base/64)*64 + (col_base%64)/2 + 16c.
                float rowsum = 0.f;
                if (TPR == 2 && PSA_RELOAD_S) {      // the scores were only reduced so far: fetch them again
#pragma unroll
                    for (int c = 0; c < NCH; ++c) load32(c, sreg[c]);
                    if (!SYM) tc_wait_ld();
                }
                if (SEP) {
                    // S_j is in registers: the issuer may overwrite it with S_{j+1} while the exponentials run
                    tc_fence_before();
                    mbar_arrive(&bars.s_free[t]);
                    // P and O are still in use by PV_{j-1} until its commit.  A wait given up here is not
                    // acted on before the next pair barrier, so that the two threads of a row stay together.
                    if (j > 0) {
                        ok = mbar_wait(&bars.o_done[t], (j - 1) & 1, abortp);
                        ok = __all_sync(0xffffffffu, ok);
                        tc_fence_after();
                    }
                }
                if (ok) {
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        uint32_t pk[16];
                        const int kc = col_base + 32 * c;            // first key column of the chunk
                        rowsum += diag ? exp_chunk32<Cfg::POLY_OF_4, true>(sreg[c], sl2, -m_run, kc, cb, pk)
                                       : exp_chunk32<Cfg::POLY_OF_4, false>(sreg[c], sl2, -m_run, kc, r, pk);
                        tmem_st16(SEP ? tP + (kc >> 1) : tS + (kc >> 6) * 64 + ((kc & 63) >> 1), pk);
                    }
                }
                l_run = fmaf(l_run, alpha, rowsum);
                if (ok && j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rare: a row maximum grew by > 2^8
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
                mbar_arrive(&bars.p_ready[t]);
            }
            if (ok) ok = mbar_wait(&bars.o_done[t], (nkv - 1) & 1, abortp);
            if (TPR == 2) xch_sum[t][part][r] = l_run;
            if (named_bar_all(ok, tile_bar, 32 * SOFTMAX_WARPS_PER_TILE)) {
                // ---- epilogue: y = O / l (the division of Eq. 2, applied once per output row)
                tc_fence_after();
                const float inv = 1.f / (TPR == 2 ? l_run + xch_sum[t][part ^ 1][r] : l_run);
                uint8_t* stage = sQ + t * Cfg::TILE_BYTES;     // Q_t is no longer read by any MMA
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
                if (sw == t * SOFTMAX_WARPS_PER_TILE && lane == 0) {
                    for (int u = 0; u < Cfg::SUB; ++u)
                        tma_store_3d(&maps.o, stage + u * 16384, col0 + 64 * u, It * TILE, b);
                    tma_store_commit();
                    tma_store_wait_read();   // smem may be released; the writes complete on their own
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, 512);
}


// Phase 1 of the symmetric scheme (paper Sec. 4.1): one CTA per unordered tile pair {I, J}, J <= I,
// computes S_IJ = scale * X_I X_J^T once and stores it at (I, J) and, transposed, at (J, I): the
// mirror block costs stores, no MACs.  S: [heads_in_pass, n, n] fp32.
template <int D>
__global__ void __launch_bounds__(128, 2)
sym_scores_kernel(const __grid_constant__ CUtensorMap mapX, float* __restrict__ Sg, int n, int H, int bh0,
                  float scale, DeviceCounters* dc) {
    constexpr int SUB = D / 64, TILE_BYTES = 128 * D * 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + TILE_BYTES;
    __shared__ uint64_t full_bar, acc_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ float tr[4][32][33];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = row_tiles(n);
    const int np = sym_pairs(T);
    const int hl = blockIdx.x / np;                 // head inside this pass
    int I, J;
    sym_pair(blockIdx.x - hl * np, &I, &J);
    const int bh = bh0 + hl, b = bh / H, h = bh - b * H;
    const int col0 = h * D;
    const size_t npad = (size_t)T * TILE;            // the scratch is padded to whole tiles

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
            tma_load_3d(sA + u * 16384, &mapX, &full_bar, col0 + 64 * u, I * TILE, b);
            tma_load_3d(sB + u * 16384, &mapX, &full_bar, col0 + 64 * u, J * TILE, b);
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
        tc_fence_after();
        float* Sh = Sg + (size_t)hl * npad * npad;
        const int r = warp * 32 + lane;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + c0, v);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float s = __uint_as_float(v[i]) * scale;
                tr[warp][lane][i] = s;
                if (I != J)  // mirror block: element (J*128 + c0 + i, I*128 + r); lanes run along a row
                    Sh[((size_t)J * TILE + c0 + i) * npad + (size_t)I * TILE + r] = s;
            }
            __syncwarp();
#pragma unroll
            for (int rr = 0; rr < 32; ++rr)  // direct block, lanes run along a row
                Sh[((size_t)I * TILE + warp * 32 + rr) * npad + (size_t)J * TILE + c0 + lane] = tr[warp][rr][lane];
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 0) tmem_dealloc(tmem, 128);
}

constexpr size_t SYM_SCRATCH_CAP = size_t(2) << 30;  // bytes of score scratch per pass

int sym_heads_per_pass(int B, int H, int n) {
    const size_t npad = (size_t)row_tiles(n) * TILE;
    const size_t per_head = npad * npad * sizeof(float);
    size_t hp = SYM_SCRATCH_CAP / per_head;
    if (hp < 1) hp = 1;
    if (hp > (size_t)B * H) hp = (size_t)B * H;
    return (int)hp;
}

template <int D>
int launch_attention(const void* Q, const void* K, const void* V, void* out, float* S, int B, int H, int n,
                     float scale, int scheme, DeviceCounters* dc, cudaStream_t stream) {
    using Cfg = AttnCfg<D>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attn_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(sym_scores_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     2 * Cfg::TILE_BYTES + 1024);
        if (e != cudaSuccess) { set_cuda_error(e, "cudaFuncSetAttribute(attention)"); return PSA_ERR_CUDA; }
        attr_set = true;
    }
    const uint64_t cols = (uint64_t)H * D;
    AttnMaps maps;
    if (!make_tensor_map_bf16_3d(&maps.q, Q, B, n, cols, 128) || !make_tensor_map_bf16_3d(&maps.k, K, B, n, cols, 128) ||
        !make_tensor_map_bf16_3d(&maps.v, V, B, n, cols, 128) || !make_tensor_map_bf16_3d(&maps.o, out, B, n, cols, 128))
        return PSA_ERR_CUDA;
    const int P = ctas_per_head(n);
    cudaError_t e;
    if (scheme != PSA_SYMMETRIC) {
        attn_kernel<D, false><<<B * H * P, ATTN_THREADS, Cfg::SMEM, stream>>>(maps, nullptr, n, H, scheme, 0, B * H,
                                                                             lpt_group(scheme, B * H, n, D),
                                                                             scale * LOG2E, dc);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_cuda_error(e, "attn_kernel launch"); return PSA_ERR_CUDA; }
        return PSA_OK;
    }
    const int hp = sym_heads_per_pass(B, H, n);
    const int np = sym_pairs(row_tiles(n));
    for (int bh0 = 0; bh0 < B * H; bh0 += hp) {
        const int heads = min(hp, B * H - bh0);
        sym_scores_kernel<D><<<heads * np, 128, 2 * Cfg::TILE_BYTES + 1024, stream>>>(maps.q, S, n, H, bh0, scale, dc);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_cuda_error(e, "sym_scores_kernel launch"); return PSA_ERR_CUDA; }
        attn_kernel<D, true><<<heads * P, ATTN_THREADS, Cfg::SMEM, stream>>>(maps, S, n, H, PSA_SYMMETRIC, bh0, heads, 1, LOG2E, dc);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_cuda_error(e, "attn_kernel(symmetric) launch"); return PSA_ERR_CUDA; }
    }
    return PSA_OK;
}

}  // namespace

size_t bf16_symmetric_scratch_bytes(int B, int H, int n) {
    const size_t npad = (size_t)row_tiles(n) * TILE;
    return (size_t)sym_heads_per_pass(B, H, n) * npad * npad * sizeof(float);
}

int bf16_attention(const void* Q, const void* K, const void* V, void* out, float* S, size_t s_bytes, int B, int H,
                   int n, int d, float scale, int scheme, DeviceCounters* dc, cudaStream_t stream) {
    if (scheme == PSA_SYMMETRIC && (!S || s_bytes < bf16_symmetric_scratch_bytes(B, H, n))) return PSA_ERR_WORKSPACE;
#ifndef PSA_NO_PERSIST
    if (scheme != PSA_SYMMETRIC) return bf16_attention_persist(Q, K, V, out, B, H, n, d, scale, scheme, dc, stream);
#endif
    if (d == 64) return launch_attention<64>(Q, K, V, out, S, B, H, n, scale, scheme, dc, stream);
    if (d == 128) return launch_attention<128>(Q, K, V, out, S, B, H, n, scale, scheme, dc, stream);
    return PSA_ERR_UNSUPPORTED;
}

}  // namespace psa
