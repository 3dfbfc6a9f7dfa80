// Fused attention core of the bf16 path for the FULL and MASKED schemes: phases 1-3 of the paper
// (Eq. 1-3) per (batch, head) and pair of 128-row query tiles, never materialising the n x n weight
// matrix, as ONE persistent kernel: a CTA per SM walks the tile scheduler's work list.
//
//   phase 1  S = Q K^T            tcgen05 MMA, operands staged by TMA, accumulator in TMEM
//   phase 2  softmax              a warp reads 16 query rows of S from TMEM in the quad layout, keeps a
//                                 running row maximum m and row sum l (the division of Eq. 2 is
//                                 applied once to the output row), writes P = exp2(..) as bf16 to TMEM
//   phase 3  O += P V             tcgen05 MMA with P read from TMEM and V (row-major = MN-major) from
//                                 shared memory, accumulator O in TMEM
//
// Which (row tile, column tile) blocks exist is decided by the tile scheduler (psa_sched.h): for the
// masked scheme (paper Sec. 5) column tiles beyond the diagonal are absent from every loop in this
// file -- not loaded, not multiplied, not exponentiated -- and only the block on the diagonal carries
// an element predicate.
//
// Work items (one per pair of row tiles of one head) are listed heaviest first inside L2-sized groups
// of heads; a CTA takes its first item by its index and every further one from a device counter, so
// the list is consumed longest-processing-time-first whatever the items' run times turn out to be
// (the role of the paper's pairing of long rows with short ones, Sec. 5.2: balance).  Because the CTA
// lives on, the operand rings, the barriers' phases and the TMEM allocation carry over from item to
// item: the next item's K, V and Q tiles are requested while the current item's last blocks are still
// in the softmax, and its first scores are computed while the other row tile's output is written.
//
// CTA layout (576 threads; 608 at d = 64): warp 0 = scheduler + TMA producer, warp 1 = MMA issuer, warps 2-9 =
// softmax and epilogue of row tile 0, warps 10-17 = the same for row tile 1 (d = 64: warp 18 = MMA issuer of row
// tile 1, warp 1 that of row tile 0).  Within a tile's eight warps, warp w owns the 16 rows
// 32 (w % 4) + 16 (w / 4) .. + 15 (a warp may touch only its own quarter of the TMEM lanes) and all 128 columns of S.
// TMEM columns, d = 128: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_t (bf16, two keys per
// column) overlays the first 64 columns of S_t.  d = 64: S0 S1 | P0 P1 [256,384) | O0 O1 [384,512): P has
// its own columns, so S of the next key block is computed while the softmax of the current one runs.
#include "psa_internal.h"
#include "psa_sched.h"
#include "psa_softmax.cuh"
#include "psa_tma.h"
#include "sm100.cuh"

namespace psa {

namespace {

template <int D>
struct PCfg {
    static constexpr int SUB = D / 64;                  // 64-column sub-tiles per 128-row tile
    static constexpr int TILE_BYTES = 128 * D * 2;      // one Q, K or V tile
    static constexpr int KSTAGES = D == 128 ? 2 : 4;
    static constexpr int VSTAGES = D == 128 ? 2 : 4;
    // output staging: one [16 rows x 64 columns] bf16 buffer per softmax warp, used for each 64-column half in turn
    static constexpr int STAGE_BYTES = 16 * 64 * 2;
    static constexpr int STAGE_BUFS = 2 * SOFTMAX_WARPS_PER_TILE;
    static constexpr int SMEM = (2 + KSTAGES + VSTAGES) * TILE_BYTES + STAGE_BUFS * STAGE_BYTES + 1024;
    static constexpr bool SEP_P = D == 64;
    static constexpr int TMEM_S = 0, TMEM_P = 256, TMEM_O = SEP_P ? 384 : 256;
};

struct PMaps {
    CUtensorMap q, k, v, o;
};

struct PBars {
    uint64_t item_full[2], item_empty[2];
    uint64_t q_full[2], q_empty[2];
    uint64_t k_full[8], k_empty[8], v_full[4], v_empty[4];
    uint64_t s_full[2], s_free[2], p_ready[2], o_done[2];
};

// d = 64 has an MMA-issuing thread per row tile slot (warp 1 for slot 0, the last warp for slot 1): a block there is
// half the tensor work of d = 128 but as many instructions to issue, and one thread was measured to be the limit.
constexpr int ISSUER1_WARP = CTRL_WARPS + 2 * SOFTMAX_WARPS_PER_TILE;
template <int D> __host__ __device__ constexpr int persist_threads() { return ATTN_THREADS + (D == 64 ? 32 : 0); }
template <int D> __host__ __device__ constexpr int item_readers() { return (D == 64 ? 2 : 1) + 2 * SOFTMAX_WARPS_PER_TILE; }   // issuers + one lane per softmax warp

// KVS ("keys are the values"): K and V are one tensor (the case the paper mentions in Sec. 3.1 beside query = key =
// value).  A key tile is then loaded once and serves phase 1 as the K-major operand and phase 3 as the MN-major
// one; the shared-memory stages of the V ring extend the K ring, and a tile is released behind its PV.
template <int D, bool KVS>
__global__ void __launch_bounds__(persist_threads<D>(), 1)
attn_persist_kernel(const __grid_constant__ PMaps maps, const __grid_constant__ SchedParams sp, int H, int scheme,
                    int nitems, float sl2, DeviceCounters* dc, DeviceCounters* dc_next) {
    using Cfg = PCfg<D>;
    constexpr bool SEP = Cfg::SEP_P;
    constexpr int VST = Cfg::VSTAGES;
    constexpr int KST = KVS ? Cfg::KSTAGES + Cfg::VSTAGES : Cfg::KSTAGES;     // stages of the K ring
    // d = 128 with distinct K and V: V_j and K_{j+1} are needed by the same step of the issuing thread and released by
    // it together, so they travel as one stage (K slot s and V slot s, one full and one empty barrier: v_full / v_empty):
    // pair p of an item is (V_{p-1}, K_p), p = 0 .. blocks, the first without a V and the last without a K.  The
    // issuing thread then probes one barrier and commits one release per key block instead of two of each.
    constexpr bool PAIRED = !SEP && !KVS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                          // 2 tiles
    uint8_t* sK = sQ + 2 * Cfg::TILE_BYTES;                      // KSTAGES tiles
    uint8_t* sV = sK + Cfg::KSTAGES * Cfg::TILE_BYTES;           // VSTAGES tiles (KVS: stages KSTAGES.. of the K ring)
    uint8_t* sStage = sV + VST * Cfg::TILE_BYTES;                // STAGE_BUFS output staging tiles
    __shared__ PBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ int item_ring[2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = sp.n, T = sp.T;
    const int masked = sp.masked;
    // An item index is decoded without divisions (psa_sched.h); single-tile items at the end of the list exist at
    // d = 64 only (a lone row tile gains nothing at d = 128: the host puts split_from beyond the list there).
    auto item_work = [&](int idx) -> CtaWork { return item_work_fast(sp, idx); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(&bars.item_full[t], 1);
            mbar_init(&bars.item_empty[t], item_readers<D>());
            mbar_init(&bars.q_full[t], 1);
            mbar_init(&bars.q_empty[t], 1);
            mbar_init(&bars.s_full[t], 1);
            mbar_init(&bars.s_free[t], SOFTMAX_WARPS_PER_TILE);       // one arrival per softmax warp
            mbar_init(&bars.p_ready[t], SOFTMAX_WARPS_PER_TILE);
            mbar_init(&bars.o_done[t], 1);
        }
        for (int s = 0; s < 8; ++s) {
            // (with an issuer per slot, an operand tile collects one release from each of them)
            mbar_init(&bars.k_full[s], 1); mbar_init(&bars.k_empty[s], SEP ? 2 : 1);
        }
        for (int s = 0; s < 4; ++s) { mbar_init(&bars.v_full[s], 1); mbar_init(&bars.v_empty[s], SEP ? 2 : 1); }
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;
    // Everything above (barriers, TMEM) overlaps the end of the kernel before this one in the stream; global memory
    // is touched only from here on.
    grid_launch_dependents();
    grid_dependency_wait();
    // the counter block of the NEXT call on this workspace is cleared here, off that call's critical path
    if (threadIdx.x == 0 && blockIdx.x == 0 && dc_next) *dc_next = DeviceCounters{0, 0, 0, 0, 0, 0, 0};

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ scheduler + TMA producer
            // kc, vc: K and V tiles requested so far (ring position); qc[t]: loads of Q buffer t so far.
            uint32_t kc = 0, vc = 0, qc[2] = {0, 0};
            int idx = blockIdx.x;          // the grid never exceeds the item count
            bool ok = true;
            for (uint32_t it = 0; ok; ++it) {
                const int slot = it & 1;
                if (it >= 2) ok = mbar_wait(&bars.item_empty[slot], ((it >> 1) - 1) & 1, abortp);
                if (!ok) break;
                item_ring[slot] = idx < nitems ? idx : -1;
                mbar_arrive(&bars.item_full[slot]);
                if (idx >= nitems) break;
                const CtaWork work = item_work(idx);
                int next = -1;
                const int b = work.bh / H, h = work.bh - b * H;
                const int nkv0 = kv_tiles(work.tile0, T, scheme);
                const int nkv1 = work.ntiles > 1 ? kv_tiles(work.tile0 + 1, T, scheme) : 0;
                const int maxkv = max(nkv0, nkv1);
                if constexpr (PAIRED) {
                    for (int p = 0; p <= maxkv && ok; ++p) {           // pair p = (V_{p-1}, K_p); vc counts pairs here
                        const int s = vc % VST;
                        if (vc >= (uint32_t)VST) ok = mbar_wait(&bars.v_empty[s], ((vc / VST) - 1) & 1, abortp);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&bars.v_full[s], ((p > 0) + (p < maxkv)) * Cfg::TILE_BYTES);
                        if (p < maxkv)
                            for (int u = 0; u < Cfg::SUB; ++u)
                                tma_load_4d(sK + s * Cfg::TILE_BYTES + u * 16384, &maps.k, &bars.v_full[s], 64 * u, h,
                                            p * TILE, b);
                        if (p > 0)
                            for (int u = 0; u < Cfg::SUB; ++u)
                                tma_load_4d(sV + s * Cfg::TILE_BYTES + u * 16384, &maps.v, &bars.v_full[s], 64 * u, h,
                                            (p - 1) * TILE, b);
                        ++vc;
                        if (p == 0) {
                            for (int t = 0; t < work.ntiles && ok; ++t) {
                                if (qc[t] > 0) ok = mbar_wait(&bars.q_empty[t], (qc[t] - 1) & 1, abortp);
                                if (!ok) break;
                                mbar_arrive_expect_tx(&bars.q_full[t], Cfg::TILE_BYTES);
                                for (int u = 0; u < Cfg::SUB; ++u)
                                    tma_load_4d(sQ + t * Cfg::TILE_BYTES + u * 16384, &maps.q, &bars.q_full[t],
                                                64 * u, h, (work.tile0 + t) * TILE, b);
                                ++qc[t];
                            }
                            if (!ok) break;
                        }
                        // the next item's index is fetched behind the item's first loads and long before it is needed
                        if (p == 1) next = (int)gridDim.x + (int)atomicAdd(&dc->next_item, 1u);
                    }
                } else {
                    for (int j = 0; j < maxkv && ok; ++j) {
                        {
                            const int s = kc % KST;
                            if (kc >= (uint32_t)KST) ok = mbar_wait(&bars.k_empty[s], ((kc / KST) - 1) & 1, abortp);
                            if (!ok) break;
                            mbar_arrive_expect_tx(&bars.k_full[s], Cfg::TILE_BYTES);
                            for (int u = 0; u < Cfg::SUB; ++u)
                                tma_load_4d(sK + s * Cfg::TILE_BYTES + u * 16384, &maps.k, &bars.k_full[s], 64 * u, h,
                                            j * TILE, b);
                            ++kc;
                        }
                        if (j == 0) {
                            for (int t = 0; t < work.ntiles && ok; ++t) {
                                if (qc[t] > 0) ok = mbar_wait(&bars.q_empty[t], (qc[t] - 1) & 1, abortp);
                                if (!ok) break;
                                mbar_arrive_expect_tx(&bars.q_full[t], Cfg::TILE_BYTES);
                                for (int u = 0; u < Cfg::SUB; ++u)
                                    tma_load_4d(sQ + t * Cfg::TILE_BYTES + u * 16384, &maps.q, &bars.q_full[t],
                                                64 * u, h, (work.tile0 + t) * TILE, b);
                                ++qc[t];
                            }
                            if (!ok) break;
                        }
                        if constexpr (!KVS) {
                            const int s = vc % VST;
                            if (vc >= (uint32_t)VST) ok = mbar_wait(&bars.v_empty[s], ((vc / VST) - 1) & 1, abortp);
                            if (!ok) break;
                            mbar_arrive_expect_tx(&bars.v_full[s], Cfg::TILE_BYTES);
                            for (int u = 0; u < Cfg::SUB; ++u)
                                tma_load_4d(sV + s * Cfg::TILE_BYTES + u * 16384, &maps.v, &bars.v_full[s], 64 * u, h,
                                            j * TILE, b);
                            ++vc;
                        }
                        // the next item's index is fetched behind the item's first loads (the atomic's round trip of about
                        // a thousand cycles would otherwise delay them) and long before it is needed
                        if (j == 0) next = (int)gridDim.x + (int)atomicAdd(&dc->next_item, 1u);
                    }
                }
                idx = next;
            }
            if (*abortp) {  // let copies already issued land before shared memory is released
                for (int t = 0; t < 2; ++t)
                    if (qc[t] > 0) mbar_wait_drain(&bars.q_full[t], (qc[t] - 1) & 1);
                for (uint32_t c = kc > (uint32_t)KST ? kc - KST : 0; c < kc; ++c)
                    mbar_wait_drain(&bars.k_full[c % KST], (c / KST) & 1);
                for (uint32_t c = vc > (uint32_t)VST ? vc - VST : 0; c < vc; ++c)
                    mbar_wait_drain(&bars.v_full[c % VST], (c / VST) & 1);
            }
        }
    } else if (SEP && (warp == 1 || warp == ISSUER1_WARP)) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer of row tile slot t (d = 64)
            // The slot's blocks form a chain S_0, S_1 | PV_0, S_2 | PV_1, ...: with P in its own TMEM columns S_{j+1}
            // needs only that the softmax warps have read S_j, PV_j needs P_j.  The thread issues the links in that
            // order, sleeping on the barriers of each; the two slots' threads walk the item list independently.
            const int t = warp == 1 ? 0 : 1;
            const uint32_t idescS = umma_idesc_bf16(128, 128, UMMA_K_MAJOR, UMMA_K_MAJOR);
            const uint32_t idescO = umma_idesc_bf16(128, D, UMMA_K_MAJOR, UMMA_MN_MAJOR);
            unsigned long long qk_blocks = 0, pv_blocks = 0;
            const uint32_t q_lo = umma_desc_lo_kmajor(smem_u32(sQ + t * Cfg::TILE_BYTES));
            const uint32_t k_lo = umma_desc_lo_kmajor(smem_u32(sK));
            const uint32_t v_lo = umma_desc_lo_mnmajor(smem_u32(KVS ? sK : sV), 16384);     // KVS: V_j is the tile of K_j
            const uint32_t dS = tmem + Cfg::TMEM_S + t * 128, dO = tmem + Cfg::TMEM_O + t * D;
            const uint32_t aP = tmem + Cfg::TMEM_P + t * 64;
            uint32_t kbase = 0, vbase = 0;      // ring positions of the current item's first K and V tile
            uint32_t parts = 0;                 // earlier items in which this slot had rows
            uint32_t blk0 = 0;                  // blocks of this slot in all earlier items
            bool ok = true;
            auto mma_S = [&](uint32_t kc) {     // S = Q K^T with K at ring position kc (phase 1, Eq. 1)
                const uint32_t k = k_lo + (kc % KST) * (Cfg::TILE_BYTES >> 4);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    umma_ss(dS, umma_desc_join(q_lo + off, UMMA_DESC_HI_SW128), umma_desc_join(k + off, UMMA_DESC_HI_SW128),
                            idescS, kk != 0);
                }
                ++qk_blocks;
            };
            auto mma_PV = [&](uint32_t vc, bool first) {   // O (+)= P V with V at ring position vc (phase 3, Eq. 3)
                const uint32_t v = v_lo + (vc % (KVS ? KST : VST)) * (Cfg::TILE_BYTES >> 4);
                if (first) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, kk != 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8, umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, 1);
                }
                ++pv_blocks;
            };
            // an operand tile has two releases to collect, one per slot; a slot whose partner has no block j gives both
            auto release = [&](uint64_t* bar, bool both) {
                umma_commit(bar);
                if (both) umma_commit(bar);
            };
            for (uint32_t it = 0; ok; ++it) {
                ok = mbar_wait(&bars.item_full[it & 1], (it >> 1) & 1, abortp);
                if (!ok) break;
                const int idx = item_ring[it & 1];
                mbar_arrive(&bars.item_empty[it & 1]);
                if (idx < 0) break;
                const CtaWork work = item_work(idx);
                const int nk0 = kv_tiles(work.tile0, T, scheme);
                const int nk1 = work.ntiles > 1 ? kv_tiles(work.tile0 + 1, T, scheme) : 0;
                const int nkv = t ? nk1 : nk0, nkv_other = t ? nk0 : nk1;
                if (nkv > 0) {
                    // first scores of the item (the softmax warps must have taken the slot's previous scores out of TMEM)
                    ok = mbar_wait(&bars.q_full[t], parts & 1, abortp) &&
                         mbar_wait(&bars.k_full[kbase % KST], (kbase / KST) & 1, abortp);
                    if (ok && blk0 > 0) ok = mbar_wait(&bars.s_free[t], (blk0 - 1) & 1, abortp);
                    if (!ok) break;
                    tc_fence_after();
                    mma_S(kbase);
                    umma_commit(&bars.s_full[t]);
                    if constexpr (!KVS) release(&bars.k_empty[kbase % KST], 0 >= nkv_other);
                    if (nkv == 1) umma_commit(&bars.q_empty[t]);
                    for (int j = 0; j < nkv && ok; ++j) {
                        const uint32_t vc = vbase + j, kc = kbase + j + 1;
                        if (j + 1 < nkv) {
                            // S_{j+1} as soon as S_j has been read: it runs under the exponentials of block j
                            ok = mbar_wait(&bars.k_full[kc % KST], (kc / KST) & 1, abortp) &&
                                 mbar_wait(&bars.s_free[t], (blk0 + j) & 1, abortp);
                            if (!ok) break;
                            tc_fence_after();
                            mma_S(kc);
                            umma_commit(&bars.s_full[t]);
                            if constexpr (!KVS) release(&bars.k_empty[kc % KST], j + 1 >= nkv_other);
                            if (j + 1 == nkv - 1) umma_commit(&bars.q_empty[t]);
                        }
                        if constexpr (!KVS) ok = mbar_wait(&bars.v_full[vc % VST], (vc / VST) & 1, abortp);
                        if (ok) ok = mbar_wait(&bars.p_ready[t], (blk0 + j) & 1, abortp);
                        if (!ok) break;
                        tc_fence_after();
                        mma_PV(KVS ? kbase + j : vc, j == 0);
                        umma_commit(&bars.o_done[t]);
                        if constexpr (KVS) release(&bars.k_empty[(kbase + j) % KST], j >= nkv_other);    // the tile's last use
                        else release(&bars.v_empty[vc % VST], j >= nkv_other);
                    }
                    ++parts;
                    blk0 += nkv;
                }
                kbase += max(nk0, nk1);
                vbase += max(nk0, nk1);
            }
            const unsigned long long block_macs = (unsigned long long)TILE * TILE * D;
            if (qk_blocks) atomicAdd(&dc->qk_macs, qk_blocks * block_macs);
            if (pv_blocks) {
                atomicAdd(&dc->pv_macs, pv_blocks * block_macs);
                atomicAdd(&dc->exps, pv_blocks * (unsigned long long)(TILE * TILE));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            // (d = 128) Each row tile's blocks form a chain S_0, PV_0, S_1, PV_1, ...  The two tiles' chains are issued
            // alternately: while the softmax warps of one tile work on their scores, the tensor pipe runs the
            // other tile's MMAs, and it is this half-step offset that keeps the pipe busy.  P overlays S, so PV_j
            // and S_{j+1} of a tile go back to back under one commit, and the thread sleeps on what each link
            // needs, tile 0 then tile 1 then tile 0 ...
            const uint32_t idescS = umma_idesc_bf16(128, 128, UMMA_K_MAJOR, UMMA_K_MAJOR);
            const uint32_t idescO = umma_idesc_bf16(128, D, UMMA_K_MAJOR, UMMA_MN_MAJOR);
            unsigned long long qk_blocks = 0, pv_blocks = 0;
            const uint32_t q_lo[2] = {umma_desc_lo_kmajor(smem_u32(sQ)), umma_desc_lo_kmajor(smem_u32(sQ + Cfg::TILE_BYTES))};
            const uint32_t k_lo = umma_desc_lo_kmajor(smem_u32(sK));
            const uint32_t v_lo = umma_desc_lo_mnmajor(smem_u32(KVS ? sK : sV), 16384);     // KVS: V_j is the tile of K_j
            const uint32_t tS0 = tmem + Cfg::TMEM_S, tO0 = tmem + Cfg::TMEM_O;
            uint32_t kbase = 0, vbase = 0;      // ring positions of the current item's first K and V tile
            uint32_t parts[2] = {0, 0};         // earlier items in which tile slot t had rows
            uint32_t blk0[2] = {0, 0};          // blocks of tile slot t in all earlier items
            bool ok = true;
            // S_t = Q_t K^T with K at ring position kc (phase 1, Eq. 1): D/16 MMAs of 128x128x16.
            auto mma_S = [&](int t, uint32_t kc) {
                const uint32_t q = q_lo[t], k = k_lo + (kc % KST) * (Cfg::TILE_BYTES >> 4);
                const uint32_t dS = tS0 + t * 128;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    umma_ss(dS, umma_desc_join(q + off, UMMA_DESC_HI_SW128), umma_desc_join(k + off, UMMA_DESC_HI_SW128),
                            idescS, kk != 0);
                }
                ++qk_blocks;
            };
            // O_t (+)= P_t V with V at ring position vc (phase 3, Eq. 3): 8 MMAs of 128 x D x 16.
            auto mma_PV = [&](int t, uint32_t vc, bool first) {
                const uint32_t v = v_lo + (vc % (KVS ? KST : VST)) * (Cfg::TILE_BYTES >> 4);
                const uint32_t dO = tO0 + t * D;
                const uint32_t aP = SEP ? tmem + Cfg::TMEM_P + t * 64 : tS0 + t * 128;
                if (first) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8,
                                umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, kk != 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ts(dO, aP + kk * 8,
                                umma_desc_join(v + kk * (2048 >> 4), UMMA_DESC_HI_SW128), idescO, 1);
                }
                ++pv_blocks;
            };
            for (uint32_t it = 0; ok; ++it) {
                ok = mbar_wait(&bars.item_full[it & 1], (it >> 1) & 1, abortp);
                if (!ok) break;
                const int idx = item_ring[it & 1];
                mbar_arrive(&bars.item_empty[it & 1]);
                if (idx < 0) break;
                const CtaWork work = item_work(idx);
                const int nkv[2] = {kv_tiles(work.tile0, T, scheme),
                                    work.ntiles > 1 ? kv_tiles(work.tile0 + 1, T, scheme) : 0};
                const int maxkv = max(nkv[0], nkv[1]);
                {
                    // first scores of both tiles (PAIRED: kbase = vbase = the ring position of the item's pair 0, which
                    // holds K_0 alone; pair j + 1 holds V_j and K_{j+1})
                    if constexpr (PAIRED) ok = mbar_wait(&bars.v_full[vbase % VST], (vbase / VST) & 1, abortp);
                    else ok = mbar_wait(&bars.k_full[kbase % KST], (kbase / KST) & 1, abortp);
                    for (int t = 0; t < work.ntiles && ok; ++t) {
                        ok = mbar_wait(&bars.q_full[t], parts[t] & 1, abortp);
                        if (!ok) break;
                        tc_fence_after();
                        mma_S(t, kbase);
                        umma_commit(&bars.s_full[t]);
                        if (nkv[t] == 1) umma_commit(&bars.q_empty[t]);
                    }
                    if (!ok) break;
                    if constexpr (PAIRED) umma_commit(&bars.v_empty[vbase % VST]);
                    else if constexpr (!KVS) umma_commit(&bars.k_empty[kbase % KST]);
                    for (int j = 0; j < maxkv && ok; ++j) {
                        for (int t = 0; t < work.ntiles && ok; ++t) {
                            if (j >= nkv[t]) continue;
                            const uint32_t vc = vbase + j + (PAIRED ? 1 : 0), kc = kbase + j + 1;
                            const bool has_next = j + 1 < nkv[t];
                            // Operand tiles first.  A probe of a barrier costs this thread 150-200 cycles beside the
                            // busy softmax warps, so slot 1 does not repeat the ones slot 0 made for the same block.
                            if constexpr (!KVS)
                                if (t == 0 || j >= nkv[0]) ok = mbar_wait(&bars.v_full[vc % VST], (vc / VST) & 1, abortp);
                            if constexpr (!PAIRED)
                                if (ok && has_next && (t == 0 || j + 1 >= nkv[0]))
                                    ok = mbar_wait(&bars.k_full[kc % KST], (kc / KST) & 1, abortp);
                            if (ok) ok = mbar_wait(&bars.p_ready[t], (blk0[t] + j) & 1, abortp);
                            if (!ok) break;
                            tc_fence_after();
                            mma_PV(t, KVS ? kbase + j : vc, j == 0);
                            if (has_next) mma_S(t, kc);
                            umma_commit(&bars.o_done[t]);
                            // an operand tile is released behind its last user in this fixed order
                            const bool last_v = t == work.ntiles - 1 || j >= nkv[t + 1];
                            if (last_v) umma_commit(KVS ? &bars.k_empty[(kbase + j) % KST] : &bars.v_empty[vc % VST]);
                            if (has_next) {
                                if constexpr (!KVS && !PAIRED)
                                    if (t == work.ntiles - 1 || j + 1 >= nkv[t + 1]) umma_commit(&bars.k_empty[kc % KST]);
                                if (j + 1 == nkv[t] - 1) umma_commit(&bars.q_empty[t]);
                            }
                        }
                    }
                }
                kbase += maxkv + (PAIRED ? 1 : 0);
                vbase += maxkv + (PAIRED ? 1 : 0);
                for (int t = 0; t < work.ntiles; ++t) { ++parts[t]; blk0[t] += nkv[t]; }
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
        // Eight warps per row tile.  A warp owns 16 rows (TMEM lanes) and reads them in the quad layout (sm100.cuh): the
        // four threads of a quad share two rows, A and B = A + 8, each holding every fourth pair of their columns, so a
        // row maximum or row sum is two shuffles inside the quad and the warps never wait for one another.
        const int sw = warp - CTRL_WARPS;
        const int t = sw / SOFTMAX_WARPS_PER_TILE;              // row tile slot of this warp
        const int wq = sw % SOFTMAX_WARPS_PER_TILE;             // warp inside the slot
        const int q = warp & 3;                                 // TMEM lane quarter this warp may access
        const int row0 = q * 32 + (wq >> 2) * 16;               // first of the warp's 16 rows inside the tile
        const int rA = row0 + (lane >> 2), rB = rA + 8;         // this thread's rows
        const int cq = 2 * (lane & 3);                          // its first column inside every group of 8
        const uint32_t lane_off = static_cast<uint32_t>(row0) << 16;
        const uint32_t tS = tmem + Cfg::TMEM_S + t * 128 + lane_off;
        const uint32_t tO = tmem + Cfg::TMEM_O + t * D + lane_off;
        const uint32_t tP = SEP ? tmem + Cfg::TMEM_P + t * 64 + lane_off : tS;     // P: 64 columns, over S at d = 128
        uint8_t* stage = sStage + (t * SOFTMAX_WARPS_PER_TILE + wq) * Cfg::STAGE_BYTES;   // this warp's output staging buffer
        uint32_t my_items = 0;                                  // items this tile slot took part in
        uint32_t blk = 0;                                       // blocks this tile slot has processed, all items
        bool store_pending = false;                             // a TMA store of this warp may still be reading `stage`
        bool ok = true;
        // Takes entry `it` of the item ring: the item's index, -1 at the end of the list, -2 when the wait ran out.
        auto take_item = [&](uint32_t it) -> int {
            if (!__all_sync(0xffffffffu, mbar_wait(&bars.item_full[it & 1], (it >> 1) & 1, abortp))) return -2;
            const int idx = item_ring[it & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.item_empty[it & 1]);
            return idx;
        };
        uint32_t it = 0;
        int idx = take_item(it++);
        CtaWork work = idx >= 0 ? item_work(idx) : CtaWork{};
        while (idx >= 0) {
            if (t >= work.ntiles) {                             // no rows for this slot in this item
                idx = take_item(it++);
                if (idx >= 0) work = item_work(idx);
                continue;
            }
            const int b = work.bh / H, h = work.bh - b * H;
            const int It = work.tile0 + t;
            const int nkv = kv_tiles(It, T, scheme);
            float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;       // running maxima (log2 units) and row sums
            for (int j = 0; j < nkv; ++j, ++blk) {
                if (SEP) {
                    ok = mbar_wait(&bars.s_full[t], blk & 1, abortp);                 // every S has its own commit
                } else {
                    // block 0 waits for the item's first S; later blocks for the commit behind PV_{j-1} and S_j
                    if (j == 0) ok = mbar_wait(&bars.s_full[t], my_items & 1, abortp);
                    else ok = mbar_wait(&bars.o_done[t], (blk - 1) & 1, abortp);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // Element predicate: on the diagonal block of the masked scheme keys beyond the row's own index,
                // and on a ragged last block keys beyond the sequence, carry no weight.  cbA, cbB = last kept columns.
                const int nvalid = min(TILE, n - j * TILE);
                const bool on_diag = masked && (j == It);
                const bool diag = on_diag || nvalid < TILE;
                const int cbA = min(on_diag ? rA : TILE - 1, nvalid - 1);
                const int cbB = min(on_diag ? rB : TILE - 1, nvalid - 1);
                // ---- the rows' 2 x 64 scores of this block
                uint32_t s0[32], s1[32];
                tc_fence_after();
                tmem_ld_quad64(tS, s0);
                tmem_ld_quad64(tS + 64, s1);
                tc_wait_ld();
                if (SEP) {
                    // S is in registers: the issuer may overwrite it with the next scores while the exponentials run
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars.s_free[t]);
                }
                // ---- pass 1: row maxima of the block, completed inside the quad
                float bA = -INFINITY, bB = -INFINITY;
                if (diag) {
                    mask_quad64(s0, cq, cbA, cbB);
                    mask_quad64(s1, 64 + cq, cbA, cbB);
                }
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
                // ---- pass 2: P = exp2(S*sl2 - m) as bf16, keys 0-63 then keys 64-127
                float sumA = 0.f, sumB = 0.f;
                uint32_t pk[16];
                exp_quad64(s0, sl2, -mA, -mB, pk, sumA, sumB);
                if (SEP && blk > 0) {
                    // P and O are still in use by the PV before this one until its commit
                    ok = mbar_wait(&bars.o_done[t], (blk - 1) & 1, abortp);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                }
                tmem_st_quad32(tP, pk);
                exp_quad64(s1, sl2, -mA, -mB, pk, sumA, sumB);
                tmem_st_quad32(tP + 32, pk);
                lA = fmaf(lA, alphaA, sumA);
                lB = fmaf(lB, alphaB, sumB);
                if (j > 0 && __any_sync(0xffffffffu, alphaA != 1.f || alphaB != 1.f)) {   // rare: a row maximum grew by > 2^8
                    const int nA = __popc(__ballot_sync(0xffffffffu, (lane & 3) == 0 && alphaA != 1.f));
                    const int nB = __popc(__ballot_sync(0xffffffffu, (lane & 3) == 0 && alphaB != 1.f));
                    if (lane == 0) atomicAdd(&dc->rescales, (unsigned long long)(nA + nB));
#pragma unroll 1
                    for (int c = 0; c < D / 64; ++c) {
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
                if (lane == 0) mbar_arrive(&bars.p_ready[t]);      // (one arrival per warp: 32 on one barrier serialise)
            }
            if (!ok) break;
            // The next item is taken and decoded now, while the last PV runs, rather than after the epilogue.
            const int idx_next = take_item(it++);
            if (idx_next == -2) break;
            const CtaWork work_next = idx_next >= 0 ? item_work(idx_next) : CtaWork{};
            ok = mbar_wait(&bars.o_done[t], (blk - 1) & 1, abortp);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // ---- epilogue: y = O / l (the division of Eq. 2, applied once per output row), bf16.  The warp writes its
            // 16 rows, 64 columns at a time, into its own staging buffer and one lane hands the buffer to TMA.
            tc_fence_after();
            const float invA = 1.f / quad_sum(lA), invB = 1.f / quad_sum(lB);
#pragma unroll
            for (int u = 0; u < Cfg::SUB; ++u) {
                uint32_t v[32];
                tmem_ld_quad64(tO + 64 * u, v);
                tc_wait_ld();
                if (store_pending) {        // the store that last used the buffer must have read it
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                }
#pragma unroll
                for (int g = 0; g < 8; ++g) {       // columns 8g + cq, 8g + cq + 1 of rows A and B: 16-byte chunk g of the row
                    const uint32_t a = pack_bf16x2(__uint_as_float(v[4 * g]) * invA, __uint_as_float(v[4 * g + 1]) * invA);
                    const uint32_t bb = pack_bf16x2(__uint_as_float(v[4 * g + 2]) * invB, __uint_as_float(v[4 * g + 3]) * invB);
                    *reinterpret_cast<uint32_t*>(stage + swz128_offset(lane >> 2, g) + 2 * cq) = a;
                    *reinterpret_cast<uint32_t*>(stage + swz128_offset((lane >> 2) + 8, g) + 2 * cq) = bb;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_4d(&maps.o, stage, 64 * u, h, It * TILE + row0, b);
                    tma_store_commit();
                }
                store_pending = true;
            }
            // (the next write to O_t, PV_0 of the tile's next item, waits for P of that item, which every
            // thread of the tile signals only after these reads)
            tc_fence_before();
            ++my_items;
            idx = idx_next;
            work = work_next;
        }
        if (store_pending && lane == 0) tma_store_wait_read();   // shared memory may be released; the writes complete on their own
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// D: head size the kernel works with (64 or 128); d: the tensors' head size, d <= D, a multiple of 8 (the columns
// between d and D are zero-filled by the loads and dropped by the stores).
template <int D, bool KVS>
int launch_persist(const void* Q, const void* K, const void* V, void* out, int B, int H, int n, int d, float scale,
                   int scheme, DeviceCounters* dc, DeviceCounters* dc_next, cudaStream_t stream) {
    using Cfg = PCfg<D>;
    static DeviceSetup setup;
    const int sm_count = device_setup(&setup, [] {
        return cudaFuncSetAttribute(attn_persist_kernel<D, KVS>, cudaFuncAttributeMaxDynamicSharedMemorySize, PCfg<D>::SMEM);
    }, "attention kernel set-up");
    if (sm_count <= 0) return PSA_ERR_CUDA;
    PMaps maps;
    if (!make_tensor_map_bf16_4d(&maps.q, Q, B, n, H, d, 128) || !make_tensor_map_bf16_4d(&maps.k, K, B, n, H, d, 128) ||
        !make_tensor_map_bf16_4d(&maps.v, V, B, n, H, d, 128) || !make_tensor_map_bf16_4d(&maps.o, out, B, n, H, d, 16))
        return PSA_ERR_CUDA;
    const long long pairs = (long long)B * H * ctas_per_head(n);
    const long long split = D == 64 ? split_point(scheme, pairs, n, sm_count) : pairs;
    const long long nitems = pairs + (pairs - split);          // pairs, then the rest as single row tiles
    if (nitems > 0x7fffffffLL - sm_count) return PSA_ERR_SHAPE;
    const int grid = (int)(nitems < sm_count ? nitems : sm_count);
    const SchedParams sp = sched_params(n, scheme == PSA_MASKED, B * H, lpt_group(scheme, B * H, n, d),
                                        split == pairs ? 0x7fffffff : (int)split);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(persist_threads<D>());
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits for its predecessor itself
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, attn_persist_kernel<D, KVS>, maps, sp, H, scheme, (int)nitems,
                                             scale * LOG2E, dc, dc_next);
    if (e != cudaSuccess) { set_cuda_error(e, "attn_persist_kernel launch"); return PSA_ERR_CUDA; }
    return PSA_OK;
}

}  // namespace

// FULL and MASKED schemes.  `dc->next_item` must be zero when the kernel starts (the per-call clearing of the
// counter block does that); the kernel is launched once per call.
int bf16_attention_persist(const void* Q, const void* K, const void* V, void* out, int B, int H, int n, int d,
                           float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next, cudaStream_t stream) {
    if (scheme != PSA_FULL && scheme != PSA_MASKED) return PSA_ERR_SCHEME_ARGS;
    if (d < 8 || d > 128 || d % 8) return PSA_ERR_UNSUPPORTED;
    if (K == V) {     // one tensor for keys and values: each key tile is loaded once
        if (d <= 64) return launch_persist<64, true>(Q, K, V, out, B, H, n, d, scale, scheme, dc, dc_next, stream);
        return launch_persist<128, true>(Q, K, V, out, B, H, n, d, scale, scheme, dc, dc_next, stream);
    }
    if (d <= 64) return launch_persist<64, false>(Q, K, V, out, B, H, n, d, scale, scheme, dc, dc_next, stream);
    return launch_persist<128, false>(Q, K, V, out, B, H, n, d, scale, scheme, dc, dc_next, stream);
}

}  // namespace psa
