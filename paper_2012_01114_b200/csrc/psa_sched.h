// Tile scheduler of the bf16 path: which 128x128 blocks of the weight matrix exist for a scheme,
// and which CTA owns them.  Pure integer functions, compiled for both host and device so that the
// analytic census (psa_skip_count) walks exactly the list the kernels walk.
//
// A block that the scheme makes redundant is absent from the list: it is never loaded, never
// multiplied and never exponentiated (paper Sec. 4.1 for the symmetric scheme, Sec. 5.1 for the
// masked one), as opposed to being computed and masked afterwards.
#pragma once
#include <stdint.h>

#include "../../include/psa.h"

#if defined(__CUDACC__)
#define PSA_HD __host__ __device__ __forceinline__
#else
#define PSA_HD inline
#endif

namespace psa {

constexpr int TILE = 128;          // rows and columns of one block of the weight matrix
constexpr int TILES_PER_CTA = 2;   // a CTA owns two consecutive row tiles of one (batch, head)

// Division of a 32-bit unsigned number by a divisor fixed for a whole launch, as a multiply-high and two shifts
// (the kernels decode a work-item index several thousand times per CTA; the hardware has no integer divide, and
// the compiler's general sequence costs a single thread several hundred cycles per item).  For d >= 2:
//     l = ceil(log2 d),  m = floor(2^32 (2^l - d) / d) + 1,  n / d = (t + ((n - t) >> 1)) >> (l - 1),  t = hi32(m n)
// exact for every 32-bit n (the round-up method with a 33-bit multiplier, its top bit folded into the second shift).
struct FastDiv {
    uint32_t d, m, s;      // divisor, multiplier, l - 1   (d = 1: m = 0, s = 0 and the quotient is n itself)
};
PSA_HD FastDiv fastdiv_make(uint32_t d) {
    FastDiv f;
    f.d = d; f.m = 0; f.s = 0;
    if (d <= 1) return f;
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    f.m = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
    f.s = l - 1;
    return f;
}
PSA_HD uint32_t fastdiv_hi32(uint32_t a, uint32_t b) {
#if defined(__CUDA_ARCH__)
    return __umulhi(a, b);
#else
    return (uint32_t)(((uint64_t)a * b) >> 32);
#endif
}
PSA_HD uint32_t fastdiv(uint32_t n, const FastDiv& f) {
    if (f.d <= 1) return n;
    const uint32_t t = fastdiv_hi32(f.m, n);
    return (t + ((n - t) >> 1)) >> f.s;
}

struct CtaWork {
    int bh;        // batch * heads + head
    int tile0;     // first row tile owned
    int ntiles;    // 1 or 2 row tiles owned
};

PSA_HD int row_tiles(int n) { return (n + TILE - 1) / TILE; }   // the last tile may be ragged
PSA_HD int ctas_per_head(int n) { return (row_tiles(n) + TILES_PER_CTA - 1) / TILES_PER_CTA; }

// CTA index -> work, for a launch over `nbh` (batch, head) units taken in groups of `group` heads.
// Inside a group the order is: every head's heaviest pair of row tiles first, then every head's next
// heaviest, ... so that the hardware's in-order CTA dispatch amounts to longest-processing-time-first
// scheduling over the group (the role of the paper's pairing of long rows with short ones, Sec. 5.2:
// balance).  Groups follow one another, which keeps the K and V that concurrently running CTAs read
// to one group's worth (L2 reuse).  group = 1 is plain head-major order.
PSA_HD CtaWork cta_work(int cta, int n, int scheme_masked, int nbh, int group) {
    const int P = ctas_per_head(n);
    const int full_groups = nbh / group;
    int g = cta / (group * P);
    if (g > full_groups) g = full_groups;
    const int off = cta - g * group * P;
    const int size = g < full_groups ? group : nbh - full_groups * group;   // heads in this group
    const int r = off / size;
    CtaWork w;
    w.bh = g * group + (off - r * size);
    const int p = scheme_masked ? (P - 1 - r) : r;
    w.tile0 = p * TILES_PER_CTA;
    const int left = row_tiles(n) - w.tile0;
    w.ntiles = left < TILES_PER_CTA ? left : TILES_PER_CTA;
    return w;
}
// The same list with a tail of single row tiles: items with an index at or beyond `split_from` are the two tiles of
// pair split_from + (item - split_from) / 2, one item each (see split_point; every pair must have two tiles).
PSA_HD CtaWork cta_work_split(int item, int n, int scheme_masked, int nbh, int group, int split_from) {
    if (item < split_from) return cta_work(item, n, scheme_masked, nbh, group);
    CtaWork w = cta_work(split_from + ((item - split_from) >> 1), n, scheme_masked, nbh, group);
    w.tile0 += (item - split_from) & 1;
    w.ntiles = 1;
    return w;
}
// The same decoding with every division replaced by FastDiv: the launch's constants are prepared once on the host.
struct SchedParams {
    int n, masked, nbh, group, P, T, full_groups, tail, split_from;
    FastDiv by_group_items;   // / (group * P)
    FastDiv by_group;         // / group
    FastDiv by_tail;          // / tail   (heads in the last, partial group; 0 if none)
};
PSA_HD SchedParams sched_params(int n, int scheme_masked, int nbh, int group, int split_from) {
    SchedParams sp;
    sp.n = n; sp.masked = scheme_masked; sp.nbh = nbh; sp.group = group; sp.split_from = split_from;
    sp.P = ctas_per_head(n); sp.T = row_tiles(n);
    sp.full_groups = nbh / group;
    sp.tail = nbh - sp.full_groups * group;
    sp.by_group_items = fastdiv_make((uint32_t)group * (uint32_t)sp.P);
    sp.by_group = fastdiv_make((uint32_t)group);
    sp.by_tail = fastdiv_make((uint32_t)(sp.tail > 0 ? sp.tail : 1));
    return sp;
}
PSA_HD CtaWork cta_work_fast(const SchedParams& sp, int cta) {
    int g = (int)fastdiv((uint32_t)cta, sp.by_group_items);
    if (g > sp.full_groups) g = sp.full_groups;
    const int off = cta - g * sp.group * sp.P;
    const bool full = g < sp.full_groups;
    const int size = full ? sp.group : sp.tail;
    const int r = (int)fastdiv((uint32_t)off, full ? sp.by_group : sp.by_tail);
    CtaWork w;
    w.bh = g * sp.group + (off - r * size);
    const int p = sp.masked ? (sp.P - 1 - r) : r;
    w.tile0 = p * TILES_PER_CTA;
    const int left = sp.T - w.tile0;
    w.ntiles = left < TILES_PER_CTA ? left : TILES_PER_CTA;
    return w;
}
// ... and with the tail of single row tiles (cta_work_split)
PSA_HD CtaWork item_work_fast(const SchedParams& sp, int item) {
    if (item < sp.split_from) return cta_work_fast(sp, item);
    CtaWork w = cta_work_fast(sp, sp.split_from + ((item - sp.split_from) >> 1));
    w.tile0 += (item - sp.split_from) & 1;
    w.ntiles = 1;
    return w;
}

// Work items of a launch over `pairs` pairs of row tiles on `sms` persistent CTAs: the first split_point() items are
// pairs, the rest single row tiles.  Where all CTAs do the same work (FULL) and the last round of pairs would occupy
// at most half of the CTAs, those pairs are handed out as single tiles instead, so that twice as many CTAs share
// that round (a lone row tile takes less time than a pair at d_k = 64 and the same time at d_k = 128).
PSA_HD long long split_point(int scheme, long long pairs, int n, int sms) {
    if (scheme != PSA_FULL || (row_tiles(n) & 1) || sms <= 0) return pairs;
    const long long r = pairs % sms;
    if (r == 0 || 2 * r > sms) return pairs;
    return pairs - r;
}
// Heads per group: as many as keep the group's K and V (bf16) within a fraction of L2; the schemes whose
// CTAs all do the same work gain nothing from reordering and keep head-major order.
#ifndef PSA_LPT_MB
#define PSA_LPT_MB 64
#endif
#ifndef PSA_LPT_ALL_FACTOR
#define PSA_LPT_ALL_FACTOR 4
#endif
PSA_HD int lpt_group(int scheme, int nbh, int n, int d) {
    if (scheme != PSA_MASKED) return 1;
    const long long per_head = (long long)n * d * 2 * 2;
    // (all heads in one group while their K and V together stay within about twice L2: CTAs that work on one head
    // at the same time stream its key blocks in step, so the footprint at any moment is far below the total, and
    // one longest-first list over everything balances best; measured on n = 8192 with 32 heads)
    if (per_head * nbh <= ((long long)PSA_LPT_ALL_FACTOR * PSA_LPT_MB) << 20) return nbh;
    long long g = ((long long)PSA_LPT_MB << 20) / per_head;
    if (g < 1) g = 1;
    if (g > nbh) g = nbh;
    return (int)g;
}

// Number of key/value tiles row tile I visits in phases 1-3 of the fused kernel (FULL, MASKED) or
// in phases 2-3 (SYMMETRIC): column tiles 0 .. kv_tiles-1.
PSA_HD int kv_tiles(int I, int T, int scheme) { return scheme == PSA_MASKED ? I + 1 : T; }

// Phase 1 of the symmetric scheme: one block per unordered pair {I, J}; block t of a head,
// t in [0, T(T+1)/2), is (I, J) with J <= I, enumerated row by row.
PSA_HD void sym_pair(int t, int* I, int* J) {
    int i = 0;
    while ((i + 1) * (i + 2) / 2 <= t) ++i;
    *I = i;
    *J = t - i * (i + 1) / 2;
}
PSA_HD int sym_pairs(int T) { return T * (T + 1) / 2; }

}  // namespace psa
