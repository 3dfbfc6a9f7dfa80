/*
 * psa_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of single-layer self-attention as the paper
 * "Parallel Scheduling Self-attention Mechanism: Generalization and Optimization"
 * defines it, with the paper's two redundancy-skipping schemes.  It exists so that
 * the CUDA library can be checked against something a reader can compare with the
 * paper by eye.  It shares no code with the CUDA path and must never be called by
 * it; only the test-suite, the smoke check and the benchmark's CPU-baseline leg
 * load this file.
 *
 * What it follows (paper section / equation):
 *   phase 1  w'_ij = sum_l q_i[l] k_j[l]                       Eq. 1
 *   phase 2  w_ij  = exp(w'_ij) / sum_j exp(w'_ij)             Eq. 2 (EAC step, then division step)
 *   phase 3  y_i   = sum_j w_ij v_j                            Eq. 3 (upper limit read as n)
 *   projection q,k,v = x * {Q,K,V matrices}                    Sec. 3.1 ("typical MVM")
 *   operation counts dn^2 MAC + n^2 EAC + n^2 div + dn^2 MAC   Sec. 3.2
 *   scheme 1 (query = key = value): one member of each pair (w'_ij, w'_ji) is computed
 *            in phase 1, the other is a copy; phases 2, 3 unchanged      Sec. 4.1, 4.2
 *   scheme 2 (masked): only the n(n+1)/2 weights on and below the main diagonal take
 *            part in all three phases                                     Sec. 5.1
 *
 * Readings taken where the paper is silent (each also listed in the design notes):
 *   - `scale` multiplies the phase-1 dot product (Eq. 1 has no 1/sqrt(d); scale = 1 gives
 *     the literal equation).
 *   - exp is evaluated on w' minus the row maximum; mathematically equal to Eq. 2.
 *   - the main diagonal is kept by the mask (Sec. 5.1 lists the diagonal among the weights that
 *     remain, together with everything below it).
 *
 * Counters are incremented inside the loops that do the work, so they are a census of
 * the operations performed, not a formula.
 *
 * Parity pins: every function below is pinned by tests that do not call it to make
 * their expectation (table values printed by the paper, closed forms, brute force,
 * library routines); see tests/test_oracle_*.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { PSA_O_FULL = 0, PSA_O_SYMMETRIC = 1, PSA_O_MASKED = 2 };
enum { PSA_O_SEL_MINIMAL = 0, PSA_O_SEL_PAPER = 1 };

typedef struct {
    uint64_t mac1; /* phase-1 multiply-accumulates            */
    uint64_t eac;  /* phase-2 exponent-accumulate operations  */
    uint64_t div;  /* phase-2 divisions                       */
    uint64_t mac3; /* phase-3 multiply-accumulates            */
} psa_oracle_counts;

/* ---- Sec. 3.1: projection, a plain matrix product  out[r,c] = sum_k X[r,k] W[k,c] ---- */
int psa_oracle_project(const double *X, const double *W, long rows, long D, long N, double *out)
{
    if (!X || !W || !out || rows < 0 || D <= 0 || N <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        double *o = out + r * N;
        for (long c = 0; c < N; ++c) o[c] = 0.0;
        for (long k = 0; k < D; ++k) {
            const double x = X[r * D + k];
            const double *w = W + k * N;
            for (long c = 0; c < N; ++c) o[c] += x * w[c];
        }
    }
    return 0;
}

/* Round every element to the nearest bfloat16 value (ties to even).  Used only to
 * attribute error to the bf16 intermediate that a 16-bit pipeline stores. */
void psa_oracle_round_bf16(double *a, long count)
{
    for (long t = 0; t < count; ++t) {
        float f = (float)a[t]; /* inputs of interest are already fp32-representable or close */
        uint32_t u;
        memcpy(&u, &f, 4);
        if ((u & 0x7f800000u) != 0x7f800000u) {
            uint32_t lsb = (u >> 16) & 1u;
            u += 0x7fffu + lsb;
        }
        u &= 0xffff0000u;
        memcpy(&f, &u, 4);
        a[t] = (double)f;
    }
}

/* Sec. 4.2 selection rule for scheme 1: is w'_ij (0-based i, j) one of the weights that
 * phase 1 computes?  "minimal": the diagonal and the lower triangle.  "paper": the
 * cyclic diagonals (i - j) mod n = 0..h' (h' = (n-1)/2 for odd n, n/2-1 for even n), and
 * for even n the whole cyclic diagonal n/2, which is its own mirror image and is computed
 * in full for balance (d*n/2 redundant MACs accepted). */
static int sym_selected(long i, long j, long n, int selection)
{
    if (selection == PSA_O_SEL_MINIMAL) return j <= i;
    long off = (i - j) % n;
    if (off < 0) off += n;
    long hp = (n % 2) ? (n - 1) / 2 : n / 2 - 1;
    if (off <= hp) return 1;
    if (n % 2 == 0 && off == n / 2) return 1;
    return 0;
}

static double dot_scaled(const double *a, const double *b, long d, double scale)
{
    double s = 0.0;
    for (long l = 0; l < d; ++l) s += a[l] * b[l];
    return scale * s;
}

/*
 * One head: n query/key/value vectors of dimension d (row strides ldq/ldk/ldv doubles).
 * Three phases in the paper's order over a materialised n x n weight matrix.
 *   scheme FULL      every (i,j)
 *   scheme MASKED    j <= i only; nothing above the diagonal is read, written or counted
 *   scheme SYMMETRIC K and V are ignored: q = k = v = Q (Sec. 4.1); phase 1 computes the
 *                    selected weights and copies each remaining w'_ij from w'_ji.
 * Y       n x d (row stride ldy)                      required
 * Wout    n x n final weights w_ij, or NULL           positions never touched hold 0
 * Sout    n x n phase-1 values w'_ij, or NULL         positions never touched hold NaN
 * counts  census of this call (overwritten)
 */
int psa_oracle_slice(const double *Q, const double *K, const double *V, long n, long d, long ldq,
                     long ldk, long ldv, double scale, int scheme, int selection, double *Y,
                     long ldy, double *Wout, double *Sout, psa_oracle_counts *counts)
{
    if (!Q || !Y || n <= 0 || d <= 0) return 1;
    if (scheme == PSA_O_SYMMETRIC) {
        K = Q; V = Q; ldk = ldq; ldv = ldq;
    } else if (scheme != PSA_O_FULL && scheme != PSA_O_MASKED) {
        return 2;
    }
    if (!K || !V) return 1;
    double *S = (double *)malloc((size_t)n * (size_t)n * sizeof(double));
    if (!S) return 3;
    for (long t = 0; t < n * n; ++t) S[t] = NAN;
    uint64_t mac1 = 0, eac = 0, ndiv = 0, mac3 = 0;

    /* ---- phase 1 (Eq. 1) ---- */
    if (scheme == PSA_O_SYMMETRIC) {
#pragma omp parallel for schedule(dynamic, 8) reduction(+ : mac1)
        for (long i = 0; i < n; ++i)
            for (long j = 0; j < n; ++j)
                if (sym_selected(i, j, n, selection)) {
                    S[i * n + j] = dot_scaled(Q + i * ldq, K + j * ldk, d, scale);
                    mac1 += (uint64_t)d;
                }
        /* data reuse (Sec. 4.1): the other member of each pair is a copy, no MACs */
#pragma omp parallel for schedule(static)
        for (long i = 0; i < n; ++i)
            for (long j = 0; j < n; ++j)
                if (!sym_selected(i, j, n, selection)) S[i * n + j] = S[j * n + i];
    } else {
#pragma omp parallel for schedule(dynamic, 8) reduction(+ : mac1)
        for (long i = 0; i < n; ++i) {
            long jend = (scheme == PSA_O_MASKED) ? i + 1 : n;
            for (long j = 0; j < jend; ++j) {
                S[i * n + j] = dot_scaled(Q + i * ldq, K + j * ldk, d, scale);
                mac1 += (uint64_t)d;
            }
        }
    }
    if (Sout) memcpy(Sout, S, (size_t)n * (size_t)n * sizeof(double));

    /* ---- phase 2 (Eq. 2): step 1 exponent-accumulate, step 2 division ---- */
#pragma omp parallel for schedule(dynamic, 8) reduction(+ : eac, ndiv)
    for (long i = 0; i < n; ++i) {
        long jend = (scheme == PSA_O_MASKED) ? i + 1 : n;
        double *row = S + i * n;
        double mx = row[0];
        for (long j = 1; j < jend; ++j)
            if (row[j] > mx) mx = row[j];
        double sum = 0.0;
        for (long j = 0; j < jend; ++j) {
            row[j] = exp(row[j] - mx);
            sum += row[j];
            eac += 1;
        }
        for (long j = 0; j < jend; ++j) {
            row[j] = row[j] / sum;
            ndiv += 1;
        }
        for (long j = jend; j < n; ++j) row[j] = 0.0; /* never used below; zero for Wout */
    }
    if (Wout) memcpy(Wout, S, (size_t)n * (size_t)n * sizeof(double));

    /* ---- phase 3 (Eq. 3) ---- */
#pragma omp parallel for schedule(dynamic, 8) reduction(+ : mac3)
    for (long i = 0; i < n; ++i) {
        long jend = (scheme == PSA_O_MASKED) ? i + 1 : n;
        double *y = Y + i * ldy;
        for (long c = 0; c < d; ++c) y[c] = 0.0;
        for (long j = 0; j < jend; ++j) {
            const double w = S[i * n + j];
            const double *v = V + j * ldv;
            for (long c = 0; c < d; ++c) y[c] += w * v[c];
            mac3 += (uint64_t)d;
        }
    }
    free(S);
    if (counts) {
        counts->mac1 = mac1; counts->eac = eac; counts->div = ndiv; counts->mac3 = mac3;
    }
    return 0;
}

/*
 * The same arithmetic, in the same order, for a chosen set of query rows only (one
 * weight row in memory at a time), so that single outputs of a large problem can be
 * checked.  rows[t] are 0-based; Y is nrows x d with row stride d.  For scheme SYMMETRIC
 * a weight that phase 1 would have copied is obtained as the dot product its mirror
 * position computes (operands in that position's order).  No counters: a subset of rows
 * is not a census.
 */
int psa_oracle_rows(const double *Q, const double *K, const double *V, long n, long d, long ldq,
                    long ldk, long ldv, double scale, int scheme, int selection, const long *rows,
                    long nrows, double *Y)
{
    if (!Q || !Y || !rows || n <= 0 || d <= 0 || nrows < 0) return 1;
    if (scheme == PSA_O_SYMMETRIC) {
        K = Q; V = Q; ldk = ldq; ldv = ldq;
    } else if (scheme != PSA_O_FULL && scheme != PSA_O_MASKED) {
        return 2;
    }
    if (!K || !V) return 1;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long t = 0; t < nrows; ++t) {
        long i = rows[t];
        double *row = (i < 0 || i >= n) ? NULL : (double *)malloc((size_t)n * sizeof(double));
        if (!row) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        long jend = (scheme == PSA_O_MASKED) ? i + 1 : n;
        for (long j = 0; j < jend; ++j) {
            if (scheme == PSA_O_SYMMETRIC && !sym_selected(i, j, n, selection))
                row[j] = dot_scaled(Q + j * ldq, K + i * ldk, d, scale); /* copy of w'_ji */
            else
                row[j] = dot_scaled(Q + i * ldq, K + j * ldk, d, scale);
        }
        double mx = row[0];
        for (long j = 1; j < jend; ++j)
            if (row[j] > mx) mx = row[j];
        double sum = 0.0;
        for (long j = 0; j < jend; ++j) {
            row[j] = exp(row[j] - mx);
            sum += row[j];
        }
        for (long j = 0; j < jend; ++j) row[j] = row[j] / sum;
        double *y = Y + t * d;
        for (long c = 0; c < d; ++c) y[c] = 0.0;
        for (long j = 0; j < jend; ++j) {
            const double w = row[j];
            const double *v = V + j * ldv;
            for (long c = 0; c < d; ++c) y[c] += w * v[c];
        }
        free(row);
    }
    return bad;
}

/*
 * Tile-granular census (design reading of "computations never issued" for hardware that
 * issues whole bm x bn blocks of the weight matrix at once): a block is issued iff it
 * holds at least one weight the scheme needs in that phase.  Enumerates blocks and, inside
 * each, elements, literally.  With bm = bn = 1 this is the paper's element count.
 *   phase 1: FULL all; MASKED j <= i; SYMMETRIC the selected members (Sec. 4.2)
 *   phase 3: FULL all; MASKED j <= i; SYMMETRIC all (Sec. 4.1: phases 2, 3 unchanged)
 * issued_* count bm*bn*d MACs per issued block (blocks are clipped at n); useful_* count
 * d MACs per needed element.
 */
typedef struct {
    uint64_t issued_mac1, issued_mac3, useful_mac1, useful_mac3, tiles1, tiles3;
} psa_oracle_tile_counts;

int psa_oracle_tiles(long n, long d, int scheme, int selection, long bm, long bn,
                     psa_oracle_tile_counts *out)
{
    if (!out || n <= 0 || d <= 0 || bm <= 0 || bn <= 0) return 1;
    memset(out, 0, sizeof(*out));
    for (long I = 0; I * bm < n; ++I)
        for (long J = 0; J * bn < n; ++J) {
            long i1 = (I + 1) * bm < n ? (I + 1) * bm : n;
            long j1 = (J + 1) * bn < n ? (J + 1) * bn : n;
            uint64_t need1 = 0, need3 = 0;
            for (long i = I * bm; i < i1; ++i)
                for (long j = J * bn; j < j1; ++j) {
                    int n1, n3;
                    if (scheme == PSA_O_FULL) { n1 = 1; n3 = 1; }
                    else if (scheme == PSA_O_MASKED) { n1 = (j <= i); n3 = n1; }
                    else if (scheme == PSA_O_SYMMETRIC) { n1 = sym_selected(i, j, n, selection); n3 = 1; }
                    else return 2;
                    need1 += (uint64_t)n1; need3 += (uint64_t)n3;
                }
            uint64_t area = (uint64_t)(i1 - I * bm) * (uint64_t)(j1 - J * bn);
            out->useful_mac1 += need1 * (uint64_t)d;
            out->useful_mac3 += need3 * (uint64_t)d;
            if (need1) { out->issued_mac1 += area * (uint64_t)d; out->tiles1 += 1; }
            if (need3) { out->issued_mac3 += area * (uint64_t)d; out->tiles3 += 1; }
        }
    return 0;
}
