/*
 * psa.h -- C interface of libpsa: skip-scheduled single-layer multi-head self-attention for
 * NVIDIA B200 (sm_100a).
 *
 * The library computes, per (batch item, head), the three phases of self-attention
 *     phase 1  S_ij = scale * sum_c q_i[c] k_j[c]                 (paper Eq. 1; scale = 1/sqrt(d_k))
 *     phase 2  w_ij = exp(S_ij) / sum_j exp(S_ij)                 (paper Eq. 2)
 *     phase 3  y_i  = sum_j w_ij v_j                              (paper Eq. 3)
 * optionally preceded by the projections q,k,v = x*Wq, x*Wk, x*Wv (paper Sec. 3.1), under one of
 * three schemes that decide which weights are ever issued (never "computed, then masked"):
 *     PSA_FULL       the original definition (paper Sec. 3.2)
 *     PSA_SYMMETRIC  query = key = value: one member of each pair (S_ij, S_ji) is computed in
 *                    phase 1 and reused for the other; phases 2 and 3 are unchanged (paper Sec. 4)
 *     PSA_MASKED     decoder mask: only weights with j <= i take part, in all phases (paper Sec. 5)
 *
 * General conventions
 *   - Unless an entry point says "host", every data pointer is a DEVICE pointer owned by the
 *     caller.  The library neither frees nor keeps it after the call returns, except the workspace
 *     registered with psa_set_workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls enqueue
 *     work on it and return without waiting; argument errors are reported immediately and launch
 *     nothing.  Conditions only the device can see (a bounded wait that expired) are recorded in a
 *     device status word and reported by psa_last_issued.
 *   - All tensors are dense, row-major, 16-byte aligned:
 *         X    [batch, n, d_model]
 *         W*   [d_model, heads*d_k]      head h owns columns h*d_k .. (h+1)*d_k-1
 *         Q,K,V[batch, n, heads, d_k]
 *         out  [batch, n, heads*d_k]
 *   - Every function returns a psa_status (0 = PSA_OK) unless stated otherwise.
 *   - Calls that share a workspace must be ordered on one stream; the library is not re-entrant
 *     across streams.
 */
#ifndef PSA_H_
#define PSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { PSA_FULL = 0, PSA_SYMMETRIC = 1, PSA_MASKED = 2 } psa_scheme;
typedef enum { PSA_F32 = 0, PSA_BF16 = 1 } psa_dtype;

typedef enum {
    PSA_OK = 0,
    PSA_ERR_NULL = 1,        /* a required pointer is NULL                                     */
    PSA_ERR_SHAPE = 2,       /* a size is <= 0 or overflows                                    */
    PSA_ERR_UNSUPPORTED = 3, /* shape outside what the kernels cover (see each entry point)     */
    PSA_ERR_ALIGN = 4,       /* a pointer is not 16-byte aligned                               */
    PSA_ERR_SCHEME_ARGS = 5, /* unknown scheme, or PSA_SYMMETRIC given distinct k/v operands   */
    PSA_ERR_WORKSPACE = 6,   /* registered workspace too small and growing it failed           */
    PSA_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed (psa_last_cuda_error)        */
    PSA_ERR_TIMEOUT = 8,     /* a bounded device-side wait expired; results are invalid        */
    PSA_ERR_NUMERIC = 9      /* reserved                                                       */
} psa_status;

/*
 * Multiply-accumulate census of one call (summed over batch and heads).
 *   proj_macs       projection MACs (paper Sec. 3.1; not part of the paper's own count)
 *   qk_macs         phase-1 MACs issued      pv_macs   phase-3 MACs issued
 *   exps            phase-2 exponentials evaluated
 *   useful_*        the paper's element-level counts for the scheme (Sec. 3.2, 4.2, 5.2):
 *                   FULL d*n^2 each; MASKED d*n(n+1)/2 each; SYMMETRIC d*n(n+1)/2 and d*n^2
 * The bf16 path issues whole 128x128 blocks of the weight matrix, so issued >= useful there (a
 * block on the diagonal, or a ragged last block, is issued in full); the fp32 path skips element by element, issued = useful.
 */
typedef struct {
    uint64_t proj_macs, qk_macs, pv_macs, exps, useful_qk_macs, useful_pv_macs;
} psa_counts;

/*
 * Projections + attention, bf16 in / bf16 out, fp32 accumulation (paper Sec. 3.1 then Eq. 1-3).
 *   X, Wq, Wk, Wv, out   device, bf16, layouts above.
 *   PSA_SYMMETRIC: q = k = v = X*Wq (paper Sec. 4.1); Wk and Wv must be NULL or equal to Wq.
 * Supported: d_k any multiple of 8 up to 256 (PSA_SYMMETRIC: up to 128).  The kernels work on heads of 64, 128 or
 * 256 columns; a shorter head is zero-padded by the tile loads, and the census counts the padded width as issued; any n >= 1 (a last block of
 * fewer than 128 vectors is zero-filled and its keys carry no weight); d_model and heads*d_k multiples of 64.
 * Needs a workspace of psa_workspace_bytes(...) (grown on demand, see psa_set_workspace).
 */
int psa_attention(const void* X, const void* Wq, const void* Wk, const void* Wv, int batch, int heads, int n,
                  int d_model, int d_k, int scheme, void* out, void* stream);

/* Same computation in fp32 storage and fp32 arithmetic on CUDA cores, element-exact skipping
 * (issued = useful).  Supported: n <= 1024, d_k <= 128 (any d_model). */
int psa_attention_f32(const void* X, const void* Wq, const void* Wk, const void* Wv, int batch, int heads, int n,
                      int d_model, int d_k, int scheme, void* out, void* stream);

/*
 * Attention core only (paper Eq. 1-3 with q, k, v given; Sec. 3.1 last paragraph).
 *   dtype PSA_BF16 or PSA_F32 selects the path and the storage type of Q, K, V, out.
 *   PSA_SYMMETRIC: K and V must be NULL or equal to Q.
 *   PSA_FULL / PSA_MASKED with K == V (one tensor for keys and values, paper Sec. 3.1): each key tile is loaded
 *   once and serves both phases.
 * Shape limits as for psa_attention / psa_attention_f32 (heads*d_k need not be a multiple of 64 here).
 */
int psa_attention_core(const void* Q, const void* K, const void* V, int batch, int heads, int n, int d_k,
                       int scheme, int dtype, void* out, void* stream);

/*
 * psa_attention / psa_attention_f32 with HOST buffers (pageable or pinned): copies X and the
 * projection matrices to the device, runs the layer, copies `out` back and waits for `stream`.
 * dtype selects bf16 or fp32 storage.  The staging buffers are part of the workspace.
 */
int psa_attention_host(const void* X_host, const void* Wq_host, const void* Wk_host, const void* Wv_host,
                       int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, void* out_host,
                       void* stream);

/*
 * psa_attention_core with HOST buffers (paper Eq. 1-3 with q, k, v given): copies Q, K, V (one tensor for
 * PSA_SYMMETRIC, where K_host and V_host are NULL or equal to Q_host) to staging buffers in the workspace,
 * runs the core, copies `out` back to out_host and waits for `stream`.  Layouts, shape limits and errors as for
 * psa_attention_core; pinned host memory makes the copies asynchronous up to the final wait.
 */
int psa_attention_core_host(const void* Q_host, const void* K_host, const void* V_host, int batch, int heads, int n,
                            int d_k, int scheme, int dtype, void* out_host, void* stream);

/*
 * Attention block: the layer above followed by the output projection over the concatenated heads,
 *     z[b, i, :] = sum_h y^(h)[b, i, :] * Wo[h*d_k : (h+1)*d_k, :],
 * y^(h) being the output of paper Eq. 3 for head h.  The paper's three phases end at y (Sec. 3.2) and it
 * leaves the rest of the model to future work (Sec. 7); the multi-head remark of Sec. 3.1 implies that
 * the heads' outputs are combined afterwards, and this is the usual way: one more product of the kind
 * Sec. 3.1 calls a typical matrix-vector multiplication, run by the projection kernel.
 *   X, Wq, Wk, Wv   as for psa_attention / psa_attention_f32 (dtype selects bf16 or fp32 storage).
 *   Wo              device, [heads*d_k, d_model] row-major, same type; never NULL.
 *   out             device, [batch, n, d_model] row-major, same type (caller-owned).
 * y is kept in the workspace in the storage type (bf16 on the bf16 path) between the two steps; the
 * workspace is psa_block_workspace_bytes(...).  No residual connection and no bias are added.
 * After this call psa_last_issued reports proj_macs = input projections + batch*n*heads*d_k*d_model
 * (the output projection); psa_skip_count describes the layer part only.
 * Shape limits and errors as for psa_attention / psa_attention_f32; argument errors launch nothing.
 */
int psa_attention_block(const void* X, const void* Wq, const void* Wk, const void* Wv, const void* Wo, int batch,
                        int heads, int n, int d_model, int d_k, int scheme, int dtype, void* out, void* stream);
/*
 * The attention block with a residual input (the skip connection a transformer block wraps around its attention
 * sub-layer; the paper leaves the complete model to future work, Sec. 7):
 *     z[b, i, :] = R[b, i, :] + sum_h y^(h)[b, i, :] * Wo[h*d_k : (h+1)*d_k, :].
 *   R   device, [batch, n, d_model] row-major, same type as the other tensors, caller-owned, read only; usually X
 *       itself; NULL gives psa_attention_block.  R must not be `out` (PSA_ERR_SCHEME_ARGS).
 * The sum is formed in fp32 in the epilogue of the output projection, before the rounding to the storage type.
 * Everything else as for psa_attention_block.
 */
int psa_attention_block_residual(const void* X, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                                 const void* R, int batch, int heads, int n, int d_model, int d_k, int scheme,
                                 int dtype, void* out, void* stream);
size_t psa_block_workspace_bytes(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype);

/*
 * Analytic census: what the tile scheduler will issue for this shape and scheme (paper Sec. 3.2,
 * 4.2, 5.2 for the useful_* fields).  Host only, launches nothing.  d_model = 0 means "core only"
 * (proj_macs = 0).
 */
int psa_skip_count(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, psa_counts* counts);

/*
 * Measured census: waits for `stream`, then returns the counters the kernels of the last call
 * accumulated on the device (one increment per block of work actually issued) and that call's
 * device status (PSA_OK or PSA_ERR_TIMEOUT).
 */
int psa_last_issued(void* stream, psa_counts* counts);

/*
 * Diagnostic of the bf16 path's online softmax (paper Eq. 2 evaluated block by block along the keys):
 * waits for `stream`, then stores in *rescales how often, during the last call, a query row's running
 * maximum was raised after the row's first key block -- each such event multiplies the row's partial
 * output and partial row sum by exp(old maximum - new maximum).  The kernels raise the maximum only
 * when it has grown by more than 2^8, so on inputs whose scores stay within a few units of each other
 * the count is zero; it is nonzero when later keys carry much larger scores than earlier ones.
 * The fp32 path finds each row's maximum before its first exponential and always reports zero.
 */
int psa_last_rescales(void* stream, uint64_t* rescales);

/* Bytes of scratch memory a call with these arguments needs (projected q, k, v; the symmetric
 * scheme's score matrix; counters).  with_host_staging != 0 adds psa_attention_host's buffers. */
size_t psa_workspace_bytes(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype,
                           int with_host_staging);

/*
 * Registers caller-owned device memory (256-byte aligned) as the workspace; it must stay valid
 * until replaced or until psa_set_workspace(NULL, 0).  Without a registered workspace, or when it
 * is too small, the library keeps a private one and grows it with cudaMalloc (synchronously, on
 * the first call that needs more).
 */
int psa_set_workspace(void* dev_ptr, size_t bytes);

/*
 * Per-kernel timing for benchmarks.  psa_profile_begin(max_calls) makes each of the next max_calls
 * calls of psa_attention / psa_attention_f32 / psa_attention_core / psa_attention_host record CUDA
 * events on the caller's stream before the projection kernel, between projection and attention,
 * and after attention.  psa_profile_end waits for those events, returns the summed durations in
 * milliseconds and the number of calls recorded, and releases the events.  Not thread-safe against
 * concurrent attention calls.
 */
int psa_profile_begin(int max_calls);
int psa_profile_end(float* proj_ms_sum, float* attn_ms_sum, int* calls);

/*
 * Allocation-free variant of the fp32 symmetric-scheme attention core.  (The paper has no
 * counterpart: this is a packaging of psa_attention_core(X, NULL, NULL, ..., PSA_SYMMETRIC, PSA_F32)
 * for one kind of caller, not another algorithm.)
 *
 * Who it is for: callers that must not allocate device memory at call time -- a service whose device
 * memory is budgeted and handed out once at start-up, a plug-in inside a host program that owns the
 * allocator, a latency-critical loop where cudaMalloc (which may synchronise the whole device) is
 * unacceptable.  The other entry points fall back on cudaMalloc for their workspace when none is
 * registered; this one never calls cudaMalloc, cudaFree or any allocating routine.
 *
 * How: the scratch the symmetric scheme needs (the score matrix S of every (batch, head), written once
 * per unordered pair and mirrored, plus the operation counters) lives in a fixed array inside the
 * library image, PSA_NOALLOC_SCRATCH_BYTES long.  Every GPU that loads the library holds that array
 * until the process exits.
 *
 *   X     device, fp32, [batch, n, heads, d_k]: query = key = value        (caller-owned, read only)
 *   out   device, fp32, [batch, n, heads*d_k]                              (caller-owned)
 *   Limits: n <= 1024, d_k <= 128, and batch*heads*n*n <= PSA_NOALLOC_MAX_SCORES; a larger problem
 *   returns PSA_ERR_WORKSPACE (psa_last_cuda_error() gives the sizes) and launches nothing.
 *
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call before starting any stream capture.  All calls share the one array, which keeps
 * the previous call's contents: the call clears the counters it needs at zero and overwrites every
 * score it later reads, but two calls whose kernels overlap on the GPU (different streams without an
 * ordering between them) race on it -- order them.  psa_last_issued does not report on this entry.
 */
#define PSA_NOALLOC_MAX_SCORES (1u << 20)
#define PSA_NOALLOC_SCRATCH_BYTES (256u + 4u * PSA_NOALLOC_MAX_SCORES)
int psa_attention_sym_f32_noalloc(const void* X, int batch, int heads, int n, int d_k, void* out, void* stream);

/*
 * Measured rates of the SM pipes that phase 2 (paper Eq. 2) runs on, for the benchmark's second ceiling
 * (the paper has no counterpart; it counts one exponent-accumulate per weight, Sec. 3.2).  Runs three short
 * kernels on every SM (16 warps each, 8 independent instructions in flight per thread) and reports
 * results per SM clock per SM, median over the SMs, best of three repetitions:
 *   ex2_per_clk_per_sm               ex2.approx.ftz.f32 alone (the special-function unit)
 *   fma_per_clk_per_sm               fma.rn.f32 alone
 *   softmax_weights_per_clk_per_sm   the per-weight mix of the softmax's exponential pass:
 *                                    fma (scale and shift), ex2, add (row sum), half a bf16x2 pack
 * Synchronises `stream`; uses (and may grow) the workspace; psa_last_issued has nothing to report afterwards.
 */
typedef struct {
    double ex2_per_clk_per_sm, fma_per_clk_per_sm, softmax_weights_per_clk_per_sm;
    int sm_count;
} psa_pipe_rates;
int psa_measure_pipe_rates(psa_pipe_rates* rates, void* stream);

/*
 * Self-test of the failure path every kernel of the library shares (no counterpart in the paper).  All device-
 * side waits are bounded; one that runs out raises a flag, the CTA's other waiters leave at their next poll,
 * every role reaches the common teardown (tensor memory is freed) and PSA_ERR_TIMEOUT is written to the
 * device status word.  A correct run never takes that path, so this call enqueues a one-CTA kernel built on
 * the same skeleton whose barrier nobody completes, with a wait limit of `limit_us` microseconds
 * (1 .. 100000).  It returns PSA_OK once the kernel is queued; the following psa_last_issued(stream, &c)
 * must then return PSA_ERR_TIMEOUT with all counters zero, and later calls on the same context work as usual.
 * Nothing traps or spins without a bound.
 */
int psa_selftest_wait_expiry(unsigned limit_us, void* stream);

/* Text for a psa_status; never NULL. */
const char* psa_status_string(int status);

/* Text of the last CUDA error seen by the calling thread's most recent failing call ("" if none). */
const char* psa_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PSA_H_ */
