// Internal declarations shared by the translation units of libpsa (not part of the public interface).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/psa.h"

namespace psa {

// Device-resident counters of one call, zeroed (stream-ordered) before its first kernel.
// Kernels add to them once per block of work they actually issue.
struct DeviceCounters {
    unsigned long long proj_macs;
    unsigned long long qk_macs;
    unsigned long long pv_macs;
    unsigned long long exps;
    int status;  // PSA_OK or PSA_ERR_TIMEOUT
    unsigned int next_item;  // work-list cursor of the persistent attention kernel
    // (row, key block) events of the bf16 online softmax in which a row's running maximum was raised after the
    // row's first block, so that its partial output and row sum were rescaled (diagnostic, psa_last_rescales)
    unsigned long long rescales;
};

// ---- fp32 CUDA-core path (psa_f32.cu) ----
// out[w][r, c] = sum_k X[r, k] W[w][k, c] for w < nW.
// `residual` ([rows, N], may be null) is added to every output.
cudaError_t f32_project(const float* X, const float* const W[3], float* const out[3], int nW, int rows, int D,
                        int N, const float* residual, DeviceCounters* dc, cudaStream_t stream);
// Q, K, V, out: [B, n, H, d] fp32.  S: scratch [B*H, n, n] fp32, used by PSA_SYMMETRIC only.
cudaError_t f32_attention(const float* Q, const float* K, const float* V, float* out, float* S, int B, int H,
                          int n, int d, float scale, int scheme, DeviceCounters* dc, cudaStream_t stream);

// Small layers in one launch (projections and the three phases of a (batch, head) per CTA, all in shared memory):
// f32_fused_fits says whether a shape qualifies.  X [B, n, D], W* [D, H*d] (Wk, Wv ignored for PSA_SYMMETRIC).
bool f32_fused_fits(int n, int D, int d, int scheme);
cudaError_t f32_fused_layer(const float* X, const float* Wq, const float* Wk, const float* Wv, float* out, int B, int H,
                            int n, int D, int d, float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next,
                            cudaStream_t stream);   // (dc_next, if given, is cleared by the kernel for the next call)

// ---- bf16 tcgen05 path (psa_gemm.cu, psa_attn.cu) ----
// C[w][M, N] = A[M, K] * Bw[w][K, N] (+ residual[M, N], bf16, may be null), bf16 row-major, fp32 accumulation.
// Returns a psa_status.
int bf16_project(const void* A, const void* const Bw[3], void* const C[3], int nW, int M, int K, int N,
                 const void* residual, DeviceCounters* dc, cudaStream_t stream);
// Q, K, V, out: [B, n, H, d] bf16.  S: scratch for PSA_SYMMETRIC (bf16_symmetric_scratch_bytes:
// one 64 KB fp32 image per score block at or below the block diagonal, for the heads of one pass).
// `dc_next`, if not null, is a second counter block that the call's attention kernel clears (FULL, MASKED only).
int bf16_attention(const void* Q, const void* K, const void* V, void* out, float* S, size_t s_bytes, int B,
                   int H, int n, int d, float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next,
                   cudaStream_t stream);
size_t bf16_symmetric_scratch_bytes(int B, int H, int n);
// PSA_FULL and PSA_MASKED for 128 < d <= 256: one row tile per CTA (psa_attn_wide.cu).
int bf16_attention_wide(const void* Q, const void* K, const void* V, void* out, int B, int H, int n, int d, float scale,
                        int scheme, DeviceCounters* dc, cudaStream_t stream);
// The persistent fused kernel behind bf16_attention for PSA_FULL and PSA_MASKED (psa_attn_persist.cu).
int bf16_attention_persist(const void* Q, const void* K, const void* V, void* out, int B, int H, int n, int d,
                           float scale, int scheme, DeviceCounters* dc, DeviceCounters* dc_next, cudaStream_t stream);

// Once-per-device set-up of a kernel family.  Function attributes (the dynamic shared-memory limit) belong to the
// device that is current when they are set, and the SM count differs between devices, so both are kept per
// device ordinal.  device_setup() returns the current device's SM count (> 0), having run `configure` (which sets
// the family's attributes) the first time that device is seen; 0 on failure (error text set).  Thread-safe.
constexpr int MAX_DEVICES = 64;
struct DeviceSetup {
    bool done[MAX_DEVICES];
    int sm_count[MAX_DEVICES];
};
int device_setup(DeviceSetup* st, cudaError_t (*configure)(), const char* what);

// Self-test of the bounded-wait failure path (psa_selftest.cu): a one-CTA kernel whose barrier nobody completes.
cudaError_t launch_wait_expiry(DeviceCounters* dc, unsigned limit_us, cudaStream_t stream);

// Pipe-rate measurement (psa_pipes.cu): three kernels (ex2, fma, softmax mix), each storing per SM the cycles its
// slowest warp took for pipe_results_per_launch_per_sm() results.
cudaError_t launch_pipe_rates(unsigned long long* cycles, float* sink, int sms, cudaStream_t stream);
double pipe_results_per_launch_per_sm();

void set_cuda_error(cudaError_t e, const char* where);
void set_error_text(const char* text);

}  // namespace psa
