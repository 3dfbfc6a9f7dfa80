// C interface of libpsa: argument checking, workspace management, the host twin of the tile
// scheduler (psa_skip_count) and dispatch to the fp32 and bf16 kernel families.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "psa_internal.h"
#include "psa_sched.h"

namespace psa {

namespace {

thread_local char g_err_text[256] = "";

struct Context {
    std::mutex mu;
    void* user_ws = nullptr;
    size_t user_bytes = 0;
    void* own_ws = nullptr;
    size_t own_bytes = 0;
    DeviceCounters* last_dc = nullptr;  // counters of the most recent call
    // The workspace starts with two counter blocks.  The bf16 FULL / MASKED path uses them in turn: the attention
    // kernel of a call clears the block of the next call, so that no clearing copy has to run ahead of the
    // call's first kernel.  `clean_ws` is the workspace whose block `next_block` is known to be clear.
    char* clean_ws = nullptr;
    int next_block = 0;
    std::vector<cudaEvent_t> prof_events;  // 3 per profiled call
    int prof_calls = 0, prof_max = 0;
    psa_counts last_useful = {0, 0, 0, 0, 0, 0};
};
// One context per device ordinal: workspace, counters and profiling state belong to the device that was current
// when they were created.  Every entry point works on the context of the calling thread's current device.
Context g_ctxs[MAX_DEVICES];
std::mutex g_setup_mu;

Context* current_ctx() {
    int dev = 0;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return nullptr; }
    if (dev < 0 || dev >= MAX_DEVICES) { set_error_text("device ordinal beyond the library's table"); return nullptr; }
    return &g_ctxs[dev];
}

constexpr size_t COUNTER_BYTES = 256;          // two counter blocks
constexpr size_t COUNTER_BLOCK_BYTES = 128;
static_assert(sizeof(DeviceCounters) <= COUNTER_BLOCK_BYTES, "counter block too small");
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, bool with_proj) {
    if (scheme != PSA_FULL && scheme != PSA_SYMMETRIC && scheme != PSA_MASKED) return PSA_ERR_SCHEME_ARGS;
    if (dtype != PSA_F32 && dtype != PSA_BF16) return PSA_ERR_UNSUPPORTED;
    if (batch <= 0 || heads <= 0 || n <= 0 || d_k <= 0 || (with_proj && d_model <= 0)) return PSA_ERR_SHAPE;
    if ((double)batch * heads * n * (double)d_k > 4.0e12 || (double)batch * n * (double)(with_proj ? d_model : 1) > 4.0e12)
        return PSA_ERR_SHAPE;
    if ((long long)batch * n > 0x7fffffffLL || (long long)heads * d_k > 0x7fffffffLL) return PSA_ERR_SHAPE;
    if (dtype == PSA_BF16) {
        // heads of up to 256 columns for the full and masked schemes; the symmetric scheme's kernels stop at 128
        if (d_k < 8 || d_k > (scheme == PSA_SYMMETRIC ? 128 : 256) || d_k % 8 != 0) return PSA_ERR_UNSUPPORTED;
        if (with_proj && (d_model % 64 != 0)) return PSA_ERR_UNSUPPORTED;
    } else {
        if (n > 1024 || d_k > 128) return PSA_ERR_UNSUPPORTED;
    }
    return PSA_OK;
}

struct WsLayout {
    size_t q, k, v, s, s_bytes, xs, wq, wk, wv, outs, total;
};

WsLayout ws_layout(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, bool with_proj,
                   bool staging) {
    const size_t es = dtype == PSA_BF16 ? 2 : 4;
    const size_t qkv = align_up((size_t)batch * n * heads * d_k * es, 256);
    WsLayout L;
    memset(&L, 0, sizeof(L));
    size_t off = COUNTER_BYTES;
    if (with_proj) {
        L.q = off; off += qkv;
        if (scheme == PSA_SYMMETRIC) { L.k = L.q; L.v = L.q; }
        else { L.k = off; off += qkv; L.v = off; off += qkv; }
    }
    if (scheme == PSA_SYMMETRIC) {
        L.s_bytes = dtype == PSA_BF16 ? bf16_symmetric_scratch_bytes(batch, heads, n)
                                      : align_up((size_t)batch * heads * n * n * sizeof(float), 256);
        L.s = off; off += L.s_bytes;
    }
    if (staging) {
        const size_t xb = align_up((size_t)batch * n * d_model * es, 256);
        const size_t wb = align_up((size_t)d_model * heads * d_k * es, 256);
        L.xs = off; off += xb;
        L.wq = off; off += wb;
        if (scheme == PSA_SYMMETRIC) { L.wk = L.wq; L.wv = L.wq; }
        else { L.wk = off; off += wb; L.wv = off; off += wb; }
        L.outs = off; off += qkv;
    }
    L.total = off;
    return L;
}

// Returns the base of a workspace of at least `bytes`, or nullptr (error text set).
char* acquire_ws(Context& cx, size_t bytes) {
    if (cx.user_ws && cx.user_bytes >= bytes) return static_cast<char*>(cx.user_ws);
    if (cx.own_ws && cx.own_bytes >= bytes) return static_cast<char*>(cx.own_ws);
    if (cx.own_ws) {
        cudaDeviceSynchronize();
        cudaFree(cx.own_ws);
        cx.own_ws = nullptr;
        cx.own_bytes = 0;
    }
    void* p = nullptr;
    const cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMalloc(workspace)"); return nullptr; }
    cx.own_ws = p;
    cx.clean_ws = nullptr;          // fresh memory: no counter block is known to be clear
    cx.own_bytes = bytes;
    return static_cast<char*>(p);
}

void useful_counts(int batch, int heads, int n, int d_model, int d_k, int scheme, bool with_proj, psa_counts* c) {
    const uint64_t bh = (uint64_t)batch * heads, N = n, d = d_k;
    const uint64_t tri = N * (N + 1) / 2;
    c->useful_qk_macs = bh * d * (scheme == PSA_FULL ? N * N : tri);
    c->useful_pv_macs = bh * d * (scheme == PSA_MASKED ? tri : N * N);
    const uint64_t nproj = scheme == PSA_SYMMETRIC ? 1 : 3;
    c->proj_macs = with_proj ? nproj * (uint64_t)batch * N * (uint64_t)d_model * (uint64_t)heads * d : 0;
}

int run_layer(Context& cx, const void* X, const void* Wq, const void* Wk, const void* Wv, const void* Q, const void* K,
              const void* V, int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, void* out,
              cudaStream_t stream, bool with_proj, char* ws, const WsLayout& L) {
    // the paths whose last kernel clears the other counter block: the fused bf16 kernel and the one-launch fp32 layer
    const bool fused_f32 = with_proj && dtype == PSA_F32 && f32_fused_fits(n, d_model, d_k, scheme);
    const bool turns = (dtype == PSA_BF16 && scheme != PSA_SYMMETRIC && d_k <= 128) || fused_f32;
    int block = 0;
    cudaError_t e = cudaSuccess;
    if (turns && cx.clean_ws == ws) {
        block = cx.next_block;
    } else {
        e = cudaMemsetAsync(ws, 0, 2 * COUNTER_BLOCK_BYTES, stream);
        if (e != cudaSuccess) { set_cuda_error(e, "cudaMemsetAsync(counters)"); return PSA_ERR_CUDA; }
    }
    cx.clean_ws = nullptr;           // until this call's kernels are known to be queued
    DeviceCounters* dc = reinterpret_cast<DeviceCounters*>(ws + block * COUNTER_BLOCK_BYTES);
    DeviceCounters* dc_next = turns ? reinterpret_cast<DeviceCounters*>(ws + (block ^ 1) * COUNTER_BLOCK_BYTES) : nullptr;
    cx.last_dc = dc;
    memset(&cx.last_useful, 0, sizeof(psa_counts));
    useful_counts(batch, heads, n, d_model, d_k, scheme, with_proj, &cx.last_useful);
    const float scale = 1.0f / sqrtf((float)d_k);
    const int nW = scheme == PSA_SYMMETRIC ? 1 : 3;
    cudaEvent_t* pev = nullptr;
    if (cx.prof_calls < cx.prof_max) pev = &cx.prof_events[3 * cx.prof_calls++];
    struct EventTail {  // records the closing event on every exit path
        cudaEvent_t* ev; cudaStream_t st;
        ~EventTail() { if (ev) cudaEventRecord(ev[2], st); }
    } tail{pev, stream};
    if (pev) cudaEventRecord(pev[0], stream);
    if (fused_f32) {
        // a small fp32 layer runs as one launch; q, k, v never leave shared memory
        if (pev) cudaEventRecord(pev[1], stream);
        e = f32_fused_layer(static_cast<const float*>(X), static_cast<const float*>(Wq), static_cast<const float*>(Wk),
                            static_cast<const float*>(Wv), static_cast<float*>(out), batch, heads, n, d_model, d_k, scale,
                            scheme, dc, dc_next, stream);
        if (e != cudaSuccess) { set_cuda_error(e, "f32_fused_layer"); return PSA_ERR_CUDA; }
        cx.clean_ws = ws;               // the other block will be clear once this call has run
        cx.next_block = block ^ 1;
        return PSA_OK;
    }
    if (with_proj) {
        void* outs[3] = {ws + L.q, ws + L.k, ws + L.v};
        const void* Ws[3] = {Wq, nW == 3 ? Wk : Wq, nW == 3 ? Wv : Wq};
        if (dtype == PSA_F32) {
            e = f32_project(static_cast<const float*>(X), reinterpret_cast<const float* const*>(Ws),
                            reinterpret_cast<float* const*>(outs), nW, batch * n, d_model, heads * d_k, nullptr, dc, stream);
            if (e != cudaSuccess) { set_cuda_error(e, "f32_project"); return PSA_ERR_CUDA; }
        } else {
            int rc = bf16_project(X, Ws, outs, nW, batch * n, d_model, heads * d_k, nullptr, dc, stream);
            if (rc != PSA_OK) return rc;
        }
        Q = ws + L.q; K = ws + L.k; V = ws + L.v;
    }
    if (pev) cudaEventRecord(pev[1], stream);
    float* S = scheme == PSA_SYMMETRIC ? reinterpret_cast<float*>(ws + L.s) : nullptr;
    if (dtype == PSA_F32) {
        e = f32_attention(static_cast<const float*>(Q), static_cast<const float*>(K), static_cast<const float*>(V),
                          static_cast<float*>(out), S, batch, heads, n, d_k, scale, scheme, dc, stream);
        if (e != cudaSuccess) { set_cuda_error(e, "f32_attention"); return PSA_ERR_CUDA; }
        return PSA_OK;
    }
    const int rc = bf16_attention(Q, K, V, out, S, L.s_bytes, batch, heads, n, d_k, scale, scheme, dc, dc_next, stream);
    if (rc == PSA_OK && turns) {        // the other block will be clear once this call has run
        cx.clean_ws = ws;
        cx.next_block = block ^ 1;
    }
    return rc;
}

int layer_entry(const void* X, const void* Wq, const void* Wk, const void* Wv, int batch, int heads, int n,
                int d_model, int d_k, int scheme, int dtype, void* out, void* stream) {
    g_err_text[0] = 0;
    int rc = check_shape(batch, heads, n, d_model, d_k, scheme, dtype, true);
    if (rc != PSA_OK) return rc;
    if (!X || !Wq || !out) return PSA_ERR_NULL;
    if (scheme == PSA_SYMMETRIC) {
        if ((Wk && Wk != Wq) || (Wv && Wv != Wq)) return PSA_ERR_SCHEME_ARGS;
    } else if (!Wk || !Wv) {
        return PSA_ERR_NULL;
    }
    if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(out)) return PSA_ERR_ALIGN;
    if (dtype == PSA_BF16 && (heads * d_k) % 64 != 0) return PSA_ERR_UNSUPPORTED;
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    const WsLayout L = ws_layout(batch, heads, n, d_model, d_k, scheme, dtype, true, false);
    char* ws = acquire_ws(cx, L.total);
    if (!ws) return PSA_ERR_WORKSPACE;
    return run_layer(cx, X, Wq, Wk, Wv, nullptr, nullptr, nullptr, batch, heads, n, d_model, d_k, scheme, dtype, out,
                     static_cast<cudaStream_t>(stream), true, ws, L);
}

}  // namespace

int device_setup(DeviceSetup* st, cudaError_t (*configure)(), const char* what) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { set_cuda_error(e, what); return 0; }
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (!st->done[dev]) {
        int sms = 0;
        e = configure();
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess || sms <= 0) { set_cuda_error(e, what); return 0; }
        st->sm_count[dev] = sms;
        st->done[dev] = true;
    }
    return st->sm_count[dev];
}

void set_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_err_text, sizeof(g_err_text), "%s: %s", where, cudaGetErrorString(e));
}
void set_error_text(const char* text) { snprintf(g_err_text, sizeof(g_err_text), "%s", text); }

}  // namespace psa

using namespace psa;

extern "C" {

int psa_attention(const void* X, const void* Wq, const void* Wk, const void* Wv, int batch, int heads, int n,
                  int d_model, int d_k, int scheme, void* out, void* stream) {
    return layer_entry(X, Wq, Wk, Wv, batch, heads, n, d_model, d_k, scheme, PSA_BF16, out, stream);
}

int psa_attention_f32(const void* X, const void* Wq, const void* Wk, const void* Wv, int batch, int heads, int n,
                      int d_model, int d_k, int scheme, void* out, void* stream) {
    return layer_entry(X, Wq, Wk, Wv, batch, heads, n, d_model, d_k, scheme, PSA_F32, out, stream);
}

int psa_attention_core(const void* Q, const void* K, const void* V, int batch, int heads, int n, int d_k,
                       int scheme, int dtype, void* out, void* stream) {
    g_err_text[0] = 0;
    int rc = check_shape(batch, heads, n, 0, d_k, scheme, dtype, false);
    if (rc != PSA_OK) return rc;
    if (!Q || !out) return PSA_ERR_NULL;
    if (scheme == PSA_SYMMETRIC) {
        if ((K && K != Q) || (V && V != Q)) return PSA_ERR_SCHEME_ARGS;
        K = Q; V = Q;
    } else if (!K || !V) {
        return PSA_ERR_NULL;
    }
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out)) return PSA_ERR_ALIGN;
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    const WsLayout L = ws_layout(batch, heads, n, 0, d_k, scheme, dtype, false, false);
    char* ws = acquire_ws(cx, L.total);
    if (!ws) return PSA_ERR_WORKSPACE;
    return run_layer(cx, nullptr, nullptr, nullptr, nullptr, Q, K, V, batch, heads, n, 0, d_k, scheme, dtype, out,
                     static_cast<cudaStream_t>(stream), false, ws, L);
}

int psa_attention_host(const void* X_host, const void* Wq_host, const void* Wk_host, const void* Wv_host,
                       int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, void* out_host,
                       void* stream_v) {
    g_err_text[0] = 0;
    int rc = check_shape(batch, heads, n, d_model, d_k, scheme, dtype, true);
    if (rc != PSA_OK) return rc;
    if (!X_host || !Wq_host || !out_host) return PSA_ERR_NULL;
    if (scheme == PSA_SYMMETRIC) {
        if ((Wk_host && Wk_host != Wq_host) || (Wv_host && Wv_host != Wq_host)) return PSA_ERR_SCHEME_ARGS;
    } else if (!Wk_host || !Wv_host) {
        return PSA_ERR_NULL;
    }
    if (dtype == PSA_BF16 && (heads * d_k) % 64 != 0) return PSA_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    const WsLayout L = ws_layout(batch, heads, n, d_model, d_k, scheme, dtype, true, true);
    char* ws = acquire_ws(cx, L.total);
    if (!ws) return PSA_ERR_WORKSPACE;
    const size_t es = dtype == PSA_BF16 ? 2 : 4;
    const size_t xb = (size_t)batch * n * d_model * es, wb = (size_t)d_model * heads * d_k * es;
    const size_t ob = (size_t)batch * n * heads * d_k * es;
    cudaError_t e = cudaMemcpyAsync(ws + L.xs, X_host, xb, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ws + L.wq, Wq_host, wb, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && scheme != PSA_SYMMETRIC) {
        e = cudaMemcpyAsync(ws + L.wk, Wk_host, wb, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ws + L.wv, Wv_host, wb, cudaMemcpyHostToDevice, stream);
    }
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMemcpyAsync(H2D)"); return PSA_ERR_CUDA; }
    rc = run_layer(cx, ws + L.xs, ws + L.wq, ws + L.wk, ws + L.wv, nullptr, nullptr, nullptr, batch, heads, n, d_model,
                   d_k, scheme, dtype, ws + L.outs, stream, true, ws, L);
    if (rc != PSA_OK) return rc;
    e = cudaMemcpyAsync(out_host, ws + L.outs, ob, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMemcpyAsync(D2H)/sync"); return PSA_ERR_CUDA; }
    return PSA_OK;
}

int psa_attention_core_host(const void* Q_host, const void* K_host, const void* V_host, int batch, int heads, int n,
                            int d_k, int scheme, int dtype, void* out_host, void* stream_v) {
    g_err_text[0] = 0;
    int rc = check_shape(batch, heads, n, 0, d_k, scheme, dtype, false);
    if (rc != PSA_OK) return rc;
    if (!Q_host || !out_host) return PSA_ERR_NULL;
    const bool sym = scheme == PSA_SYMMETRIC;
    if (sym) {
        if ((K_host && K_host != Q_host) || (V_host && V_host != Q_host)) return PSA_ERR_SCHEME_ARGS;
    } else if (!K_host || !V_host) {
        return PSA_ERR_NULL;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    const WsLayout L = ws_layout(batch, heads, n, 0, d_k, scheme, dtype, false, false);
    const size_t tb = (size_t)batch * n * heads * d_k * (dtype == PSA_BF16 ? 2 : 4), tba = align_up(tb, 256);
    const size_t q_off = align_up(L.total, 256), k_off = q_off + tba, v_off = k_off + tba;
    const size_t o_off = sym ? k_off : v_off + tba;          // the symmetric scheme stages one input tensor
    char* ws = acquire_ws(cx, o_off + tba);
    if (!ws) return PSA_ERR_WORKSPACE;
    cudaError_t e = cudaMemcpyAsync(ws + q_off, Q_host, tb, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && !sym) {
        e = cudaMemcpyAsync(ws + k_off, K_host, tb, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ws + v_off, V_host, tb, cudaMemcpyHostToDevice, stream);
    }
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMemcpyAsync(H2D)"); return PSA_ERR_CUDA; }
    const void* q = ws + q_off;
    rc = run_layer(cx, nullptr, nullptr, nullptr, nullptr, q, sym ? q : ws + k_off, sym ? q : ws + v_off, batch, heads, n,
                   0, d_k, scheme, dtype, ws + o_off, stream, false, ws, L);
    if (rc != PSA_OK) return rc;
    e = cudaMemcpyAsync(out_host, ws + o_off, tb, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMemcpyAsync(D2H)/sync"); return PSA_ERR_CUDA; }
    return PSA_OK;
}

int psa_attention_block(const void* X, const void* Wq, const void* Wk, const void* Wv, const void* Wo, int batch,
                        int heads, int n, int d_model, int d_k, int scheme, int dtype, void* out, void* stream_v) {
    return psa_attention_block_residual(X, Wq, Wk, Wv, Wo, nullptr, batch, heads, n, d_model, d_k, scheme, dtype, out,
                                        stream_v);
}

int psa_attention_block_residual(const void* X, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                                 const void* R, int batch, int heads, int n, int d_model, int d_k, int scheme,
                                 int dtype, void* out, void* stream_v) {
    g_err_text[0] = 0;
    int rc = check_shape(batch, heads, n, d_model, d_k, scheme, dtype, true);
    if (rc != PSA_OK) return rc;
    if (!X || !Wq || !Wo || !out) return PSA_ERR_NULL;
    if (scheme == PSA_SYMMETRIC) {
        if ((Wk && Wk != Wq) || (Wv && Wv != Wq)) return PSA_ERR_SCHEME_ARGS;
    } else if (!Wk || !Wv) {
        return PSA_ERR_NULL;
    }
    if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(Wo) || !aligned16(out) ||
        !aligned16(R))
        return PSA_ERR_ALIGN;
    if (R == out) return PSA_ERR_SCHEME_ARGS;      // the residual is read while the output is written
    if (dtype == PSA_BF16 && (heads * d_k) % 64 != 0) return PSA_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    const WsLayout L = ws_layout(batch, heads, n, d_model, d_k, scheme, dtype, true, false);
    const size_t y_off = align_up(L.total, 256);
    const size_t y_bytes = (size_t)batch * n * heads * d_k * (dtype == PSA_BF16 ? 2 : 4);
    char* ws = acquire_ws(cx, y_off + align_up(y_bytes, 256));
    if (!ws) return PSA_ERR_WORKSPACE;
    void* y = ws + y_off;
    rc = run_layer(cx, X, Wq, Wk, Wv, nullptr, nullptr, nullptr, batch, heads, n, d_model, d_k, scheme, dtype, y, stream,
                   true, ws, L);
    if (rc != PSA_OK) return rc;
    // z = y * Wo with the projection kernel; its MACs are added to the call's counter block
    const void* Ws[3] = {Wo, Wo, Wo};
    void* outs[3] = {out, out, out};
    if (dtype == PSA_F32) {
        cudaError_t e = f32_project(static_cast<const float*>(y), reinterpret_cast<const float* const*>(Ws),
                                    reinterpret_cast<float* const*>(outs), 1, batch * n, heads * d_k, d_model,
                                    static_cast<const float*>(R), cx.last_dc, stream);
        if (e != cudaSuccess) { set_cuda_error(e, "f32_project(Wo)"); return PSA_ERR_CUDA; }
        return PSA_OK;
    }
    return bf16_project(y, Ws, outs, 1, batch * n, heads * d_k, d_model, R, cx.last_dc, stream);
}

size_t psa_block_workspace_bytes(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype) {
    if (d_model <= 0 || check_shape(batch, heads, n, d_model, d_k, scheme, dtype, true) != PSA_OK) return 0;
    const WsLayout L = ws_layout(batch, heads, n, d_model, d_k, scheme, dtype, true, false);
    return align_up(L.total, 256) + align_up((size_t)batch * n * heads * d_k * (dtype == PSA_BF16 ? 2 : 4), 256);
}

int psa_skip_count(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype, psa_counts* c) {
    if (!c) return PSA_ERR_NULL;
    const bool with_proj = d_model > 0;
    int rc = check_shape(batch, heads, n, d_model, d_k, scheme, dtype, with_proj);
    if (rc != PSA_OK) return rc;
    memset(c, 0, sizeof(*c));
    useful_counts(batch, heads, n, d_model, d_k, scheme, with_proj, c);
    const uint64_t bh = (uint64_t)batch * heads;
    if (dtype == PSA_F32) {  // element-exact skipping
        c->qk_macs = c->useful_qk_macs;
        c->pv_macs = c->useful_pv_macs;
        c->exps = c->useful_pv_macs / (uint64_t)d_k;
        return PSA_OK;
    }
    // bf16: walk the CTA list and each CTA's block list exactly as the kernels do.  (Where the kernel hands the last
    // pairs of a launch out as single row tiles, split_point in psa_sched.h, those are the same row tiles with the
    // same block lists taken one at a time: the census does not depend on the grouping.)
    const int T = row_tiles(n);
    // (a head size below the 64, 128 or 256 columns the kernels work with is zero-padded by the loads: the padded
    // width is what the tensor core is issued)
    const uint64_t block_macs = (uint64_t)TILE * TILE * (d_k <= 64 ? 64 : (d_k <= 128 ? 128 : 256));
    uint64_t qk_blocks = 0, pv_blocks = 0, exps = 0;
    const int P = ctas_per_head(n);
    for (int cta = 0; cta < P; ++cta) {  // every head has the same list
        const CtaWork w = cta_work(cta, n, scheme == PSA_MASKED, 1, 1);
        for (int t = 0; t < w.ntiles; ++t) {
            const int I = w.tile0 + t, kv = kv_tiles(I, T, scheme);
            pv_blocks += kv;
            if (scheme != PSA_SYMMETRIC) qk_blocks += kv;
            exps += (uint64_t)kv * TILE * TILE;      // every weight of an issued block is exponentiated
        }
    }
    if (scheme == PSA_SYMMETRIC) {
        for (int t = 0; t < sym_pairs(T); ++t) {
            int I, J;
            sym_pair(t, &I, &J);
            if (J <= I) ++qk_blocks;
        }
    }
    c->qk_macs = bh * qk_blocks * block_macs;
    c->pv_macs = bh * pv_blocks * block_macs;
    c->exps = bh * exps;
    return PSA_OK;
}

int psa_last_issued(void* stream, psa_counts* c) {
    if (!c) return PSA_ERR_NULL;
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    if (!cx.last_dc) return PSA_ERR_NULL;
    DeviceCounters h;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaMemcpy(&h, cx.last_dc, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { set_cuda_error(e, "psa_last_issued"); return PSA_ERR_CUDA; }
    *c = cx.last_useful;
    c->proj_macs = h.proj_macs;
    c->qk_macs = h.qk_macs;
    c->pv_macs = h.pv_macs;
    c->exps = h.exps;
    return h.status;
}

int psa_measure_pipe_rates(psa_pipe_rates* r, void* stream_v) {
    g_err_text[0] = 0;
    if (!r) return PSA_ERR_NULL;
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || sms <= 0) { set_cuda_error(e, "psa_measure_pipe_rates"); return PSA_ERR_CUDA; }
    const size_t cyc_bytes = align_up(3 * (size_t)sms * sizeof(unsigned long long), 256);
    char* ws = acquire_ws(cx, COUNTER_BYTES + cyc_bytes + 256);
    if (!ws) return PSA_ERR_WORKSPACE;
    cx.clean_ws = nullptr;
    cx.last_dc = nullptr;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    unsigned long long* cyc = reinterpret_cast<unsigned long long*>(ws + COUNTER_BYTES);
    std::vector<unsigned long long> h(3 * (size_t)sms);
    double best[3] = {0, 0, 0};
    for (int rep = 0; rep < 3; ++rep) {       // the first repetition warms the clocks up; the best is kept
        e = cudaMemsetAsync(cyc, 0, cyc_bytes, stream);
        if (e == cudaSuccess) e = launch_pipe_rates(cyc, reinterpret_cast<float*>(ws + COUNTER_BYTES + cyc_bytes), sms, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
        if (e == cudaSuccess) e = cudaMemcpy(h.data(), cyc, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) { set_cuda_error(e, "psa_measure_pipe_rates"); return PSA_ERR_CUDA; }
        for (int m = 0; m < 3; ++m) {
            std::vector<unsigned long long> v(h.begin() + (size_t)m * sms, h.begin() + (size_t)(m + 1) * sms);
            std::sort(v.begin(), v.end());
            const double med = (double)v[v.size() / 2];
            if (med > 0 && pipe_results_per_launch_per_sm() / med > best[m]) best[m] = pipe_results_per_launch_per_sm() / med;
        }
    }
    r->ex2_per_clk_per_sm = best[0];
    r->fma_per_clk_per_sm = best[1];
    r->softmax_weights_per_clk_per_sm = best[2];
    r->sm_count = sms;
    return PSA_OK;
}

int psa_selftest_wait_expiry(unsigned limit_us, void* stream_v) {
    g_err_text[0] = 0;
    if (limit_us == 0 || limit_us > 100000u) return PSA_ERR_SHAPE;     // at most 0.1 s (1.6 s for the slowest waiter)
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    char* ws = acquire_ws(cx, COUNTER_BYTES);
    if (!ws) return PSA_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t e = cudaMemsetAsync(ws, 0, 2 * COUNTER_BLOCK_BYTES, stream);
    if (e == cudaSuccess) e = launch_wait_expiry(reinterpret_cast<DeviceCounters*>(ws), limit_us, stream);
    if (e != cudaSuccess) { set_cuda_error(e, "psa_selftest_wait_expiry"); return PSA_ERR_CUDA; }
    cx.clean_ws = nullptr;
    cx.last_dc = reinterpret_cast<DeviceCounters*>(ws);
    memset(&cx.last_useful, 0, sizeof(psa_counts));
    return PSA_OK;
}

int psa_last_rescales(void* stream, uint64_t* rescales) {
    if (!rescales) return PSA_ERR_NULL;
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    if (!cx.last_dc) return PSA_ERR_NULL;
    DeviceCounters h;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaMemcpy(&h, cx.last_dc, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { set_cuda_error(e, "psa_last_rescales"); return PSA_ERR_CUDA; }
    *rescales = h.rescales;
    return PSA_OK;
}

size_t psa_workspace_bytes(int batch, int heads, int n, int d_model, int d_k, int scheme, int dtype,
                           int with_host_staging) {
    const bool with_proj = d_model > 0;
    if (check_shape(batch, heads, n, d_model, d_k, scheme, dtype, with_proj) != PSA_OK) return 0;
    return ws_layout(batch, heads, n, d_model, d_k, scheme, dtype, with_proj, with_host_staging != 0 && with_proj).total;
}

int psa_set_workspace(void* dev_ptr, size_t bytes) {
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255u)) return PSA_ERR_ALIGN;
    cx.user_ws = dev_ptr;
    cx.user_bytes = dev_ptr ? bytes : 0;
    cx.last_dc = nullptr;
    cx.clean_ws = nullptr;
    return PSA_OK;
}

int psa_profile_begin(int max_calls) {
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    for (cudaEvent_t e : cx.prof_events) cudaEventDestroy(e);
    cx.prof_events.clear();
    cx.prof_calls = 0;
    cx.prof_max = 0;
    if (max_calls <= 0 || max_calls > 100000) return PSA_ERR_SHAPE;
    cx.prof_events.resize(3 * (size_t)max_calls);
    for (size_t i = 0; i < cx.prof_events.size(); ++i) {
        cudaError_t e = cudaEventCreate(&cx.prof_events[i]);
        if (e != cudaSuccess) {
            set_cuda_error(e, "cudaEventCreate");
            for (size_t k = 0; k < i; ++k) cudaEventDestroy(cx.prof_events[k]);
            cx.prof_events.clear();
            return PSA_ERR_CUDA;
        }
    }
    cx.prof_max = max_calls;
    return PSA_OK;
}

int psa_profile_end(float* proj_ms_sum, float* attn_ms_sum, int* calls) {
    Context* cp = current_ctx();
    if (!cp) return PSA_ERR_CUDA;
    Context& cx = *cp;
    std::lock_guard<std::mutex> lock(cx.mu);
    float p = 0.f, a = 0.f;
    int rc = PSA_OK;
    for (int c = 0; c < cx.prof_calls; ++c) {
        cudaEvent_t* ev = &cx.prof_events[3 * c];
        float t0 = 0.f, t1 = 0.f;
        cudaError_t e = cudaEventSynchronize(ev[2]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t0, ev[0], ev[1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t1, ev[1], ev[2]);
        if (e != cudaSuccess) { set_cuda_error(e, "psa_profile_end"); rc = PSA_ERR_CUDA; break; }
        p += t0; a += t1;
    }
    if (proj_ms_sum) *proj_ms_sum = p;
    if (attn_ms_sum) *attn_ms_sum = a;
    if (calls) *calls = cx.prof_calls;
    for (cudaEvent_t e : cx.prof_events) cudaEventDestroy(e);
    cx.prof_events.clear();
    cx.prof_calls = 0;
    cx.prof_max = 0;
    return rc;
}

const char* psa_status_string(int status) {
    switch (status) {
        case PSA_OK: return "ok";
        case PSA_ERR_NULL: return "a required pointer is NULL";
        case PSA_ERR_SHAPE: return "invalid size";
        case PSA_ERR_UNSUPPORTED: return "shape or number type not supported by this path";
        case PSA_ERR_ALIGN: return "pointer not sufficiently aligned";
        case PSA_ERR_SCHEME_ARGS: return "unknown scheme, or operands inconsistent with the scheme";
        case PSA_ERR_WORKSPACE: return "workspace unavailable";
        case PSA_ERR_CUDA: return "CUDA call failed";
        case PSA_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case PSA_ERR_NUMERIC: return "numeric failure";
        default: return "unknown status";
    }
}

const char* psa_last_cuda_error(void) { return g_err_text; }

}  // extern "C"
