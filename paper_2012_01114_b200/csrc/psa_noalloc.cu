// psa_attention_sym_f32_noalloc: the fp32 symmetric-scheme attention core for callers that are not
// allowed to allocate device memory.
//
// The regular entry points keep the symmetric scheme's score matrix (and the operation counters)
// in a workspace that the library obtains with cudaMalloc when the caller has registered none.
// Some callers cannot tolerate that: code running inside a memory-budgeted service where every
// byte of device memory is handed out up front, plug-ins loaded into a host application that owns
// the allocator, and real-time loops in which an allocation (which may synchronise the device)
// is not acceptable.  For them the scratch lives in a fixed array that is part of the library image.
//
// The price: every GPU that loads the library carries the array (PSA_NOALLOC_SCRATCH_BYTES) until
// the process exits, the problem size is capped, and all calls share the one array.
#include <stdio.h>

#include <mutex>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr size_t NOALLOC_COUNTER_BYTES = 256;
constexpr size_t NOALLOC_MAX_SCORES = size_t(1) << 20;  // batch * heads * n * n fp32 values (4 MiB)
constexpr size_t NOALLOC_BYTES = NOALLOC_COUNTER_BYTES + NOALLOC_MAX_SCORES * sizeof(float);
static_assert(NOALLOC_BYTES == PSA_NOALLOC_SCRATCH_BYTES, "header constant out of date");
static_assert(sizeof(DeviceCounters) <= NOALLOC_COUNTER_BYTES, "counter block too small");

// Device-resident scratch: [0, 256) operation counters, then the score matrices.  In host code this
// name is only a handle for the runtime's symbol table; the device address is looked up below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

unsigned char* g_scratch_addr[MAX_DEVICES];  // device address of the array, per device ordinal (0 = not looked up)
std::mutex g_scratch_mu;                     // guards the table above

}  // namespace
}  // namespace psa

using namespace psa;

extern "C" int psa_attention_sym_f32_noalloc(const void* X, int batch, int heads, int n, int d_k, void* out,
                                             void* stream_v) {
    set_error_text("");
    if (!X || !out) return PSA_ERR_NULL;
    if (batch <= 0 || heads <= 0 || n <= 0 || d_k <= 0) return PSA_ERR_SHAPE;
    if (n > 1024 || d_k > 128) return PSA_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(out)) & 15u) return PSA_ERR_ALIGN;
    const unsigned long long scores = (unsigned long long)batch * heads * n * (unsigned long long)n;
    if (scores > NOALLOC_MAX_SCORES) {
        char msg[200];
        snprintf(msg, sizeof(msg),
                 "psa_attention_sym_f32_noalloc: batch*heads*n*n = %llu exceeds the built-in scratch of %llu scores",
                 scores, (unsigned long long)NOALLOC_MAX_SCORES);
        set_error_text(msg);
        return PSA_ERR_WORKSPACE;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return PSA_ERR_CUDA; }
    if (dev < 0 || dev >= MAX_DEVICES) return PSA_ERR_UNSUPPORTED;
    unsigned char* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mu);
        if (!g_scratch_addr[dev]) {  // first call on this device: resolve the array's device address
            unsigned char* p = nullptr;
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
            if (e != cudaSuccess || !p) { set_cuda_error(e, "cudaGetSymbolAddress(scratch)"); return PSA_ERR_CUDA; }
            g_scratch_addr[dev] = p;
        }
        base = g_scratch_addr[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    DeviceCounters* dc = reinterpret_cast<DeviceCounters*>(base);
    // The array keeps what the previous call left.  The counters must start at zero; the score region
    // needs no clearing because phase 1 writes every element that phases 2-3 read.
    e = cudaMemsetAsync(dc, 0, sizeof(DeviceCounters), stream);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMemsetAsync(noalloc counters)"); return PSA_ERR_CUDA; }
    float* S = reinterpret_cast<float*>(base + NOALLOC_COUNTER_BYTES);
    const float* x = static_cast<const float*>(X);
    e = f32_attention(x, x, x, static_cast<float*>(out), S, batch, heads, n, d_k, 1.0f / sqrtf((float)d_k),
                      PSA_SYMMETRIC, dc, stream);
    if (e != cudaSuccess) { set_cuda_error(e, "f32_attention(noalloc)"); return PSA_ERR_CUDA; }
    return PSA_OK;
}
