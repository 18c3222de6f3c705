// Attention for callers that cannot allocate device memory.
//
// Some code that wants to run the split-KV attention kernels has no allocator to ask for the
// scratch the split partials need: a plug-in running inside another engine's memory plan where
// every byte is already spoken for, a callback on a path where cudaMalloc is forbidden because
// it would synchronise the device, a process whose memory pool is owned by a different runtime.
// For them this file keeps ONE fixed scratch area inside the library image itself, a file-scope
// __device__ array, and offers an entry point that uses it.  Every GPU that loads the library
// holds the array (SPARSK_STATIC_SCRATCH_BYTES) until the process exits.
#include <cstdint>
#include <cstdio>
#include <mutex>

#include "../../include/sparsk.h"
#include <cuda_runtime.h>


static __device__ __align__(256) unsigned char g_static_scratch[SPARSK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
char *g_scratch_addr[MAX_DEVICES];  // device address of g_static_scratch, per device, once known

void say(char *err, size_t n, const char *fmt, long a = 0, long b = 0)
{
    if (err && n) snprintf(err, n, fmt, a, b);
}
}  // namespace

extern "C" int sparsk_attention_static(const sparsk_attn_args *args, void *cuda_stream, char *err, size_t err_len)
{
    if (err && err_len) err[0] = 0;
    if (!args) {
        say(err, err_len, "args is NULL");
        return SPARSK_EINVAL;
    }
    const size_t need = sparsk_attention_scratch_bytes(args->n_rows, args->n_q_heads, args->head_dim);
    if (need == 0) {
        say(err, err_len, "n_rows, n_q_heads or head_dim is invalid");
        return SPARSK_EINVAL;
    }
    if (need > (size_t)SPARSK_STATIC_SCRATCH_BYTES) {
        say(err, err_len, "this call needs %ld bytes of scratch but the built-in area holds %ld; "
                          "use fewer rows per call or sparsk_attention with your own scratch",
            (long)need, (long)SPARSK_STATIC_SCRATCH_BYTES);
        return SPARSK_ECAPACITY;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        say(err, err_len, "no usable current CUDA device");
        return SPARSK_ECUDA;
    }
    char *scratch = nullptr;
    {
        // In host code the array's name is only a handle; the address kernels can use has to be
        // asked for, once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess || !p) {
                say(err, err_len, "cudaGetSymbolAddress failed on device %ld (error %ld)", dev, (long)e);
                return SPARSK_ECUDA;
            }
            g_scratch_addr[dev] = static_cast<char *>(p);
        }
        scratch = g_scratch_addr[dev];
    }
    // Nothing in the area has to start at zero: the two counters are rewritten by every call and,
    // as long as the groups partition the rows and none exceeds max_grp_rows (the documented
    // precondition of sparsk_attention), every partial cell a call reads is one it wrote first.
    // A row outside every group would be merged from whatever an earlier call left here.
    const int rc = sparsk_attention(args, scratch, need, cuda_stream);
    if (rc == SPARSK_EINVAL) say(err, err_len, "sparsk_attention rejected the arguments");
    if (rc == SPARSK_ECUDA) say(err, err_len, "a kernel launch failed");
    return rc;
}
