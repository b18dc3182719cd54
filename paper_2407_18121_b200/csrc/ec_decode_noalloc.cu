// ec_decode_step_noalloc: the decode step for callers that cannot allocate device memory.
//
// The ordinary ec_decode_step needs a caller-provided workspace (per-unit arrival counters
// and the per-split partial results that the last CTA of a unit merges). Some hosts cannot provide one: an inference
// server that hands all of the GPU's memory to its own pool at start-up and forbids
// cudaMalloc afterwards, a plug-in whose execute callback may not allocate, or a latency-
// critical loop that cannot afford cudaMalloc's implicit device synchronisation. For them
// the scratch lives in the library itself, in a fixed device array.
#include "ec_common.cuh"

#include <mutex>

namespace {

// Built-in scratch: kNoAllocBytes per GPU that loads the library, held until the process exits.
constexpr size_t kNoAllocBytes = 2u << 20;   // 2 MiB
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices];   // device address of g_noalloc_scratch, per device ordinal

// In host code `g_noalloc_scratch` is only a handle; the address a kernel can use has to be
// asked for, once per device, with that device current.
int scratch_address(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return EC_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return EC_OK;
}

}  // namespace

extern "C" {

size_t ec_decode_noalloc_capacity(void) { return kNoAllocBytes; }

int ec_decode_step_noalloc(const void *q, const void *k_new, const void *v_new, ec_cache *c, float scale,
                           void *out, int *evicted_slot, int *slot_written, void *stream)
{
    ec::NvtxRange nvtx_range("ec_decode_step_noalloc");
    // the caller owns *c: check it before anything is computed from its fields
    int cst = ec::check_cache(c);
    if (cst != EC_OK) return cst;
    // the same size rule as the ordinary call, measured against the fixed array
    const size_t need = ec_decode_workspace(c);
    if (need == 0 || need > kNoAllocBytes) return EC_ERR_TOO_LARGE;
    void *scratch = nullptr;
    int st = scratch_address(&scratch);
    if (st != EC_OK) return st;
    // What has to start at zero (the arrival counters at the head of the array) is cleared by
    // ec_decode_step itself with a memset node before its kernel; the partial results are
    // rewritten by every launch before they are read.
    return ec_decode_step(q, k_new, v_new, c, scale, out, evicted_slot, slot_written, scratch, kNoAllocBytes, stream);
}

}  // extern "C"
