// Shared device helpers and internal launch declarations of the Elastic Cache library.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <nvtx3/nvToolsExt.h>

#include "ec.h"

namespace ec {

// A named range around every entry point that enqueues work, visible to profilers that listen to
// NVTX (header-only: without such a tool attached the calls return at once).
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};

constexpr int kStatusBytes = 256;   // status block at the head of an importance workspace

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Eight bf16 values held in one 16-byte vector -> eight floats.
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    f[0] = bf16lo(v.x); f[1] = bf16hi(v.x);
    f[2] = bf16lo(v.y); f[3] = bf16hi(v.y);
    f[4] = bf16lo(v.z); f[5] = bf16hi(v.z);
    f[6] = bf16lo(v.w); f[7] = bf16hi(v.w);
}

__device__ __forceinline__ uint32_t pack2(float a, float b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a (low half), .y = b
    return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    uint4 v;
    v.x = pack2(f[0], f[1]);
    v.y = pack2(f[2], f[3]);
    v.z = pack2(f[4], f[5]);
    v.w = pack2(f[6], f[7]);
    return v;
}

// Read-only streaming load (data never written by the running kernel).
__device__ __forceinline__ uint4 ldg_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- host-only argument checks (ec_api.cu); each returns an ec_status ----
int check_importance_args(const void *Q, const void *K, const float *scores, const float *lse, int N, int H, int T, int D,
                          float scale, const void *ws, size_t ws_bytes);
int check_select_compact_args(const void *K, const void *V, const float *scores, int N, int H, int T, int D, int n_keep,
                              int share, int compaction, const void *Kc, const void *Vc, int cap,
                              const int32_t *anchor_pos, const int32_t *bucket_len, const void *ws, size_t ws_bytes);
int check_cache(const ec_cache *c);

// ---- launchers implemented in the .cu files (all asynchronous on `stream`) ----
cudaError_t launch_importance(const void *Q, const void *K, float *scores, float *lse_out, const float *lse_in,
                              int N, int H, int Tq, int P, int D, float scale, int statistic, double beta, void *ws,
                              cudaStream_t stream);
size_t importance_workspace_bytes(int N, int H, int T, int D);
// passed as launch_importance's lse_in: the normaliser already lies in the workspace (see there)
static const float *const kLseInWorkspace = reinterpret_cast<const float *>(static_cast<uintptr_t>(1));
cudaError_t launch_attention(const void *Q, const void *K, const void *V, void *out, float *lse_out, int N, int H,
                             int Tq, int P, int D, float scale, void *ws, cudaStream_t stream);
cudaError_t launch_wait_selftest(void *ws, unsigned limit_us, cudaStream_t stream);

cudaError_t launch_select(const float *scores, int units, int T, int n_keep, int share, int protect_ends,
                          int32_t *anchor_pos, int32_t *bucket_len, float *mean_ws, cudaStream_t stream);
cudaError_t launch_gather(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int D,
                          int n_keep, void *Kc, void *Vc, int cap, cudaStream_t stream);

// K_all/V_all [units, P + Tq, D] <- cache rows in queue order (slot j below `base`, ring slots
// base + (ring_head + j - base) % ring after it; ring = 0 means no ring yet) followed by the new rows.
cudaError_t launch_concat(const void *Kc, const void *Vc, int units, int cap, int D, int P, int base, int ring,
                          int ring_head, const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                          cudaStream_t stream);
// The same with the cache rows' slots given as a host list: queue position j comes from slot slots[j].
cudaError_t launch_concat_listed(const void *Kc, const void *Vc, int units, int cap, int D, int P, const int *slots_host,
                                 const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                                 cudaStream_t stream);
cudaError_t launch_merge(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int D,
                         int n_keep, void *Kc, void *Vc, int cap, cudaStream_t stream);

int decode_splits(int units, int rows);
// splits > 1: `counters` (units ints) must be zero when the launch starts; the kernel leaves them zero.
// defer_from >= 0: the kernels in front on `stream` are decode steps that write no cache row below defer_from.
cudaError_t launch_decode(const void *q, const void *k_new, const void *v_new, void *Kc, void *Vc,
                          int units, int D, int cap, int len, int write_slot, int defer_from, float scale, void *out,
                          float *partials, int *counters, int splits, cudaStream_t stream);

}  // namespace ec
